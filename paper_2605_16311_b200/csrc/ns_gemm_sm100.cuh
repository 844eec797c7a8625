// Newton-Schulz products on the 5th-generation tensor cores (sm_100a):
//   grouped, persistent, warp-specialised bf16 GEMM  D[M x N] = sum_k a(i,k) b(j,k)
//   - operands staged by TMA (3-D tiled tensor maps, 128-byte swizzle) into a multi-stage
//     shared-memory ring guarded by mbarriers,
//   - tcgen05.mma (kind::f16, bf16 x bf16 -> fp32) issued by one thread, accumulators in TMEM,
//     double-buffered so the epilogue of tile t overlaps the main loop of tile t+1,
//   - epilogue warps read TMEM with tcgen05.ld and apply the fused Newton-Schulz epilogues
//     (Gram scaling, 1.5 Y + Q Y, sign + pack, weight update).
// One launch covers every (parameter, worker) product of one Newton-Schulz half-iteration: each
// CTA (or CTA pair) walks a host-built list of tiles (problem, tile_m, tile_n).
//
// Two shapes of the same kernel (template parameter CTAS):
//   CTAS = 1: one CTA per 128 x BN tile, tcgen05.mma.cta_group::1.
//   CTAS = 2: a cluster of two CTAs on neighbouring SMs shares a 256 x BN tile (cta_group::2): CTA r
//             stages rows [128 r, 128 r + 128) of A and columns [BN/2 r, BN/2 (r+1)) of B, the MMA is
//             issued by CTA 0 alone and reads both shared memories, and each CTA keeps and drains the
//             accumulator of its own 128 rows.  Per flop this halves the operand bytes every SM has
//             to pull from L2, which is what bounds the 128 x 128 shape.  Barriers that cross the
//             pair: the "stage full" barrier lives in CTA 0 and counts the TMA bytes of both CTAs;
//             "stage empty" and "accumulator full" are signalled in both CTAs by a multicast
//             tcgen05.commit; "accumulator empty" lives in CTA 0 and collects the epilogue warps of both.
//             No TMA load uses cluster multicast.
//
// Operand layouts in shared memory (one 64-wide K block per stage):
//   K-major  (contiguous along K):  rows of 128 bytes, TMA box {64 k, R rows}, 8-row swizzle atoms
//            of 1024 bytes; descriptor SBO = 1024, a 16-element K step advances the start by 32 bytes.
//   MN-major (contiguous along M/N): per 64 rows of M/N one 8 KB chunk = 64 k-rows of 128 bytes,
//            TMA box {64 mn, 64 k}; descriptor LBO = 8192 (next chunk), SBO = 1024 (next 8 k-rows),
//            a 16-element K step advances the start by 2048 bytes.
// Epilogue traffic also goes through TMA: the Y_k tile that enters as 1.5*C is prefetched into a ring
// of 64-column chunk buffers (128-byte swizzle; hi half and lo half, or two fp32 halves for the first
// iteration's momentum) by a dedicated thread, eight math warps (two per TMEM lane quarter) overwrite the
// chunk in place, and the same dedicated thread sends it off with TMA stores; the math warps touch global
// memory directly only for payload words and the final weight update.  The math warps never wait for each
// other: per chunk they wait on the buffer's "C landed / buffer free" mbarrier and arrive on its "results
// written" mbarrier.
// Gram products are symmetric: only tiles on or above the diagonal are scheduled and an off-diagonal tile is
// also stored transposed.  A problem may carry up to three operand pairs ("segments") that are accumulated
// into the same tile along K: split-precision products (hi hi + lo hi + hi lo) of the spectral scale.
// Warps (416 threads): 0 = TMA of the A operand, 1 and 12 = MMA issue (alternate K blocks), 2..9 = epilogue math,
// 10 = epilogue TMA, 11 = TMA of the B operand.  The single threads of warps 0, 1, 11 and 12 sit on the critical path of
// every K block (512 tensor-core cycles on a CTA pair): the MMA threads form their descriptors by adding a step to
// precomputed words and take turns, so that one prepares while the other's instructions run, and the copies of a stage
// are split over two threads.
// Every wait is bounded: after the launch's wait limit (two seconds by default) a waiting thread records
// STATUS_TIMEOUT in the status word, raises a CTA-wide abort flag and the CTA drains and exits (TMEM is freed).
#pragma once

#include <type_traits>

#include <cuda.h>

#include "common.cuh"

namespace signmuon {

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;
constexpr int EPI_WARPS = 8;                 // EPI_WARPS / 4 warps per TMEM lane quarter, each NCOL of a chunk's 64 columns
constexpr int EPI_NCOL = 256 / EPI_WARPS;    // columns of a chunk one math thread owns (32 or 16)
static_assert(EPI_WARPS == 8 || EPI_WARPS == 16, "8 or 16 epilogue math warps");
constexpr int GEMM_THREADS = 32 * (7 + EPI_WARPS);   // warp 0: TMA of the A operand, warp 1: MMA issue (even K blocks), then the
                                                     // epilogue math warps, the epilogue TMA warp (C loads, result stores), the
                                                     // TMA warp of the B operand, last warp: MMA issue (odd K blocks)
constexpr uint64_t DEFAULT_WAIT_LIMIT_NS = 2000000000ull;   // two seconds unless the caller sets another limit

struct GemmLaunchArgs {
  const CUtensorMap* tmaps;
  const GemmProblem* problems;
  const TileEntry* tiles;
  const uint32_t* cta_tile_start;   // [gridDim.x + 1]
  const ParamDev* params;
  uint32_t* status;
  float lr;
  uint64_t wait_limit_ns;           // after this long a waiting thread gives up and the CTA aborts
  PeerList peers;                   // other GPUs' payload buffers that also receive the packed words (n = 0: none)
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait. Returns false when the CTA is aborting (this or another thread ran out of time).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint64_t limit_ns) {
  uint32_t spins = 0;
  uint64_t t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_ns) {
        *abort_flag = 1;
        atomicExch(status, (uint32_t)STATUS_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// Same load inside a CTA pair: the completion bytes may be credited to a barrier of the peer CTA.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// Barrier over every thread of every CTA of the cluster (all threads of a warp must arrive together).
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// CTA-pair form: the MMA spans both CTAs; the commit arrives on the barrier at the same offset in both.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, int x, int y, int z, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Loads 32 consecutive fp32 columns of this thread's TMEM lane and waits for them.  Load and wait sit in
// one asm statement so that no use of the destination registers can be scheduled before the wait.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_ld_cols(uint32_t taddr, float (&v)[32]) { tc_ld32(taddr, v); }
__device__ __forceinline__ void tc_ld_cols(uint32_t taddr, float (&v)[16]) { tc_ld16(taddr, v); }

// Shared-memory matrix descriptor (128-byte swizzle).  Bits: [0,14) start >> 4, [16,30) LBO >> 4,
// [32,46) SBO >> 4, [46,48) = 1 (descriptor version), [61,64) = 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// High word of such a descriptor with a stride byte offset of 1024 (every operand tile here), and the MMA issued from
// the two descriptor words of each operand (A and B share the high word).  kind::f16 takes bf16 x bf16 -> fp32 with
// K = 16 per instruction, kind::f8f6f4 E4M3 x E4M3 -> fp32 with K = 32 (32 bytes either way).
constexpr uint32_t SMEM_DESC_HI_SBO1024 = ((1024u >> 4) & 0x3fffu) | (1u << 14) | (2u << 29);
template <bool PAIR, bool FP8>
__device__ __forceinline__ void tc_mma_words(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                             uint32_t accumulate) {
  if (PAIR && FP8) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
  } else if (PAIR) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
  } else if (FP8) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
  }
}

// Instruction descriptor: D fp32 (bits [4,6) = 1), A/B format in bits [7,10) and [10,13) (kind::f16: 1 = bf16;
// kind::f8f6f4: 0 = E4M3), bit 15 / 16: A / B contiguous along M / N, bits [17,23) N >> 3, bits [24,29) M >> 4
// (M = 128 for one CTA, 256 for a CTA pair).
__device__ __forceinline__ uint32_t instr_desc(int m, int n, int a_mn, int b_mn, int fp8 = 0) {
  uint32_t d = 0;
  d |= 1u << 4;
  if (!fp8) {
    d |= 1u << 7;
    d |= 1u << 10;
  }
  d |= (uint32_t)(a_mn & 1) << 15;
  d |= (uint32_t)(b_mn & 1) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(m >> 4) << 24;
  return d;
}

// ------------------------------------------------------------------------------------------ kernel
constexpr uint32_t EPI_HALF_BYTES = 128 * 128;        // 128 rows x 128 bytes (one swizzled half)
constexpr uint32_t EPI_BUF_BYTES = 2 * EPI_HALF_BYTES;

// Issues the TMA loads of the C chunk (64 columns from column `col0`) of a tile into an epilogue buffer.
// (c_mode, the two tensor maps and the batch slot are the problem's, read once per tile by the caller)
__device__ __forceinline__ void epi_issue_c_load(int c_mode, const CUtensorMap* map0, const CUtensorMap* map1, int batch_c,
                                                 int row0, int col0, uint32_t buf, uint32_t bar) {
  if (c_mode == C_F32) {
    mbar_expect_tx(bar, EPI_BUF_BYTES);
    tma_load_3d(buf, map0, col0, row0, batch_c, bar);
    tma_load_3d(buf + EPI_HALF_BYTES, map0, col0 + 32, row0, batch_c, bar);
  } else if (c_mode == C_HILO) {
    mbar_expect_tx(bar, EPI_BUF_BYTES);
    tma_load_3d(buf, map0, col0, row0, batch_c, bar);
    tma_load_3d(buf + EPI_HALF_BYTES, map1, col0, row0, batch_c, bar);
  } else {
    mbar_expect_tx(bar, EPI_HALF_BYTES);
    tma_load_3d(buf, map0, col0, row0, batch_c, bar);
  }
}

template <int BN, int STAGES, int EPI_BUFS, int CTAS, int KIND>
__global__ void __launch_bounds__(GEMM_THREADS, 1) ns_gemm_tc_kernel(const __grid_constant__ GemmLaunchArgs args) {
  constexpr int B_ROWS = BN / CTAS;                            // rows of the B operand this CTA stages
  constexpr int TILE_M = GEMM_BM * CTAS;                       // rows of the output tile of the CTA (pair)
  constexpr uint32_t A_BYTES = GEMM_BM * GEMM_BK * 2;          // 16 KB
  constexpr uint32_t B_BYTES = B_ROWS * GEMM_BK * 2;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN;                       // two accumulator buffers
  // KIND 0: a launch of Gram products only (no C operand, bf16 output: ring buffers of one half);
  // KIND 1: a launch of apply products (C operand, hi/lo output, pack or weight update).
  // (a Gram chunk buffer holds the bf16 chunk and, in its second half, the transposed copy for the mirror tile)
  constexpr uint32_t BUF_BYTES = EPI_BUF_BYTES;
  static_assert(KIND == 0 || KIND == 1, "Gram or apply launch");
  static_assert(CTAS == 1 || CTAS == 2, "one CTA or a CTA pair");
  static_assert(B_ROWS % 64 == 0, "B rows per CTA: whole 64-row chunks");
  static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "TMEM columns: power of two");
  static_assert(EPI_BUFS >= 2 && EPI_BUFS <= 8, "chunk ring: 2 to 8 buffers (2 = no prefetch of C)");

  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[STAGES];
  __shared__ uint64_t empty_bar[STAGES];
  __shared__ uint64_t tmem_full_bar[2];
  __shared__ uint64_t tmem_empty_bar[2];
  __shared__ uint64_t c_full_bar[EPI_BUFS];      // chunk buffer holds its C operand / may be overwritten
  __shared__ uint64_t buf_ready_bar[EPI_BUFS];   // the eight math warps have written their results into it
  __shared__ uint64_t row_pair_bar[4];           // the math warps of a lane quarter (fp32 C chunks only)
  __shared__ uint32_t tmem_slot;
  __shared__ uint32_t abort_word;
  __shared__ uint32_t issue_turn;               // index of the next K block whose MMAs may be issued (two issuing threads)

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  volatile uint32_t* abort_flag = &abort_word;
  const uint32_t cta_rank = (CTAS == 2) ? cluster_cta_rank() : 0u;     // 0 issues the MMAs of the pair
  const uint32_t work_id = (CTAS == 2) ? (blockIdx.x >> 1) : blockIdx.x;

  if (threadIdx.x == 0) {
    abort_word = 0;
    issue_turn = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&tmem_full_bar[a]), 2);          // one commit of each MMA-issuing thread
      mbar_init(smem_u32(&tmem_empty_bar[a]), EPI_WARPS * CTAS);
    }
    for (int b = 0; b < EPI_BUFS; ++b) {
      mbar_init(smem_u32(&c_full_bar[b]), 1);
      mbar_init(smem_u32(&buf_ready_bar[b]), EPI_WARPS);
    }
    for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&row_pair_bar[i]), EPI_WARPS / 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) {   // the same warp of both CTAs allocates the pair's columns
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // the peer's barriers are initialised before anything signals them
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;

  const uint32_t tile_begin = args.cta_tile_start[work_id];
  const uint32_t tile_end = args.cta_tile_start[work_id + 1];

  auto load_operand = [&](uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    if (CTAS == 2) tma_load_3d_pair(dst, map, x, y, z, bar);
    else tma_load_3d(dst, map, x, y, z, bar);
  };
  const int row_shift = (int)cta_rank * GEMM_BM;   // this CTA's rows inside the tile of the pair

  if (warp == 0 || warp == 3 + EPI_WARPS || warp >= 5 + EPI_WARPS) {
    // ===================================================================== TMA producers
    // Four threads feed the operand ring, two for the even and two for the odd K blocks: one of each pair loads the A
    // tiles (and, in CTA 0, posts the bytes a stage expects), the other the B tiles.  The two threads of a K block wait
    // on the same "stage empty" barrier.  A B copy may complete before the A thread has posted the expected bytes of
    // its stage: the barrier's transaction count is signed, and its phase cannot end before that post, which is also
    // the phase's only pending arrival.  (One thread issuing all copies of a stage - four when both operands are
    // MN-major - was the bound of those launches.)
    if (lane == 0) {
      const bool do_a = (warp == 0 || warp == 5 + EPI_WARPS);
      const uint32_t my_parity = (warp >= 5 + EPI_WARPS) ? 1u : 0u;   // this thread serves the even or the odd K blocks
      uint32_t it = 0;   // running k-block counter across tiles
      const uint32_t full0 = (CTAS == 2) ? map_to_cta(smem_u32(&full_bar[0]), 0) : smem_u32(&full_bar[0]);
      bool ok = true;
      for (uint32_t t = tile_begin; t < tile_end && ok; ++t) {
        const TileEntry te = args.tiles[t];
        const GemmProblem& pr = args.problems[te.problem];
        const CUtensorMap* map = args.tmaps + (do_a ? pr.tmapA : pr.tmapB);
        // this CTA's rows of its operand
        const int r0 = do_a ? te.tm * TILE_M + (int)cta_rank * GEMM_BM : te.tn * BN + (int)cta_rank * B_ROWS;
        const int batch = pr.batch;
        const int mn = do_a ? pr.a_mn : pr.b_mn;
        // FP8 operands (Gram launches only): a stage still holds 128 bytes along K, i.e. 128 elements instead of 64,
        // and an MN-major tile is one 128-wide chunk of 128 k-rows instead of two 64-wide chunks of 64
        const bool fp8 = KIND == 0 && pr.fp8 != 0;
        const int kelem = fp8 ? 2 * GEMM_BK : GEMM_BK;
        const int nk = (pr.K + kelem - 1) / kelem;
        const int nseg = pr.nseg > 1 ? pr.nseg : 1;           // split-precision products: segments along K
        // Diagonal tile of a one-segment Gram product: this CTA's B rows are its A rows, so B is not loaded
        // and the MMA reads the A tile for both operands (B_ROWS == GEMM_BM and equal box shapes).
        const bool share_ab = KIND == 0 && B_ROWS == GEMM_BM && pr.diag_share != 0 && te.tm == te.tn;
        const uint32_t stage_tx = share_ab ? CTAS * A_BYTES : CTAS * STAGE_BYTES;
        const bool skip = !do_a && share_ab;
        const int chunks = (do_a ? GEMM_BM : B_ROWS) / 64;
        for (int seg = 0; seg < nseg && ok; ++seg) {
          if (seg == 1) map = args.tmaps + (do_a ? pr.tmapA2 : pr.tmapB2);
          else if (seg == 2) map = args.tmaps + (do_a ? pr.tmapA3 : pr.tmapB3);
          for (int kb = 0; kb < nk; ++kb, ++it) {
            if ((it & 1u) != my_parity) continue;
            const uint32_t s = it % (uint32_t)STAGES, par = ((it / (uint32_t)STAGES) & 1u) ^ 1u;   // ring position, parity of its "empty" barrier
            if (!mbar_wait(smem_u32(&empty_bar[0]) + 8u * s, par, abort_flag, args.status, args.wait_limit_ns)) { ok = false; break; }
            // the "full" barrier of the pair is CTA 0's: it expects the bytes of both CTAs
            const uint32_t fb = full0 + 8u * s;
            if (do_a && cta_rank == 0) mbar_expect_tx(smem_u32(&full_bar[0]) + 8u * s, stage_tx);
            const uint32_t dst = smem_base + s * STAGE_BYTES + (do_a ? 0u : A_BYTES);
            const int k0 = kb * kelem;
            if (skip) {
            } else if (!mn) {
              load_operand(dst, map, k0, r0, batch, fb);
            } else if (fp8) {
              load_operand(dst, map, r0, k0, batch, fb);
            } else {
              for (int c = 0; c < chunks; ++c) load_operand(dst + c * 8192, map, r0 + 64 * c, k0, batch, fb);
            }
          }
        }
      }
      if (!ok) {
        // Abort path: let the copies already issued land before the CTA's shared memory goes away.
        if (cta_rank == 0 && do_a && my_parity == 0) {
          const uint32_t pending = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
          for (uint32_t j = 0; j < pending; ++j) {
            const uint32_t i2 = it - 1 - j;
            uint32_t spins = 0;
            while (!mbar_try_wait(smem_u32(&full_bar[i2 % STAGES]), (i2 / STAGES) & 1u) && ++spins < (1u << 22)) {}
          }
        } else {
          // the barrier that counts these copies is not this thread's to poll: give them a fixed 100 us
          const uint64_t t0 = global_timer_ns();
          while (global_timer_ns() - t0 < 100000ull) {}
        }
      }
    }
  } else if (warp == 1 || warp == 4 + EPI_WARPS) {
    // ===================================================================== MMA issuers (CTA 0 of a pair)
    // A tcgen05.mma occupies its issuing thread for as long as the tensor core takes to accept it, and whatever
    // else that thread does between two instructions (barrier waits, descriptor arithmetic, the commit) is time in
    // which the tensor pipe has nothing to do: measured, every cycle of such work lengthens a K block by a cycle.
    // So two threads issue alternate K blocks.  Each prepares its K block (waits for the stage, forms the
    // descriptors) while the other one's instructions run, then waits for its turn, issues its four instructions
    // and passes the turn on.  The turn (a K-block counter in shared memory, handed over between
    // tcgen05.fence::before_thread_sync and ::after_thread_sync) keeps the instructions of a tile in K order, so the
    // accumulation order - and with it every result bit - does not depend on timing.  A commit covers the MMAs of its
    // own thread only: each thread frees the stages it consumed, and both commit to the accumulator's barrier.
    if (lane == 0 && cta_rank == 0) {
      const uint32_t me = (warp == 1) ? 0u : 1u;
      const uint32_t turn_addr = smem_u32(&issue_turn);
      uint32_t tcount = 0;
      uint32_t it0 = 0;                            // index of the tile's first K block in the CTA's K-block sequence
      bool ok = true;
      for (uint32_t t = tile_begin; t < tile_end && ok; ++t, ++tcount) {
        const TileEntry te = args.tiles[t];
        const GemmProblem& pr = args.problems[te.problem];
        const int a_mn = pr.a_mn, b_mn = pr.b_mn;
        const bool fp8 = KIND == 0 && pr.fp8 != 0;
        const int kelem = fp8 ? 2 * GEMM_BK : GEMM_BK;
        const uint32_t nk = (uint32_t)(((pr.K + kelem - 1) / kelem) * (pr.nseg > 1 ? pr.nseg : 1));
        const uint32_t idesc = instr_desc(TILE_M, BN, a_mn, b_mn, fp8 ? 1 : 0);
        // MN-major operands: bytes between the 16 (bf16) or 32 (FP8) k-rows of consecutive instructions, and between
        // 128-byte-wide chunks along M/N (a 128-row FP8 tile is a single chunk)
        const uint32_t mn_step = fp8 ? 4096u : 2048u, mn_lbo = fp8 ? 16384u : 8192u;
        const bool share_ab = KIND == 0 && B_ROWS == GEMM_BM && pr.diag_share != 0 && te.tm == te.tn;
        const uint32_t acc = tcount & 1u;
        const uint32_t acc_round = tcount >> 1;
        if (!mbar_wait(smem_u32(&tmem_empty_bar[acc]), (acc_round & 1u) ^ 1u, abort_flag, args.status, args.wait_limit_ns)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        // The descriptors of a tile differ only in their start-address field: the low word is the stage's address
        // field plus a per-tile constant (leading byte offset), advanced by a per-tile step for each of the four
        // instructions of a K block; the high word (stride byte offset 1024, version, 128-byte swizzle) never changes.
        const uint32_t a_lo_const = ((a_mn ? mn_lbo : 16u) >> 4) << 16, b_lo_const = ((b_mn ? mn_lbo : 16u) >> 4) << 16;
        const uint32_t a_step = (a_mn ? mn_step : 32u) >> 4, b_step = (b_mn ? mn_step : 32u) >> 4;
        const uint32_t b_off = share_ab ? 0u : A_BYTES;
        auto run_tile = [&](auto fp8_tag) {
          constexpr bool FP8 = decltype(fp8_tag)::value;
          // this thread's K blocks of the tile: those whose index in the CTA's sequence has its parity
          for (uint32_t kb = (it0 + me) & 1u; kb < nk; kb += 2) {
            const uint32_t it = it0 + kb;
            const uint32_t s = it % (uint32_t)STAGES, par = (it / (uint32_t)STAGES) & 1u;
            if (!mbar_wait(smem_u32(&full_bar[0]) + 8u * s, par, abort_flag, args.status, args.wait_limit_ns)) { ok = false; break; }
            const uint32_t sa = smem_base + s * STAGE_BYTES;
            const uint32_t a_lo = ((sa >> 4) & 0x3fffu) | a_lo_const, b_lo = (((sa + b_off) >> 4) & 0x3fffu) | b_lo_const;
            // wait for the turn (bounded like every other wait)
            {
              uint32_t v, spins = 0;
              uint64_t t_first = 0;
              for (;;) {
                asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(turn_addr) : "memory");
                if (v == it) break;
                if ((++spins & 1023u) == 0) {
                  if (*abort_flag) { ok = false; break; }
                  const uint64_t now = global_timer_ns();
                  if (t_first == 0) t_first = now;
                  else if (now - t_first > args.wait_limit_ns) {
                    *abort_flag = 1;
                    atomicExch(args.status, (uint32_t)STATUS_TIMEOUT);
                    ok = false;
                    break;
                  }
                }
              }
              if (!ok) break;
            }
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < GEMM_BK / 16; ++kk)
              tc_mma_words<CTAS == 2, FP8>(d_tmem, a_lo + kk * a_step, b_lo + kk * b_step, SMEM_DESC_HI_SBO1024, idesc,
                                           (kb | (uint32_t)kk) != 0 ? 1u : 0u);
            tc_fence_before();
            asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(turn_addr), "r"(it + 1u) : "memory");
            // frees the stage (in both CTAs of a pair) once these MMAs have read it
            if (CTAS == 2) tc_commit_pair(smem_u32(&empty_bar[0]) + 8u * s); else tc_commit(smem_u32(&empty_bar[0]) + 8u * s);
          }
        };
        if (fp8) run_tile(std::integral_constant<bool, true>{}); else run_tile(std::integral_constant<bool, false>{});
        if (ok) {                                    // this thread's share of the accumulator is complete
          if (CTAS == 2) tc_commit_pair(smem_u32(&tmem_full_bar[acc])); else tc_commit(smem_u32(&tmem_full_bar[acc]));
        }
        it0 += nk;
      }
    }
  } else {
    // ===================================================================== epilogue
    // Chunks (64 output columns of this CTA's 128 rows) are numbered g = 0, 1, ... across the CTA's tiles;
    // chunk g lives in ring buffer g % EPI_BUFS.  For every chunk the TMA thread (warp 2 + EPI_WARPS) first makes the
    // buffer available - it waits until the store that last used the buffer has left shared memory, then
    // either starts the C loads on c_full_bar (bytes expected) or just arrives on it - and it does so
    // PREFETCH chunks ahead of the chunk whose results it sends off.  A math warp waits on c_full_bar,
    // reads its accumulator columns, combines, writes the results in place and arrives on buf_ready_bar;
    // the TMA thread waits on that and issues the stores.
    constexpr uint32_t PREFETCH = EPI_BUFS;      // every buffer is handed out again as soon as its store has left it
    if (warp == 2 + EPI_WARPS) {
      // ------------------------------------------------------------------- epilogue TMA thread
      if (lane == 0) {
        bool ok = true;
        // load-side cursor
        uint32_t pf_t = tile_begin, pf_g = 0;
        int pf_ch = 0, pf_n = 0, pf_row0 = 0, pf_n0 = 0;
        const GemmProblem* pf_pr = nullptr;
        const CUtensorMap* pf_map0 = nullptr;
        const CUtensorMap* pf_map1 = nullptr;
        int pf_cmode = 0, pf_batch = 0;
        bool pf_live = false;
        uint32_t pf_issued = 0;
        auto pf_enter_tile = [&]() {
          if (pf_t >= tile_end) return;
          const TileEntry te = args.tiles[pf_t];
          pf_pr = &args.problems[te.problem];
          pf_row0 = te.tm * TILE_M + row_shift;
          pf_n0 = te.tn * BN;
          pf_n = (pf_pr->N - pf_n0 + 63) / 64;
          if (pf_n > BN / 64) pf_n = BN / 64;
          pf_live = KIND == 1 && pf_pr->tma_c != 0 && pf_row0 < pf_pr->M;
          pf_cmode = pf_pr->c_mode; pf_batch = pf_pr->batch_c;
          pf_map0 = args.tmaps + pf_pr->tmapC0; pf_map1 = args.tmaps + pf_pr->tmapC1;
          pf_ch = 0;
        };
        auto pf_step = [&]() {                   // makes the buffer of chunk pf_g available to the math warps
          if (pf_t >= tile_end) return;
          const uint32_t nb = pf_g % EPI_BUFS;
          if (pf_live) {
            epi_issue_c_load(pf_cmode, pf_map0, pf_map1, pf_batch, pf_row0, pf_n0 + pf_ch * 64, epi_base + nb * BUF_BYTES,
                             smem_u32(&c_full_bar[nb]));
            ++pf_issued;
          } else {
            mbar_arrive(smem_u32(&c_full_bar[nb]));
          }
          ++pf_g;
          if (++pf_ch == pf_n) { ++pf_t; pf_enter_tile(); }
        };
        pf_enter_tile();
        for (uint32_t j = 0; j + 1 <= PREFETCH; ++j) pf_step();
        uint32_t g = 0;
        for (uint32_t t = tile_begin; t < tile_end && ok; ++t) {
          const TileEntry te = args.tiles[t];
          const GemmProblem& pr = args.problems[te.problem];
          const int row0 = te.tm * TILE_M + row_shift;
          const int n0 = te.tn * BN;
          int n_chunks = (pr.N - n0 + 63) / 64;
          if (n_chunks > BN / 64) n_chunks = BN / 64;
          const bool rows_live = row0 < pr.M;
          const int epi = (KIND == 0) ? (int)EPI_GRAM : pr.epi;
          const bool store_hi = (KIND == 0 || epi == EPI_APPLY || (epi == EPI_APPLY_PACK && pr.store_out)) &&
                                pr.tma_out != 0 && rows_live;
          const bool store_lo = (KIND == 1 && epi == EPI_APPLY && pr.hi_only == 0) || (KIND == 0 && pr.gram_lo != 0);
          const bool mirror = KIND == 0 && pr.sym != 0 && pr.gram_lo == 0 && te.tn != te.tm && rows_live;
          const CUtensorMap* mapO0 = args.tmaps + pr.tmapO0;
          const CUtensorMap* mapO1 = args.tmaps + pr.tmapO1;
          const CUtensorMap* mapOT = args.tmaps + pr.tmapOT;
          const int batch_o = pr.batch_o, prM = pr.M;
          for (int ch = 0; ch < n_chunks; ++ch, ++g) {
            const uint32_t b = g % EPI_BUFS;
            const uint32_t buf = epi_base + b * BUF_BYTES;
            const int col0 = n0 + ch * 64;
            if (!mbar_wait(smem_u32(&buf_ready_bar[b]), (g / EPI_BUFS) & 1u, abort_flag, args.status, args.wait_limit_ns)) { ok = false; break; }
            if (store_hi) {
              tma_store_3d(mapO0, col0, row0, batch_o, buf);
              if (store_lo) tma_store_3d(mapO1, col0, row0, batch_o, buf + EPI_HALF_BYTES);
              if (mirror) {                      // rows col0.. of the output, columns row0.. (two 64-column boxes)
                tma_store_3d(mapOT, row0, col0, batch_o, buf + EPI_HALF_BYTES);
                if (row0 + 64 < prM) tma_store_3d(mapOT, row0 + 64, col0, batch_o, buf + EPI_HALF_BYTES + 8192u);
              }
            }
            bulk_commit();
            // The buffer goes straight to chunk g + EPI_BUFS: wait until this store has read it out of shared
            // memory (a few hundred cycles), then start that chunk's C loads (or just release the buffer).
            bulk_wait_read<0>();
            pf_step();
          }
        }
        if (!ok && pf_issued) {                  // abort path: give the loads in flight a fixed 100 us to land
          const uint64_t t0 = global_timer_ns();
          while (global_timer_ns() - t0 < 100000ull) {}
        }
        bulk_wait_all();                         // stores must be complete before the CTA retires
      }
    } else {
      // ------------------------------------------------------------------- epilogue math warps (2 .. 9)
      const int q = warp & 3;                    // TMEM lane quarter this warp may read
      constexpr int NC = EPI_NCOL;               // columns per thread
      constexpr int UNITS = NC / 8;              // 16-byte units of bf16 per thread
      const int sub = (warp - 2) >> 2;           // which NC of a chunk's 64 columns
      const int r_in = q * 32 + lane;            // row of the tile this thread owns
      const uint32_t row_off = (uint32_t)r_in * 128u;
      const uint32_t sw = (uint32_t)(r_in & 7);
      uint32_t g = 0, tcount = 0, f32_chunks = 0;
      bool ok = true;
      for (uint32_t t = tile_begin; t < tile_end && ok; ++t, ++tcount) {
        const TileEntry te = args.tiles[t];
        const GemmProblem& pr = args.problems[te.problem];
        // the fields used per chunk, read once per tile
        const int prM = pr.M, prN = pr.N, c_mode = pr.c_mode;
        const int epi = (KIND == 0) ? (int)EPI_GRAM : pr.epi;
        const int row0 = te.tm * TILE_M + row_shift;
        const int row = row0 + r_in;
        const int n0 = te.tn * BN;
        int n_chunks = (prN - n0 + 63) / 64;
        if (n_chunks > BN / 64) n_chunks = BN / 64;
        const float scale = pr.scale_ptr ? __ldg(pr.scale_ptr) : pr.scale_imm;
        const float own = pr.own_coef;           // coefficient of the own term (1.5 for one Newton-Schulz step)
        // a CTA whose 128 rows lie wholly below the matrix moves nothing through TMA (it still drains TMEM)
        const bool rows_live = row0 < prM;
        const bool tma_c = KIND == 1 && pr.tma_c != 0 && rows_live, tma_out = pr.tma_out != 0;
        const bool store_hi = KIND == 0 || epi == EPI_APPLY || (epi == EPI_APPLY_PACK && pr.store_out);
        const bool store_lo = (KIND == 1 && epi == EPI_APPLY && pr.hi_only == 0) || (KIND == 0 && pr.gram_lo != 0);
        const bool mirror = KIND == 0 && pr.sym != 0 && pr.gram_lo == 0 && te.tn != te.tm && rows_live;   // off-diagonal Gram tile
        // symmetric result with hi/lo outputs: the hi part of an off-diagonal tile also goes to the transposed place
        const bool mirror_hi = pr.sym != 0 && pr.mirror_hi != 0 && te.tn != te.tm && row < prM;
        bf16* const out_t = reinterpret_cast<bf16*>(pr.out) + row;
        const int64_t ld_out = pr.ld_out;
        const bf16* c2_hi = nullptr;
        const bf16* c2_lo = nullptr;
        if (KIND == 1 && pr.C2 != nullptr && row < prM) {
          c2_hi = pr.C2 + (size_t)row * ld_out;
          c2_lo = pr.C2_lo + (size_t)row * ld_out;
        }
        const float c2_coef = pr.c2_coef;
        const uint32_t acc = tcount & 1u;
        const uint32_t acc_round = tcount >> 1;
        ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_round & 1u, abort_flag, args.status, args.wait_limit_ns);
        ok = __all_sync(0xffffffffu, ok);        // the whole warp takes the same exit
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16) + (uint32_t)(sub * NC);
#pragma unroll 1
        for (int ch = 0; ch < n_chunks; ++ch, ++g) {
          const uint32_t b = g % EPI_BUFS;
          const uint32_t buf = epi_base + b * BUF_BYTES;
          const int col0 = n0 + ch * 64 + sub * NC;    // first of this thread's columns
          // second linear term of a chain product: this thread's NC columns of its row, hi and lo parts (one cache line
          // each), requested before the waits so that their latency is hidden
          if (KIND == 1 && c2_hi != nullptr && col0 < prN) {
            asm volatile("prefetch.global.L1 [%0];" ::"l"(c2_hi + col0));
            asm volatile("prefetch.global.L1 [%0];" ::"l"(c2_lo + col0));
          }
          ok = mbar_wait(smem_u32(&c_full_bar[b]), (g / EPI_BUFS) & 1u, abort_flag, args.status, args.wait_limit_ns);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          float v[NC];
          tc_ld_cols(taddr + ch * 64, v);
          if (ch == n_chunks - 1) {              // last read of this accumulator: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (CTAS == 2) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));
              else mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
            }
          }
          if (KIND == 1 && c2_hi != nullptr) {
#pragma unroll
            for (int u = 0; u < UNITS; ++u) {
              if (col0 + u * 8 >= prN) break;
              const uint4 uh = __ldg(reinterpret_cast<const uint4*>(c2_hi + col0 + u * 8));
              const uint4 ul = __ldg(reinterpret_cast<const uint4*>(c2_lo + col0 + u * 8));
              const uint32_t wh[4] = {uh.x, uh.y, uh.z, uh.w};
              const uint32_t wl[4] = {ul.x, ul.y, ul.z, ul.w};
              float* o = v + u * 8;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                o[2 * e] = fmaf(c2_coef, __uint_as_float(wh[e] << 16) + __uint_as_float(wl[e] << 16), o[2 * e]);
                o[2 * e + 1] = fmaf(c2_coef, __uint_as_float(wh[e] & 0xffff0000u) + __uint_as_float(wl[e] & 0xffff0000u),
                                    o[2 * e + 1]);
              }
            }
          }
          if (KIND == 0) {
            const float f = -0.5f * scale;
#pragma unroll
            for (int j = 0; j < NC; ++j) v[j] *= f;
          } else if (tma_c) {
            if (c_mode == C_F32) {               // half h of the buffer = fp32 columns 32 h .. 32 h + 31
              const uint32_t fhalf = (uint32_t)(sub * NC) >> 5, funit0 = ((uint32_t)(sub * NC) & 31u) >> 2;
#pragma unroll
              for (int cc = 0; cc < NC / 4; ++cc) {
                const uint32_t c16 = funit0 + (uint32_t)cc;
                const uint4 u = lds128(buf + fhalf * EPI_HALF_BYTES + row_off + ((c16 ^ sw) << 4));
                float* o = v + cc * 4;
                o[0] = scale * fmaf(own, __uint_as_float(u.x), o[0]);
                o[1] = scale * fmaf(own, __uint_as_float(u.y), o[1]);
                o[2] = scale * fmaf(own, __uint_as_float(u.z), o[2]);
                o[3] = scale * fmaf(own, __uint_as_float(u.w), o[3]);
              }
              // The bf16 results go to this thread's units of BOTH halves, i.e. into fp32 columns that other warps
              // of this lane quarter still have to read: all of them finish reading before any writes.
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&row_pair_bar[q]));
              ok = mbar_wait(smem_u32(&row_pair_bar[q]), f32_chunks & 1u, abort_flag, args.status, args.wait_limit_ns);
              ++f32_chunks;
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
            } else {
              const bool has_lo = c_mode == C_HILO;
#pragma unroll
              for (int c = 0; c < UNITS; ++c) {
                const uint32_t c16 = (uint32_t)(sub * UNITS + c);
                const uint4 uh = lds128(buf + row_off + ((c16 ^ sw) << 4));
                uint4 ul = make_uint4(0, 0, 0, 0);
                if (has_lo) ul = lds128(buf + EPI_HALF_BYTES + row_off + ((c16 ^ sw) << 4));
                const uint32_t wh[4] = {uh.x, uh.y, uh.z, uh.w};
                const uint32_t wl[4] = {ul.x, ul.y, ul.z, ul.w};
                float* o = v + c * 8;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float c0 = __uint_as_float(wh[e] << 16) + __uint_as_float(wl[e] << 16);
                  const float c1 = __uint_as_float(wh[e] & 0xffff0000u) + __uint_as_float(wl[e] & 0xffff0000u);
                  o[2 * e] = scale * fmaf(own, c0, o[2 * e]);
                  o[2 * e + 1] = scale * fmaf(own, c1, o[2 * e + 1]);
                }
              }
            }
          } else if (KIND == 1) {
            apply_c_direct<NC>(pr, scale, row, col0, v);
          }
          // ---- outputs
          if (mirror_hi) {
            // lanes hold consecutive rows: one column of the tile is 64 contiguous bytes of the transposed tile
#pragma unroll
            for (int j = 0; j < NC; ++j)
              if (col0 + j < prN) out_t[(size_t)(col0 + j) * ld_out] = __float2bfloat16_rn(v[j]);
          }
          if (store_hi) {
            if (tma_out) {
#pragma unroll
              for (int c = 0; c < UNITS; ++c) {
                const uint32_t c16 = (uint32_t)(sub * UNITS + c);
                const float* o = v + c * 8;
                uint32_t wh[4], wl[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  wh[e] = pack_bf16x2(o[2 * e], o[2 * e + 1]);
                  wl[e] = pack_bf16x2(o[2 * e] - __uint_as_float(wh[e] << 16),
                                      o[2 * e + 1] - __uint_as_float(wh[e] & 0xffff0000u));
                }
                sts128(buf + row_off + ((c16 ^ sw) << 4), make_uint4(wh[0], wh[1], wh[2], wh[3]));
                if (store_lo) sts128(buf + EPI_HALF_BYTES + row_off + ((c16 ^ sw) << 4), make_uint4(wl[0], wl[1], wl[2], wl[3]));
              }
              if (mirror) {
                // transposed copy: element (j, r) of a 64 x 128 chunk kept as two {64 x 64} swizzled boxes
                const uint32_t tb = buf + EPI_HALF_BYTES + (uint32_t)(r_in >> 6) * 8192u + (uint32_t)(r_in & 7) * 2u;
                const uint32_t unit = (uint32_t)(r_in & 63) >> 3;
#pragma unroll
                for (int j = 0; j < NC; ++j) {
                  const uint16_t h = __bfloat16_as_ushort(__float2bfloat16_rn(v[j]));
                  const uint32_t jj = (uint32_t)(sub * NC + j);
                  asm volatile("st.shared.u16 [%0], %1;" ::"r"(tb + jj * 128u + ((unit ^ (jj & 7u)) << 4)), "h"(h) : "memory");
                }
              }
              fence_async_smem();
            } else {
              store_out_direct<NC>(pr, row, col0, v, store_lo);
            }
          }
          if (KIND == 1 && epi == EPI_APPLY_PACK) {
            if (NC == 32) pack_bits_direct(pr, row, col0, v, args.peers); else pack_bits16_direct(pr, row, col0, v, args.peers);
          } else if (KIND == 1 && epi == EPI_APPLY_UPDATE) {
            update_weights_direct<NC>(pr, args.params, args.lr, row, col0, v);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&buf_ready_bar[b]));   // this warp's part of the chunk is in shared memory
        }
      }
    }
  }

  tc_fence_before();
  if (CTAS == 2) {
    // neither CTA may retire (or free TMEM) while the peer can still signal its barriers or read its operands
    cluster_sync_all();
    if (warp == 1)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  } else {
    __syncthreads();
    if (warp == 1)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Self-test of the bounded wait: one thread waits, with the same mbar_wait as the product kernel, on an mbarrier
// that nothing ever arrives at.  The wait runs out after `limit_ns`, the status word receives STATUS_TIMEOUT
// and the kernel returns normally; the context stays usable.
__global__ void wait_timeout_probe_kernel(uint32_t* status, uint64_t limit_ns) {
  __shared__ uint64_t never_bar;
  __shared__ uint32_t abort_word;
  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(smem_u32(&never_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    volatile uint32_t* abort_flag = &abort_word;
    mbar_wait(smem_u32(&never_bar), 0u, abort_flag, status, limit_ns);
  }
}

template <int BN, int STAGES, int EPI_BUFS, int CTAS, int KIND>
constexpr size_t ns_gemm_tc_smem_bytes() {
  return (size_t)STAGES * (GEMM_BM * GEMM_BK * 2 + (BN / CTAS) * GEMM_BK * 2) +
         (size_t)EPI_BUFS * EPI_BUF_BYTES + 1024;
}

}  // namespace signmuon
