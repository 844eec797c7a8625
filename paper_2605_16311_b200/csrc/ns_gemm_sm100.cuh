// Newton-Schulz products on the 5th-generation tensor cores (sm_100a):
//   grouped, persistent, warp-specialised bf16 GEMM  D[M x N] = sum_k a(i,k) b(j,k)
//   - operands staged by TMA (3-D tiled tensor maps, 128-byte swizzle) into a multi-stage
//     shared-memory ring guarded by mbarriers,
//   - tcgen05.mma (kind::f16, bf16 x bf16 -> fp32) issued by one thread, accumulators in TMEM,
//     double-buffered so the epilogue of tile t overlaps the main loop of tile t+1,
//   - epilogue warps read TMEM with tcgen05.ld and apply the fused Newton-Schulz epilogues
//     (Gram scaling, 1.5 Y + Q Y, sign + pack, weight update).
// One launch covers every (parameter, worker) product of one Newton-Schulz half-iteration: each
// CTA walks a host-built list of tiles (problem, tile_m, tile_n).
//
// Operand layouts in shared memory (one 64-wide K block per stage):
//   K-major  (contiguous along K):  rows of 128 bytes, TMA box {64 k, R rows}, 8-row swizzle atoms
//            of 1024 bytes; descriptor SBO = 1024, a 16-element K step advances the start by 32 bytes.
//   MN-major (contiguous along M/N): per 64 rows of M/N one 8 KB chunk = 64 k-rows of 128 bytes,
//            TMA box {64 mn, 64 k}; descriptor LBO = 8192 (next chunk), SBO = 1024 (next 8 k-rows),
//            a 16-element K step advances the start by 2048 bytes.
// Every wait is bounded: after about two seconds a waiting thread records STATUS_TIMEOUT in the
// status word, raises a CTA-wide abort flag and the CTA drains and exits (TMEM is freed).
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace signmuon {

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;
constexpr int GEMM_THREADS = 192;            // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

struct GemmLaunchArgs {
  const CUtensorMap* tmaps;
  const GemmProblem* problems;
  const TileEntry* tiles;
  const uint32_t* cta_tile_start;   // [gridDim.x + 1]
  const ParamDev* params;
  uint32_t* status;
  float lr;
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
                                          uint32_t* status) {
  uint32_t spins = 0;
  uint64_t t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > WAIT_LIMIT_NS) {
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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

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

// Instruction descriptor, kind::f16: D fp32 (bits [4,6) = 1), A/B bf16 (bits [7,10) = [10,13) = 1),
// bit 15 / 16: A / B contiguous along M / N, bits [17,23) N >> 3, bits [24,29) M >> 4.
__device__ __forceinline__ uint32_t instr_desc(int n, int a_mn, int b_mn) {
  uint32_t d = 0;
  d |= 1u << 4;
  d |= 1u << 7;
  d |= 1u << 10;
  d |= (uint32_t)(a_mn & 1) << 15;
  d |= (uint32_t)(b_mn & 1) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(GEMM_BM >> 4) << 24;
  return d;
}

// ------------------------------------------------------------------------------------------ kernel
template <int BN, int STAGES>
__global__ void __launch_bounds__(GEMM_THREADS, 1) ns_gemm_tc_kernel(const GemmLaunchArgs args) {
  constexpr uint32_t A_BYTES = GEMM_BM * GEMM_BK * 2;          // 16 KB
  constexpr uint32_t B_BYTES = BN * GEMM_BK * 2;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN;                       // two accumulator buffers
  static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "TMEM columns: power of two");

  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[STAGES];
  __shared__ uint64_t empty_bar[STAGES];
  __shared__ uint64_t tmem_full_bar[2];
  __shared__ uint64_t tmem_empty_bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ uint32_t abort_word;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  volatile uint32_t* abort_flag = &abort_word;

  if (threadIdx.x == 0) {
    abort_word = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&tmem_full_bar[a]), 1);
      mbar_init(smem_u32(&tmem_empty_bar[a]), 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;

  const uint32_t tile_begin = args.cta_tile_start[blockIdx.x];
  const uint32_t tile_end = args.cta_tile_start[blockIdx.x + 1];

  if (warp == 0) {
    // ===================================================================== TMA producer
    if (lane == 0) {
      uint32_t it = 0;   // running k-block counter across tiles
      bool ok = true;
      for (uint32_t t = tile_begin; t < tile_end && ok; ++t) {
        const TileEntry te = args.tiles[t];
        const GemmProblem& pr = args.problems[te.problem];
        const CUtensorMap* mapA = args.tmaps + pr.tmapA;
        const CUtensorMap* mapB = args.tmaps + pr.tmapB;
        const int m0 = te.tm * GEMM_BM, n0 = te.tn * BN, batch = pr.batch;
        const int a_mn = pr.a_mn, b_mn = pr.b_mn;
        const int nk = (pr.K + GEMM_BK - 1) / GEMM_BK;
        for (int kb = 0; kb < nk; ++kb, ++it) {
          const uint32_t s = it % STAGES;
          const uint32_t round = it / STAGES;
          if (!mbar_wait(smem_u32(&empty_bar[s]), (round & 1u) ^ 1u, abort_flag, args.status)) { ok = false; break; }
          const uint32_t fb = smem_u32(&full_bar[s]);
          mbar_expect_tx(fb, STAGE_BYTES);
          const uint32_t sa = smem_base + s * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          const int k0 = kb * GEMM_BK;
          if (!a_mn) {
            tma_load_3d(sa, mapA, k0, m0, batch, fb);
          } else {
#pragma unroll
            for (int c = 0; c < GEMM_BM / 64; ++c) tma_load_3d(sa + c * 8192, mapA, m0 + 64 * c, k0, batch, fb);
          }
          if (!b_mn) {
            tma_load_3d(sb, mapB, k0, n0, batch, fb);
          } else {
#pragma unroll
            for (int c = 0; c < BN / 64; ++c) tma_load_3d(sb + c * 8192, mapB, n0 + 64 * c, k0, batch, fb);
          }
        }
      }
      if (!ok) {
        // Abort path: let the copies already issued land before the CTA's shared memory goes away.
        const uint32_t pending = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
        for (uint32_t j = 0; j < pending; ++j) {
          const uint32_t i2 = it - 1 - j;
          uint32_t spins = 0;
          while (!mbar_try_wait(smem_u32(&full_bar[i2 % STAGES]), (i2 / STAGES) & 1u) && ++spins < (1u << 22)) {}
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================================== MMA issuer
    if (lane == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (uint32_t t = tile_begin; t < tile_end && ok; ++t, ++tcount) {
        const TileEntry te = args.tiles[t];
        const GemmProblem& pr = args.problems[te.problem];
        const int a_mn = pr.a_mn, b_mn = pr.b_mn;
        const int nk = (pr.K + GEMM_BK - 1) / GEMM_BK;
        const uint32_t idesc = instr_desc(BN, a_mn, b_mn);
        const uint32_t acc = tcount & 1u;
        const uint32_t acc_round = tcount >> 1;
        if (!mbar_wait(smem_u32(&tmem_empty_bar[acc]), (acc_round & 1u) ^ 1u, abort_flag, args.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < nk; ++kb, ++it) {
          const uint32_t s = it % STAGES;
          const uint32_t round = it / STAGES;
          if (!mbar_wait(smem_u32(&full_bar[s]), round & 1u, abort_flag, args.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int kk = 0; kk < GEMM_BK / 16; ++kk) {
            const uint64_t adesc = a_mn ? smem_desc(sa + kk * 2048, 8192, 1024) : smem_desc(sa + kk * 32, 16, 1024);
            const uint64_t bdesc = b_mn ? smem_desc(sb + kk * 2048, 8192, 1024) : smem_desc(sb + kk * 32, 16, 1024);
            tc_mma_f16(d_tmem, adesc, bdesc, idesc, (kb | kk) != 0 ? 1u : 0u);
          }
          tc_commit(smem_u32(&empty_bar[s]));        // frees the stage once these MMAs have read it
        }
        if (ok) tc_commit(smem_u32(&tmem_full_bar[acc]));   // accumulator complete
      }
    }
  } else {
    // ===================================================================== epilogue (warps 2..5)
    const int q = warp & 3;                      // TMEM lane quarter this warp may read
    uint32_t tcount = 0;
    for (uint32_t t = tile_begin; t < tile_end; ++t, ++tcount) {
      const TileEntry te = args.tiles[t];
      const GemmProblem& pr = args.problems[te.problem];
      const uint32_t acc = tcount & 1u;
      const uint32_t acc_round = tcount >> 1;
      bool ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_round & 1u, abort_flag, args.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = te.tm * GEMM_BM + q * 32 + lane;
      const int n0 = te.tn * BN;
      const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        if (n0 + c * 32 >= pr.N) break;          // warp-uniform
        float v[32];
        tc_ld32(taddr + c * 32, v);
        epilogue_row32(pr, args.params, args.lr, row, n0 + c * 32, v);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

template <int BN, int STAGES>
constexpr size_t ns_gemm_tc_smem_bytes() {
  return (size_t)STAGES * (GEMM_BM * GEMM_BK * 2 + BN * GEMM_BK * 2) + 1024;
}

}  // namespace signmuon
