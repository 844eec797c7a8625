// Newton-Schulz iteration carried out in Gram space, on chip, for matrices whose short side s is at most 256.
//
// With A_k = Y_k Y_k^T (short side) the step Y_{k+1} = (3/2 I - A_k / 2) Y_k gives
//     A_{k+1} = P_k A_k P_k = 9/4 A_k - 3/2 A_k^2 + 1/4 A_k^3,        P_k = 3/2 I - A_k / 2,
//     Y_K     = T_K Y_0,   T_{k+1} = P_k T_k,   T_0 = I,
// so K iterations need Y only twice: once for A_0 (a Gram launch) and once for T_K Y_0 (an apply launch).  All
// matrices in between are s x s, symmetric and commute.  Writing T_k = t_k I + F_k with t_k = (3/2)^k keeps the
// large multiple of the identity out of the bf16 operands:
//     F_{k+1} = 3/2 F_k - t_k / 2 A_k - 1/2 A_k F_k,   F_0 = 0.
// This kernel runs that chain for one (matrix, worker) problem per CTA pair without touching global memory between
// iterations: A_k lives in shared memory as a bf16 hi/lo pair (hi is the tensor-core operand, hi + lo the value used
// in the fp32 combinations), the accumulator of the A-chain and Z_k = -2 F_k live in tensor memory, and the three
// products of an iteration (A A, A (A A), A F) are tcgen05.mma instructions of the pair (M = N = 256, K = s).
//
// Per CTA (rank r of the pair): rows [128 r, 128 r + 128) of every matrix.  A symmetric matrix serves as the A operand
// (its rows) and as the B operand (b(j,k) = X[j][k], rows again), so each CTA only ever needs its own rows: what its
// threads compute is what its next MMA reads.  Thread = row = TMEM lane; the four warps that share a tensor-memory lane
// quarter split the 32-column chunks between them (a thread always meets the same (row, chunk) cells, so the
// combination phases need no barrier of their own).  Shared memory: A_hi, A_lo and X (S_hi or F_hi), 64 KB each,
// K-major with 128-byte swizzle in four 64-column blocks.  Tensor memory: D0 (A-chain), D1 (Z).
//
//   input : Q_hi, Q_lo = hi/lo pair of -A_0 / 2 (what the Gram launch stores), [s][ldq] bf16
//   output: F_K as a hi/lo pair, written over the input; the apply launch then forms
//           Y_K = (1/sigma) (F_K Mom + (3/2)^K Mom).
// Every wait is bounded (see ns_gemm_sm100.cuh); the barrier structure does not depend on whether a wait ran out.
#pragma once

#include "ns_gemm_sm100.cuh"

namespace signmuon {

struct ChainProblem {
  bf16* q_hi;             // in: hi(-A_0 / 2), out: hi(F_K); [s][ldq]
  bf16* q_lo;             // in: lo(-A_0 / 2), out: lo(F_K)
  int32_t s, ldq;
};

struct ChainLaunchArgs {
  const ChainProblem* problems;
  const uint32_t* order;        // problem indices, grouped by CTA pair
  const uint32_t* pair_start;   // [pairs + 1] into `order`
  uint32_t* status;
  uint64_t wait_limit_ns;
  int32_t K;                    // Newton-Schulz iterations (>= 2)
};

constexpr int CHAIN_COLGROUPS = 4;                           // warps that share a lane quarter, each walking every 4th chunk
constexpr int CHAIN_THREADS = 128 * CHAIN_COLGROUPS;
constexpr uint32_t CHAIN_BUF_BYTES = 128 * 256 * 2;            // 128 rows x 256 columns of bf16
constexpr size_t CHAIN_SMEM_BYTES = 3 * CHAIN_BUF_BYTES + 1024;

__device__ __forceinline__ void tc_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory address of the 16-byte unit that holds columns [8 u, 8 u + 8) of row `row` of an operand buffer.
__device__ __forceinline__ uint32_t chain_unit_addr(uint32_t buf, int row, int u) {
  return buf + (uint32_t)(u >> 3) * 16384u + (uint32_t)row * 128u + ((((uint32_t)u & 7u) ^ ((uint32_t)row & 7u)) << 4);
}
// Writes 32 consecutive values (columns [32 ch, 32 ch + 32) of row `row`) as bf16 hi (and lo) units.
__device__ __forceinline__ void chain_store_row32(uint32_t buf_hi, uint32_t buf_lo, int row, int ch, const float (&v)[32]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint32_t wh[4], wl[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = v[q * 8 + 2 * e], b = v[q * 8 + 2 * e + 1];
      wh[e] = pack_bf16x2(a, b);
      wl[e] = pack_bf16x2(a - __uint_as_float(wh[e] << 16), b - __uint_as_float(wh[e] & 0xffff0000u));
    }
    sts128(chain_unit_addr(buf_hi, row, ch * 4 + q), make_uint4(wh[0], wh[1], wh[2], wh[3]));
    if (buf_lo) sts128(chain_unit_addr(buf_lo, row, ch * 4 + q), make_uint4(wl[0], wl[1], wl[2], wl[3]));
  }
}
// Reads columns [32 ch, 32 ch + 32) of row `row` as hi + lo.
__device__ __forceinline__ void chain_load_row32(uint32_t buf_hi, uint32_t buf_lo, int row, int ch, float (&v)[32]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 h = lds128(chain_unit_addr(buf_hi, row, ch * 4 + q));
    const uint4 l = lds128(chain_unit_addr(buf_lo, row, ch * 4 + q));
    const uint32_t wh[4] = {h.x, h.y, h.z, h.w}, wl[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[q * 8 + 2 * e] = __uint_as_float(wh[e] << 16) + __uint_as_float(wl[e] << 16);
      v[q * 8 + 2 * e + 1] = __uint_as_float(wh[e] & 0xffff0000u) + __uint_as_float(wl[e] & 0xffff0000u);
    }
  }
}

__global__ void __launch_bounds__(CHAIN_THREADS, 1) ns_chain_kernel(const __grid_constant__ ChainLaunchArgs args) {
  extern __shared__ uint8_t chain_smem_raw[];
  __shared__ uint64_t mma_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ uint32_t abort_word;

  const uint32_t smem_base = (smem_u32(chain_smem_raw) + 1023u) & ~1023u;
  const uint32_t buf_ahi = smem_base, buf_alo = smem_base + CHAIN_BUF_BYTES, buf_x = smem_base + 2 * CHAIN_BUF_BYTES;
  const int warp = threadIdx.x >> 5;
  const int quarter = warp & 3;                         // tensor-memory lane quarter this warp may access
  const int cg = warp >> 2;                             // which of the 32-column chunks this warp walks: cg, cg + 4, ...
  const int row = quarter * 32 + (threadIdx.x & 31);    // row of this CTA's 128 = TMEM lane
  const uint32_t rank = cluster_cta_rank();             // rank 0 issues the pair's MMAs
  const uint32_t pair = blockIdx.x >> 1;
  volatile uint32_t* abort_flag = &abort_word;

  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(smem_u32(&mma_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);  // this warp's lane quarter
  const uint32_t d0 = t_lane, d1 = t_lane + 256u;                        // A-chain accumulator, Z = -2 F
  const uint32_t d0_mma = tmem_base, d1_mma = tmem_base + 256u;

  uint32_t phase = 0;                                   // parity of the next completion of mma_bar
  bool ok = true;                                       // false once a wait ran out: work is skipped, barriers are kept

  // One product D (+)= X Y^T-form with both operands K-major in shared memory (rows = this CTA's 128 rows of X as
  // A operand and of Y as B operand), contraction over the first k16 blocks of 16 columns.
  auto issue_product = [&](uint32_t d_tmem, uint32_t buf_a, uint32_t buf_b, uint32_t idesc, int k16, bool accumulate) {
    // descriptor low words: start address (16-byte units) | leading byte offset 16; K-major, stride byte offset 1024
    const uint32_t a_lo = ((buf_a >> 4) & 0x3fffu) | (1u << 16), b_lo = ((buf_b >> 4) & 0x3fffu) | (1u << 16);
    for (int ks = 0; ks < k16; ++ks) {
      const uint32_t off16 = (uint32_t)(ks >> 2) * (16384u >> 4) + (uint32_t)(ks & 3) * 2u;
      tc_mma_words<true, false>(d_tmem, a_lo + off16, b_lo + off16, SMEM_DESC_HI_SBO1024, idesc,
                                (accumulate || ks > 0) ? 1u : 0u);
    }
  };
  // Everything the threads of both CTAs wrote (shared memory, tensor memory) becomes visible to the MMAs issued next.
  auto publish = [&]() {
    tc_wait_st();
    fence_async_smem();
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
  };
  auto await_mma = [&]() {
    if (ok) ok = mbar_wait(smem_u32(&mma_bar), phase, abort_flag, args.status, args.wait_limit_ns);
    phase ^= 1u;
    tc_fence_after();
  };

  const uint32_t p_begin = args.pair_start[pair], p_end = args.pair_start[pair + 1];
  for (uint32_t pi = p_begin; pi < p_end; ++pi) {
    const ChainProblem pr = args.problems[args.order[pi]];
    const int s = pr.s;
    // The pair's MMA is always 256 x 256 (each CTA supplies 128 rows of either operand; rows and columns past s are
    // zero in shared memory); only the contraction length follows s.
    const int k16 = (s + 15) >> 4;                      // contraction in steps of 16 columns
    const int chunks = (s + 31) >> 5;                   // 32-column chunks a thread walks over
    const uint32_t idesc = instr_desc(256, 256, 0, 0);
    const int grow = (int)rank * 128 + row;             // row of the s x s matrices this thread owns
    const bool live = grow < s;

    // ---- load -A_0/2 (hi/lo), form A_0 = -2 (hi + lo): A buffers <- split(A_0), D1 <- Z_1 = A_0 (F_1 = -A_0 / 2)
    for (int ch = cg; ch < chunks; ch += CHAIN_COLGROUPS) {
      float a[32];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int c0 = ch * 32 + q * 8;
        uint4 h = make_uint4(0, 0, 0, 0), l = make_uint4(0, 0, 0, 0);
        if (live && c0 < s) {                           // (ldq is a multiple of 8: whole units stay inside the row's pitch)
          h = *reinterpret_cast<const uint4*>(pr.q_hi + (int64_t)grow * pr.ldq + c0);
          l = *reinterpret_cast<const uint4*>(pr.q_lo + (int64_t)grow * pr.ldq + c0);
        }
        const uint32_t wh[4] = {h.x, h.y, h.z, h.w}, wl[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float v0 = -2.f * (__uint_as_float(wh[e] << 16) + __uint_as_float(wl[e] << 16));
          const float v1 = -2.f * (__uint_as_float(wh[e] & 0xffff0000u) + __uint_as_float(wl[e] & 0xffff0000u));
          a[q * 8 + 2 * e] = (c0 + 2 * e < s) ? v0 : 0.f;             // the pitch padding beyond column s is not data
          a[q * 8 + 2 * e + 1] = (c0 + 2 * e + 1 < s) ? v1 : 0.f;
        }
      }
      chain_store_row32(buf_ahi, buf_alo, row, ch, a);
      tc_st32(d1 + ch * 32, a);
    }

    float t = 1.f;                                      // t_k = (3/2)^k
    for (int k = 0; k < args.K; ++k) {
      const bool last = (k == args.K - 1);
      if (k > 0) {
        // X <- hi(F_k), F_k = -Z_k / 2;  D1 <- 3/2 Z_k + t_k A_k  (the MMA then adds A_k F_k: Z_{k+1})
        for (int ch = cg; ch < chunks; ch += CHAIN_COLGROUPS) {
          float z[32], a[32];
          tc_ld32(d1 + ch * 32, z);
          chain_load_row32(buf_ahi, buf_alo, row, ch, a);
          float f[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const bool in = live && (ch * 32 + j < s);  // columns past s may hold another problem's leftovers
            const float zj = in ? z[j] : 0.f;
            f[j] = -0.5f * zj;
            z[j] = fmaf(1.5f, zj, t * a[j]);
          }
          chain_store_row32(buf_x, 0u, row, ch, f);
          tc_st32(d1 + ch * 32, z);
        }
      }
      publish();
      if (rank == 0 && threadIdx.x == 0 && ok) {
        if (k > 0) issue_product(d1_mma, buf_ahi, buf_x, idesc, k16, true);          // Z_{k+1} = ... + A_k F_k
        if (!last) issue_product(d0_mma, buf_ahi, buf_ahi, idesc, k16, false);        // S = A_k A_k
        tc_commit_pair(smem_u32(&mma_bar));
      }
      await_mma();
      if (!last) {
        // X <- hi(S);  D0 <- 9 A_k - 6 S  (the MMA then adds A_k S: 4 A_{k+1})
        for (int ch = cg; ch < chunks; ch += CHAIN_COLGROUPS) {
          float sv[32], a[32];
          tc_ld32(d0 + ch * 32, sv);
          chain_load_row32(buf_ahi, buf_alo, row, ch, a);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const bool in = live && (ch * 32 + j < s);
            sv[j] = in ? sv[j] : 0.f;
            a[j] = fmaf(9.f, a[j], -6.f * sv[j]);
          }
          chain_store_row32(buf_x, 0u, row, ch, sv);
          tc_st32(d0 + ch * 32, a);
        }
        publish();
        if (rank == 0 && threadIdx.x == 0 && ok) {
          issue_product(d0_mma, buf_ahi, buf_x, idesc, k16, true);                    // 4 A_{k+1} = 9 A_k - 6 S + A_k S
          tc_commit_pair(smem_u32(&mma_bar));
        }
        await_mma();
        // A buffers <- split(A_{k+1})
        for (int ch = cg; ch < chunks; ch += CHAIN_COLGROUPS) {
          float v[32];
          tc_ld32(d0 + ch * 32, v);
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = (live && (ch * 32 + j < s)) ? 0.25f * v[j] : 0.f;
          chain_store_row32(buf_ahi, buf_alo, row, ch, v);
        }
      }
      t *= 1.5f;
    }

    // ---- F_K = -Z_K / 2 as a hi/lo pair, over the input (tensor-memory reads are warp-wide: every lane takes them)
    for (int ch = cg; ch < chunks; ch += CHAIN_COLGROUPS) {
      float z[32];
      tc_ld32(d1 + ch * 32, z);
      if (!(live && ok)) continue;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int c0 = ch * 32 + q * 8;
        if (c0 >= s) continue;
        uint32_t wh[4], wl[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float a = -0.5f * z[q * 8 + 2 * e], b = -0.5f * z[q * 8 + 2 * e + 1];
          wh[e] = pack_bf16x2(a, b);
          wl[e] = pack_bf16x2(a - __uint_as_float(wh[e] << 16), b - __uint_as_float(wh[e] & 0xffff0000u));
        }
        // (columns [s, ldq) of the last unit are pitch padding: writing them is harmless)
        *reinterpret_cast<uint4*>(pr.q_hi + (int64_t)grow * pr.ldq + c0) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
        *reinterpret_cast<uint4*>(pr.q_lo + (int64_t)grow * pr.ldq + c0) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
      }
    }
    // the next problem overwrites shared and tensor memory: every read of this one is complete in both CTAs
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
  }

  tc_fence_before();
  cluster_sync_all();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

}  // namespace signmuon
