// Shared device-side structures of the SignMuon step (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace signmuon {

typedef __nv_bfloat16 bf16;

// Device status word values (first word of the status area in the workspace).
enum : uint32_t { STATUS_OK = 0, STATUS_TIMEOUT = 1 };

// One entry per parameter block, uploaded when the caller's pointers change.
struct ParamDev {
  void* W;              // [rows][cols] weight_dtype, in/out
  const void* G;        // [M][rows][cols] grad_dtype
  float* mom;           // [M][rows*cols] float32 momentum (state buffer)
  bf16* y0;             // matrix params: Newton-Schulz operand buffer 0, [M][rows][ldy]
  bf16* y1;             // matrix params: operand buffer 1 (ping-pong partner)
  bf16* ylo;            // optional: receives bf16(Mom - bf16(Mom)), the lo part of the first operand (same layout
                        // as y0); set when the Newton-Schulz products run in split precision
  float* scales;        // matrix params: [M][2] = {1/max(sigma,eps)^2, 1/max(sigma,eps)}
  float* partials;      // matrix params: [M][chunks_per_worker] per-block sums of squares
  int64_t d;            // rows*cols
  int32_t rows, cols;
  int32_t ldy;          // row pitch of the bf16 operand buffers (cols rounded up to 8)
  int32_t kind, wdtype, gdtype;
  uint32_t word_off;    // first word of this parameter inside a worker's payload
  uint32_t n_words;     // ceil(d / 32)
  uint32_t chunks_per_worker;  // momentum-kernel blocks (= norm partials) per worker
  float upd_scale;      // 1, or 1/sqrt(rows*cols) for the Eq. 2 normalisation
  int32_t vec_ok;       // 16-byte vector path allowed (d % 8 == 0 and ldy == cols)
  uint8_t* sbar8;       // matrix params with the local polar step: the vote matrix once more as FP8 (E4M3) +-1 bytes,
                        // [rows][ld8]: operand of the step's first Gram product (null: not kept)
  int32_t ld8;          // row pitch of sbar8 in bytes (cols rounded up to 16)
  int32_t yk_buf;       // matrix params: which operand buffer (0: y0, 1: y1) holds Y_K after the last apply product
  int32_t avg_workers;  // > 1: the momentum takes the mean of this many workers' gradients (Muon rule), G is [avg][rows][cols]
  // power iteration (scale = spectral): un-normalised vectors and their norms
  float* pi_v;          // [M][cols]
  float* pi_u;          // [M][rows]
  float* pi_scal;       // [M][2] = {||v||, ||u||}
  const float* pi_start;// [M][cols] the caller's start vectors
};

// Epilogues of the Newton-Schulz products.
//
// The iterate is kept as a bf16 pair: `hi` = bf16(y) is the tensor-core operand, `lo` = bf16(y - hi)
// the remainder, so that the dominant term 1.5 * Y_k of  Y_{k+1} = 1.5 Y_k + (-A/2) Y_k  enters
// with ~16 mantissa bits while the product uses `hi` only.  An entry of Y_K near zero is the
// difference of its own term and the product term; carrying its own term in bf16 alone would
// decide such signs with a 2^-9 relative error of a term that is not small.
enum : int32_t {
  EPI_GRAM = 0,          // out = bf16(-0.5 * scale * acc)                      (the "-A/2" of 3I/2 - A/2)
  EPI_APPLY = 1,         // y = scale * (acc + own * C), own = 1.5; out = hi(y), out_lo = lo(y)   (Y_{k+1})
  EPI_APPLY_PACK = 2,    // sign bits of y -> payload words (hi(y) optionally stored)
  EPI_APPLY_UPDATE = 3   // W -= lr * y                                          (local polar step)
};

enum : int32_t {
  C_BF16 = 0,            // C = hi only (exact for the +-1 vote matrix)
  C_HILO = 1,            // C = hi + lo
  C_F32 = 2              // C = float32 momentum (first iteration)
};

// One product D[M x N] = A * B^T-like contraction over K with bf16 operands.
//   a(i,k) = A[i*a_sm + k*a_sk],  b(j,k) = B[j*b_sn + k*b_sk]   (element strides)
struct GemmProblem {
  const bf16* A;
  const bf16* B;
  int64_t a_sm, a_sk, b_sn, b_sk;
  int32_t M, N, K;
  int32_t tmapA, tmapB;   // indices into the tensor-map array (tensor-core kernel)
  int32_t batch;          // third TMA coordinate (worker slot)
  int32_t a_mn, b_mn;     // 1: operand is contiguous along M/N (not along K)
  int32_t epi;
  void* out;              // bf16 output (GRAM: -A/2; APPLY*: hi part of Y_{k+1})
  bf16* out_lo;           // APPLY: lo part of Y_{k+1} (same pitch as out)
  int64_t ld_out;
  const void* C;          // APPLY*: Y_k (bf16 hi, or float32 momentum when c_mode == C_F32)
  const bf16* C_lo;       // APPLY*: lo part of Y_k when c_mode == C_HILO
  int64_t ldc;
  const float* scale_ptr; // optional per-problem scale read from memory (else scale_imm)
  float scale_imm;
  int32_t c_mode;
  int32_t store_out;      // APPLY_PACK: also write hi(y)
  int32_t param;          // APPLY_UPDATE: index into the ParamDev table
  uint32_t* bits_out;     // APPLY_PACK: first payload word of this (param, worker)
  // TMA-staged epilogue (tensor-core kernel): tensor maps with {64 x 128} bf16 or {32 x 128} fp32 boxes
  int32_t tma_c, tma_out; // 1: C arrives / results leave through TMA, 0: direct global accesses
  int32_t tmapC0, tmapC1; // C hi (or fp32 momentum) and C lo
  int32_t tmapO0, tmapO1; // out hi and out lo
  int32_t batch_c, batch_o;
  // Gram products (tensor-core kernel): the result is symmetric, so only tiles on or above the diagonal are
  // scheduled and every off-diagonal tile is also written transposed through the {64 x 64}-box map tmapOT
  int32_t sym, tmapOT;
  // Split-precision products: up to three operand pairs (hi hi, lo hi, hi lo) accumulated into the same
  // tile, every segment contracting over the same K.
  int32_t nseg;           // 0 or 1: one pair
  int32_t tmapA2, tmapB2, tmapA3, tmapB3;
  float own_coef;         // APPLY*: coefficient of the own term, y = scale * (acc + own_coef * C): 1.5 for one Newton-Schulz
                          // step; 1.5^K when the product applies K steps at once (iteration carried out in Gram space)
  int32_t hi_only;        // EPI_APPLY: store hi(y) only (the lo buffer is still being read as an operand)
  int32_t fp8;            // operands are FP8 (E4M3) bytes: 128 elements per 128-byte row, tensor-core kind f8f6f4.  Used for
                          // the first Gram product of the local polar step, whose operand is the exact +-1 vote matrix
  int32_t gram_lo;        // EPI_GRAM: also store lo(-A/2) through tmapO1 (then the tile is not mirrored)
  int32_t diag_share;     // EPI_GRAM, one segment: on diagonal tiles the B operand is the A tile (not loaded twice)
  // Products of the Gram-space chain through memory (s x s, symmetric operands and results)
  int32_t mirror_hi;      // sym != 0: every off-diagonal tile also stores hi(result) transposed with plain stores (used
                          // where the transposed copy through tmapOT is not available: hi/lo outputs)
  const bf16* C2;         // EPI_APPLY: second linear term (hi part), same shape and pitch as the output, read with plain
  const bf16* C2_lo;      //            loads; y = scale * (acc + own_coef * C + c2_coef * (C2 + C2_lo))
  float c2_coef;
};

// Payload buffers of other GPUs that receive every payload word this GPU packs (the exchange of Alg. 3 fused into
// the pack: plain stores into peer-mapped memory instead of a separate all-gather).  All payload buffers share one
// layout, so a peer's copy of a word lives at the same offset: delta[p] = peer p's buffer - this GPU's buffer (bytes).
constexpr int MAX_PAYLOAD_PEERS = 7;
struct PeerList {
  int32_t n;
  int32_t reserved;
  int64_t delta[MAX_PAYLOAD_PEERS];
};
__device__ __forceinline__ void store_payload_word(uint32_t* own, uint32_t word, const PeerList& peers) {
  *own = word;
  for (int p = 0; p < peers.n; ++p)
    *reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(own) + peers.delta[p]) = word;
}

struct TileEntry {
  uint32_t problem;       // index relative to the launch's first problem
  uint16_t tm, tn;        // tile coordinates (units of 128 rows / BN columns)
};

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Stores NC floats as bf16 (hi) and optionally the bf16 remainders (lo) at row pointer offsets.
template <int NC>
__device__ __forceinline__ void store_hi_lo(bf16* o, bf16* olo, const float (&v)[NC], bool vec, int n_valid) {
  if (vec) {
#pragma unroll
    for (int q = 0; q < NC / 8; ++q) {
      uint32_t w[4], wl[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a = v[q * 8 + 2 * e], b = v[q * 8 + 2 * e + 1];
        w[e] = pack_bf16x2(a, b);
        wl[e] = pack_bf16x2(a - __uint_as_float(w[e] << 16), b - __uint_as_float(w[e] & 0xffff0000u));
      }
      reinterpret_cast<uint4*>(o)[q] = make_uint4(w[0], w[1], w[2], w[3]);
      if (olo) reinterpret_cast<uint4*>(olo)[q] = make_uint4(wl[0], wl[1], wl[2], wl[3]);
    }
  } else {
#pragma unroll
    for (int j = 0; j < NC; ++j) {
      if (j < n_valid) {
        const bf16 h = __float2bfloat16_rn(v[j]);
        o[j] = h;
        if (olo) olo[j] = __float2bfloat16_rn(v[j] - __bfloat162float(h));
      }
    }
  }
}

// ---- epilogue building blocks, each over 32 consecutive columns [col0, col0+32) of output row `row`;
// rows/columns outside the problem are skipped.

// v <- scale * (v + own * C) with C read directly from global memory (own = 1.5 for a Newton-Schulz step).
template <int NC = 32>
__device__ __forceinline__ void apply_c_direct(const GemmProblem& pr, float scale, int row, int col0, float* v) {
  if (row >= pr.M || col0 >= pr.N) return;
  const bool full = (col0 + NC <= pr.N);
  const int n_valid = full ? NC : pr.N - col0;
  const float own = pr.own_coef;
  if (pr.c_mode == C_F32) {
    const float* c = reinterpret_cast<const float*>(pr.C) + (int64_t)row * pr.ldc + col0;
    if (full && ((pr.ldc & 3) == 0)) {
      const float4* c4 = reinterpret_cast<const float4*>(c);
#pragma unroll
      for (int q = 0; q < NC / 4; ++q) {
        const float4 t = __ldg(c4 + q);
        v[4 * q] = scale * fmaf(own, t.x, v[4 * q]);
        v[4 * q + 1] = scale * fmaf(own, t.y, v[4 * q + 1]);
        v[4 * q + 2] = scale * fmaf(own, t.z, v[4 * q + 2]);
        v[4 * q + 3] = scale * fmaf(own, t.w, v[4 * q + 3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC; ++j) v[j] = (j < n_valid) ? scale * fmaf(own, __ldg(c + j), v[j]) : 0.f;
    }
  } else {
    const bf16* c = reinterpret_cast<const bf16*>(pr.C) + (int64_t)row * pr.ldc + col0;
    const bf16* cl = pr.c_mode == C_HILO ? pr.C_lo + (int64_t)row * pr.ldc + col0 : nullptr;
    if (full && ((pr.ldc & 7) == 0)) {
#pragma unroll
      for (int q = 0; q < NC / 8; ++q) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(c) + q);
        uint4 u = make_uint4(0, 0, 0, 0);
        if (cl) u = *(reinterpret_cast<const uint4*>(cl) + q);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
        const uint32_t wl[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float c0 = __uint_as_float(w[e] << 16) + __uint_as_float(wl[e] << 16);
          const float c1 = __uint_as_float(w[e] & 0xffff0000u) + __uint_as_float(wl[e] & 0xffff0000u);
          v[q * 8 + 2 * e] = scale * fmaf(own, c0, v[q * 8 + 2 * e]);
          v[q * 8 + 2 * e + 1] = scale * fmaf(own, c1, v[q * 8 + 2 * e + 1]);
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC; ++j) {
        float cv = 0.f;
        if (j < n_valid) cv = __bfloat162float(c[j]) + (cl ? __bfloat162float(cl[j]) : 0.f);
        v[j] = (j < n_valid) ? scale * fmaf(own, cv, v[j]) : 0.f;
      }
    }
  }
}

// out <- hi(v) (and out_lo <- lo(v)) written directly to global memory.
template <int NC = 32>
__device__ __forceinline__ void store_out_direct(const GemmProblem& pr, int row, int col0, const float* v, bool with_lo) {
  if (row >= pr.M || col0 >= pr.N) return;
  const bool full = (col0 + NC <= pr.N);
  const int n_valid = full ? NC : pr.N - col0;
  bf16* o = reinterpret_cast<bf16*>(pr.out) + (int64_t)row * pr.ld_out + col0;
  bf16* ol = (with_lo && pr.out_lo) ? pr.out_lo + (int64_t)row * pr.ld_out + col0 : nullptr;
  const float(&vv)[NC] = *reinterpret_cast<const float(*)[NC]>(v);
  store_hi_lo<NC>(o, ol, vv, full && ((pr.ld_out & 7) == 0), n_valid);
}

// One payload word from 32 consecutive columns (only issued for parameters with cols % 32 == 0).
__device__ __forceinline__ void pack_bits_direct(const GemmProblem& pr, int row, int col0, const float* v,
                                                 const PeerList& peers) {
  if (row >= pr.M || col0 + 32 > pr.N) return;
  uint32_t word = 0;
#pragma unroll
  for (int j = 0; j < 32; ++j) word |= (v[j] >= 0.f ? 1u : 0u) << j;
  store_payload_word(pr.bits_out + (((int64_t)row * pr.N + col0) >> 5), word, peers);
}
// Half a payload word from 16 consecutive columns (col0 a multiple of 16; little-endian words: the lower
// columns are the lower half).
__device__ __forceinline__ void pack_bits16_direct(const GemmProblem& pr, int row, int col0, const float* v,
                                                   const PeerList& peers) {
  if (row >= pr.M || col0 + 16 > pr.N) return;
  uint32_t half = 0;
#pragma unroll
  for (int j = 0; j < 16; ++j) half |= (v[j] >= 0.f ? 1u : 0u) << j;
  uint16_t* own = reinterpret_cast<uint16_t*>(pr.bits_out) + (((int64_t)row * pr.N + col0) >> 4);
  *own = (uint16_t)half;
  for (int p = 0; p < peers.n; ++p)
    *reinterpret_cast<uint16_t*>(reinterpret_cast<char*>(own) + peers.delta[p]) = (uint16_t)half;
}

// W <- W - lr * v (local polar step's last epilogue).
template <int NC = 32>
__device__ __forceinline__ void update_weights_direct(const GemmProblem& pr, const ParamDev* params, float lr, int row,
                                                      int col0, const float* v) {
  if (row >= pr.M || col0 >= pr.N) return;
  const bool full = (col0 + NC <= pr.N);
  const int n_valid = full ? NC : pr.N - col0;
  const ParamDev& pd = params[pr.param];
  if (pd.wdtype == 0) {
    float* w = reinterpret_cast<float*>(pd.W) + (int64_t)row * pr.N + col0;
    if (full && ((pr.N & 3) == 0)) {
      float4* w4 = reinterpret_cast<float4*>(w);
#pragma unroll
      for (int q = 0; q < NC / 4; ++q) {
        float4 t = w4[q];
        t.x = fmaf(-lr, v[4 * q], t.x);
        t.y = fmaf(-lr, v[4 * q + 1], t.y);
        t.z = fmaf(-lr, v[4 * q + 2], t.z);
        t.w = fmaf(-lr, v[4 * q + 3], t.w);
        w4[q] = t;
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC; ++j)
        if (j < n_valid) w[j] = fmaf(-lr, v[j], w[j]);
    }
  } else {
    bf16* w = reinterpret_cast<bf16*>(pd.W) + (int64_t)row * pr.N + col0;
    if (full && ((pr.N & 7) == 0)) {
      uint4* w4 = reinterpret_cast<uint4*>(w);
#pragma unroll
      for (int q = 0; q < NC / 8; ++q) {
        const uint4 t = w4[q];
        const uint32_t in[4] = {t.x, t.y, t.z, t.w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          o[e] = pack_bf16x2(fmaf(-lr, v[q * 8 + 2 * e], __uint_as_float(in[e] << 16)),
                             fmaf(-lr, v[q * 8 + 2 * e + 1], __uint_as_float(in[e] & 0xffff0000u)));
        w4[q] = make_uint4(o[0], o[1], o[2], o[3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC; ++j)
        if (j < n_valid) w[j] = __float2bfloat16_rn(fmaf(-lr, v[j], __bfloat162float(w[j])));
    }
  }
}

// Whole epilogue of 32 columns with direct global accesses (diagnostic kernel and ragged fallbacks).
__device__ __forceinline__ void epilogue_row32(const GemmProblem& pr, const ParamDev* params, float lr,
                                               int row, int col0, float (&v)[32], const PeerList& peers) {
  if (row >= pr.M || col0 >= pr.N) return;
  const float scale = pr.scale_ptr ? __ldg(pr.scale_ptr) : pr.scale_imm;
  if (pr.epi == EPI_GRAM) {
    const float f = -0.5f * scale;
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] *= f;
    store_out_direct(pr, row, col0, v, false);
    return;
  }
  apply_c_direct(pr, scale, row, col0, v);
  if (pr.epi == EPI_APPLY || (pr.epi == EPI_APPLY_PACK && pr.store_out))
    store_out_direct(pr, row, col0, v, pr.epi == EPI_APPLY && pr.hi_only == 0);
  if (pr.epi == EPI_APPLY_PACK) pack_bits_direct(pr, row, col0, v, peers);
  else if (pr.epi == EPI_APPLY_UPDATE) update_weights_direct(pr, params, lr, row, col0, v);
}

}  // namespace signmuon
