// Memory-bound kernels of the SignMuon step: momentum (+ Frobenius norm + bf16 operand),
// fused plain-parameter update, stand-alone sign pack, and majority vote + weight update.
#pragma once

#include "common.cuh"

namespace signmuon {

constexpr int EW_THREADS = 256;
constexpr int MOM_CHUNK = 8192;        // entries per block of the momentum kernel (256 threads x 8 x 4)
constexpr int PLAIN_CHUNK = 2048;      // entries per block of the plain-parameter kernel (8 warps x 256)
constexpr int VOTE_THREADS = 128;      // vote kernel: 4 warps per block, 4 consecutive payload words per thread (128-bit loads)
constexpr int PACK_CHUNK = 1024;       // entries per block of the stand-alone pack kernel (small: it only sees small, ragged matrices)

// Finds the list slot whose block range contains `block` (`starts` is ascending, one entry per slot).
__device__ __forceinline__ int find_slot(const uint32_t* __restrict__ starts, int n, uint32_t block) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (__ldg(starts + mid) <= block) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

template <typename T> __device__ __forceinline__ float load_as_float(const T* p);
template <> __device__ __forceinline__ float load_as_float<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_as_float<bf16>(const bf16* p) {
  return __bfloat162float(*p);
}

// Loads 8 consecutive elements (16-byte aligned for bf16, 32-byte span for float) as floats.
__device__ __forceinline__ void load8(const float* p, float (&x)[8]) {
  const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void load8(const bf16* p, float (&x)[8]) {
  const uint4 a = __ldcs(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    x[2 * e] = __uint_as_float(w[e] << 16);
    x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
  }
}

// ---------------------------------------------------------------------------------------------
// Momentum of the matrix parameters (Alg. 2: weight decay + momentum; Alg. 4: ||Mom||_F):
//   Mom <- beta Mom + (1-beta)(G + lambda W);  Y0 = bf16(Mom);  partial[block] = sum Mom^2.
// Grid: one block per MOM_CHUNK entries of one (parameter, worker).
// ---------------------------------------------------------------------------------------------
template <typename GT, typename WT>
__device__ __forceinline__ void momentum_block(const ParamDev& pd, int m, uint32_t chunk, float beta,
                                               float lambda, float& sumsq) {
  const int64_t d = pd.d;
  const GT* g = reinterpret_cast<const GT*>(pd.G) + (int64_t)m * d;
  const WT* w = reinterpret_cast<const WT*>(pd.W);
  float* mom = pd.mom + (int64_t)m * d;
  bf16* y = pd.y0 + (int64_t)m * pd.rows * pd.ldy;
  bf16* ylo = pd.ylo ? pd.ylo + (int64_t)m * pd.rows * pd.ldy : nullptr;
  const int64_t base = (int64_t)chunk * MOM_CHUNK;
  const float omb = 1.f - beta;
  const int avg = pd.avg_workers;                 // > 1: mean gradient of that many workers (m is 0 then)
  const float inv_avg = 1.f / (float)(avg > 1 ? avg : 1);
  if (pd.vec_ok) {
#pragma unroll
    for (int it = 0; it < MOM_CHUNK / (EW_THREADS * 8); ++it) {
      const int64_t i = base + ((int64_t)it * EW_THREADS + threadIdx.x) * 8;
      if (i < d) {   // d % 8 == 0 on this path
        float gv[8], mv[8];
        load8(g + i, gv);
        load8(mom + i, mv);
        if (avg > 1) {
          for (int k = 1; k < avg; ++k) {
            float t[8];
            load8(g + (int64_t)k * d + i, t);
#pragma unroll
            for (int e = 0; e < 8; ++e) gv[e] += t[e];
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) gv[e] *= inv_avg;
        }
        if (lambda != 0.f) {
          float wv[8];
          load8(w + i, wv);
#pragma unroll
          for (int e = 0; e < 8; ++e) gv[e] = fmaf(lambda, wv[e], gv[e]);
        }
        uint32_t packed[4];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          mv[e] = fmaf(beta, mv[e], omb * gv[e]);
          sumsq = fmaf(mv[e], mv[e], sumsq);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __nv_bfloat162 h = __floats2bfloat162_rn(mv[2 * e], mv[2 * e + 1]);
          packed[e] = *reinterpret_cast<uint32_t*>(&h);
        }
        float4* mo = reinterpret_cast<float4*>(mom + i);
        mo[0] = make_float4(mv[0], mv[1], mv[2], mv[3]);
        mo[1] = make_float4(mv[4], mv[5], mv[6], mv[7]);
        *reinterpret_cast<uint4*>(y + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        if (ylo) {
          uint32_t lo[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            lo[e] = pack_bf16x2(mv[2 * e] - __uint_as_float(packed[e] << 16),
                                mv[2 * e + 1] - __uint_as_float(packed[e] & 0xffff0000u));
          *reinterpret_cast<uint4*>(ylo + i) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
    }
  } else {
    const int64_t end = (base + MOM_CHUNK < d) ? base + MOM_CHUNK : d;
    for (int64_t i = base + threadIdx.x; i < end; i += EW_THREADS) {
      float gv = load_as_float<GT>(g + i);
      if (avg > 1) {
        for (int k = 1; k < avg; ++k) gv += load_as_float<GT>(g + (int64_t)k * d + i);
        gv *= inv_avg;
      }
      if (lambda != 0.f) gv = fmaf(lambda, load_as_float<WT>(w + i), gv);
      const float mv = fmaf(beta, mom[i], omb * gv);
      mom[i] = mv;
      sumsq = fmaf(mv, mv, sumsq);
      const int64_t r = i / pd.cols;
      const int64_t c = i - r * pd.cols;
      const bf16 h = __float2bfloat16_rn(mv);
      y[r * pd.ldy + c] = h;
      if (ylo) ylo[r * pd.ldy + c] = __float2bfloat16_rn(mv - __bfloat162float(h));
    }
  }
}

__global__ void __launch_bounds__(EW_THREADS) momentum_kernel(const ParamDev* __restrict__ params,
                                                              const int32_t* __restrict__ list,
                                                              const uint32_t* __restrict__ starts, int n_list,
                                                              float beta, float lambda) {
  const int slot = find_slot(starts, n_list, blockIdx.x);
  const ParamDev pd = params[list[slot]];
  const uint32_t local = blockIdx.x - starts[slot];
  const int m = local / pd.chunks_per_worker;
  const uint32_t chunk = local - m * pd.chunks_per_worker;
  float sumsq = 0.f;
  if (pd.gdtype == 0) {
    if (pd.wdtype == 0) momentum_block<float, float>(pd, m, chunk, beta, lambda, sumsq);
    else momentum_block<float, bf16>(pd, m, chunk, beta, lambda, sumsq);
  } else {
    if (pd.wdtype == 0) momentum_block<bf16, float>(pd, m, chunk, beta, lambda, sumsq);
    else momentum_block<bf16, bf16>(pd, m, chunk, beta, lambda, sumsq);
  }
  __shared__ float red[EW_THREADS / 32];
  sumsq = warp_sum(sumsq);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sumsq;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < EW_THREADS / 32; ++i) t += red[i];
    pd.partials[(int64_t)m * pd.chunks_per_worker + chunk] = t;
  }
}

// One warp per (matrix parameter, worker): fixed-order sum of the block partials in double,
// then the two scale factors the Newton-Schulz epilogues use.
__global__ void finalize_norms_kernel(const ParamDev* __restrict__ params, const int32_t* __restrict__ list,
                                      int n_list, int num_workers, float eps) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= n_list * num_workers) return;
  const ParamDev& pd = params[list[warp / num_workers]];
  const int m = warp % num_workers;
  const float* part = pd.partials + (int64_t)m * pd.chunks_per_worker;
  double acc = 0.0;
  for (uint32_t i = lane; i < pd.chunks_per_worker; i += 32) acc += (double)part[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const double sigma = fmax(sqrt(acc), (double)eps);
    pd.scales[2 * m] = (float)(1.0 / (sigma * sigma));
    pd.scales[2 * m + 1] = (float)(1.0 / sigma);
  }
}

// ---------------------------------------------------------------------------------------------
// Plain parameters: the whole step in one pass (no Newton-Schulz): momentum of every worker,
// bit = (Mom >= 0), ballot-packed payload words, majority vote in registers, weight update.
// Each warp owns 128 consecutive entries; lane l holds entries base + 32 k + l, k = 0..3, so that
// one __ballot_sync per (worker, k) yields one payload word.
// ---------------------------------------------------------------------------------------------
// Stores 8 consecutive elements.
__device__ __forceinline__ void store8(float* p, const float (&x)[8]) {
  __stcs(reinterpret_cast<float4*>(p), make_float4(x[0], x[1], x[2], x[3]));
  __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(x[4], x[5], x[6], x[7]));
}
__device__ __forceinline__ void store8(bf16* p, const float (&x)[8]) {
  __stcs(reinterpret_cast<uint4*>(p), make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]),
                                                 pack_bf16x2(x[4], x[5]), pack_bf16x2(x[6], x[7])));
}

// Vector form of the plain-parameter step for a warp whose 256 entries are all inside the parameter and
// 16-byte aligned: lane l owns entries base + 8 l .. + 7 (128-bit accesses), its 8 sign bits form one byte
// and four neighbouring lanes' bytes one payload word (OR within the 4-lane group).  Two workers are in
// flight at a time so that a lane keeps 6 vector loads outstanding.
template <typename GT, typename WT>
__device__ __forceinline__ void plain_warp_vec(const ParamDev& pd, int64_t base, int M, float beta, float lambda,
                                               float step, uint32_t* __restrict__ bits,
                                               uint32_t* __restrict__ vote_words, int64_t bits_pitch, int do_vote,
                                               const PeerList& peers) {
  const int lane = threadIdx.x & 31;
  const int64_t d = pd.d;
  const int64_t i0 = base + 8 * lane;
  const GT* __restrict__ g = reinterpret_cast<const GT*>(pd.G) + i0;
  float* __restrict__ mom = pd.mom + i0;
  WT* w = reinterpret_cast<WT*>(pd.W) + i0;
  const float omb = 1.f - beta;
  const unsigned group = 0xfu << (lane & ~3);            // this lane's 4-lane group
  const int shift = (lane & 3) * 8;
  const int64_t word = (base >> 5) + (lane >> 2);        // the payload word this group builds
  uint32_t* out = bits + pd.word_off + word;
  float wv[8];
  load8(w, wv);
  int count[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) count[e] = 0;
  auto finish = [&](float (&gv)[8], float (&mv)[8], int m) {
    uint32_t byte = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      mv[e] = fmaf(beta, mv[e], omb * fmaf(lambda, wv[e], gv[e]));
      const bool b = mv[e] >= 0.f;
      count[e] += b ? 1 : 0;
      byte |= (b ? 1u : 0u) << e;
    }
    store8(mom + (int64_t)m * d, mv);
    const uint32_t wordv = __reduce_or_sync(group, byte << shift);
    if ((lane & 3) == 0) store_payload_word(out + (int64_t)m * bits_pitch, wordv, peers);
  };
  int m = 0;
  for (; m + 1 < M; m += 2) {
    float g0[8], m0[8], g1[8], m1[8];
    load8(g + (int64_t)m * d, g0);
    load8(mom + (int64_t)m * d, m0);
    load8(g + (int64_t)(m + 1) * d, g1);
    load8(mom + (int64_t)(m + 1) * d, m1);
    finish(g0, m0, m);
    finish(g1, m1, m + 1);
  }
  if (m < M) {
    float g0[8], m0[8];
    load8(g + (int64_t)m * d, g0);
    load8(mom + (int64_t)m * d, m0);
    finish(g0, m0, m);
  }
  if (!do_vote) return;      // the workers of this pass are a subset: vote and update follow the payload exchange
  uint32_t vbyte = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const bool plus = 2 * count[e] >= M;
    vbyte |= (plus ? 1u : 0u) << e;
    wv[e] -= plus ? step : -step;
  }
  store8(w, wv);
  const uint32_t vword = __reduce_or_sync(group, vbyte << shift);
  if ((lane & 3) == 0) vote_words[pd.word_off + word] = vword;
}

template <typename GT, typename WT>
__device__ __forceinline__ void plain_warp_scalar(const ParamDev& pd, int64_t base, int M, float beta, float lambda,
                                                  float step, uint32_t* __restrict__ bits,
                                                  uint32_t* __restrict__ vote_words, int64_t bits_pitch, int do_vote,
                                                  const PeerList& peers);

template <typename GT, typename WT>
__device__ __forceinline__ void plain_block(const ParamDev& pd, uint32_t chunk, int M, float beta,
                                            float lambda, float step, uint32_t* __restrict__ bits,
                                            uint32_t* __restrict__ vote_words, int64_t bits_pitch, int do_vote,
                                            const PeerList& peers) {
  const int warp = threadIdx.x >> 5;
  const int64_t d = pd.d;
  if ((d & 7) == 0 && (int64_t)chunk * PLAIN_CHUNK + (warp + 1) * 256 <= d) {
    plain_warp_vec<GT, WT>(pd, (int64_t)chunk * PLAIN_CHUNK + warp * 256, M, beta, lambda, step, bits, vote_words,
                           bits_pitch, do_vote, peers);
    return;
  }
  // ragged tail (or an unaligned parameter): the warp's 256 entries as two scalar passes of 128
  for (int pass = 0; pass < 2; ++pass)
    plain_warp_scalar<GT, WT>(pd, (int64_t)chunk * PLAIN_CHUNK + warp * 256 + pass * 128, M, beta, lambda, step, bits,
                              vote_words, bits_pitch, do_vote, peers);
}

template <typename GT, typename WT>
__device__ __forceinline__ void plain_warp_scalar(const ParamDev& pd, int64_t base, int M, float beta,
                                                  float lambda, float step, uint32_t* __restrict__ bits,
                                                  uint32_t* __restrict__ vote_words, int64_t bits_pitch, int do_vote,
                                                  const PeerList& peers) {
  const int lane = threadIdx.x & 31;
  const int64_t d = pd.d;
  if (base >= d) return;
  const GT* g = reinterpret_cast<const GT*>(pd.G);
  WT* w = reinterpret_cast<WT*>(pd.W);
  const float omb = 1.f - beta;
  int count[4] = {0, 0, 0, 0};
  float wv[4];
  bool valid[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int64_t i = base + 32 * k + lane;
    valid[k] = i < d;
    wv[k] = valid[k] ? load_as_float<WT>(w + i) : 0.f;
  }
  const int64_t word0 = base >> 5;
  for (int m = 0; m < M; ++m) {
    const GT* gm = g + (int64_t)m * d;
    float* mm = pd.mom + (int64_t)m * d;
    float mv[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int64_t i = base + 32 * k + lane;
      float gv = valid[k] ? load_as_float<GT>(gm + i) : 0.f;
      float old = valid[k] ? __ldcs(mm + i) : 0.f;
      gv = fmaf(lambda, wv[k], gv);
      mv[k] = fmaf(beta, old, omb * gv);
    }
    uint32_t mine = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int64_t i = base + 32 * k + lane;
      if (valid[k]) __stcs(mm + i, mv[k]);
      const bool b = valid[k] && (mv[k] >= 0.f);
      count[k] += b ? 1 : 0;
      const uint32_t word = __ballot_sync(0xffffffffu, b);
      if (lane == k) mine = word;
    }
    if (lane < 4 && word0 + lane < pd.n_words)
      store_payload_word(bits + (int64_t)m * bits_pitch + pd.word_off + word0 + lane, mine, peers);
  }
  if (!do_vote) return;
  uint32_t vmine = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int64_t i = base + 32 * k + lane;
    const bool plus = valid[k] && (2 * count[k] >= M);
    const uint32_t word = __ballot_sync(0xffffffffu, plus);
    if (lane == k) vmine = word;
    if (valid[k]) {
      const float nw = wv[k] - (plus ? step : -step);
      if (sizeof(WT) == 4) reinterpret_cast<float*>(w)[i] = nw;
      else reinterpret_cast<bf16*>(w)[i] = __float2bfloat16_rn(nw);
    }
  }
  if (lane < 4 && word0 + lane < pd.n_words) vote_words[pd.word_off + word0 + lane] = vmine;
}

__global__ void __launch_bounds__(EW_THREADS) plain_params_kernel(const ParamDev* __restrict__ params,
                                                                  const int32_t* __restrict__ list,
                                                                  const uint32_t* __restrict__ starts, int n_list,
                                                                  int M, float beta, float lambda, float lr,
                                                                  uint32_t* __restrict__ bits,
                                                                  uint32_t* __restrict__ vote_words,
                                                                  int64_t bits_pitch, int do_vote,
                                                                  const __grid_constant__ PeerList peers) {
  const int slot = find_slot(starts, n_list, blockIdx.x);
  const ParamDev pd = params[list[slot]];
  const uint32_t chunk = blockIdx.x - starts[slot];
  const float step = lr * pd.upd_scale;
  if (pd.gdtype == 0) {
    if (pd.wdtype == 0) plain_block<float, float>(pd, chunk, M, beta, lambda, step, bits, vote_words, bits_pitch, do_vote, peers);
    else plain_block<float, bf16>(pd, chunk, M, beta, lambda, step, bits, vote_words, bits_pitch, do_vote, peers);
  } else {
    if (pd.wdtype == 0) plain_block<bf16, float>(pd, chunk, M, beta, lambda, step, bits, vote_words, bits_pitch, do_vote, peers);
    else plain_block<bf16, bf16>(pd, chunk, M, beta, lambda, step, bits, vote_words, bits_pitch, do_vote, peers);
  }
}

// ---------------------------------------------------------------------------------------------
// Stand-alone sign + pack (Alg. 3 "PackBits") for matrix parameters whose rows do not hold whole
// payload words (cols % 32 != 0), and for K = 0.  Source: bf16 Y_K [M][rows][ldy] in the operand buffer the
// parameter's last apply product wrote, or for K = 0 the float32 momentum itself.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS) pack_kernel(const ParamDev* __restrict__ params,
                                                          const int32_t* __restrict__ list,
                                                          const uint32_t* __restrict__ starts, int n_list,
                                                          int from_momentum,
                                                          uint32_t* __restrict__ bits, int64_t bits_pitch,
                                                          const __grid_constant__ PeerList peers) {
  const int slot = find_slot(starts, n_list, blockIdx.x);
  const ParamDev pd = params[list[slot]];
  const uint32_t local = blockIdx.x - starts[slot];
  const uint32_t cpw = (uint32_t)((pd.d + PACK_CHUNK - 1) / PACK_CHUNK);
  const int m = local / cpw;
  const uint32_t chunk = local - m * cpw;
  const int lane = threadIdx.x & 31;
  const bf16* y = (pd.yk_buf ? pd.y1 : pd.y0) + (int64_t)m * pd.rows * pd.ldy;   // where this parameter's Y_K was left
  const float* mom = pd.mom + (int64_t)m * pd.d;
  const int64_t base = (int64_t)chunk * PACK_CHUNK;
#pragma unroll 4
  for (int it = 0; it < PACK_CHUNK / EW_THREADS; ++it) {
    const int64_t i = base + (int64_t)it * EW_THREADS + threadIdx.x;
    bool b = false;
    if (i < pd.d) {
      if (from_momentum) {
        b = mom[i] >= 0.f;
      } else {
        const int64_t r = i / pd.cols;
        const int64_t c = i - r * pd.cols;
        b = __bfloat162float(y[r * pd.ldy + c]) >= 0.f;
      }
    }
    const uint32_t word = __ballot_sync(0xffffffffu, b);
    const int64_t wi = i >> 5;
    if (lane == 0 && wi < pd.n_words) store_payload_word(bits + (int64_t)m * bits_pitch + pd.word_off + wi, word, peers);
  }
}

// ---------------------------------------------------------------------------------------------
// Majority vote from the packed words (App. B: c = sum_m b^(m), S = sign(2c - M), ties -> +1) and
// the weight update W <- W - eta S (Alg. 3), or, for the local polar step, S as a bf16 +-1 matrix.
//
// Two streaming kernels.  vote_kernel reads the payload (the workers' rows are 128-byte aligned in the workspace, so
// a lane reads four consecutive words of a worker as one 128-bit load, eight rows in flight) and writes the vote
// words; the 32 per-position counts of a word are kept as bit-sliced counter planes (about three logic operations
// per worker word instead of 32 unpacks) and the comparison c >= ceil(M/2) is the carry out of a bit-sliced addition
// of 2^PLANES - ceil(M/2).  update_kernel reads the vote words back (1/8 byte per entry, from L2) and moves the weights
// (or the +-1 matrix) as 128-bit vectors, eight per thread in flight.  Split this way each kernel keeps few registers
// per byte in flight; one fused kernel held both the payload rows and the weight vectors and ran at lower occupancy.
// ---------------------------------------------------------------------------------------------
template <int PLANES>
struct VoteCounter {
  uint32_t c[PLANES];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int b = 0; b < PLANES; ++b) c[b] = 0;
  }
  __device__ __forceinline__ void add(uint32_t carry) {
#pragma unroll
    for (int b = 0; b < PLANES; ++b) {
      const uint32_t t = c[b] & carry;
      c[b] ^= carry;
      carry = t;
    }
  }
  // bit set <=> count >= ceil(M/2) <=> 2c - M >= 0
  __device__ __forceinline__ uint32_t majority(int M) const {
    const uint32_t add = (1u << PLANES) - (uint32_t)((M + 1) >> 1);
    uint32_t carry = 0;
#pragma unroll
    for (int b = 0; b < PLANES; ++b) {
      const uint32_t kb = ((add >> b) & 1u) ? 0xffffffffu : 0u;
      carry = (c[b] & kb) | (carry & (c[b] ^ kb));
    }
    return carry;
  }
};

// vote_kernel: payload rows -> vote words, over a few contiguous word ranges of the payload (the matrix parameters'
// words; everything when the plain parameters are voted here too).  The vote of a bit position does not depend on
// the parameter it belongs to, so the kernel needs no parameter table: a thread owns four consecutive words of the
// concatenated ranges.  Range bounds are multiples of four words (rounded outwards by the host: a few neighbouring
// words of a plain parameter or pad words may be voted again, with the same result).
constexpr int MAX_VOTE_RANGES = 8;
struct VoteRanges {
  int32_t n;
  int32_t reserved;
  int64_t begin[MAX_VOTE_RANGES];     // first word of the range
  int64_t quads_before[MAX_VOTE_RANGES + 1];   // four-word groups in the ranges before this one; [n] = total
};
template <int PLANES>
__global__ void __launch_bounds__(VOTE_THREADS) vote_kernel(const __grid_constant__ VoteRanges ranges, int M,
                                                            const uint32_t* __restrict__ bits,
                                                            uint32_t* __restrict__ vote_words, int64_t bits_pitch) {
  constexpr int ROWS = 8;                               // worker rows in flight per lane
  // the update kernel that follows may start its prologue (and request its weights) while this grid still runs
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t q = (int64_t)blockIdx.x * VOTE_THREADS + threadIdx.x;
  if (q >= ranges.quads_before[ranges.n]) return;
  int r = 0;
#pragma unroll
  for (int i = 1; i < MAX_VOTE_RANGES; ++i)
    if (i < ranges.n && q >= ranges.quads_before[i]) r = i;
  const int64_t g = ranges.begin[r] + 4 * (q - ranges.quads_before[r]);
  VoteCounter<PLANES> cnt[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) cnt[j].clear();
  const uint32_t* col = bits + g;
  int m = 0;
  for (; m + ROWS <= M; m += ROWS) {
    uint4 v[ROWS];
#pragma unroll
    for (int k = 0; k < ROWS; ++k) v[k] = __ldcs(reinterpret_cast<const uint4*>(col + (int64_t)(m + k) * bits_pitch));
#pragma unroll
    for (int k = 0; k < ROWS; ++k) { cnt[0].add(v[k].x); cnt[1].add(v[k].y); cnt[2].add(v[k].z); cnt[3].add(v[k].w); }
  }
  if (m + 4 <= M) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = __ldcs(reinterpret_cast<const uint4*>(col + (int64_t)(m + k) * bits_pitch));
#pragma unroll
    for (int k = 0; k < 4; ++k) { cnt[0].add(v[k].x); cnt[1].add(v[k].y); cnt[2].add(v[k].z); cnt[3].add(v[k].w); }
    m += 4;
  }
  for (; m < M; ++m) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(col + (int64_t)m * bits_pitch));
    cnt[0].add(v.x); cnt[1].add(v.y); cnt[2].add(v.z); cnt[3].add(v.w);
  }
  *reinterpret_cast<uint4*>(vote_words + g) =
      make_uint4(cnt[0].majority(M), cnt[1].majority(M), cnt[2].majority(M), cnt[3].majority(M));
}

// update_kernel: vote words -> W <- W - eta S (Alg. 3 "Update parameters"), or S as a bf16 +-1 matrix in the local
// polar step's operand slot.  A block owns UPD_VECS 128-bit vectors of one parameter (4 float32 or 8 bf16 entries
// each, all inside one vote word), a thread eight of them, all requested before the first is used.
constexpr int UPD_VECS = EW_THREADS * 8;
// (SBAR is a template parameter so that the plain weight update does not carry the registers of the +-1 matrix stores.)
template <typename WT, bool SBAR>
__device__ __forceinline__ void update_block(const ParamDev& pd, uint32_t chunk, int lp_slot, float step,
                                             const uint32_t* __restrict__ vote_words) {
  constexpr bool write_sbar = SBAR;
  const int64_t d = pd.d;
  WT* w = reinterpret_cast<WT*>(pd.W);
  bf16* sbar = pd.y0 + (int64_t)lp_slot * pd.rows * pd.ldy;   // the slot after the own workers' slots of operand buffer 0
  const uint32_t* vw = vote_words + pd.word_off;
  const bool vec = write_sbar ? (pd.vec_ok != 0) : ((d & 7) == 0);
  const int epv = (write_sbar || sizeof(WT) == 2) ? 8 : 4;
  if (vec) {
    uint4* vbase = write_sbar ? reinterpret_cast<uint4*>(sbar) : reinterpret_cast<uint4*>(w);
    const int64_t n_vec = d / epv;
    const int64_t i0 = (int64_t)chunk * UPD_VECS + threadIdx.x;
    uint4 x[8];
    uint32_t vword[8];
    if (!write_sbar) {
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int64_t i = i0 + it * EW_THREADS;
        if (i < n_vec) x[it] = __ldcs(vbase + i);
      }
    }
    // the vote words come from the grid launched just before this one, which may still be running
    asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int64_t i = i0 + it * EW_THREADS;
      if (i < n_vec) vword[it] = __ldcg(vw + ((i * epv) >> 5));
    }
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int64_t i = i0 + it * EW_THREADS;
      if (i >= n_vec) continue;
      uint4 o;
      if (!write_sbar && sizeof(WT) == 4) {             // 4 float32: a nibble of the vote word
        const uint32_t b4 = vword[it] >> ((i & 7) * 4);
        o.x = __float_as_uint(__uint_as_float(x[it].x) - ((b4 & 1u) ? step : -step));
        o.y = __float_as_uint(__uint_as_float(x[it].y) - ((b4 & 2u) ? step : -step));
        o.z = __float_as_uint(__uint_as_float(x[it].z) - ((b4 & 4u) ? step : -step));
        o.w = __float_as_uint(__uint_as_float(x[it].w) - ((b4 & 8u) ? step : -step));
      } else {                                          // 8 bf16: a byte of the vote word
        const uint32_t b8 = vword[it] >> ((i & 3) * 8);
        const uint32_t in[4] = {x[it].x, x[it].y, x[it].z, x[it].w};
        uint32_t ov[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool p0 = (b8 >> (2 * e)) & 1u, p1 = (b8 >> (2 * e + 1)) & 1u;
          if (write_sbar) ov[e] = (p0 ? 0x3f80u : 0xbf80u) | ((p1 ? 0x3f80u : 0xbf80u) << 16);      // bf16 +-1
          else ov[e] = pack_bf16x2(__uint_as_float(in[e] << 16) - (p0 ? step : -step),
                                   __uint_as_float(in[e] & 0xffff0000u) - (p1 ? step : -step));
        }
        o = make_uint4(ov[0], ov[1], ov[2], ov[3]);
        if (write_sbar && pd.sbar8) {                   // the same eight signs as E4M3 bytes (+1 = 0x38, -1 = 0xb8)
          uint32_t lo4 = 0, hi4 = 0;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            lo4 |= (((b8 >> e) & 1u) ? 0x38u : 0xb8u) << (8 * e);
            hi4 |= (((b8 >> (4 + e)) & 1u) ? 0x38u : 0xb8u) << (8 * e);
          }
          int64_t off = i * 8;                          // dense when the byte pitch equals the column count
          if (pd.ld8 != pd.cols) {
            const int64_t r = off / pd.cols;
            off = r * pd.ld8 + (off - r * pd.cols);
          }
          __stcs(reinterpret_cast<uint2*>(pd.sbar8 + off), make_uint2(lo4, hi4));
        }
      }
      __stcs(vbase + i, o);
    }
    return;
  }
  // scalar path: rows that are padded in the operand buffer (the +-1 matrix of a parameter whose column count is
  // not a multiple of 8), or d not a multiple of 8.  The block covers the same entries as on the vector path.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t e_begin = (int64_t)chunk * UPD_VECS * epv;
  const int64_t e_end = (e_begin + (int64_t)UPD_VECS * epv < d) ? e_begin + (int64_t)UPD_VECS * epv : d;
  for (int64_t i = e_begin + threadIdx.x; i < e_end; i += EW_THREADS) {
    const bool plus = (__ldcg(vw + (i >> 5)) >> (i & 31)) & 1u;
    if (write_sbar) {
      int64_t o = i;
      if (pd.ldy != pd.cols) {
        const int64_t r = i / pd.cols;
        o = r * pd.ldy + (i - r * pd.cols);
      }
      sbar[o] = __float2bfloat16_rn(plus ? 1.f : -1.f);
      if (pd.sbar8) {
        const int64_t r = i / pd.cols;
        pd.sbar8[r * pd.ld8 + (i - r * pd.cols)] = plus ? (uint8_t)0x38 : (uint8_t)0xb8;
      }
    } else {
      const float nw = load_as_float<WT>(w + i) - (plus ? step : -step);
      if (sizeof(WT) == 4) reinterpret_cast<float*>(w)[i] = nw;
      else reinterpret_cast<bf16*>(w)[i] = __float2bfloat16_rn(nw);
    }
  }
}

// LP = the local polar step follows: matrix parameters then receive the +-1 matrix instead of a weight update.  Two
// kernels, so that the plain weight update (LP = false) is compiled without the registers of the other path.
template <bool LP>
__global__ void __launch_bounds__(EW_THREADS, 4) update_kernel(const ParamDev* __restrict__ params,
                                                            const int32_t* __restrict__ list,
                                                            const uint32_t* __restrict__ starts, int n_list, int lp_slot,
                                                            float lr, const uint32_t* __restrict__ vote_words) {
  const int slot = find_slot(starts, n_list, blockIdx.x);
  const ParamDev pd = params[list[slot]];
  const uint32_t chunk = blockIdx.x - starts[slot];
  const float step = lr * pd.upd_scale;
  if (LP && pd.kind == 0) {                  // plain parameters are updated directly (no local polar step)
    if (pd.wdtype == 0) update_block<float, true>(pd, chunk, lp_slot, step, vote_words);
    else update_block<bf16, true>(pd, chunk, lp_slot, step, vote_words);
  } else {
    if (pd.wdtype == 0) update_block<float, false>(pd, chunk, lp_slot, step, vote_words);
    else update_block<bf16, false>(pd, chunk, lp_slot, step, vote_words);
  }
}

// ---------------------------------------------------------------------------------------------
// Integer sign sums (Alg. 2: "sum_signs <- sum_m S^(m)", all-reduce with SUM on int8).
// sign_sum_kernel: per payload bit position the sum of the +-1 signs of `rows` payload rows, one int8 per
// position (2 c - rows, c = number of set bits); thread t owns word t (32 positions, 32 bytes of output).
// sums_to_vote_kernel: S = sign(sum), ties -> +1, packed back into vote words (bit = sum >= 0).
// Pad positions carry bit 0 in every payload, so their sum is -rows (negative after any reduction): the vote
// keeps them 0.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS) sign_sum_kernel(const uint32_t* __restrict__ bits, int64_t bits_pitch,
                                                              int64_t words, int rows, int8_t* __restrict__ sums) {
  const int64_t w = (int64_t)blockIdx.x * EW_THREADS + threadIdx.x;
  if (w >= words) return;
  VoteCounter<8> cnt;
  cnt.clear();
  for (int m = 0; m < rows; ++m) cnt.add(__ldg(bits + (int64_t)m * bits_pitch + w));
  uint32_t out[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int j = q * 4 + e;
      int c = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) c |= (int)((cnt.c[b] >> j) & 1u) << b;
      packed |= (uint32_t)(uint8_t)(int8_t)(2 * c - rows) << (8 * e);
    }
    out[q] = packed;
  }
  uint4* o = reinterpret_cast<uint4*>(sums + w * 32);
  o[0] = make_uint4(out[0], out[1], out[2], out[3]);
  o[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

__global__ void __launch_bounds__(EW_THREADS) sums_to_vote_kernel(const int8_t* __restrict__ sums, int64_t words,
                                                                  uint32_t* __restrict__ vote_words) {
  const int64_t w = (int64_t)blockIdx.x * EW_THREADS + threadIdx.x;
  if (w >= words) return;
  const uint4* in = reinterpret_cast<const uint4*>(sums + w * 32);
  const uint4 a = __ldg(in), b = __ldg(in + 1);
  const uint32_t v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
  uint32_t word = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int8_t sv = (int8_t)((v[q] >> (8 * e)) & 0xffu);
      word |= (sv >= 0 ? 1u : 0u) << (q * 4 + e);
    }
  vote_words[w] = word;
}

// ---------------------------------------------------------------------------------------------
// Hand-shake of the fused exchange.  publish_payload_kernel runs after the last kernel that stores payload words:
// it makes those stores visible system-wide and writes this step's sequence number into slot `my_rank` of every
// peer's flag array.  await_payloads_kernel runs before the vote: lane r waits until slot r of this GPU's own flag
// array has reached the sequence number, at most `limit_ns`; a wait that runs out records STATUS_TIMEOUT.
// ---------------------------------------------------------------------------------------------
struct FlagList {
  int32_t n;
  int32_t reserved;
  uint32_t* flags[MAX_PAYLOAD_PEERS];
};
__global__ void publish_payload_kernel(const __grid_constant__ FlagList peers, int my_rank, uint32_t seq) {
  if (threadIdx.x < peers.n) {
    __threadfence_system();
    volatile uint32_t* f = peers.flags[threadIdx.x] + my_rank;
    *f = seq;
    __threadfence_system();
  }
}
__global__ void await_payloads_kernel(const uint32_t* own_flags, int n_ranks, int my_rank, uint32_t seq,
                                      uint64_t limit_ns, uint32_t* status) {
  const int r = threadIdx.x;
  if (r >= n_ranks || r == my_rank) return;
  const volatile uint32_t* f = own_flags + r;
  uint64_t t0 = 0;
  uint32_t spins = 0;
  // (sequence numbers wrap: compare as a signed distance)
  while ((int32_t)(*f - seq) < 0) {
    if ((++spins & 63u) == 0) {
      uint64_t now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) { atomicExch(status, (uint32_t)STATUS_TIMEOUT); return; }
    }
  }
  __threadfence_system();
}

// ---------------------------------------------------------------------------------------------
// Sign agreement (the quantity the paper's training scripts log next to the communication volume):
// per worker, the number of payload bits equal to the vote.  blockIdx.y = worker; pad bits are zero in
// every payload and in the vote, so they count as agreeing and the host subtracts them.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS) sign_agreement_kernel(const uint32_t* __restrict__ bits,
                                                                    const uint32_t* __restrict__ vote_words,
                                                                    int64_t words_per_worker, int64_t bits_pitch,
                                                                    unsigned long long* __restrict__ agree) {
  const int m = blockIdx.y;
  const uint32_t* mine = bits + (int64_t)m * bits_pitch;
  unsigned int acc = 0;   // at most 32 bits x (words / threads) per thread: far below 2^32
  for (int64_t i = (int64_t)blockIdx.x * EW_THREADS + threadIdx.x; i < words_per_worker; i += (int64_t)gridDim.x * EW_THREADS)
    acc += __popc(~(__ldg(mine + i) ^ __ldg(vote_words + i)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ unsigned int red[EW_THREADS / 32];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
#pragma unroll
    for (int i = 0; i < EW_THREADS / 32; ++i) t += red[i];
    atomicAdd(agree + m, t);    // integer: the result does not depend on the order
  }
}

}  // namespace signmuon
