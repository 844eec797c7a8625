// Spectral-norm estimate by power iteration (Alg. 5) for every (matrix parameter, worker), the scale of
// Alg. 4 with scale = spectral:
//     v <- v0 / (||v0|| + eps);  P times { u <- X v, u <- u / (||u|| + eps);  v <- X^T u, v <- v / (||v|| + eps) };
//     sigma = ||X v||.
// X is the float32 momentum.  The vectors are kept un-normalised together with their norms; a matvec divides
// its input by (norm + eps) while reading it.  Memory-bound: each matvec reads X once (4 bytes per entry).
#pragma once

#include "elementwise.cuh"

namespace signmuon {

constexpr int PI_ROWS_PER_BLOCK = 8;     // X v: one warp per row
constexpr int PI_COLS_PER_BLOCK = 128;   // X^T u: 32 lanes x 4 columns, 8 warps stride over the rows

enum : int32_t { PI_NORM_START = 0, PI_NORM_U = 1, PI_NORM_V = 2, PI_NORM_SIGMA = 3 };

// One block per (matrix parameter, worker): Euclidean norm of a vector, fixed summation order (double).
//   PI_NORM_START: v <- v0 (copied from the caller's start vectors), scal[0] = ||v0||
//   PI_NORM_U:     scal[1] = ||u||          PI_NORM_V: scal[0] = ||v||
//   PI_NORM_SIGMA: sigma = ||u|| (u holds X v): scales = {1/max(sigma,eps)^2, 1/max(sigma,eps)}
__global__ void __launch_bounds__(EW_THREADS) pi_norm_kernel(const ParamDev* __restrict__ params,
                                                             const int32_t* __restrict__ list, int num_workers,
                                                             int mode, float eps) {
  const ParamDev& pd = params[list[blockIdx.x / num_workers]];
  const int m = blockIdx.x % num_workers;
  const bool on_u = (mode == PI_NORM_U || mode == PI_NORM_SIGMA);
  const int n = on_u ? pd.rows : pd.cols;
  float* vec = on_u ? pd.pi_u + (int64_t)m * pd.rows : pd.pi_v + (int64_t)m * pd.cols;
  const float* src = (mode == PI_NORM_START) ? pd.pi_start + (int64_t)m * pd.cols : vec;
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += EW_THREADS) {
    const float x = src[i];
    if (mode == PI_NORM_START) vec[i] = x;
    acc += (double)x * (double)x;
  }
  __shared__ double red[EW_THREADS / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < EW_THREADS / 32; ++i) t += red[i];
    const double nrm = sqrt(t);
    if (mode == PI_NORM_SIGMA) {
      const double sigma = fmax(nrm, (double)eps);
      pd.scales[2 * m] = (float)(1.0 / (sigma * sigma));
      pd.scales[2 * m + 1] = (float)(1.0 / sigma);
    } else {
      pd.pi_scal[2 * m + (on_u ? 1 : 0)] = (float)nrm;
    }
  }
}

// u_raw = X (v / (||v|| + eps)): one warp per row, lanes stride over the columns (coalesced 128-byte reads).
__global__ void __launch_bounds__(EW_THREADS) pi_xv_kernel(const ParamDev* __restrict__ params,
                                                           const int32_t* __restrict__ list,
                                                           const uint32_t* __restrict__ starts, int n_list, float eps) {
  const int slot = find_slot(starts, n_list, blockIdx.x);
  const ParamDev& pd = params[list[slot]];
  const uint32_t local = blockIdx.x - starts[slot];
  const uint32_t bpw = (uint32_t)((pd.rows + PI_ROWS_PER_BLOCK - 1) / PI_ROWS_PER_BLOCK);
  const int m = local / bpw;
  const int row = (int)(local - m * bpw) * PI_ROWS_PER_BLOCK + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= pd.rows) return;
  const float* x = pd.mom + (int64_t)m * pd.d + (int64_t)row * pd.cols;
  const float* v = pd.pi_v + (int64_t)m * pd.cols;
  const float inv = 1.f / (pd.pi_scal[2 * m] + eps);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  int j = lane;
  for (; j + 96 < pd.cols; j += 128) {
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[k] = fmaf(__ldcs(x + j + 32 * k), __ldg(v + j + 32 * k), acc[k]);
  }
  for (; j < pd.cols; j += 32) acc[0] = fmaf(__ldcs(x + j), __ldg(v + j), acc[0]);
  const float s = warp_sum((acc[0] + acc[1]) + (acc[2] + acc[3]));
  if (lane == 0) pd.pi_u[(int64_t)m * pd.rows + row] = s * inv;
}

// v_raw = X^T (u / (||u|| + eps)): a block owns 128 columns; warp w adds rows w, w + 8, ...; lane l holds
// columns l, l + 32, l + 64, l + 96 of the strip; the eight warps' partial sums are added in a fixed order.
__global__ void __launch_bounds__(EW_THREADS) pi_xtu_kernel(const ParamDev* __restrict__ params,
                                                            const int32_t* __restrict__ list,
                                                            const uint32_t* __restrict__ starts, int n_list, float eps) {
  const int slot = find_slot(starts, n_list, blockIdx.x);
  const ParamDev& pd = params[list[slot]];
  const uint32_t local = blockIdx.x - starts[slot];
  const uint32_t bpw = (uint32_t)((pd.cols + PI_COLS_PER_BLOCK - 1) / PI_COLS_PER_BLOCK);
  const int m = local / bpw;
  const int col0 = (int)(local - m * bpw) * PI_COLS_PER_BLOCK;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* x = pd.mom + (int64_t)m * pd.d;
  const float* u = pd.pi_u + (int64_t)m * pd.rows;
  const float inv = 1.f / (pd.pi_scal[2 * m + 1] + eps);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  bool in[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) in[k] = col0 + lane + 32 * k < pd.cols;
  for (int i = warp; i < pd.rows; i += EW_THREADS / 32) {
    const float ui = __ldg(u + i);
    const float* xr = x + (int64_t)i * pd.cols + col0 + lane;
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (in[k]) acc[k] = fmaf(__ldcs(xr + 32 * k), ui, acc[k]);
  }
  __shared__ float part[EW_THREADS / 32][PI_COLS_PER_BLOCK];
#pragma unroll
  for (int k = 0; k < 4; ++k) part[warp][lane + 32 * k] = acc[k];
  __syncthreads();
  if (threadIdx.x < PI_COLS_PER_BLOCK && col0 + threadIdx.x < pd.cols) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < EW_THREADS / 32; ++w) t += part[w][threadIdx.x];
    pd.pi_v[(int64_t)m * pd.cols + col0 + threadIdx.x] = t * inv;
  }
}

}  // namespace signmuon
