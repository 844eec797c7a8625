// signmuon_momentum_norm_noalloc: the momentum + Frobenius-norm stage of the SignMuon step for one
// matrix, for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off the table - a step body being recorded into
// a larger pipeline whose memory plan is frozen, a plugin living inside another framework's caching
// allocator that must not grow its pool, a real-time loop that may not take the allocator lock.  The
// regular path gets its scratch (the per-block partial sums of the two-stage norm reduction) from the
// caller-provided workspace; this entry point keeps that scratch in a fixed array that is part of the
// library image instead, so a caller only brings inputs and outputs.
//
// Consequences of the fixed array, all of them visible to the caller:
//   * it has a hard capacity (SIGNMUON_NOALLOC_MAX_PARTIALS partial sums, one per 8192 entries per
//     worker); larger problems are refused with SIGNMUON_ERR_TOO_LARGE, nothing is launched;
//   * every GPU that loads the library carries the array (256 KB) until the process exits;
//   * all calls share it.  The partial sums a call uses are fully rewritten by that call before they
//     are read, so nothing has to be cleared between calls, but two calls that overlap on the GPU
//     (different streams, no ordering between them) race on it.  Keep calls stream-ordered.
//   * the first call on each device looks up the array's device address (cudaGetSymbolAddress with
//     that device current).  Make that first call outside any stream capture.  That first call is also
//     where the CUDA runtime may load this library's device code onto the GPU and place the array
//     (lazy module loading): "allocates nothing" describes every call after it, and this one as far as
//     the library's own code goes.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/signmuon.h"

namespace {

typedef __nv_bfloat16 bf16;

constexpr int NA_THREADS = 256;
constexpr int NA_CHUNK = 8192;                       // entries per block
constexpr int NA_MAX_DEVICES = 64;

// The scratch. In host code this name is only a handle for cudaGetSymbolAddress, never a pointer
// that a kernel may be given.
static __device__ __align__(256) float g_noalloc_partials[SIGNMUON_NOALLOC_MAX_PARTIALS];

std::mutex g_setup_mutex;
float* g_partials_addr[NA_MAX_DEVICES] = {};         // per device: device address of the array above

// Looks up (once per device, with that device current) the device address of the scratch array.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return SIGNMUON_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_partials_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_partials) != cudaSuccess || !p) return SIGNMUON_ERR_CUDA;
    g_partials_addr[dev] = static_cast<float*>(p);
  }
  *out = g_partials_addr[dev];
  return SIGNMUON_OK;
}

__device__ __forceinline__ void na_load8(const float* p, float (&x)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *(reinterpret_cast<const float4*>(p) + 1);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void na_load8(const bf16* p, float (&x)[8]) {
  const uint4 a = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    x[2 * e] = __uint_as_float(w[e] << 16);
    x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
  }
}

// Mom <- beta Mom + (1 - beta)(G + lambda W); operand = bf16(Mom); partials[worker][block] = sum Mom^2.
// Same arithmetic, in the same order, as the regular momentum kernel's vector path.
template <typename GT, typename WT>
__global__ void __launch_bounds__(NA_THREADS) momentum_noalloc_kernel(const GT* __restrict__ grads,
                                                                      const WT* __restrict__ weights,
                                                                      float* __restrict__ mom, bf16* __restrict__ operand,
                                                                      float* __restrict__ partials, int64_t d,
                                                                      uint32_t chunks_per_worker, float beta,
                                                                      float lambda) {
  const uint32_t m = blockIdx.x / chunks_per_worker;
  const uint32_t chunk = blockIdx.x - m * chunks_per_worker;
  const GT* g = grads + (int64_t)m * d;
  float* mo = mom + (int64_t)m * d;
  bf16* y = operand + (int64_t)m * d;
  const int64_t base = (int64_t)chunk * NA_CHUNK;
  const float omb = 1.f - beta;
  float sumsq = 0.f;
#pragma unroll
  for (int it = 0; it < NA_CHUNK / (NA_THREADS * 8); ++it) {
    const int64_t i = base + ((int64_t)it * NA_THREADS + threadIdx.x) * 8;
    if (i < d) {
      float gv[8], mv[8];
      na_load8(g + i, gv);
      na_load8(mo + i, mv);
      if (lambda != 0.f) {
        float wv[8];
        na_load8(weights + i, wv);
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
      float4* o = reinterpret_cast<float4*>(mo + i);
      o[0] = make_float4(mv[0], mv[1], mv[2], mv[3]);
      o[1] = make_float4(mv[4], mv[5], mv[6], mv[7]);
      *reinterpret_cast<uint4*>(y + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    }
  }
  __shared__ float red[NA_THREADS / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sumsq += __shfl_xor_sync(0xffffffffu, sumsq, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sumsq;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < NA_THREADS / 32; ++i) t += red[i];
    partials[(int64_t)m * chunks_per_worker + chunk] = t;
  }
}

// One warp per worker: fixed-order sum of that worker's partials, then 1/max(sigma,eps)^2 and 1/max(sigma,eps).
__global__ void norm_noalloc_kernel(const float* __restrict__ partials, uint32_t chunks_per_worker, int num_workers,
                                    float eps, float* __restrict__ scales) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= num_workers) return;
  const float* part = partials + (int64_t)warp * chunks_per_worker;
  double acc = 0.0;
  for (uint32_t i = lane; i < chunks_per_worker; i += 32) acc += (double)part[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const double sigma = fmax(sqrt(acc), (double)eps);
    scales[2 * warp] = (float)(1.0 / (sigma * sigma));
    scales[2 * warp + 1] = (float)(1.0 / sigma);
  }
}

// Launches return their own status (cudaLaunchKernelEx), so an earlier, unrelated error that is still
// pending in the runtime is neither reported as this call's nor cleared by it.
cudaLaunchConfig_t launch_config(unsigned blocks, unsigned threads, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks, 1, 1);
  cfg.blockDim = dim3(threads, 1, 1);
  cfg.stream = s;
  return cfg;
}

template <typename GT, typename WT>
cudaError_t launch_noalloc(const void* g, const void* w, float* mom, void* operand, float* partials, int64_t d,
                           uint32_t cpw, int M, float beta, float lambda, cudaStream_t s) {
  const cudaLaunchConfig_t cfg = launch_config(cpw * (uint32_t)M, NA_THREADS, s);
  return cudaLaunchKernelEx(&cfg, momentum_noalloc_kernel<GT, WT>, static_cast<const GT*>(g),
                            static_cast<const WT*>(w), mom, static_cast<bf16*>(operand), partials, d, cpw, beta, lambda);
}

}  // namespace

extern "C" int signmuon_momentum_norm_noalloc(const void* dev_grads, int32_t grad_dtype, const void* dev_weights,
                                              int32_t weight_dtype, float* dev_momentum, void* dev_operand_bf16,
                                              float* dev_scales, int64_t rows, int64_t cols, int32_t num_workers,
                                              float momentum, float weight_decay, float eps, void* cuda_stream) {
  if (!dev_grads || !dev_momentum || !dev_operand_bf16 || !dev_scales) return SIGNMUON_ERR_INVALID_ARG;
  if (grad_dtype != SIGNMUON_F32 && grad_dtype != SIGNMUON_BF16) return SIGNMUON_ERR_INVALID_ARG;
  if (weight_dtype != SIGNMUON_F32 && weight_dtype != SIGNMUON_BF16) return SIGNMUON_ERR_INVALID_ARG;
  if (num_workers < 1 || num_workers > 255) return SIGNMUON_ERR_INVALID_ARG;
  if (!(momentum >= 0.f && momentum < 1.f) || !(weight_decay >= 0.f)) return SIGNMUON_ERR_INVALID_ARG;
  if (weight_decay != 0.f && !dev_weights) return SIGNMUON_ERR_INVALID_ARG;
  if (rows < 1 || cols < 1 || rows > (1 << 24) || cols > (1 << 24)) return SIGNMUON_ERR_BAD_SHAPE;
  const int64_t d = rows * cols;
  if (d % 8 != 0) return SIGNMUON_ERR_BAD_SHAPE;      // 16-byte vector accesses per worker slab
  const int64_t cpw = (d + NA_CHUNK - 1) / NA_CHUNK;
  if (cpw * num_workers > SIGNMUON_NOALLOC_MAX_PARTIALS) return SIGNMUON_ERR_TOO_LARGE;
  const uintptr_t align = reinterpret_cast<uintptr_t>(dev_grads) | reinterpret_cast<uintptr_t>(dev_momentum) |
                          reinterpret_cast<uintptr_t>(dev_operand_bf16) | reinterpret_cast<uintptr_t>(dev_weights);
  if ((align & 15) || (reinterpret_cast<uintptr_t>(dev_scales) & 3)) return SIGNMUON_ERR_MISALIGNED;
  if (!(eps > 0.f)) eps = 1e-12f;

  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return SIGNMUON_ERR_CUDA;
  if (major != 10) return SIGNMUON_ERR_UNSUPPORTED_ARCH;   // the library image holds sm_100a code only

  float* partials = nullptr;                           // device address of g_noalloc_partials on this device
  const int rc = scratch_for_current_device(&partials);
  if (rc != SIGNMUON_OK) return rc;

  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  const uint32_t c = (uint32_t)cpw;
  cudaError_t err;
  if (grad_dtype == SIGNMUON_F32) {
    if (weight_dtype == SIGNMUON_F32)
      err = launch_noalloc<float, float>(dev_grads, dev_weights, dev_momentum, dev_operand_bf16, partials, d, c, num_workers, momentum, weight_decay, s);
    else
      err = launch_noalloc<float, bf16>(dev_grads, dev_weights, dev_momentum, dev_operand_bf16, partials, d, c, num_workers, momentum, weight_decay, s);
  } else {
    if (weight_dtype == SIGNMUON_F32)
      err = launch_noalloc<bf16, float>(dev_grads, dev_weights, dev_momentum, dev_operand_bf16, partials, d, c, num_workers, momentum, weight_decay, s);
    else
      err = launch_noalloc<bf16, bf16>(dev_grads, dev_weights, dev_momentum, dev_operand_bf16, partials, d, c, num_workers, momentum, weight_decay, s);
  }
  if (err != cudaSuccess) return SIGNMUON_ERR_CUDA;
  const cudaLaunchConfig_t ncfg = launch_config((unsigned)(num_workers * 32 + 255) / 256, 256, s);
  err = cudaLaunchKernelEx(&ncfg, norm_noalloc_kernel, static_cast<const float*>(partials), c, (int)num_workers, eps,
                           dev_scales);
  return err == cudaSuccess ? SIGNMUON_OK : SIGNMUON_ERR_CUDA;
}
