// Diagnostic CUDA-core version of the Newton-Schulz products: same problems, tiles and epilogues
// as the tensor-core kernel, plain shared-memory tiling, fp32 accumulation of bf16 operands.
// Selected by SIGNMUON_FLAG_SIMT_GEMM; used to tell an epilogue/layout mistake from a
// tensor-core descriptor mistake.  Not a performance path.
#pragma once

#include "common.cuh"

namespace signmuon {

__global__ void __launch_bounds__(128) ns_gemm_simt_kernel(const GemmProblem* __restrict__ problems,
                                                           const TileEntry* __restrict__ tiles, int bn,
                                                           const ParamDev* __restrict__ params, float lr,
                                                           const __grid_constant__ PeerList peers) {
  __shared__ float As[128][33];
  __shared__ float Bs[32][33];
  const TileEntry te = tiles[blockIdx.x];
  const GemmProblem pr = problems[te.problem];
  const int m0 = te.tm * 128;
  const int n0 = te.tn * bn;
  const int tid = threadIdx.x;
  for (int c0 = n0; c0 < n0 + bn && c0 < pr.N; c0 += 32) {
    float acc[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
    for (int k0 = 0; k0 < pr.K; k0 += 32) {
      for (int idx = tid; idx < 128 * 32; idx += 128) {
        int i, k;
        if (pr.a_mn) { i = idx & 127; k = idx >> 7; } else { i = idx >> 5; k = idx & 31; }
        float x = 0.f;
        if (m0 + i < pr.M && k0 + k < pr.K)
          x = __bfloat162float(pr.A[(int64_t)(m0 + i) * pr.a_sm + (int64_t)(k0 + k) * pr.a_sk]);
        As[i][k] = x;
      }
      for (int idx = tid; idx < 32 * 32; idx += 128) {
        int j, k;
        if (pr.b_mn) { j = idx & 31; k = idx >> 5; } else { j = idx >> 5; k = idx & 31; }
        float x = 0.f;
        if (c0 + j < pr.N && k0 + k < pr.K)
          x = __bfloat162float(pr.B[(int64_t)(c0 + j) * pr.b_sn + (int64_t)(k0 + k) * pr.b_sk]);
        Bs[j][k] = x;
      }
      __syncthreads();
#pragma unroll 4
      for (int k = 0; k < 32; ++k) {
        const float a = As[tid][k];
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[j] = fmaf(a, Bs[j][k], acc[j]);
      }
      __syncthreads();
    }
    epilogue_row32(pr, params, lr, m0 + tid, c0, acc, peers);
  }
}

}  // namespace signmuon
