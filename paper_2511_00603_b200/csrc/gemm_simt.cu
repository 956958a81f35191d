// Grouped GEMM on the CUDA cores: C_g = epi(A_g W_g^T + bias_g), 64 x 64 tiles, fp32 accumulate.
// This is the plain comparator of the tcgen05 kernel (same descriptors, same epilogues); it is
// selected by epara_config.gemm_impl = EPARA_GEMM_SIMT and used to localise a disagreement.
#include "common.cuh"
#include "kernels.h"

namespace epara {

__device__ __forceinline__ int find_group(const GemmGroup* groups, int n, int tile) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (groups[mid].tile_start <= tile) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmGroup* __restrict__ groups, int n_groups) {
  __shared__ float As[16][SIMT_TILE + 4];
  __shared__ float Ws[16][SIMT_TILE + 4];
  pdl_launch_dependents();
  pdl_wait();
  const int gi = find_group(groups, n_groups, blockIdx.x);
  const GemmGroup& g = groups[gi];
  const int local = blockIdx.x - g.tile_start;
  const int tm = local / g.tiles_n, tn = local % g.tiles_n;
  const int m0 = tm * SIMT_TILE, n0 = tn * SIMT_TILE;
  const int M = g.M, N = g.N, K = g.K;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int lr = threadIdx.x >> 2, lc = (threadIdx.x & 3) * 4;   // loader: row 0..63, k offset 0,4,8,12
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int k = k0 + lc + i;
      As[lc + i][lr] = (m0 + lr < M && k < K) ? bf2f(g.A[(size_t)(m0 + lr) * g.lda + k]) : 0.f;
      Ws[lc + i][lr] = (n0 + lr < N && k < K) ? bf2f(g.W[(size_t)(n0 + lr) * g.ldw + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; w[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      v[j] = acc[i][j];
      if ((g.epi & EPI_BIAS) && n < N) v[j] += bf2f(g.bias[n]);
      if (g.epi & EPI_GELU) v[j] = gelu_erf(v[j]);
    }
    if (g.epi & EPI_RESID_F32) {
      float* C = reinterpret_cast<float*>(g.C) + (size_t)m * g.ldc;
#pragma unroll
      for (int j = 0; j < 4; ++j) { const int n = n0 + tx * 4 + j; if (n < N) C[n] += v[j]; }
    } else if (g.epi & EPI_SWIGLU) {
      bf16* C = reinterpret_cast<bf16*>(g.C) + (size_t)m * g.ldc;
#pragma unroll
      for (int j = 0; j < 4; j += 2) {
        const int n = n0 + tx * 4 + j;
        if (n + 1 < N) C[n >> 1] = f2bf(silu_f(v[j]) * v[j + 1]);
      }
    } else {
      bf16* C = reinterpret_cast<bf16*>(g.C) + (size_t)m * g.ldc;
#pragma unroll
      for (int j = 0; j < 4; ++j) { const int n = n0 + tx * 4 + j; if (n < N) C[n] = f2bf(v[j]); }
    }
  }
}

void launch_gemm_simt(const GemmGroup* groups, int n_groups, int total_tiles, cudaStream_t st) {
  if (n_groups == 0 || total_tiles == 0) return;
  gemm_simt_kernel<<<total_tiles, 256, 0, st>>>(groups, n_groups);
}

}  // namespace epara
