// Weight-streaming grouped GEMM for groups of at most 16 rows (a latency-sensitive batch, a
// single decode request): C_g = epi(A_g W_g^T + bias_g) with M <= 16.
//
// With so few rows the work is reading W once; a 128-row tensor-core tile would leave most SMs idle
// on the narrow matrices and spend its time on zero rows.  Here one block of 8 warps owns 16
// consecutive rows of W (16 output columns) over the whole K, so a GEMM gives N / 16 blocks and
// every block has all of its loads in flight at once.  K is cut into 32-wide k-blocks dealt to the
// warps round-robin (warp w takes k-blocks w, w + 8, ...): in one k-block lane (gq, tq) reads 16
// contiguous bytes of W rows gq and gq + 8 and of activation row gq, which feed two
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate) with W as the 16-row operand and the batch as the
// 8 columns.  The k order inside an MMA is a permutation of memory order, the same one for both
// operands, which leaves every dot product unchanged.  The 8 warps' partial sums are added in warp
// order in shared memory, then the epilogue (bias, GELU, SwiGLU, fp32 residual) writes the outputs.
// An output row's value never depends on the other rows of the batch.
#include "common.cuh"
#include "kernels.h"

namespace epara {

namespace {

constexpr int RS_ROWS = 16;       // W rows (output columns) per block
constexpr int RS_WARPS = 8;
constexpr int RS_U = 4;           // k-blocks in flight per warp

__device__ __forceinline__ uint4 ldg_w(const bf16* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Activations are written by the kernel before this one: an ordinary (coherent) load that the
// compiler cannot move above the dependency wait.
__device__ __forceinline__ uint4 ld_act(const bf16* p) {
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ void mma16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ int find_group_rs(const GemmGroup* groups, int n, int item) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (groups[mid].tile_start <= item) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// NT: batch tiles of 8 rows (1: M <= 8, 2: M <= 16).
template <int NT>
__global__ void __launch_bounds__(RS_WARPS * 32, NT == 1 ? 3 : 2)
gemm_stream_kernel(const GemmGroup* __restrict__ groups, int n_groups) {
  __shared__ float red[RS_WARPS][NT][RS_ROWS][8];
  __shared__ float outv[NT][8][RS_ROWS + 1];
  pdl_launch_dependents();
  const GemmGroup& g = groups[find_group_rs(groups, n_groups, blockIdx.x)];
  const int n0 = (blockIdx.x - g.tile_start) * RS_ROWS;
  const int M = g.M, N = g.N, K = g.K;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gq = lane >> 2, tq = lane & 3;
  const int nkb = (K + 31) >> 5;

  const bool w_lo_ok = n0 + gq < N, w_hi_ok = n0 + gq + 8 < N;
  const bf16* w_lo = g.W + (size_t)(n0 + gq) * g.ldw + tq * 8;
  const bf16* w_hi = g.W + (size_t)(n0 + gq + 8) * g.ldw + tq * 8;
  const bf16* x_row[NT];
  bool x_ok[NT];
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    x_ok[t] = t * 8 + gq < M;
    x_row[t] = g.A + (size_t)(t * 8 + gq) * g.lda + tq * 8;
  }
  float acc[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t) { acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f; }

  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  // The weights are never written by a kernel, so the first batch of W loads is issued before the
  // wait on the earlier kernels of the stream; the activations are read after it.
  bool first = true;
  for (int kb0 = warp; kb0 < nkb || first; kb0 += RS_WARPS * RS_U) {
    uint4 wl[RS_U], wh[RS_U], xv[NT][RS_U];
#pragma unroll
    for (int u = 0; u < RS_U; ++u) {
      const int k = (kb0 + u * RS_WARPS) * 32;
      const bool k_ok = k + tq * 8 < K;              // K is a multiple of 8: a 16-byte piece is all in or all out
      wl[u] = (k_ok && w_lo_ok) ? ldg_w(w_lo + k) : zero4;
      wh[u] = (k_ok && w_hi_ok) ? ldg_w(w_hi + k) : zero4;
    }
    if (first) { pdl_wait(); first = false; }
#pragma unroll
    for (int u = 0; u < RS_U; ++u) {
      const int k = (kb0 + u * RS_WARPS) * 32;
      const bool k_ok = k + tq * 8 < K;
#pragma unroll
      for (int t = 0; t < NT; ++t)
        xv[t][u] = (k_ok && x_ok[t]) ? ld_act(x_row[t] + k) : zero4;
    }
#pragma unroll
    for (int u = 0; u < RS_U; ++u) {
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        mma16816(acc[t], wl[u].x, wh[u].x, wl[u].y, wh[u].y, xv[t][u].x, xv[t][u].y);
        mma16816(acc[t], wl[u].z, wh[u].z, wl[u].w, wh[u].w, xv[t][u].z, xv[t][u].w);
      }
    }
  }
  // accumulator layout: acc[0], acc[1] = (W row gq, batch rows 2tq, 2tq+1); acc[2], acc[3] = (W row gq+8, same)
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    red[warp][t][gq][2 * tq] = acc[t][0];
    red[warp][t][gq][2 * tq + 1] = acc[t][1];
    red[warp][t][gq + 8][2 * tq] = acc[t][2];
    red[warp][t][gq + 8][2 * tq + 1] = acc[t][3];
  }
  __syncthreads();
  const int epi = g.epi;
  for (int idx = threadIdx.x; idx < NT * 8 * RS_ROWS; idx += RS_WARPS * 32) {
    const int r = idx % RS_ROWS, bm = (idx / RS_ROWS) % 8, t = idx / (RS_ROWS * 8);
    float v = red[0][t][r][bm];
#pragma unroll
    for (int w = 1; w < RS_WARPS; ++w) v += red[w][t][r][bm];
    const int n = n0 + r;
    if ((epi & EPI_BIAS) && n < N) v += bf2f(g.bias[n]);
    if (epi & EPI_GELU) v = gelu_erf(v);
    outv[t][bm][r] = v;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < NT * 8 * RS_ROWS; idx += RS_WARPS * 32) {
    const int r = idx % RS_ROWS, bm = (idx / RS_ROWS) % 8, t = idx / (RS_ROWS * 8);
    const int m = t * 8 + bm, n = n0 + r;
    if (m >= M || n >= N) continue;
    const float v = outv[t][bm][r];
    if (epi & EPI_RESID_F32) {
      float* C = reinterpret_cast<float*>(g.C) + (size_t)m * g.ldc + n;
      *C += v;
    } else if (epi & EPI_SWIGLU) {
      if ((r & 1) == 0 && n + 1 < N)
        reinterpret_cast<bf16*>(g.C)[(size_t)m * g.ldc + (n >> 1)] = f2bf(silu_f(v) * outv[t][bm][r + 1]);
    } else {
      reinterpret_cast<bf16*>(g.C)[(size_t)m * g.ldc + n] = f2bf(v);
    }
  }
}

}  // namespace

int gemm_stream_tiles(int N) { return (N + RS_ROWS - 1) / RS_ROWS; }

cudaError_t launch_gemm_stream(const GemmGroup* groups, int n_groups, int total_items, int max_rows, cudaStream_t st) {
  if (n_groups == 0 || total_items == 0) return cudaSuccess;
  if (max_rows > 16) return cudaErrorInvalidValue;
  if (max_rows <= 8) return launch_pdl(gemm_stream_kernel<1>, dim3(total_items), dim3(RS_WARPS * 32), 0, st, groups, n_groups);
  return launch_pdl(gemm_stream_kernel<2>, dim3(total_items), dim3(RS_WARPS * 32), 0, st, groups, n_groups);
}

}  // namespace epara
