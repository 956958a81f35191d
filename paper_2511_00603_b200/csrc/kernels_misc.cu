// Bandwidth-trivial kernels of a step: input gather / embedding / patchify, LayerNorm and
// RMSNorm, RoPE + KV append, ViT token assembly, logits scatter + argmax.
// Every launch is grouped: blockIdx.y selects the group (one model), blockIdx.x a unit of work
// inside it; blocks beyond a group's extent return at once.
#include "common.cuh"
#include "kernels.h"

namespace epara {

// ------------------------------------------------------------------ gather
// Row and embedding gathers take one block per row (a handful of rows per step); the patch gather takes
// GATHER_PATCH_ROWS patch rows per block, so that a thread has several 16-byte loads in flight.
__global__ void __launch_bounds__(128) gather_kernel(const GatherGroup* __restrict__ groups) {
  const GatherGroup g = groups[blockIdx.y];
  if ((int)blockIdx.x >= g.blocks) return;      // (descriptors are not written by kernels: no wait needed to leave)
  pdl_launch_dependents();
  pdl_wait();
  if (g.kind == GATHER_ROWS) {
    const int b = blockIdx.x;
    const uint4* src = reinterpret_cast<const uint4*>(g.reqs[b].input);
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(g.out) + (size_t)b * g.ld);
    for (int i = threadIdx.x; i < g.width / 8; i += blockDim.x) dst[i] = src[i];
  } else if (g.kind == GATHER_EMB) {
    const int b = blockIdx.x;              // one block per token row
    const int tok = g.rows[b].token;
    const uint4* src = reinterpret_cast<const uint4*>(g.emb + (size_t)tok * g.width);
    float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(g.out) + (size_t)b * g.width);
    for (int i = threadIdx.x; i < g.width / 8; i += blockDim.x) {
      float f[8];
      unpack8(src[i], f);
      dst[2 * i] = make_float4(f[0], f[1], f[2], f[3]);
      dst[2 * i + 1] = make_float4(f[4], f[5], f[6], f[7]);
    }
  } else {  // GATHER_PATCH: row (b*np + i*gw + j), column c*p*p + u*p + v  <-  img[b][c][p*i+u][p*j+v]
    const int p = g.patch, gw = g.img / p, np = gw * gw;
    const int vec_per_row = p / 8, vecs = g.width / 8;
    const int row0 = blockIdx.x * GATHER_PATCH_ROWS;
    const int nrows = min(GATHER_PATCH_ROWS, g.B * np - row0);
#pragma unroll 4
    for (int idx = threadIdx.x; idx < nrows * vecs; idx += blockDim.x) {
      const int row = row0 + idx / vecs, e = idx % vecs;
      const int b = row / np, pi = row % np;
      const int i = pi / gw, j = pi % gw;
      const int cu = e / vec_per_row, v8 = e % vec_per_row;   // cu = c*p + u
      const int c = cu / p, u = cu % p;
      const bf16* img = reinterpret_cast<const bf16*>(g.reqs[b].input);
      const bf16* s = img + ((size_t)c * g.img + (size_t)(p * i + u)) * g.img + p * j + v8 * 8;
      reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(g.out) + (size_t)row * g.width)[e] = *reinterpret_cast<const uint4*>(s);
    }
  }
}

void launch_gather(const GatherGroup* groups, int n_groups, int max_blocks, cudaStream_t st) {
  if (n_groups == 0 || max_blocks == 0) return;
  launch_pdl(gather_kernel, dim3(max_blocks, n_groups), dim3(128), 0, st, groups);
}

// ------------------------------------------------------------------ norms
// Rows are held in registers between the statistics pass and the write.  Narrow rows
// (d <= 1024) take one warp per row, 8 rows per block; wider rows one block per row.
constexpr int NORM_THREADS = 256;
constexpr int NORM_WARP_D = 1024;

template <bool WARP>
__device__ __forceinline__ void norm_row(const NormGroup& g, int row, float* red) {
  constexpr int STRIDE = WARP ? 32 : NORM_THREADS;
  const int t = WARP ? (threadIdx.x & 31) : threadIdx.x;
  const int nvec = g.d >> 2;
  const float4* x = reinterpret_cast<const float4*>(g.x + (size_t)(g.row_index ? g.row_index[row] : row) * g.x_stride);
  float4 v[8];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = t + i * STRIDE;
    if (c < nvec) {
      v[i] = x[c];
      s += (g.kind == NORM_LN) ? (v[i].x + v[i].y) + (v[i].z + v[i].w)
                               : (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
    }
  }
  s = WARP ? warp_sum(s) : block_sum(s, red);
  float mean = 0.f, rstd;
  const float inv_d = 1.0f / (float)g.d;
  if (g.kind == NORM_LN) {
    mean = s * inv_d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = t + i * STRIDE;
      if (c < nvec) {
        const float a = v[i].x - mean, b = v[i].y - mean, cc = v[i].z - mean, dd = v[i].w - mean;
        q += (a * a + b * b) + (cc * cc + dd * dd);
      }
    }
    q = WARP ? warp_sum(q) : block_sum(q, red);
    rstd = 1.0f / sqrtf(q * inv_d + g.eps);
  } else {
    rstd = 1.0f / sqrtf(s * inv_d + g.eps);
  }
  uint2* y = reinterpret_cast<uint2*>(g.y + (size_t)row * g.d);
  const uint2* gm = reinterpret_cast<const uint2*>(g.gamma);
  const uint2* bt = reinterpret_cast<const uint2*>(g.beta);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = t + i * STRIDE;
    if (c < nvec) {
      const uint2 gg = __ldg(gm + c);
      float ga[4] = {__uint_as_float(gg.x << 16), __uint_as_float(gg.x & 0xffff0000u),
                     __uint_as_float(gg.y << 16), __uint_as_float(gg.y & 0xffff0000u)};
      float be[4] = {0.f, 0.f, 0.f, 0.f};
      if (g.kind == NORM_LN) {
        const uint2 bb = __ldg(bt + c);
        be[0] = __uint_as_float(bb.x << 16); be[1] = __uint_as_float(bb.x & 0xffff0000u);
        be[2] = __uint_as_float(bb.y << 16); be[3] = __uint_as_float(bb.y & 0xffff0000u);
      }
      uint2 o;
      o.x = pack2((v[i].x - mean) * rstd * ga[0] + be[0], (v[i].y - mean) * rstd * ga[1] + be[1]);
      o.y = pack2((v[i].z - mean) * rstd * ga[2] + be[2], (v[i].w - mean) * rstd * ga[3] + be[3]);
      y[c] = o;
    }
  }
}

// Narrow rows (d <= 512): one warp takes ROWS rows at once, all their loads in flight together.  Two rows
// keep the kernel at 64 registers, so four blocks (32 warps) share an SM: with more registers per
// thread the occupancy, not the loads per warp, limited the bandwidth.
constexpr int NORM_NARROW_D = 512;
constexpr int NORM_NARROW_ROWS = 2;
__device__ __forceinline__ void norm_rows_narrow(const NormGroup& g, int row0) {
  const int lane = threadIdx.x & 31;
  const int nvec = g.d >> 2;
  float4 v[NORM_NARROW_ROWS][4];
#pragma unroll
  for (int r = 0; r < NORM_NARROW_ROWS; ++r) {
    const bool live = row0 + r < g.M;
    const float4* x = reinterpret_cast<const float4*>(g.x + (size_t)((live && g.row_index) ? g.row_index[row0 + r] : row0 + r) * g.x_stride);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = lane + i * 32;
      v[r][i] = (live && c < nvec) ? x[c] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  const float inv_d = 1.0f / (float)g.d;
  const uint2* gm = reinterpret_cast<const uint2*>(g.gamma);
  const uint2* bt = reinterpret_cast<const uint2*>(g.beta);
#pragma unroll
  for (int r = 0; r < NORM_NARROW_ROWS; ++r) {
    if (row0 + r >= g.M) break;                  // uniform across the warp
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      s += (g.kind == NORM_LN) ? (v[r][i].x + v[r][i].y) + (v[r][i].z + v[r][i].w)
                               : (v[r][i].x * v[r][i].x + v[r][i].y * v[r][i].y) + (v[r][i].z * v[r][i].z + v[r][i].w * v[r][i].w);
    s = warp_sum(s);
    float mean = 0.f, rstd;
    if (g.kind == NORM_LN) {
      mean = s * inv_d;
      float q = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (lane + i * 32 < nvec) {
          const float a = v[r][i].x - mean, b = v[r][i].y - mean, cc = v[r][i].z - mean, dd = v[r][i].w - mean;
          q += (a * a + b * b) + (cc * cc + dd * dd);
        }
      }
      q = warp_sum(q);
      rstd = 1.0f / sqrtf(q * inv_d + g.eps);
    } else {
      rstd = 1.0f / sqrtf(s * inv_d + g.eps);
    }
    uint2* y = reinterpret_cast<uint2*>(g.y + (size_t)(row0 + r) * g.d);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = lane + i * 32;
      if (c < nvec) {
        const uint2 gg = __ldg(gm + c);
        const float ga[4] = {__uint_as_float(gg.x << 16), __uint_as_float(gg.x & 0xffff0000u),
                             __uint_as_float(gg.y << 16), __uint_as_float(gg.y & 0xffff0000u)};
        float be[4] = {0.f, 0.f, 0.f, 0.f};
        if (g.kind == NORM_LN) {
          const uint2 bb = __ldg(bt + c);
          be[0] = __uint_as_float(bb.x << 16); be[1] = __uint_as_float(bb.x & 0xffff0000u);
          be[2] = __uint_as_float(bb.y << 16); be[3] = __uint_as_float(bb.y & 0xffff0000u);
        }
        uint2 o;
        o.x = pack2((v[r][i].x - mean) * rstd * ga[0] + be[0], (v[r][i].y - mean) * rstd * ga[1] + be[1]);
        o.y = pack2((v[r][i].z - mean) * rstd * ga[2] + be[2], (v[r][i].w - mean) * rstd * ga[3] + be[3]);
        y[c] = o;
      }
    }
  }
}

// Blocks a group of M rows of width d needs (device copy of norm_blocks).
__device__ __forceinline__ int norm_blocks_dev(int M, int d) {
  constexpr int wpb = NORM_THREADS / 32;
  if (d <= NORM_NARROW_D) return (M + wpb * NORM_NARROW_ROWS - 1) / (wpb * NORM_NARROW_ROWS);
  return d <= NORM_WARP_D ? (M + wpb - 1) / wpb : M;
}

__global__ void __launch_bounds__(NORM_THREADS, 4) norm_kernel(const NormGroup* __restrict__ groups) {
  __shared__ float red[32];
  const NormGroup g = groups[blockIdx.y];
  if ((int)blockIdx.x >= norm_blocks_dev(g.M, g.d)) return;   // beyond this group's rows: nothing to wait for
  pdl_launch_dependents();
  pdl_wait();
  if (g.d <= NORM_NARROW_D) {
    const int row0 = (blockIdx.x * (NORM_THREADS / 32) + (threadIdx.x >> 5)) * NORM_NARROW_ROWS;
    if (row0 < g.M) norm_rows_narrow(g, row0);
  } else if (g.d <= NORM_WARP_D) {
    const int row = blockIdx.x * (NORM_THREADS / 32) + (threadIdx.x >> 5);
    if (row < g.M) norm_row<true>(g, row, red);
  } else {
    norm_row<false>(g, blockIdx.x, red);
  }
}

// Blocks a group of M rows of width d needs.
int norm_blocks(int M, int d) {
  const int wpb = NORM_THREADS / 32;
  if (d <= NORM_NARROW_D) return (M + wpb * NORM_NARROW_ROWS - 1) / (wpb * NORM_NARROW_ROWS);
  return d <= NORM_WARP_D ? (M + wpb - 1) / wpb : M;
}

void launch_norm(const NormGroup* groups, int n_groups, int max_blocks, cudaStream_t st) {
  if (n_groups == 0 || max_blocks == 0) return;
  launch_pdl(norm_kernel, dim3(max_blocks, n_groups), dim3(NORM_THREADS), 0, st, groups);
}

// ------------------------------------------------------------------ RoPE + KV append
// One block per token row (a decode request has one row, a prompt chunk one per token).  The row's token sits
// at position `pos` of its sequence: q and k are rotated there
// (interleaved pairs; cos and sin come from the model's table, computed from fp64 angles when the
// model was placed), q in place, k and v written to the cache page table[pos/16], slot pos%16.
// The page id comes from the caller's block table and is checked against the pool's page count.
__global__ void __launch_bounds__(256) rope_append_kernel(const RopeGroup* __restrict__ groups) {
  const RopeGroup g = groups[blockIdx.y];
  const int b = blockIdx.x;               // token row
  if (b >= g.B) return;
  pdl_launch_dependents();
  pdl_wait();
  const RowDesc rd = g.rows[b];
  const int pos = rd.pos, hd = g.hd, half = hd >> 1;
  const float2* cs = g.cs + (size_t)pos * half;
  const int page = g.reqs[rd.req].table[pos / 16], slot = pos % 16;
  // a page id outside the pool is reported and nothing is written for this row (q stays unrotated)
  if (page < 0 || page >= g.kv_pages) {
    if (threadIdx.x == 0) atomicExch(g.status, ERR_PAGE_APPEND);
    return;
  }
  bf16* row = g.qkv + (size_t)b * (g.Hq + 2 * g.Hkv) * hd;
  const int n_rot = (g.Hq + g.Hkv) * half;
  for (int e = threadIdx.x; e < n_rot; e += blockDim.x) {
    const int h = e / half, j = e % half;
    const float2 t = __ldg(cs + j);
    __nv_bfloat162* p2 = reinterpret_cast<__nv_bfloat162*>(row + (size_t)h * hd) + j;
    const float2 v = __bfloat1622float2(*p2);
    const float x0 = v.x * t.x - v.y * t.y, x1 = v.x * t.y + v.y * t.x;
    const __nv_bfloat162 o = __floats2bfloat162_rn(x0, x1);
    if (h < g.Hq) {
      *p2 = o;
    } else {
      const int kh = h - g.Hq;
      bf16* dst = g.kv_layer + (((size_t)page * 2 + 0) * g.Hkv + kh) * 16 * hd + (size_t)slot * hd;
      reinterpret_cast<__nv_bfloat162*>(dst)[j] = o;
    }
  }
  const bf16* vsrc = row + (size_t)(g.Hq + g.Hkv) * hd;
  for (int e = threadIdx.x; e < g.Hkv * half; e += blockDim.x) {
    const int kh = e / half, j = e % half;
    bf16* dst = g.kv_layer + (((size_t)page * 2 + 1) * g.Hkv + kh) * 16 * hd + (size_t)slot * hd;
    reinterpret_cast<__nv_bfloat162*>(dst)[j] = reinterpret_cast<const __nv_bfloat162*>(vsrc + (size_t)kh * hd)[j];
  }
}

void launch_rope_append(const RopeGroup* groups, int n_groups, int max_B, cudaStream_t st) {
  if (n_groups == 0 || max_B == 0) return;
  launch_pdl(rope_append_kernel, dim3(max_B, n_groups), dim3(256), 0, st, groups);
}

// ------------------------------------------------------------------ ViT token assembly
constexpr int ASSEMBLE_ROWS = 8;           // token rows per block
__global__ void __launch_bounds__(256) assemble_kernel(const AssembleGroup* __restrict__ groups) {
  const AssembleGroup g = groups[blockIdx.y];
  const int row0 = blockIdx.x * ASSEMBLE_ROWS;
  if (row0 >= g.B * g.T) return;
  pdl_launch_dependents();
  pdl_wait();
  const int nrows = min(ASSEMBLE_ROWS, g.B * g.T - row0), vecs = g.d / 8;
#pragma unroll 2
  for (int idx = threadIdx.x; idx < nrows * vecs; idx += blockDim.x) {
    const int row = row0 + idx / vecs, i = idx % vecs;
    const int b = row / g.T, t = row % g.T;
    const bf16* src = (t == 0) ? g.cls : g.E + ((size_t)b * (g.T - 1) + (t - 1)) * g.d;
    float a[8], p[8];
    unpack8(reinterpret_cast<const uint4*>(src)[i], a);
    unpack8(reinterpret_cast<const uint4*>(g.pos + (size_t)t * g.d)[i], p);
    float4* z = reinterpret_cast<float4*>(g.z + (size_t)row * g.d);
    z[2 * i] = make_float4(a[0] + p[0], a[1] + p[1], a[2] + p[2], a[3] + p[3]);
    z[2 * i + 1] = make_float4(a[4] + p[4], a[5] + p[5], a[6] + p[6], a[7] + p[7]);
  }
}

void launch_assemble(const AssembleGroup* groups, int n_groups, int max_rows, cudaStream_t st) {
  if (n_groups == 0 || max_rows == 0) return;
  launch_pdl(assemble_kernel, dim3((max_rows + ASSEMBLE_ROWS - 1) / ASSEMBLE_ROWS, n_groups), dim3(256), 0, st, groups);
}

// ------------------------------------------------------------------ output scatter + argmax
// One block per request: copies its logits row to the request's buffer and writes the index of
// the maximum (lowest index on ties; NaNs never win).  Rows are read 8 values (16 bytes) at a time.
constexpr int OUT_THREADS = 512;
__global__ void __launch_bounds__(OUT_THREADS) output_kernel(const OutputGroup* __restrict__ groups) {
  __shared__ float sv[OUT_THREADS / 32];
  __shared__ int si[OUT_THREADS / 32];
  const OutputGroup g = groups[blockIdx.y];
  const int b = blockIdx.x;
  if (b >= g.B) return;
  pdl_launch_dependents();
  pdl_wait();
  const ReqDesc r = g.reqs[b];
  const bf16* src = g.logits + (size_t)b * g.ld;          // 16-byte aligned: ld is a multiple of 8
  bf16* dst = reinterpret_cast<bf16*>(r.out_logits);
  const bool dst_vec = dst && (reinterpret_cast<uintptr_t>(dst) & 15) == 0;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  const int nvec = g.N >> 3;
  for (int i = threadIdx.x; i < nvec; i += OUT_THREADS) {
    const uint4 u = reinterpret_cast<const uint4*>(src)[i];
    if (dst_vec) {
      reinterpret_cast<uint4*>(dst)[i] = u;
    } else if (dst) {
      const bf16* e = reinterpret_cast<const bf16*>(&u);
#pragma unroll
      for (int k = 0; k < 8; ++k) dst[i * 8 + k] = e[k];
    }
    float f[8];
    unpack8(u, f);
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (f[k] > best || (f[k] == best && bi == 0x7fffffff)) { best = f[k]; bi = i * 8 + k; }   // ascending index: the first maximum stays
  }
  for (int i = (nvec << 3) + threadIdx.x; i < g.N; i += OUT_THREADS) {   // ragged end
    const bf16 v = src[i];
    if (dst) dst[i] = v;
    const float f = bf2f(v);
    if (f > best || (f == best && i < bi)) { best = f; bi = i; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
  }
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { sv[w] = best; si[w] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < OUT_THREADS / 32; ++k)
      if (sv[k] > best || (sv[k] == best && si[k] < bi)) { best = sv[k]; bi = si[k]; }
    if (bi == 0x7fffffff) bi = 0;
    if (r.out_argmax) *r.out_argmax = bi;
  }
}

void launch_output(const OutputGroup* groups, int n_groups, int max_B, cudaStream_t st) {
  if (n_groups == 0 || max_B == 0) return;
  launch_pdl(output_kernel, dim3(max_B, n_groups), dim3(OUT_THREADS), 0, st, groups);
}

}  // namespace epara
