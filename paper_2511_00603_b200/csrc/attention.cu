// Attention kernels.
//
// Decode (one query token per request, paged KV cache, GQA): the KV axis of every request is
// cut into fixed chunks of ATTN_CHUNK tokens; one block handles (chunk, kv head, request) for
// all G query heads that share the kv head, so every K/V byte is read once.  The chunk size is
// a constant, hence a request's reduction order never depends on what else is in the step.
// A page's (K or V, head) tile is 16 x hd contiguous bf16; a warp reads it with 128-bit loads,
// lanes covering consecutive 16-byte pieces.  Partials (m, l, o) go to scratch and a second
// kernel merges the chunks in order.
//
// Encoder (ViT): full bidirectional attention of T tokens per (image, head).
#include "common.cuh"
#include "kernels.h"

namespace epara {

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

template <int HD, int G>
__global__ void __launch_bounds__(128) attn_decode_kernel(const AttnDecGroup* __restrict__ groups, int n_groups) {
  constexpr int LPT = HD / 8;        // lanes per token row
  constexpr int TPW = 32 / LPT;      // tokens per warp-wide load
  constexpr int NL = 16 / TPW;       // loads per page tile
  constexpr float LOG2E = 1.4426950408889634f;

  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.z >= groups[i].req_start) gi = i;
  const AttnDecGroup& g = groups[gi];
  const int b = blockIdx.z - g.req_start;
  const int kvh = blockIdx.y;
  if (kvh >= g.Hkv) return;
  const AttnReq rq = g.reqs[b];
  const int chunk = blockIdx.x;
  const int t_begin = chunk * ATTN_CHUNK;
  if (t_begin >= rq.len) return;
  const int t_end = min(rq.len, t_begin + ATTN_CHUNK);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = lane % LPT, ts = lane / LPT;

  // q of the G heads sharing this kv head, pre-scaled by log2(e)/sqrt(hd)
  float q[G][8];
  const float scale = LOG2E * rsqrtf((float)HD);
#pragma unroll
  for (int h = 0; h < G; ++h) {
    const uint4 u = *reinterpret_cast<const uint4*>(g.q + (size_t)b * g.q_stride + (size_t)(kvh * G + h) * HD + c * 8);
    unpack8(u, q[h]);
#pragma unroll
    for (int e = 0; e < 8; ++e) q[h][e] *= scale;
  }
  float m[G], l[G], acc[G][8];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -1e30f; l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[h][e] = 0.f;
  }

  const int page_begin = t_begin / 16, page_end = (t_end + 15) / 16;
  for (int pg = page_begin + warp; pg < page_end; pg += 4) {
    const int page = rq.table[pg];
    const uint4* kt = reinterpret_cast<const uint4*>(g.kv_layer + (((size_t)page * 2 + 0) * g.Hkv + kvh) * 16 * HD);
    const uint4* vt = reinterpret_cast<const uint4*>(g.kv_layer + (((size_t)page * 2 + 1) * g.Hkv + kvh) * 16 * HD);
    uint4 kr[NL], vr[NL];
#pragma unroll
    for (int i = 0; i < NL; ++i) kr[i] = ldg_stream(kt + i * 32 + lane);
#pragma unroll
    for (int i = 0; i < NL; ++i) vr[i] = ldg_stream(vt + i * 32 + lane);
    float s[NL][G];
#pragma unroll
    for (int i = 0; i < NL; ++i) {
      float kf[8];
      unpack8(kr[i], kf);
      const bool valid = (pg * 16 + i * TPW + ts) < t_end;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) d = fmaf(q[h][e], kf[e], d);
#pragma unroll
        for (int o = 1; o < LPT; o <<= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        s[i][h] = valid ? d : -INFINITY;
      }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
      float mn = m[h];
#pragma unroll
      for (int i = 0; i < NL; ++i) mn = fmaxf(mn, s[i][h]);
      const float sc = exp2f(m[h] - mn);
      m[h] = mn;
      l[h] *= sc;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[h][e] *= sc;
#pragma unroll
      for (int i = 0; i < NL; ++i) s[i][h] = exp2f(s[i][h] - mn);
    }
#pragma unroll
    for (int i = 0; i < NL; ++i) {
      float vf[8];
      unpack8(vr[i], vf);
      if ((pg * 16 + i * TPW + ts) >= t_end) {   // slots past the length may hold anything, NaN included
#pragma unroll
        for (int e = 0; e < 8; ++e) vf[e] = 0.f;
      }
#pragma unroll
      for (int h = 0; h < G; ++h) {
        l[h] += s[i][h];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[h][e] = fmaf(s[i][h], vf[e], acc[h][e]);
      }
    }
  }

  // merge the TPW token sub-groups of the warp (lanes that share c)
#pragma unroll
  for (int o = LPT; o < 32; o <<= 1) {
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float om = __shfl_xor_sync(0xffffffffu, m[h], o);
      const float ol = __shfl_xor_sync(0xffffffffu, l[h], o);
      const float mn = fmaxf(m[h], om);
      const float a = exp2f(m[h] - mn), bb = exp2f(om - mn);
      l[h] = l[h] * a + ol * bb;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float oa = __shfl_xor_sync(0xffffffffu, acc[h][e], o);
        acc[h][e] = acc[h][e] * a + oa * bb;
      }
      m[h] = mn;
    }
  }
  // merge the 4 warps through shared memory, in warp order
  __shared__ float sm_m[4][G], sm_l[4][G], sm_o[4][G][HD];
  if (ts == 0) {
#pragma unroll
    for (int h = 0; h < G; ++h) {
      if (c == 0) { sm_m[warp][h] = m[h]; sm_l[warp][h] = l[h]; }
#pragma unroll
      for (int e = 0; e < 8; ++e) sm_o[warp][h][c * 8 + e] = acc[h][e];
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * HD; idx += 128) {
    const int h = idx / HD, e = idx % HD;
    float mm = sm_m[0][h];
#pragma unroll
    for (int w = 1; w < 4; ++w) mm = fmaxf(mm, sm_m[w][h]);
    float ll = 0.f, oo = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float a = exp2f(sm_m[w][h] - mm);
      ll += sm_l[w][h] * a;
      oo += sm_o[w][h][e] * a;
    }
    float* dst = g.partial + (((size_t)b * g.Hq + (kvh * G + h)) * g.max_chunks + chunk) * (HD + 2);
    dst[2 + e] = oo;
    if (e == 0) { dst[0] = mm; dst[1] = ll; }
  }
}

// One block per (query head, request): merges the chunk partials in chunk order.
__global__ void attn_combine_kernel(const AttnDecGroup* __restrict__ groups, int n_groups) {
  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.y >= groups[i].req_start) gi = i;
  const AttnDecGroup& g = groups[gi];
  const int b = blockIdx.y - g.req_start, hq = blockIdx.x;
  if (hq >= g.Hq) return;
  const int HD = g.hd;
  const int n_chunks = (g.reqs[b].len + ATTN_CHUNK - 1) / ATTN_CHUNK;
  const float* p = g.partial + ((size_t)b * g.Hq + hq) * g.max_chunks * (HD + 2);
  float mm = -1e30f;
  for (int ch = 0; ch < n_chunks; ++ch) mm = fmaxf(mm, p[(size_t)ch * (HD + 2)]);
  for (int e = threadIdx.x; e < HD; e += blockDim.x) {
    float ll = 0.f, oo = 0.f;
    for (int ch = 0; ch < n_chunks; ++ch) {
      const float* pc = p + (size_t)ch * (HD + 2);
      const float a = exp2f(pc[0] - mm);
      ll += pc[1] * a;
      oo += pc[2 + e] * a;
    }
    g.out[((size_t)b * g.Hq + hq) * HD + e] = f2bf(oo / ll);
  }
}

template <int HD, int G>
static cudaError_t launch_dec(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_chunks,
                              cudaStream_t st) {
  attn_decode_kernel<HD, G><<<dim3(max_chunks, max_Hkv, total_B), 128, 0, st>>>(groups, n_groups);
  return cudaGetLastError();
}

cudaError_t launch_attn_decode(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_chunks,
                               int hd, int gqa, cudaStream_t st) {
  if (n_groups == 0 || total_B == 0) return cudaSuccess;
  if (total_B > 65535 || max_Hkv > 65535) return cudaErrorInvalidValue;
#define EPARA_DEC(HD_, G_) if (hd == HD_ && gqa == G_) return launch_dec<HD_, G_>(groups, n_groups, total_B, max_Hkv, max_chunks, st);
  EPARA_DEC(64, 1) EPARA_DEC(64, 2) EPARA_DEC(64, 4) EPARA_DEC(64, 8)
  EPARA_DEC(128, 1) EPARA_DEC(128, 2) EPARA_DEC(128, 4) EPARA_DEC(128, 8)
  EPARA_DEC(16, 1) EPARA_DEC(16, 2) EPARA_DEC(16, 4)
  EPARA_DEC(32, 1) EPARA_DEC(32, 2) EPARA_DEC(32, 4)
#undef EPARA_DEC
  return cudaErrorInvalidValue;
}

cudaError_t launch_attn_combine(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hq, int hd,
                                cudaStream_t st) {
  if (n_groups == 0 || total_B == 0) return cudaSuccess;
  attn_combine_kernel<<<dim3(max_Hq, total_B), hd < 32 ? 32 : hd, 0, st>>>(groups, n_groups);
  return cudaGetLastError();
}

__global__ void attn_fill_reqs_kernel(AttnReq* reqs, const int32_t* kv_lens, const int32_t* tables, int stride, int B) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) { reqs[b].table = tables + (size_t)b * stride; reqs[b].len = kv_lens[b]; reqs[b].pad = 0; }
}

void launch_attn_fill_reqs(AttnReq* reqs, const int32_t* kv_lens, const int32_t* tables, int stride, int B,
                           cudaStream_t st) {
  if (B == 0) return;
  attn_fill_reqs_kernel<<<(B + 127) / 128, 128, 0, st>>>(reqs, kv_lens, tables, stride, B);
}

// ------------------------------------------------------------------ encoder attention
// One block per (image, head, block of ENC_QB query rows); K and V of the head sit in shared
// memory as bf16; one thread per query row runs an online softmax over all T keys.
constexpr int ENC_QB = 64;
int attn_encoder_q_blocks(int T) { return (T + ENC_QB - 1) / ENC_QB; }

template <int HD>
__global__ void __launch_bounds__(ENC_QB) attn_encoder_kernel(const AttnEncGroup* __restrict__ groups, int n_groups) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.x >= groups[i].blk_start) gi = i;
  const AttnEncGroup& g = groups[gi];
  const int local = blockIdx.x - g.blk_start;
  const int qb = local % g.q_blocks, bh = local / g.q_blocks;
  const int h = bh % g.H, b = bh / g.H;
  const int T = g.T, d = g.H * HD;
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);
  bf16* Vs = Ks + (size_t)T * HD;
  const bf16* base = g.qkv + (size_t)b * T * 3 * d + (size_t)h * HD;
  for (int i = threadIdx.x; i < T * (HD / 8); i += blockDim.x) {
    const int t = i / (HD / 8), cc = i % (HD / 8);
    reinterpret_cast<uint4*>(Ks)[i] = *reinterpret_cast<const uint4*>(base + (size_t)t * 3 * d + d + cc * 8);
    reinterpret_cast<uint4*>(Vs)[i] = *reinterpret_cast<const uint4*>(base + (size_t)t * 3 * d + 2 * d + cc * 8);
  }
  __syncthreads();
  const int row = qb * ENC_QB + threadIdx.x;
  if (row >= T) return;
  float q[HD], o[HD];
  const float scale = 1.4426950408889634f * rsqrtf((float)HD);
#pragma unroll
  for (int cc = 0; cc < HD / 8; ++cc) {
    unpack8(*reinterpret_cast<const uint4*>(base + (size_t)row * 3 * d + cc * 8), q + cc * 8);
  }
#pragma unroll
  for (int e = 0; e < HD; ++e) { q[e] *= scale; o[e] = 0.f; }
  float m = -1e30f, l = 0.f;
  for (int t = 0; t < T; ++t) {
    float s = 0.f;
#pragma unroll
    for (int cc = 0; cc < HD / 8; ++cc) {
      float kf[8];
      unpack8(reinterpret_cast<const uint4*>(Ks + (size_t)t * HD)[cc], kf);
#pragma unroll
      for (int e = 0; e < 8; ++e) s = fmaf(q[cc * 8 + e], kf[e], s);
    }
    if (s > m) {
      const float sc = exp2f(m - s);
      l *= sc;
#pragma unroll
      for (int e = 0; e < HD; ++e) o[e] *= sc;
      m = s;
    }
    const float p = exp2f(s - m);
    l += p;
#pragma unroll
    for (int cc = 0; cc < HD / 8; ++cc) {
      float vf[8];
      unpack8(reinterpret_cast<const uint4*>(Vs + (size_t)t * HD)[cc], vf);
#pragma unroll
      for (int e = 0; e < 8; ++e) o[cc * 8 + e] = fmaf(p, vf[e], o[cc * 8 + e]);
    }
  }
  const float inv = 1.0f / l;
  bf16* out = g.out + ((size_t)b * T + row) * d + (size_t)h * HD;
#pragma unroll
  for (int cc = 0; cc < HD / 8; ++cc) {
    uint4 u;
    u.x = pack2(o[cc * 8 + 0] * inv, o[cc * 8 + 1] * inv);
    u.y = pack2(o[cc * 8 + 2] * inv, o[cc * 8 + 3] * inv);
    u.z = pack2(o[cc * 8 + 4] * inv, o[cc * 8 + 5] * inv);
    u.w = pack2(o[cc * 8 + 6] * inv, o[cc * 8 + 7] * inv);
    reinterpret_cast<uint4*>(out)[cc] = u;
  }
}

cudaError_t launch_attn_encoder(const AttnEncGroup* groups, int n_groups, int total_blocks, int max_T,
                                cudaStream_t st) {
  if (n_groups == 0 || total_blocks == 0) return cudaSuccess;
  const size_t smem = (size_t)max_T * 64 * 2 * sizeof(bf16);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(attn_encoder_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  attn_encoder_kernel<64><<<total_blocks, ENC_QB, smem, st>>>(groups, n_groups);
  return cudaGetLastError();
}

}  // namespace epara
