// Attention kernels.
//
// Decode (one query token per request, paged KV cache, GQA): the KV axis of every request is
// cut into fixed chunks of ATTN_CHUNK tokens; one block handles (chunk, kv head, request) for
// all G query heads that share the kv head, so every K/V byte is read once.  The chunk size is
// a constant, hence a request's reduction order never depends on what else is in the step.
// A page's (K or V, head) tile is 16 x hd contiguous bf16; a warp reads it with 128-bit loads,
// lanes covering consecutive 16-byte pieces.  Partials (m, l, o) go to scratch; the block of a
// (request, kv head) that finishes last merges the chunks in chunk order (finish_chunk).
//
// Encoder (ViT): full bidirectional attention of T tokens per (image, head).
#include <cstring>

#include "../../include/epara.h"
#include "common.cuh"
#include "kernels.h"

namespace epara {

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Merge of the chunk partials of one (request, query head) element e, in chunk order.  Every load is
// independent of the running sums: unrolled, they are all in flight together.
template <int HD>
__device__ __forceinline__ float merge_chunks(const float* p, int n_chunks, int e) {
  float mm = -1e30f;
#pragma unroll 8
  for (int ch = 0; ch < n_chunks; ++ch) mm = fmaxf(mm, __ldcg(p + (size_t)ch * (HD + 2)));
  float ll = 0.f, oo = 0.f;
#pragma unroll 8
  for (int ch = 0; ch < n_chunks; ++ch) {
    const float* pc = p + (size_t)ch * (HD + 2);
    const float a = exp2f(__ldcg(pc) - mm);
    ll += __ldcg(pc + 1) * a;
    oo += __ldcg(pc + 2 + e) * a;
  }
  return oo / ll;
}

// Last step of a decode-attention block: the four warps' (m, l, o) of this chunk sit in shared
// memory.  They are merged in warp order.  A request of a single chunk is finished right here.
// Otherwise the chunk's partial goes to scratch.  With `fused` a per-(request, kv head) counter is
// bumped and the block that arrives last (no block waits for another) merges all chunks in chunk
// order, writes the output and leaves the counter at zero for the next launch; without it a second
// kernel (attn_combine_kernel) does the same merge.  The arithmetic and its order are the same in both
// cases, so the result depends neither on which block is last nor on the mode.
template <int HD, int G>
__device__ __forceinline__ void finish_chunk(const AttnDecGroup& g, int b, int row, int kvh, int chunk, int len, int fused,
                                             const float (*sm_m)[G], const float (*sm_l)[G],
                                             const float (*sm_o)[G][HD]) {
  __shared__ int s_last;
  const int n_chunks = (len + ATTN_CHUNK - 1) / ATTN_CHUNK;
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
    if (n_chunks == 1) {
      g.out[((size_t)row * g.Hq + (kvh * G + h)) * HD + e] = f2bf(oo / ll);
    } else {
      float* dst = g.partial + (((size_t)b * g.Hq + (kvh * G + h)) * g.max_chunks + chunk) * (HD + 2);
      __stcg(dst + 2 + e, oo);
      if (e == 0) { __stcg(dst, mm); __stcg(dst + 1, ll); }
    }
  }
  if (n_chunks == 1 || !fused) return;
  __syncthreads();                      // all partials of the block are written ...
  if (threadIdx.x == 0) {
    __threadfence();                    // ... and visible device-wide before the arrival is counted
    int* cnt = g.counters + (size_t)b * g.Hkv + kvh;
    const int last = (atomicAdd(cnt, 1) == n_chunks - 1);
    if (last) atomicExch(cnt, 0);
    s_last = last;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int idx = threadIdx.x; idx < G * HD; idx += 128) {
    const int h = idx / HD, e = idx % HD;
    const float* p = g.partial + ((size_t)b * g.Hq + (kvh * G + h)) * g.max_chunks * (HD + 2);
    g.out[((size_t)row * g.Hq + (kvh * G + h)) * HD + e] = f2bf(merge_chunks<HD>(p, n_chunks, e));
  }
}

// Separate merge for launches with many blocks: one block per (query head, request) of more than one chunk.
template <int HD>
__global__ void __launch_bounds__(HD) attn_combine_kernel(const AttnDecGroup* __restrict__ groups, int n_groups) {
  pdl_launch_dependents();
  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.y >= groups[i].req_start) gi = i;
  const AttnDecGroup& g = groups[gi];
  const int b = blockIdx.y - g.req_start, hq = blockIdx.x;
  pdl_wait();
  if (hq >= g.Hq) return;
  const AttnReq rq = g.reqs[b];
  const int n_chunks = (rq.len + ATTN_CHUNK - 1) / ATTN_CHUNK;
  if (n_chunks == 1) return;            // finished by the attention kernel itself
  const float* p = g.partial + ((size_t)b * g.Hq + hq) * g.max_chunks * (HD + 2);
  const int e = threadIdx.x;
  g.out[((size_t)rq.row * g.Hq + hq) * HD + e] = f2bf(merge_chunks<HD>(p, n_chunks, e));
}

template <int HD, int G>
__global__ void __launch_bounds__(128) attn_decode_kernel(const AttnDecGroup* __restrict__ groups, int n_groups, int fused) {
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
  if (g.reqs_stable && blockIdx.x * ATTN_CHUNK >= g.reqs[b].len) return;   // nothing to do and nothing to wait for
  pdl_launch_dependents();
  pdl_wait();                 // q, the appended K/V row and (single-kernel entry) the request table come from earlier kernels
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
    const uint4 u = *reinterpret_cast<const uint4*>(g.q + (size_t)rq.row * g.q_stride + (size_t)(kvh * G + h) * HD + c * 8);
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
    if (page < 0 || page >= g.kv_pages) {          // outside the pool: reported, read as absent
      if (lane == 0) atomicExch(g.status, ERR_PAGE_ATTEND);
      continue;
    }
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
  finish_chunk<HD, G>(g, b, rq.row, kvh, chunk, rq.len, fused, sm_m, sm_l, sm_o);
}

// Tensor-core variant for hd 64 / 128.  Same work split (chunk, kv head, request; 4 warps, warp w
// takes pages w, w+4, w+8, w+12 of the chunk) and the same partial format, but the pages are
// brought into shared memory with 16-byte cp.async copies -- all of a warp's pages are in flight
// at once and no registers are tied up by loads -- and Q K^T and P V run on mma.sync m16n8k16
// with the G query heads of the kv head as the first G rows of the 16-row A operand.  Rows of a
// staged tile are 128-byte segments whose 16-byte pieces are XOR-swizzled by the token index, so
// ldmatrix reads are free of bank conflicts.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// 16-byte copy that writes zeros instead when `valid` is false (the source is not read then)
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, bool valid) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma_bf16_m16n8k16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

template <int HD, int G, int NSLOT>
__global__ void __launch_bounds__(128) attn_decode_mma_kernel(const AttnDecGroup* __restrict__ groups, int n_groups, int fused) {
  constexpr int ROWB = HD * 2;              // bytes per token row
  constexpr int TILE = 16 * ROWB;           // bytes per (K or V) page tile
  constexpr int CPR = HD / 8;               // 16-byte pieces per row
  constexpr int KS = HD / 16;               // k-steps of Q K^T
  constexpr float LOG2E = 1.4426950408889634f;
  extern __shared__ __align__(128) unsigned char dsm[];

  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.z >= groups[i].req_start) gi = i;
  const AttnDecGroup& g = groups[gi];
  const int b = blockIdx.z - g.req_start;
  const int kvh = blockIdx.y;
  if (kvh >= g.Hkv) return;
  if (g.reqs_stable && blockIdx.x * ATTN_CHUNK >= g.reqs[b].len) return;   // nothing to do and nothing to wait for
  pdl_launch_dependents();
  pdl_wait();                 // q, the appended K/V row and (single-kernel entry) the request table come from earlier kernels
  const AttnReq rq = g.reqs[b];
  const int chunk = blockIdx.x;
  const int t_begin = chunk * ATTN_CHUNK;
  if (t_begin >= rq.len) return;
  const int t_end = min(rq.len, t_begin + ATTN_CHUNK);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gq = lane >> 2, tq = lane & 3;
  const int Hkv = g.Hkv;
  const bf16* kv_layer = g.kv_layer;
  const long long kv_pages = g.kv_pages;
  uint32_t bad_mask = 0;                    // pages of this warp whose id was outside the pool (warp-uniform)

  // ---- issue all copies of this warp's pages (up to 4), one commit group per page
  unsigned char* wsm = dsm + warp * (NSLOT * 2 * TILE);
  const uint32_t wsm_u = (uint32_t)__cvta_generic_to_shared(wsm);
  const int page_begin = t_begin / 16, page_end = (t_end + 15) / 16;
  // page i of this warp goes to slot i % NSLOT; one commit group per page (empty past the end)
  auto issue = [&](int i) {
    const int pg = page_begin + warp + 4 * i;
    if (i < 4 && pg < page_end) {
      const int page = rq.table[pg];
      if (page < 0 || page >= kv_pages) {            // outside the pool: reported, read as absent
        if (lane == 0) atomicExch(g.status, ERR_PAGE_ATTEND);
        bad_mask |= 1u << i;
        cp_async_commit();
        return;
      }
      const unsigned char* kt = reinterpret_cast<const unsigned char*>(kv_layer + (((size_t)page * 2 + 0) * Hkv + kvh) * 16 * HD);
      const unsigned char* vt = reinterpret_cast<const unsigned char*>(kv_layer + (((size_t)page * 2 + 1) * Hkv + kvh) * 16 * HD);
      const uint32_t kd = wsm_u + (i % NSLOT) * 2 * TILE, vd = kd + TILE;
#pragma unroll
      for (int j = 0; j < (16 * CPR) / 32; ++j) {
        const int piece = j * 32 + lane, r = piece / CPR, c = piece % CPR;
        const uint32_t off = r * ROWB + (c & ~7) * 16 + (((c & 7) ^ (r & 7)) << 4);
        cp_async16(kd + off, kt + piece * 16);
        cp_async16(vd + off, vt + piece * 16);
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int i = 0; i < NSLOT; ++i) issue(i);

  // ---- Q fragments: rows 0..G-1 of the A operand are the query heads of this kv head
  uint32_t qa[KS][4];
  {
    const bf16* qrow = g.q + (size_t)rq.row * g.q_stride + (size_t)(kvh * G + gq) * HD;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = (gq < G) ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * tq) : 0u;
      qa[ks][2] = (gq < G) ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * tq) : 0u;
      qa[ks][1] = 0u;
      qa[ks][3] = 0u;
    }
  }
  const float scale = LOG2E * rsqrtf((float)HD);
  float o[HD / 8][4];
#pragma unroll
  for (int n = 0; n < HD / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m_run = -1e30f, l_run = 0.f;
  const int lm_row = lane & 7, lm_mat = lane >> 3;

  auto process = [&](int i) {
    const int pg = page_begin + warp + 4 * i;
    if (pg >= page_end || (bad_mask & (1u << i))) return;
    const uint32_t kd = wsm_u + (i % NSLOT) * 2 * TILE, vd = kd + TILE;
    const int tok0 = pg * 16;
    if (tok0 + 16 > t_end) {
      // slots past the length may hold anything (NaN included): zero those V rows
      const int valid = t_end - tok0;
      for (int piece = lane; piece < 16 * CPR; piece += 32) {
        const int r = piece / CPR, c = piece % CPR;
        if (r >= valid)
          *reinterpret_cast<uint4*>(wsm + (i % NSLOT) * 2 * TILE + TILE + r * ROWB + (c & ~7) * 16 + (((c & 7) ^ (r & 7)) << 4)) =
              make_uint4(0, 0, 0, 0);
      }
      __syncwarp();
    }
    // S = Q K^T for 16 tokens: two 8-token tiles
    float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int r = (lm_mat >> 1) * 8 + lm_row, c = ks * 2 + (lm_mat & 1);
      uint32_t kr[4];
      ldsm_x4(kr, kd + r * ROWB + (c & ~7) * 16 + (((c & 7) ^ (r & 7)) << 4));
      mma_bf16_m16n8k16(sc[0], qa[ks], kr[0], kr[1]);
      mma_bf16_m16n8k16(sc[1], qa[ks], kr[2], kr[3]);
    }
    // row gq of the tile: tokens tok0 + j*8 + 2*tq (+1)
    float s[4];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int t0 = tok0 + j * 8 + 2 * tq;
      s[2 * j] = (t0 < t_end) ? sc[j][0] * scale : -INFINITY;
      s[2 * j + 1] = (t0 + 1 < t_end) ? sc[j][1] * scale : -INFINITY;
    }
    float mx = fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3]));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float mn = fmaxf(m_run, mx);
    const float resc = exp2f(m_run - mn);
    m_run = mn;
    l_run *= resc;
#pragma unroll
    for (int n = 0; n < HD / 8; ++n) { o[n][0] *= resc; o[n][1] *= resc; }
    const float p0 = exp2f(s[0] - mn), p1 = exp2f(s[1] - mn), p2 = exp2f(s[2] - mn), p3 = exp2f(s[3] - mn);
    l_run += (p0 + p1) + (p2 + p3);
    // P enters the tensor core as bf16; to keep fp32-level accuracy it is split into a bf16 head
    // and a bf16 remainder (p = hi + lo up to 2^-17 relative), and P V is two MMAs per tile
    uint32_t pa[4], pb[4];
    pa[0] = pack2(p0, p1); pa[1] = 0u; pa[2] = pack2(p2, p3); pa[3] = 0u;
    pb[0] = pack2(p0 - __uint_as_float(pa[0] << 16), p1 - __uint_as_float(pa[0] & 0xffff0000u));
    pb[2] = pack2(p2 - __uint_as_float(pa[2] << 16), p3 - __uint_as_float(pa[2] & 0xffff0000u));
    pb[1] = 0u; pb[3] = 0u;
    // O += P V
#pragma unroll
    for (int np = 0; np < HD / 16; ++np) {
      const int r = (lm_mat & 1) * 8 + lm_row, c = 2 * np + (lm_mat >> 1);
      uint32_t vr[4];
      ldsm_x4_trans(vr, vd + r * ROWB + (c & ~7) * 16 + (((c & 7) ^ (r & 7)) << 4));
      mma_bf16_m16n8k16(o[2 * np], pa, vr[0], vr[1]);
      mma_bf16_m16n8k16(o[2 * np + 1], pa, vr[2], vr[3]);
      mma_bf16_m16n8k16(o[2 * np], pb, vr[0], vr[1]);
      mma_bf16_m16n8k16(o[2 * np + 1], pb, vr[2], vr[3]);
    }
  };
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    cp_async_wait<NSLOT - 1>();              // page i has landed (one group is committed per step)
    __syncwarp();
    process(i);
    __syncwarp();                            // the slot is free again
    issue(i + NSLOT);
  }

  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);

  // ---- merge the 4 warps through shared memory, in warp order (same layout as the SIMT kernel)
  __shared__ float sm_m[4][G], sm_l[4][G], sm_o[4][G][HD];
  if (gq < G) {
    if (tq == 0) { sm_m[warp][gq] = m_run; sm_l[warp][gq] = l_run; }
#pragma unroll
    for (int n = 0; n < HD / 8; ++n) {
      sm_o[warp][gq][n * 8 + 2 * tq] = o[n][0];
      sm_o[warp][gq][n * 8 + 2 * tq + 1] = o[n][1];
    }
  }
  __syncthreads();
  finish_chunk<HD, G>(g, b, rq.row, kvh, chunk, rq.len, fused, sm_m, sm_l, sm_o);
}

template <int HD, int G>
static cudaError_t launch_dec_mma(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_chunks,
                                  int fused, cudaStream_t st) {
  constexpr int NSLOT = 2;                           // pages in flight per warp
  constexpr int SMEM = 4 * NSLOT * 2 * 16 * HD * 2;  // 4 warps x NSLOT pages x (K + V) tiles
  cudaError_t e = cudaFuncSetAttribute(attn_decode_mma_kernel<HD, G, NSLOT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  return launch_pdl(attn_decode_mma_kernel<HD, G, NSLOT>, dim3(max_chunks, max_Hkv, total_B), dim3(128), SMEM, st, groups, n_groups, fused);
}

template <int HD, int G>
static cudaError_t launch_dec(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_chunks,
                              int fused, cudaStream_t st) {
  return launch_pdl(attn_decode_kernel<HD, G>, dim3(max_chunks, max_Hkv, total_B), dim3(128), 0, st, groups, n_groups, fused);
}

// Few blocks (up to two waves): the last block of a (request, kv head) merges the chunks itself and the
// step saves a launch.  Many blocks: the counter round trip at the end of every block costs more than
// a second kernel, so the merge runs as attn_combine_kernel.
bool attn_decode_fused(int total_B, int max_Hkv, int max_chunks, int sm_count) {
  return (long long)total_B * max_Hkv * max_chunks <= 10ll * sm_count;
}

cudaError_t launch_attn_decode(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_Hq,
                               int max_chunks, int hd, int gqa, int fused, cudaStream_t st) {
  if (n_groups == 0 || total_B == 0) return cudaSuccess;
  if (total_B > 65535 || max_Hkv > 65535) return cudaErrorInvalidValue;
  cudaError_t e = cudaErrorInvalidValue;
#define EPARA_DEC(HD_, G_) if (hd == HD_ && gqa == G_) e = launch_dec<HD_, G_>(groups, n_groups, total_B, max_Hkv, max_chunks, fused, st);
#define EPARA_DEC_MMA(HD_, G_) if (hd == HD_ && gqa == G_) e = launch_dec_mma<HD_, G_>(groups, n_groups, total_B, max_Hkv, max_chunks, fused, st);
  EPARA_DEC_MMA(64, 1) EPARA_DEC_MMA(64, 2) EPARA_DEC_MMA(64, 4) EPARA_DEC_MMA(64, 8)
  EPARA_DEC_MMA(128, 1) EPARA_DEC_MMA(128, 2) EPARA_DEC_MMA(128, 4) EPARA_DEC_MMA(128, 8)
#undef EPARA_DEC_MMA
  EPARA_DEC(16, 1) EPARA_DEC(16, 2) EPARA_DEC(16, 4)
  EPARA_DEC(32, 1) EPARA_DEC(32, 2) EPARA_DEC(32, 4)
#undef EPARA_DEC
  if (e != cudaSuccess || fused || max_chunks <= 1) return e;
  const dim3 grid(max_Hq, total_B);
  switch (hd) {
    case 16: return launch_pdl(attn_combine_kernel<16>, grid, dim3(16), 0, st, groups, n_groups);
    case 32: return launch_pdl(attn_combine_kernel<32>, grid, dim3(32), 0, st, groups, n_groups);
    case 64: return launch_pdl(attn_combine_kernel<64>, grid, dim3(64), 0, st, groups, n_groups);
    case 128: return launch_pdl(attn_combine_kernel<128>, grid, dim3(128), 0, st, groups, n_groups);
  }
  return cudaErrorInvalidValue;
}

// Set-up kernel of the single-kernel entry points.  It writes the group descriptor (passed by value, so
// that no host buffer has to outlive the call) to `dst`, clears the status word and the chunk counters,
// and fills the request table.  The lengths come from caller device memory: they are clamped to
// [0, max_len], the range the scratch and the tables were sized for, so that no chunk index can leave the
// partial buffer.  A request of length 0 attends to nothing and its output row is left unwritten.
__global__ void attn_prepare_kernel(AttnDecGroup g, AttnDecGroup* dst, AttnReq* reqs, const int32_t* kv_lens,
                                    const int32_t* tables, int stride, int max_len, int n_counters) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0) { *dst = g; *g.status = 0; }
  if (i < g.B) {
    reqs[i].table = tables + (size_t)i * stride;
    reqs[i].len = min(max(kv_lens[i], 0), max_len);
    reqs[i].row = i;
  }
  for (int c = i; c < n_counters; c += gridDim.x * blockDim.x) g.counters[c] = 0;
}

void launch_attn_prepare(const AttnDecGroup& g, AttnDecGroup* dst, AttnReq* reqs, const int32_t* kv_lens,
                         const int32_t* tables, int stride, int max_len, int n_counters, cudaStream_t st) {
  if (g.B == 0) return;
  attn_prepare_kernel<<<(g.B + 127) / 128, 128, 0, st>>>(g, dst, reqs, kv_lens, tables, stride, max_len, n_counters);
}

// ------------------------------------------------------------------ encoder attention
// One block per (image, head, block of up to 112 query rows); one warp per 16 query rows.
// K and V of the head are staged once in shared memory (bf16, rows padded to 72 elements so
// that ldmatrix rows fall in distinct banks); each warp runs a flash-style loop over 64-key
// blocks with mma.sync m16n8k16 (bf16 in, fp32 accumulate): S = Q K^T, online softmax in the
// exp2 domain, O += P V.  Keys beyond T are masked; their padded rows are zero.
constexpr int ENC_ROWS = 112;      // query rows per block (7 warps): two blocks share an SM
constexpr int ENC_LD = 72;         // padded row length of K and V in shared memory
int attn_encoder_q_blocks(int T) { return (T + ENC_ROWS - 1) / ENC_ROWS; }
static int enc_key_pad(int T) { return (T + 63) / 64 * 64; }

__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__global__ void __launch_bounds__(ENC_ROWS * 2, 2) attn_encoder_kernel(const AttnEncGroup* __restrict__ groups, int n_groups) {
  constexpr int HD = 64;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_launch_dependents();
  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.x >= groups[i].blk_start) gi = i;
  const AttnEncGroup& g = groups[gi];
  pdl_wait();
  const int local = blockIdx.x - g.blk_start;
  const int qb = local % g.q_blocks, bh = local / g.q_blocks;
  const int h = bh % g.H, b = bh / g.H;
  const int T = g.T, d = g.H * HD;
  const int Tp = (T + 63) / 64 * 64;
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);
  bf16* Vs = Ks + (size_t)Tp * ENC_LD;
  const bf16* base = g.qkv + (size_t)b * T * 3 * d + (size_t)h * HD;
  // K and V are brought in by cp.async, one commit group per block of 64 keys, all in flight at once;
  // the loop below waits for block after block, so the first scores start while later keys still load
  const int nblk = Tp >> 6;
  {
    const uint32_t ks_u = (uint32_t)__cvta_generic_to_shared(Ks), vs_u = (uint32_t)__cvta_generic_to_shared(Vs);
    for (int blk = 0; blk < nblk; ++blk) {
      for (int i = threadIdx.x; i < 64 * (HD / 8); i += blockDim.x) {
        const int t = blk * 64 + (i >> 3), cc = i & 7;
        const bool valid = t < T;
        const bf16* src = base + (size_t)(valid ? t : 0) * 3 * d + cc * 8;
        cp_async16_zfill(ks_u + (uint32_t)(t * ENC_LD + cc * 8) * 2u, src + d, valid);
        cp_async16_zfill(vs_u + (uint32_t)(t * ENC_LD + cc * 8) * 2u, src + 2 * d, valid);
      }
      cp_async_commit();
    }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = qb * ENC_ROWS + warp * 16;
  const bool active = row0 < T;             // idle warps still take part in the block barriers below
  const int gq = lane >> 2, tq = lane & 3;
  // Q fragments of the warp's 16 rows: 4 k-steps of 16
  uint32_t qa[4][4];
  {
    const int r_lo = row0 + gq, r_hi = row0 + gq + 8;
    const bf16* q_lo = base + (size_t)min(r_lo, T - 1) * 3 * d;
    const bf16* q_hi = base + (size_t)min(r_hi, T - 1) * 3 * d;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      qa[ks][0] = *reinterpret_cast<const uint32_t*>(q_lo + ks * 16 + 2 * tq);
      qa[ks][1] = *reinterpret_cast<const uint32_t*>(q_hi + ks * 16 + 2 * tq);
      qa[ks][2] = *reinterpret_cast<const uint32_t*>(q_lo + ks * 16 + 2 * tq + 8);
      qa[ks][3] = *reinterpret_cast<const uint32_t*>(q_hi + ks * 16 + 2 * tq + 8);
    }
  }
  const float scale = 1.4426950408889634f * rsqrtf((float)HD);
  float o[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m_lo = -1e30f, m_hi = -1e30f, l_lo = 0.f, l_hi = 0.f;
  const uint32_t ks_base = (uint32_t)__cvta_generic_to_shared(Ks);
  const uint32_t vs_base = (uint32_t)__cvta_generic_to_shared(Vs);
  // ldmatrix lane addressing: lanes 0-7 rows of matrix 0, 8-15 matrix 1, 16-23 matrix 2, 24-31 matrix 3
  const int lm_row = lane & 7, lm_mat = lane >> 3;
  for (int kb = 0; kb < Tp; kb += 64) {
    // at most (blocks after this one) copy groups may still be pending
    switch (nblk - 1 - (kb >> 6)) {
      case 0: cp_async_wait<0>(); break;
      case 1: cp_async_wait<1>(); break;
      case 2: cp_async_wait<2>(); break;
      case 3: cp_async_wait<3>(); break;
      case 4: cp_async_wait<4>(); break;
      case 5: cp_async_wait<5>(); break;
      case 6: cp_async_wait<6>(); break;
      default: cp_async_wait<7>(); break;
    }
    __syncthreads();
    if (!active) continue;
    // the last block of keys is ragged (197 = 3 x 64 + 5): only its 16-key groups that hold real keys are computed
    const int np_lim = (min(64, T - kb) + 15) >> 4;
    float sc[8][4];
#pragma unroll
    for (int n = 0; n < 8; ++n) { sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f; }
    // S = Q K^T : for key tiles (pairs of 8 keys) and k-steps
#pragma unroll
    for (int np = 0; np < 4; ++np) {        // key tiles 2np, 2np+1
      if (np >= np_lim) continue;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        // matrices: (keys 2np*8.., k lo), (keys 2np*8.., k hi), (keys (2np+1)*8.., k lo), (.., k hi)
        const int key = kb + (2 * np + (lm_mat >> 1)) * 8 + lm_row;
        const int kcol = ks * 16 + (lm_mat & 1) * 8;
        uint32_t r[4];
        ldmatrix_x4(r, ks_base + (uint32_t)(key * ENC_LD + kcol) * 2u);
        mma_bf16_16816(sc[2 * np], qa[ks], r[0], r[1]);
        mma_bf16_16816(sc[2 * np + 1], qa[ks], r[2], r[3]);
      }
    }
    // online softmax (rows gq and gq+8 of the warp tile).  The running maximum is kept in units of the raw
    // scores (the scale is positive), so that scaling and subtracting the maximum are one FMA per score;
    // only the ragged last block of keys needs masking.
    if (kb + 64 > T) {
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        const int key = kb + n * 8 + 2 * tq;
        if (key >= T) { sc[n][0] = -INFINITY; sc[n][2] = -INFINITY; }
        if (key + 1 >= T) { sc[n][1] = -INFINITY; sc[n][3] = -INFINITY; }
      }
    }
    float mx_lo = m_lo, mx_hi = m_hi;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      mx_lo = fmaxf(mx_lo, fmaxf(sc[n][0], sc[n][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(sc[n][2], sc[n][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float a_lo = exp2f((m_lo - mx_lo) * scale), a_hi = exp2f((m_hi - mx_hi) * scale);
    m_lo = mx_lo; m_hi = mx_hi;
    const float nm_lo = -m_lo * scale, nm_hi = -m_hi * scale;
    l_lo *= a_lo; l_hi *= a_hi;
#pragma unroll
    for (int n = 0; n < 8; ++n) { o[n][0] *= a_lo; o[n][1] *= a_lo; o[n][2] *= a_hi; o[n][3] *= a_hi; }
    uint32_t pa[4][4];                       // P as A fragments: 4 k-steps of 16 keys
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      if ((n >> 1) >= np_lim) continue;      // all keys of the group are masked: never read below
      const float p0 = exp2f(fmaf(sc[n][0], scale, nm_lo)), p1 = exp2f(fmaf(sc[n][1], scale, nm_lo));
      const float p2 = exp2f(fmaf(sc[n][2], scale, nm_hi)), p3 = exp2f(fmaf(sc[n][3], scale, nm_hi));
      l_lo += p0 + p1;
      l_hi += p2 + p3;
      pa[n >> 1][(n & 1) * 2 + 0] = pack2(p0, p1);
      pa[n >> 1][(n & 1) * 2 + 1] = pack2(p2, p3);
    }
    // O += P V : k = keys (4 steps of 16), n = head dims (8 tiles of 8)
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      if (ks >= np_lim) continue;
#pragma unroll
      for (int np = 0; np < 4; ++np) {      // dim tiles 2np, 2np+1
        // matrices: (keys lo 8, dims 2np*8..), (keys hi 8, dims 2np*8..), (keys lo, dims (2np+1)*8..), (keys hi, ..)
        const int key = kb + ks * 16 + (lm_mat & 1) * 8 + lm_row;
        const int col = (2 * np + (lm_mat >> 1)) * 8;
        uint32_t r[4];
        ldmatrix_x4_trans(r, vs_base + (uint32_t)(key * ENC_LD + col) * 2u);
        mma_bf16_16816(o[2 * np], pa[ks], r[0], r[1]);
        mma_bf16_16816(o[2 * np + 1], pa[ks], r[2], r[3]);
      }
    }
  }
  if (!active) return;
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const float i_lo = 1.0f / l_lo, i_hi = 1.0f / l_hi;
  const int r_lo = row0 + gq, r_hi = row0 + gq + 8;
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    if (r_lo < T)
      *reinterpret_cast<uint32_t*>(g.out + ((size_t)b * T + r_lo) * d + (size_t)h * HD + n * 8 + 2 * tq) =
          pack2(o[n][0] * i_lo, o[n][1] * i_lo);
    if (r_hi < T)
      *reinterpret_cast<uint32_t*>(g.out + ((size_t)b * T + r_hi) * d + (size_t)h * HD + n * 8 + 2 * tq) =
          pack2(o[n][2] * i_hi, o[n][3] * i_hi);
  }
}

cudaError_t launch_attn_encoder(const AttnEncGroup* groups, int n_groups, int total_blocks, int max_T,
                                cudaStream_t st) {
  if (n_groups == 0 || total_blocks == 0) return cudaSuccess;
  const size_t smem = (size_t)enc_key_pad(max_T) * ENC_LD * 2 * sizeof(bf16);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(attn_encoder_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  const int rows = max_T < ENC_ROWS ? max_T : ENC_ROWS;
  const int warps = (rows + 15) / 16;
  return launch_pdl(attn_encoder_kernel, dim3(total_blocks), dim3(warps * 32), smem, st, groups, n_groups);
}

}  // namespace epara

// ------------------------------------------------------------------ decode attention without caller scratch
// Scratch of epara_decode_attention_static: one array per GPU that loads this library, held until
// the process exits.  Host code may not hand `g_static_scratch` itself to a kernel (on the host the
// name is only a stand-in for the symbol); the device address is looked up once per device below.
namespace {
constexpr size_t STATIC_SCRATCH_BYTES = EPARA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];
constexpr int MAX_DEVICES = 64;
unsigned char* g_static_ptr[MAX_DEVICES] = {nullptr};
int g_static_sm[MAX_DEVICES] = {0};
}  // namespace

extern "C" int epara_decode_attention_static(int device, void* cuda_stream, const void* q, int q_stride,
                                             const void* kv_layer, long long kv_pages, const int32_t* kv_lens,
                                             const int32_t* tables, int table_stride, void* out, int B, int Hq, int Hkv,
                                             int hd, int max_len) {
  using namespace epara;
  if (!q || !kv_layer || !kv_lens || !tables || !out || B < 0 || Hkv <= 0 || Hq <= 0 || Hq % Hkv || max_len <= 0 || hd <= 0 ||
      kv_pages <= 0)
    return EPARA_E_INVALID;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(kv_layer) & 15) || (q_stride % 8))
    return EPARA_E_INVALID;
  if (device < 0 || device >= MAX_DEVICES) return EPARA_E_INVALID;
  const int chunks = (max_len + ATTN_CHUNK - 1) / ATTN_CHUNK;
  const size_t req_bytes = ((size_t)B * sizeof(AttnReq) + 255) / 256 * 256;
  const size_t part_bytes = ((size_t)B * Hq * chunks * (hd + 2) * sizeof(float) + 255) / 256 * 256;
  const size_t need = 256 + req_bytes + part_bytes + (size_t)B * Hq * sizeof(int);
  if (need > STATIC_SCRATCH_BYTES) return EPARA_E_RESOURCE;   // problem too large for the built-in scratch
  if (B == 0) return EPARA_OK;
  if (cudaSetDevice(device) != cudaSuccess) return EPARA_E_CUDA;
  if (!g_static_ptr[device]) {
    // first call on this device: resolve the device address of the array (this device is current)
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return EPARA_E_CUDA;
    int sm = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sm <= 0) return EPARA_E_CUDA;
    g_static_sm[device] = sm;
    g_static_ptr[device] = static_cast<unsigned char*>(p);
  }
  unsigned char* s = g_static_ptr[device];
  cudaStream_t st = (cudaStream_t)cuda_stream;
  AttnDecGroup g;
  memset(&g, 0, sizeof(g));
  AttnReq* reqs = reinterpret_cast<AttnReq*>(s + 256);
  g.q = (const bf16*)q; g.q_stride = q_stride; g.kv_layer = (const bf16*)kv_layer; g.reqs = reqs; g.out = (bf16*)out;
  g.partial = reinterpret_cast<float*>(s + 256 + req_bytes);
  g.counters = reinterpret_cast<int*>(s + 256 + req_bytes + part_bytes);
  g.B = B; g.Hq = Hq; g.Hkv = Hkv; g.hd = hd; g.max_chunks = chunks; g.req_start = 0;
  g.status = reinterpret_cast<int*>(s + DEC_STATUS_OFFSET);
  g.kv_pages = kv_pages;
  // The array keeps the previous call's contents.  The set-up kernel rewrites the descriptor and the
  // request table and clears the status word and the chunk counters (the parts that must start at
  // zero); every partial that is read is written first by this call's attention kernel.
  launch_attn_prepare(g, reinterpret_cast<AttnDecGroup*>(s), reqs, kv_lens, tables, table_stride, max_len, B * Hq, st);
  cudaError_t e = launch_attn_decode(reinterpret_cast<const AttnDecGroup*>(s), 1, B, Hkv, Hq, chunks, hd, Hq / Hkv,
                                     attn_decode_fused(B, Hkv, chunks, g_static_sm[device]) ? 1 : 0, st);
  if (e == cudaErrorInvalidValue) return EPARA_E_UNSUPPORTED;
  return e == cudaSuccess ? EPARA_OK : EPARA_E_CUDA;
}

extern "C" int epara_decode_attention_static_status(int device, int* code) {
  if (!code || device < 0 || device >= MAX_DEVICES) return EPARA_E_INVALID;
  *code = 0;
  if (!g_static_ptr[device]) return EPARA_OK;                 // never used on this device
  if (cudaSetDevice(device) != cudaSuccess) return EPARA_E_CUDA;
  if (cudaMemcpy(code, g_static_ptr[device] + epara::DEC_STATUS_OFFSET, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return EPARA_E_CUDA;
  return *code ? EPARA_E_DEVICE : EPARA_OK;
}

extern "C" size_t epara_static_scratch_bytes(void) { return STATIC_SCRATCH_BYTES; }

