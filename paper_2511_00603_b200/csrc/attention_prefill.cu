// Causal attention of prompt chunks over the paged KV cache (the prefill phase of a decoder request).
//
// A request brings n_tok query tokens (rows row_start .. of the qkv matrix); token t sits at position
// kv_len + t and attends to positions 0 .. kv_len + t.  The chunk's own k, v have been appended to the
// cache by the RoPE kernel, so every key and value is read from the cache through the block table.
// One block of 4 warps per (request, query head, tile of 64 query tokens); warp w owns 16 query rows.
// Keys are walked in blocks of 64: K and V of the block are gathered page by page into shared memory with
// 16-byte cp.async copies (double-buffered: block kb + 1 loads while block kb is computed), rows padded
// by 8 elements so that ldmatrix reads are free of bank conflicts.  Per block: S = Q K^T on mma.sync
// m16n8k16 (bf16 in, fp32 accumulate), causal mask, online softmax in the exp2 domain, O += P V with P fed
// as a bf16 head plus a bf16 remainder.
// Keys past the chunk's reach are zero-filled and masked; a page id outside the pool is reported in the
// step's status word and its keys are treated the same way (never dereferenced).
// A token's result depends only on its own sequence: tiles and key blocks are fixed by (kv_len, t).
#include "common.cuh"
#include "kernels.h"

namespace epara {

namespace {

__device__ __forceinline__ void cp16_zfill(uint32_t dst, const void* src, bool valid) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm4(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_trans(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

constexpr int KB = 64;                       // keys per block

template <int HD>
__global__ void __launch_bounds__(128, 2) attn_prefill_kernel(const AttnPrefillGroup* __restrict__ groups, int n_groups) {
  constexpr int LD = HD + 8;                 // padded row length in shared memory (elements)
  constexpr int KS = HD / 16;                // k-steps of Q K^T
  constexpr int NT = HD / 8;                 // 8-wide tiles of the head dimension
  constexpr int CPR = HD / 8;                // 16-byte pieces per row
  constexpr int STAGE = 2 * KB * LD;         // elements per stage: K block then V block
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* sm = reinterpret_cast<bf16*>(smem_raw);

  pdl_launch_dependents();
  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if ((int)blockIdx.x >= groups[i].blk_start) gi = i;
  const AttnPrefillGroup& g = groups[gi];
  const int local = blockIdx.x - g.blk_start;
  if (local >= g.n_blocks) return;
  int ri = 0;
  for (int i = 1; i < g.n_reqs; ++i) if (local >= g.reqs[i].blk_start) ri = i;
  const PrefillReq rq = g.reqs[ri];
  const int tiles = (rq.n_tok + PREFILL_TILE - 1) / PREFILL_TILE;
  const int lb = local - rq.blk_start;
  const int hq = lb / tiles, tile = lb - hq * tiles;
  const int kvh = hq / (g.Hq / g.Hkv);
  const int Hkv = g.Hkv;
  const bf16* kv_layer = g.kv_layer;
  const long long kv_pages = g.kv_pages;
  pdl_wait();                                 // q and the chunk's k, v come from the kernels before this one

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gq = lane >> 2, tq = lane & 3;
  const int t0 = tile * PREFILL_TILE;
  const int tw0 = t0 + warp * 16;             // first query token of this warp
  const bool active = tw0 < rq.n_tok;
  // keys this block needs: positions 0 .. kv_len + (last token of the tile)
  const int n_keys = rq.kv_len + min(rq.n_tok, t0 + PREFILL_TILE);
  const int nblk = (n_keys + KB - 1) / KB;
  // the last key this warp's rows may see
  const int warp_last_key = rq.kv_len + min(rq.n_tok - 1, tw0 + 15);

  auto load_block = [&](int kb, int stage) {
    const uint32_t ks_u = (uint32_t)__cvta_generic_to_shared(sm + stage * STAGE);
    const uint32_t vs_u = ks_u + KB * LD * 2;
    for (int idx = threadIdx.x; idx < KB * CPR; idx += 128) {
      const int r = idx / CPR, c = idx - r * CPR;
      const int j = kb * KB + r;
      bool valid = j < n_keys;
      int page = 0;
      if (valid) {
        page = rq.table[j >> 4];
        if (page < 0 || page >= kv_pages) {   // outside the pool: reported, read as absent
          atomicExch(g.status, ERR_PAGE_ATTEND);
          valid = false;
          page = 0;
        }
      }
      const bf16* kp = kv_layer + (((size_t)page * 2 + 0) * Hkv + kvh) * 16 * HD + (size_t)(j & 15) * HD + c * 8;
      const bf16* vp = kp + (size_t)Hkv * 16 * HD;
      const uint32_t o = (uint32_t)(r * LD + c * 8) * 2u;
      cp16_zfill(ks_u + o, valid ? kp : kv_layer, valid);
      cp16_zfill(vs_u + o, valid ? vp : kv_layer, valid);
    }
  };

  load_block(0, 0);
  cp_commit();

  // Q fragments of the warp's 16 rows (rows past the chunk are clamped to its last token and never stored)
  uint32_t qa[KS][4];
  {
    const int r_lo = min(tw0 + gq, rq.n_tok - 1), r_hi = min(tw0 + gq + 8, rq.n_tok - 1);
    const bf16* q_lo = g.qkv + (size_t)(rq.row_start + r_lo) * g.q_stride + (size_t)hq * HD;
    const bf16* q_hi = g.qkv + (size_t)(rq.row_start + r_hi) * g.q_stride + (size_t)hq * HD;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = *reinterpret_cast<const uint32_t*>(q_lo + ks * 16 + 2 * tq);
      qa[ks][1] = *reinterpret_cast<const uint32_t*>(q_hi + ks * 16 + 2 * tq);
      qa[ks][2] = *reinterpret_cast<const uint32_t*>(q_lo + ks * 16 + 2 * tq + 8);
      qa[ks][3] = *reinterpret_cast<const uint32_t*>(q_hi + ks * 16 + 2 * tq + 8);
    }
  }
  const float scale = 1.4426950408889634f * rsqrtf((float)HD);
  float o[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m_lo = -1e30f, m_hi = -1e30f, l_lo = 0.f, l_hi = 0.f;
  const int lm_row = lane & 7, lm_mat = lane >> 3;
  // last key each of this lane's two rows may attend to (causal)
  const int lim_lo = rq.kv_len + tw0 + gq, lim_hi = lim_lo + 8;

  for (int kb = 0; kb < nblk; ++kb) {
    const int stage = kb & 1;
    cp_wait_all();                            // this thread's copies of block kb have landed ...
    __syncthreads();                          // ... everyone's have, and everyone is done with block kb - 1
    if (kb + 1 < nblk) load_block(kb + 1, stage ^ 1);
    cp_commit();
    if (!active || kb * KB > warp_last_key) continue;     // nothing in this block for this warp's rows
    const uint32_t ks_base = (uint32_t)__cvta_generic_to_shared(sm + stage * STAGE);
    const uint32_t vs_base = ks_base + KB * LD * 2;
    float sc[8][4];
#pragma unroll
    for (int n = 0; n < 8; ++n) { sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f; }
#pragma unroll
    for (int np = 0; np < 4; ++np) {
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int key = (2 * np + (lm_mat >> 1)) * 8 + lm_row;
        const int kcol = ks * 16 + (lm_mat & 1) * 8;
        uint32_t r[4];
        ldsm4(r, ks_base + (uint32_t)(key * LD + kcol) * 2u);
        mma16816(sc[2 * np], qa[ks], r[0], r[1]);
        mma16816(sc[2 * np + 1], qa[ks], r[2], r[3]);
      }
    }
    // causal mask: only blocks that reach past the smallest limit of the warp's rows need it
    if (kb * KB + KB - 1 > rq.kv_len + tw0) {
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        const int key = kb * KB + n * 8 + 2 * tq;
        if (key > lim_lo) sc[n][0] = -INFINITY;
        if (key + 1 > lim_lo) sc[n][1] = -INFINITY;
        if (key > lim_hi) sc[n][2] = -INFINITY;
        if (key + 1 > lim_hi) sc[n][3] = -INFINITY;
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
    for (int n = 0; n < NT; ++n) { o[n][0] *= a_lo; o[n][1] *= a_lo; o[n][2] *= a_hi; o[n][3] *= a_hi; }
    // P enters the tensor core as bf16; to keep fp32-level accuracy it is split into a bf16 head and a bf16
    // remainder (p = hi + lo up to 2^-17 relative) and P V is two MMAs per tile, as in the decode kernel
    uint32_t pa[4][4], pb[4][4];              // A fragments: 4 k-steps of 16 keys
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const float p0 = exp2f(fmaf(sc[n][0], scale, nm_lo)), p1 = exp2f(fmaf(sc[n][1], scale, nm_lo));
      const float p2 = exp2f(fmaf(sc[n][2], scale, nm_hi)), p3 = exp2f(fmaf(sc[n][3], scale, nm_hi));
      l_lo += p0 + p1;
      l_hi += p2 + p3;
      const uint32_t h01 = pack2(p0, p1), h23 = pack2(p2, p3);
      pa[n >> 1][(n & 1) * 2 + 0] = h01;
      pa[n >> 1][(n & 1) * 2 + 1] = h23;
      pb[n >> 1][(n & 1) * 2 + 0] = pack2(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xffff0000u));
      pb[n >> 1][(n & 1) * 2 + 1] = pack2(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xffff0000u));
    }
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        const int key = ks * 16 + (lm_mat & 1) * 8 + lm_row;
        const int col = (2 * np + (lm_mat >> 1)) * 8;
        uint32_t r[4];
        ldsm4_trans(r, vs_base + (uint32_t)(key * LD + col) * 2u);
        mma16816(o[2 * np], pa[ks], r[0], r[1]);
        mma16816(o[2 * np + 1], pa[ks], r[2], r[3]);
        mma16816(o[2 * np], pb[ks], r[0], r[1]);
        mma16816(o[2 * np + 1], pb[ks], r[2], r[3]);
      }
    }
  }
  cp_wait_all();
  if (!active) return;
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const float i_lo = 1.0f / l_lo, i_hi = 1.0f / l_hi;
  const int r_lo = tw0 + gq, r_hi = tw0 + gq + 8;
  const size_t ostride = (size_t)g.Hq * HD;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    if (r_lo < rq.n_tok)
      *reinterpret_cast<uint32_t*>(g.out + (size_t)(rq.row_start + r_lo) * ostride + (size_t)hq * HD + n * 8 + 2 * tq) =
          pack2(o[n][0] * i_lo, o[n][1] * i_lo);
    if (r_hi < rq.n_tok)
      *reinterpret_cast<uint32_t*>(g.out + (size_t)(rq.row_start + r_hi) * ostride + (size_t)hq * HD + n * 8 + 2 * tq) =
          pack2(o[n][2] * i_hi, o[n][3] * i_hi);
  }
}

template <int HD>
cudaError_t launch_prefill(const AttnPrefillGroup* groups, int n_groups, int total_blocks, cudaStream_t st) {
  constexpr int SMEM = 2 * 2 * KB * (HD + 8) * 2;
  cudaError_t e = cudaFuncSetAttribute(attn_prefill_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  return launch_pdl(attn_prefill_kernel<HD>, dim3(total_blocks), dim3(128), SMEM, st, groups, n_groups);
}

}  // namespace

cudaError_t launch_attn_prefill(const AttnPrefillGroup* groups, int n_groups, int total_blocks, int hd, cudaStream_t st) {
  if (n_groups == 0 || total_blocks == 0) return cudaSuccess;
  if (hd == 64) return launch_prefill<64>(groups, n_groups, total_blocks, st);
  if (hd == 128) return launch_prefill<128>(groups, n_groups, total_blocks, st);
  return cudaErrorInvalidValue;
}

}  // namespace epara
