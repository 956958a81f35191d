// Encoder (bidirectional) attention on the sm_100a tensor cores, head dimension 64, up to 224 tokens.
//
// One persistent CTA per SM walks over (image, head) items.  Per item, with T tokens, KP = T rounded
// up to 16 key columns and one or two tiles of 128 query rows:
//   warp 0 (one lane)  TMA producer: the Q tiles (128 x 64), the K tile and the V tile (KP x 64) of the
//                      item straight out of the qkv activation matrix [rows, 3d] (128-byte swizzle);
//   warp 1 (one lane)  MMA issuer: S_m = Q_m K^T (tcgen05.mma M 128, N KP, K 64) into TMEM for both
//                      query tiles, later O_m = P_m V (M 128, N 64, K KP) into a third TMEM region;
//   warps 2..13        384 workers; thread = (query row, part of the key columns).  V is consumed by the MMA as the TMA wrote it
//                      (tokens x 64 is the MN-major form of the B operand); the workers only zero its rows
//                      >= T.  Softmax: the thread reads its part of the row of S from TMEM once and keeps it in
//                      registers: maximum (the parts meet in shared memory), then p = exp2((s - max) * scale)
//                      with the row sum in fp32; P goes to shared memory as bf16 in the K-major
//                      128-byte-swizzled layout the MMA reads as its A operand.  Key columns >= T are masked
//                      by selection.  Last two of the three parts read half of O each from TMEM, divide by the row sum and
//                      store bf16 (rows >= T are not stored).
// Rows of the Q / K / V tiles past the image's T tokens belong to the next image or lie past the matrix
// (TMA fills those with zeros); they only ever reach masked columns, zeroed V^T columns or rows that
// are not stored.  Every mbarrier wait is bounded: when one runs out the kernel records a code in
// *status, all roles leave their loops, TMEM is freed and the kernel returns.
#include "common.cuh"
#include "kernels.h"
#include "tcgen05.cuh"

namespace epara {

namespace {

using namespace tc;

constexpr int ET_NS = 3;                              // worker threads per query row: each takes a part of the key columns
constexpr int ET_WORKERS = 128 * ET_NS;
constexpr int ET_THREADS = 64 + ET_WORKERS;
constexpr int ET_NB = (ENC_TC_MAX_T / 16 + ET_NS - 1) / ET_NS;   // 16-column blocks per thread at most (5)
constexpr int ET_OUT_PARTS = 2;                       // parts that store output: 32 of the 64 dims each
constexpr int ET_Q_BYTES = 128 * 128;                 // one query tile: 128 rows of 128 bytes
constexpr int ET_KV_BYTES = ENC_TC_MAX_T * 128;       // K or V tile at the largest KP (224 rows)
constexpr int ET_P_BLOCK = 128 * 128;                 // P: one 64-key block = 128 rows of 128 bytes
constexpr int ET_OFF_Q = 0;
constexpr int ET_OFF_K = 2 * ET_Q_BYTES;
constexpr int ET_OFF_V = ET_OFF_K + ET_KV_BYTES;
constexpr int ET_OFF_P = ET_OFF_V + ET_KV_BYTES;
constexpr int ET_OFF_L = ET_OFF_P + 4 * ET_P_BLOCK;   // partial row sums [2 tiles][parts][128] fp32, then partial maxima (4 KB each at most)
constexpr int ET_OFF_BAR = ET_OFF_L + 8192;
static_assert(2 * 2 * ET_NS * 128 * 4 <= 8192, "row sums and maxima");
constexpr size_t ET_SMEM = 1024 + ET_OFF_BAR + 256;
static_assert(ET_OFF_V % 1024 == 0 && ET_OFF_P % 1024 == 0, "swizzle atoms are 1024 bytes");
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// TMEM columns: S_0 and S_1.  O_m = P_m V is written over the first 64 columns of S_m, which the softmax
// has read out by then; the next item's S_m waits until O_m has been read out in turn.
constexpr int ET_S_COL0 = 0, ET_S_COL1 = 256;

enum { B_FULL_QK = 0, B_FULL_V, B_QK_FREE, B_V_FREE, B_S_FULL0, B_S_FULL1,
       B_P_READY0, B_P_READY1, B_O_FULL0, B_O_FULL1, B_O_EMPTY0, B_O_EMPTY1, B_MX0, B_MX1, B_COUNT };

// V tile as the B operand of P V: tokens (the K dimension of the MMA) x 64 dims (N), dims contiguous =
// MN-major.  Rows of 128 bytes, 128-byte swizzle, 8-token groups 1024 bytes apart; N = 64 is a single
// 128-byte row, so the only stride in play is the one between 8-token groups (given in both offset fields).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)(1024 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

struct ItemRef {
  const AttnEncGroup* g;
  int b, h;
};
__device__ __forceinline__ ItemRef find_item(const AttnEncGroup* groups, int n_groups, int item) {
  int gi = 0;
  for (int i = 1; i < n_groups; ++i) if (item >= groups[i].blk_start) gi = i;
  ItemRef r;
  r.g = groups + gi;
  const int local = item - r.g->blk_start;
  r.b = local / r.g->H;
  r.h = local - r.b * r.g->H;
  return r;
}

__global__ void __launch_bounds__(ET_THREADS, 1)
attn_encoder_tc_kernel(const AttnEncGroup* __restrict__ groups, int n_groups, int total_items, int* __restrict__ status) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bars = base + ET_OFF_BAR;
  auto bar = [&](int i) { return bars + 8u * i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + ET_OFF_BAR + 8 * B_COUNT);
  static_assert(8 * B_COUNT + 16 <= 256, "barrier area");
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* sm_l = reinterpret_cast<float*>(base_ptr + ET_OFF_L);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    mbar_init(bar(B_FULL_QK), 1); mbar_init(bar(B_FULL_V), 1); mbar_init(bar(B_QK_FREE), 1);
    mbar_init(bar(B_V_FREE), 1);
    mbar_init(bar(B_S_FULL0), 1); mbar_init(bar(B_S_FULL1), 1);
    mbar_init(bar(B_P_READY0), ET_WORKERS); mbar_init(bar(B_P_READY1), ET_WORKERS);
    mbar_init(bar(B_O_FULL0), 1); mbar_init(bar(B_O_FULL1), 1);
    mbar_init(bar(B_O_EMPTY0), ET_WORKERS); mbar_init(bar(B_O_EMPTY1), ET_WORKERS);
    mbar_init(bar(B_MX0), ET_WORKERS); mbar_init(bar(B_MX1), ET_WORKERS);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                  // the qkv matrix comes from the kernel before this one

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      const AttnEncGroup* g_prev = nullptr;
      uint32_t it = 0;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++it) {
        const ItemRef r = find_item(groups, n_groups, item);
        const AttnEncGroup* g = r.g;
        if (g != g_prev) { tensormap_acquire(&g->tmQ); tensormap_acquire(&g->tmKV); g_prev = g; }
        const int T = g->T, KP = g->KP, d = g->H * 64, n_mt = (T + 127) >> 7;
        const int row0 = r.b * T;
        // Q and K: free once both S = Q K^T of the previous item are complete
        if (!mbar_wait<false>(bar(B_QK_FREE), (it & 1u) ^ 1u, abort_flag)) { ok = false; atomicExch(status, 11); break; }
        mbar_expect_tx(bar(B_FULL_QK), (uint32_t)(n_mt * ET_Q_BYTES + KP * 128));
        for (int m = 0; m < n_mt; ++m)
          tma_load_2d(base + ET_OFF_Q + m * ET_Q_BYTES, &g->tmQ, r.h * 64, row0 + m * 128, bar(B_FULL_QK));
        tma_load_2d(base + ET_OFF_K, &g->tmKV, d + r.h * 64, row0, bar(B_FULL_QK));
        // V: free once the last P V of the previous item is complete
        if (!mbar_wait<false>(bar(B_V_FREE), (it & 1u) ^ 1u, abort_flag)) { ok = false; atomicExch(status, 12); break; }
        mbar_expect_tx(bar(B_FULL_V), (uint32_t)(KP * 128));
        tma_load_2d(base + ET_OFF_V, &g->tmKV, 2 * d + r.h * 64, row0, bar(B_FULL_V));
      }
      if (!ok) *abort_flag = 1;
      // copies in flight when a wait gave up: the consumers have left, so nothing reads them; let them land
      if (!ok) {
        volatile int never = 0;
        mbar_wait<false>(bar(B_FULL_QK), (it & 1u), &never);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // Order of issue per item: P_0 V, P_1 V, then Q_0 K^T and Q_1 K^T of the NEXT item, each as soon as
    // the workers have read O_0 / O_1 out of the TMEM region it overwrites -- the scores of the next item
    // are waiting in TMEM when the softmax warps get there.
    // Barriers of the first query tile complete once per item, those of the second once per item with two
    // tiles: each has its own use counter (items of different models mix).
    if (lane == 0) {
      bool ok = true;
      uint32_t cnt_s[2] = {0, 0};               // S = Q K^T issued so far, per tile index
      uint32_t cnt_pv[2] = {0, 0};              // P V issued so far, per tile index
      uint32_t cnt_qk = 0;                      // items whose Q / K have been consumed
      // Q_m K^T of an item (its Q and K must have landed: caller waited FULL_QK)
      auto issue_s = [&](const AttnEncGroup* g, int m) -> bool {
        // the region still holds O_m of the previous item with this tile until the workers have read it
        if (!mbar_wait<false>(bar(B_O_EMPTY0 + m), (cnt_s[m] & 1u) ^ 1u, abort_flag)) { atomicExch(status, 14); return false; }
        tc_fence_after();
        const uint32_t idesc_s = make_idesc(g->KP);
        const uint64_t dq = make_smem_desc(base + ET_OFF_Q + m * ET_Q_BYTES), dk = make_smem_desc(base + ET_OFF_K);
        const uint32_t d_tmem = tmem_base + (uint32_t)(m ? ET_S_COL1 : ET_S_COL0);
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f16(d_tmem, dq + (uint64_t)(k * 2), dk + (uint64_t)(k * 2), idesc_s, k > 0 ? 1u : 0u);
        mma_commit(bar(B_S_FULL0 + m));
        ++cnt_s[m];
        return true;
      };
      auto wait_qk = [&]() -> bool {
        if (!mbar_wait<false>(bar(B_FULL_QK), cnt_qk & 1u, abort_flag)) { atomicExch(status, 13); return false; }
        tc_fence_after();
        ++cnt_qk;
        return true;
      };
      uint32_t it = 0;
      const AttnEncGroup* g_next = nullptr;
      if ((int)blockIdx.x < total_items) {
        g_next = find_item(groups, n_groups, blockIdx.x).g;
        const int n_mt = (g_next->T + 127) >> 7;
        ok = wait_qk();
        for (int m = 0; m < n_mt && ok; ++m) ok = issue_s(g_next, m);
        if (ok) mma_commit(bar(B_QK_FREE));     // arrives when every MMA issued so far is complete
      }
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++it) {
        const AttnEncGroup* g = g_next;
        const int KP = g->KP, n_mt = (g->T + 127) >> 7;
        const bool has_next = item + (int)gridDim.x < total_items;
        int n_mt_next = 0;
        if (has_next) {
          g_next = find_item(groups, n_groups, item + gridDim.x).g;
          n_mt_next = (g_next->T + 127) >> 7;
        }
        for (int m = 0; m < n_mt && ok; ++m) {
          if (!mbar_wait<false>(bar(B_P_READY0 + m), cnt_pv[m] & 1u, abort_flag)) { ok = false; atomicExch(status, 16); break; }
          tc_fence_after();                     // (P_READY also says that every worker has read S_m out)
          const uint32_t idesc_o = make_idesc(64) | (1u << 16);     // B operand MN-major
          const uint32_t d_tmem = tmem_base + (uint32_t)(m ? ET_S_COL1 : ET_S_COL0);
          const int ksteps = KP >> 4;
          for (int k = 0; k < ksteps; ++k) {
            const uint64_t dp = make_smem_desc(base + ET_OFF_P + (k >> 2) * ET_P_BLOCK) + (uint64_t)((k & 3) * 2);
            const uint64_t dv = make_smem_desc_mn(base + ET_OFF_V + k * 2048);   // 16 tokens = two 8-token groups
            mma_f16(d_tmem, dp, dv, idesc_o, k > 0 ? 1u : 0u);
          }
          mma_commit(bar(B_O_FULL0 + m));
          if (m == n_mt - 1) mma_commit(bar(B_V_FREE));     // V may be overwritten once this P V is complete
          ++cnt_pv[m];
        }
        // scores of the next item
        if (ok && has_next) {
          ok = wait_qk();
          for (int m = 0; m < n_mt_next && ok; ++m) ok = issue_s(g_next, m);
          if (ok) mma_commit(bar(B_QK_FREE));
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ workers (warps 2.., ET_WORKERS threads)
    // Thread (quarter, lane, part): query row quarter*32 + lane of the current tile, and one part of the
    // key columns for the softmax; parts 0 and 1 also store one half of the 64 output dims.
    const int quarter = warp & 3, row = quarter * 32 + lane, part = (warp - 2) >> 2;
    const int wtid = threadIdx.x - 64;
    const float scale = 1.4426950408889634f * 0.125f;       // log2(e) / sqrt(64)
    float* sm_mx = sm_l + 2 * ET_NS * 128;                  // [2 tiles][parts][128] partial row maxima
    bool ok = true;
    uint32_t it = 0;
    uint32_t cnt_m[2] = {0, 0};                             // tiles processed so far, per tile index
    int prev_last = -1;                                     // last tile index of the previous item
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++it) {
      const ItemRef r = find_item(groups, n_groups, item);
      const AttnEncGroup* g = r.g;
      const int T = g->T, KP = g->KP, d = g->H * 64, n_mt = (T + 127) >> 7;
      // ---- softmax of the item's tiles: this thread's half of the key columns
      // the KP / 16 blocks of 16 columns are dealt to the parts as evenly as possible
      const int nb = KP >> 4, nb_lo = nb / ET_NS, nb_rem = nb % ET_NS;
      const int b_lo = part * nb_lo + min(part, nb_rem);
      const int c_lo = b_lo * 16, c_hi = c_lo + (nb_lo + (part < nb_rem ? 1 : 0)) * 16;
      for (int m = 0; m < n_mt && ok; ++m) {
        if (!mbar_wait<false>(bar(B_S_FULL0 + m), cnt_m[m] & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 18); break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(m ? ET_S_COL1 : ET_S_COL0);
        // The thread's half of the row (at most 112 columns) is read from TMEM once, all loads in flight
        // together, and stays in registers for both the maximum and the exponentials.
        const int n16 = (c_hi - c_lo) >> 4;                 // 16-column blocks of this part: 0..ET_NB
        uint32_t v[16 * ET_NB];
#pragma unroll
        for (int b16 = 0; b16 < ET_NB; ++b16)
          if (b16 < n16) tmem_ld16_nowait(taddr + (uint32_t)(c_lo + 16 * b16), v + 16 * b16);
        tmem_ld_wait();
#pragma unroll
        for (int b16 = 0; b16 < ET_NB; ++b16) tmem_regs_ready16(v + 16 * b16);
        tc_fence_before();                                  // (this thread's reads of S_m are over; P_READY tells the MMA warp)
        // row maximum (four independent chains); columns past the image become -inf (uniform branch per block)
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int b16 = 0; b16 < ET_NB; ++b16) {
          if (b16 >= n16) break;
          const int c = c_lo + 16 * b16;
          if (c + 16 > T) {
#pragma unroll
            for (int j = 0; j < 16; ++j) if (c + j >= T) v[16 * b16 + j] = 0xff800000u;
          }
#pragma unroll
          for (int j = 16 * b16; j < 16 * b16 + 16; j += 4) {
            mx0 = fmaxf(mx0, __uint_as_float(v[j])); mx1 = fmaxf(mx1, __uint_as_float(v[j + 1]));
            mx2 = fmaxf(mx2, __uint_as_float(v[j + 2])); mx3 = fmaxf(mx3, __uint_as_float(v[j + 3]));
          }
        }
        sm_mx[(m * ET_NS + part) * 128 + row] = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        // the two halves of a row meet here (an mbarrier, so that the wait is bounded like all others)
        mbar_arrive(bar(B_MX0 + m));
        if (!mbar_wait<false>(bar(B_MX0 + m), cnt_m[m] & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 22); break; }
        float mx = sm_mx[(m * ET_NS) * 128 + row];
#pragma unroll
        for (int p2 = 1; p2 < ET_NS; ++p2) mx = fmaxf(mx, sm_mx[(m * ET_NS + p2) * 128 + row]);
        const float nms = -mx * scale;
        // P may be overwritten once the P V of the tile before this one is complete
        if (m > 0 || prev_last >= 0) {
          const int pm = m > 0 ? 0 : prev_last;
          if (!mbar_wait<false>(bar(B_O_FULL0 + pm), (cnt_m[pm] - 1u) & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 19); break; }
        }
        // p = exp2(s * scale - max * scale), row sum, bf16 P in the swizzled K-major layout
        float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
        unsigned char* prow = base_ptr + ET_OFF_P + (row >> 3) * 1024 + (row & 7) * 128;
        const int sw = row & 7;
#pragma unroll
        for (int i = 0; i < 2 * ET_NB; ++i) {               // 16-byte pieces of 8 keys; piece index kc, block kc / 8
          if (i >= 2 * n16) break;
          const float p0 = ex2_approx(fmaf(__uint_as_float(v[8 * i]), scale, nms));
          const float p1 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 1]), scale, nms));
          const float p2 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 2]), scale, nms));
          const float p3 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 3]), scale, nms));
          const float p4 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 4]), scale, nms));
          const float p5 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 5]), scale, nms));
          const float p6 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 6]), scale, nms));
          const float p7 = ex2_approx(fmaf(__uint_as_float(v[8 * i + 7]), scale, nms));
          l0 += p0 + p4; l1 += p1 + p5; l2 += p2 + p6; l3 += p3 + p7;
          const int kc = (c_lo >> 3) + i;
          *reinterpret_cast<uint4*>(prow + (kc >> 3) * ET_P_BLOCK + (((kc & 7) ^ sw) << 4)) =
              make_uint4(pack2(p0, p1), pack2(p2, p3), pack2(p4, p5), pack2(p6, p7));
        }
        sm_l[(m * ET_NS + part) * 128 + row] = (l0 + l1) + (l2 + l3);
        if (m == 0) {
          // V is consumed by the tensor core as the TMA wrote it.  Its rows T .. KP-1 are another image's tokens
          // or stale memory; they meet P columns that are exactly zero, but 0 x NaN is NaN: zero them before the
          // first tile's P is reported (every P V of the item is issued after that report).  Waiting for V
          // only here leaves its load, which starts when the previous item's last P V is done, a whole
          // softmax to arrive.
          if (!mbar_wait<false>(bar(B_FULL_V), it & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 20); break; }
          if (wtid < (KP - T) * 8)
            *reinterpret_cast<uint4*>(base_ptr + ET_OFF_V + (T + (wtid >> 3)) * 128 + (wtid & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();                      // P (and the zeroed V rows) must be visible to the tensor core's reads
        mbar_arrive(bar(B_P_READY0 + m));
        ++cnt_m[m];
      }
      // ---- outputs: parts 0 and 1 read one half of the 64 dims of their row, for each tile
      for (int m = 0; m < n_mt && ok; ++m) {
        if (!mbar_wait<false>(bar(B_O_FULL0 + m), (cnt_m[m] - 1u) & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 21); break; }
        if (part >= ET_OUT_PARTS) { mbar_arrive(bar(B_O_EMPTY0 + m)); continue; }
        tc_fence_after();
        const uint32_t oaddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((m ? ET_S_COL1 : ET_S_COL0) + part * 32);
        uint32_t o[32];
        tmem_ld32(oaddr, o);
        tc_fence_before();
        mbar_arrive(bar(B_O_EMPTY0 + m));                   // the next item's S_m may overwrite the region
        const int q = m * 128 + row;
        if (q < T) {
          // (all parts' sums were published before P_READY, which the P V -- and so O_FULL -- waited for)
          float l = sm_l[(m * ET_NS) * 128 + row];
#pragma unroll
          for (int p2 = 1; p2 < ET_NS; ++p2) l += sm_l[(m * ET_NS + p2) * 128 + row];
          const float inv = 1.0f / l;
          uint4* dst = reinterpret_cast<uint4*>(g->out + ((size_t)r.b * T + q) * d + (size_t)r.h * 64 + part * 32);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            dst[k] = make_uint4(pack2(__uint_as_float(o[8 * k]) * inv, __uint_as_float(o[8 * k + 1]) * inv),
                                pack2(__uint_as_float(o[8 * k + 2]) * inv, __uint_as_float(o[8 * k + 3]) * inv),
                                pack2(__uint_as_float(o[8 * k + 4]) * inv, __uint_as_float(o[8 * k + 5]) * inv),
                                pack2(__uint_as_float(o[8 * k + 6]) * inv, __uint_as_float(o[8 * k + 7]) * inv));
        }
      }
      prev_last = n_mt - 1;
    }
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace

cudaError_t launch_attn_encoder_tc(const AttnEncGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                                   cudaStream_t st) {
  if (n_groups == 0 || total_items == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(attn_encoder_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ET_SMEM);
  if (e != cudaSuccess) return e;
  const int grid = total_items < sm_count ? total_items : sm_count;
  return launch_pdl(attn_encoder_tc_kernel, dim3(grid), dim3(ET_THREADS), ET_SMEM, st, groups, n_groups, total_items, status);
}

}  // namespace epara
