// Grouped bf16 GEMM on the sm_100a tensor cores: C_g = epi(A_g W_g^T + bias_g).
//
// One persistent launch covers every group (one group = one model's GEMM in this wave, with its
// own M, N, K, tile width bn in {128, 256} and k-split count).  Work items -- (tile, k range) --
// are numbered group after group; CTA i takes items i, i + grid, ...  Inside a CTA three roles
// run concurrently:
//   warp 0 (one lane)  TMA producer: for each 64-wide k-block loads the A tile (128 x 64) and the
//                      W tile (bn x 64) into a ring of shared-memory stages (plain, non-multicast
//                      cp.async.bulk.tensor; out-of-range rows/columns arrive as zeros);
//   warp 1 (one lane)  MMA issuer: tcgen05.mma (M 128, N bn, K 16) from shared memory into one
//                      of two TMEM accumulators (256 columns each), releasing stages with
//                      tcgen05.commit;
//   warps 2..17        epilogue: tcgen05.ld of the finished accumulator (four warps per TMEM lane
//                      quarter, a quarter of the tile's columns each), bias / GELU / SwiGLU / fp32 residual
//                      update, bf16 store -- while the MMA warp already fills the other accumulator.
// Split-k (weight-streaming groups with few tiles): every k range of a tile writes its fp32
// partial; the range that finishes last (an atomic counter per tile, no waiting) adds the partials
// in range order and runs the epilogue, so the result does not depend on arrival order.
// The K reduction of an output element is the same sequence whatever else is in the launch.
// Every mbarrier wait is bounded: when a wait runs out the kernel records a code in *status, all
// roles leave their loops, TMEM is freed and the kernel returns.
//
// Two kernels share this pipeline and its epilogue: gemm_tc_kernel (one CTA per 128-row tile; groups of
// 17 to 128 rows and the split-k groups) and gemm_tc_pair_kernel further down (two CTAs of a cluster per
// 256-row tile, tcgen05 cta_group::2; every other group of more than 128 rows).
#include "common.cuh"
#include "kernels.h"
#include "tcgen05.cuh"

namespace epara {

namespace {

using namespace tc;

// The operand ring holds 192 KB: 4 stages of 48 KB (A 128 x 64 + W 256 x 64) when some group of the
// launch has 256-wide tiles, 6 stages of 32 KB when all tiles are 128 wide (more loads in flight for
// the weight-streaming groups).  The geometry is a launch parameter.
constexpr int MAX_STAGES = 6;
constexpr int A_BYTES = TC_BM * TC_BK * 2;          // 16 KB
constexpr int B_BYTES_MAX = TC_BN_MAX * TC_BK * 2;  // 32 KB
constexpr int RING_BYTES = 4 * (A_BYTES + B_BYTES_MAX);
constexpr int ACC_COLS = TC_BN_MAX;                 // TMEM columns per accumulator
constexpr int TMEM_COLS = 2 * ACC_COLS;             // 512: the whole TMEM of the SM
constexpr int EPI_WARPS = 16;
constexpr int N_THREADS = 64 + EPI_WARPS * 32;
constexpr int STAGE_OUT_BYTES = EPI_WARPS * 2048;    // epilogue staging: 2 KB (32 rows x 64 bytes) per warp
constexpr size_t SMEM_BYTES = 1024 + (size_t)RING_BYTES + STAGE_OUT_BYTES + 256;

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(EPI_WARPS * 32) : "memory"); }

__device__ __forceinline__ int find_group_tc(const GemmGroup* groups, int n, int item) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (groups[mid].tile_start <= item) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Register copy of a group's scalar fields for the epilogue threads.  The descriptors live in
// global memory and the epilogue is full of asm statements that clobber memory, so reading
// fields through the descriptor pointer would reload them (at L2 latency) again and again.
struct GView {
  const bf16* bias;
  void* C;
  float* partial;
  int* counters;
  const CUtensorMap* tmC;
  int M, N, K, ldc, epi, tile_start, tiles_m, tiles_n, bn, ksplit, c_rows;
};
__device__ __forceinline__ GView load_view(const GemmGroup* g) {
  GView v;
  v.bias = g->bias; v.C = g->C; v.partial = g->partial; v.counters = g->counters;
  v.M = g->M; v.N = g->N; v.K = g->K; v.ldc = g->ldc; v.epi = g->epi; v.tile_start = g->tile_start;
  v.tiles_m = g->tiles_m; v.tiles_n = g->tiles_n; v.bn = g->bn; v.ksplit = g->ksplit;
  v.tmC = &g->tmC; v.c_rows = g->c_rows;
  return v;
}

// A work item of a group: tile (tm, tn) and k-block range [kb0, kb1).
struct Item {
  int m0, n0, tile, split, kb0, kb1;
};
template <class G>
__device__ __forceinline__ Item decode_item(const G& g, int local) {
  Item it;
  it.split = local % g.ksplit;
  it.tile = local / g.ksplit;
  it.m0 = (it.tile / g.tiles_n) * TC_BM;
  it.n0 = (it.tile % g.tiles_n) * g.bn;
  const int kblocks = (g.K + TC_BK - 1) / TC_BK;
  const int per = (kblocks + g.ksplit - 1) / g.ksplit;
  it.kb0 = it.split * per;
  it.kb1 = min(kblocks, it.kb0 + per);
  return it;
}

// Per-thread copy of the fields the single-thread roles need, refreshed only when the item leaves
// the current group (descriptor reads from global memory are latency the MMA issuer cannot hide).
struct GroupCache {
  const GemmGroup* g;
  int start, end, tiles_n, ksplit, bn, kblocks, K;
};
__device__ __forceinline__ void group_cache(GroupCache& c, const GemmGroup* groups, int n_groups, int item) {
  if (c.g != nullptr && item >= c.start && item < c.end) return;
  const GemmGroup* g = groups + find_group_tc(groups, n_groups, item);
  c.g = g;
  c.start = g->tile_start;
  c.tiles_n = g->tiles_n;
  c.ksplit = g->ksplit;
  c.bn = g->bn;
  c.end = c.start + g->tiles_m * g->tiles_n * g->ksplit;
  c.K = g->K;
  c.kblocks = (c.K + TC_BK - 1) / TC_BK;
}
__device__ __forceinline__ Item decode_item(const GroupCache& c, int item) {
  const int local = item - c.start;
  Item it;
  it.split = local % c.ksplit;
  it.tile = local / c.ksplit;
  it.m0 = (it.tile / c.tiles_n) * TC_BM;
  it.n0 = (it.tile % c.tiles_n) * c.bn;
  const int per = (c.kblocks + c.ksplit - 1) / c.ksplit;
  it.kb0 = it.split * per;
  it.kb1 = min(c.kblocks, it.kb0 + per);
  return it;
}

// Epilogue of 4 consecutive columns [n, n+4) of one row (split-k reduction path).
__device__ __forceinline__ void epilogue4(const GView& g, int m, int n, float4 a) {
  const int N = g.N;
  float v[4] = {a.x, a.y, a.z, a.w};
  const bool full = (n + 4 <= N);
  if (g.epi & EPI_BIAS) {
#pragma unroll
    for (int j = 0; j < 4; ++j) if (n + j < N) v[j] += bf2f(g.bias[n + j]);
  }
  if (g.epi & EPI_GELU) {
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = gelu_erf(v[j]);
  }
  if (g.epi & EPI_RESID_F32) {
    float* C = reinterpret_cast<float*>(g.C) + (size_t)m * g.ldc + n;
    if (full) {
      float4 c = *reinterpret_cast<float4*>(C);
      c.x += v[0]; c.y += v[1]; c.z += v[2]; c.w += v[3];
      *reinterpret_cast<float4*>(C) = c;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) if (n + j < N) C[j] += v[j];
    }
  } else if (g.epi & EPI_SWIGLU) {
    bf16* C = reinterpret_cast<bf16*>(g.C) + (size_t)m * g.ldc + (n >> 1);
    if (full) {
      *reinterpret_cast<uint32_t*>(C) = pack2(silu_f(v[0]) * v[1], silu_f(v[2]) * v[3]);
    } else {
      if (n + 1 < N) C[0] = f2bf(silu_f(v[0]) * v[1]);
    }
  } else {
    bf16* C = reinterpret_cast<bf16*>(g.C) + (size_t)m * g.ldc + n;
    if (full) {
      *reinterpret_cast<uint2*>(C) = make_uint2(pack2(v[0], v[1]), pack2(v[2], v[3]));
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) if (n + j < N) C[j] = f2bf(v[j]);
    }
  }
}

// Split-k reduction of one tile by the 256 epilogue threads: positions (row, 4 columns) are swept
// coalesced along the row, U positions x up to KSMAX ranges of loads in flight per thread; the
// ranges of a position are added in range order.
template <int U, int KSMAX>
__device__ __forceinline__ void splitk_reduce(const GView& g, const Item& it, int et, size_t pld) {
  const int rows = min(TC_BM, g.M - it.m0);
  const int cols4 = (min(g.bn, g.N - it.n0) + 3) >> 2;
  const int npos = rows * cols4;
  const size_t sstride = (size_t)g.tiles_m * TC_BM * pld;
  const float* p0 = g.partial + (size_t)it.m0 * pld + it.n0;
  const int ks = g.ksplit;
  constexpr int STEP = EPI_WARPS * 32;
  for (int base_pos = et; base_pos < npos; base_pos += STEP * U) {
    float4 pv[U][KSMAX];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int pos = base_pos + u * STEP;
      const int r = pos / cols4, c4 = pos - r * cols4;
#pragma unroll
      for (int s2 = 0; s2 < KSMAX; ++s2)
        if (s2 < ks && pos < npos)
          pv[u][s2] = __ldcg(reinterpret_cast<const float4*>(p0 + (size_t)r * pld + c4 * 4 + s2 * sstride));
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int pos = base_pos + u * STEP;
      if (pos < npos) {
        float4 a4 = pv[u][0];
#pragma unroll
        for (int s2 = 1; s2 < KSMAX; ++s2)
          if (s2 < ks) { a4.x += pv[u][s2].x; a4.y += pv[u][s2].y; a4.z += pv[u][s2].z; a4.w += pv[u][s2].w; }
        const int r = pos / cols4, c4 = pos - r * cols4;
        epilogue4(g, it.m0 + r, it.n0 + c4 * 4, a4);
      }
    }
  }
}

// Direct epilogue of one warp for one tile, with no block-level barrier.  Warp (quarter, part) owns
// rows quarter*32..+31 and the part-th quarter of the tile's columns.  Per chunk (32 accumulator
// columns; 16 for an fp32 residual) each lane turns its row's values into outputs and parks them in
// the warp's 2 KB staging area (64-byte rows, SwiGLU 32-byte rows, 16-byte pieces in the TMA swizzle
// pattern, which also keeps the stores free of bank conflicts); one lane then hands the 32-row box to
// the TMA unit: a plain store for bf16 outputs, a reduce-add for the fp32 residual (the addition
// happens at L2; the SM never reads C).  The hardware clips rows and columns outside the tensor.
// The accumulator is handed back to the MMA warp as soon as this warp's last chunk has left TMEM.
// MODE: 0 bf16 output, 1 SwiGLU, 2 fp32 residual.
// REMOTE: tempty is a shared::cluster address (the accumulator barrier of the pair's leader).
template <int MODE, bool REMOTE = false>
__device__ __forceinline__ void epi_direct(const GView& g, const Item& it, uint32_t taddr, unsigned char* wst, int quarter,
                                           int part, int lane, uint2 bias_reg, uint32_t tempty) {
  constexpr int CW = (MODE == 2) ? 16 : 32;                  // accumulator columns per chunk
  const uint32_t wst_u = smem_u32(wst);
  const int y0 = it.m0 + quarter * 32;
  const bool box_ok = y0 < g.c_rows;                         // some row of this warp's box is inside the tensor
  const int c_begin = part * (g.bn >> 2);
  const int c_end = min(c_begin + (g.bn >> 2), g.N - it.n0);
  if (c_begin >= c_end) {                                    // nothing to do for this warp: release at once
    tc_fence_before();
    __syncwarp();
    if (lane == 0) { if (REMOTE) mbar_arrive_cluster(tempty); else mbar_arrive(tempty); }
    return;
  }
#pragma unroll 1
  for (int c = c_begin; c < c_end; c += CW) {
    const int n = it.n0 + c;
    float v[CW];
    {
      uint32_t r[CW];
      if (MODE == 2) tmem_ld16(taddr + (uint32_t)c, r); else tmem_ld32(taddr + (uint32_t)c, r);
#pragma unroll
      for (int j = 0; j < CW; ++j) v[j] = __uint_as_float(r[j]);
    }
    if (c + CW >= c_end) {                                   // that was this warp's last read of the accumulator
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { if (REMOTE) mbar_arrive_cluster(tempty); else mbar_arrive(tempty); }
    }
    if (g.epi & EPI_BIAS) {
      // the bias values of this chunk sit in consecutive lanes of bias_reg (zero past N)
      const int lane0 = (c - c_begin) >> 2;
#pragma unroll
      for (int jj = 0; jj < CW / 2; ++jj) {
        const uint32_t w = __shfl_sync(0xffffffffu, (jj & 1) ? bias_reg.y : bias_reg.x, lane0 + (jj >> 1));
        v[2 * jj] += __uint_as_float(w << 16);
        v[2 * jj + 1] += __uint_as_float(w & 0xffff0000u);
      }
    }
    if (g.epi & EPI_GELU) {
#pragma unroll
      for (int j = 0; j < CW; ++j) v[j] = gelu_erf(v[j]);
    }
    // the previous box of this warp must have been read out of the staging area
    if (lane == 0) bulk_wait_read0();
    __syncwarp();
    if (MODE == 2) {
      unsigned char* srow = wst + lane * 64;
      const int sw = (lane >> 1) & 3;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        *reinterpret_cast<float4*>(srow + ((k ^ sw) << 4)) = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
    } else if (MODE == 1) {
      unsigned char* srow = wst + lane * 32;                 // 32 columns -> 16 outputs -> 2 pieces
      const int sw = (lane >> 2) & 1;
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        uint4 o;
        o.x = pack2(silu_f(v[16 * k]) * v[16 * k + 1], silu_f(v[16 * k + 2]) * v[16 * k + 3]);
        o.y = pack2(silu_f(v[16 * k + 4]) * v[16 * k + 5], silu_f(v[16 * k + 6]) * v[16 * k + 7]);
        o.z = pack2(silu_f(v[16 * k + 8]) * v[16 * k + 9], silu_f(v[16 * k + 10]) * v[16 * k + 11]);
        o.w = pack2(silu_f(v[16 * k + 12]) * v[16 * k + 13], silu_f(v[16 * k + 14]) * v[16 * k + 15]);
        *reinterpret_cast<uint4*>(srow + ((k ^ sw) << 4)) = o;
      }
    } else {
      unsigned char* srow = wst + lane * 64;                 // 32 columns -> 4 pieces
      const int sw = (lane >> 1) & 3;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint4 o;
        o.x = pack2(v[8 * k], v[8 * k + 1]); o.y = pack2(v[8 * k + 2], v[8 * k + 3]);
        o.z = pack2(v[8 * k + 4], v[8 * k + 5]); o.w = pack2(v[8 * k + 6], v[8 * k + 7]);
        *reinterpret_cast<uint4*>(srow + ((k ^ sw) << 4)) = o;
      }
    }
    fence_async_smem();                      // the staged values must be visible to the TMA unit
    __syncwarp();
    if (lane == 0 && box_ok) {
      if (MODE == 2) tma_reduce_add_2d(g.tmC, wst_u, n, y0);
      else tma_store_2d(g.tmC, wst_u, MODE == 1 ? (n >> 1) : n, y0);
      bulk_commit();
    }
  }
}

__global__ void __launch_bounds__(N_THREADS, 1)
gemm_tc_kernel(const GemmGroup* __restrict__ groups, int n_groups, int total_items, int* __restrict__ status,
               int STAGES, int STAGE_BYTES) {
  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte aligned tile area (128-byte swizzle atoms are 1024 bytes)
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  unsigned char* stage_out = base_ptr + RING_BYTES;
  const uint32_t bars = base + RING_BYTES + STAGE_OUT_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * MAX_STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + RING_BYTES + STAGE_OUT_BYTES + 8 * (2 * MAX_STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* last_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);
  volatile int* votes = reinterpret_cast<volatile int*>(tmem_slot + 4);   // one per epilogue warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), EPI_WARPS); }
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane != 0) {
      pdl_wait();
      // ---------------------------------------------------------- L2 prefetch of residual tiles
      // The fp32 residual epilogue reads C before it adds to it; these lanes ask L2 for the C tiles of
      // this CTA's items ahead of time so that those reads do not wait on HBM.
      for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const GemmGroup& g = groups[find_group_tc(groups, n_groups, item)];
        if (!(g.epi & EPI_RESID_F32)) continue;
        const Item it = decode_item(g, item - g.tile_start);
        if (it.split != g.ksplit - 1) continue;        // once per tile
        const int ncols = min(g.bn, g.N - it.n0);
        for (int r = lane - 1; r < TC_BM && it.m0 + r < g.M; r += 31) {
          const float* rowp = reinterpret_cast<const float*>(g.C) + (size_t)(it.m0 + r) * g.ldc + it.n0;
          for (int c = 0; c < ncols; c += 32)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + c));
        }
      }
    }
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t issued_mask = 0, last_parity = 0;
      const GemmGroup* g_prev = nullptr;
      GroupCache gc;
      gc.g = nullptr;
      // Weights are never written by a kernel: the W tiles of this CTA's first k-blocks (the stages are
      // all free) are requested before the wait on the earlier kernels of the stream, the A tiles after it.
      int npre = 0;
      if ((int)blockIdx.x < total_items) {
        group_cache(gc, groups, n_groups, blockIdx.x);
        const GemmGroup* g = gc.g;
        const Item it = decode_item(gc, blockIdx.x);
        tensormap_acquire(&g->tmA);
        tensormap_acquire(&g->tmW);
        g_prev = g;
        const uint32_t bytes = A_BYTES + (uint32_t)gc.bn * TC_BK * 2;
        npre = min(STAGES, it.kb1 - it.kb0);
        for (int i = 0; i < npre; ++i) {
          mbar_expect_tx(full_bar(i), bytes);
          tma_load_2d(base + i * STAGE_BYTES + A_BYTES, &g->tmW, (it.kb0 + i) * TC_BK, it.n0, full_bar(i));
        }
        pdl_wait();
        for (int i = 0; i < npre; ++i) {
          tma_load_2d(base + i * STAGE_BYTES, &g->tmA, (it.kb0 + i) * TC_BK, it.m0, full_bar(i));
          issued_mask |= 1u << i;
        }
        if (npre == STAGES) { stage = 0; phase = 1u; } else { stage = npre; }
      } else {
        pdl_wait();
      }
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        group_cache(gc, groups, n_groups, item);
        const GemmGroup* g = gc.g;
        const Item it = decode_item(gc, item);
        if (g != g_prev) {                     // the maps were written by a host copy: acquire once per group
          tensormap_acquire(&g->tmA);
          tensormap_acquire(&g->tmW);
          g_prev = g;
        }
        const uint32_t bytes = A_BYTES + (uint32_t)gc.bn * TC_BK * 2;
        for (int kb = it.kb0 + npre; kb < it.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 1); break; }
          mbar_expect_tx(full_bar(stage), bytes);
          const uint32_t sa = base + stage * STAGE_BYTES;
          tma_load_2d(sa, &g->tmA, kb * TC_BK, it.m0, full_bar(stage));
          tma_load_2d(sa + A_BYTES, &g->tmW, kb * TC_BK, it.n0, full_bar(stage));
          issued_mask |= 1u << stage;
          last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        npre = 0;
      }
      if (!ok) {
        *abort_flag = 1;
        // let copies already in flight land before the CTA's shared memory goes away
        for (int s = 0; s < STAGES; ++s)
          if (issued_mask & (1u << s)) {
            volatile int never = 0;
            mbar_wait(full_bar(s), (last_parity >> s) & 1u, &never);
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      GroupCache gc;
      gc.g = nullptr;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        group_cache(gc, groups, n_groups, item);
        const Item it = decode_item(gc, item);
        const uint32_t idesc = make_idesc(gc.bn);
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 2); break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_COLS);
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; atomicExch(status, 3); break; }
          tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES;
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)
            mma_f16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
          mma_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        mma_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..17)
    pdl_wait();
    const int ew = warp - 2;
    const int et = threadIdx.x - 64;          // 0..255 among the epilogue threads
    const int quarter = warp & 3;             // TMEM lanes 32*quarter .. +31 belong to this warp
    const int part = ew >> 2;                 // which quarter of the tile's columns this warp owns
    const int row = quarter * 32 + lane;      // row of the tile this thread reads from TMEM
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    GView g;
    int g_end = -1;
    g.tile_start = 0;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      if (item >= g_end || item < g.tile_start) {
        g = load_view(groups + find_group_tc(groups, n_groups, item));
        g_end = g.tile_start + g.tiles_m * g.tiles_n * g.ksplit;
        if (lane == 0) tensormap_acquire(g.tmC);
      }
      const Item it = decode_item(g, item - g.tile_start);
      // bias of this warp's columns, 4 values per lane, requested before the accumulator is awaited
      uint2 bias_reg = make_uint2(0u, 0u);
      if (g.epi & EPI_BIAS) {
        const int nb = it.n0 + part * (g.bn >> 2) + lane * 4;
        if (lane * 4 >= (g.bn >> 2)) {
          // beyond this warp's columns
        } else if (nb + 4 <= g.N) {
          bias_reg = __ldg(reinterpret_cast<const uint2*>(g.bias + nb));
        } else {
          unsigned short e[4] = {0, 0, 0, 0};
#pragma unroll
          for (int j = 0; j < 4; ++j) if (nb + j < g.N) e[j] = __bfloat16_as_ushort(g.bias[nb + j]);
          bias_reg = make_uint2((uint32_t)e[0] | ((uint32_t)e[1] << 16), (uint32_t)e[2] | ((uint32_t)e[3] << 16));
        }
      }
      bool got = mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
      if (g.ksplit > 1) {
        // the split path uses block-level barriers among the epilogue warps: leave together
        if (lane == 0) votes[ew] = got ? 1 : 0;
        epi_barrier();
        for (int w = 0; w < EPI_WARPS; ++w) got = got && (votes[w] != 0);
        epi_barrier();
      }
      if (!got) { ok = false; if (lane == 0) atomicExch(status, 4); break; }
      tc_fence_after();
      const int m = it.m0 + row;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * ACC_COLS);
      const bool split = g.ksplit > 1;
      const size_t pld = (size_t)g.tiles_n * g.bn;                                   // partial row length
      if (split) {
        float* pdst = g.partial + ((size_t)it.split * g.tiles_m * TC_BM + m) * pld + it.n0;
#pragma unroll 1
        for (int c = part * 32; c < g.bn; c += 128) {
          if (it.n0 + c >= g.N) break;           // uniform across the warp
          uint32_t r[32];
          tmem_ld32(taddr + (uint32_t)c, r);
          if (m < g.M) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              __stcg(reinterpret_cast<float4*>(pdst + c + j),
                     make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                 __uint_as_float(r[j + 3])));
          }
        }
        // the accumulator is drained: hand it back to the MMA warp
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
        // count this k range; the one that arrives last reduces all ranges in order
        __threadfence();
        epi_barrier();
        if (et == 0) {
          const int old = atomicAdd(g.counters + it.tile, 1);
          const int last = (old == g.ksplit - 1);
          if (last) atomicExch(g.counters + it.tile, 0);
          *last_flag = last;
        }
        epi_barrier();
        const bool last = *last_flag != 0;
        if (last) {
          __threadfence();
          if (g.ksplit <= 2) splitk_reduce<4, 2>(g, it, et, pld);
          else if (g.ksplit <= 4) splitk_reduce<2, 4>(g, it, et, pld);
          else splitk_reduce<1, 8>(g, it, et, pld);
        }
        epi_barrier();                         // last_flag may be rewritten only after everyone read it
      } else {
        // direct epilogue (see epi_direct), specialised by output mode
        unsigned char* wst = stage_out + ew * 2048;
        if (g.epi & EPI_RESID_F32) epi_direct<2>(g, it, taddr, wst, quarter, part, lane, bias_reg, tempty_bar(acc));
        else if (g.epi & EPI_SWIGLU) epi_direct<1>(g, it, taddr, wst, quarter, part, lane, bias_reg, tempty_bar(acc));
        else epi_direct<0>(g, it, taddr, wst, quarter, part, lane, bias_reg, tempty_bar(acc));
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    // The kernel that follows may already be resident and is released the moment this grid completes:
    // the staged boxes must have reached global memory, not merely have left shared memory.
    if (lane == 0) bulk_wait_done0();
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------- tile pairs
// The same pipeline for 256 x bn tiles worked by two CTAs of a cluster (the two SMs of a TPC): each CTA
// loads its own 128 rows of A and bn / 2 rows of W per k-block (32 KB instead of 48: six ring stages, and
// a third less traffic from L2 per flop, which is what bounds the one-CTA kernel on all 148 SMs), rank 0
// issues one M = 256 MMA for both, the accumulator rows of a CTA's half live in its own TMEM and its own
// epilogue warps write them out.  Warp 0 loads A, warp 18 loads W, warp 1 of rank 0 issues the MMAs, warps
// 2..17 are the epilogue.  Barriers: every CTA's loads are counted on rank 0's full barrier;
// the MMA completion is reported to the empty / accumulator-full barriers of both CTAs; the epilogue
// warps of both report a drained accumulator to rank 0.  Only groups with ksplit = 1 take this path; a
// work item is one 256-row tile, GemmGroup::tiles_m counts 256-row tiles.
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_STAGE_BYTES = RING_BYTES / PAIR_STAGES;     // 32 KB: A 16 KB + at most 128 rows of W

template <class G>
__device__ __forceinline__ Item decode_item_pair(const G& g, int local, int rank) {
  Item it;
  it.split = 0;
  it.tile = local;
  it.m0 = (local / g.tiles_n) * (2 * TC_BM) + rank * TC_BM;
  it.n0 = (local % g.tiles_n) * g.bn;
  it.kb0 = 0;
  it.kb1 = (g.K + TC_BK - 1) / TC_BK;
  return it;
}

// A producer that gives up cannot await its copies in flight (their bytes are counted on the leader's
// barrier, which may never complete once the peer has given up too): it sleeps this long instead, far
// more than a copy takes, before the CTAs meet at the closing cluster barrier.
constexpr unsigned long long PAIR_DRAIN_NS = 200000ull;
constexpr int PAIR_W_WARP = 2 + EPI_WARPS;                     // the warp after the epilogue warps loads W
constexpr int PAIR_THREADS = N_THREADS + 32;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PAIR_THREADS, 1)
gemm_tc_pair_kernel(const GemmGroup* __restrict__ groups, int n_groups, int total_items, int* __restrict__ status) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  unsigned char* stage_out = base_ptr + RING_BYTES;
  const uint32_t bars = base + RING_BYTES + STAGE_OUT_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * MAX_STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + RING_BYTES + STAGE_OUT_BYTES + 8 * (2 * MAX_STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < PAIR_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                        // the peer's barriers exist before anything is reported to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane != 0) {
      // L2 prefetch of the fp32 residual tiles this CTA will add to (see the one-CTA kernel)
      pdl_wait();
      for (int item = pair; item < total_items; item += n_pairs) {
        const GemmGroup& g = groups[find_group_tc(groups, n_groups, item)];
        if (!(g.epi & EPI_RESID_F32)) continue;
        const Item it = decode_item_pair(g, item - g.tile_start, rank);
        const int ncols = min(g.bn, g.N - it.n0);
        for (int r = lane - 1; r < TC_BM && it.m0 + r < g.M; r += 31) {
          const float* rowp = reinterpret_cast<const float*>(g.C) + (size_t)(it.m0 + r) * g.ldc + it.n0;
          for (int c = 0; c < ncols; c += 32)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + c));
        }
      }
    }
    // ------------------------------------------------------------ TMA producer of A (one per CTA)
    // One thread issues a TMA load in some 150 cycles; with both operands on one thread a k-block costs it
    // more than the 512 cycles its MMAs take once tiles are short.  So the two operands have a thread each.
    if (lane == 0) {
      pdl_wait();
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const GemmGroup* g_prev = nullptr;
      GroupCache gc;
      gc.g = nullptr;
      for (int item = pair; item < total_items && ok; item += n_pairs) {
        group_cache(gc, groups, n_groups, item);
        const GemmGroup* g = gc.g;
        const Item it = decode_item_pair(gc, item - gc.start, rank);
        if (g != g_prev) { tensormap_acquire(&g->tmA); g_prev = g; }
        const uint32_t bytes = 2u * (A_BYTES + (uint32_t)(gc.bn >> 1) * TC_BK * 2);   // both CTAs' boxes of a k-block
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 31); break; }
          if (rank == 0) mbar_expect_tx(full_bar(stage), bytes);
          tma_load_2d_pair(base + stage * PAIR_STAGE_BYTES, &g->tmA, kb * TC_BK, it.m0, mapa_shared(full_bar(stage), 0));
          if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) { *abort_flag = 1; drain_sleep(PAIR_DRAIN_NS); }
    }
  } else if (warp == PAIR_W_WARP) {
    // ------------------------------------------------------------ TMA producer of W (one per CTA)
    // Weights are never written by a kernel, so this thread does not wait for the earlier kernels of the
    // stream: the first stages' W boxes are on their way while those still run.  (Bytes that land before
    // rank 0 has announced them leave the barrier's count negative for a while, which is allowed; the
    // phase cannot complete before that thread's own arrival.)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const GemmGroup* g_prev = nullptr;
      GroupCache gc;
      gc.g = nullptr;
      for (int item = pair; item < total_items && ok; item += n_pairs) {
        group_cache(gc, groups, n_groups, item);
        const GemmGroup* g = gc.g;
        const Item it = decode_item_pair(gc, item - gc.start, rank);
        if (g != g_prev) { tensormap_acquire(&g->tmW); g_prev = g; }
        const int n_half = it.n0 + rank * (gc.bn >> 1);
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 35); break; }
          tma_load_2d_pair(base + stage * PAIR_STAGE_BYTES + A_BYTES, &g->tmW, kb * TC_BK, n_half, mapa_shared(full_bar(stage), 0));
          if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) { *abort_flag = 1; drain_sleep(PAIR_DRAIN_NS); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (rank 0 only)
    if (lane == 0 && rank == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      GroupCache gc;
      gc.g = nullptr;
      for (int item = pair; item < total_items && ok; item += n_pairs) {
        group_cache(gc, groups, n_groups, item);
        const uint32_t idesc = make_idesc_pair(gc.bn);
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 32); break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_COLS);
        for (int kb = 0; kb < gc.kblocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; atomicExch(status, 33); break; }
          tc_fence_after();
          const uint32_t sa = base + stage * PAIR_STAGE_BYTES;
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)
            mma_f16_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          mma_commit_pair(empty_bar(stage));
          if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        mma_commit_pair(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..17 of both CTAs)
    pdl_wait();
    const int ew = warp - 2;
    const int quarter = warp & 3;
    const int part = ew >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    GView g;
    int g_end = -1;
    g.tile_start = 0;
    for (int item = pair; item < total_items && ok; item += n_pairs) {
      if (item >= g_end || item < g.tile_start) {
        g = load_view(groups + find_group_tc(groups, n_groups, item));
        g_end = g.tile_start + g.tiles_m * g.tiles_n;
        if (lane == 0) tensormap_acquire(g.tmC);
      }
      const Item it = decode_item_pair(g, item - g.tile_start, rank);
      uint2 bias_reg = make_uint2(0u, 0u);
      if (g.epi & EPI_BIAS) {
        const int nb = it.n0 + part * (g.bn >> 2) + lane * 4;
        if (lane * 4 >= (g.bn >> 2)) {
          // beyond this warp's columns
        } else if (nb + 4 <= g.N) {
          bias_reg = __ldg(reinterpret_cast<const uint2*>(g.bias + nb));
        } else {
          unsigned short e[4] = {0, 0, 0, 0};
#pragma unroll
          for (int j = 0; j < 4; ++j) if (nb + j < g.N) e[j] = __bfloat16_as_ushort(g.bias[nb + j]);
          bias_reg = make_uint2((uint32_t)e[0] | ((uint32_t)e[1] << 16), (uint32_t)e[2] | ((uint32_t)e[3] << 16));
        }
      }
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 34); break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * ACC_COLS);
      unsigned char* wst = stage_out + ew * 2048;
      const uint32_t te = mapa_shared(tempty_bar(acc), 0);
      if (g.epi & EPI_RESID_F32) epi_direct<2, true>(g, it, taddr, wst, quarter, part, lane, bias_reg, te);
      else if (g.epi & EPI_SWIGLU) epi_direct<1, true>(g, it, taddr, wst, quarter, part, lane, bias_reg, te);
      else epi_direct<0, true>(g, it, taddr, wst, quarter, part, lane, bias_reg, te);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_done0();
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                        // neither CTA leaves while the other may still read its operands or signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------- fused MLP block
// z += GELU(h W1^T + b1) W2^T + b2 for encoder blocks with d <= 384: the 4d-wide hidden tensor never leaves
// the SM.  A cluster of two CTAs works one 256-row tile (cta_group::2, as in the tile-pair kernel).  Per tile
// the CTA's 128 rows of h stay in shared memory (d / 64 k-blocks of 16 KB); the hidden layer is taken in chunks
// of 128 columns:
//   S = h W1_c^T         (M 256, N 128, K d)  into tensor-memory columns 384..511,
//   P = bf16(GELU(S + b1_c)) by the 16 epilogue warps, written to shared memory in the K-major 128-byte-swizzled
//                        layout an A operand has (two blocks of 128 rows x 64 columns),
//   O += P W2_c^T        (M 256, N d, K 128)  into columns 0..d-1 (two MMAs of N = d / 2 per k step when d > 256),
// and after the last chunk O + b2 is added to z through the same TMA reduce-add epilogue as any fp32-residual
// GEMM.  The rounding points are those of the unfused pair of GEMMs (the hidden tensor is rounded to bf16 once,
// the k order of both contractions is ascending), so a request's bits do not change with the kernel.
// The two contractions have an issuing thread each (warp 1 for S, the last warp for O): the chains only meet
// through the epilogue warps (S -> P), so the tensor core works on the next chunk's S while this chunk's GELU is
// computed and on this chunk's O while the next S is read out, and neither thread's issue time (some 80 cycles
// per tcgen05.mma) delays the other chain.  Weights stream through two rings of two 24 KB slots (W1: three k-blocks
// of a chunk half per slot; W2: one k-block of a chunk half per slot), each with its own producer thread.
// P's 32 KB double as the staging area of the final epilogue (P is idle by then).
constexpr int MLP_SLOT_BYTES = 24 * 1024;
constexpr int MLP_SLOTS = 4;                                   // two for W1 (0, 1), two for W2 (2, 3)
constexpr int MLP_O_WARP = PAIR_W_WARP + 1;                    // issues the second contraction
constexpr int MLP_THREADS = PAIR_THREADS + 32;
constexpr int MLP_X_BYTES = 6 * A_BYTES;                       // d <= 384: at most six k-blocks of 128 x 64
constexpr int MLP_P_BYTES = 2 * A_BYTES;                       // 128 rows x 128 hidden columns, bf16
constexpr int MLP_OFF_P = MLP_X_BYTES;
constexpr int MLP_OFF_RING = MLP_OFF_P + MLP_P_BYTES;
constexpr int MLP_OFF_BAR = MLP_OFF_RING + MLP_SLOTS * MLP_SLOT_BYTES;
constexpr size_t MLP_SMEM_BYTES = 1024 + (size_t)MLP_OFF_BAR + 256;
static_assert(MLP_SMEM_BYTES <= 227 * 1024, "shared memory of one SM");
static_assert(STAGE_OUT_BYTES <= MLP_P_BYTES, "the final epilogue stages its boxes in P");
constexpr int MLP_S_COL = 384;                                 // S behind the output accumulator
constexpr int MLP_CHUNK = 128;
enum { MB_W_FULL = 0, MB_W_EMPTY = MLP_SLOTS, MB_X_FULL = 2 * MLP_SLOTS, MB_X_EMPTY, MB_S_FULL, MB_S_EMPTY, MB_P_FULL,
       MB_P_EMPTY, MB_O_FULL, MB_O_EMPTY, MB_STAGE_FREE, MB_COUNT };
static_assert(8 * MB_COUNT + 16 <= 256, "barrier area");

__device__ __forceinline__ int find_group_mlp(const MlpGroup* groups, int n, int item) {
  int gi = 0;
  for (int i = 1; i < n; ++i) if (groups[i].tile_start <= item) gi = i;
  return gi;
}
// Geometry of a group in registers (the single-thread roles cannot hide descriptor loads).
struct MlpGeo {
  const MlpGroup* g;
  int start, end, kb1, nc, n2, n2i, slots1;
};
__device__ __forceinline__ void mlp_geo(MlpGeo& c, const MlpGroup* groups, int n_groups, int item) {
  if (c.g != nullptr && item >= c.start && item < c.end) return;
  const MlpGroup* g = groups + find_group_mlp(groups, n_groups, item);
  c.g = g;
  c.start = g->tile_start;
  c.end = c.start + g->tiles_m;
  const int d = g->d;
  c.kb1 = d >> 6;                       // k-blocks of the first contraction
  c.nc = g->F / MLP_CHUNK;              // chunks of the hidden layer
  c.n2i = d > 256 ? 2 : 1;              // MMAs per k step of the second contraction
  c.n2 = d / c.n2i;                     // and their N
  c.slots1 = (c.kb1 + 2) / 3;           // ring slots of one W1 chunk (three k-blocks of 64 rows each per slot)
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MLP_THREADS, 1)
gemm_mlp_pair_kernel(const MlpGroup* __restrict__ groups, int n_groups, int total_items, int* __restrict__ status) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bars = base + MLP_OFF_BAR;
  auto bar = [&](int i) { return bars + 8u * i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + MLP_OFF_BAR + 8 * MB_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < MLP_SLOTS; ++s) { mbar_init(bar(MB_W_FULL + s), 1); mbar_init(bar(MB_W_EMPTY + s), 1); }
    mbar_init(bar(MB_X_FULL), 1); mbar_init(bar(MB_X_EMPTY), 1);
    mbar_init(bar(MB_S_FULL), 1); mbar_init(bar(MB_S_EMPTY), 2 * EPI_WARPS);
    mbar_init(bar(MB_P_FULL), 2 * EPI_WARPS); mbar_init(bar(MB_P_EMPTY), 1);
    mbar_init(bar(MB_O_FULL), 1); mbar_init(bar(MB_O_EMPTY), 2 * EPI_WARPS);
    mbar_init(bar(MB_STAGE_FREE), EPI_WARPS);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                        // the peer's barriers exist before anything is reported to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer of h and W1 (one per CTA)
    // Per tile: the CTA's rows of h (once the tile before has been used by its last S), then W1 chunk by chunk.
    if (lane == 0) {
      bool ok = true;
      bool waited = false;
      const MlpGroup* g_prev = nullptr;
      MlpGeo gc;
      gc.g = nullptr;
      int slot = 0;
      uint32_t phase = 0, t = 0;
      for (int item = pair; item < total_items && ok; item += n_pairs, ++t) {
        mlp_geo(gc, groups, n_groups, item);
        const MlpGroup* g = gc.g;
        if (g != g_prev) { tensormap_acquire(&g->tmX); tensormap_acquire(&g->tmW1); g_prev = g; }
        const int m0 = (item - gc.start) * (2 * TC_BM) + rank * TC_BM;
        if (!mbar_wait(bar(MB_X_EMPTY), (t & 1u) ^ 1u, abort_flag)) { ok = false; atomicExch(status, 41); break; }
        if (!waited) { pdl_wait(); waited = true; }   // h is written by the kernel before this one
        if (rank == 0) mbar_expect_tx(bar(MB_X_FULL), 2u * (uint32_t)gc.kb1 * A_BYTES);
        for (int kb = 0; kb < gc.kb1; ++kb)
          tma_load_2d_pair(base + kb * A_BYTES, &g->tmX, kb * TC_BK, m0, mapa_shared(bar(MB_X_FULL), 0));
        for (int c = 0; c < gc.nc && ok; ++c) {
          for (int s1 = 0; s1 < gc.slots1; ++s1) {
            if (!mbar_wait(bar(MB_W_EMPTY + slot), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 42); break; }
            const int kb_lo = s1 * 3, kb_hi = min(gc.kb1, kb_lo + 3);
            if (rank == 0) mbar_expect_tx(bar(MB_W_FULL + slot), 2u * (uint32_t)(kb_hi - kb_lo) * (64 * 128));
            for (int kb = kb_lo; kb < kb_hi; ++kb)
              tma_load_2d_pair(base + MLP_OFF_RING + slot * MLP_SLOT_BYTES + (kb - kb_lo) * (64 * 128), &g->tmW1, kb * TC_BK,
                               c * MLP_CHUNK + rank * 64, mapa_shared(bar(MB_W_FULL + slot), 0));
            if (++slot == 2) { slot = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) { *abort_flag = 1; drain_sleep(PAIR_DRAIN_NS); }
    }
  } else if (warp == PAIR_W_WARP) {
    // ------------------------------------------------------------ TMA producer of W2 (one per CTA)
    // (Weights are never written by a kernel: no wait for earlier kernels.)
    if (lane == 0) {
      int slot = 0;
      uint32_t phase = 0;
      bool ok = true;
      const MlpGroup* g_prev = nullptr;
      MlpGeo gc;
      gc.g = nullptr;
      for (int item = pair; item < total_items && ok; item += n_pairs) {
        mlp_geo(gc, groups, n_groups, item);
        const MlpGroup* g = gc.g;
        if (g != g_prev) { tensormap_acquire(&g->tmW2); g_prev = g; }
        const int half = gc.n2 >> 1;                         // rows of one MMA's B operand held by this CTA
        for (int c = 0; c < gc.nc && ok; ++c) {
          for (int j = 0; j < 2; ++j) {                      // the chunk's two k-blocks
            if (!mbar_wait(bar(MB_W_EMPTY + 2 + slot), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 43); break; }
            if (rank == 0) mbar_expect_tx(bar(MB_W_FULL + 2 + slot), 2u * (uint32_t)gc.n2i * (uint32_t)half * 128u);
            for (int i = 0; i < gc.n2i; ++i)
              tma_load_2d_pair(base + MLP_OFF_RING + (2 + slot) * MLP_SLOT_BYTES + i * half * 128, &g->tmW2, (2 * c + j) * TC_BK,
                               i * gc.n2 + rank * half, mapa_shared(bar(MB_W_FULL + 2 + slot), 0));
            if (++slot == 2) { slot = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) { *abort_flag = 1; drain_sleep(PAIR_DRAIN_NS); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer of S = h W1_c^T (rank 0 only)
    if (lane == 0 && rank == 0) {
      int slot = 0;
      uint32_t phase = 0;
      uint32_t n_s = 0, t = 0;                // chunks issued, tiles started
      bool ok = true;
      MlpGeo gc;
      gc.g = nullptr;
      const uint32_t idesc_s = make_idesc_pair(MLP_CHUNK);
      for (int item = pair; item < total_items && ok; item += n_pairs, ++t) {
        mlp_geo(gc, groups, n_groups, item);
        if (!mbar_wait(bar(MB_X_FULL), t & 1u, abort_flag)) { ok = false; atomicExch(status, 49); break; }
        for (int c = 0; c < gc.nc && ok; ++c, ++n_s) {
          // S is free once the epilogue warps have read the chunk before out of it
          if (n_s > 0 && !mbar_wait(bar(MB_S_EMPTY), (n_s - 1) & 1u, abort_flag)) { ok = false; atomicExch(status, 44); break; }
          tc_fence_after();
          for (int s1 = 0; s1 < gc.slots1; ++s1) {
            if (!mbar_wait(bar(MB_W_FULL + slot), phase, abort_flag)) { ok = false; atomicExch(status, 45); break; }
            tc_fence_after();
            const int kb_lo = s1 * 3, kb_hi = min(gc.kb1, kb_lo + 3);
            for (int kb = kb_lo; kb < kb_hi; ++kb) {
              const uint64_t da = make_smem_desc(base + kb * A_BYTES);
              const uint64_t db = make_smem_desc(base + MLP_OFF_RING + slot * MLP_SLOT_BYTES + (kb - kb_lo) * (64 * 128));
#pragma unroll
              for (int k = 0; k < TC_BK / 16; ++k)
                mma_f16_pair(tmem_base + MLP_S_COL, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc_s, (kb > 0 || k > 0) ? 1u : 0u);
            }
            mma_commit_pair(bar(MB_W_EMPTY + slot));
            if (++slot == 2) { slot = 0; phase ^= 1u; }
          }
          if (!ok) break;
          mma_commit_pair(bar(MB_S_FULL));
          if (c == gc.nc - 1) mma_commit_pair(bar(MB_X_EMPTY));     // the tile's rows of h are no longer needed
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == MLP_O_WARP) {
    // ------------------------------------------------------------ MMA issuer of O += P W2_c^T (rank 0 only)
    if (lane == 0 && rank == 0) {
      int slot = 0;
      uint32_t phase = 0;
      uint32_t n_o = 0, t = 0;
      bool ok = true;
      MlpGeo gc;
      gc.g = nullptr;
      for (int item = pair; item < total_items && ok; item += n_pairs, ++t) {
        mlp_geo(gc, groups, n_groups, item);
        const uint32_t idesc_o = make_idesc_pair(gc.n2);
        const int half = gc.n2 >> 1;
        for (int c = 0; c < gc.nc && ok; ++c, ++n_o) {
          if (!mbar_wait(bar(MB_P_FULL), n_o & 1u, abort_flag)) { ok = false; atomicExch(status, 46); break; }
          // the first chunk overwrites O: the tile before must have been read out of it
          if (c == 0 && t > 0 && !mbar_wait(bar(MB_O_EMPTY), (t - 1) & 1u, abort_flag)) { ok = false; atomicExch(status, 47); break; }
          tc_fence_after();
          for (int j = 0; j < 2; ++j) {
            if (!mbar_wait(bar(MB_W_FULL + 2 + slot), phase, abort_flag)) { ok = false; atomicExch(status, 48); break; }
            tc_fence_after();
            const uint64_t da = make_smem_desc(base + MLP_OFF_P + j * A_BYTES);
#pragma unroll
            for (int k = 0; k < TC_BK / 16; ++k)
              for (int i = 0; i < gc.n2i; ++i) {
                const uint64_t db = make_smem_desc(base + MLP_OFF_RING + (2 + slot) * MLP_SLOT_BYTES + i * half * 128);
                mma_f16_pair(tmem_base + (uint32_t)(i * gc.n2), da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc_o,
                             (c > 0 || j > 0 || k > 0) ? 1u : 0u);
              }
            mma_commit_pair(bar(MB_W_EMPTY + 2 + slot));
            if (++slot == 2) { slot = 0; phase ^= 1u; }
          }
          if (!ok) break;
          mma_commit_pair(bar(MB_P_EMPTY));
          if (c == gc.nc - 1) mma_commit_pair(bar(MB_O_FULL));
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------ epilogue warps (2..17 of both CTAs)
    pdl_wait();
    const int ew = warp - 2;
    const int quarter = warp & 3;
    const int part = ew >> 2;
    const int row = quarter * 32 + lane;
    bool ok = true;
    uint32_t n_c = 0, t = 0;                  // chunks and tiles done by this warp
    const MlpGroup* g = nullptr;
    int g_start = 0, g_end = -1, nc = 0, d = 0, c_rows = 0;
    const bf16 *b1 = nullptr, *b2 = nullptr;
    const uint32_t s_taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(MLP_S_COL + part * 32);
    unsigned char* prow = base_ptr + MLP_OFF_P + (part >> 1) * A_BYTES + row * 128;
    const int piece0 = (part & 1) * 4, sw = row & 7;
    const uint32_t s_empty_r = mapa_shared(bar(MB_S_EMPTY), 0), p_full_r = mapa_shared(bar(MB_P_FULL), 0);
    const uint32_t o_empty_r = mapa_shared(bar(MB_O_EMPTY), 0);
    for (int item = pair; item < total_items && ok; item += n_pairs, ++t) {
      if (item >= g_end || item < g_start) {
        g = groups + find_group_mlp(groups, n_groups, item);
        g_start = g->tile_start; g_end = g_start + g->tiles_m;
        nc = g->F / MLP_CHUNK; d = g->d; c_rows = g->c_rows; b1 = g->b1; b2 = g->b2;
        if (lane == 0) tensormap_acquire(&g->tmC);
      }
      for (int c = 0; c < nc && ok; ++c, ++n_c) {
        // this warp's 32 hidden columns of the chunk: bias values four per lane in lanes 0..7
        uint2 bias_reg = make_uint2(0u, 0u);
        if (b1 != nullptr && lane < 8) bias_reg = __ldg(reinterpret_cast<const uint2*>(b1 + c * MLP_CHUNK + part * 32 + lane * 4));
        if (!mbar_wait(bar(MB_S_FULL), n_c & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 50); break; }
        tc_fence_after();
        float v[32];
        {
          uint32_t r[32];
          tmem_ld32(s_taddr, r);
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(s_empty_r);       // the next chunk's S may be issued
        if (b1 != nullptr) {
#pragma unroll
          for (int jj = 0; jj < 16; ++jj) {
            const uint32_t w = __shfl_sync(0xffffffffu, (jj & 1) ? bias_reg.y : bias_reg.x, jj >> 1);
            v[2 * jj] += __uint_as_float(w << 16);
            v[2 * jj + 1] += __uint_as_float(w & 0xffff0000u);
          }
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
        // P still feeds the second contraction of the chunk before; at a tile's first chunk it also was the
        // staging area of the final epilogue of the tile before, which every warp of this CTA must have left
        if (n_c > 0 && !mbar_wait(bar(MB_P_EMPTY), (n_c - 1) & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 51); break; }
        if (c == 0 && t > 0 && !mbar_wait(bar(MB_STAGE_FREE), (t - 1) & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 52); break; }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          uint4 o;
          o.x = pack2(v[8 * k], v[8 * k + 1]); o.y = pack2(v[8 * k + 2], v[8 * k + 3]);
          o.z = pack2(v[8 * k + 4], v[8 * k + 5]); o.w = pack2(v[8 * k + 6], v[8 * k + 7]);
          *reinterpret_cast<uint4*>(prow + (((piece0 + k) ^ sw) << 4)) = o;
        }
        fence_async_smem();                     // P must be visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(p_full_r);
      }
      if (!ok) break;
      // ---- the tile's output: O + b2 added to z (TMA reduce-add), staged in P
      GView gv;
      gv.bias = b2; gv.C = nullptr; gv.partial = nullptr; gv.counters = nullptr; gv.tmC = &g->tmC;
      gv.M = g->M; gv.N = d; gv.K = g->F; gv.ldc = d; gv.epi = EPI_RESID_F32 | (b2 != nullptr ? EPI_BIAS : 0);
      gv.tile_start = g_start; gv.tiles_m = g_end - g_start; gv.tiles_n = 1; gv.bn = d; gv.ksplit = 1; gv.c_rows = c_rows;
      Item it;
      it.split = 0; it.tile = item - g_start; it.m0 = it.tile * (2 * TC_BM) + rank * TC_BM; it.n0 = 0; it.kb0 = 0; it.kb1 = 0;
      uint2 bias_reg = make_uint2(0u, 0u);
      if (b2 != nullptr) {
        const int nb = part * (d >> 2) + lane * 4;
        if (lane * 4 < (d >> 2)) bias_reg = __ldg(reinterpret_cast<const uint2*>(b2 + nb));
      }
      if (!mbar_wait(bar(MB_O_FULL), t & 1u, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 53); break; }
      tc_fence_after();
      const uint32_t o_taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
      epi_direct<2, true>(gv, it, o_taddr, base_ptr + MLP_OFF_P + ew * 2048, quarter, part, lane, bias_reg, o_empty_r);
      if (lane == 0) { bulk_wait_read0(); mbar_arrive(bar(MB_STAGE_FREE)); }   // this warp's boxes have left P
    }
    if (lane == 0) bulk_wait_done0();
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                        // neither CTA leaves while the other may still read its operands or signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

}  // namespace

// Tile width and k-split of a GEMM whose row capacity is rows_cap (fixed when the model is placed,
// so a request's reduction order never depends on the batch it happens to share).
void gemm_tc_config(long long rows_cap, int N, int K, int epi, int sm_count, int* bn, int* ksplit) {
  auto padded = [&](int b) { return (N + b - 1) / b * b; };
  const int kblocks = (K + TC_BK - 1) / TC_BK;
  if (rows_cap <= 0) { *bn = 128; *ksplit = 1; return; }
  if (rows_cap > 256) {                       // dense: tensor-bound; a 128 x 256 MMA runs at about twice the
    *bn = (N > 128) ? 256 : 128;              // efficiency of a 128 x 128 one, which outweighs padded columns
    // fp32-residual outputs leave in 16-column boxes, so their tiles may be 192 wide (48 columns per
    // epilogue warp): N = 384 then fills two tiles exactly instead of wasting a quarter of two 256-wide ones
    if ((epi & EPI_RESID_F32) && N % 192 == 0 && padded(192) < padded(256)) *bn = 192;
    *ksplit = 1;
    return;
  }
  // weight streaming: the widest tile (most W bytes in flight per stage).  Splitting K pays only when
  // a handful of tiles would each stream a very long K: measured on B200 (whole decode steps of the 1B
  // decoder at batch 32 and 128), splitting from K = 1024 or 2048 on, into 4 to 8 ranges, changed the
  // step time by -2 % to +9 %: the fixed cost of a split item (partials, counter, reduction) eats the gain.
  // One CTA streams only about 80 GB/s through its 4-stage ring, so when 256-wide tiles would leave
  // SMs without work, 128-wide tiles (twice as many CTAs) stream faster.
  const int tiles_m = (int)((rows_cap + TC_BM - 1) / TC_BM);
  *bn = (N > 128 && tiles_m * (padded(256) / 256) * 10 >= sm_count * 7) ? 256 : 128;
  const int tiles = tiles_m * (padded(*bn) / *bn);
  int ks = 1;
  if (kblocks >= 64 && tiles * 8 <= sm_count) {
    ks = kblocks / 16;
    if (ks > 8) ks = 8;
    while (ks > 1 && (ks - 1) * ((kblocks + ks - 1) / ks) >= kblocks) --ks;   // no empty range
  }
  *ksplit = ks;
}

cudaError_t launch_gemm_tc(const GemmGroup* groups, int n_groups, int total_items, int max_bn, int* status, int sm_count,
                           cudaStream_t st) {
  if (n_groups == 0 || total_items == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int grid = total_items < sm_count ? total_items : sm_count;
  const int stages = max_bn <= 128 ? 6 : 4;
  const int stage_bytes = RING_BYTES / stages;
  return launch_pdl(gemm_tc_kernel, dim3(grid), dim3(N_THREADS), SMEM_BYTES, st, groups, n_groups, total_items, status,
                    stages, stage_bytes);
}

// A GEMM takes the tile-pair kernel when it has more than one 128-row tile at capacity and is not split
// along K; decided from the same placement-time quantities as the tile width, never from the batch.
// Weight-streaming groups (129..256 rows) gain too: the pair reads every W box from HBM once, each CTA
// half of it, where two one-CTA row tiles each load all of it.
bool gemm_tc_pair_eligible(long long rows_cap, int N, int K, int epi, int bn, int ksplit) {
  (void)N; (void)K; (void)epi;
  return rows_cap > TC_BM && ksplit == 1 && (bn == 128 || bn == 192 || bn == 256);
}

cudaError_t launch_gemm_tc_pair(const GemmGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                                cudaStream_t st) {
  if (n_groups == 0 || total_items == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int pairs = total_items < sm_count / 2 ? total_items : sm_count / 2;
  return launch_pdl(gemm_tc_pair_kernel, dim3(2 * pairs), dim3(PAIR_THREADS), SMEM_BYTES, st, groups, n_groups, total_items, status);
}

// The fused MLP kernel takes an encoder block when its accumulators fit the tensor memory (d <= 384 beside one
// 128-column chunk of S), the shapes tile evenly, and the model has more than one 128-row tile at capacity.
bool gemm_mlp_eligible(long long rows_cap, int d, int F) {
  return rows_cap > TC_BM && d >= 64 && d <= 384 && d % 64 == 0 && F >= 128 && F % 128 == 0;
}

cudaError_t launch_gemm_mlp_pair(const MlpGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                                 cudaStream_t st) {
  if (n_groups == 0 || total_items == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(gemm_mlp_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MLP_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int pairs = total_items < sm_count / 2 ? total_items : sm_count / 2;
  return launch_pdl(gemm_mlp_pair_kernel, dim3(2 * pairs), dim3(MLP_THREADS), MLP_SMEM_BYTES, st, groups, n_groups, total_items, status);
}

}  // namespace epara
