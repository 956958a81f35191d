// Grouped bf16 GEMM for groups of 17 to 128 rows (decode batches, classification heads): C = epi(A W^T + bias)
// with the operands swapped on the tensor core.
//
// With so few rows of A the work is streaming W once.  A 128-row tile of A would be mostly padding and a stage
// of the operand ring would hold as many activation bytes as weight bytes.  Here the MMA's 128-row operand is
// a tile of W (128 output columns) and the batch is the MMA's N (the row capacity rounded up to 16, at most
// 128): D[n, m] = sum_k W[n, k] A[m, k].  The accumulator holds C transposed: TMEM lane = output column, TMEM
// column = batch row.
//
// What bounds these kernels is how many bytes of W a CTA has in flight: at full rate HBM answers a request after
// about 5 us, so the whole device needs some 30 MB outstanding, about 200 KB per SM (measured: a CTA's ingest is
// its ring size divided by that latency, whatever the tile shape).  Activation tiles come from L2, a fraction of
// that latency away, and must not take ring space from W: the two operands have rings of their own, ten stages of
// 16 KB for W and two to four short-lived stages for the activations.
//
// A matrix has only N / 128 such tiles (16 to 24 for the projections of a 1B-scale decoder), too few CTAs to pull
// HBM bandwidth.  So K is cut into S ranges (S in {1, 2, 4, 8}, fixed from N and K when the model is placed) and
// the S CTAs of a thread-block cluster work one tile: each accumulates its k range in its own TMEM.  CTA r owns a
// share of the tile's output columns: once every CTA of the cluster is past its last MMA (a cluster barrier: the
// slices land in the owners' idle operand rings), every CTA sends the matching slice of its fp32 partial into CTA
// r's shared memory (distributed-shared-memory stores, which nobody waits for), and after a second cluster barrier
// CTA r adds the S slices in rank order out of its own shared memory and runs the epilogue for its columns.  No partial ever
// travels through global memory and the reduction order is fixed, so a request's bits do not depend on timing or
// on what else is in the launch.
//
// Roles per CTA: warp 0 (one lane) TMA producer of W -- it does not wait for the earlier kernels of the stream,
// weights being static, so its ring is full when they finish; warp 6 (one lane) TMA producer of the activations;
// warp 1 (one lane) tcgen05.mma issuer; warps 2..5 read the accumulator (one TMEM lane quarter each).  Every mbarrier wait is bounded; a CTA that gives up
// records a code in *status and still meets its cluster at the barriers.
#include "common.cuh"
#include "kernels.h"
#include "tcgen05.cuh"

namespace epara {

namespace {

using namespace tc;

constexpr int SW_BM = 128;                       // W rows (output columns) per tile
constexpr int SW_W_BYTES = SW_BM * TC_BK * 2;    // 16 KB
constexpr int SW_RING_BYTES_1 = 192 * 1024;      // one CTA per SM
constexpr int SW_RING_BYTES_2 = 104 * 1024;      // two CTAs per SM: launches with more CTAs than SMs, where a second
                                                 // MMA-issuing thread per SM and no second wave pay (the LM head:
                                                 // 45 -> 31 us at 128 rows), while launches that fit one wave were a
                                                 // little faster with the deeper ring
constexpr int SW_W_STAGES_MAX = 10;
constexpr int SW_A_STAGES_MAX = 4;
constexpr int SW_THREADS_EPI = 128;
constexpr int SW_A_WARP = 6;                     // the warp after the accumulator warps loads the activations
constexpr int SW_THREADS = 64 + SW_THREADS_EPI + 32;
constexpr int SW_TMEM_COLS = 128;
inline size_t sw_smem(int ring_bytes) { return 1024 + (size_t)ring_bytes + 256; }

__device__ __forceinline__ int find_group_sw(const GemmGroup* groups, int n, int item) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (groups[mid].tile_start <= item) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// S: CTAs per cluster = k ranges per tile.  One cluster per (group, tile of 128 output columns).
template <int S>
__global__ void __launch_bounds__(SW_THREADS, 2)
gemm_swap_kernel(const GemmGroup* __restrict__ groups, int n_groups, int* __restrict__ status, int ring_bytes) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bars = base + ring_bytes;
  auto wfull_bar = [&](int s) { return bars + 8u * s; };
  auto wempty_bar = [&](int s) { return bars + 8u * (SW_W_STAGES_MAX + s); };
  auto afull_bar = [&](int s) { return bars + 8u * (2 * SW_W_STAGES_MAX + s); };
  auto aempty_bar = [&](int s) { return bars + 8u * (2 * SW_W_STAGES_MAX + SW_A_STAGES_MAX + s); };
  const uint32_t tfull_bar = bars + 8u * (2 * SW_W_STAGES_MAX + 2 * SW_A_STAGES_MAX);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + ring_bytes + 8 * (2 * SW_W_STAGES_MAX + 2 * SW_A_STAGES_MAX + 1));
  static_assert(8 * (2 * SW_W_STAGES_MAX + 2 * SW_A_STAGES_MAX + 1) + 16 <= 256, "barrier area");
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  bool acc_ok = true;
  const int rank = S == 1 ? 0 : (int)cluster_ctarank();
  const int item = blockIdx.x / S;
  pdl_launch_dependents();

  const GemmGroup* g = groups + find_group_sw(groups, n_groups, item);
  const int nb = g->bn;                           // batch rows as the MMA's N: multiple of 16, at most 128
  const int n0 = (item - g->tile_start) * SW_BM;  // first output column (W row) of the tile
  const int kblocks = (g->K + TC_BK - 1) / TC_BK;
  const int per = (kblocks + S - 1) / S;
  const int kb0 = rank * per, kb1 = min(kblocks, kb0 + per);
  const bool empty = kb0 >= kb1;                  // K too short for this rank: its partial is zero
  // activation ring first (a_stages tiles of nb x 64), then the W ring (w_stages tiles of 128 x 64)
  const int a_bytes = nb * TC_BK * 2;
  const int a_stages = nb > 64 ? 2 : SW_A_STAGES_MAX;
  const int w_stages = min(SW_W_STAGES_MAX, (ring_bytes - a_stages * a_bytes) / SW_W_BYTES);
  const uint32_t w_base = base + a_stages * a_bytes;        // a multiple of 2 KB from a 1 KB-aligned base ...
  static_assert(SW_W_BYTES % 1024 == 0, "swizzle atoms");   // ... since nb is a multiple of 16

  if (threadIdx.x == 0) {
    for (int s = 0; s < w_stages; ++s) { mbar_init(wfull_bar(s), 1); mbar_init(wempty_bar(s), 1); }
    for (int s = 0; s < a_stages; ++s) { mbar_init(afull_bar(s), 1); mbar_init(aempty_bar(s), 1); }
    mbar_init(tfull_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)SW_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer of W (tmW: box of 128 rows)
    if (lane == 0) {
      tensormap_acquire(&g->tmW);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(wempty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 41); break; }
        mbar_expect_tx(wfull_bar(stage), (uint32_t)SW_W_BYTES);
        tma_load_2d(w_base + stage * SW_W_BYTES, &g->tmW, kb * TC_BK, n0, wfull_bar(stage));
        if (++stage == w_stages) { stage = 0; phase ^= 1u; }
      }
      pdl_wait();                                  // (every thread of the kernel waits once, see common.cuh)
      if (!ok) { *abort_flag = 1; drain_sleep(200000ull); }
    }
  } else if (warp == SW_A_WARP) {
    // ------------------------------------------------------------ TMA producer of the activations (tmA: box of nb rows)
    if (lane == 0) {
      tensormap_acquire(&g->tmA);
      pdl_wait();
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(aempty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 44); break; }
        mbar_expect_tx(afull_bar(stage), (uint32_t)a_bytes);
        tma_load_2d(base + stage * a_bytes, &g->tmA, kb * TC_BK, 0, afull_bar(stage));
        if (++stage == a_stages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) { *abort_flag = 1; drain_sleep(200000ull); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc(nb);
      int ws = 0, as = 0;
      uint32_t wphase = 0, aphase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(afull_bar(as), aphase, abort_flag)) { ok = false; atomicExch(status, 45); break; }
        if (!mbar_wait(wfull_bar(ws), wphase, abort_flag)) { ok = false; atomicExch(status, 42); break; }
        tc_fence_after();
        const uint64_t dw = make_smem_desc(w_base + ws * SW_W_BYTES), da = make_smem_desc(base + as * a_bytes);
#pragma unroll
        for (int k = 0; k < TC_BK / 16; ++k)
          mma_f16(tmem_base, dw + (uint64_t)(k * 2), da + (uint64_t)(k * 2), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
        mma_commit(wempty_bar(ws));
        mma_commit(aempty_bar(as));
        if (++ws == w_stages) { ws = 0; wphase ^= 1u; }
        if (++as == a_stages) { as = 0; aphase ^= 1u; }
      }
      if (!ok) *abort_flag = 1;
      else if (!empty) mma_commit(tfull_bar);
    }
  } else if (warp < SW_A_WARP) {
    // ------------------------------------------------------------ wait for this CTA's accumulator (warps 2..5)
    pdl_wait();
    acc_ok = empty || mbar_wait(tfull_bar, 0u, abort_flag);
    if (!acc_ok) {
      if (lane == 0) atomicExch(status, 43);
      *abort_flag = 1;
    }
  }
  // The slices go into the owners' operand rings, which must be idle: every CTA of the cluster has to be past
  // its last MMA before anyone sends.
  __syncthreads();
  if (S > 1) cluster_sync_all();
  if (warp >= 2 && warp < SW_A_WARP) {
    // ------------------------------------------------------------ accumulator -> the owners' shared memory
    // Output column n0 + row (TMEM lane `row`) belongs to CTA row / RP of the cluster.  Its buffer, over the idle
    // operand ring, is [S sources][nb batch rows][RP columns] fp32; this CTA fills plane `rank` of every owner.
    constexpr int RP = SW_BM / S;                     // columns per owner
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t dst = (S == 1 ? base : mapa_shared(base, (uint32_t)(row / RP))) + (uint32_t)(rank * nb * RP + (row % RP)) * 4u;
    tc_fence_after();
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    for (int c = 0; c < nb; c += 16) {
      uint32_t r[16];
      if (empty || !acc_ok) {
#pragma unroll
        for (int j = 0; j < 16; ++j) r[j] = 0u;      // no k-block for this rank (or a wait that ran out): a zero partial
      } else {
        tmem_ld16(taddr + (uint32_t)c, r);
      }
#pragma unroll
      for (int j = 0; j < 16; ++j)
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst + (uint32_t)((c + j) * RP) * 4u), "f"(__uint_as_float(r[j])) : "memory");
    }
    tc_fence_before();
  }
  __syncthreads();
  if (S > 1) cluster_sync_all();                     // every slice has reached its owner (release / acquire)

  if (warp >= 2 && warp < SW_A_WARP) {
    // ------------------------------------------------------------ reduction in rank order + epilogue
    // This CTA owns output columns n0 + rank * RP .. + RP - 1.  A thread takes four consecutive columns of the
    // batch rows t / CG, t / CG + 128 / CG, ..., two rows per pass: the S slices of both rows (and, for a residual
    // output, the old values of C) are requested together, then added in rank order.
    constexpr int RP = SW_BM / S;                    // columns per CTA
    constexpr int CG = RP / 4;                       // 4-column pieces per batch row
    constexpr int MSTEP = SW_THREADS_EPI / CG;       // batch rows per pass over the threads
    const int t = threadIdx.x - 64;
    const int col = (t % CG) * 4;                    // within this CTA's columns
    const int n = n0 + rank * RP + col;
    // (scalar copies: the descriptor lives in global memory, and with stores in the loop every g-> would be read again)
    const int M = g->M, N = g->N, epi = g->epi, ldc = g->ldc;
    void* const Cptr = g->C;
    const bf16* const bias_ptr = g->bias;
    const float* const red = reinterpret_cast<const float*>(base_ptr);
    float bias[4] = {0.f, 0.f, 0.f, 0.f};
    if (epi & EPI_BIAS) {
#pragma unroll
      for (int j = 0; j < 4; ++j) if (n + j < N) bias[j] = bf2f(bias_ptr[n + j]);
    }
    const bool full = n + 4 <= N;
#pragma unroll 1
    for (int m0 = t / CG; m0 < nb; m0 += 2 * MSTEP) {
      float4 old[2], part[2][S];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int m = m0 + u * MSTEP;
        old[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if ((epi & EPI_RESID_F32) && m < M && n < N) {
          const float* cf = reinterpret_cast<const float*>(Cptr) + (size_t)m * ldc + n;
          if (full) old[u] = *reinterpret_cast<const float4*>(cf);
          else { old[u].x = cf[0]; if (n + 1 < N) old[u].y = cf[1]; if (n + 2 < N) old[u].z = cf[2]; }
        }
#pragma unroll
        for (int q = 0; q < S; ++q)
          part[u][q] = m < nb ? *reinterpret_cast<const float4*>(red + (q * nb + m) * RP + col) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int m = m0 + u * MSTEP;
        float v[4] = {part[u][0].x, part[u][0].y, part[u][0].z, part[u][0].w};
#pragma unroll
        for (int q = 1; q < S; ++q) { v[0] += part[u][q].x; v[1] += part[u][q].y; v[2] += part[u][q].z; v[3] += part[u][q].w; }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[j] += bias[j];
          if (epi & EPI_GELU) v[j] = gelu_erf(v[j]);
        }
        if (m >= M || n >= N) continue;
        if (epi & EPI_SWIGLU) {
          // gate and up are adjacent output columns
          bf16* cb = reinterpret_cast<bf16*>(Cptr) + (size_t)m * ldc + (n >> 1);
          if (full) *reinterpret_cast<uint32_t*>(cb) = pack2(silu_f(v[0]) * v[1], silu_f(v[2]) * v[3]);
          else if (n + 1 < N) {
            cb[0] = f2bf(silu_f(v[0]) * v[1]);
            if (n + 3 < N) cb[1] = f2bf(silu_f(v[2]) * v[3]);
          }
        } else if (epi & EPI_RESID_F32) {
          float* cf = reinterpret_cast<float*>(Cptr) + (size_t)m * ldc + n;
          if (full) *reinterpret_cast<float4*>(cf) = make_float4(old[u].x + v[0], old[u].y + v[1], old[u].z + v[2], old[u].w + v[3]);
          else { cf[0] = old[u].x + v[0]; if (n + 1 < N) cf[1] = old[u].y + v[1]; if (n + 2 < N) cf[2] = old[u].z + v[2]; }
        } else {
          bf16* cb = reinterpret_cast<bf16*>(Cptr) + (size_t)m * ldc + n;
          if (full) *reinterpret_cast<uint2*>(cb) = make_uint2(pack2(v[0], v[1]), pack2(v[2], v[3]));
          else {
#pragma unroll
            for (int j = 0; j < 4; ++j) if (n + j < N) cb[j] = f2bf(v[j]);
          }
        }
      }
    }
  }
  // (after the barrier above nobody touches another CTA's shared memory, so the CTAs may leave one by one)
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)SW_TMEM_COLS) : "memory");
  }
}

template <int S>
cudaError_t launch_swap(const GemmGroup* groups, int n_groups, int total_items, int* status, int sm_count, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(gemm_swap_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sw_smem(SW_RING_BYTES_1));
  if (e != cudaSuccess) return e;
  // (clusters of eight one-SM CTAs were slow to place: 25.8 us against 15.4 with two CTAs per SM, 2048 x 8192 at 128 rows)
  const int ring_bytes = (total_items * S > sm_count || S == 8) ? SW_RING_BYTES_2 : SW_RING_BYTES_1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(total_items * S);
  cfg.blockDim = dim3(SW_THREADS);
  cfg.dynamicSmemBytes = sw_smem(ring_bytes);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = S;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_swap_kernel<S>, groups, n_groups, status, ring_bytes);
}

}  // namespace

// k ranges per tile: doubled while the CTAs still fit two per SM and every range keeps at least four k-blocks
// (sixteen for the step from four to eight ranges, which pays only on a long K: 19.6 -> 15.4 us for 2048 x 8192 at
// 128 rows, nothing for 2048 x 2048).
int gemm_swap_ksplit(int N, int K, int sm_count) {
  const int tiles = (N + SW_BM - 1) / SW_BM, kblocks = (K + TC_BK - 1) / TC_BK;
  int s = 1;
  while (s < 8 && tiles * s * 2 <= 2 * sm_count && kblocks / (s * 2) >= (s == 4 ? 16 : 4)) s *= 2;
  return s;
}

int gemm_swap_tiles(int N) { return (N + SW_BM - 1) / SW_BM; }

cudaError_t launch_gemm_swap(const GemmGroup* groups, int n_groups, int total_items, int ksplit, int* status, int sm_count,
                             cudaStream_t st) {
  if (n_groups == 0 || total_items == 0) return cudaSuccess;
  switch (ksplit) {
    case 1: return launch_swap<1>(groups, n_groups, total_items, status, sm_count, st);
    case 2: return launch_swap<2>(groups, n_groups, total_items, status, sm_count, st);
    case 4: return launch_swap<4>(groups, n_groups, total_items, status, sm_count, st);
    case 8: return launch_swap<8>(groups, n_groups, total_items, status, sm_count, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace epara
