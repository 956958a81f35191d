// Grouped bf16 GEMM on the sm_100a tensor cores: C_g = epi(A_g W_g^T + bias_g).
//
// One persistent launch covers every group (one group = one model's GEMM in this wave, with its
// own M, N, K).  Tiles of 128 x TC_BN are numbered group after group; CTA i takes tiles
// i, i + grid, ...  Inside a CTA three roles run concurrently:
//   warp 0 (one lane)  TMA producer: for each 64-wide k-block loads the A tile (128 x 64) and the
//                      W tile (TC_BN x 64) into a ring of shared-memory stages (plain, non-multicast
//                      cp.async.bulk.tensor; out-of-range rows/columns arrive as zeros);
//   warp 1 (one lane)  MMA issuer: tcgen05.mma (M 128, N TC_BN, K 16) from shared memory into one
//                      of two TMEM accumulators, releasing stages with tcgen05.commit;
//   warps 2..5         epilogue: tcgen05.ld of the finished accumulator, bias / GELU / SwiGLU /
//                      fp32 residual update, bf16 store -- while the MMA warp already fills the
//                      other accumulator.
// The K reduction of an output element is always the same sequence of k-blocks, whatever else is
// in the launch, so results do not depend on co-resident groups.
// Every mbarrier wait is bounded: when a wait runs out the kernel records a code in *status, all
// roles leave their loops, TMEM is freed and the kernel returns.
#include "common.cuh"
#include "kernels.h"

namespace epara {

namespace {

constexpr int STAGES = 6;
constexpr int A_BYTES = TC_BM * TC_BK * 2;          // 16 KB
constexpr int B_BYTES = TC_BN * TC_BK * 2;          // 16 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TMEM_COLS = 2 * TC_BN;                // two accumulators
constexpr int N_THREADS = 192;
constexpr size_t SMEM_BYTES = 1024 + (size_t)STAGES * STAGE_BYTES + 256;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait for the phase with the given parity.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    if (done) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = globaltimer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > WAIT_LIMIT_NS) return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* tm) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(tm) : "memory");
}

// K-major operand tile in shared memory, rows of 128 bytes, 128-byte swizzle, 8-row groups 1024
// bytes apart (what a TMA box of 64 bf16 x rows with SWIZZLE_128B produces).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);           // start address
  d |= (uint64_t)1 << 16;                           // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset
  d |= (uint64_t)1 << 46;                           // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                           // SWIZZLE_128B
  return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = TC_BN.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TC_BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);

__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(IDESC), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ int find_group_tc(const GemmGroup* groups, int n, int tile) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (groups[mid].tile_start <= tile) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Epilogue of 32 consecutive columns [n, n+32) of one row.
__device__ __forceinline__ void epilogue_row(const GemmGroup& g, int m, int n, const uint32_t* r) {
  const int N = g.N;
  float v[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
  const bool full = (n + 32 <= N);
  if (g.epi & EPI_BIAS) {
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        float b[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(g.bias + n + j)), b);
#pragma unroll
        for (int e = 0; e < 8; ++e) v[j + e] += b[e];
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (n + j < N) v[j] += bf2f(g.bias[n + j]);
    }
  }
  if (g.epi & EPI_GELU) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
  }
  if (g.epi & EPI_RESID_F32) {
    float* C = reinterpret_cast<float*>(g.C) + (size_t)m * g.ldc + n;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        float4 c = *reinterpret_cast<float4*>(C + j);
        c.x += v[j]; c.y += v[j + 1]; c.z += v[j + 2]; c.w += v[j + 3];
        *reinterpret_cast<float4*>(C + j) = c;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (n + j < N) C[j] += v[j];
    }
  } else if (g.epi & EPI_SWIGLU) {
    bf16* C = reinterpret_cast<bf16*>(g.C) + (size_t)m * g.ldc + (n >> 1);
    if (full) {
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        o[j] = pack2(silu_f(v[4 * j]) * v[4 * j + 1], silu_f(v[4 * j + 2]) * v[4 * j + 3]);
      reinterpret_cast<uint4*>(C)[0] = make_uint4(o[0], o[1], o[2], o[3]);
      reinterpret_cast<uint4*>(C)[1] = make_uint4(o[4], o[5], o[6], o[7]);
    } else {
#pragma unroll
      for (int j = 0; j < 32; j += 2) if (n + j + 1 < N) C[j >> 1] = f2bf(silu_f(v[j]) * v[j + 1]);
    }
  } else {
    bf16* C = reinterpret_cast<bf16*>(g.C) + (size_t)m * g.ldc + n;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint4 o;
        o.x = pack2(v[j], v[j + 1]); o.y = pack2(v[j + 2], v[j + 3]);
        o.z = pack2(v[j + 4], v[j + 5]); o.w = pack2(v[j + 6], v[j + 7]);
        *reinterpret_cast<uint4*>(C + j) = o;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (n + j < N) C[j] = f2bf(v[j]);
    }
  }
}

__global__ void __launch_bounds__(N_THREADS, 1)
gemm_tc_kernel(const GemmGroup* __restrict__ groups, int n_groups, int total_tiles, int* __restrict__ status) {
  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte aligned tile area (128-byte swizzle atoms are 1024 bytes)
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bars = base + STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0;
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
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t issued_mask = 0, last_parity = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const GemmGroup* g = groups + find_group_tc(groups, n_groups, tile);
        const int local = tile - g->tile_start;
        const int m0 = (local / g->tiles_n) * TC_BM, n0 = (local % g->tiles_n) * TC_BN;
        tensormap_acquire(&g->tmA);
        tensormap_acquire(&g->tmW);
        const int kblocks = (g->K + TC_BK - 1) / TC_BK;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 1); break; }
          mbar_expect_tx(full_bar(stage), STAGE_BYTES);
          const uint32_t sa = base + stage * STAGE_BYTES;
          tma_load_2d(sa, &g->tmA, kb * TC_BK, m0, full_bar(stage));
          tma_load_2d(sa + A_BYTES, &g->tmW, kb * TC_BK, n0, full_bar(stage));
          issued_mask |= 1u << stage;
          last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
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
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const GemmGroup* g = groups + find_group_tc(groups, n_groups, tile);
        const int kblocks = (g->K + TC_BK - 1) / TC_BK;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; atomicExch(status, 2); break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TC_BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; atomicExch(status, 3); break; }
          tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES;
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)
            mma_f16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), (kb > 0 || k > 0) ? 1u : 0u);
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
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;             // TMEM lanes 32*quarter .. +31 belong to this warp
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const GemmGroup& g = groups[find_group_tc(groups, n_groups, tile)];
      const int local = tile - g.tile_start;
      const int m0 = (local / g.tiles_n) * TC_BM, n0 = (local % g.tiles_n) * TC_BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; if (lane == 0) atomicExch(status, 4); break; }
      tc_fence_after();
      const int m = m0 + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * TC_BN);
#pragma unroll 1
      for (int c = 0; c < TC_BN; c += 32) {
        if (n0 + c >= g.N) break;              // uniform across the warp
        uint32_t r[32];
        tmem_ld32(taddr + (uint32_t)c, r);
        if (m < g.M) epilogue_row(g, m, n0 + c, r);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

}  // namespace

cudaError_t launch_gemm_tc(const GemmGroup* groups, int n_groups, int total_tiles, int* status, int sm_count,
                           cudaStream_t st) {
  if (n_groups == 0 || total_tiles == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int grid = total_tiles < sm_count ? total_tiles : sm_count;
  gemm_tc_kernel<<<grid, N_THREADS, SMEM_BYTES, st>>>(groups, n_groups, total_tiles, status);
  return cudaGetLastError();
}

}  // namespace epara
