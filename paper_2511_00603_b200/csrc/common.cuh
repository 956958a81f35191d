// Small device helpers shared by the kernels.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include "desc.h"

namespace epara {

// Programmatic dependent launch.  Every kernel of a step is launched with programmatic stream
// serialisation: it may become resident while the kernel before it in the stream is still running,
// which hides launch latency and set-up.  pdl_launch_dependents() lets the next kernel start
// launching; pdl_wait() returns once all earlier kernels have completed and their writes are
// visible.  Rule: a kernel touches nothing that an earlier kernel of the stream writes or reads
// before its pdl_wait(); weights and the step's descriptors (uploaded by a copy that completes
// before the first kernel) may be read earlier.  Every kernel waits at least once, so completion
// is transitive along the stream.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// (one thread per block is enough; a block that exits counts as having triggered)
__device__ __forceinline__ void pdl_launch_dependents() {
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ float bf2f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ bf16 f2bf(float v) { return __float2bfloat16_rn(v); }

// 8 bf16 packed in a uint4 -> 8 floats (bf16 is the top half of an fp32).
__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
}

__device__ __forceinline__ unsigned pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<unsigned*>(&v);
}

// GELU in its erf form, 0.5 x (1 + erf(x / sqrt 2)).  erf comes from the rational approximation
// 1 - erf(z) = (1 + a1 z + ... + a6 z^6)^-16 for z >= 0 (Abramowitz & Stegun 7.1.28, |error| <= 3e-7),
// one reciprocal and no branches; 1 + erf of a negative argument is taken as 1 - erf(|z|) directly,
// so the negative tail has no cancellation.  Absolute error of the result below 1e-6.
__device__ __forceinline__ float gelu_erf(float x) {
  const float z = fabsf(x) * 0.70710678118654752f;
  float p = 0.0000430638f;
  p = fmaf(p, z, 0.0002765672f);
  p = fmaf(p, z, 0.0001520143f);
  p = fmaf(p, z, 0.0092705272f);
  p = fmaf(p, z, 0.0422820123f);
  p = fmaf(p, z, 0.0705230784f);
  p = fmaf(p, z, 1.0f);
  p *= p; p *= p; p *= p; p *= p;
  const float r = __fdividef(1.0f, p);        // 1 - erf(|z|); for huge |x| p is inf or huge and r is 0
  return 0.5f * x * (x > 0.f ? 2.0f - r : r);
}
__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum for blocks of up to 1024 threads; `red` is 32 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < nw) ? red[l] : 0.f;
  t = warp_sum(t);
  return t;
}

}  // namespace epara
