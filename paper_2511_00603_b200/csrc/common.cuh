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

// GELU in its erf form, 0.5 x (1 + erf(x / sqrt 2)), evaluated as 0.5 x (1 + tanh(x P(x^2))) with
// P(t) = a + b t + c t^2 fitted (minimax over |x| <= 8) so that tanh(x P(x^2)) follows erf(x / sqrt 2):
// the formula itself is within 2.6e-5 of the erf form everywhere.  t is clamped at 64, where the
// argument is already past saturation, because c < 0 would turn P around for |x| > 11.  tanh comes
// from the hardware approximation (relative error 2^-11 of tanh), which bounds the absolute error of
// the result by about 2.5e-4 |x|: below the rounding of the bf16 store for x > 0, and of the size of
// that rounding at the typical magnitude of the tensor for the small negative outputs.
// Seven FMA-pipe instructions and one special-function instruction per element.
__device__ __forceinline__ float gelu_erf(float x) {
  const float t = fminf(x * x, 64.0f);
  float p = fmaf(t, -3.51516781e-4f, 3.70056460e-2f);
  p = fmaf(t, p, 7.97507884e-1f);
  float th;
  asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(x * p));
  const float hx = 0.5f * x;
  return fmaf(hx, th, hx);
}
// x / (1 + e^-x) with the fast division (2 ulp; the denominator is at least 1, and an overflowed e^-x gives 0,
// the limit).  The IEEE division's special-case path, which a zero numerator takes, measured 3x slower in
// the epilogue loops.
__device__ __forceinline__ float silu_f(float x) { return __fdividef(x, 1.0f + __expf(-x)); }

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
