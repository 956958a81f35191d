// Self-test of the bounded wait every tensor-core kernel relies on: one thread waits on an mbarrier
// that nothing ever arrives at, with a short limit, and must come back by itself with the status word
// set.  This is the only way the give-up path is exercised without making a real kernel misbehave.
#include "../../include/epara.h"
#include "common.cuh"
#include "tcgen05.cuh"

namespace epara {
namespace {

__global__ void __launch_bounds__(32, 1) bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    tc::mbar_init(tc::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // phase 0 of a fresh barrier with one pending arrival never completes: the wait must run out
    const bool done = tc::mbar_wait<true>(tc::smem_u32(&bar), 0u, &abort_flag, limit_ns);
    if (!done) atomicExch(status, ERR_SELFTEST_WAIT);
  }
}

}  // namespace
}  // namespace epara

extern "C" int epara_selftest_bounded_wait(int device, void* cuda_stream, unsigned long long limit_ns, int* status_dev,
                                           int* code) {
  if (!status_dev || !code || limit_ns == 0 || limit_ns > 1000000000ull) return EPARA_E_INVALID;
  *code = 0;
  if (cudaSetDevice(device) != cudaSuccess) return EPARA_E_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemsetAsync(status_dev, 0, sizeof(int), st) != cudaSuccess) return EPARA_E_CUDA;
  epara::bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status_dev, limit_ns);
  if (cudaGetLastError() != cudaSuccess) return EPARA_E_CUDA;
  if (cudaMemcpyAsync(code, status_dev, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return EPARA_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return EPARA_E_CUDA;
  return *code != 0 ? EPARA_E_DEVICE : EPARA_OK;
}
