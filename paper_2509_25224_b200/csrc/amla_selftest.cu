// Self-test of the bounded device-side wait (diagnostic; not on the decode path).
//
// Every wait inside the decode kernels gives up after a time limit, records kStatusTimeout in the status word and lets
// the kernel return, so that a lost signal shows up as AMLA_ERR_DEVICE_TIMEOUT instead of a hung GPU.  This kernel
// makes that path observable without disturbing a real decode: one warp initialises an mbarrier that nothing ever
// arrives on, waits on it through the same mbar_wait the kernels use, with a caller-chosen (short) limit, and
// records the outcome.  No TMA, no tensor memory, no second CTA: when the limit passes, the kernel simply ends.
#include "amla_common.cuh"
#include "amla_sm100.cuh"

namespace amla {

__global__ void __launch_bounds__(32, 1) wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar_storage;
  const uint32_t bar = sm100::smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    *status = kStatusOk;
    sm100::mbar_init(bar, 1);
  }
  __syncwarp();
  // phase 0 never completes: there is no arrival
  const bool ok = __all_sync(0xffffffffu, sm100::mbar_wait(bar, 0, limit_ns));
  if (!ok && threadIdx.x == 0) atomicExch(status, kStatusTimeout);
}

cudaError_t launch_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t stream) {
  wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
  return cudaGetLastError();
}

}  // namespace amla
