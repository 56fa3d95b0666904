// Test-only probe (compiled into the wait-test variant of the library, never into the product): one warp waits,
// with the library's bounded wait, on an mbarrier that nothing ever arrives at.  No TMA, no tensor-core work and
// no TMEM is involved; the wait gives up after its cycle limit, records MOSAIC_E_DEVICE_TIMEOUT and the kernel
// returns normally.
#include "tc_common.cuh"

namespace mosaic {

__global__ void wait_probe_kernel(int* status, int* result) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(s32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const long long t0 = clock64();
  const bool ok = mbar_wait(s32(&bar), 0, &abort_flag, status);   // phase 0 never completes
  const long long dt = clock64() - t0;
  if (threadIdx.x == 0) { result[0] = ok ? 1 : 0; result[1] = (int)(dt >> 10); }
}

}  // namespace mosaic

// Launches the probe on `cuda_stream`; `status` and `result` are device pointers (1 and 2 ints).
extern "C" int mosaic_test_wait_probe(int* status, int* result, void* cuda_stream) {
  mosaic::wait_probe_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(status, result);
  return cudaGetLastError() == cudaSuccess ? 0 : -5;
}
