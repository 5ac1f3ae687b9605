// Diagnostic entry point: shows, without harming the device, what the kernels do when a barrier they wait on
// is never satisfied.  One block waits on an mbarrier that nothing arrives at, through the same bounded-wait
// helper the decode kernel uses; the wait gives up after its limit (about 0.2 s), raises
// TRANSMLA_DEV_TIMEOUT in the status word, later waits return at once, and the kernel ends normally.
#include "common.cuh"

namespace transmla {

__global__ void bounded_wait_probe_kernel(int32_t* dev_status, long long* cycles_out) {
  __shared__ uint64_t bar_storage;
  __shared__ int abort_s;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const long long t0 = clock64();
  mbar_wait(bar, 0, &abort_s, dev_status);  // expires: nobody arrives
  const long long t1 = clock64();
  mbar_wait(bar, 0, &abort_s, dev_status);  // returns at once: the block has already given up
  const long long t2 = clock64();
  if (threadIdx.x == 0 && cycles_out != nullptr) {
    cycles_out[0] = t1 - t0;
    cycles_out[1] = t2 - t1;
  }
}

}  // namespace transmla

extern "C" transmla_status_t transmla_selftest_bounded_wait(int32_t* dev_status, long long* cycles_out, void* stream) {
  if (dev_status == nullptr) return TRANSMLA_ERR_NULL;
  transmla::bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(dev_status, cycles_out);
  return cudaGetLastError() == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}
