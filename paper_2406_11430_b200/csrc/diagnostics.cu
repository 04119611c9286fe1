// Self-test of the give-up path of the bounded waits (l2kv_selftest_wait_timeout).
#include "async_copy.cuh"

namespace l2kv {

// One thread block waits on an mbarrier that expects one arrival which never comes; no copy
// targets the barrier or shared memory, so giving up leaves nothing in flight.
__global__ void __launch_bounds__(32) wait_timeout_kernel(int32_t* status_word) {
  __shared__ __align__(8) unsigned long long s_bar;
  const uint32_t bar = smem_u32(&s_bar);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait<10>(bar, 0);        // 1024 polls, then false
  if (!ok) record_timeout(status_word);
}

}  // namespace l2kv

extern "C" int l2kv_selftest_wait_timeout(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return L2KV_ERR_INVALID_ARG;
  if (workspace_bytes < (size_t)l2kv::kStatusBytes) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  l2kv::wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<int32_t*>(workspace));
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}
