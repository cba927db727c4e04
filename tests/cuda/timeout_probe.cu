// Test-only kernel (built by tests/test_gpu_timeout.py, not part of the library): one warp calls the
// library's bounded barrier wait on an mbarrier that nothing ever arrives at, with a limit of about a
// millisecond instead of the library's default.  The wait runs out, records SPARKATTN_E_DEVICE_TIMEOUT and
// the wait id in the status words of the workspace, and the kernel returns normally: no trap, no fault,
// nothing left spinning.
#include "../../paper_2609_23153_b200/csrc/common.cuh"

using namespace sparkattn;

__global__ void timeout_probe_kernel(int32_t* status, unsigned long long limit_ns, int wait_id) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0, &abort_flag, status, wait_id, limit_ns);
  // word 2: threads whose wait gave up; word 3: threads that (wrongly) saw the barrier flip
  atomicAdd(status + (ok ? 3 : 2), 1);
}

extern "C" int timeout_probe(void* workspace, unsigned long long limit_ns, int wait_id, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, s) != cudaSuccess) return -1;
  timeout_probe_kernel<<<1, 32, 0, s>>>(static_cast<int32_t*>(workspace), limit_ns, wait_id);
  return cudaGetLastError() == cudaSuccess ? 0 : -1;
}
