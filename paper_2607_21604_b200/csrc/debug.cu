// Test hooks that are not part of the serving surface.
#include "tc_common.cuh"

// One warp waits on a barrier that nothing arrives at, with the bounded wait of the tensor-core
// kernels; when the limit runs out it records AKVS_ERR_TIMEOUT and returns like they do.
__global__ void wait_timeout_kernel(int32_t* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (!tc::mbar_wait(&bar, 0, &abort_flag, limit_cycles)) {
      abort_flag = 1;
      set_status(status, AKVS_ERR_TIMEOUT);
    }
  }
  __syncthreads();
}

extern "C" int32_t akvs_debug_wait_timeout(void* workspace, int64_t limit_cycles, void* stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return AKVS_ERR_WORKSPACE;
  long long lim = limit_cycles < 1000 ? 1000 : (limit_cycles > 200000000ll ? 200000000ll : limit_cycles);
  wait_timeout_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(reinterpret_cast<int32_t*>(workspace), lim);
  AKVS_LAUNCHED();
  return AKVS_OK;
}
