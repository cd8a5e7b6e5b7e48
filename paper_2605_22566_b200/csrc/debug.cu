// Diagnostics behind the gf_debug_* entry points: nothing here is on the attention path.
#include "gf_device.cuh"

namespace gf {
namespace {

// One warp waits, with the given limit, on a barrier that nobody ever arrives at: the bounded wait
// must run out, record the give-up status and return, and the kernel must end.
__global__ void k_wait_probe(int32_t* status, long long limit, int32_t* returned) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool done = mbar_wait(&bar, 0, status, limit);
    *returned = done ? 1 : 2;  // 2: the wait gave up
  }
}

}  // namespace

int launch_wait_probe(int32_t* status, long long limit, int32_t* returned, cudaStream_t st) {
  k_wait_probe<<<1, 32, 0, st>>>(status, limit, returned);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
