// A wait that cannot succeed, on purpose bounded: the same bounded-wait helper and the same status
// word the kernels of this library use, so that the "a wait gave up" path — poll limit reached,
// H2O_ERR_TIMEOUT recorded, kernel returns normally, context stays usable — can be exercised without
// hanging or faulting anything.  The barrier below expects one arrival that nobody ever makes.
#include "h2o_internal.cuh"
#include "sm100_ptx.cuh"

namespace h2o {

namespace {

__global__ void wait_probe_kernel(int32_t* status, uint32_t polls) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  bool done = false;
  for (uint32_t it = 0; it < polls && !done; ++it) done = ptx::mbar_try_wait(&bar, 0);
  if (!done && threadIdx.x == 0) atomicCAS(status, 0, H2O_ERR_TIMEOUT);
}

}  // namespace

cudaError_t launch_wait_probe(const CacheView& c, uint32_t polls, cudaStream_t stream) {
  wait_probe_kernel<<<1, 32, 0, stream>>>(c.status, polls);
  return cudaGetLastError();
}

}  // namespace h2o
