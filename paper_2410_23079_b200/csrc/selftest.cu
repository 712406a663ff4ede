// Self-test of the library's failure detection: what happens when a bounded on-device wait runs out.
//
// Every mbarrier wait in the tensor-core prefill kernels gives up after a fixed number of polls,
// records BUZZ_ERR_TIMEOUT in the device status word and lets the CTA run to its end. In a correct
// build no wait ever expires, so that path would otherwise never execute. This entry point runs it
// on purpose, harmlessly: ONE CTA initialises an mbarrier that expects one arrival, nobody arrives,
// one thread waits on it through the same bounded wait the prefill kernels use (with a small poll
// limit), the wait gives up, the status word is set the same way, and the kernel returns by itself.
// Nothing traps, nothing spins without a limit, and the context stays usable.
#include "buzz_internal.cuh"
#include "sm100_ptx.cuh"

namespace {

__global__ void __launch_bounds__(32)
wait_expiry_kernel(int32_t* status, uint32_t polls) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    sm100::fence_barrier_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    // phase 0 never completes: the barrier's single expected arrival is never made
    if (!sm100::mbar_wait(&bar, 0, polls)) buzz_set_status(status, BUZZ_ERR_TIMEOUT, -1, (int)polls);
  }
}

}  // namespace

extern "C" int buzz_selftest_wait_expiry(buzz_t c, int polls, void* stream) {
  if (!c || polls < 1 || polls > (1 << 16)) return BUZZ_ERR_INVALID;
  (void)cudaGetLastError();
  wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(c->st.status, (uint32_t)polls);
  c->launches += 1;
  c->last_kind = 2;
  return cudaGetLastError() == cudaSuccess ? BUZZ_OK : BUZZ_ERR_CUDA;
}
