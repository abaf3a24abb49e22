// hga_selftest_bounded_wait: exercises the bounded mbarrier wait that every tensor-core kernel of
// this library uses, with a short limit and on a barrier that nothing completes, so that the
// give-up path (abort flag, clean exit, HGA_STATUS_WAIT_TIMEOUT in the status word) can be checked
// on a GPU without making a product kernel misbehave.  No TMA, no tensor memory.
#include "hga_common.cuh"
#include "hga_sm100.cuh"

namespace hga {

namespace {

__global__ void __launch_bounds__(64)
k_selftest_bounded_wait(long long cycle_limit, int32_t* status_word, long long* waited_cycles) {
  __shared__ uint64_t never;      // one arrival expected, none ever made
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&never, 1);
    abort_flag = 0;
    sm100::fence_barrier_init();
  }
  __syncthreads();
  volatile int* abort = &abort_flag;
  // warp 0 waits for the barrier with the short limit; warp 1 waits with the product limit and must
  // be released by the abort flag warp 0 raises, as the other roles of a product kernel are
  const long long t0 = clock64();
  const bool ok = threadIdx.x < 32 ? sm100::mbar_wait_bounded(&never, 0, abort, cycle_limit)
                                   : sm100::mbar_wait_bounded(&never, 0, abort);
  const long long waited = clock64() - t0;
  const bool all_gave_up = __syncthreads_and(!ok);
  if (threadIdx.x == 0) {
    if (all_gave_up && abort_flag) atomicOr(status_word, HGA_STATUS_WAIT_TIMEOUT);
    if (waited_cycles) *waited_cycles = waited;
  }
}

}  // namespace

}  // namespace hga

extern "C" int hga_selftest_bounded_wait(uint32_t cycle_limit, int32_t* status_word, long long* waited_cycles,
                                         void* stream) {
  if (!status_word) return HGA_ERR_NULL;
  if (cycle_limit < 1 || cycle_limit > (1u << 24)) return HGA_ERR_SHAPE;
  hga::k_selftest_bounded_wait<<<1, 64, 0, (cudaStream_t)stream>>>((long long)cycle_limit, status_word, waited_cycles);
  hga::count_launch(HGA_KERNELS_AUX);
  return hga::record_cuda(cudaGetLastError());
}
