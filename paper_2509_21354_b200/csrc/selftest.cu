// kvE_selftest_timeout: makes the two bounded-wait helpers of the library run out on purpose, safely.
// Every kernel of the library waits on mbarriers (copies landing, tensor-core commits, peers of a cluster) through
// mbar_wait_bounded / mbar_wait_cluster_bounded; when such a wait gives up, the kernel records KVE_ERR_TIMEOUT in the
// status word and leaves in order.  Here a barrier is armed with bytes (or an arrival) that nothing ever delivers and
// the wait limit is a few thousand polls / two milliseconds: the kernel must return, the status word must read
// KVE_ERR_TIMEOUT, and the context must stay usable.  Nothing faults, traps or spins without a bound.
#include "gate_rnn.cuh"

namespace kve {

// which 0: a CTA waits for 16 bytes of a bulk copy that is never issued (the wait of the copy pipelines)
__global__ void __launch_bounds__(32) kve_selftest_cta_wait_kernel(int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
    mbar_arrive_expect_tx(&bar, 16);      // the arrival is there, the bytes never come: the phase cannot complete
  }
  __syncwarp();
  const bool ok = mbar_wait_bounded(&bar, 0, 4096);
  if (!ok && threadIdx.x == 0) set_status(status, ERR_TIMEOUT);
}

// which 1: the two CTAs of a cluster each wait for an arrival from the peer that the peer never sends (the wait of the
// recurrence kernel); both give up after two milliseconds, then leave together like that kernel does
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(32) kve_selftest_cluster_wait_kernel(int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  cluster_sync_all();
  const bool ok = mbar_wait_cluster_bounded(&bar, 0, 2000000ull);
  if (!ok && threadIdx.x == 0) set_status(status, ERR_TIMEOUT);
  cluster_sync_all();      // nobody leaves while a peer could still address its shared memory
}

cudaError_t launch_selftest_timeout(int which, int32_t* status, cudaStream_t st) {
  if (which == 0) kve_selftest_cta_wait_kernel<<<1, 32, 0, st>>>(status);
  else kve_selftest_cluster_wait_kernel<<<2, 32, 0, st>>>(status);
  return cudaGetLastError();
}

}  // namespace kve
