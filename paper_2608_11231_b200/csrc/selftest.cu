// Self-test of the bounded device-side wait: the give-up path that every tensor-core kernel of the library
// shares (tc::mbar_wait) is taken on purpose, with a small poll limit, by a kernel that does nothing else.
// It neither faults nor hangs: the wait returns false after `poll_limit` polls, the status word is set, the
// kernel ends.
#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

__global__ void selftest_bounded_wait_kernel(uint32_t poll_limit, int32_t *status) {
    __shared__ uint64_t bar;
    __shared__ volatile int dead;
    if (threadIdx.x == 0) {
        dead = 0;
        tc::mbar_init(&bar, 1);      // one arrival expected: none ever comes
        tc::mbar_fence_init();
    }
    __syncthreads();
    const bool done = tc::mbar_wait(&bar, 0, &dead, status, poll_limit);
    // after the first wait has run out, every later wait in the CTA returns at once
    const bool again = tc::mbar_wait(&bar, 0, &dead, status, poll_limit);
    if (done || again) atomicExch(status + 1, 1);   // must not happen: word 1 of the header flags it
}

}  // namespace

cudaError_t launch_selftest_bounded_wait(uint32_t poll_limit, int32_t *status, cudaStream_t s) {
    selftest_bounded_wait_kernel<<<1, 64, 0, s>>>(poll_limit, status);
    return cudaGetLastError();
}

}  // namespace lkv
