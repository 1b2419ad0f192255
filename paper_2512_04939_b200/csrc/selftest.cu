// Self-test of the bounded-wait protocol that every pipelined kernel of the library relies on.
//
// A kernel whose mbarrier wait is never satisfied must not hang: the wait gives up after its
// cycle limit, raises the CTA's abort flag and the context's device status word, every other
// wait in the CTA sees the flag and gives up as well, and the kernel returns normally, leaving
// the context usable.  The production kernels never get there on valid input, so this one-CTA
// kernel walks the same helpers (mbar_wait, mbar_wait_warp, WaitCtl) on a barrier that nobody
// arrives on, with a short limit.  Nothing faults, traps or spins without a bound.
#include "common.cuh"
#include "runtime.h"

namespace lv {

__global__ void __launch_bounds__(64, 1)
bounded_wait_selftest_kernel(long long limit_cycles, uint32_t* status, uint32_t* outcome) {
  __shared__ uint64_t never_arrived;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&never_arrived, 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  const WaitCtl ctl{&abort_flag, status, limit_cycles};
  bool done;
  if (threadIdx.x < 32) {
    // warp 0: one elected thread waits like a producer / issuer thread does
    done = true;
    if (elect_one()) done = mbar_wait(&never_arrived, 0, ctl);
    done = __all_sync(0xffffffffu, done ? 1 : 0) != 0;
  } else {
    // warp 1: the warp-uniform flavour of the softmax / epilogue warps; it gives up either on its own
    // limit or on warp 0's abort flag, whichever comes first
    done = mbar_wait_warp(&never_arrived, 0, ctl);
  }
  __syncthreads();
  // bit 0 / bit 1: warp 0 / warp 1 came back from its wait claiming that the phase had completed
  if ((threadIdx.x & 31) == 0 && done) atomicOr(outcome, 1u << (threadIdx.x >> 5));
  if (threadIdx.x == 0) atomicOr(outcome, 4u);  // the kernel reached its end
}

cudaError_t launch_bounded_wait_selftest(litevggt_ctx* ctx, long long limit_cycles, uint32_t* outcome, cudaStream_t s,
                                         int* launches) {
  cudaError_t e = cudaMemsetAsync(outcome, 0, sizeof(uint32_t), s);
  if (e != cudaSuccess) return e;
  bounded_wait_selftest_kernel<<<1, 64, 0, s>>>(limit_cycles, ctx->ws.status, outcome);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace lv
