// Self-test of the bounded device-side wait that every tensor-core kernel of the library relies on.
#include "kernels.h"
#include "tc_common.cuh"

namespace ast {
namespace {

// One warp waits, with a limit of `limit` polls, on an mbarrier at which nobody ever arrives.  The wait must give up and
// the kernel must return with the error word set, exactly as the pipelines do when a hand-off never comes.
__global__ void bounded_wait_probe(int* err, uint32_t limit) {
    __shared__ uint64_t bar;
    const uint32_t b = tc::smem_u32(&bar);
    if (threadIdx.x == 0) tc::mbar_init(b, 1);
    __syncthreads();
    const bool ok = tc::mbar_wait_limit(b, 0u, limit);
    if (!__syncthreads_and(ok ? 1 : 0) && threadIdx.x == 0) atomicExch(err, 1);
}

}  // namespace

void launch_bounded_wait_probe(int* err, unsigned limit, cudaStream_t st) { bounded_wait_probe<<<1, 32, 0, st>>>(err, limit); }

}  // namespace ast
