// Self-test of the bounded-wait plumbing.  Every mbarrier wait of the tensor-core kernels gives up after a fixed
// number of attempts, records a bit in the context's device error word and lets its thread block run to its exit;
// the host then reports TREEKV_ERR_TIMEOUT from treekv_get_stats until treekv_reset.  In a healthy run no wait
// ever gives up, so this file provides the one place where it does by construction: a kernel of one thread block
// that waits, with the same helper and a small attempt limit, on a barrier that nothing will ever signal, with no
// asynchronous operation outstanding.  It touches nothing of the cache.
#include "common.cuh"
#include "ctx.cuh"
#include "tma.cuh"

using namespace treekv;

namespace {
constexpr unsigned kErrSelfTestWait = 64u;

__global__ void wait_giveup_kernel(DevStats* stats, uint32_t attempts) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t addr = smem_addr_u32(&bar);
    if (threadIdx.x == 0) { mbar_init(addr, 1); mbar_fence_init(); }
    __syncthreads();
    // phase 0 of a fresh barrier with one expected arrival and no arriver never completes
    if (threadIdx.x == 0 && !mbar_wait_limit(addr, 0, attempts)) atomicOr(&stats->error, kErrSelfTestWait);
}
}  // namespace

extern "C" treekv_status treekv_selftest_wait_giveup(treekv_ctx* ctx, int attempts, void* stream) {
    if (!ctx || attempts < 1 || attempts > 4096) return TREEKV_ERR_INVALID_ARG;
    wait_giveup_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->cv.stats, (uint32_t)attempts);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return TREEKV_ERR_CUDA; }
    ctx->launches += 1;
    return TREEKV_OK;
}
