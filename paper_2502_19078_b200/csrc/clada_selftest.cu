// Self-test of the bounded waits: the decode kernels' two wait primitives (an mbarrier wait and the grid
// barrier) are made to run out in a harmless form -- a barrier nobody arrives at, a grid barrier that
// expects one CTA more than the grid has -- with a small poll limit, so that the give-up branch, the
// status bit and the recovery by clada_workspace_init can be exercised without any kernel ever hanging.
#include "common.cuh"
#include "ffn_common.cuh"

namespace clada {

__global__ void __launch_bounds__(64, 1)
bounded_wait_selftest_kernel(WsCtrl *ctrl, unsigned poll_limit, int32_t *report, int32_t *status) {
    __shared__ uint64_t bar;
    __shared__ int gave_up;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);  // one arrival expected; none will come
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        gave_up = 0;
    }
    __syncthreads();
    // every thread waits for phase 0 of the barrier, as the consumers of a ring stage do
    if (!mbar_wait(smem_u32(&bar), 0, poll_limit)) atomicOr(&gave_up, 1);
    __syncthreads();
    const bool mbar_gave_up = gave_up != 0;
    // the grid barrier of a grid of gridDim.x CTAs that is told to expect one more
    const bool barrier_ok = grid_barrier(ctrl, gridDim.x + 1u, 32, poll_limit);
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        report[0] = mbar_gave_up ? 1 : 0;
        report[1] = barrier_ok ? 0 : 1;
    }
    if (threadIdx.x == 0 && (mbar_gave_up || !barrier_ok) && status) atomicOr(status, CLADA_STATUS_TIMEOUT);
}

}  // namespace clada

using namespace clada;

extern "C" int clada_selftest_bounded_waits(void *ws, size_t ws_bytes, uint32_t poll_limit, int32_t *report,
                                            int32_t *status, void *stream) {
    if (!ws || !report) return CLADA_ERR_NULL;
    if (ws_bytes < kWsCtrlBytes || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    if (poll_limit == 0 || poll_limit > (1u << 20)) return CLADA_ERR_SHAPE;  // at most about a second per wait
    bounded_wait_selftest_kernel<<<2, 64, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<WsCtrl *>(ws), poll_limit,
                                                                               report, status);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}
