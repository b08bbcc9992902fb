// Neuron selection by threshold (Eq. base_threshold, last line; Algorithm 2 mask generation) and
// the order-statistic helper that places a threshold at a given sparsity.
#include <math.h>

#include "common.cuh"
#include "nvtx_ranges.cuh"

namespace clada {

constexpr int kSelThreads = 1024;

// One CTA per sequence.  Each warp owns a contiguous run of 32-neuron chunks, so warp ballots give
// ascending positions directly: pass 1 counts, a scan over warp totals gives each warp its base,
// pass 2 writes.
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float *__restrict__ scores, int d_ff, const float *__restrict__ tau,
              int64_t tau_stride, uint8_t *__restrict__ mask, int32_t *__restrict__ idx,
              int32_t *__restrict__ count) {
    const int b = blockIdx.x;
    const float *A = scores + (size_t)b * d_ff;
    const float t = tau[(size_t)b * tau_stride];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kSelThreads / kWarp;
    const int chunks = (d_ff + kWarp - 1) / kWarp;
    const int per_warp = (chunks + kWarps - 1) / kWarps;
    const int c0 = warp * per_warp, c1 = min(chunks, c0 + per_warp);

    int n = 0;
    for (int c = c0; c < c1; ++c) {
        const int j = c * kWarp + lane;
        const bool keep = j < d_ff && A[j] >= t;
        n += __popc(__ballot_sync(0xffffffffu, keep));
    }
    __shared__ int s_tot[kWarps];
    if (lane == 0) s_tot[warp] = n;
    __syncthreads();
    int base = 0, total = 0;
    for (int w = 0; w < kWarps; ++w) {
        const int v = s_tot[w];
        base += (w < warp) ? v : 0;
        total += v;
    }
    for (int c = c0; c < c1; ++c) {
        const int j = c * kWarp + lane;
        const bool keep = j < d_ff && A[j] >= t;
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        if (j < d_ff && mask) mask[(size_t)b * d_ff + j] = keep ? 1 : 0;
        if (keep && idx) idx[(size_t)b * d_ff + base + __popc(bal & ((1u << lane) - 1u))] = j;
        base += __popc(bal);
    }
    if (threadIdx.x == 0 && count) count[b] = total;
}

// r-th smallest (0-based) of non-negative floats by most-significant-byte-first radix selection
// on their bit patterns (monotone for non-negative IEEE floats).
__device__ float radix_select(const float *__restrict__ A, int n, int r, int *s_hist, int *s_pick) {
    uint32_t prefix = 0, pmask = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) s_hist[i] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += blockDim.x) {
            const uint32_t u = __float_as_uint(A[j]);
            if ((u & pmask) == prefix) atomicAdd(&s_hist[(u >> shift) & 255u], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int acc = 0, bin = 0;
            for (; bin < 255; ++bin) {
                if (acc + s_hist[bin] > r) break;
                acc += s_hist[bin];
            }
            s_pick[0] = bin;
            s_pick[1] = r - acc;
        }
        __syncthreads();
        prefix |= (uint32_t)s_pick[0] << shift;
        pmask |= 255u << shift;
        r = s_pick[1];
        __syncthreads();
    }
    return __uint_as_float(prefix);
}

__global__ void __launch_bounds__(kSelThreads)
tau_from_sparsity_kernel(const float *__restrict__ scores, int d_ff, int k_cut,
                         float *__restrict__ tau_base) {
    __shared__ int s_hist[256];
    __shared__ int s_pick[2];
    const int b = blockIdx.x;
    const float *A = scores + (size_t)b * d_ff;
    float out;
    if (k_cut <= 0) {
        out = 0.f;
    } else if (k_cut >= d_ff) {
        out = INFINITY;
    } else {
        const float lo = radix_select(A, d_ff, k_cut - 1, s_hist, s_pick);
        const float hi = radix_select(A, d_ff, k_cut, s_hist, s_pick);
        out = __fadd_rn(__fmul_rn(0.5f, lo), __fmul_rn(0.5f, hi));
    }
    if (threadIdx.x == 0) tau_base[b] = out;
}

}  // namespace clada

using namespace clada;

extern "C" {

int clada_select(const float *scores, int32_t B, int32_t d_ff, const float *tau, int64_t tau_stride,
                 uint8_t *mask, int32_t *idx, int32_t *count, void *stream) {
    CLADA_RANGE("clada_select");
    if (!scores || !tau) return CLADA_ERR_NULL;
    if (B <= 0 || d_ff <= 0 || tau_stride < 0) return CLADA_ERR_SHAPE;
    select_kernel<<<B, kSelThreads, 0, static_cast<cudaStream_t>(stream)>>>(scores, d_ff, tau, tau_stride,
                                                                           mask, idx, count);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

int clada_tau_from_sparsity(const float *scores, int32_t B, int32_t d_ff, float rho, float *tau_base,
                            void *stream) {
    CLADA_RANGE("clada_tau_from_sparsity");
    if (!scores || !tau_base) return CLADA_ERR_NULL;
    if (B <= 0 || d_ff <= 0 || !(rho >= 0.f && rho <= 1.f)) return CLADA_ERR_SHAPE;
    const int k_cut = (int)floor((double)rho * d_ff + 0.5);
    tau_from_sparsity_kernel<<<B, kSelThreads, 0, static_cast<cudaStream_t>(stream)>>>(scores, d_ff, k_cut,
                                                                                     tau_base);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

}  // extern "C"
