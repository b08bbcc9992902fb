// Offline error-controlled threshold search (Eq. base_threshold):
//   tau_base = argmax eps  s.t.  mean over validation samples x of CETT(x; eps) <= bound,
//   CETT(x; eps) = || sum_{A_j(x) < eps} n_j(x) ||_F / || MLP(x) ||_F.
//
// For one sample, cutting the k lowest-scored neurons gives the numerator ||C_k||, C_k = sum of the outputs
// n_j = z_{:,j} (outer) W_out,j of the first k neurons in ascending score order, and C_F is the dense output:
// one pass over the neurons in that order yields CETT for every cut size.  Steps:
//   1. scores and z (neuron-major) from the prefill-statistics GEMM;
//   2. per sample, neurons sorted by score (bitonic sort of (score, index) keys in shared memory);
//   3. per sample, the running sum C over a (32 tokens x 128 columns) tile per CTA, 4 x 4 elements per
//      thread in registers; after each neuron the tile's sum of squares goes to a per-tile partial row;
//   4. per sample, partial rows added in tile order (fp64): cum[k] = ||C_k||^2;
//   5. every score of every sample is a candidate eps; a candidate is feasible if the mean over samples
//      of sqrt(cum[k_x(eps)] / cum[F]) is within the bound (k_x by binary search); the largest feasible wins.
#include <math.h>

#include <algorithm>

#include "common.cuh"
#include "nvtx_ranges.cuh"
#include "prefix_common.cuh"

namespace clada {

constexpr int kSortThreads = 1024;
constexpr int kMaxSortN = 16384;

// Ascending by (score, index): 64-bit keys, scores are non-negative so their bit patterns order them.
__global__ void __launch_bounds__(kSortThreads)
cett_sort_kernel(const float *__restrict__ scores, int d_ff, int n_pow2, int32_t *__restrict__ order,
                 float *__restrict__ sorted) {
    extern __shared__ unsigned long long s_keys[];
    const int b = blockIdx.x;
    const float *A = scores + (size_t)b * d_ff;
    for (int i = threadIdx.x; i < n_pow2; i += kSortThreads)
        s_keys[i] = i < d_ff ? (((unsigned long long)__float_as_uint(A[i]) << 32) | (unsigned)i) : ~0ull;
    __syncthreads();
    for (int k = 2; k <= n_pow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < n_pow2; i += kSortThreads) {
                const int l = i ^ j;
                if (l > i) {
                    const unsigned long long a = s_keys[i], c = s_keys[l];
                    const bool up = (i & k) == 0;
                    if ((a > c) == up) {
                        s_keys[i] = c;
                        s_keys[l] = a;
                    }
                }
            }
            __syncthreads();
        }
    }
    for (int i = threadIdx.x; i < d_ff; i += kSortThreads) {
        order[(size_t)b * d_ff + i] = (int32_t)(s_keys[i] & 0xffffffffull);
        sorted[(size_t)b * d_ff + i] = __uint_as_float((unsigned)(s_keys[i] >> 32));
    }
}

constexpr int kCumThreads = 256;
constexpr int kCumTok = 32, kCumCol = 128, kCumChunk = 32;

// Grid (column tiles, token tiles) of ONE sample whose tokens are rows [t0, t1) of the prompt batch.
template <typename T>
__global__ void __launch_bounds__(kCumThreads)
cett_cumulative_kernel(const float *__restrict__ zt, long long zt_stride, const T *__restrict__ Wd_t, int d_model,
                       int d_ff, const int32_t *__restrict__ order, long long t0, long long t1,
                       float *__restrict__ partials) {
    __shared__ float s_z[kCumChunk][kCumTok];
    __shared__ float s_w[kCumChunk][kCumCol];
    __shared__ float s_q[kCumThreads / kWarp][kCumChunk];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tx = tid & 31, ty = tid >> 5;  // 4 columns x 4 tokens per thread
    const long long tok0 = t0 + (long long)blockIdx.y * kCumTok;
    const int col0 = blockIdx.x * kCumCol;
    const int tile = blockIdx.y * gridDim.x + blockIdx.x;
    float c[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = 0.f;

    for (int k0 = 0; k0 < d_ff; k0 += kCumChunk) {
        // stage this chunk's z slices (32 tokens) and W_out slices (128 columns), zero outside the sample
        for (int e = tid; e < kCumChunk * kCumTok; e += kCumThreads) {
            const int kk = e / kCumTok, tt = e % kCumTok;
            float v = 0.f;
            if (k0 + kk < d_ff && tok0 + tt < t1) v = zt[(size_t)order[k0 + kk] * zt_stride + tok0 + tt];
            s_z[kk][tt] = v;
        }
        for (int e = tid; e < kCumChunk * kCumCol; e += kCumThreads) {
            const int kk = e / kCumCol, cc = e % kCumCol;
            float v = 0.f;
            if (k0 + kk < d_ff && col0 + cc < d_model)
                v = Elem<T>::to_float(Wd_t[(size_t)order[k0 + kk] * d_model + col0 + cc]);
            s_w[kk][cc] = v;
        }
        __syncthreads();
#pragma unroll 4
        for (int kk = 0; kk < kCumChunk; ++kk) {
            const float4 zv = *reinterpret_cast<const float4 *>(&s_z[kk][ty * 4]);
            const float4 wv = *reinterpret_cast<const float4 *>(&s_w[kk][tx * 4]);
            const float z4[4] = {zv.x, zv.y, zv.z, zv.w}, w4[4] = {wv.x, wv.y, wv.z, wv.w};
            float q = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    c[i][j] = fmaf(z4[i], w4[j], c[i][j]);
                    q = fmaf(c[i][j], c[i][j], q);
                }
            q = warp_sum(q);
            if (lane == 0) s_q[warp][kk] = q;
        }
        __syncthreads();
        if (tid < kCumChunk && k0 + tid < d_ff) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kCumThreads / kWarp; ++w) s += s_q[w][tid];
            partials[(size_t)tile * d_ff + k0 + tid] = s;
        }
        __syncthreads();
    }
}

// cum[b, 0] = 0, cum[b, k+1] = sum over the sample's tiles of partials[tile, k], in tile order, fp64.
__global__ void cett_reduce_kernel(const float *__restrict__ partials, int n_tiles, int d_ff,
                                   double *__restrict__ cum_b) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k == 0) cum_b[0] = 0.0;
    if (k >= d_ff) return;
    double s = 0.0;
    for (int t = 0; t < n_tiles; ++t) s += (double)partials[(size_t)t * d_ff + k];
    cum_b[k + 1] = s;
}

__device__ __forceinline__ float mean_cett_at(float eps, const float *__restrict__ sorted,
                                              const double *__restrict__ cum, int B, int d_ff) {
    double mean = 0.0;
    for (int x = 0; x < B; ++x) {
        const float *sx = sorted + (size_t)x * d_ff;
        int lo = 0, hi = d_ff;  // first index with sx[i] >= eps = number of scores below eps
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sx[mid] < eps) lo = mid + 1; else hi = mid;
        }
        const double dense = cum[(size_t)x * (d_ff + 1) + d_ff];
        if (dense > 0.0) mean += sqrt(cum[(size_t)x * (d_ff + 1) + lo] / dense);
    }
    return (float)(mean / B);
}

// best: bit pattern of the largest feasible candidate (non-negative floats order as unsigned integers).
__global__ void cett_search_kernel(const float *__restrict__ scores, const float *__restrict__ sorted,
                                   const double *__restrict__ cum, int B, int d_ff, float bound,
                                   unsigned *__restrict__ best) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * d_ff) return;
    const float eps = scores[i];
    if (!(eps >= 0.f)) return;
    if (mean_cett_at(eps, sorted, cum, B, d_ff) <= bound) atomicMax(best, __float_as_uint(eps));
}

__global__ void cett_result_kernel(const unsigned *__restrict__ best, const float *__restrict__ sorted,
                                   const double *__restrict__ cum, int B, int d_ff, float *__restrict__ tau_base,
                                   float *__restrict__ mean_cett) {
    if (threadIdx.x || blockIdx.x) return;
    const float tau = __uint_as_float(*best);
    *tau_base = tau;
    if (mean_cett) *mean_cett = mean_cett_at(tau, sorted, cum, B, d_ff);
}

// ---- workspace ------------------------------------------------------------------------------

struct CettLayout {
    size_t partials, zt, order, sorted, cum, tile_partials, best, total;
};

static size_t align256(size_t n) { return (n + 255) & ~(size_t)255; }

static CettLayout cett_layout(const clada_layer *L, const int64_t *off, int32_t B) {
    CettLayout lay;
    const long long T_total = off[B];
    long long max_tiles = 1;
    for (int b = 0; b < B; ++b) {
        const long long tt = (off[b + 1] - off[b] + kCumTok - 1) / kCumTok;
        max_tiles = std::max(max_tiles, tt * ((L->d_model + kCumCol - 1) / kCumCol));
    }
    size_t p = kWsCtrlBytes;
    lay.partials = p;      p += align256(prefix_partials_bytes_cuda_core(off, B, L->d_ff));
    lay.zt = p;            p += align256((size_t)L->d_ff * (size_t)std::max<long long>(T_total, 1) * sizeof(float));
    lay.order = p;         p += align256((size_t)B * L->d_ff * sizeof(int32_t));
    lay.sorted = p;        p += align256((size_t)B * L->d_ff * sizeof(float));
    lay.cum = p;           p += align256((size_t)B * (L->d_ff + 1) * sizeof(double));
    lay.tile_partials = p; p += align256((size_t)max_tiles * L->d_ff * sizeof(float));
    lay.best = p;          p += 256;
    lay.total = p;
    return lay;
}

static int check_offsets(const int64_t *off, int32_t B) {
    if (!off) return CLADA_ERR_NULL;
    if (B <= 0) return CLADA_ERR_SHAPE;
    if (B > kMaxSeqs) return CLADA_ERR_UNSUPPORTED;
    for (int b = 0; b <= B; ++b)
        if (off[b] < 0 || (b > 0 && off[b] < off[b - 1])) return CLADA_ERR_SHAPE;
    return CLADA_OK;
}

}  // namespace clada

using namespace clada;

extern "C" {

size_t clada_cett_workspace_bytes(const clada_layer *layer, const int64_t *seq_offsets, int32_t B) {
    if (!layer || layer->d_model <= 0 || layer->d_ff <= 0 || check_offsets(seq_offsets, B) != CLADA_OK) return 0;
    return cett_layout(layer, seq_offsets, B).total;
}

int clada_cett_threshold_search(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                                float bound, float *tau_base, float *mean_cett, float *scores, void *ws,
                                size_t ws_bytes, int32_t *status, void *stream) {
    CLADA_RANGE("clada_cett_threshold_search");
    (void)status;
    int rc = validate_layer(layer, true);
    if (rc != CLADA_OK) return rc;
    if (!X || !tau_base || !scores) return CLADA_ERR_NULL;
    if (!aligned16(X)) return CLADA_ERR_ALIGN;
    if ((rc = check_offsets(seq_offsets, B)) != CLADA_OK) return rc;
    if (!(bound >= 0.f)) return CLADA_ERR_SHAPE;
    if (layer->d_ff > kMaxSortN) return CLADA_ERR_UNSUPPORTED;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    const CettLayout lay = cett_layout(layer, seq_offsets, B);
    if (ws_bytes < lay.total) return CLADA_ERR_WORKSPACE;
    char *base = static_cast<char *>(ws);
    float *partials = reinterpret_cast<float *>(base + lay.partials);
    float *zt = reinterpret_cast<float *>(base + lay.zt);
    int32_t *order = reinterpret_cast<int32_t *>(base + lay.order);
    float *sorted = reinterpret_cast<float *>(base + lay.sorted);
    double *cum = reinterpret_cast<double *>(base + lay.cum);
    float *tile_partials = reinterpret_cast<float *>(base + lay.tile_partials);
    unsigned *best = reinterpret_cast<unsigned *>(base + lay.best);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int F = layer->d_ff, d = layer->d_model;
    const long long T_total = seq_offsets[B];

    // 1. scores and z
    rc = run_prefix_scores_with_z(layer, X, seq_offsets, B, scores, partials, zt, st);
    if (rc != CLADA_OK) return rc;
    // 2. neurons in ascending score order, per sample
    static bool configured[64] = {};
    DeviceInfo di;
    if ((rc = device_info(&di)) != CLADA_OK) return rc;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(cett_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kMaxSortN * (int)sizeof(unsigned long long)));
        configured[di.device & 63] = true;
    }
    int n_pow2 = 1;
    while (n_pow2 < F) n_pow2 <<= 1;
    cett_sort_kernel<<<B, kSortThreads, (size_t)n_pow2 * sizeof(unsigned long long), st>>>(scores, F, n_pow2, order,
                                                                                      sorted);
    CLADA_CUDA_TRY(cudaGetLastError());
    // 3 + 4. cumulative cut norms, sample by sample (the tile partials are reused)
    for (int b = 0; b < B; ++b) {
        const long long t0 = seq_offsets[b], t1 = seq_offsets[b + 1];
        double *cum_b = cum + (size_t)b * (F + 1);
        const int tok_tiles = (int)((t1 - t0 + kCumTok - 1) / kCumTok), col_tiles = (d + kCumCol - 1) / kCumCol;
        const int n_tiles = tok_tiles * col_tiles;
        if (n_tiles > 0) {
            dim3 grid(col_tiles, tok_tiles);
            if (layer->dtype == CLADA_F32)
                cett_cumulative_kernel<float><<<grid, kCumThreads, 0, st>>>(
                    zt, T_total, static_cast<const float *>(layer->w_down_t), d, F, order + (size_t)b * F, t0, t1,
                    tile_partials);
            else if (layer->dtype == CLADA_BF16)
                cett_cumulative_kernel<__nv_bfloat16><<<grid, kCumThreads, 0, st>>>(
                    zt, T_total, static_cast<const __nv_bfloat16 *>(layer->w_down_t), d, F, order + (size_t)b * F, t0,
                    t1, tile_partials);
            else
                cett_cumulative_kernel<__half><<<grid, kCumThreads, 0, st>>>(
                    zt, T_total, static_cast<const __half *>(layer->w_down_t), d, F, order + (size_t)b * F, t0, t1,
                    tile_partials);
            CLADA_CUDA_TRY(cudaGetLastError());
        }
        cett_reduce_kernel<<<(F + 255) / 256, 256, 0, st>>>(tile_partials, n_tiles, F, cum_b);
        CLADA_CUDA_TRY(cudaGetLastError());
    }
    // 5. the largest feasible candidate
    CLADA_CUDA_TRY(cudaMemsetAsync(best, 0, sizeof(unsigned), st));
    cett_search_kernel<<<(B * F + 255) / 256, 256, 0, st>>>(scores, sorted, cum, B, F, bound, best);
    CLADA_CUDA_TRY(cudaGetLastError());
    cett_result_kernel<<<1, 32, 0, st>>>(best, sorted, cum, B, F, tau_base, mean_cett);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

// The curve of one sample, for inspection and tests: cett[k] = CETT with the k lowest-scored neurons cut,
// k = 0 .. d_ff, read back from the workspace of the last clada_cett_threshold_search on the same arguments.
int clada_cett_curve(const clada_layer *layer, const int64_t *seq_offsets, int32_t B, int32_t sample,
                     const void *ws, size_t ws_bytes, double *cum_out, int32_t *order_out, void *stream) {
    CLADA_RANGE("clada_cett_curve");
    if (!layer || !ws || !cum_out) return CLADA_ERR_NULL;
    int rc = check_offsets(seq_offsets, B);
    if (rc != CLADA_OK) return rc;
    if (sample < 0 || sample >= B) return CLADA_ERR_SHAPE;
    const CettLayout lay = cett_layout(layer, seq_offsets, B);
    if (ws_bytes < lay.total) return CLADA_ERR_WORKSPACE;
    const char *base = static_cast<const char *>(ws);
    const int F = layer->d_ff;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CLADA_CUDA_TRY(cudaMemcpyAsync(cum_out, base + lay.cum + (size_t)sample * (F + 1) * sizeof(double),
                                   (size_t)(F + 1) * sizeof(double), cudaMemcpyDeviceToDevice, st));
    if (order_out)
        CLADA_CUDA_TRY(cudaMemcpyAsync(order_out, base + lay.order + (size_t)sample * F * sizeof(int32_t),
                                       (size_t)F * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return CLADA_OK;
}

}  // extern "C"
