// Prefill statistics (Eq. neuron_activation) on CUDA cores, fp32 accumulation, any dtype:
//   z[t,j] = silu(x_t . w_gate_j) * (x_t . w_up_j),   A[b,j] = sqrt(sum_{t in b} z[t,j]^2) * ||W_out,j||
// plus the fp64 guard-band refinement and the one-call prefill entry point.
//
// The GEMM never writes z: each CTA owns a (token tile, neuron tile) pair that lies inside one
// prompt, keeps both accumulators (gate and up) in registers, and its epilogue squares and sums
// over the tile's tokens into one fp32 partial per neuron.  A second kernel adds a prompt's
// partials in tile order, so scores are bit-identical run to run.
#include <math.h>

#include "common.cuh"
#include "nvtx_ranges.cuh"
#include "prefix_common.cuh"

namespace clada {

constexpr int BM = 64, BN = 64, BK = 32, kPfThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kPfThreads)
prefix_partials_kernel(const T *__restrict__ X, const T *__restrict__ Wg, const T *__restrict__ Wu,
                       int d_model, int d_ff, const SeqTable tab, float *__restrict__ partials,
                       float *__restrict__ zt, long long zt_stride, int act) {
    constexpr int E = Elem<T>::kPerVec;
    __shared__ __align__(16) float Xs[BK][BM + 4];
    __shared__ __align__(16) float Gs[BK][BN + 4];
    __shared__ __align__(16) float Us[BK][BN + 4];
    __shared__ float s_red[16][BN + 1];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;  // 16 x 16 threads, 4 x 4 outputs each
    const int n0 = blockIdx.x * BN;
    int b;
    long long t0, t1;
    locate_tile(tab, blockIdx.y, BM, b, t0, t1);

    float ag[4][4], au[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) ag[i][j] = au[i][j] = 0.f;

    constexpr int kVecPerRow = BK / E;            // 16-byte vectors per tile row
    constexpr int kVecPerTile = BM * kVecPerRow;  // BM == BN
    for (int k0 = 0; k0 < d_model; k0 += BK) {
        for (int v = tid; v < kVecPerTile; v += kPfThreads) {
            const int r = v / kVecPerRow, c = (v % kVecPerRow) * E;
            const bool kin = k0 + c < d_model;  // d_model % 8 == 0, so a vector is all in or all out
            float fx[E], fg[E], fu[E];
            uint4 qx = make_uint4(0, 0, 0, 0), qg = qx, qu = qx;
            if (kin && t0 + r < t1) qx = *reinterpret_cast<const uint4 *>(X + (size_t)(t0 + r) * d_model + k0 + c);
            if (kin && n0 + r < d_ff) {
                qg = *reinterpret_cast<const uint4 *>(Wg + (size_t)(n0 + r) * d_model + k0 + c);
                if (Wu) qu = *reinterpret_cast<const uint4 *>(Wu + (size_t)(n0 + r) * d_model + k0 + c);  // null: no gate projection
            }
            Elem<T>::unpack(qx, fx);
            Elem<T>::unpack(qg, fg);
            Elem<T>::unpack(qu, fu);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                Xs[c + e][r] = fx[e];
                Gs[c + e][r] = fg[e];
                Us[c + e][r] = fu[e];
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a = *reinterpret_cast<const float4 *>(&Xs[k][ty * 4]);
            const float4 g = *reinterpret_cast<const float4 *>(&Gs[k][tx * 4]);
            const float4 u = *reinterpret_cast<const float4 *>(&Us[k][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w};
            const float gv[4] = {g.x, g.y, g.z, g.w};
            const float uv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    ag[i][j] = fmaf(av[i], gv[j], ag[i][j]);
                    au[i][j] = fmaf(av[i], uv[j], au[i][j]);
                }
        }
        __syncthreads();
    }
    // epilogue: z^2 summed over this thread's 4 tokens, then over the 16 thread rows in order
    // (the offline threshold search also wants z itself, neuron-major: zt[j, t])
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float z = neuron_value_f(act, ag[i][j], au[i][j]);  // padded token rows give exactly 0
            s = fmaf(z, z, s);
            const long long t = t0 + ty * 4 + i;
            if (zt && t < t1 && n0 + tx * 4 + j < d_ff) zt[(size_t)(n0 + tx * 4 + j) * zt_stride + t] = z;
        }
        s_red[ty][tx * 4 + j] = s;
    }
    __syncthreads();
    if (tid < BN && n0 + tid < d_ff) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < 16; ++r) s += s_red[r][tid];
        partials[(size_t)blockIdx.y * d_ff + n0 + tid] = s;
    }
}

__global__ void prefix_finalize_kernel(const float *__restrict__ partials, const SeqTable tab, int tile, int d_ff,
                                       const float *__restrict__ w_down_norm, float *__restrict__ scores) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = blockIdx.y;
    if (j >= d_ff) return;
    int first = 0;
    for (int q = 0; q < b; ++q) first += tiles_of(tab.off[q + 1] - tab.off[q], tile);
    const int n = tiles_of(tab.off[b + 1] - tab.off[b], tile);
    float s = 0.f;
    for (int t = 0; t < n; ++t) s += partials[(size_t)(first + t) * d_ff + j];
    scores[(size_t)b * d_ff + j] = __fmul_rn(sqrtf(s), w_down_norm[j]);
}

// Chunked prefill: the same tile sums added into a running sum of squares per (prompt, neuron) ...
__global__ void prefix_accumulate_kernel(const float *__restrict__ partials, const SeqTable tab, int tile, int d_ff,
                                         float *__restrict__ sumsq) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = blockIdx.y;
    if (j >= d_ff) return;
    int first = 0;
    for (int q = 0; q < b; ++q) first += tiles_of(tab.off[q + 1] - tab.off[q], tile);
    const int n = tiles_of(tab.off[b + 1] - tab.off[b], tile);
    float s = sumsq[(size_t)b * d_ff + j];
    for (int t = 0; t < n; ++t) s += partials[(size_t)(first + t) * d_ff + j];
    sumsq[(size_t)b * d_ff + j] = s;
}

// ... and, after the last chunk, the scores from it.
__global__ void prefix_finish_kernel(const float *__restrict__ sumsq, int B, int d_ff,
                                     const float *__restrict__ w_down_norm, float *__restrict__ scores) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)B * d_ff) return;
    scores[i] = __fmul_rn(sqrtf(sumsq[i]), w_down_norm[i % d_ff]);
}

// ---- guard band -----------------------------------------------------------------------------

struct GuardMults {
    int n;
    float m[8];
};

__global__ void guard_candidates_kernel(const float *__restrict__ scores, int B, int d_ff,
                                        const float *__restrict__ tau_base, const GuardMults gm,
                                        float rel_band, int *__restrict__ n_cand, int2 *__restrict__ cand) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * d_ff) return;
    const int b = i / d_ff, j = i % d_ff;
    const float a = scores[i];
    bool near = false;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < gm.n) {
            const float thr = tau_base[b] * gm.m[g];
            near |= fabsf(a - thr) <= rel_band * fabsf(thr);
        }
    }
    if (near) cand[atomicAdd(n_cand, 1)] = make_int2(b, j);
}

constexpr int kRefThreads = 1024;

// A 16-byte vector widened to fp64 (exact).  For bf16 the double is assembled from the bit fields with
// integer operations: converting through the float-to-double instruction runs at a sixteenth of the ALU
// rate and was the guard band's bottleneck.  Zeros, denormals, inf and NaN take the conversion.
template <typename T> struct Widen;
template <> struct Widen<float> {
    __device__ static __forceinline__ void run(const uint4 &v, double (&o)[4]) {
        o[0] = (double)__uint_as_float(v.x); o[1] = (double)__uint_as_float(v.y);
        o[2] = (double)__uint_as_float(v.z); o[3] = (double)__uint_as_float(v.w);
    }
};
__device__ __forceinline__ double bf16_bits_to_double(uint32_t b) {  // b: 16 significant bits
    const uint32_t ex = (b >> 7) & 0xffu;
    if (ex == 0u || ex == 255u) return (double)__uint_as_float(b << 16);
    const uint32_t hi = ((b & 0x8000u) << 16) | ((ex + 896u) << 20) | ((b & 0x7fu) << 13);
    return __hiloint2double((int)hi, 0);
}
// IEEE half: 1 sign, 5 exponent (bias 15), 10 fraction bits -> double (bias 1023, fraction at bit 42 of 52).
__device__ __forceinline__ double f16_bits_to_double(uint32_t b) {  // b: 16 significant bits
    const uint32_t ex = (b >> 10) & 0x1fu;
    if (ex == 0u || ex == 31u) return (double)__half2float(__ushort_as_half((unsigned short)b));
    const uint32_t hi = ((b & 0x8000u) << 16) | ((ex + 1008u) << 20) | ((b & 0x3ffu) << 10);
    return __hiloint2double((int)hi, 0);
}
template <> struct Widen<__half> {
    __device__ static __forceinline__ void run(const uint4 &v, double (&o)[8]) {
        o[0] = f16_bits_to_double(v.x & 0xffffu); o[1] = f16_bits_to_double(v.x >> 16);
        o[2] = f16_bits_to_double(v.y & 0xffffu); o[3] = f16_bits_to_double(v.y >> 16);
        o[4] = f16_bits_to_double(v.z & 0xffffu); o[5] = f16_bits_to_double(v.z >> 16);
        o[6] = f16_bits_to_double(v.w & 0xffffu); o[7] = f16_bits_to_double(v.w >> 16);
    }
};
template <> struct Widen<__nv_bfloat16> {
    __device__ static __forceinline__ void run(const uint4 &v, double (&o)[8]) {
        o[0] = bf16_bits_to_double(v.x & 0xffffu); o[1] = bf16_bits_to_double(v.x >> 16);
        o[2] = bf16_bits_to_double(v.y & 0xffffu); o[3] = bf16_bits_to_double(v.y >> 16);
        o[4] = bf16_bits_to_double(v.z & 0xffffu); o[5] = bf16_bits_to_double(v.z >> 16);
        o[6] = bf16_bits_to_double(v.w & 0xffffu); o[7] = bf16_bits_to_double(v.w >> 16);
    }
};

// How many CTAs share one candidate's prompt: with fewer candidates than CTAs, each candidate's tokens are
// dealt to several CTAs (the partial sums meet in guard_finish_kernel), so the whole GPU works on the band.
constexpr int kRefMaxUnits = 512;  // (candidate, split) partial sums held in the workspace
__host__ __device__ inline int guard_splits(int total, int n_ctas) {
    if (total <= 0 || total >= n_ctas) return 1;
    int s = n_ctas / total;
    if (s > 32) s = 32;
    while (s > 1 && total * s > kRefMaxUnits) --s;
    return s;
}

// One CTA per (candidate, split) (grid-stride).  The candidate's gate and up rows are widened to fp64 once
// into shared memory; each of the 32 warps takes every (32 * splits)-th token of the prompt, lanes split
// d_model by 16-byte vectors, products and sums in fp64.  Warp and CTA sums are taken in a fixed order.
template <typename T>
__global__ void __launch_bounds__(kRefThreads)
guard_refine_kernel(const T *__restrict__ X, const T *__restrict__ Wg, const T *__restrict__ Wu,
                    const T *__restrict__ Wd_t, int d_model, int d_ff, const SeqTable tab,
                    const int *__restrict__ n_cand, const int2 *__restrict__ cand,
                    float *__restrict__ scores, int act, double2 *__restrict__ part) {
    constexpr int E = Elem<T>::kPerVec;
    constexpr int kWarps = kRefThreads / kWarp;
    extern __shared__ __align__(16) double s_rows[];  // gate row | up row, fp64
    __shared__ double s_zz[kWarps];
    __shared__ double s_nn[kWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int vpr = d_model / E;
    const int total = *n_cand;
    const int S = guard_splits(total, (int)gridDim.x);
    for (int unit = blockIdx.x; unit < total * S; unit += gridDim.x) {
        const int c = unit / S, split = unit % S;
        const int b = cand[c].x, j = cand[c].y;
        const uint4 *wg = reinterpret_cast<const uint4 *>(Wg + (size_t)j * d_model);
        const uint4 *wu = reinterpret_cast<const uint4 *>(Wu + (size_t)j * d_model);
        const uint4 *wd = reinterpret_cast<const uint4 *>(Wd_t + (size_t)j * d_model);
        for (int v = threadIdx.x; v < vpr; v += kRefThreads) {
            double g[E], u[E];
            Widen<T>::run(wg[v], g);
            if (Wu) {
                Widen<T>::run(wu[v], u);
            } else {  // no gate projection: the u factor is not used
#pragma unroll
                for (int e = 0; e < E; ++e) u[e] = 0.0;
            }
#pragma unroll
            for (int e = 0; e < E; ++e) {  // element-major: lanes then read consecutive doubles
                s_rows[e * vpr + v] = g[e];
                s_rows[d_model + e * vpr + v] = u[e];
            }
        }
        __syncthreads();
        double zz = 0.0;
        for (long long t = tab.off[b] + warp + (long long)kWarps * split; t < tab.off[b + 1]; t += (long long)kWarps * S) {
            const uint4 *x = reinterpret_cast<const uint4 *>(X + (size_t)t * d_model);
            double g = 0.0, u = 0.0;
#pragma unroll 4
            for (int v = lane; v < vpr; v += kWarp) {  // four independent 16-byte loads in flight
                double fx[E];
                Widen<T>::run(x[v], fx);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    g = fma(s_rows[e * vpr + v], fx[e], g);
                    u = fma(s_rows[d_model + e * vpr + v], fx[e], u);
                }
            }
            g = warp_sum(g);
            u = warp_sum(u);
            const double z = neuron_value_d(act, g, u);
            zz += z * z;
        }
        double nn = 0.0;
        for (int v = threadIdx.x; v < vpr; v += kRefThreads) {
            double fd[E];
            Widen<T>::run(wd[v], fd);
#pragma unroll
            for (int e = 0; e < E; ++e) nn = fma(fd[e], fd[e], nn);
        }
        nn = warp_sum(nn);
        if (lane == 0) {
            s_zz[warp] = zz;
            s_nn[warp] = nn;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            double a = 0.0, n2 = 0.0;
            for (int w = 0; w < kWarps; ++w) {
                a += s_zz[w];
                n2 += s_nn[w];
            }
            if (S == 1)
                scores[(size_t)b * d_ff + j] = (float)(sqrt(a) * sqrt(n2));
            else
                part[unit] = make_double2(a, n2);  // this split's share of the sum over tokens
        }
        __syncthreads();
    }
}

// The splits of a candidate added in split order (only launched work when candidates were split).
__global__ void guard_finish_kernel(const int *__restrict__ n_cand, const int2 *__restrict__ cand, int n_ctas, int d_ff,
                                    const double2 *__restrict__ part, float *__restrict__ scores) {
    const int total = *n_cand;
    const int S = guard_splits(total, n_ctas);
    if (S == 1) return;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < total; c += gridDim.x * blockDim.x) {
        double a = 0.0;
        for (int s = 0; s < S; ++s) a += part[c * S + s].x;
        scores[(size_t)cand[c].x * d_ff + cand[c].y] = (float)(sqrt(a) * sqrt(part[c * S].y));
    }
}

// ---- host side ------------------------------------------------------------------------------

static int build_table(const int64_t *seq_offsets, int32_t B, SeqTable *tab, int *n_mtiles) {
    if (!seq_offsets) return CLADA_ERR_NULL;
    if (B <= 0) return CLADA_ERR_SHAPE;
    if (B > kMaxSeqs) return CLADA_ERR_UNSUPPORTED;
    tab->B = B;
    long long tiles = 0;
    for (int b = 0; b <= B; ++b) {
        tab->off[b] = seq_offsets[b];
        if (seq_offsets[b] < 0 || (b > 0 && seq_offsets[b] < seq_offsets[b - 1])) return CLADA_ERR_SHAPE;
        if (b > 0) tiles += tiles_of(seq_offsets[b] - seq_offsets[b - 1], BM);
    }
    if (tiles > 65535) return CLADA_ERR_UNSUPPORTED;
    *n_mtiles = (int)tiles;
    return CLADA_OK;
}

static size_t partials_bytes(int n_mtiles, int d_ff) {
    return (((size_t)n_mtiles * d_ff * sizeof(float)) + 255) & ~(size_t)255;
}

template <typename T>
static int run_scores(const clada_layer *L, const void *X, const SeqTable &tab, int n_mtiles, float *scores,
                      float *partials, cudaStream_t st, float *zt = nullptr, long long zt_stride = 0) {
    if (n_mtiles > 0) {
        dim3 grid((L->d_ff + BN - 1) / BN, n_mtiles);
        prefix_partials_kernel<T><<<grid, kPfThreads, 0, st>>>(
            static_cast<const T *>(X), static_cast<const T *>(L->w_gate), static_cast<const T *>(L->w_up),
            L->d_model, L->d_ff, tab, partials, zt, zt_stride, L->activation);
        CLADA_CUDA_TRY(cudaGetLastError());
    }
    return launch_prefix_finalize(partials, tab, BM, L->d_ff, L->w_down_norm, scores, st);
}

int run_prefix_scores_with_z(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                             float *scores, float *partials, float *zt, cudaStream_t st) {
    SeqTable tab;
    int n_mtiles = 0;
    int rc = build_table(seq_offsets, B, &tab, &n_mtiles);
    if (rc != CLADA_OK) return rc;
    if (layer->dtype == CLADA_F32)
        return run_scores<float>(layer, X, tab, n_mtiles, scores, partials, st, zt, seq_offsets[B]);
    if (layer->dtype == CLADA_BF16)
        return run_scores<__nv_bfloat16>(layer, X, tab, n_mtiles, scores, partials, st, zt, seq_offsets[B]);
    return run_scores<__half>(layer, X, tab, n_mtiles, scores, partials, st, zt, seq_offsets[B]);
}

size_t prefix_partials_bytes_cuda_core(const int64_t *seq_offsets, int32_t B, int d_ff) {
    long long tiles = 0;
    for (int b = 0; b < B; ++b) tiles += tiles_of(seq_offsets[b + 1] - seq_offsets[b], BM);
    return partials_bytes((int)tiles, d_ff);
}

int launch_prefix_finalize(const float *partials, const SeqTable &tab, int tile, int d_ff,
                           const float *w_down_norm, float *scores, cudaStream_t st) {
    dim3 fgrid((d_ff + 255) / 256, tab.B);
    prefix_finalize_kernel<<<fgrid, 256, 0, st>>>(partials, tab, tile, d_ff, w_down_norm, scores);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

}  // namespace clada

using namespace clada;

extern "C" {

int clada_prefix_scores(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                        float *scores, void *ws, size_t ws_bytes, int32_t *status, void *stream) {
    CLADA_RANGE("clada_prefix_scores");
    (void)status;
    int rc = validate_layer(layer, true);
    if (rc != CLADA_OK) return rc;
    if (!X || !scores) return CLADA_ERR_NULL;
    if (!aligned16(X)) return CLADA_ERR_ALIGN;
    SeqTable tab;
    int n_mtiles = 0;
    rc = build_table(seq_offsets, B, &tab, &n_mtiles);
    if (rc != CLADA_OK) return rc;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    if (ws_bytes < kWsCtrlBytes + partials_bytes(n_mtiles, layer->d_ff)) return CLADA_ERR_WORKSPACE;
    float *partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (layer->dtype == CLADA_F32) return run_scores<float>(layer, X, tab, n_mtiles, scores, partials, st);
    // bf16 / fp16: tensor cores (128-token tiles: never more partial rows than the 64-token tiling above)
    rc = run_prefix_partials_tc(layer, X, tab, seq_offsets[B], partials, status, st);
    if (rc != CLADA_OK) return rc;
    return launch_prefix_finalize(partials, tab, kTcTokenTile, layer->d_ff, layer->w_down_norm, scores, st);
}

int clada_prefix_accumulate(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                            float *sumsq, void *Z, void *ws, size_t ws_bytes, int32_t *status, void *stream) {
    CLADA_RANGE("clada_prefix_accumulate");
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!X || !sumsq) return CLADA_ERR_NULL;
    if (!aligned16(X) || (Z && !aligned16(Z))) return CLADA_ERR_ALIGN;
    if (Z && layer->dtype == CLADA_F32) return CLADA_ERR_UNSUPPORTED;  // hidden activations: tensor-core route only
    if (Z && layer->d_ff % 8 != 0) return CLADA_ERR_SHAPE;  // rows of Z are written as 16-byte vectors
    SeqTable tab;
    int n_mtiles = 0;
    rc = build_table(seq_offsets, B, &tab, &n_mtiles);
    if (rc != CLADA_OK) return rc;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    if (ws_bytes < kWsCtrlBytes + partials_bytes(n_mtiles, layer->d_ff)) return CLADA_ERR_WORKSPACE;
    float *partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int tile = BM;
    if (layer->dtype == CLADA_F32) {
        if (n_mtiles > 0) {
            dim3 grid((layer->d_ff + BN - 1) / BN, n_mtiles);
            prefix_partials_kernel<float><<<grid, kPfThreads, 0, st>>>(
                static_cast<const float *>(X), static_cast<const float *>(layer->w_gate),
                static_cast<const float *>(layer->w_up), layer->d_model, layer->d_ff, tab, partials, nullptr, 0,
                layer->activation);
            CLADA_CUDA_TRY(cudaGetLastError());
        }
    } else {
        rc = run_prefix_partials_tc(layer, X, tab, seq_offsets[B], partials, status, st, Z);
        if (rc != CLADA_OK) return rc;
        tile = kTcTokenTile;
    }
    dim3 agrid((layer->d_ff + 255) / 256, tab.B);
    prefix_accumulate_kernel<<<agrid, 256, 0, st>>>(partials, tab, tile, layer->d_ff, sumsq);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

int clada_prefix_finish(const clada_layer *layer, const float *sumsq, int32_t B, float *scores, void *stream) {
    CLADA_RANGE("clada_prefix_finish");
    int rc = validate_layer(layer, true);
    if (rc != CLADA_OK) return rc;
    if (!sumsq || !scores) return CLADA_ERR_NULL;
    if (B <= 0) return CLADA_ERR_SHAPE;
    const size_t n = (size_t)B * layer->d_ff;
    prefix_finish_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        sumsq, B, layer->d_ff, layer->w_down_norm, scores);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

int clada_prefill_down(const clada_layer *layer, const void *w_down, const void *Z, int64_t T, void *Y,
                       int32_t y_dtype, void *ws, size_t ws_bytes, int32_t *status, void *stream) {
    CLADA_RANGE("clada_prefill_down");
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!w_down || !Z || !Y) return CLADA_ERR_NULL;
    if (T < 0) return CLADA_ERR_SHAPE;
    if (layer->dtype == CLADA_F32) return CLADA_ERR_UNSUPPORTED;  // tensor-core route: bf16 / fp16 layers
    if (!dtype_ok(y_dtype)) return CLADA_ERR_DTYPE;
    if (layer->d_ff % 8 != 0) return CLADA_ERR_SHAPE;  // rows of Z and of w_down must be 16-byte multiples
    if (!aligned16(w_down) || !aligned16(Z) || !aligned16(Y)) return CLADA_ERR_ALIGN;
    if (ws && ((reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < kWsCtrlBytes)) return CLADA_ERR_WORKSPACE;
    // the scratch behind the workspace's control block (which this call leaves alone) holds split partial outputs
    void *scratch = ws ? static_cast<char *>(ws) + kWsCtrlBytes : nullptr;
    return run_down_tc(layer, w_down, Z, T, Y, y_dtype, scratch, ws ? ws_bytes - kWsCtrlBytes : 0, status,
                       static_cast<cudaStream_t>(stream));
}

int clada_refine_scores(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                        const float *tau_base, const float *guard_mults, int32_t n_guard, float rel_band,
                        float *scores, void *ws, size_t ws_bytes, int32_t *status, void *stream) {
    CLADA_RANGE("clada_refine_scores");
    (void)status;
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!X || !scores || !tau_base || !guard_mults) return CLADA_ERR_NULL;
    if (n_guard <= 0 || n_guard > 8 || !(rel_band >= 0.f)) return CLADA_ERR_SHAPE;
    if (!aligned16(X)) return CLADA_ERR_ALIGN;
    SeqTable tab;
    int n_mtiles = 0;
    rc = build_table(seq_offsets, B, &tab, &n_mtiles);
    if (rc != CLADA_OK) return rc;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    // candidate counter, split partial sums and candidate list live behind the partials region of clada_prefix_scores
    const size_t off = kWsCtrlBytes + partials_bytes(n_mtiles, layer->d_ff);
    const size_t part_bytes = kRefMaxUnits * sizeof(double2);
    const size_t need = off + 256 + part_bytes + (size_t)B * layer->d_ff * sizeof(int2);
    if (ws_bytes < need) return CLADA_ERR_WORKSPACE;
    int *n_cand = reinterpret_cast<int *>(static_cast<char *>(ws) + off);
    double2 *part = reinterpret_cast<double2 *>(static_cast<char *>(ws) + off + 256);
    int2 *cand = reinterpret_cast<int2 *>(static_cast<char *>(ws) + off + 256 + part_bytes);
    GuardMults gm;
    gm.n = n_guard;
    for (int g = 0; g < 8; ++g) gm.m[g] = g < n_guard ? guard_mults[g] : 0.f;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CLADA_CUDA_TRY(cudaMemsetAsync(n_cand, 0, sizeof(int), st));
    const int n = B * layer->d_ff;
    guard_candidates_kernel<<<(n + 255) / 256, 256, 0, st>>>(scores, B, layer->d_ff, tau_base, gm, rel_band,
                                                             n_cand, cand);
    CLADA_CUDA_TRY(cudaGetLastError());
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    const int grid = di.num_sms;
    const size_t rows_smem = 2 * (size_t)layer->d_model * sizeof(double);
    static bool configured[64] = {};
    if (!configured[di.device & 63]) {  // up to 128 KB of dynamic shared memory
        CLADA_CUDA_TRY(cudaFuncSetAttribute(guard_refine_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            2 * kMaxDModel * (int)sizeof(double)));
        CLADA_CUDA_TRY(cudaFuncSetAttribute(guard_refine_kernel<__nv_bfloat16>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            2 * kMaxDModel * (int)sizeof(double)));
        CLADA_CUDA_TRY(cudaFuncSetAttribute(guard_refine_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            2 * kMaxDModel * (int)sizeof(double)));
        configured[di.device & 63] = true;
    }
    if (layer->dtype == CLADA_F32)
        guard_refine_kernel<float><<<grid, kRefThreads, rows_smem, st>>>(
            static_cast<const float *>(X), static_cast<const float *>(layer->w_gate),
            static_cast<const float *>(layer->w_up), static_cast<const float *>(layer->w_down_t),
            layer->d_model, layer->d_ff, tab, n_cand, cand, scores, layer->activation, part);
    else if (layer->dtype == CLADA_BF16)
        guard_refine_kernel<__nv_bfloat16><<<grid, kRefThreads, rows_smem, st>>>(
            static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(layer->w_gate),
            static_cast<const __nv_bfloat16 *>(layer->w_up), static_cast<const __nv_bfloat16 *>(layer->w_down_t),
            layer->d_model, layer->d_ff, tab, n_cand, cand, scores, layer->activation, part);
    else
        guard_refine_kernel<__half><<<grid, kRefThreads, rows_smem, st>>>(
            static_cast<const __half *>(X), static_cast<const __half *>(layer->w_gate),
            static_cast<const __half *>(layer->w_up), static_cast<const __half *>(layer->w_down_t),
            layer->d_model, layer->d_ff, tab, n_cand, cand, scores, layer->activation, part);
    CLADA_CUDA_TRY(cudaGetLastError());
    guard_finish_kernel<<<2, 256, 0, st>>>(n_cand, cand, grid, layer->d_ff, part, scores);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

int clada_prefix_select(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                        const float *tau_base, const float *guard_mults, int32_t n_guard, float *scores,
                        uint8_t *mask, int32_t *idx, int32_t *count, void *ws, size_t ws_bytes,
                        int32_t *status, void *stream) {
    CLADA_RANGE("clada_prefix_select");
    int rc = clada_prefix_scores(layer, X, seq_offsets, B, scores, ws, ws_bytes, status, stream);
    if (rc != CLADA_OK || !tau_base) return rc;
    if (n_guard > 0 && guard_mults) {
        rc = clada_refine_scores(layer, X, seq_offsets, B, tau_base, guard_mults, n_guard, 1e-4f, scores, ws,
                                 ws_bytes, status, stream);
        if (rc != CLADA_OK) return rc;
    }
    return clada_select(scores, B, layer->d_ff, tau_base, 1, mask, idx, count, stream);
}

}  // extern "C"
