// Per-token cognitive load (Eqs. surprisal, entropy) and the token-aware threshold
// (Eq. final_threshold).
//
// A cluster of CTAs per vocabulary row.  Each thread streams 16-byte vectors of logits and keeps a running
// (max m, Z = sum e^{l-m}, W = sum e^{l-m}(l-m)).  At each level (CTA, then cluster) the maximum is reduced
// first, every statistic is moved to it once, and Z and W are summed, always in the same order.  With
// logZ = log Z:
//   surprisal = m + logZ - l[token],   entropy = logZ - W / Z.
#include <math.h>

#include <cooperative_groups.h>

#include "common.cuh"
#include "nvtx_ranges.cuh"

namespace cg = cooperative_groups;

namespace clada {

struct SoftStat {
    float m, z, w;
};

__device__ __forceinline__ SoftStat stat_empty() { return SoftStat{-INFINITY, 0.f, 0.f}; }

// Move a statistic to a new (not smaller) reference maximum.
__device__ __forceinline__ void stat_rebase(SoftStat &a, float m_new) {
    if (a.m == -INFINITY) {
        a.m = m_new;  // nothing accumulated yet
        return;
    }
    const float dm = a.m - m_new;  // <= 0
    const float sc = expf(dm);
    a.w = (a.w + dm * a.z) * sc;
    a.z = a.z * sc;
    a.m = m_new;
}

template <int N>
__device__ __forceinline__ void stat_add(SoftStat &a, const float (&l)[N], bool &bad) {
    float cm = -INFINITY;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        bad |= !(l[i] < INFINITY);  // +inf or NaN
        cm = fmaxf(cm, l[i]);
    }
    if (cm == -INFINITY) return;  // the whole chunk has probability zero
    if (cm > a.m) stat_rebase(a, cm);
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const float t = l[i] - a.m;
        const float e = expf(t);
        a.z += e;
        a.w += (t == -INFINITY) ? 0.f : e * t;
    }
}

template <typename T>
__device__ __forceinline__ float load_logit(const T *row, int64_t i) {
    return Elem<T>::to_float(row[i]);
}

constexpr int kCogThreads = 512;
constexpr int kCogMaxCluster = 8;

// Grid (cluster size, B): the CTAs of a cluster split one vocabulary row into equal slices, leave their
// slice statistics in shared memory, and rank 0 reads them over distributed shared memory, merges them
// in rank order and writes the row's outputs.  tau_base == nullptr: cognitive load only.
template <typename T>
__global__ void __launch_bounds__(kCogThreads)
cogload_kernel(const T *__restrict__ logits, int64_t V, int64_t row_stride,
               const int32_t *__restrict__ token_id, float *__restrict__ surprisal,
               float *__restrict__ entropy, int32_t *__restrict__ status,
               const float *__restrict__ tau_base, const float *__restrict__ lambda,
               const float *__restrict__ gamma, float tau_s, float tau_H, int L,
               float *__restrict__ tau_final, int32_t *__restrict__ level_out) {
    constexpr int E = Elem<T>::kPerVec;
    cg::cluster_group cluster = cg::this_cluster();
    const int n_slices = (int)cluster.num_blocks(), slice = (int)cluster.block_rank();
    const int b = blockIdx.y;
    const T *row = logits + (size_t)b * row_stride;
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    // First cluster phase: "every CTA of the cluster has started", which a write into another CTA's shared
    // memory needs.  Arrive now, wait only just before that write: by then the phase has long completed.
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    pdl_wait();

    SoftStat st = stat_empty();
    bool bad = false;

    // Loads that only the last steps need are issued first, so that their latency hides under the row's:
    // the chosen token and its logit (two dependent loads), and the first adjustment operands per thread.
    int32_t tok = 0;
    bool tok_ok = false;
    float tok_logit = 0.f;
    float adj_base = 0.f, adj_lambda = 0.f, adj_gamma = 0.f;
    if (slice == 0) {
        if (tid == 0) {
            tok = token_id[b];
            tok_ok = tok >= 0 && tok < V;
            if (tok_ok) tok_logit = load_logit(row, tok);
        }
        if (tau_base != nullptr && tid < L) {
            adj_base = tau_base[(size_t)b * L + tid];
            adj_lambda = lambda[tid];
            adj_gamma = gamma[tid];
        }
    }

    // The row as scalar head (up to the first 16-byte boundary), 16-byte vectors, scalar tail; the
    // vectors are dealt to the slices in contiguous runs, head and tail go to slice 0.
    const uintptr_t addr = reinterpret_cast<uintptr_t>(row);
    int64_t head = ((16 - (addr & 15)) & 15) / sizeof(T);
    if (head > V) head = V;
    const int64_t nvec = (V - head) / E;
    const int64_t tail0 = head + nvec * E;
    if (slice == 0 && tid < head) {
        float l[1] = {load_logit(row, tid)};
        stat_add(st, l, bad);
    }
    const uint4 *vrow = reinterpret_cast<const uint4 *>(row + head);
    const int64_t v0 = nvec * slice / n_slices, v1 = nvec * (slice + 1) / n_slices;
    // eight vectors in flight per thread
    for (int64_t v = v0 + tid; v < v1; v += 8 * (int64_t)kCogThreads) {
        uint4 q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t vi = v + u * (int64_t)kCogThreads;
            q[u] = make_uint4(0, 0, 0, 0);
            if (vi < v1) q[u] = ldg_stream(vrow + vi);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (v + u * (int64_t)kCogThreads < v1) {
                float l[E];
                Elem<T>::unpack(q[u], l);
                stat_add(st, l, bad);
            }
        }
    }
    if (slice == 0 && tail0 + tid < V) {
        float l[1] = {load_logit(row, tail0 + tid)};
        stat_add(st, l, bad);
    }

    // CTA reduction, in a fixed order.  Merging statistics pairwise costs two exponentials per merge on a
    // serial chain (13 levels from thread to row); instead the maximum is reduced first (compares only),
    // every thread moves its statistic to it once, and Z and W are then plain sums.
    __shared__ float s_max[kCogThreads / kWarp];
    __shared__ float2 s_zw[kCogThreads / kWarp];
    __shared__ SoftStat s_all[kCogMaxCluster];  // on rank 0: every slice's statistic, written by its owner
    __shared__ int s_bad;
    __shared__ float s_out[2];
    float wm = st.m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
    if (tid == 0) s_bad = 0;
    if ((tid & 31) == 0) s_max[tid >> 5] = wm;
    __syncthreads();
    if (bad) atomicOr(&s_bad, 1);
    float cm = s_max[0];
#pragma unroll
    for (int w = 1; w < kCogThreads / kWarp; ++w) cm = fmaxf(cm, s_max[w]);
    float z = 0.f, wsum = 0.f;
    if (st.z > 0.f) {  // (a thread without finite logits adds nothing; cm is finite here)
        const float dm = st.m - cm;  // <= 0
        const float sc = expf(dm);
        z = st.z * sc;
        wsum = (st.w + dm * st.z) * sc;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        z += __shfl_xor_sync(0xffffffffu, z, o);
        wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
    }
    if ((tid & 31) == 0) s_zw[tid >> 5] = make_float2(z, wsum);
    __syncthreads();
    if (tid < kWarp) {  // warp 0 adds the 16 warp sums by butterfly (same bits on every lane)
        float2 v = tid < kCogThreads / kWarp ? s_zw[tid] : make_float2(0.f, 0.f);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            v.x += __shfl_xor_sync(0xffffffffu, v.x, o);
            v.y += __shfl_xor_sync(0xffffffffu, v.y, o);
        }
        SoftStat tot = SoftStat{cm, v.x, v.y};
        if (s_bad) tot.z = NAN;  // carries the non-finite flag to rank 0
        // every CTA started (first phase) before anyone writes into rank 0's shared memory
        asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
        if (tid == 0) *cluster.map_shared_rank(&s_all[slice], 0) = tot;
    } else {
        asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
    }
    cluster.sync();  // the statistics have landed; the other CTAs are done and may leave
    if (slice == 0) {
        if (tid < kWarp) {
            // lane r takes slice r's statistic; maximum first, one move per lane, then sums
            SoftStat mine = stat_empty();
            if (tid < n_slices) mine = s_all[tid];
            float rm = mine.m;
#pragma unroll
            for (int o = kCogMaxCluster / 2; o > 0; o >>= 1) rm = fmaxf(rm, __shfl_xor_sync(0xffffffffu, rm, o));
            float rz = mine.z, rw = mine.w;  // a NaN Z (non-finite flag) stays NaN through the sums
            if (mine.z > 0.f) {
                const float dm = mine.m - rm;
                const float sc = expf(dm);
                rz = mine.z * sc;
                rw = (mine.w + dm * mine.z) * sc;
            }
#pragma unroll
            for (int o = kCogMaxCluster / 2; o > 0; o >>= 1) {
                rz += __shfl_xor_sync(0xffffffffu, rz, o);
                rw += __shfl_xor_sync(0xffffffffu, rw, o);
            }
            const SoftStat tot = SoftStat{rm, rz, rw};
            if (tid == 0) {
                int flags = 0;
                float s, h;
                if (!(tot.z > 0.f)) {  // a +inf / NaN logit (z is NaN), or no finite logit at all
                    flags |= CLADA_STATUS_NONFINITE_LOGIT;
                    s = h = NAN;
                } else {
                    const float logz = logf(tot.z);
                    h = logz - tot.w / tot.z;
                    if (!tok_ok) {
                        flags |= CLADA_STATUS_BAD_TOKEN;
                        s = NAN;
                    } else {
                        s = (tot.m + logz) - tok_logit;
                    }
                }
                surprisal[b] = s;
                entropy[b] = h;
                // which of the four thresholds of Eq. final_threshold this token selects
                if (level_out) level_out[b] = (s > tau_s ? 1 : 0) + (h > tau_H ? 2 : 0);
                s_out[0] = s;
                s_out[1] = h;
                if (flags && status) atomicOr(status, flags);
            }
        }
        if (tau_base != nullptr) {
            __syncthreads();
            const float s = s_out[0], h = s_out[1];
            if (tid < L) {  // operands fetched at the start
                float mult = 1.0f;
                if (s > tau_s) mult = __fadd_rn(mult, adj_lambda);
                if (h > tau_H) mult = __fadd_rn(mult, adj_gamma);
                tau_final[(size_t)b * L + tid] = __fmul_rn(adj_base, mult);
            }
            for (int l = tid + kCogThreads; l < L; l += kCogThreads) {
                float mult = 1.0f;
                if (s > tau_s) mult = __fadd_rn(mult, lambda[l]);
                if (h > tau_H) mult = __fadd_rn(mult, gamma[l]);
                tau_final[(size_t)b * L + l] = __fmul_rn(tau_base[(size_t)b * L + l], mult);
            }
        }
    }
}

__global__ void adjust_threshold_kernel(const float *__restrict__ tau_base,
                                        const float *__restrict__ lambda,
                                        const float *__restrict__ gamma, float tau_s, float tau_H,
                                        const float *__restrict__ surprisal,
                                        const float *__restrict__ entropy, int B, int L,
                                        float *__restrict__ tau_final) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * L) return;
    const int b = i / L, l = i % L;
    float mult = 1.0f;
    if (surprisal[b] > tau_s) mult = __fadd_rn(mult, lambda[l]);
    if (entropy[b] > tau_H) mult = __fadd_rn(mult, gamma[l]);
    tau_final[i] = __fmul_rn(tau_base[i], mult);
}

static int launch_cogload(const void *logits, int32_t dtype, int32_t B, int64_t V, int64_t row_stride,
                          const int32_t *token_id, float *surprisal, float *entropy,
                          int32_t *status, const float *tau_base, const float *lambda,
                          const float *gamma, float tau_s, float tau_H, int L, float *tau_final,
                          int32_t *level_out, void *stream) {
    if (!logits || !token_id || !surprisal || !entropy) return CLADA_ERR_NULL;
    if (!dtype_ok(dtype)) return CLADA_ERR_DTYPE;
    if (B <= 0 || V <= 0 || row_stride < V) return CLADA_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(logits) % elem_size(dtype)) return CLADA_ERR_ALIGN;
    cudaLaunchConfig_t cfg = {};
    // one CTA per 4096 logits of a row, at most a portable cluster of 8
    int n_slices = 1;
    while (n_slices < kCogMaxCluster && (int64_t)n_slices * 4096 < V) n_slices *= 2;
    if (B > 65535) return CLADA_ERR_UNSUPPORTED;
    cfg.gridDim = dim3(n_slices, B);
    cfg.blockDim = dim3(kCogThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = n_slices;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (dtype == CLADA_F32)
        CLADA_CUDA_TRY(cudaLaunchKernelEx(&cfg, cogload_kernel<float>, static_cast<const float *>(logits), V,
                                          row_stride, token_id, surprisal, entropy, status, tau_base, lambda, gamma,
                                          tau_s, tau_H, L, tau_final, level_out));
    else if (dtype == CLADA_BF16)
        CLADA_CUDA_TRY(cudaLaunchKernelEx(&cfg, cogload_kernel<__nv_bfloat16>,
                                          static_cast<const __nv_bfloat16 *>(logits), V, row_stride, token_id,
                                          surprisal, entropy, status, tau_base, lambda, gamma, tau_s, tau_H, L,
                                          tau_final, level_out));
    else
        CLADA_CUDA_TRY(cudaLaunchKernelEx(&cfg, cogload_kernel<__half>, static_cast<const __half *>(logits), V,
                                          row_stride, token_id, surprisal, entropy, status, tau_base, lambda, gamma,
                                          tau_s, tau_H, L, tau_final, level_out));
    return CLADA_OK;
}

}  // namespace clada

using namespace clada;

extern "C" {

int clada_cogload(const void *logits, int32_t logits_dtype, int32_t B, int64_t V, int64_t row_stride,
                  const int32_t *token_id, float *surprisal, float *entropy, int32_t *status,
                  void *stream) {
    CLADA_RANGE("clada_cogload");
    return launch_cogload(logits, logits_dtype, B, V, row_stride, token_id, surprisal, entropy, status,
                          nullptr, nullptr, nullptr, 0.f, 0.f, 0, nullptr, nullptr, stream);
}

// Surprisal and entropy as clada_cogload, plus the load level I(s > tau_s) + 2 I(H > tau_H) that indexes
// the nested lists' counts (the same comparisons as Eq. final_threshold's indicators).
int clada_cogload_level(const void *logits, int32_t logits_dtype, int32_t B, int64_t V, int64_t row_stride,
                        const int32_t *token_id, float tau_s, float tau_H, float *surprisal, float *entropy,
                        int32_t *level, int32_t *status, void *stream) {
    CLADA_RANGE("clada_cogload_level");
    if (!level) return CLADA_ERR_NULL;
    return launch_cogload(logits, logits_dtype, B, V, row_stride, token_id, surprisal, entropy, status,
                          nullptr, nullptr, nullptr, tau_s, tau_H, 0, nullptr, level, stream);
}

int clada_adjust_threshold(const float *tau_base, const float *lambda, const float *gamma, float tau_s,
                           float tau_H, const float *surprisal, const float *entropy, int32_t B,
                           int32_t L, float *tau_final, void *stream) {
    CLADA_RANGE("clada_adjust_threshold");
    if (!tau_base || !lambda || !gamma || !surprisal || !entropy || !tau_final) return CLADA_ERR_NULL;
    if (B <= 0 || L <= 0) return CLADA_ERR_SHAPE;
    const int threads = 128;
    const int blocks = (B * L + threads - 1) / threads;
    adjust_threshold_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        tau_base, lambda, gamma, tau_s, tau_H, surprisal, entropy, B, L, tau_final);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

int clada_cogload_adjust(const void *logits, int32_t logits_dtype, int32_t B, int64_t V,
                         int64_t row_stride, const int32_t *token_id, const float *tau_base,
                         const float *lambda, const float *gamma, float tau_s, float tau_H, int32_t L,
                         float *surprisal, float *entropy, float *tau_final, int32_t *status,
                         void *stream) {
    CLADA_RANGE("clada_cogload_adjust");
    if (!tau_base || !lambda || !gamma || !tau_final) return CLADA_ERR_NULL;
    if (L <= 0) return CLADA_ERR_SHAPE;
    return launch_cogload(logits, logits_dtype, B, V, row_stride, token_id, surprisal, entropy, status,
                          tau_base, lambda, gamma, tau_s, tau_H, L, tau_final, nullptr, stream);
}

}  // extern "C"
