// Nested index lists: the four masks of a sequence in one list.
//
// Eq. final_threshold yields tau_base * m with m in {1, 1+lambda, 1+gamma, (1+lambda)+gamma}, and a kept set
// is { j : A_j >= tau }, so every kept set is a leading part of the neurons listed in descending order of
// score.  Once after prefill, per sequence:
//   order  = neurons by descending score, equal scores by ascending index        [d_ff] int32
//   counts = |{ j : A_j >= tau_base * m_k }| for the four multipliers            [4]    int32
// A decode step then needs the load level k = I(s > tau_s) + 2 I(H > tau_H) (clada_cogload_level) and reads
// order[0 .. counts[k]): no per-step threshold test, ranking or compaction, and the per-sequence state
// is one int32 list instead of the fp32 scores plus masks.
//
// Rank sort: a neuron's place in the list is the number of neurons that come before it -- those with a larger
// score, or an equal score and a smaller index -- so every place can be computed independently and exactly.
// A sequence is shared by several CTAs; each holds the whole score vector in shared memory (as bit patterns:
// scores are norms, so the patterns of the positive ones order them; see score_key for the rest) and ranks its slice, one warp per neuron, lanes
// striding over the vector.  The four counts come from the first CTA of the sequence by a block-wide sum.  The
// multipliers are formed on the host exactly as the adjustment kernel forms them (fp32, one addition at a time),
// the thresholds with one fp32 multiplication.
#include <math.h>

#include <algorithm>

#include "common.cuh"
#include "nvtx_ranges.cuh"

namespace clada {

constexpr int kNestThreads = 1024;
constexpr int kNestMaxN = 32768;  // the score vector must fit shared memory (4 bytes per neuron)

struct NestMults {
    float m[4];
};

// Sort key of a score: scores are norms, so the bit patterns of the positive ones order them.  What is not a
// positive number is put where the selection A_j >= tau puts it: NaN compares false with every threshold and
// sorts after everything (key 0); zero of either sign and anything negative sort just before it (key 1).
__device__ __forceinline__ unsigned score_key(float a) {
    if (a > 0.f) return __float_as_uint(a) + 1u;
    return a != a ? 0u : 1u;
}

__global__ void __launch_bounds__(kNestThreads)
nested_build_kernel(const float *__restrict__ scores, int d_ff, const float *__restrict__ tau_base,
                    long long tau_stride, const NestMults mults, int32_t *__restrict__ order,
                    int32_t *__restrict__ counts) {
    extern __shared__ unsigned s_key[];
    __shared__ int s_part[kNestThreads / kWarp][4];
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *A = scores + (size_t)b * d_ff;
    for (int i = tid; i < d_ff; i += kNestThreads) s_key[i] = score_key(A[i]);
    __syncthreads();
    const int e0 = (int)(((long long)d_ff * blockIdx.x) / gridDim.x);
    const int e1 = (int)(((long long)d_ff * (blockIdx.x + 1)) / gridDim.x);
    // before(e) = #{k < e : key_k >= key_e} + #{k > e : key_k > key_e}: one comparison per pair, four pairs per
    // 16-byte shared-memory load; the vector that holds e and the ragged end of the row go element by element.
    const uint4 *s_vec = reinterpret_cast<const uint4 *>(s_key);
    const int nvec = d_ff / 4;
    for (int e = e0 + warp; e < e1; e += kNestThreads / kWarp) {
        const unsigned a = s_key[e];
        const int ev = e >> 2;
        int before = 0;
        for (int v = lane; v < min(ev, nvec); v += kWarp) {
            const uint4 q = s_vec[v];
            before += (q.x >= a) + (q.y >= a) + (q.z >= a) + (q.w >= a);
        }
        for (int v = ev + 1 + lane; v < nvec; v += kWarp) {
            const uint4 q = s_vec[v];
            before += (q.x > a) + (q.y > a) + (q.z > a) + (q.w > a);
        }
        {
            int k = -1;  // lanes 0..3: the vector around e; lanes 4..: the elements after the last whole vector
            if (lane < 4) {
                if (ev < nvec) k = ev * 4 + lane;
            } else if (nvec * 4 + lane - 4 < d_ff) {
                k = nvec * 4 + lane - 4;
            }
            if (k >= 0 && k != e) {
                const unsigned v = s_key[k];
                before += k < e ? (v >= a) : (v > a);
            }
        }
        before = warp_sum(before);
        if (lane == 0) order[(size_t)b * d_ff + before] = e;
    }
    if (blockIdx.x == 0) {
        float tau[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) tau[k] = __fmul_rn(tau_base[(size_t)b * tau_stride], mults.m[k]);
        int c[4] = {0, 0, 0, 0};
        for (int i = tid; i < d_ff; i += kNestThreads) {
            const float a = A[i];
#pragma unroll
            for (int k = 0; k < 4; ++k) c[k] += (a >= tau[k]) ? 1 : 0;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int w = warp_sum(c[k]);
            if (lane == 0) s_part[warp][k] = w;
        }
        __syncthreads();
        if (tid < 4) {
            int tot = 0;
            for (int w = 0; w < kNestThreads / kWarp; ++w) tot += s_part[w][tid];
            counts[(size_t)b * 4 + tid] = tot;
        }
    }
}

// For many sequences of a wide layer the pairwise count above is more work than a sort: one CTA per sequence,
// (score, index) keys in shared memory, bitonic network; the counts as above.  d_ff <= 16384 (8-byte keys of the
// next power of two in shared memory).
constexpr int kNestSortMaxN = 16384;

__global__ void __launch_bounds__(kNestThreads)
nested_sort_kernel(const float *__restrict__ scores, int d_ff, int n_pow2, const float *__restrict__ tau_base,
                    long long tau_stride, const NestMults mults, int32_t *__restrict__ order,
                    int32_t *__restrict__ counts) {
    extern __shared__ unsigned long long s_key64[];
    __shared__ int s_part[kNestThreads / kWarp][4];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *A = scores + (size_t)b * d_ff;
    float tau[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) tau[k] = __fmul_rn(tau_base[(size_t)b * tau_stride], mults.m[k]);
    // Complementing the score's key turns the ascending network into descending score, and the index in the
    // low word breaks ties upward.
    int c[4] = {0, 0, 0, 0};
    for (int i = tid; i < n_pow2; i += kNestThreads) {
        unsigned long long key = ~0ull;  // padding sorts last
        if (i < d_ff) {
            const float a = A[i];
            key = ((unsigned long long)(~score_key(a)) << 32) | (unsigned)i;
#pragma unroll
            for (int k = 0; k < 4; ++k) c[k] += (a >= tau[k]) ? 1 : 0;
        }
        s_key64[i] = key;
    }
    __syncthreads();
    for (int k = 2; k <= n_pow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < n_pow2; i += kNestThreads) {
                const int l = i ^ j;
                if (l > i) {
                    const unsigned long long x = s_key64[i], y = s_key64[l];
                    const bool ascending = (i & k) == 0;
                    if ((x > y) == ascending) {
                        s_key64[i] = y;
                        s_key64[l] = x;
                    }
                }
            }
            __syncthreads();
        }
    }
    for (int i = tid; i < d_ff; i += kNestThreads) order[(size_t)b * d_ff + i] = (int32_t)(s_key64[i] & 0xffffffffull);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int w = warp_sum(c[k]);
        if (lane == 0) s_part[warp][k] = w;
    }
    __syncthreads();
    if (tid < 4) {
        int tot = 0;
        for (int w = 0; w < kNestThreads / kWarp; ++w) tot += s_part[w][tid];
        counts[(size_t)b * 4 + tid] = tot;
    }
}


}  // namespace clada

using namespace clada;

extern "C" int clada_nested_build(const float *scores, int32_t B, int32_t d_ff, const float *tau_base,
                                  int64_t tau_stride, float lambda, float gamma, int32_t *order, int32_t *counts,
                                  void *stream) {
    CLADA_RANGE("clada_nested_build");
    if (!scores || !tau_base || !order || !counts) return CLADA_ERR_NULL;
    if (B <= 0 || d_ff <= 0 || tau_stride < 0) return CLADA_ERR_SHAPE;
    if (d_ff > kNestMaxN || B > 65535) return CLADA_ERR_UNSUPPORTED;
    NestMults mults;
    {
        // level k = I(s > tau_s) + 2 I(H > tau_H); the sums are taken as the adjustment takes them:
        // start from 1, add lambda if the first indicator holds, then gamma if the second does
        volatile float one = 1.0f;
        volatile float m1 = one + lambda;
        volatile float m2 = one + gamma;
        volatile float m3 = m1 + gamma;
        mults.m[0] = one;
        mults.m[1] = m1;
        mults.m[2] = m2;
        mults.m[3] = m3;
    }
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(nested_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kNestMaxN * (int)sizeof(unsigned)));
        CLADA_CUDA_TRY(cudaFuncSetAttribute(nested_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kNestSortMaxN * (int)sizeof(unsigned long long)));
        configured[di.device & 63] = true;
    }
    // The pairwise count costs B * d_ff^2 comparisons spread over the device, the sort a fixed ~0.2 ms for up to
    // one sequence per SM: take the sort for many wide sequences.
    if (d_ff <= kNestSortMaxN && (double)B * d_ff * d_ff > 6e8) {
        int n_pow2 = 2;
        while (n_pow2 < d_ff) n_pow2 <<= 1;
        nested_sort_kernel<<<B, kNestThreads, (size_t)n_pow2 * sizeof(unsigned long long),
                             static_cast<cudaStream_t>(stream)>>>(scores, d_ff, n_pow2, tau_base, tau_stride, mults,
                                                                  order, counts);
        CLADA_CUDA_TRY(cudaGetLastError());
        return CLADA_OK;
    }
    // enough CTAs per sequence to occupy the device, at least 32 neurons each
    int split = (di.num_sms + B - 1) / B;
    split = std::max(1, std::min(split, (d_ff + 31) / 32));
    nested_build_kernel<<<dim3(split, B), kNestThreads, (size_t)d_ff * sizeof(unsigned),
                          static_cast<cudaStream_t>(stream)>>>(scores, d_ff, tau_base, tau_stride, mults, order,
                                                               counts);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}
