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
// One CTA per sequence: (score, index) keys in shared memory, bitonic network, then the four counts by a
// block-wide sum.  The multipliers are formed on the host exactly as the adjustment kernel forms them
// (fp32, one addition at a time), the thresholds with one fp32 multiplication.
#include <math.h>

#include "common.cuh"

namespace clada {

constexpr int kNestThreads = 1024;
constexpr int kNestMaxN = 16384;  // keys of the next power of two must fit shared memory (128 KB)

struct NestMults {
    float m[4];
};

__global__ void __launch_bounds__(kNestThreads)
nested_build_kernel(const float *__restrict__ scores, int d_ff, int n_pow2, const float *__restrict__ tau_base,
                    long long tau_stride, const NestMults mults, int32_t *__restrict__ order,
                    int32_t *__restrict__ counts) {
    extern __shared__ unsigned long long s_key[];
    __shared__ int s_part[kNestThreads / kWarp][4];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *A = scores + (size_t)b * d_ff;
    float tau[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) tau[k] = __fmul_rn(tau_base[(size_t)b * tau_stride], mults.m[k]);
    // Scores are norms (non-negative), so their bit patterns order them; complementing the pattern turns
    // the ascending network into descending score, and the index in the low word breaks ties upward.
    int c[4] = {0, 0, 0, 0};
    for (int i = tid; i < n_pow2; i += kNestThreads) {
        unsigned long long key = ~0ull;  // padding sorts last
        if (i < d_ff) {
            const float a = A[i];
            key = ((unsigned long long)(~__float_as_uint(a)) << 32) | (unsigned)i;
#pragma unroll
            for (int k = 0; k < 4; ++k) c[k] += (a >= tau[k]) ? 1 : 0;
        }
        s_key[i] = key;
    }
    __syncthreads();
    for (int k = 2; k <= n_pow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < n_pow2; i += kNestThreads) {
                const int l = i ^ j;
                if (l > i) {
                    const unsigned long long x = s_key[i], y = s_key[l];
                    const bool ascending = (i & k) == 0;
                    if ((x > y) == ascending) {
                        s_key[i] = y;
                        s_key[l] = x;
                    }
                }
            }
            __syncthreads();
        }
    }
    for (int i = tid; i < d_ff; i += kNestThreads) order[(size_t)b * d_ff + i] = (int32_t)(s_key[i] & 0xffffffffull);
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
    if (!scores || !tau_base || !order || !counts) return CLADA_ERR_NULL;
    if (B <= 0 || d_ff <= 0 || tau_stride < 0) return CLADA_ERR_SHAPE;
    if (d_ff > kNestMaxN || B > 65535) return CLADA_ERR_UNSUPPORTED;
    int n_pow2 = 2;
    while (n_pow2 < d_ff) n_pow2 <<= 1;
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
                                            kNestMaxN * (int)sizeof(unsigned long long)));
        configured[di.device & 63] = true;
    }
    nested_build_kernel<<<B, kNestThreads, (size_t)n_pow2 * sizeof(unsigned long long),
                          static_cast<cudaStream_t>(stream)>>>(scores, d_ff, n_pow2, tau_base, tau_stride, mults,
                                                               order, counts);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}
