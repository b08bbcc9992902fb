// Pieces shared by the two batched decode kernels (CUDA-core tile kernel, tensor-core tile kernel): the launch
// parameters, the prologue that builds a CTA's share of the union of a tile's kept sets, and the epilogue that
// sums the CTAs' partial outputs.
#pragma once

#include "common.cuh"
#include "ffn_common.cuh"

namespace clada {

struct FfnBatchParams {
    const void *w_gate, *w_up, *w_down_t;
    const void *x;           // sequence b at x + b * x_stride (bytes)
    size_t x_stride;
    const float *scores;     // [BT, d_ff]
    const unsigned *keep_words;  // [BT, chunks] keep bits A_bj >= tau_b per 32-neuron chunk, or null: test the scores here
    const float *tau;        // sequence b at tau[b * tau_stride]
    long long tau_stride;
    void *y;                 // sequence b at y + b * y_stride (bytes)
    size_t y_stride;
    int y_dtype;
    float *partials;         // [gridDim.x, BT, d_model]
    WsCtrl *ctrl;
    int32_t *status;
    int d_model, d_ff;
    int act;                 // clada_activation of the layer
};

constexpr int kBatchMaxBatches = 4;  // prologue batches: d_ff <= 4 * 32 * kFfnThreads

// Prologue of a tile of BT sequences, run by all kFfnThreads threads of the CTA: every sequence's keep bits
// A_bj >= tau_b per 32-neuron chunk (s_balb), their union (s_bal), the union's ranks by a block scan, and this
// CTA's equal share of the union in ascending order: s_list[i] = neuron, s_keep[i] = bit b set iff sequence b
// keeps it.  s_tau must hold the BT thresholds (visible to all threads).  Returns the share's size.
template <int BT, int NT = kFfnThreads>
__device__ __forceinline__ int batch_union_share(const FfnBatchParams &p, const float *s_tau, unsigned *s_bal,
                                                 unsigned *s_balb, int *s_list, int *s_keep, int *s_wtot,
                                                 const uint64_t keep_policy) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff;
    const int chunks = (F + kWarp - 1) / kWarp;
    // ---- prologue: keep-bits per sequence, their union, ranks of the union -----------------------
    const int n_batches = (chunks + NT - 1) / NT;
    {
        int slot = tid + (cta * 37) % NT;
        if (slot >= NT) slot -= NT;
        for (int bt = 0; bt < n_batches; ++bt) {
            const int q = bt * NT + slot;
            if (q >= chunks) continue;
            const int j0 = q * kWarp;
            unsigned wu = 0;
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                unsigned w = 0;
                if (p.keep_words) {  // the words of the whole batch were computed once by keep_words_kernel
                    w = p.keep_words[(size_t)b * chunks + q];
                    s_balb[b * chunks + q] = w;
                    wu |= w;
                    continue;
                }
                const float *sc = p.scores + (size_t)b * F;
                const float tau = s_tau[b];
                if (((reinterpret_cast<uintptr_t>(sc) & 15u) == 0) && j0 + kWarp <= F) {
                    float4 v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = ld_keep4(reinterpret_cast<const float4 *>(sc + j0) + u, keep_policy);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        w |= (v[u].x >= tau ? 1u : 0u) << (4 * u);
                        w |= (v[u].y >= tau ? 1u : 0u) << (4 * u + 1);
                        w |= (v[u].z >= tau ? 1u : 0u) << (4 * u + 2);
                        w |= (v[u].w >= tau ? 1u : 0u) << (4 * u + 3);
                    }
                } else {
                    for (int u = 0; u < kWarp; ++u)
                        if (j0 + u < F && ld_keep(sc + j0 + u, keep_policy) >= tau) w |= 1u << u;
                }
                s_balb[b * chunks + q] = w;
                wu |= w;
            }
            s_bal[q] = wu;
        }
    }
    __syncthreads();
    unsigned bal[kBatchMaxBatches];
    int first_rank[kBatchMaxBatches];
    int n_act = 0;
#pragma unroll
    for (int bt = 0; bt < kBatchMaxBatches; ++bt) {
        bal[bt] = 0u;
        first_rank[bt] = 0;
        if (bt >= n_batches) continue;  // uniform
        const int q = bt * NT + tid;
        if (q < chunks) bal[bt] = s_bal[q];
        const int cnt = __popc(bal[bt]);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < kWarp; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (bt > 0) __syncthreads();
        if (lane == kWarp - 1) s_wtot[warp] = incl;
        __syncthreads();
        int wbase = 0, btot = 0;
#pragma unroll
        for (int w = 0; w < (NT / kWarp); ++w) {
            const int v = s_wtot[w];
            wbase += (w < warp) ? v : 0;
            btot += v;
        }
        first_rank[bt] = n_act + wbase + incl - cnt;
        n_act += btot;
    }
    const int r0 = (int)(((int64_t)n_act * cta) / n_ctas);
    const int r1 = (int)(((int64_t)n_act * (cta + 1)) / n_ctas);
#pragma unroll
    for (int bt = 0; bt < kBatchMaxBatches; ++bt) {
        if (bt >= n_batches) continue;  // uniform
        const int q = bt * NT + tid;
        const int fr = first_rank[bt];
        const bool in_share = q < chunks && fr < r1 && fr + __popc(bal[bt]) > r0;
        unsigned todo = __ballot_sync(0xffffffffu, in_share);
        while (todo) {
            const int t = __ffs(todo) - 1;
            todo &= todo - 1;
            const unsigned wb = __shfl_sync(0xffffffffu, bal[bt], t);
            const int wfr = __shfl_sync(0xffffffffu, fr, t);
            const int qq = bt * NT + warp * kWarp + t;
            const int rank = wfr + __popc(wb & ((1u << lane) - 1u));
            if (((wb >> lane) & 1u) && rank >= r0 && rank < r1) {
                int bits = 0;
#pragma unroll
                for (int b = 0; b < BT; ++b) bits |= (int)((s_balb[b * chunks + qq] >> lane) & 1u) << b;
                s_list[rank - r0] = qq * kWarp + lane;
                s_keep[rank - r0] = bits;
            }
        }
    }
    return r1 - r0;
}

// Epilogue of a tile: after the grid barrier every CTA sums a slice of (sequence, column group) pairs over all
// CTAs' partial rows [n_ctas][BT][d_model] in CTA order (a warp per group of 4 columns: lane l adds rows l,
// l+32, ..., then the 32 lane sums combine by butterfly) and writes y.
template <int BT, int NT = kFfnThreads>
__device__ __forceinline__ void batch_column_sums(const FfnBatchParams &p) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x, d = p.d_model;
    const int ngroups = d / 4;
    for (int it = cta + warp * n_ctas; it < BT * ngroups; it += n_ctas * (NT / kWarp)) {
        const int b = it / ngroups, q = it % ngroups;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int rb = 0; rb < n_ctas; rb += 5 * kWarp) {
            float4 v[5];
#pragma unroll
            for (int u = 0; u < 5; ++u) {
                const int r = rb + u * kWarp + lane;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (r < n_ctas)
                    v[u] = __ldcg(reinterpret_cast<const float4 *>(p.partials + ((size_t)r * BT + b) * d) + q);
            }
#pragma unroll
            for (int u = 0; u < 5; ++u) {
                s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w;
            }
        }
        s.x = warp_sum(s.x); s.y = warp_sum(s.y); s.z = warp_sum(s.z); s.w = warp_sum(s.w);
        if (lane == 0) {
            char *yb = static_cast<char *>(p.y) + b * p.y_stride;
            if (p.y_dtype == CLADA_F32) {
                reinterpret_cast<float4 *>(yb)[q] = s;
            } else {
                reinterpret_cast<uint2 *>(yb)[q] = pack4_16bit(p.y_dtype, s);
            }
        }
    }
}

// Keep bits of a whole batch, once per decode call: words[b][q] bit u = (scores[b][32 q + u] >= tau_b).  Every CTA
// of every tile launch then reads 4 bytes per (sequence, chunk) instead of testing 128 bytes of scores.
int launch_keep_words(const float *scores, int B, int d_ff, const float *tau, long long tau_stride, unsigned *words,
                      cudaStream_t st);
inline size_t keep_words_bytes(int B, int d_ff) {
    return (((size_t)B * ((d_ff + 31) / 32) * sizeof(unsigned)) + 255) & ~(size_t)255;
}

// The tensor-core tile kernel (clada_ffn_batch_tc.cu): whether it takes this layer and tile, and its launch.
bool ffn_batch_tc_supported(const clada_layer *layer, int bt);
int launch_ffn_batch_tc(const FfnBatchParams &p, int dtype, int bt, cudaStream_t st);

// The dense pass for 3-16 sequences of a 16-bit layer (clada_ffn_batch_dense.cu): every row of the layer is read
// once for the whole launch.  At the sparsities the method runs at (40-60 % per sequence) three kept sets already
// cover 80-95 % of the layer, and the pass streams faster than the tile kernels (which read only the union, at a
// lower rate): measured on a 4096 x 14336 layer, four sequences at 40 % take 67 us densely and 85 us as a tile.
// Two sequences keep the tile kernel: their union leaves a quarter of the layer out.
constexpr int kDenseMinSeqs = 3;
constexpr int kDenseMaxSeqs = 16;
bool ffn_batch_dense_supported(const clada_layer *layer, int B);
size_t ffn_batch_dense_scratch_bytes(const clada_layer *layer, int B);
int launch_ffn_batch_dense(const clada_layer *layer, int B, const void *x, const float *scores, const float *tau,
                           long long tau_stride, void *y, int y_dtype, void *ws, int32_t *status, cudaStream_t st);

}  // namespace clada
