// Shared by the two prefill-statistics paths (CUDA-core and tensor-core): the prompt table passed by
// value to kernels, token-tile bookkeeping, and the finalize step.
#pragma once

#include "common.cuh"

namespace clada {

constexpr int kMaxSeqs = 128;
struct SeqTable {
    int B;
    long long off[kMaxSeqs + 1];
};

// Token tiles of `tile` rows never straddle prompts: prompt b owns tiles_of(T_b, tile) of them.
__host__ __device__ inline int tiles_of(long long rows, int tile) { return (int)((rows + tile - 1) / tile); }

#ifdef __CUDACC__
// Which prompt and which token range a global token-tile index falls in.
__device__ inline void locate_tile(const SeqTable &tab, int ttile, int tile, int &b, long long &t0, long long &t1) {
    int first = 0;
    for (b = 0; b < tab.B - 1; ++b) {
        const int n = tiles_of(tab.off[b + 1] - tab.off[b], tile);
        if (ttile < first + n) break;
        first += n;
    }
    t0 = tab.off[b] + (long long)(ttile - first) * tile;
    t1 = min(t0 + tile, tab.off[b + 1]);
}
#endif

// scores[b,j] = sqrt(sum over prompt b's tiles of partials[tile,j]) * w_down_norm[j], tiles in order.
int launch_prefix_finalize(const float *partials, const SeqTable &tab, int tile, int d_ff,
                           const float *w_down_norm, float *scores, cudaStream_t st);

// CUDA-core scores for any dtype that also leave z, neuron-major (zt[j, t], row stride T_total), for the
// offline threshold search; partials must hold prefix_partials_bytes_cuda_core() bytes.
int run_prefix_scores_with_z(const clada_layer *layer, const void *X, const int64_t *seq_offsets, int32_t B,
                             float *scores, float *partials, float *zt, cudaStream_t st);
size_t prefix_partials_bytes_cuda_core(const int64_t *seq_offsets, int32_t B, int d_ff);

// Tensor-core partial sums (bf16 layers, 128-token tiles).  partials: [sum_b tiles_of(T_b, 128), d_ff].
// z_out (optional): the hidden activations [T_total, d_ff] in the layer's element type.
int run_prefix_partials_tc(const clada_layer *layer, const void *X, const SeqTable &tab, long long T_total,
                           float *partials, int32_t *status, cudaStream_t st, void *z_out = nullptr);

// Y [T, d_model] = Z [T, d_ff] . w_down[d_model, d_ff]^T on the tensor cores (16-bit element types).  scratch
// (optional, 16-byte aligned): down_split_scratch_bytes() bytes let a short prompt's tiles be split along K.
int run_down_tc(const clada_layer *layer, const void *w_down, const void *Z, long long T, void *Y, int y_dtype,
                void *scratch, size_t scratch_bytes, int32_t *status, cudaStream_t st);
size_t down_split_scratch_bytes(const clada_layer *layer, long long T, int num_sms);
constexpr int kTcTokenTile = 128;

}  // namespace clada
