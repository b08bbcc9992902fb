// The single-sequence decode launch (clada_ffn.cu) as the decode entry points (clada_decode.cu) see it.
#pragma once

#include "common.cuh"
#include "ffn_common.cuh"

namespace clada {

struct FfnParams {
    const void *w_gate, *w_up, *w_down_t;
    const void *x;        // [d_model]
    const float *scores;  // [d_ff]
    const float *tau;     // one float
    void *y;              // [d_model]
    int y_dtype;
    uint8_t *mask_out;    // [d_ff] or null
    int32_t *idx_out;     // [d_ff] or null
    int32_t *count_out;   // one int or null
    float *partials;      // [gridDim.x, consumer groups, d_model]
    WsCtrl *ctrl;
    int32_t *status;
    int d_model, d_ff;
    int act;              // clada_activation of the layer
    // Nested index lists instead of scores and a threshold (order != null): the kept set is
    // order[0 .. counts[*level]), neurons in descending order of score.
    const int32_t *order;   // [d_ff]
    const int32_t *counts;  // [4]
    const int32_t *level;   // one int in 0..3
};

constexpr int kSingleMaxDff = 4 * kWarp * kFfnThreads;  // four prologue batches of one 32-neuron chunk per thread

// One launch for one sequence of a layer of the given clada_dtype.
int launch_ffn_single(const FfnParams &p, int dtype, cudaStream_t st);

}  // namespace clada
