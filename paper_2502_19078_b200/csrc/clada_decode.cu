// The decode entry points of the C ABI: host-side checks, the choice of launches for a batch (one dense pass for
// 3-16 sequences of a 16-bit layer, else tiles of 4 or 2 sequences, else one launch per sequence), the scratch
// each choice needs, and the entry that allocates nothing.
#include <algorithm>

#include "common.cuh"
#include "nvtx_ranges.cuh"
#include "ffn_batch.cuh"
#include "ffn_common.cuh"
#include "ffn_single.cuh"

using namespace clada;

// Host-side checks of a decode call; nothing is enqueued here.
static int decode_validate(const clada_layer *layer, const void *x, int32_t B, const float *scores,
                           const float *tau_final, int64_t tau_stride, const void *y, int32_t y_dtype) {
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!x || !scores || !tau_final || !y) return CLADA_ERR_NULL;
    if (B <= 0 || tau_stride < 0) return CLADA_ERR_SHAPE;
    if (!dtype_ok(y_dtype)) return CLADA_ERR_DTYPE;
    if (!aligned16(x) || !aligned16(y)) return CLADA_ERR_ALIGN;
    if (layer->d_ff > kSingleMaxDff) return CLADA_ERR_UNSUPPORTED;
    return CLADA_OK;
}

// Sequences per launch for the next `remaining` sequences of a batch, at most max_tile (16, 4, 2 or 1): three or
// more sequences of a 16-bit layer go through the layer in one dense pass, up to 16 per launch; otherwise tiles of
// 4 or 2 read the union of their kept sets (a tile kernel that takes 4 sequences of this layer also takes 2).
static int decode_tile(const clada_layer *layer, int remaining, int max_tile, bool *dense) {
    *dense = false;
    if (max_tile >= kDenseMaxSeqs && remaining >= kDenseMinSeqs) {
        const int n = remaining < kDenseMaxSeqs ? remaining : kDenseMaxSeqs;
        if (ffn_batch_dense_supported(layer, n)) {
            *dense = true;
            return n;
        }
    }
    const int bt = ffn_batch_tile(layer, remaining);
    return bt < max_tile ? bt : (max_tile < 4 ? max_tile : 4);
}

// Whether any launch of the call is a tile of 2 or 4 sequences (those read the batch's keep words).
static bool decode_has_tiles(const clada_layer *layer, int32_t B, int max_tile) {
    for (int b = 0; b < B;) {
        bool dense;
        const int bt = decode_tile(layer, B - b, max_tile, &dense);
        if (bt > 1 && !dense) return true;
        b += bt;
    }
    return false;
}

// Scratch bytes a decode call needs when its launches take at most max_tile sequences: the control words, the
// largest per-launch scratch (dense pass: a partial output per group of CTAs and the groups' hidden activations;
// tile: one fp32 partial output row per (CTA, sequence of the tile); single sequence: one row per consumer group),
// and behind it the batch's keep words when tiles are launched.
static size_t decode_scratch_bytes(const clada_layer *layer, int32_t B, int num_sms, int max_tile) {
    const int vpr = layer->d_model / (layer->dtype == CLADA_F32 ? 4 : 8);
    size_t launch = 0;
    bool tiles = false;
    for (int b = 0; b < B;) {
        bool dense;
        const int bt = decode_tile(layer, B - b, max_tile, &dense);
        size_t need;
        if (dense) {
            need = ffn_batch_dense_scratch_bytes(layer, bt);
        } else {
            need = (size_t)num_sms * (bt > 1 ? bt : ffn_groups(vpr)) * layer->d_model * sizeof(float);
            tiles = tiles || bt > 1;
        }
        launch = std::max(launch, need);
        b += bt;
    }
    launch = (launch + 255) & ~(size_t)255;
    return kWsCtrlBytes + launch + (tiles ? keep_words_bytes_of(B, layer->d_ff) : 0);
}

// The launches of a validated decode call whose scratch holds tiles of up to max_tile sequences.
static int decode_enqueue(const clada_layer *layer, const void *x, int32_t B, const float *scores,
                          const float *tau_final, int64_t tau_stride, void *y, int32_t y_dtype,
                          uint8_t *mask_out, int32_t *idx_out, int32_t *count_out, void *ws, int max_tile,
                          int32_t *status, void *stream) {
    int rc;
    const size_t esz = elem_size(layer->dtype);
    const size_t ysz = elem_size(y_dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Tiles of sequences: the keep bits of the whole batch are computed once, into the end of the scratch, and
    // every CTA of every tile launch reads those words instead of testing the score vectors itself.
    unsigned *words = nullptr;
    if (decode_has_tiles(layer, B, max_tile)) {
        DeviceInfo di;
        rc = device_info(&di);
        if (rc != CLADA_OK) return rc;
        const size_t total = decode_scratch_bytes(layer, B, di.num_sms, max_tile);
        words = reinterpret_cast<unsigned *>(static_cast<char *>(ws) + total - keep_words_bytes_of(B, layer->d_ff));
        rc = launch_keep_words(scores, B, layer->d_ff, tau_final, tau_stride, words, st);
        if (rc != CLADA_OK) return rc;
    }
    const size_t chunks = (size_t)(layer->d_ff + 31) / 32;
    int b = 0;
    while (b < B) {
        // Tiles of 4 or 2 sequences read each row of the union of their kept sets once.
        bool dense;
        const int bt = decode_tile(layer, B - b, max_tile, &dense);
        if (bt > 1) {
            if (mask_out || idx_out || count_out) {  // the batch kernels compute y only
                rc = clada_select(scores + (size_t)b * layer->d_ff, bt, layer->d_ff, tau_final + (size_t)b * tau_stride,
                                  tau_stride, mask_out ? mask_out + (size_t)b * layer->d_ff : nullptr,
                                  idx_out ? idx_out + (size_t)b * layer->d_ff : nullptr,
                                  count_out ? count_out + b : nullptr, stream);
                if (rc != CLADA_OK) return rc;
            }
            if (dense)
                rc = launch_ffn_batch_dense(layer, bt, static_cast<const char *>(x) + (size_t)b * layer->d_model * esz,
                                            scores + (size_t)b * layer->d_ff, tau_final + (size_t)b * tau_stride,
                                            tau_stride, static_cast<char *>(y) + (size_t)b * layer->d_model * ysz,
                                            y_dtype, ws, status, st);
            else
                rc = launch_ffn_batch(layer, bt, static_cast<const char *>(x) + (size_t)b * layer->d_model * esz,
                                      scores + (size_t)b * layer->d_ff, tau_final + (size_t)b * tau_stride, tau_stride,
                                      static_cast<char *>(y) + (size_t)b * layer->d_model * ysz, y_dtype, ws,
                                      words + (size_t)b * chunks, status, st);
            if (rc != CLADA_OK) return rc;
            b += bt;
            continue;
        }
        FfnParams p;
        p.w_gate = layer->w_gate;
        p.w_up = layer->w_up;
        p.w_down_t = layer->w_down_t;
        p.x = static_cast<const char *>(x) + (size_t)b * layer->d_model * esz;
        p.scores = scores + (size_t)b * layer->d_ff;
        p.tau = tau_final + (size_t)b * tau_stride;
        p.y = static_cast<char *>(y) + (size_t)b * layer->d_model * ysz;
        p.y_dtype = y_dtype;
        p.mask_out = mask_out ? mask_out + (size_t)b * layer->d_ff : nullptr;
        p.idx_out = idx_out ? idx_out + (size_t)b * layer->d_ff : nullptr;
        p.count_out = count_out ? count_out + b : nullptr;
        p.partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
        p.ctrl = static_cast<WsCtrl *>(ws);
        p.status = status;
        p.d_model = layer->d_model;
        p.d_ff = layer->d_ff;
        p.act = layer->activation;
        p.order = nullptr;
        p.counts = nullptr;
        p.level = nullptr;
        rc = launch_ffn_single(p, layer->dtype, st);
        if (rc != CLADA_OK) return rc;
        ++b;
    }
    return CLADA_OK;
}

static int decode_with_workspace(const clada_layer *layer, const void *x, int32_t B, const float *scores,
                                 const float *tau_final, int64_t tau_stride, void *y, int32_t y_dtype,
                                 uint8_t *mask_out, int32_t *idx_out, int32_t *count_out, void *ws,
                                 size_t ws_bytes, int32_t *status, void *stream) {
    int rc = decode_validate(layer, x, B, scores, tau_final, tau_stride, y, y_dtype);
    if (rc != CLADA_OK) return rc;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    // the dense pass when the workspace holds its scratch (clada_workspace_bytes asks for it), else tiles of 4
    int max_tile = kDenseMaxSeqs;
    if (ws_bytes < decode_scratch_bytes(layer, B, di.num_sms, max_tile)) max_tile = 4;
    if (ws_bytes < decode_scratch_bytes(layer, B, di.num_sms, max_tile)) return CLADA_ERR_WORKSPACE;
    return decode_enqueue(layer, x, B, scores, tau_final, tau_stride, y, y_dtype, mask_out, idx_out, count_out, ws,
                          max_tile, status, stream);
}

extern "C" int clada_sparse_ffn_decode(const clada_layer *layer, const void *x, int32_t B,
                                       const float *scores, const float *tau_final, int64_t tau_stride,
                                       void *y, int32_t y_dtype, uint8_t *mask_out, int32_t *idx_out,
                                       int32_t *count_out, void *ws, size_t ws_bytes, int32_t *status,
                                       void *stream) {
    CLADA_RANGE("clada_sparse_ffn_decode");
    return decode_with_workspace(layer, x, B, scores, tau_final, tau_stride, y, y_dtype, mask_out, idx_out,
                                 count_out, ws, ws_bytes, status, stream);
}

// Decode from nested index lists (clada_nested_build): no scores, no threshold, no compaction -- the
// kept set of sequence b is the leading counts[b][level[b]] entries of order[b].  One launch per sequence.
extern "C" int clada_sparse_ffn_decode_nested(const clada_layer *layer, const void *x, int32_t B,
                                              const int32_t *order, const int32_t *counts, const int32_t *level,
                                              void *y, int32_t y_dtype, int32_t *count_out, void *ws,
                                              size_t ws_bytes, int32_t *status, void *stream) {
    CLADA_RANGE("clada_sparse_ffn_decode_nested");
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!x || !order || !counts || !level || !y) return CLADA_ERR_NULL;
    if (B <= 0) return CLADA_ERR_SHAPE;
    if (!dtype_ok(y_dtype)) return CLADA_ERR_DTYPE;
    if (!aligned16(x) || !aligned16(y)) return CLADA_ERR_ALIGN;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    if (ws_bytes < decode_scratch_bytes(layer, 1, di.num_sms, 1)) return CLADA_ERR_WORKSPACE;
    const size_t esz = elem_size(layer->dtype), ysz = elem_size(y_dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int b = 0; b < B; ++b) {
        FfnParams p = {};
        p.w_gate = layer->w_gate;
        p.w_up = layer->w_up;
        p.w_down_t = layer->w_down_t;
        p.x = static_cast<const char *>(x) + (size_t)b * layer->d_model * esz;
        p.y = static_cast<char *>(y) + (size_t)b * layer->d_model * ysz;
        p.y_dtype = y_dtype;
        p.count_out = count_out ? count_out + b : nullptr;
        p.partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
        p.ctrl = static_cast<WsCtrl *>(ws);
        p.status = status;
        p.d_model = layer->d_model;
        p.d_ff = layer->d_ff;
        p.act = layer->activation;
        p.order = order + (size_t)b * layer->d_ff;
        p.counts = counts + (size_t)b * 4;
        p.level = level + b;
        rc = launch_ffn_single(p, layer->dtype, st);
        if (rc != CLADA_OK) return rc;
    }
    return CLADA_OK;
}

// One decode step of a whole stack.  A single sequence runs all layers in one persistent launch
// (clada_ffn_stack.cu); a batch runs the per-layer call in a native loop (one C call per token instead
// of one per layer; the launches chain with programmatic dependent launch).
extern "C" int clada_sparse_ffn_decode_layers(const clada_layer *layers, int32_t L, const void *x, int32_t B,
                                              const float *scores, const float *tau_final, void *y,
                                              int32_t y_dtype, void *ws, size_t ws_bytes, int32_t *status,
                                              void *stream) {
    CLADA_RANGE("clada_sparse_ffn_decode_layers");
    if (!layers || !x || !scores || !tau_final || !y) return CLADA_ERR_NULL;
    if (L <= 0 || B <= 0) return CLADA_ERR_SHAPE;
    if (!dtype_ok(y_dtype)) return CLADA_ERR_DTYPE;
    for (int l = 0; l < L; ++l) {  // validate everything before enqueueing anything
        int rc = validate_layer(&layers[l], false);
        if (rc != CLADA_OK) return rc;
        if (layers[l].d_model != layers[0].d_model || layers[l].d_ff != layers[0].d_ff ||
            layers[l].dtype != layers[0].dtype)
            return CLADA_ERR_SHAPE;
    }
    if (!aligned16(x) || !aligned16(y)) return CLADA_ERR_ALIGN;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    const size_t d = (size_t)layers[0].d_model, F = (size_t)layers[0].d_ff;
    const size_t x_layer = (size_t)B * d * elem_size(layers[0].dtype), y_layer = (size_t)B * d * elem_size(y_dtype);
    if (ffn_stack_supported(layers, L, B, ws_bytes))
        return launch_ffn_stack(layers, L, x, x_layer, scores, tau_final, 1, y, y_layer, y_dtype, ws, ws_bytes, status,
                                static_cast<cudaStream_t>(stream));
    for (int l = 0; l < L; ++l) {
        int rc = decode_with_workspace(&layers[l], static_cast<const char *>(x) + l * x_layer, B,
                                       scores + (size_t)l * B * F, tau_final + l, L,
                                       static_cast<char *>(y) + l * y_layer, y_dtype, nullptr, nullptr, nullptr, ws,
                                       ws_bytes, status, stream);
        if (rc != CLADA_OK) return rc;
    }
    return CLADA_OK;
}

// ---- the entry point that allocates nothing ---------------------------------------------------
//
// Some callers may not allocate device memory at all: a plug-in that runs inside another engine's
// execution step, where the host engine owns and budgets every byte and forbids allocation calls in
// the step; a serving process that froze its memory plan at start-up; code on a latency-critical path
// where cudaMalloc would synchronise the whole device.  For them the decode kernel's scratch (its
// control words and the per-CTA partial outputs) lives in the fixed array below instead of a
// caller-provided workspace.  Every GPU that loads the library holds these kStaticScratchBytes until
// the process exits.
constexpr int kStaticMaxSms = 160;
constexpr int kStaticMaxDModel = 8192;
constexpr size_t kStaticScratchBytes = kWsCtrlBytes + (size_t)kStaticMaxSms * kStaticMaxDModel * sizeof(float);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// The array's name is only a host-side handle; kernels need its device address, which the runtime
// gives per device.  Looked up once per device, with that device current, and cached.
static int static_scratch_address(void **out) {
    constexpr int kMaxDev = 64;
    static void *cache[kMaxDev] = {};
    int dev = 0;
    CLADA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return CLADA_ERR_UNSUPPORTED;
    if (!cache[dev]) {
        void *ptr = nullptr;
        CLADA_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        cache[dev] = ptr;
    }
    *out = cache[dev];
    return CLADA_OK;
}

extern "C" int clada_sparse_ffn_decode_static(const clada_layer *layer, const void *x, int32_t B,
                                              const float *scores, const float *tau_final,
                                              int64_t tau_stride, void *y, int32_t y_dtype,
                                              uint8_t *mask_out, int32_t *idx_out, int32_t *count_out,
                                              int32_t *status, void *stream) {
    CLADA_RANGE("clada_sparse_ffn_decode_static");
    // Everything that can be refused is refused before the first enqueue.
    int rc = decode_validate(layer, x, B, scores, tau_final, tau_stride, y, y_dtype);
    if (rc != CLADA_OK) return rc;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    // The largest tile of sequences whose partial rows fit the array: a batch that the workspace entry would
    // cut into tiles of 4 runs here in tiles of 2, or one sequence per launch, when the array is too small
    // for more (same results per sequence; the weight rows are then read once per smaller tile).
    int max_tile = kDenseMaxSeqs;
    while (max_tile > 1 && decode_scratch_bytes(layer, B, di.num_sms, max_tile) > kStaticScratchBytes)
        max_tile = max_tile > 4 ? 4 : max_tile >> 1;
    if (layer->d_model > kStaticMaxDModel || di.num_sms > kStaticMaxSms ||
        decode_scratch_bytes(layer, B, di.num_sms, max_tile) > kStaticScratchBytes) {
        set_last_cuda_error(cudaErrorInvalidValue,
                            "clada_sparse_ffn_decode_static: d_model > 8192 or more than 160 SMs exceeds the "
                            "built-in scratch; use clada_sparse_ffn_decode with a workspace");
        return CLADA_ERR_UNSUPPORTED;
    }
    void *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != CLADA_OK) return rc;
    // The array keeps whatever the last call left.  The control words must start at zero (they are
    // zero after a clean call, not after one that timed out), so clear them in stream order.
    CLADA_CUDA_TRY(cudaMemsetAsync(scratch, 0, kWsCtrlBytes, static_cast<cudaStream_t>(stream)));
    return decode_enqueue(layer, x, B, scores, tau_final, tau_stride, y, y_dtype, mask_out, idx_out, count_out,
                          scratch, max_tile, status, stream);
}
