// Library plumbing: version, error strings, device info, workspace, down-projection norms.
#include <stdio.h>
#include <string.h>

#include <algorithm>

#include "common.cuh"
#include "nvtx_ranges.cuh"
#include "ffn_batch.cuh"
#include "prefix_common.cuh"

namespace clada {

static thread_local char g_last_error[512] = "";

void set_last_cuda_error(cudaError_t e, const char *where) {
    snprintf(g_last_error, sizeof g_last_error, "%s: %s (%s)", where, cudaGetErrorName(e),
             cudaGetErrorString(e));
}

int cuda_fail(cudaError_t e, const char *where) {
    set_last_cuda_error(e, where);
    (void)cudaGetLastError();  // clear a non-sticky error so the next call starts clean
    return CLADA_ERR_CUDA;
}

int validate_layer(const clada_layer *layer, bool need_norm) {
    if (!layer || !layer->w_gate || !layer->w_down_t) return CLADA_ERR_NULL;
    if (layer->activation < CLADA_ACT_SILU_GATED || layer->activation > CLADA_ACT_RELU) return CLADA_ERR_UNSUPPORTED;
    const bool gated = layer->activation != CLADA_ACT_RELU;
    if (gated && !layer->w_up) return CLADA_ERR_NULL;
    if (need_norm && !layer->w_down_norm) return CLADA_ERR_NULL;
    if (!dtype_ok(layer->dtype)) return CLADA_ERR_DTYPE;
    if (layer->d_model <= 0 || layer->d_ff <= 0 || layer->d_model % 8 != 0) return CLADA_ERR_SHAPE;
    const int max_d = layer->dtype == CLADA_F32 ? kMaxDModel / 2 : kMaxDModel;
    if (layer->d_model > max_d) return CLADA_ERR_UNSUPPORTED;
    if (!aligned16(layer->w_gate) || (gated && !aligned16(layer->w_up)) || !aligned16(layer->w_down_t))
        return CLADA_ERR_ALIGN;
    return CLADA_OK;
}

int device_info(DeviceInfo *out) {
    constexpr int kMaxDev = 64;
    static DeviceInfo cache[kMaxDev];
    static bool have[kMaxDev] = {};
    int dev = 0;
    CLADA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev >= 0 && dev < kMaxDev && have[dev]) {
        *out = cache[dev];
        return CLADA_OK;
    }
    DeviceInfo di;
    di.device = dev;
    CLADA_CUDA_TRY(cudaDeviceGetAttribute(&di.num_sms, cudaDevAttrMultiProcessorCount, dev));
    CLADA_CUDA_TRY(cudaDeviceGetAttribute(&di.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (dev >= 0 && dev < kMaxDev) {
        cache[dev] = di;
        have[dev] = true;
    }
    *out = di;
    return CLADA_OK;
}

// Row norms of w_down_t: one warp per row, 16-byte loads, fp32 accumulation.
template <typename T>
__global__ void down_norms_kernel(const T *__restrict__ w, int d_model, int d_ff, float *__restrict__ out) {
    constexpr int E = Elem<T>::kPerVec;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) / kWarp;
    const int lane = threadIdx.x % kWarp;
    if (warp >= d_ff) return;
    const uint4 *row = reinterpret_cast<const uint4 *>(w + (size_t)warp * d_model);
    const int nvec = d_model / E;
    float acc = 0.f;
    for (int v = lane; v < nvec; v += kWarp) {
        float f[E];
        Elem<T>::unpack(ldg_stream(row + v), f);
#pragma unroll
        for (int i = 0; i < E; ++i) acc = fmaf(f[i], f[i], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) out[warp] = sqrtf(acc);
}

}  // namespace clada

using namespace clada;

namespace clada {
// Measuring aid: read a buffer once with the decode kernel's kind of load (16 bytes per thread, no L1
// allocation), eight loads in flight per thread, and fold it into one word per CTA so that nothing is
// optimised away.  Gives the read-only streaming bandwidth the sparse FFN's rows could at best arrive at.
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4 *__restrict__ buf, size_t n_vec,
                                                          uint32_t *__restrict__ sink) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    uint32_t acc = 0;
    size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; v + 7 * stride < n_vec; v += 8 * stride) {
        uint4 q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) q[u] = ldg_stream(buf + v + u * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc ^= q[u].x ^ q[u].y ^ q[u].z ^ q[u].w;
    }
    for (; v < n_vec; v += stride) {
        const uint4 q = ldg_stream(buf + v);
        acc ^= q.x ^ q.y ^ q.z ^ q.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) atomicXor(sink, acc);
}
}  // namespace clada

extern "C" {

int clada_version(void) { return 100; }

const char *clada_status_string(int code) {
    switch (code) {
        case CLADA_OK: return "ok";
        case CLADA_ERR_NULL: return "a required pointer is NULL";
        case CLADA_ERR_SHAPE: return "invalid size or shape";
        case CLADA_ERR_ALIGN: return "pointer not 16-byte aligned";
        case CLADA_ERR_DTYPE: return "unknown or unsupported dtype";
        case CLADA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CLADA_ERR_CUDA: return "CUDA runtime error (see clada_last_cuda_error)";
        case CLADA_ERR_UNSUPPORTED: return "size, element type or option beyond what the kernels support";
        default: return "unknown status";
    }
}

const char *clada_last_cuda_error(void) { return g_last_error; }

size_t clada_workspace_bytes(const clada_layer *layer, int32_t B, int64_t T_total) {
    if (!layer || B <= 0 || T_total < 0 || layer->d_model <= 0 || layer->d_ff <= 0) return 0;
    DeviceInfo di;
    int sms = 148;
    if (device_info(&di) == CLADA_OK) sms = di.num_sms;
    // decode: at most four fp32 partial output rows per persistent CTA (a tile of 4 sequences; two consumer groups
    // in two buffers for the stack launch), then the keep words of the batch (4 bytes per sequence and 32 neurons)
    size_t decode = (size_t)sms * 4 * (size_t)layer->d_model * sizeof(float) +
                    ((((size_t)B * ((size_t)(layer->d_ff + 31) / 32) * sizeof(unsigned)) + 255) & ~(size_t)255);
    // one sequence through a stack of layers: the keep words of up to 128 layers behind the partial rows
    decode = std::max(decode, (size_t)sms * 4 * (size_t)layer->d_model * sizeof(float) + keep_words_bytes(128, layer->d_ff));
    // a dense pass over the layer for 3-16 sequences: a partial output per group of CTAs and the groups' hidden activations
    if (B >= kDenseMinSeqs) {
        const size_t dense = ffn_batch_dense_scratch_bytes(layer, B < kDenseMaxSeqs ? B : kDenseMaxSeqs);
        // sequences past a multiple of 16 may still run as tiles, whose keep words sit behind the launch scratch
        decode = std::max(decode, dense + ((((size_t)B * ((size_t)(layer->d_ff + 31) / 32) * sizeof(unsigned)) + 255) & ~(size_t)255));
    }
    // prefix: one fp32 partial sum of squares per (token tile, neuron); tiles hold 64 tokens
    size_t tiles = (size_t)(T_total / 64) + (size_t)B + 1;
    size_t prefix = (tiles * (size_t)layer->d_ff * sizeof(float) + 255) & ~(size_t)255;
    // guard band: candidate list (int32 pairs) per (sequence, neuron), worst case all of them
    // plus its counter (256 bytes) and up to 512 split partial sums (two doubles each)
    size_t refine = (size_t)B * (size_t)layer->d_ff * 2 * sizeof(int32_t) + 256 + 512 * 16;
    size_t scratch = decode > prefix + refine ? decode : prefix + refine;
    // dense prefill down projection of a short prompt: the fp32 partial outputs of its K splits
    if (layer->dtype != CLADA_F32) scratch = std::max(scratch, down_split_scratch_bytes(layer, T_total, sms));
    return kWsCtrlBytes + ((scratch + 255) & ~(size_t)255);
}

int clada_workspace_init(void *ws, size_t ws_bytes, void *stream) {
    if (!ws) return CLADA_ERR_NULL;
    if (ws_bytes < kWsCtrlBytes || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    CLADA_CUDA_TRY(cudaMemsetAsync(ws, 0, kWsCtrlBytes, static_cast<cudaStream_t>(stream)));
    return CLADA_OK;
}

int clada_down_norms(const clada_layer *layer, float *out, void *stream) {
    CLADA_RANGE("clada_down_norms");
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!out) return CLADA_ERR_NULL;
    const int threads = 256;
    const int blocks = (layer->d_ff + threads / kWarp - 1) / (threads / kWarp);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (layer->dtype == CLADA_F32)
        down_norms_kernel<float><<<blocks, threads, 0, st>>>(
            static_cast<const float *>(layer->w_down_t), layer->d_model, layer->d_ff, out);
    else if (layer->dtype == CLADA_BF16)
        down_norms_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(layer->w_down_t), layer->d_model, layer->d_ff, out);
    else
        down_norms_kernel<__half><<<blocks, threads, 0, st>>>(
            static_cast<const __half *>(layer->w_down_t), layer->d_model, layer->d_ff, out);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

int clada_stream_read_probe(const void *buf, size_t bytes, uint32_t *sink, void *stream) {
    if (!buf || !sink) return CLADA_ERR_NULL;
    if (bytes < 16 || !aligned16(buf)) return CLADA_ERR_ALIGN;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    stream_read_kernel<<<di.num_sms * 4, 512, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(buf), bytes / 16, sink);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

}  // extern "C"
