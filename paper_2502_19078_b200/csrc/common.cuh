// Shared host/device helpers of the CLADA CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "clada.h"

namespace clada {

constexpr int kWarp = 32;
constexpr int kMaxDModel = 8192;

// ---- host-side error plumbing -------------------------------------------------------------
void set_last_cuda_error(cudaError_t e, const char *where);
int cuda_fail(cudaError_t e, const char *where);  // records and returns CLADA_ERR_CUDA

#define CLADA_CUDA_TRY(expr)                                           \
    do {                                                               \
        cudaError_t e__ = (expr);                                      \
        if (e__ != cudaSuccess) return ::clada::cuda_fail(e__, #expr); \
    } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elem_size(int dtype) { return dtype == CLADA_F32 ? 4 : 2; }
inline bool dtype_ok(int dtype) { return dtype == CLADA_F32 || dtype == CLADA_BF16 || dtype == CLADA_F16; }
int validate_layer(const clada_layer *layer, bool need_norm);

struct DeviceInfo {
    int device;
    int num_sms;
    int max_smem_optin;
};
// Properties of the current device (cached per device).
int device_info(DeviceInfo *out);

// ---- workspace layout ---------------------------------------------------------------------
// [0, 256)            control words (grid-barrier counters), zeroed by clada_workspace_init
// [256, ...)          per-call scratch
constexpr size_t kWsCtrlBytes = 256;
struct WsCtrl {
    unsigned int arrive;  // grid barrier: CTAs that reached it
    unsigned int depart;  // CTAs that left it; the last one resets both
};

// ---- device helpers -----------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// 16-byte read-only global load that does not allocate in L1 (weights are streamed once).
__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// The two bf16 halves of a 32-bit word as fp32 (exact).
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;  // elements per 16-byte vector
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float to_float(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[8]) {
        f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
        f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
    }
    __device__ static __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
};
__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t w) {
    return __half22float2(*reinterpret_cast<const __half2 *>(&w));
}
template <> struct Elem<__half> {
    static constexpr int kPerVec = 8;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[8]) {
        const float2 a = half2_bits_to_float2(v.x), b = half2_bits_to_float2(v.y), c = half2_bits_to_float2(v.z),
                     d = half2_bits_to_float2(v.w);
        f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
    }
    __device__ static __forceinline__ float to_float(__half v) { return __half2float(v); }
};

// Four fp32 values as four 16-bit elements of the given clada_dtype (round to nearest even).
__device__ __forceinline__ uint2 pack4_16bit(int dtype, float4 s) {
    uint2 o;
    if (dtype == CLADA_BF16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(s.x, s.y), hi = __floats2bfloat162_rn(s.z, s.w);
        o.x = *reinterpret_cast<uint32_t *>(&lo);
        o.y = *reinterpret_cast<uint32_t *>(&hi);
    } else {
        __half2 lo = __floats2half2_rn(s.x, s.y), hi = __floats2half2_rn(s.z, s.w);
        o.x = *reinterpret_cast<uint32_t *>(&lo);
        o.y = *reinterpret_cast<uint32_t *>(&hi);
    }
    return o;
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start
// while its predecessor in the stream drains; it must not touch global memory the predecessor may
// write before pdl_wait() returns (the predecessor has then completed and flushed).  Both are
// no-ops for a plain launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// silu(g) = g / (1 + exp(-g)); expf keeps full fp32 accuracy.
__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + expf(-g)); }

// tanh form of GELU: 0.5 g (1 + tanh(sqrt(2/pi) (g + 0.044715 g^3))).
__device__ __forceinline__ float gelu_tanh_f(float g) {
    const float inner = 0.7978845608028654f * (g + 0.044715f * g * g * g);
    return 0.5f * g * (1.0f + tanhf(inner));
}

// Value of one neuron for one token from g = w_gate_j . x and u = w_up_j . x in the layer's FFN form
// (Eq. neuron_activation with the family's sigma; the non-gated form has no u factor).
__device__ __forceinline__ float neuron_value_f(int act, float g, float u) {
    if (act == CLADA_ACT_GELU_GATED) return gelu_tanh_f(g) * u;
    if (act == CLADA_ACT_RELU) return g > 0.f ? g : 0.f;
    return silu_f(g) * u;
}

__device__ __forceinline__ double neuron_value_d(int act, double g, double u) {
    if (act == CLADA_ACT_GELU_GATED) {
        const double inner = 0.79788456080286535588 * (g + 0.044715 * g * g * g);
        return 0.5 * g * (1.0 + tanh(inner)) * u;
    }
    if (act == CLADA_ACT_RELU) return g > 0.0 ? g : 0.0;
    return g / (1.0 + exp(-g)) * u;
}

__host__ __device__ __forceinline__ bool act_is_gated(int act) { return act != CLADA_ACT_RELU; }

#endif  // __CUDACC__

}  // namespace clada
