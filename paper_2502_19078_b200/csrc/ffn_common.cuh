// Device primitives shared by the single-sequence and the batched sparse-FFN decode kernels:
// bounded grid barrier, bounded mbarrier waits, bulk row copies with L2 policies, packed-pair unpacking.
#pragma once

#include "common.cuh"

namespace clada {

constexpr unsigned kBarrierSpinLimit = 1u << 22;  // polls of an L2 word: gives up after ~1 s at most

// Bounded grid-wide barrier on two self-resetting counters in the workspace control block.
// Returns false if the wait expired.  Thread 0 arrives and polls; the departure count (whose last
// increment resets both counters for the next launch) is another round trip to L2 that nothing waits
// for, so a thread of the otherwise idle producer warp takes it after the CTA has been released.
static __device__ bool grid_barrier(WsCtrl *ctrl, unsigned n_ctas, int depart_tid,
                                    unsigned spin_limit = kBarrierSpinLimit) {
    __shared__ int s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&ctrl->arrive, 1u);
        unsigned spins = 0, seen;
        int ok = 1;
        for (;;) {
            asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(seen) : "l"(&ctrl->arrive) : "memory");
            if (seen >= n_ctas) break;
            if (++spins > spin_limit) {
                ok = 0;
                break;
            }
        }
        s_ok = ok;
    }
    __syncthreads();
    const bool ok = s_ok != 0;
    if ((int)threadIdx.x == depart_tid && ok) {
        const unsigned left = atomicAdd(&ctrl->depart, 1u);
        if (left == n_ctas - 1) {  // last one out: everyone has seen arrive == n_ctas
            ctrl->arrive = 0;
            ctrl->depart = 0;
            __threadfence();
        }
    }
    return ok;
}

// ---- mbarrier / bulk-copy primitives (bounded waits) -------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(1000u)  // suspend for at most ~1 us per try
        : "memory");
    return ok != 0;
}
constexpr unsigned kMbarSpinLimit = 1u << 20;  // tries of at most ~1 us each: about a second
// Waits for the phase with the given parity; gives up (returns false) after `limit` tries.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned limit = kMbarSpinLimit) {
    for (unsigned i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Bulk copies move one contiguous row, global -> this CTA's shared memory, completion counted on an
// mbarrier; both addresses are 16-byte aligned and the size is a multiple of 16.
// L2 policies: weights are read once (evict first), the small per-call vectors are re-read by every
// CTA and by the next call (evict last), so the streaming rows do not push them out of L2.
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_load_row_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar,
                                                   uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ float ld_keep(const float *p, uint64_t policy) {
    float v;
    asm volatile("ld.global.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(v) : "l"(p), "l"(policy));
    return v;
}
__device__ __forceinline__ float4 ld_keep4(const float4 *p, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// A 16-byte vector as E/2 pairs of fp32 (exact), ready for the packed two-wide FMA.
template <typename T> struct Pairs;
template <> struct Pairs<float> {
    static constexpr int kPairs = 2;
    __device__ static __forceinline__ void unpack(const uint4 &v, float2 (&f)[2]) {
        f[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
        f[1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
};
template <> struct Pairs<__nv_bfloat16> {
    static constexpr int kPairs = 4;
    __device__ static __forceinline__ void unpack(const uint4 &v, float2 (&f)[4]) {
        f[0] = make_float2(bf16_lo(v.x), bf16_hi(v.x));
        f[1] = make_float2(bf16_lo(v.y), bf16_hi(v.y));
        f[2] = make_float2(bf16_lo(v.z), bf16_hi(v.z));
        f[3] = make_float2(bf16_lo(v.w), bf16_hi(v.w));
    }
};

template <> struct Pairs<__half> {
    static constexpr int kPairs = 4;
    __device__ static __forceinline__ void unpack(const uint4 &v, float2 (&f)[4]) {
        f[0] = half2_bits_to_float2(v.x);
        f[1] = half2_bits_to_float2(v.y);
        f[2] = half2_bits_to_float2(v.z);
        f[3] = half2_bits_to_float2(v.w);
    }
};

constexpr int kConsumers = 512;               // consumer threads (16 warps)
constexpr int kConsWarps = kConsumers / kWarp;
constexpr int kFfnThreads = kConsumers + 32;  // + one producer warp
constexpr int kFfnWarps = kFfnThreads / kWarp;
constexpr int kMaxStages = 16;

// Batched decode (clada_ffn_batch.cu): how many sequences the next launch should take (4, 2 or 1 = use
// the single-sequence kernel), and the launch itself for a tile of 2 or 4 sequences.
int ffn_batch_tile(const clada_layer *layer, int remaining);
int launch_ffn_batch(const clada_layer *layer, int bt, const void *x, const float *scores, const float *tau,
                     long long tau_stride, void *y, int y_dtype, void *ws, int32_t *status, cudaStream_t st);

// One sequence through a stack of layers in one persistent launch (clada_ffn_stack.cu): whether the stack
// kernel takes this call (one sequence, at least two layers of one FFN form, a workspace with two partial
// rows per SM), and the launch (x / y strides in bytes, tau stride in elements).
bool ffn_stack_supported(const clada_layer *layers, int L, int B, size_t ws_bytes);
int launch_ffn_stack(const clada_layer *layers, int L, const void *x, size_t x_stride, const float *scores,
                     const float *tau, long long tau_stride, void *y, size_t y_stride, int y_dtype, void *ws,
                     int32_t *status, cudaStream_t st);

}  // namespace clada
