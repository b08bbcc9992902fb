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
#ifndef CLADA_MBAR_SUSPEND_NS
#define CLADA_MBAR_SUSPEND_NS 1000
#endif
constexpr unsigned kMbarSuspendNs = CLADA_MBAR_SUSPEND_NS;  // a try may suspend the thread for about this long
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kMbarSuspendNs)
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
// A neuron index on its way into a row address.  The lists the kernels build hold indices below d_ff by
// construction, so the release build passes them through; a -DCLADA_DEBUG_BOUNDS build checks every one, records
// CLADA_STATUS_BAD_INDEX in the call's status word and reads row 0 instead (never a trap, never a skipped copy:
// the stage's byte count stays what its barrier expects).
__device__ __forceinline__ int guard_row(int j, int d_ff, int32_t *status) {
#ifdef CLADA_DEBUG_BOUNDS
    if ((unsigned)j >= (unsigned)d_ff) {
        if (status) atomicOr(status, CLADA_STATUS_BAD_INDEX);
        return 0;
    }
#endif
    return j;
}
// A slot of a list about to be written: always true in the release build; the checking build records an
// out-of-range slot and the caller skips the store.
__device__ __forceinline__ bool guard_slot(int i, int n, int32_t *status) {
#ifdef CLADA_DEBUG_BOUNDS
    if ((unsigned)i >= (unsigned)n) {
        if (status) atomicOr(status, CLADA_STATUS_BAD_INDEX);
        return false;
    }
#endif
    return true;
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

// ---- the consumers' loop over one share of kept neurons (single-sequence kernels) -----------------------
//
// The 512 consumer threads work as GROUPS groups of GT = 512 / GROUPS threads.  A group owns every GROUPS-th
// chunk of GS = 4 consecutive neurons of the share; within a group thread gt owns the 16-byte column vectors
// gt, gt + GT, ... of every row (x and the partial y of those columns stay in registers).  Per chunk: the gate
// and up dot products of its four neurons from the staged rows (packed two-wide FMAs), ONE group-wide reduction
// of the eight values (halving butterfly in the warp, then across the group's warps through shared memory, fixed
// order), the neuron values, and the four down rows scaled into the partial y.  (Without a gate projection and with
// one vector per thread a chunk is EIGHT neurons: the eight values are their gate sums.)  With two groups one group's
// reduction latency hides under the other's arithmetic, and a row of at most 256 vectors keeps every thread busy.
// A group never reads the other group's stages, but it watches each of them land before it moves past.
// A stage is handed back by the warps of the group that owns its neuron (kConsWarps / GROUPS arrivals per stage;
// a group needs GS <= n_stages stages at once, which the launch checks).
constexpr int GS = 4;  // neurons per group-wide reduction

__device__ __forceinline__ void group_sync(int grp, int n_threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(4 + grp), "r"(n_threads) : "memory");  // named barriers 4, 5
}

template <typename T, int NV, bool GATED, int GROUPS>
__device__ __forceinline__ void consume_share(const int my_n, const int act, const uint32_t ring,
                                              const uint32_t stage_bytes, const uint32_t row_bytes,
                                              const uint32_t down_off, const uint32_t full0, const uint32_t empty0,
                                              const int n_stages, int &cs, uint32_t &cpar,
                                              const float2 (&xr)[NV][Pairs<T>::kPairs], const bool (&vok)[NV],
                                              float2 (&acc)[NV][Pairs<T>::kPairs], float *s_dot, bool &timed_out,
                                              unsigned long long *waited_ns = nullptr) {
    constexpr int P = Pairs<T>::kPairs;
    constexpr int GT = kConsumers / GROUPS;  // threads per group
    constexpr int GW = GT / kWarp;           // warps per group
    constexpr int PER = GW / 4;              // warps each lane adds in the cross-warp sum (4 lanes per value)
    static_assert(GROUPS == 1 || GROUPS == 2, "one or two consumer groups");
    // Neurons per chunk (= per group-wide reduction of eight values): four with a gate and an up value each, or,
    // without a gate projection, eight when a row is one vector per thread (the ring then holds twelve stages or
    // more): rows that narrow are bound by the reduction's latency, not by their bytes.
    constexpr int NPC = (!GATED && NV == 1) ? 2 * GS : GS;
    const int tid = threadIdx.x, lane = tid & 31;
    const int grp = tid / GT, gt = tid - grp * GT, gw = gt >> 5;
    float(*dot)[2 * GS][GW] = reinterpret_cast<float(*)[2 * GS][GW]>(s_dot + (size_t)grp * 2 * 2 * GS * GW);
    const bool b16 = lane & 16, b8 = lane & 8, b4 = lane & 4;
    int buf = 0;
    for (int g0 = 0, chunk = 0; g0 < my_n; g0 += NPC, ++chunk) {
        if (GROUPS > 1 && (chunk & (GROUPS - 1)) != grp) {
            // The other group's chunk.  Its stages are not read here and not handed back from here, but each
            // one's copy is seen to land: bulk copies may complete out of order, and a wait by parity for the
            // NEXT use of a stage would pass at once if this use had not even completed yet.
#pragma unroll
            for (int g = 0; g < NPC; ++g) {
                if (g0 + g >= my_n) break;
                if (!timed_out && !mbar_wait(full0 + 8 * cs, cpar)) timed_out = true;
                if (++cs == n_stages) {
                    cs = 0;
                    cpar ^= 1;
                }
            }
            continue;
        }
        float pd[2 * GS];
        uint32_t st_addr[NPC];
        int st_idx[NPC];
#pragma unroll
        for (int g = 0; g < NPC; ++g) {
            const int i = g0 + g;
            float2 sg = make_float2(0.f, 0.f), su = make_float2(0.f, 0.f);
            st_idx[g] = cs;
            st_addr[g] = ring + (uint32_t)cs * stage_bytes;
            if (i < my_n) {
#ifdef CLADA_STACK_TRACE
                unsigned long long w0 = 0;
                if (waited_ns) asm volatile("mov.u64 %0, %globaltimer;" : "=l"(w0));
#endif
                if (!timed_out && !mbar_wait(full0 + 8 * cs, cpar)) timed_out = true;
#ifdef CLADA_STACK_TRACE
                if (waited_ns) {
                    unsigned long long w1;
                    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(w1));
                    *waited_ns += w1 - w0;
                }
#endif
                if (++cs == n_stages) {
                    cs = 0;
                    cpar ^= 1;
                }
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    if (!vok[k]) continue;
                    const uint32_t a = st_addr[g] + (uint32_t)(gt + k * GT) * 16u;
                    float2 fg[P], fu[P];
                    Pairs<T>::unpack(lds128(a), fg);
                    if (GATED) Pairs<T>::unpack(lds128(a + row_bytes), fu);
#pragma unroll
                    for (int e = 0; e < P; ++e) {
                        sg = __ffma2_rn(fg[e], xr[k][e], sg);
                        if (GATED) su = __ffma2_rn(fu[e], xr[k][e], su);
                    }
                }
            }
            if (NPC == GS) {
                pd[2 * g] = sg.x + sg.y;
                pd[2 * g + 1] = su.x + su.y;
            } else {
                pd[g] = sg.x + sg.y;  // no up values: the eight slots hold eight neurons' gate sums
            }
        }
        // Warp sums of the 8 values by a halving butterfly (9 shuffles): after it every lane of
        // quad q holds the warp total of value q.  Fixed order, so results repeat bit for bit.
        float b[4], c[2], v8;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float send = b16 ? pd[i] : pd[i + 4];
            b[i] = (b16 ? pd[i + 4] : pd[i]) + __shfl_xor_sync(0xffffffffu, send, 16);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float send = b8 ? b[i] : b[i + 2];
            c[i] = (b8 ? b[i + 2] : b[i]) + __shfl_xor_sync(0xffffffffu, send, 8);
        }
        v8 = (b4 ? c[1] : c[0]) + __shfl_xor_sync(0xffffffffu, b4 ? c[0] : c[1], 4);
        v8 += __shfl_xor_sync(0xffffffffu, v8, 2);
        v8 += __shfl_xor_sync(0xffffffffu, v8, 1);
        // lane 4q holds value index: bit4 -> +4, bit3 -> +2, bit2 -> +1
        if ((lane & 3) == 0) dot[buf][(b16 ? 4 : 0) + (b8 ? 2 : 0) + (b4 ? 1 : 0)][gw] = v8;
        if (GROUPS == 1)
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
        else
            group_sync(grp, GT);
        // Cross-warp sums: lane l adds PER consecutive warps of value l/4 (4 lanes per value), the quad
        // finishes by butterfly; then gate lanes form the neuron value h.
        float tot;
        if (PER == 4) {
            const float4 q4 = *reinterpret_cast<const float4 *>(&dot[buf][lane >> 2][(lane & 3) * 4]);
            tot = (q4.x + q4.y) + (q4.z + q4.w);
        } else {
            const float2 q2 = *reinterpret_cast<const float2 *>(&dot[buf][lane >> 2][(lane & 3) * 2]);
            tot = q2.x + q2.y;
        }
        tot += __shfl_xor_sync(0xffffffffu, tot, 1);
        tot += __shfl_xor_sync(0xffffffffu, tot, 2);
        const float up = __shfl_xor_sync(0xffffffffu, tot, 4);  // value 2g+1 sits 4 lanes above value 2g
        const float hval = neuron_value_f(act, tot, up);        // meaningful on lanes 8g..8g+3 (4g..4g+3 without up values)
#pragma unroll
        for (int g = 0; g < NPC; ++g) {
            const float h = __shfl_sync(0xffffffffu, hval, (NPC == GS ? 8 : 4) * g);
            if (g0 + g >= my_n) continue;
            const float2 h2 = make_float2(h, h);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                if (!vok[k]) continue;
                float2 fd[P];
                Pairs<T>::unpack(lds128(st_addr[g] + down_off + (uint32_t)(gt + k * GT) * 16u), fd);
#pragma unroll
                for (int e = 0; e < P; ++e) acc[k][e] = __ffma2_rn(h2, fd[e], acc[k][e]);
            }
        }
        // hand the stages back to the producer
        __syncwarp();
        if (lane == 0) {
#pragma unroll
            for (int g = 0; g < NPC; ++g)
                if (g0 + g < my_n) mbar_arrive(empty0 + 8 * st_idx[g]);
        }
        buf ^= 1;
    }
}

// Shared-memory floats consume_share needs for its cross-warp sums (all groups, two buffers each).
constexpr int kDotFloats = 2 * 2 * GS * kConsWarps;

// Consumer groups for a row of vpr 16-byte vectors: two groups of 256 threads when a group covers the row with one
// vector per thread (otherwise half the 512 threads would own nothing), else one group of 512.  Measured: with two
// vectors per thread in two groups (rows of 257-512 vectors) a group holds its four stages twice as long and the
// 4096-wide layers lose 6 % against one group; at 256 vectors two groups gain 9-13 %.
__host__ __device__ inline int ffn_groups(int vpr) { return vpr <= kConsumers / 2 ? 2 : 1; }

// Batched decode (clada_ffn_batch.cu): how many sequences the next launch should take (4, 2 or 1 = use
// the single-sequence kernel), and the launch itself for a tile of 2 or 4 sequences.
int ffn_batch_tile(const clada_layer *layer, int remaining);
int launch_ffn_batch(const clada_layer *layer, int bt, const void *x, const float *scores, const float *tau,
                     long long tau_stride, void *y, int y_dtype, void *ws, const unsigned *keep_words,
                     int32_t *status, cudaStream_t st);
// Keep bits of a whole batch for the tile launches (clada_ffn_batch.cu): the kernel's launch and the bytes of
// workspace its output takes (a multiple of 256).
int launch_keep_words(const float *scores, int B, int d_ff, const float *tau, long long tau_stride, unsigned *words,
                      cudaStream_t st);
size_t keep_words_bytes_of(int B, int d_ff);

// One sequence through a stack of layers in one persistent launch (clada_ffn_stack.cu): whether the stack
// kernel takes this call (one sequence, at least two layers of one FFN form, a workspace with two partial
// rows per SM), and the launch (x / y strides in bytes, tau stride in elements).
bool ffn_stack_supported(const clada_layer *layers, int L, int B, size_t ws_bytes);
int launch_ffn_stack(const clada_layer *layers, int L, const void *x, size_t x_stride, const float *scores,
                     const float *tau, long long tau_stride, void *y, size_t y_stride, int y_dtype, void *ws,
                     size_t ws_bytes, int32_t *status, cudaStream_t st);

}  // namespace clada
