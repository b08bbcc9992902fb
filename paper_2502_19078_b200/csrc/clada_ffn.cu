// Sparse gated FFN for one decode token per sequence (Algorithm 2, generation phase):
//   kept = { j : A_j >= tau_final },  y = sum_{j in kept} silu(w_gate_j . x) (w_up_j . x) w_down_t[j,:]
//
// One persistent cooperative kernel per (layer, sequence):
//   prologue  every CTA scans the F scores against tau (batched loads, warp ballots), learns the number of kept
//             neurons and takes an equal share [r0, r1) of the kept list in ascending order;
//   stream    a producer thread copies the three contiguous rows of each kept neuron into a ring of
//             shared-memory stages with bulk asynchronous copies (mbarrier-tracked), which keeps
//             ~200 KB of HBM requests in flight per SM whatever the consumers are doing.  Consumer
//             thread t owns the same 16-byte column vectors of every row (x and the partial y for
//             those columns live in registers) and reads the staged rows from shared memory;
//   epilogue  each CTA stores its fp32 partial y, all CTAs meet at a bounded grid barrier, then every
//             CTA sums a slice of columns over all partials in CTA order (deterministic) and writes y.
#include <math.h>

#include "common.cuh"

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
    float *partials;      // [gridDim.x, d_model]
    WsCtrl *ctrl;
    int32_t *status;
    int d_model, d_ff;
};

constexpr unsigned kBarrierSpinLimit = 1u << 20;  // polls ~100 ns apart: gives up after ~0.1 s

// Bounded grid-wide barrier on two self-resetting counters in the workspace control block.
// Returns false if the wait expired.
__device__ bool grid_barrier(WsCtrl *ctrl, unsigned n_ctas) {
    __shared__ int s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&ctrl->arrive, 1u);
        unsigned spins = 0;
        int ok = 1;
        while (*reinterpret_cast<volatile unsigned *>(&ctrl->arrive) < n_ctas) {
            if (++spins > kBarrierSpinLimit) {
                ok = 0;
                break;
            }
            __nanosleep(64);
        }
        __threadfence();
        s_ok = ok;
        if (ok) {
            const unsigned left = atomicAdd(&ctrl->depart, 1u);
            if (left == n_ctas - 1) {  // last one out: everyone has seen arrive == n_ctas
                ctrl->arrive = 0;
                ctrl->depart = 0;
                __threadfence();
            }
        }
    }
    __syncthreads();
    return s_ok != 0;
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
constexpr unsigned kMbarSpinLimit = 1u << 22;  // each failed try_wait already sleeps in hardware
// Waits for the phase with the given parity; gives up (returns false) after kMbarSpinLimit tries.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (unsigned i = 0; i < kMbarSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// One contiguous row, global -> this CTA's shared memory, completion counted on an mbarrier.
// Both addresses are 16-byte aligned and bytes is a multiple of 16.
__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

constexpr int kConsumers = 256;              // consumer threads (8 warps)
constexpr int kFfnThreads = kConsumers + 32;  // + one producer warp
constexpr int kMaxStages = 16;

// One CTA per SM.  Warp 8 lane 0 streams the three rows of each kept neuron of this CTA's share into
// a ring of shared-memory stages with bulk async copies (one stage = gate row | up row | down row);
// the 8 consumer warps take stages G at a time: dot products from shared memory against x in
// registers, CTA-wide sum, silu * up, then the down row is added into the register-resident partial y.
template <typename T, int NV, int G>
__global__ void __launch_bounds__(kFfnThreads, 1)
sparse_ffn_kernel(const FfnParams p, const int n_stages) {
    constexpr int E = Elem<T>::kPerVec;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nwarps = kFfnThreads / kWarp;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff, d = p.d_model;
    const int vpr = d / E;                       // 16-byte vectors per row
    const uint32_t row_bytes = (uint32_t)vpr * 16u;
    const uint32_t stage_bytes = 3u * row_bytes;

    // dynamic shared memory: ring | full[kMaxStages] | empty[kMaxStages] | kept list
    const uint32_t ring = smem_u32(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)n_stages * stage_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages);
    unsigned *s_bal = reinterpret_cast<unsigned *>(bars + 2 * kMaxStages);  // one ballot word per chunk
    int *s_list = reinterpret_cast<int *>(s_bal + (F + kWarp - 1) / kWarp);
    __shared__ int s_wtot[nwarps];
    __shared__ float s_dot[2][kConsumers / kWarp][2 * G];

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full0 + 8 * s, 1);                      // the producer's expect_tx arrival
            mbar_init(empty0 + 8 * s, kConsumers / kWarp);    // one arrival per consumer warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    // ---- prologue: threshold test and this CTA's share of the kept list -------------------------
    // Pass 1 reads the scores in batches of independent loads (one memory round trip per batch, not
    // per chunk) and leaves one ballot word per 32-neuron chunk in shared memory; pass 2 ranks from
    // those words without touching global memory again.
    const float tau = *p.tau;
    const int chunks = (F + kWarp - 1) / kWarp;
    const int per_warp = (chunks + nwarps - 1) / nwarps;
    const int c0 = warp * per_warp, c1 = min(chunks, c0 + per_warp);
    int n = 0;
    constexpr int kBatch = 16;
    for (int c = c0; c < c1; c += kBatch) {
        float v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = (c + u) * kWarp + lane;
            v[u] = (c + u < c1 && j < F) ? __ldg(p.scores + j) : -INFINITY;
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (c + u < c1) {  // warp-uniform
                const int j = (c + u) * kWarp + lane;
                const unsigned bal = __ballot_sync(0xffffffffu, j < F && v[u] >= tau);
                if (lane == 0) s_bal[c + u] = bal;
                n += __popc(bal);
            }
        }
    }
    if (lane == 0) s_wtot[warp] = n;
    __syncthreads();
    int base = 0, n_act = 0;
#pragma unroll
    for (int w = 0; w < nwarps; ++w) {
        const int v = s_wtot[w];
        base += (w < warp) ? v : 0;
        n_act += v;
    }
    const int r0 = (int)(((int64_t)n_act * cta) / n_ctas);
    const int r1 = (int)(((int64_t)n_act * (cta + 1)) / n_ctas);
    const int m0 = (int)(((int64_t)F * cta) / n_ctas);  // slice of the mask this CTA writes
    const int m1 = (int)(((int64_t)F * (cta + 1)) / n_ctas);
    for (int c = c0; c < c1; ++c) {
        const int j = c * kWarp + lane;
        const unsigned bal = s_bal[c];
        const bool keep = (bal >> lane) & 1u;
        const int rank = base + __popc(bal & ((1u << lane) - 1u));
        if (keep && rank >= r0 && rank < r1) {
            s_list[rank - r0] = j;
            if (p.idx_out) p.idx_out[rank] = j;
        }
        if (p.mask_out && j >= m0 && j < m1) p.mask_out[j] = keep ? 1 : 0;
        base += __popc(bal);
    }
    if (p.count_out && cta == 0 && tid == 0) *p.count_out = n_act;
    const int my_n = r1 - r0;
    __syncthreads();  // s_list and the mbarriers are ready

    float acc[NV][E];
    bool timed_out = false;

    if (warp == kConsumers / kWarp) {
        // ---- producer ------------------------------------------------------------------------
        if (lane == 0) {
            const char *Wg = static_cast<const char *>(p.w_gate);
            const char *Wu = static_cast<const char *>(p.w_up);
            const char *Wd = static_cast<const char *>(p.w_down_t);
            int issued = 0;
            for (int i = 0; i < my_n; ++i) {
                const int s = i % n_stages, use = i / n_stages;
                if (!mbar_wait(empty0 + 8 * s, (use & 1) ^ 1)) {  // a fresh barrier passes parity 1 at once
                    timed_out = true;
                    break;
                }
                const size_t off = (size_t)s_list[i] * row_bytes;
                const uint32_t dst = ring + (uint32_t)s * stage_bytes, bar = full0 + 8 * s;
                mbar_expect_tx(bar, stage_bytes);
                bulk_load_row(dst, Wg + off, row_bytes, bar);
                bulk_load_row(dst + row_bytes, Wu + off, row_bytes, bar);
                bulk_load_row(dst + 2 * row_bytes, Wd + off, row_bytes, bar);
                issued = i + 1;
            }
            // Never leave with copies in flight: the last use of every stage must have landed.
            for (int i = max(0, issued - n_stages); i < issued; ++i)
                if (!mbar_wait(full0 + 8 * (i % n_stages), (i / n_stages) & 1)) timed_out = true;
        }
    } else {
        // ---- consumers -----------------------------------------------------------------------
        float xr[NV][E];
        bool vok[NV];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int v = tid + i * kConsumers;
            vok[i] = v < vpr;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (vok[i]) q = *(reinterpret_cast<const uint4 *>(p.x) + v);
            Elem<T>::unpack(q, xr[i]);
#pragma unroll
            for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
        }
        int buf = 0;
        for (int g0 = 0; g0 < my_n; g0 += G, buf ^= 1) {
            float pd[2 * G];
            uint32_t st_addr[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int i = g0 + g;
                float sg = 0.f, su = 0.f;
                st_addr[g] = ring + (uint32_t)(i % n_stages) * stage_bytes;
                if (i < my_n) {
                    if (!timed_out && !mbar_wait(full0 + 8 * (i % n_stages), (i / n_stages) & 1)) timed_out = true;
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        if (!vok[k]) continue;
                        const uint32_t a = st_addr[g] + (uint32_t)(tid + k * kConsumers) * 16u;
                        float fg[E], fu[E];
                        Elem<T>::unpack(lds128(a), fg);
                        Elem<T>::unpack(lds128(a + row_bytes), fu);
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            sg = fmaf(fg[e], xr[k][e], sg);
                            su = fmaf(fu[e], xr[k][e], su);
                        }
                    }
                }
                pd[2 * g] = sg;
                pd[2 * g + 1] = su;
            }
            // CTA-wide sums in a fixed order: lanes by butterfly, then warps 0..7
#pragma unroll
            for (int k = 0; k < 2 * G; ++k) pd[k] = warp_sum(pd[k]);
            if (lane == 0) {
#pragma unroll
                for (int k = 0; k < 2 * G; ++k) s_dot[buf][warp][k] = pd[k];
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
#pragma unroll
            for (int g = 0; g < G; ++g) {
                if (g0 + g >= my_n) continue;
                float sg = 0.f, su = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumers / kWarp; ++w) {
                    sg += s_dot[buf][w][2 * g];
                    su += s_dot[buf][w][2 * g + 1];
                }
                const float h = silu_f(sg) * su;
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    if (!vok[k]) continue;
                    float fd[E];
                    Elem<T>::unpack(lds128(st_addr[g] + 2 * row_bytes + (uint32_t)(tid + k * kConsumers) * 16u), fd);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[k][e] = fmaf(h, fd[e], acc[k][e]);
                }
            }
            // hand the stages back to the producer
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (g0 + g < my_n) mbar_arrive(empty0 + 8 * ((g0 + g) % n_stages));
            }
        }
        // partial y of this CTA
        float *mine = p.partials + (size_t)cta * d;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            if (!vok[i]) continue;
            float4 *dst = reinterpret_cast<float4 *>(mine + (size_t)(tid + i * kConsumers) * E);
#pragma unroll
            for (int e = 0; e < E; e += 4)
                dst[e / 4] = make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
        }
    }
    if (timed_out && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);

    // ---- epilogue: grid barrier, deterministic column reduction ---------------------------------
    if (!grid_barrier(p.ctrl, (unsigned)n_ctas)) {
        if (tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }
    // columns in groups of 4 (float4); a warp sums one group: lane l adds partial rows l, l+32, ...
    // in order, then the 32 lane sums combine by butterfly.
    const int ngroups = d / 4;
    for (int q = cta + warp * n_ctas; q < ngroups; q += n_ctas * nwarps) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 5
        for (int r = lane; r < n_ctas; r += kWarp) {
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(p.partials + (size_t)r * d) + q);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        s.x = warp_sum(s.x); s.y = warp_sum(s.y); s.z = warp_sum(s.z); s.w = warp_sum(s.w);
        if (lane == 0) {
            if (p.y_dtype == CLADA_F32) {
                reinterpret_cast<float4 *>(p.y)[q] = s;
            } else {
                __nv_bfloat162 lo = __floats2bfloat162_rn(s.x, s.y), hi = __floats2bfloat162_rn(s.z, s.w);
                uint2 o;
                o.x = *reinterpret_cast<uint32_t *>(&lo);
                o.y = *reinterpret_cast<uint32_t *>(&hi);
                reinterpret_cast<uint2 *>(p.y)[q] = o;
            }
        }
    }
}

// ---- host side ------------------------------------------------------------------------------

template <typename T, int NV, int G>
static int launch_variant(const FfnParams &p, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_kernel<T, NV, G>;
    const size_t stage_bytes = 3 * (size_t)(p.d_model / E) * 16;
    const size_t tail = 2 * kMaxStages * sizeof(uint64_t) + (size_t)((p.d_ff + 31) / 32) * sizeof(unsigned) +
                        (size_t)(p.d_ff / di.num_sms + 2) * sizeof(int);
    const size_t budget = (size_t)di.max_smem_optin - 1024;  // leave room for the static arrays
    if (budget < tail + 2 * G * stage_bytes) return CLADA_ERR_UNSUPPORTED;
    int n_stages = (int)((budget - tail) / stage_bytes);
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    const size_t smem = (size_t)n_stages * stage_bytes + tail;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, di.max_smem_optin - 1024));
        configured[di.device & 63] = true;
    }
    FfnParams params = p;
    int stages_arg = n_stages;
    void *args[] = {&params, &stages_arg};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(di.num_sms);  // one CTA per SM: co-resident by construction, checked by the launch
    cfg.blockDim = dim3(kFfnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident: the grid barrier cannot starve
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CLADA_CUDA_TRY(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kern), args));
    return CLADA_OK;
}

template <typename T>
static int launch_ffn(const FfnParams &p, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    const int vpr = p.d_model / E;
    if (vpr <= 256) return launch_variant<T, 1, 2>(p, st);
    if (vpr <= 512) return launch_variant<T, 2, 2>(p, st);
    if (vpr <= 768) return launch_variant<T, 3, 2>(p, st);
    if (vpr <= 1024) return launch_variant<T, 4, 2>(p, st);
    return CLADA_ERR_UNSUPPORTED;
}

}  // namespace clada

using namespace clada;

extern "C" int clada_sparse_ffn_decode(const clada_layer *layer, const void *x, int32_t B,
                                       const float *scores, const float *tau_final, int64_t tau_stride,
                                       void *y, int32_t y_dtype, uint8_t *mask_out, int32_t *idx_out,
                                       int32_t *count_out, void *ws, size_t ws_bytes, int32_t *status,
                                       void *stream) {
    int rc = validate_layer(layer, false);
    if (rc != CLADA_OK) return rc;
    if (!x || !scores || !tau_final || !y) return CLADA_ERR_NULL;
    if (B <= 0 || tau_stride < 0) return CLADA_ERR_SHAPE;
    if (y_dtype != CLADA_F32 && y_dtype != CLADA_BF16) return CLADA_ERR_DTYPE;
    if (!aligned16(x) || !aligned16(y)) return CLADA_ERR_ALIGN;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return CLADA_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    const size_t need = kWsCtrlBytes + (size_t)di.num_sms * layer->d_model * sizeof(float);
    if (ws_bytes < need) return CLADA_ERR_WORKSPACE;

    const size_t esz = elem_size(layer->dtype);
    const size_t ysz = elem_size(y_dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int b = 0; b < B; ++b) {
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
        rc = layer->dtype == CLADA_F32 ? launch_ffn<float>(p, st) : launch_ffn<__nv_bfloat16>(p, st);
        if (rc != CLADA_OK) return rc;
    }
    return CLADA_OK;
}
