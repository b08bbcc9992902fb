// Sparse gated FFN decode for a tile of BT sequences at once (per-sequence masks):
//   kept_b = { j : A_bj >= tau_b },   y_b = sum_{j in kept_b} silu(w_gate_j . x_b) (w_up_j . x_b) w_down_t[j,:]
//
// The rows of a neuron are read ONCE for the whole tile: the CTAs share out the UNION of the tile's kept
// sets, stream each union neuron's three rows through the same bulk-copy ring as the single-sequence
// kernel, and every consumer thread keeps x and the partial y of its columns for all BT sequences in
// registers.  A sequence that does not keep a neuron of the union gets h = 0 for it, so each y_b is
// exactly the sum over its own kept set.  16 dot products share one CTA-wide reduction (BT = 4: two
// neurons per reduction, BT = 2: four).  Partial outputs are reduced across CTAs in a fixed order.
#include <math.h>

#include "common.cuh"
#include "ffn_batch.cuh"
#include "ffn_common.cuh"

namespace clada {

template <typename T, int NV, int BT>
__global__ void __launch_bounds__(kFfnThreads, 1)
sparse_ffn_batch_kernel(const FfnBatchParams p, const int n_stages) {
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = Pairs<T>::kPairs;
    constexpr int GB = 8 / BT;  // neurons per CTA-wide reduction: 16 dot products each time
    static_assert(BT == 2 || BT == 4, "tile of 2 or 4 sequences");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff, d = p.d_model;
    const int vpr = d / E;
    const uint32_t row_bytes = (uint32_t)vpr * 16u;
    const bool gated = act_is_gated(p.act);
    const uint32_t n_rows = gated ? 3u : 2u;  // gate | up | down, or gate | down without a gate projection
    const uint32_t stage_bytes = n_rows * row_bytes;
    const uint32_t down_off = (n_rows - 1u) * row_bytes;
    const int chunks = (F + kWarp - 1) / kWarp;
    const int list_cap = F / n_ctas + 2;

    // dynamic shared memory: ring | full | empty | union keep-bits | per-sequence keep-bits | list | keep nibbles
    const uint32_t ring = smem_u32(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)n_stages * stage_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages);
    unsigned *s_bal = reinterpret_cast<unsigned *>(bars + 2 * kMaxStages);
    unsigned *s_balb = s_bal + chunks;                      // [BT][chunks]
    int *s_list = reinterpret_cast<int *>(s_balb + BT * chunks);
    int *s_keep = s_list + list_cap;                        // bit b: sequence b keeps this neuron
    __shared__ int s_wtot[kFfnWarps];
    __shared__ float s_tau[BT];
    __shared__ __align__(16) float s_dot[2][16][kConsWarps];

    pdl_launch_dependents();
    if (tid == kConsumers) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kConsWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();

    const uint64_t keep_policy = policy_evict_last();
    if (tid < BT) s_tau[tid] = ld_keep(p.tau + (size_t)tid * p.tau_stride, keep_policy);
    float2 xr[BT][NV][P];
    bool vok[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int v = tid + i * kConsumers;
        vok[i] = tid < kConsumers && v < vpr;
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            uint4 q = make_uint4(0, 0, 0, 0);
            if (vok[i]) q = *(reinterpret_cast<const uint4 *>(static_cast<const char *>(p.x) + b * p.x_stride) + v);
            Pairs<T>::unpack(q, xr[b][i]);
        }
    }
    __syncthreads();  // thresholds are in shared memory

    const int my_n = batch_union_share<BT>(p, s_tau, s_bal, s_balb, s_list, s_keep, s_wtot, keep_policy);
    __syncthreads();  // list, keep bits and the mbarriers are ready

    bool timed_out = false;

    if (warp == kConsWarps) {
        // ---- producer (as in the single-sequence kernel) -------------------------------------------
        if (lane == 0) {
            const char *Wg = static_cast<const char *>(p.w_gate);
            const char *Wu = static_cast<const char *>(p.w_up);
            const char *Wd = static_cast<const char *>(p.w_down_t);
            const uint64_t stream_policy = policy_evict_first();
            int issued = 0;
            int s = 0;            // ring position and the parity of its current use, kept incrementally
            uint32_t par = 0;
            for (int i = 0; i < my_n; ++i) {
                if (!mbar_wait(empty0 + 8 * s, par ^ 1)) {
                    timed_out = true;
                    break;
                }
                const size_t off = (size_t)guard_row(s_list[i], p.d_ff, p.status) * row_bytes;
                const uint32_t dst = ring + (uint32_t)s * stage_bytes, bar = full0 + 8 * s;
                mbar_expect_tx(bar, stage_bytes);
                bulk_load_row_hint(dst, Wg + off, row_bytes, bar, stream_policy);
                if (gated) bulk_load_row_hint(dst + row_bytes, Wu + off, row_bytes, bar, stream_policy);
                bulk_load_row_hint(dst + down_off, Wd + off, row_bytes, bar, stream_policy);
                issued = i + 1;
                if (++s == n_stages) {
                    s = 0;
                    par ^= 1;
                }
            }
            for (int i = max(0, issued - n_stages); i < issued; ++i)
                if (!mbar_wait(full0 + 8 * (i % n_stages), (i / n_stages) & 1)) timed_out = true;
        }
    } else {
        // ---- consumers ---------------------------------------------------------------------------
        float2 acc[BT][NV][P];
#pragma unroll
        for (int b = 0; b < BT; ++b)
#pragma unroll
            for (int i = 0; i < NV; ++i)
#pragma unroll
                for (int e = 0; e < P; ++e) acc[b][i][e] = make_float2(0.f, 0.f);
        const bool b16 = lane & 16, b8 = lane & 8, b4 = lane & 4, b2 = lane & 2;
        int buf = 0;
        int cs = 0;           // ring position of the next neuron to consume, and the parity of its use
        uint32_t cpar = 0;
        for (int g0 = 0; g0 < my_n; g0 += GB, buf ^= 1) {
            float pd[16];  // value (g * BT + b) * 2 + {0: gate, 1: up}
            uint32_t st_addr[GB];
            int st_idx[GB];
#pragma unroll
            for (int g = 0; g < GB; ++g) {
                const int i = g0 + g;
                float2 sg[BT], su[BT];
#pragma unroll
                for (int b = 0; b < BT; ++b) sg[b] = su[b] = make_float2(0.f, 0.f);
                st_idx[g] = cs;
                st_addr[g] = ring + (uint32_t)cs * stage_bytes;
                if (i < my_n) {
                    if (!timed_out && !mbar_wait(full0 + 8 * cs, cpar)) timed_out = true;
                    if (++cs == n_stages) {
                        cs = 0;
                        cpar ^= 1;
                    }
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        if (!vok[k]) continue;
                        const uint32_t a = st_addr[g] + (uint32_t)(tid + k * kConsumers) * 16u;
                        float2 fg[P], fu[P];
                        Pairs<T>::unpack(lds128(a), fg);
                        if (gated) {
                            Pairs<T>::unpack(lds128(a + row_bytes), fu);
#pragma unroll
                            for (int b = 0; b < BT; ++b)
#pragma unroll
                                for (int e = 0; e < P; ++e) {
                                    sg[b] = __ffma2_rn(fg[e], xr[b][k][e], sg[b]);
                                    su[b] = __ffma2_rn(fu[e], xr[b][k][e], su[b]);
                                }
                        } else {
#pragma unroll
                            for (int b = 0; b < BT; ++b)
#pragma unroll
                                for (int e = 0; e < P; ++e) sg[b] = __ffma2_rn(fg[e], xr[b][k][e], sg[b]);
                        }
                    }
                }
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    pd[(g * BT + b) * 2] = sg[b].x + sg[b].y;
                    pd[(g * BT + b) * 2 + 1] = su[b].x + su[b].y;
                }
            }
            // Warp sums of the 16 values by a halving butterfly (16 shuffles): afterwards both lanes of pair
            // v hold the warp total of value v.  Then across the 16 warps through shared memory: lane l adds
            // 8 warps of value l / 2, the pair finishes.  Fixed order throughout.
            float b8v[8], b4v[4], b2v[2], v16;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float send = b16 ? pd[i] : pd[i + 8];
                b8v[i] = (b16 ? pd[i + 8] : pd[i]) + __shfl_xor_sync(0xffffffffu, send, 16);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float send = b8 ? b8v[i] : b8v[i + 4];
                b4v[i] = (b8 ? b8v[i + 4] : b8v[i]) + __shfl_xor_sync(0xffffffffu, send, 8);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const float send = b4 ? b4v[i] : b4v[i + 2];
                b2v[i] = (b4 ? b4v[i + 2] : b4v[i]) + __shfl_xor_sync(0xffffffffu, send, 4);
            }
            v16 = (b2 ? b2v[1] : b2v[0]) + __shfl_xor_sync(0xffffffffu, b2 ? b2v[0] : b2v[1], 2);
            v16 += __shfl_xor_sync(0xffffffffu, v16, 1);
            // value index: bit4 -> +8, bit3 -> +4, bit2 -> +2, bit1 -> +1  ( = lane >> 1 )
            if ((lane & 1) == 0) s_dot[buf][lane >> 1][warp] = v16;
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
            float tot;
            {
                const float4 *src = reinterpret_cast<const float4 *>(&s_dot[buf][lane >> 1][(lane & 1) * 8]);
                const float4 q0 = src[0], q1 = src[1];
                tot = ((q0.x + q0.y) + (q0.z + q0.w)) + ((q1.x + q1.y) + (q1.z + q1.w));
                tot += __shfl_xor_sync(0xffffffffu, tot, 1);
            }
            const float up = __shfl_xor_sync(0xffffffffu, tot, 2);  // value 2m+1 sits 2 lanes above value 2m
            const float hval = neuron_value_f(p.act, tot, up);                    // pair m = g * BT + b sits on lanes 4m, 4m+1
#pragma unroll
            for (int g = 0; g < GB; ++g) {
                float h[BT];
#pragma unroll
                for (int b = 0; b < BT; ++b) h[b] = __shfl_sync(0xffffffffu, hval, 4 * (g * BT + b));
                if (g0 + g >= my_n) continue;
                const int bits = s_keep[g0 + g];
                float2 h2[BT];
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    const float hb = ((bits >> b) & 1) ? h[b] : 0.f;  // not kept by sequence b: no contribution
                    h2[b] = make_float2(hb, hb);
                }
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    if (!vok[k]) continue;
                    float2 fd[P];
                    Pairs<T>::unpack(lds128(st_addr[g] + down_off + (uint32_t)(tid + k * kConsumers) * 16u), fd);
#pragma unroll
                    for (int b = 0; b < BT; ++b)
#pragma unroll
                        for (int e = 0; e < P; ++e) acc[b][k][e] = __ffma2_rn(h2[b], fd[e], acc[b][k][e]);
                }
            }
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int g = 0; g < GB; ++g)
                    if (g0 + g < my_n) mbar_arrive(empty0 + 8 * st_idx[g]);
            }
        }
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            float *mine = p.partials + ((size_t)cta * BT + b) * d;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                if (!vok[i]) continue;
                float4 *dst = reinterpret_cast<float4 *>(mine + (size_t)(tid + i * kConsumers) * E);
#pragma unroll
                for (int e = 0; e < P; e += 2)
                    dst[e / 2] = make_float4(acc[b][i][e].x, acc[b][i][e].y, acc[b][i][e + 1].x, acc[b][i][e + 1].y);
            }
        }
    }
    if (timed_out && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);

    // ---- epilogue: grid barrier, deterministic column reduction per sequence ----------------------
    if (!grid_barrier(p.ctrl, (unsigned)n_ctas, kConsumers)) {
        if (tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }
    batch_column_sums<BT>(p);
}


// One thread per (sequence, 32-neuron chunk): eight 16-byte loads, one keep word.
__global__ void __launch_bounds__(256)
keep_words_kernel(const float *__restrict__ scores, int B, int d_ff, const float *__restrict__ tau,
                  long long tau_stride, unsigned *__restrict__ words) {
    pdl_launch_dependents();
    pdl_wait();
    const int chunks = (d_ff + kWarp - 1) / kWarp;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * chunks) return;
    const int b = i / chunks, q = i - b * chunks;
    const float *sc = scores + (size_t)b * d_ff;
    const float t = tau[(size_t)b * tau_stride];
    const int j0 = q * kWarp;
    unsigned w = 0;
    if (((reinterpret_cast<uintptr_t>(sc) & 15u) == 0) && j0 + kWarp <= d_ff) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldg(reinterpret_cast<const float4 *>(sc + j0) + u);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            w |= (v[u].x >= t ? 1u : 0u) << (4 * u);
            w |= (v[u].y >= t ? 1u : 0u) << (4 * u + 1);
            w |= (v[u].z >= t ? 1u : 0u) << (4 * u + 2);
            w |= (v[u].w >= t ? 1u : 0u) << (4 * u + 3);
        }
    } else {
        for (int u = 0; u < kWarp; ++u)
            if (j0 + u < d_ff && sc[j0 + u] >= t) w |= 1u << u;
    }
    words[i] = w;
}

// ---- host side ------------------------------------------------------------------------------

size_t keep_words_bytes_of(int B, int d_ff) { return keep_words_bytes(B, d_ff); }

int launch_keep_words(const float *scores, int B, int d_ff, const float *tau, long long tau_stride, unsigned *words,
                      cudaStream_t st) {
    const int chunks = (d_ff + kWarp - 1) / kWarp;
    const int n = B * chunks;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((n + 255) / 256);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void *args[] = {&scores, &B, &d_ff, &tau, &tau_stride, &words};
    CLADA_CUDA_TRY(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(keep_words_kernel), args));
    return CLADA_OK;
}

template <typename T, int NV, int BT>
static int launch_batch_variant(const FfnBatchParams &p, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_batch_kernel<T, NV, BT>;
    const size_t stage_bytes = (act_is_gated(p.act) ? 3 : 2) * (size_t)(p.d_model / E) * 16;
    const size_t chunks = (size_t)(p.d_ff + 31) / 32;
    const size_t tail = 2 * kMaxStages * sizeof(uint64_t) + (1 + BT) * chunks * sizeof(unsigned) +
                        2 * (size_t)(p.d_ff / di.num_sms + 2) * sizeof(int);
    const size_t budget = (size_t)di.max_smem_optin - 4096;  // leave room for the static arrays
    if (budget < tail + 4 * stage_bytes) return CLADA_ERR_UNSUPPORTED;  // a reduction group needs up to 4 stages
    int n_stages = (int)((budget - tail) / stage_bytes);
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    const size_t smem = (size_t)n_stages * stage_bytes + tail;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
        configured[di.device & 63] = true;
    }
    FfnBatchParams params = p;
    int stages_arg = n_stages;
    void *args[] = {&params, &stages_arg};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(di.num_sms);
    cfg.blockDim = dim3(kFfnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident: the grid barrier cannot starve
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    CLADA_CUDA_TRY(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kern), args));
    return CLADA_OK;
}

int ffn_batch_tile(const clada_layer *layer, int remaining) {
    const int vpr = layer->d_model / (layer->dtype == CLADA_F32 ? 4 : 8);
    if (layer->d_ff > kBatchMaxBatches * kWarp * kFfnThreads) return 1;
    if (remaining >= 4 && vpr <= kConsumers) return 4;
    if (remaining >= 2 && vpr <= 2 * kConsumers) return 2;
    return 1;
}

int launch_ffn_batch(const clada_layer *layer, int bt, const void *x, const float *scores, const float *tau,
                     long long tau_stride, void *y, int y_dtype, void *ws, const unsigned *keep_words,
                     int32_t *status, cudaStream_t st) {
    FfnBatchParams p;
    p.w_gate = layer->w_gate;
    p.w_up = layer->w_up;
    p.w_down_t = layer->w_down_t;
    p.x = x;
    p.x_stride = (size_t)layer->d_model * elem_size(layer->dtype);
    p.scores = scores;
    p.keep_words = keep_words;
    p.tau = tau;
    p.tau_stride = tau_stride;
    p.y = y;
    p.y_stride = (size_t)layer->d_model * elem_size(y_dtype);
    p.y_dtype = y_dtype;
    p.partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
    p.ctrl = static_cast<WsCtrl *>(ws);
    p.status = status;
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.act = layer->activation;
    // 16-bit layers: the tile kernel with the gate / up contractions on the tensor cores, where it takes the shape
    if (ffn_batch_tc_supported(layer, bt)) return launch_ffn_batch_tc(p, layer->dtype, bt, st);
    const bool f32 = layer->dtype == CLADA_F32;
    const int vpr = layer->d_model / (f32 ? 4 : 8);
    const bool f16 = layer->dtype == CLADA_F16;
    if (bt == 4 && vpr <= kConsumers)
        return f32   ? launch_batch_variant<float, 1, 4>(p, st)
               : f16 ? launch_batch_variant<__half, 1, 4>(p, st)
                     : launch_batch_variant<__nv_bfloat16, 1, 4>(p, st);
    if (bt == 2 && vpr <= kConsumers)
        return f32   ? launch_batch_variant<float, 1, 2>(p, st)
               : f16 ? launch_batch_variant<__half, 1, 2>(p, st)
                     : launch_batch_variant<__nv_bfloat16, 1, 2>(p, st);
    if (bt == 2 && vpr <= 2 * kConsumers)
        return f32   ? launch_batch_variant<float, 2, 2>(p, st)
               : f16 ? launch_batch_variant<__half, 2, 2>(p, st)
                     : launch_batch_variant<__nv_bfloat16, 2, 2>(p, st);
    return CLADA_ERR_UNSUPPORTED;
}

}  // namespace clada
