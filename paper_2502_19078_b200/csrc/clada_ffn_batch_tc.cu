// Sparse gated FFN decode for a tile of BT sequences (per-sequence masks), 16-bit layers, with the gate / up
// contractions on the tensor cores:
//   kept_b = { j : A_bj >= tau_b },   y_b = sum_{j in kept_b} silu(w_gate_j . x_b) (w_up_j . x_b) w_down_t[j,:]
//
// A tile is a skinny matrix product: BT <= 4 rows of x against the gate and up rows of the union's neurons.  On
// CUDA cores every (neuron, sequence) dot product costs a 512-thread reduction and the tile kernel spends ~240
// instructions per thread and neuron; here a chunk of four neurons is ONE chain of warp-level
// mma.m16n8k16 instructions per warp: the 16 rows of the A operand are the tile's sequences (rows past BT are
// zero), the 8 columns of the B operand are the chunk's four gate rows and four up rows, and each of the 16
// consumer warps owns a slice of K = d_model (its x fragments stay in registers for the whole launch).  The
// order of k inside a slice is permuted so that one 16-byte shared-memory load per lane feeds two k-steps and
// the same 16-byte vectors of x are the A fragments.  The 16 warps' partial D tiles go to shared memory; after
// one CTA barrier every warp sums them for itself in warp order (fp32, round to nearest), forms the neuron
// values h, zeroes them for the sequences that cut the neuron, and scales the down rows into the per-thread
// partial y on the CUDA cores as before.
//
// Precision: products of two 16-bit values are exact in the tensor core; its fp32 accumulation is not IEEE
// (it truncates), so a chain is kept short -- at most 10 k-steps per accumulator, two accumulators per warp,
// everything above that is summed in fp32 on the CUDA cores -- and the outputs stay within the 1e-5 of the
// oracle that the CUDA-core kernels are held to (tested on every tile shape and on the full-size layers).
//
// Everything else is the CUDA-core tile kernel's: the union prologue, the bulk-copy ring (rows padded by 64
// bytes so that the B loads of two neighbouring neurons fall on different banks), the bounded waits, the
// deterministic column sums.
#include <math.h>

#include "common.cuh"
#include "ffn_batch.cuh"
#include "ffn_common.cuh"

namespace clada {

constexpr uint32_t kRowPad = 64;  // bytes between staged rows beyond the row itself

#ifdef CLADA_TC_TRACE
#ifndef CLADA_TC_TRACE_TID
#define CLADA_TC_TRACE_TID 0
#endif
__device__ unsigned long long *g_tc_trace = nullptr;  // [n_ctas][256 chunks][8 slots]
#define TC_TRACE(chunk, slot)                                                                              \
    do {                                                                                                   \
        if (g_tc_trace && tid == CLADA_TC_TRACE_TID && (chunk) < 256) {                                                     \
            unsigned long long t_;                                                                         \
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));                                          \
            g_tc_trace[((size_t)blockIdx.x * 256 + (chunk)) * 8 + (slot)] = t_;                            \
        }                                                                                                  \
    } while (0)
#else
#define TC_TRACE(chunk, slot) \
    do {                      \
    } while (0)
#endif

template <typename T> struct TileMma;
template <> struct TileMma<__nv_bfloat16> {
    // D (16 x 8, fp32) += A (16 x 16: rows 0-7 given, rows 8-15 zero) . B (16 x 8)
    __device__ static __forceinline__ void run(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
    }
};
template <> struct TileMma<__half> {
    __device__ static __forceinline__ void run(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
    }
};

// NV: 16-byte vectors of a row per thread (down projection); NPS: pairs of k-steps per warp, i.e. 16-byte
// vectors of x per lane (16 warps x NPS x 4 lanes of a quad cover a row of up to 64 NPS vectors).
//
// 512 threads and no producer warp: with a seventeenth warp one scheduler of the SM would hold five warps, which
// caps a thread at 96 registers -- the x fragments and the partial y then spill, and with nearly all of the SM's
// L1 carved out as shared memory every spill reload is a trip to L2 (that, not arithmetic, was what held the
// CUDA-core tile kernel at 1.2 us per neuron).  Warp 0 issues the bulk copies itself: the first ring's worth
// after the prologue, and at every chunk, right after the barrier that follows the MMAs -- by then every warp
// has finished the previous chunk's down rows -- the copies that reuse that chunk's stages.  The CTA barrier
// is the hand-back; only the "stage full" mbarriers remain.
template <typename T, int NV, int BT, int NPS, int CH>
__global__ void __launch_bounds__(kConsumers, 1)
sparse_ffn_batch_tc_kernel(const FfnBatchParams p, const int n_stages) {
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = Pairs<T>::kPairs;
    static_assert(CH >= 1 && CH <= 4, "a chunk's gate rows are columns 0-3 of the B tile, its up rows columns 4-7");
    static_assert(BT == 2 || BT == 4, "tile of 2 or 4 sequences");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff, d = p.d_model;
    const int vpr = d / E;
    const uint32_t row_bytes = (uint32_t)vpr * 16u;
    const uint32_t pitch = row_bytes + kRowPad;
    const bool gated = act_is_gated(p.act);
    const uint32_t n_rows = gated ? 3u : 2u;  // gate | up | down, or gate | down without a gate projection
    const uint32_t stage_bytes = n_rows * pitch;
    const uint32_t down_off = (n_rows - 1u) * pitch;
    const int chunks = (F + kWarp - 1) / kWarp;
    const int list_cap = F / n_ctas + 2;

    // dynamic shared memory: ring | full | union keep-bits | per-sequence keep-bits | list | keep nibbles
    const uint32_t ring = smem_u32(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)n_stages * stage_bytes);
    const uint32_t full0 = smem_u32(bars);
    unsigned *s_bal = reinterpret_cast<unsigned *>(bars + kMaxStages);
    unsigned *s_balb = s_bal + chunks;                      // [BT][chunks]
    int *s_list = reinterpret_cast<int *>(s_balb + BT * chunks);
    int *s_keep = s_list + list_cap;                        // bit b: sequence b keeps this neuron
    __shared__ int s_wtot[kConsWarps];
    __shared__ float s_tau[BT];
    __shared__ __align__(16) float s_part[2][kConsWarps][BT][8];  // per chunk parity and warp: D rows of the sequences

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) mbar_init(full0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();
    TC_TRACE(255, 0);

    const uint64_t keep_policy = policy_evict_last();
    if (tid < BT) s_tau[tid] = ld_keep(p.tau + (size_t)tid * p.tau_stride, keep_policy);
    const int g = lane >> 2, t = lane & 3;
    bool vok[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) vok[i] = tid + i * kConsumers < vpr;
    __syncthreads();  // thresholds are in shared memory

    const int my_n = batch_union_share<BT, kConsumers>(p, s_tau, s_bal, s_balb, s_list, s_keep, s_wtot, keep_policy);
    __syncthreads();  // list, keep bits and the mbarriers are ready
    TC_TRACE(255, 1);

    // ---- the copies (thread 0) -----------------------------------------------------------------------------
    // Warp 0 issues: lane l copies row l % n_rows of neuron first + l / n_rows (one bulk copy per lane, so a
    // chunk's twelve copies go out together instead of one after another from a single thread).
    auto issue = [&](int first, int count) {  // neurons [first, first + count) of the share, count <= 8
        const int q = lane / (int)n_rows, r = lane - q * (int)n_rows;
        const int i = first + q;
        const bool on = q < count;
        const int s = on ? i % n_stages : 0;
        const uint32_t bar = full0 + 8 * s;
        if (on && r == 0) mbar_expect_tx(bar, n_rows * row_bytes);
        __syncwarp();
        if (on) {
            const void *base = r == 0 ? p.w_gate : (r + 1 == (int)n_rows ? p.w_down_t : p.w_up);
            const char *src = static_cast<const char *>(base) + (size_t)guard_row(s_list[i], p.d_ff, p.status) * row_bytes;
            bulk_load_row_hint(ring + (uint32_t)s * stage_bytes + (uint32_t)r * pitch, src, row_bytes, bar,
                               policy_evict_first());
        }
    };
    if (warp == 0)
        for (int i = 0; i < min(my_n, n_stages); i += 8) issue(i, min(8, min(my_n, n_stages) - i));

    // A fragments: lane (g, t) = (lane / 4, lane % 4) holds, for each of its warp's pairs of k-steps, the
    // 16-byte vector 4 * pair + t of sequence g's x (zero for g >= BT and past the row's end).  A warp's pairs
    // are warp, warp + 16, ...: consecutive warps read consecutive 64-byte pieces of x.
    uint4 afrag[NPS];
#pragma unroll
    for (int j = 0; j < NPS; ++j) {
        const int v = 4 * (warp + kConsWarps * j) + t;
        afrag[j] = make_uint4(0u, 0u, 0u, 0u);
        if (g < BT && v < vpr)
            afrag[j] = *(reinterpret_cast<const uint4 *>(static_cast<const char *>(p.x) + g * p.x_stride) + v);
    }

    TC_TRACE(255, 2);
    bool timed_out = false;
    float2 acc[BT][NV][P];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int e = 0; e < P; ++e) acc[b][i][e] = make_float2(0.f, 0.f);
    int cs = 0;           // ring position of the chunk's first neuron, and the parity of its use
    uint32_t cpar = 0;
    // B rows of this lane: lane (g, t) feeds column g of the B tile
    const int nb = g & 3;
    const uint32_t b_off = (g >= 4 ? pitch : 0u);
    for (int g0 = 0; g0 < my_n; g0 += CH) {
        const int nn = min(CH, my_n - g0);
        TC_TRACE(g0 / CH, 0);
        // the chunk's stages: neuron q of the chunk sits in stage s0 + q (wrapped)
        const int s0 = cs;
        {
            int s = cs;
            uint32_t par = cpar;
#pragma unroll
            for (int q = 0; q < CH; ++q) {
                if (q < nn) {
                    if (!timed_out && !mbar_wait(full0 + 8 * s, par)) timed_out = true;
                    if (++s == n_stages) {
                        s = 0;
                        par ^= 1;
                    }
                }
            }
            cs = s;
            cpar = par;
        }
        auto stage_addr = [&](int q) {
            const int s = s0 + q;
            return ring + (uint32_t)(s < n_stages ? s : s - n_stages) * stage_bytes;
        };
        TC_TRACE(g0 / CH, 1);
        // ---- gate | up of four neurons for all sequences: one chain of warp-level MMAs per accumulator ----
        float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const bool row_ok = nb < nn && (g < 4 || gated);
            const uint32_t brow = stage_addr(nb) + b_off;
#pragma unroll
            for (int j = 0; j < NPS; ++j) {
                const int v = 4 * (warp + kConsWarps * j) + t;
                uint4 b = make_uint4(0u, 0u, 0u, 0u);
                if (row_ok && v < vpr) b = lds128(brow + (uint32_t)v * 16u);
                TileMma<T>::run(d0, afrag[j].x, afrag[j].y, b.x, b.y);
                TileMma<T>::run(d1, afrag[j].z, afrag[j].w, b.z, b.w);
            }
        }
        // D rows 0 .. BT-1 (lanes with g < BT), columns 2t, 2t+1
        const int pb = (g0 / CH) & 1;  // double buffer: a slow warp may still be reading the chunk before
        if (g < BT) *reinterpret_cast<float2 *>(&s_part[pb][warp][g][2 * t]) = make_float2(d0[0] + d1[0], d0[1] + d1[1]);
        TC_TRACE(g0 / CH, 2);
        __syncthreads();  // every warp is past the previous chunk's down rows and has stored its partial tile
        TC_TRACE(g0 / CH, 3);
        // the copies that reuse the previous chunk's stages
        if (warp == 0 && g0 > 0) {
            const int first = g0 - CH + n_stages;
            if (first < my_n) issue(first, min(CH, my_n - first));
        }
        // ---- sum over the 16 warps (their K slices), neuron values: every warp for itself, so that no second
        // barrier is needed.  Lane l holds value (b, n) = (l / 8, l % 8), adds the 16 partials in warp order;
        // column n + 4 is the same neuron's up row. ----
        float hval = 0.f;
        {
            const int b = lane >> 3, n = lane & 7;
            float s16 = 0.f;
            if (b < BT) {
#pragma unroll
                for (int wv = 0; wv < kConsWarps; ++wv) s16 += s_part[pb][wv][b][n];
            }
            const float up = __shfl_xor_sync(0xffffffffu, s16, 4);
            // not kept by sequence b, or past the share's end: no contribution
            if (b < BT && n < nn && ((s_keep[g0 + (n & 3)] >> b) & 1)) hval = neuron_value_f(p.act, s16, up);
        }
        TC_TRACE(g0 / CH, 4);
        TC_TRACE(g0 / CH, 5);
        // ---- down rows scaled into the partial y ---------------------------------------------------------
#pragma unroll
        for (int q = 0; q < CH; ++q) {
            float2 h2[BT];
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                const float h = __shfl_sync(0xffffffffu, hval, b * 8 + q);
                h2[b] = make_float2(h, h);
            }
            if (q >= nn) continue;
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                if (!vok[k]) continue;
                float2 fd[P];
                Pairs<T>::unpack(lds128(stage_addr(q) + down_off + (uint32_t)(tid + k * kConsumers) * 16u), fd);
#pragma unroll
                for (int b = 0; b < BT; ++b)
#pragma unroll
                    for (int e = 0; e < P; ++e) acc[b][k][e] = __ffma2_rn(h2[b], fd[e], acc[b][k][e]);
            }
        }
        TC_TRACE(g0 / CH, 6);
    }
    TC_TRACE(255, 3);
    // Never leave with copies in flight.  Every copy issued was waited for above, unless a wait gave up: then
    // thread 0 waits (bounded again) for the last ring's worth.
    if (timed_out && tid == 0) {
        const int issued = my_n;  // at most: copies are issued at most n_stages ahead of the chunk being read
        for (int i = max(0, issued - n_stages); i < issued; ++i) mbar_wait(full0 + 8 * (i % n_stages), (i / n_stages) & 1);
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
    if (timed_out && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
    TC_TRACE(255, 4);

    // ---- epilogue: grid barrier, deterministic column reduction per sequence ----------------------
    if (!grid_barrier(p.ctrl, (unsigned)n_ctas, kWarp)) {
        if (tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }
    TC_TRACE(255, 5);
    batch_column_sums<BT, kConsumers>(p);
    TC_TRACE(255, 6);
}

// ---- host side ------------------------------------------------------------------------------

// Ring stages of a launch: as many as fit beside the prologue's arrays, at most kMaxStages.
static int tc_ring_stages(const FfnBatchParams &p, int bt, const DeviceInfo &di, size_t *smem, size_t *budget) {
    const size_t stage_bytes = (act_is_gated(p.act) ? 3 : 2) * ((size_t)(p.d_model / 8) * 16 + kRowPad);
    const size_t chunks = (size_t)(p.d_ff + 31) / 32;
    const size_t tail = kMaxStages * sizeof(uint64_t) + (1 + bt) * chunks * sizeof(unsigned) +
                        2 * (size_t)(p.d_ff / di.num_sms + 2) * sizeof(int);
    *budget = (size_t)di.max_smem_optin - 6144;  // leave room for the static arrays (partial tiles: 4 KB)
    int n_stages = *budget > tail ? (int)((*budget - tail) / stage_bytes) : 0;
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    *smem = (size_t)n_stages * stage_bytes + tail;
    return n_stages;
}

template <typename T, int NV, int BT, int NPS, int CH>
static int launch_tc_variant(const FfnBatchParams &p, cudaStream_t st) {
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_batch_tc_kernel<T, NV, BT, NPS, CH>;
    size_t smem, budget;
    const int n_stages = tc_ring_stages(p, BT, di, &smem, &budget);
    if (n_stages < 2 * CH) return CLADA_ERR_UNSUPPORTED;  // the chunk being read and the chunk on its way
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
        configured[di.device & 63] = true;
    }
    FfnBatchParams params = p;
    int stages_arg = n_stages;
    void *args[] = {&params, &stages_arg};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(di.num_sms);
    cfg.blockDim = dim3(kConsumers);
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

// Rows of up to 512 vectors (d_model 4096) take 8 pairs of k-steps per warp and tiles of 4 or 2; rows of up to
// 640 vectors (d_model 5120) 10 pairs and tiles of 2 (two vectors of partial y per thread and sequence).  A chunk
// is four neurons when the ring holds eight stages or more, else three (six or seven stages: d_model 5120).
bool ffn_batch_tc_supported(const clada_layer *layer, int bt) {
    if (layer->dtype != CLADA_BF16 && layer->dtype != CLADA_F16) return false;
    const int vpr = layer->d_model / 8;
    if (!((bt == 4 && vpr <= kConsumers) || (bt == 2 && vpr <= 640))) return false;
    DeviceInfo di;
    if (device_info(&di) != CLADA_OK) return false;
    FfnBatchParams p = {};
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.act = layer->activation;
    size_t smem, budget;
    return tc_ring_stages(p, bt, di, &smem, &budget) >= 6;
}

template <typename T, int NV, int BT, int NPS>
static int launch_tc_chunked(const FfnBatchParams &p, cudaStream_t st) {
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    size_t smem, budget;
    const int n_stages = tc_ring_stages(p, BT, di, &smem, &budget);
    if (n_stages >= 8) return launch_tc_variant<T, NV, BT, NPS, 4>(p, st);
    return launch_tc_variant<T, NV, BT, NPS, 3>(p, st);
}

template <typename T>
static int launch_tc_typed(const FfnBatchParams &p, int bt, cudaStream_t st) {
    const int vpr = p.d_model / Elem<T>::kPerVec;
    if (bt == 4 && vpr <= kConsumers) return launch_tc_chunked<T, 1, 4, 8>(p, st);
    if (bt == 2 && vpr <= kConsumers) return launch_tc_chunked<T, 1, 2, 8>(p, st);
    if (bt == 2 && vpr <= 640) return launch_tc_chunked<T, 2, 2, 10>(p, st);
    return CLADA_ERR_UNSUPPORTED;
}

int launch_ffn_batch_tc(const FfnBatchParams &p, int dtype, int bt, cudaStream_t st) {
    return dtype == CLADA_BF16 ? launch_tc_typed<__nv_bfloat16>(p, bt, st) : launch_tc_typed<__half>(p, bt, st);
}

}  // namespace clada

#ifdef CLADA_TC_TRACE
extern "C" int clada_tc_trace_buffer(unsigned long long *buf) {
    CLADA_CUDA_TRY(cudaMemcpyToSymbol(clada::g_tc_trace, &buf, sizeof buf));
    return CLADA_OK;
}
#endif
