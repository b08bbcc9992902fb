// Sparse gated FFN for one decode token per sequence (Algorithm 2, generation phase):
//   kept = { j : A_j >= tau_final },  y = sum_{j in kept} silu(w_gate_j . x) (w_up_j . x) w_down_t[j,:]
//
// One persistent cooperative kernel per (layer, sequence), one CTA per SM:
//   prologue  every CTA tests all F scores against tau (the vector arrives as one bulk copy into the idle
//             ring; a warp tests 32 chunks of 32 neurons with one ballot each), a block scan ranks the
//             chunks, and the CTA takes an equal share [r0, r1) of the kept neurons in ascending order,
//             or, given a nested index list, simply copies its share of the list's head;
//   stream    a producer thread copies the three contiguous rows of each kept neuron into a ring of
//             shared-memory stages with bulk asynchronous copies (mbarrier-tracked), which keeps
//             ~200 KB of HBM requests in flight per SM whatever the consumers are doing.  Consumer
//             thread t owns the same 16-byte column vectors of every row (x and the partial y for
//             those columns live in registers) and reads the staged rows from shared memory, four
//             neurons per CTA-wide reduction;
//   epilogue  each CTA stores its fp32 partial y, all CTAs meet at a bounded grid barrier, then every
//             CTA sums a slice of columns over all partials in CTA order (deterministic) and writes y.
#include <math.h>

#include "common.cuh"
#include "ffn_common.cuh"
#include "ffn_single.cuh"

namespace clada {

// floor(n * c / n_ctas): where CTA c's even share of n items starts.  n <= 69632 and c <= n_ctas (a few
// hundred), so the product fits 32 bits and the division is the cheap one.
__device__ __forceinline__ int split_at(int n, int c, int n_ctas) {
    return (int)(((unsigned)n * (unsigned)c) / (unsigned)n_ctas);
}

constexpr int G = GS;                         // neurons per group-wide reduction (a reduction holds G stages)
constexpr int kMaxBatches = kSingleMaxDff / (kWarp * kFfnThreads);  // prologue batches

template <typename T, int NV, bool GATED, int GROUPS>
__global__ void __launch_bounds__(kFfnThreads, 1)
sparse_ffn_kernel(const FfnParams p, const int n_stages) {
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = Pairs<T>::kPairs;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff, d = p.d_model;
    const int vpr = d / E;  // 16-byte vectors per row
    const uint32_t row_bytes = (uint32_t)vpr * 16u;
    constexpr uint32_t kRows = GATED ? 3u : 2u;  // gate | up | down, or gate | down without a gate projection
    const uint32_t stage_bytes = kRows * row_bytes;
    const uint32_t down_off = (kRows - 1u) * row_bytes;
    const int chunks = (F + kWarp - 1) / kWarp;

    // dynamic shared memory: ring | full[kMaxStages] | empty[kMaxStages] | keep-bits | kept list
    const uint32_t ring = smem_u32(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)n_stages * stage_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages);
    const uint32_t sbar = smem_u32(bars + 2 * kMaxStages);  // completion of the score vector's bulk copy
    unsigned *s_bal = reinterpret_cast<unsigned *>(bars + 2 * kMaxStages + 1);  // keep-bits word per chunk
    int *s_list = reinterpret_cast<int *>(s_bal + chunks);
    __shared__ int s_wtot[kFfnWarps];
    __shared__ float s_tau;
    __shared__ __align__(16) float s_dot[kDotFloats];
    constexpr int GT = kConsumers / GROUPS;  // threads per consumer group (the producer warp counts as none)
    const int grp = tid < kConsumers ? tid / GT : 0, gt = tid - grp * GT;

    pdl_launch_dependents();  // the next kernel in the stream may be scheduled as SMs free up
    if (tid == kConsumers) {  // the producer warp sets the ring up while the others start loading
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full0 + 8 * s, 1);            // the producer's expect_tx arrival
            mbar_init(empty0 + 8 * s, kConsWarps / GROUPS);  // one arrival per warp of the group that owns the stage
        }
        mbar_init(sbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();  // everything below may read what the previous kernel wrote

    const uint64_t keep_policy = policy_evict_last();
    const bool nested = p.order != nullptr;
    __shared__ int s_cnt[5];
    if (nested) {  // the four counts and the level are independent loads: one round trip
        if (tid < 4) s_cnt[tid] = p.counts[tid];
        if (tid == 4) s_cnt[4] = *p.level;
    } else if (tid == 0) {
        s_tau = ld_keep(p.tau, keep_policy);  // one request per CTA, not one per warp
    }
    // x of this thread's columns (consumers), requested before the scan so the latencies overlap
    float2 xr[NV][P];
    bool vok[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int v = gt + i * GT;
        vok[i] = tid < kConsumers && v < vpr;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (vok[i]) q = *(reinterpret_cast<const uint4 *>(p.x) + v);
        Pairs<T>::unpack(q, xr[i]);
    }

    // ---- prologue: threshold test, ranks, this CTA's share of the kept list ---------------------
    // A batch is one 32-neuron chunk per thread; F <= 32 * kFfnThreads needs a single batch.  The keep-bits
    // words stay in registers (thread tid owns chunk tid of the batch) and are ranked by a block-wide scan.
    int n_act_o = 0, r0_o = 0, r1_o = 0;
    if (nested) {
        // The list exists already: this CTA copies its share of the leading n_act entries.  A count or
        // an index outside its range is clamped (no access leaves the layer) and reported.
        __syncthreads();
        const int lv = s_cnt[4];
        int n = s_cnt[lv & 3];
        bool bad = lv < 0 || lv > 3 || n < 0 || n > F;
        n = min(max(n, 0), F);
        n_act_o = n;
        r0_o = split_at(n, cta, n_ctas);
        r1_o = split_at(n, cta + 1, n_ctas);
        for (int i = tid; i < r1_o - r0_o; i += kFfnThreads) {
            const int j = p.order[r0_o + i];
            bad |= j < 0 || j >= F;
            s_list[i] = min(max(j, 0), F - 1);
        }
        if (bad && p.status) atomicOr(p.status, CLADA_STATUS_BAD_INDEX);
    } else {
    const bool vec_ok = (reinterpret_cast<uintptr_t>(p.scores) & 15u) == 0;
    const int n_batches = (chunks + kFfnThreads - 1) / kFfnThreads;
    unsigned bal[kMaxBatches];  // keep bits of this thread's chunk in every batch
    // The score vector comes in as ONE bulk copy into the (still idle) ring when it is aligned and fits: 148 CTAs
    // each pulling the same 44 KB through L2 with per-thread loads took ~2.4 us, the copy engine's stream about
    // half that.  Otherwise the threads load their chunks themselves.
    const bool bulk_scores = vec_ok && (F & 3) == 0 && (size_t)F * 4 <= (size_t)n_stages * stage_bytes;
    if (bulk_scores && tid == kConsumers) {
        mbar_expect_tx(sbar, (uint32_t)F * 4u);
        bulk_load_row_hint(ring, p.scores, (uint32_t)F * 4u, sbar, keep_policy);
    }
    {
        // A warp tests 32 chunks.  For chunk c every lane holds ONE neuron's score -- consecutive addresses, so a
        // load is one 128-byte line from global memory and conflict-free from shared memory -- and the chunk's
        // keep-bits word is the warp's ballot.  (One 128-byte chunk per lane, the first layout, made every load
        // touch 32 lines, or hit one bank 32 times: 1.6 us of the prologue.)
        float tau = 0.f;
        const float kNoNeuron = __int_as_float(0x7fc00000);  // NaN: no threshold keeps a position past d_ff
#pragma unroll
        for (int bt = 0; bt < kMaxBatches; ++bt) {
            bal[bt] = 0u;
            if (bt >= n_batches) continue;  // uniform
            const int q0 = bt * kFfnThreads + warp * kWarp;  // the warp's first chunk of this batch
            const bool any = q0 < chunks;                    // warp-uniform: warps past the vector's end do nothing
            // all 32 chunks whole and inside the vector: no per-element checks, constant offsets
            const bool whole = q0 + kWarp <= chunks && (q0 + kWarp) * kWarp <= F;
            float v[kWarp];
            if (!bulk_scores && any) {
                if (whole) {
                    const float *src = p.scores + (size_t)q0 * kWarp + lane;
#pragma unroll
                    for (int c = 0; c < kWarp; ++c) v[c] = ld_keep(src + c * kWarp, keep_policy);
                } else {
#pragma unroll
                    for (int c = 0; c < kWarp; ++c) {
                        const int j = (q0 + c) * kWarp + lane;
                        v[c] = (q0 + c < chunks && j < F) ? ld_keep(p.scores + j, keep_policy) : kNoNeuron;
                    }
                }
            }
            if (bt == 0) {  // the threshold arrives while the score loads are in flight
                __syncthreads();
                tau = s_tau;
                if (bulk_scores && !mbar_wait(sbar, 0) && tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
            }
            if (!any) continue;
            if (bulk_scores) {
                if (whole) {
                    const uint32_t src = ring + (uint32_t)(q0 * kWarp + lane) * 4u;
#pragma unroll
                    for (int c = 0; c < kWarp; ++c) v[c] = lds_f32(src + (uint32_t)c * (kWarp * 4u));
                } else {
#pragma unroll
                    for (int c = 0; c < kWarp; ++c) {
                        const int j = (q0 + c) * kWarp + lane;
                        v[c] = (q0 + c < chunks && j < F) ? lds_f32(ring + (uint32_t)j * 4u) : kNoNeuron;
                    }
                }
            }
            // lane c keeps the word of chunk q0 + c: thread tid owns chunk bt * kFfnThreads + tid, as below
#pragma unroll
            for (int c = 0; c < kWarp; ++c) {
                const unsigned w = __ballot_sync(0xffffffffu, v[c] >= tau);
                if (lane == c) bal[bt] = w;
            }
        }
    }
    int first_rank[kMaxBatches];  // rank of this thread's chunk's first kept neuron
    int n_act = 0;
#pragma unroll
    for (int bt = 0; bt < kMaxBatches; ++bt) {
        first_rank[bt] = 0;
        if (bt >= n_batches) continue;  // uniform
        const int cnt = __popc(bal[bt]);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < kWarp; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (bt > 0) __syncthreads();  // s_wtot free again
        if (lane == kWarp - 1) s_wtot[warp] = incl;
        __syncthreads();
        int wbase = 0, btot = 0;
#pragma unroll
        for (int w = 0; w < kFfnWarps; ++w) {
            const int v = s_wtot[w];
            wbase += (w < warp) ? v : 0;
            btot += v;
        }
        first_rank[bt] = n_act + wbase + incl - cnt;
        n_act += btot;
    }
    const int r0 = split_at(n_act, cta, n_ctas);
    const int r1 = split_at(n_act, cta + 1, n_ctas);
    const int m0 = split_at(F, cta, n_ctas);  // slice of the mask this CTA writes
    const int m1 = split_at(F, cta + 1, n_ctas);
    // Only two or three chunks hold this CTA's share: the warp that owns such a chunk writes it out
    // with one lane per neuron.
#pragma unroll
    for (int bt = 0; bt < kMaxBatches; ++bt) {
        if (bt >= n_batches) continue;  // uniform
        const int q = bt * kFfnThreads + tid;
        const int fr = first_rank[bt];
        const bool in_share = q < chunks && fr < r1 && fr + __popc(bal[bt]) > r0;
        const bool in_mask = p.mask_out && q < chunks && q * kWarp < m1 && q * kWarp + kWarp > m0;
        unsigned todo = __ballot_sync(0xffffffffu, in_share || in_mask);
        while (todo) {
            const int t = __ffs(todo) - 1;
            todo &= todo - 1;
            const unsigned wb = __shfl_sync(0xffffffffu, bal[bt], t);
            const int wfr = __shfl_sync(0xffffffffu, fr, t);
            const int j = (bt * kFfnThreads + (warp * kWarp + t)) * kWarp + lane;
            const bool keep = (wb >> lane) & 1u;
            const int rank = wfr + __popc(wb & ((1u << lane) - 1u));
            if (keep && rank >= r0 && rank < r1 && guard_slot(rank, F, p.status)) {
                s_list[rank - r0] = j;
                if (p.idx_out) p.idx_out[rank] = j;
            }
            if (p.mask_out && j >= m0 && j < m1) p.mask_out[j] = keep ? 1 : 0;
        }
    }
    n_act_o = n_act;
    r0_o = r0;
    r1_o = r1;
    }  // scores + threshold
    const int n_act = n_act_o, r0 = r0_o, r1 = r1_o;
    if (p.count_out && cta == 0 && tid == 0) *p.count_out = n_act;
    const int my_n = r1 - r0;
    if (n_act == 0) {
        // Nothing is kept (every CTA sees the same count): y = 0, written slice by slice, and there are
        // no partial sums to combine, so the grid barrier is skipped as well.
        const int ng = d / 4;  // output in groups of 4 columns
        const int q0 = split_at(ng, cta, n_ctas), q1 = split_at(ng, cta + 1, n_ctas);
        for (int q = q0 + tid; q < q1; q += kFfnThreads) {
            if (p.y_dtype == CLADA_F32)
                reinterpret_cast<float4 *>(p.y)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            else
                reinterpret_cast<uint2 *>(p.y)[q] = make_uint2(0u, 0u);
        }
        return;
    }
    __syncthreads();  // s_list and the mbarriers are ready

    bool timed_out = false;

    if (warp == kConsWarps) {
        // ---- producer ------------------------------------------------------------------------
        if (lane == 0) {
            const char *Wg = static_cast<const char *>(p.w_gate);
            const char *Wu = static_cast<const char *>(p.w_up);
            const char *Wd = static_cast<const char *>(p.w_down_t);
            const uint64_t stream_policy = policy_evict_first();
            int issued = 0;
            int s = 0;            // ring position and the parity of its current use, kept incrementally
            uint32_t par = 0;
            for (int i = 0; i < my_n; ++i) {
                if (!mbar_wait(empty0 + 8 * s, par ^ 1)) {  // a fresh barrier passes parity 1 at once
                    timed_out = true;
                    break;
                }
                const size_t off = (size_t)guard_row(s_list[i], p.d_ff, p.status) * row_bytes;
                const uint32_t dst = ring + (uint32_t)s * stage_bytes, bar = full0 + 8 * s;
                mbar_expect_tx(bar, stage_bytes);
                bulk_load_row_hint(dst, Wg + off, row_bytes, bar, stream_policy);
                if (GATED) bulk_load_row_hint(dst + row_bytes, Wu + off, row_bytes, bar, stream_policy);
                bulk_load_row_hint(dst + down_off, Wd + off, row_bytes, bar, stream_policy);
                issued = i + 1;
                if (++s == n_stages) {
                    s = 0;
                    par ^= 1;
                }
            }
            // Never leave with copies in flight: the last use of every stage must have landed.
            for (int i = max(0, issued - n_stages); i < issued; ++i)
                if (!mbar_wait(full0 + 8 * (i % n_stages), (i / n_stages) & 1)) timed_out = true;
        }
    } else {
        // ---- consumers -----------------------------------------------------------------------
        float2 acc[NV][P];
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int e = 0; e < P; ++e) acc[i][e] = make_float2(0.f, 0.f);
        int cs = 0;           // ring position of the next neuron to consume, and the parity of its use
        uint32_t cpar = 0;
        consume_share<T, NV, GATED, GROUPS>(my_n, p.act, ring, stage_bytes, row_bytes, down_off, full0, empty0, n_stages,
                                            cs, cpar, xr, vok, acc, s_dot, timed_out);
        // partial y of this consumer group
        float *mine = p.partials + ((size_t)cta * GROUPS + grp) * d;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            if (!vok[i]) continue;
            float4 *dst = reinterpret_cast<float4 *>(mine + (size_t)(gt + i * GT) * E);
#pragma unroll
            for (int e = 0; e < P; e += 2)
                dst[e / 2] = make_float4(acc[i][e].x, acc[i][e].y, acc[i][e + 1].x, acc[i][e + 1].y);
        }
    }
    if (timed_out && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);

    // ---- epilogue: grid barrier, deterministic column reduction ---------------------------------
    if (!grid_barrier(p.ctrl, (unsigned)n_ctas, kConsumers)) {
        if (tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }
    // columns in groups of 4 (float4); a warp sums one group: lane l adds partial rows l, l+32, ... (one row
    // per CTA and consumer group) in order (five loads in flight at a time), then the 32 lane sums combine by
    // butterfly.
    const int ngroups = d / 4;
    const int n_rows = n_ctas * GROUPS;
    for (int q = cta + warp * n_ctas; q < ngroups; q += n_ctas * kFfnWarps) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int rb = 0; rb < n_rows; rb += 5 * kWarp) {
            float4 v[5];
#pragma unroll
            for (int u = 0; u < 5; ++u) {
                const int r = rb + u * kWarp + lane;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (r < n_rows) v[u] = __ldcg(reinterpret_cast<const float4 *>(p.partials + (size_t)r * d) + q);
            }
#pragma unroll
            for (int u = 0; u < 5; ++u) {
                s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w;
            }
        }
        s.x = warp_sum(s.x); s.y = warp_sum(s.y); s.z = warp_sum(s.z); s.w = warp_sum(s.w);
        if (lane == 0) {
            if (p.y_dtype == CLADA_F32) {
                reinterpret_cast<float4 *>(p.y)[q] = s;
            } else {
                reinterpret_cast<uint2 *>(p.y)[q] = pack4_16bit(p.y_dtype, s);
            }
        }
    }
}

// ---- host side ------------------------------------------------------------------------------

template <typename T, int NV, bool GATED, int GROUPS>
static int launch_variant(const FfnParams &p, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_kernel<T, NV, GATED, GROUPS>;
    const size_t stage_bytes = (GATED ? 3 : 2) * (size_t)(p.d_model / E) * 16;
    const size_t tail = (2 * kMaxStages + 1) * sizeof(uint64_t) + (size_t)((p.d_ff + 31) / 32) * sizeof(unsigned) +
                        (size_t)(p.d_ff / di.num_sms + 2) * sizeof(int);
    const size_t budget = (size_t)di.max_smem_optin - 2048;  // leave room for the static arrays
    if (budget < tail + G * stage_bytes) return CLADA_ERR_UNSUPPORTED;  // a group needs G stages at once
    int n_stages = (int)((budget - tail) / stage_bytes);
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    const size_t smem = (size_t)n_stages * stage_bytes + tail;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
        configured[di.device & 63] = true;
    }
    FfnParams params = p;
    int stages_arg = n_stages;
    void *args[] = {&params, &stages_arg};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(di.num_sms);  // one CTA per SM
    cfg.blockDim = dim3(kFfnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident: the grid barrier cannot starve
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // hide the launch latency
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    CLADA_CUDA_TRY(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kern), args));
    return CLADA_OK;
}

template <typename T>
static int launch_ffn(const FfnParams &p, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    const int vpr = p.d_model / E;
    if (p.d_ff > kMaxBatches * kWarp * kFfnThreads) return CLADA_ERR_UNSUPPORTED;
    const bool gated = act_is_gated(p.act);
    if (vpr <= kConsumers / 2)  // narrow rows: two consumer groups of 256 threads, one vector per thread
        return gated ? launch_variant<T, 1, true, 2>(p, st) : launch_variant<T, 1, false, 2>(p, st);
    if (vpr <= kConsumers) return gated ? launch_variant<T, 1, true, 1>(p, st) : launch_variant<T, 1, false, 1>(p, st);
    if (vpr <= 2 * kConsumers)  // wide rows: two vectors per thread
        return gated ? launch_variant<T, 2, true, 1>(p, st) : launch_variant<T, 2, false, 1>(p, st);
    return CLADA_ERR_UNSUPPORTED;
}

int launch_ffn_single(const FfnParams &p, int dtype, cudaStream_t st) {
    return dtype == CLADA_F32    ? launch_ffn<float>(p, st)
           : dtype == CLADA_BF16 ? launch_ffn<__nv_bfloat16>(p, st)
                                 : launch_ffn<__half>(p, st);
}

}  // namespace clada
