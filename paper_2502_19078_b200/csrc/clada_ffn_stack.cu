// Sparse gated FFN of one decode token through a whole stack of layers in ONE persistent launch
// (Algorithm 2, generation phase: the loop over layers inside a decode step):
//   for l = 0 .. L-1:  kept_l = { j : A_lj >= tau_l },
//                      y_l = sum_{j in kept_l} silu(w_gate_lj . x_l) (w_up_lj . x_l) w_down_t_l[j,:]
//
// A launch per layer pays, per layer, for what does not move weight bytes: the launch ramp, the score
// test, the first rows' latency, the slowest CTA's tail, a grid barrier and the column sums.  Here the
// weight stream never stops at a layer boundary.  One cooperative CTA per SM, as in the per-layer kernel:
//   scanner   one warp builds the kept lists: it tests a layer's scores against its threshold and writes
//             this CTA's equal share of the kept neurons into one of four list buffers, up to four layers
//             ahead of the layer being streamed, so the score test is never on anybody's path.
//   producer  one thread walks layer after layer: the layer's x (one ring stage), then the three rows of
//             every kept neuron of this CTA's share, as bulk asynchronous copies into the ring.  It runs
//             ahead of the consumers by the ring's depth, across layer boundaries.
//   consumers 512 threads.  Per layer: x from its stage into registers, the share's neurons four per
//             CTA-wide reduction, the CTA's partial y to global memory, a grid barrier, then a slice of
//             columns summed over all CTAs' partials in CTA order.  While they are at the barrier the
//             copies of the next layer's rows go on into the ring.
// Partial rows are double buffered by barrier number, every wait is bounded, and the summation order is
// that of the per-layer kernel: results repeat bit for bit and equal the per-layer call's.
#include <math.h>

#include "common.cuh"
#include "ffn_common.cuh"

namespace clada {

constexpr int kMaxStackLayers = 128;  // layers per launch (their weight pointers travel as kernel parameters)
constexpr int kStackMaxDff = 65536;    // the scanner parks one keep word per 32 neurons in shared memory

struct StackLayers {
    const void *w[kMaxStackLayers][3];  // w_gate, w_up, w_down_t of every layer
};

struct StackParams {
    const char *x;        // layer l reads x + l * x_stride (bytes)
    size_t x_stride;
    const float *scores;  // layer l: scores + l * d_ff
    const float *tau;     // layer l: tau[l * tau_stride]
    long long tau_stride;
    char *y;              // layer l writes y + l * y_stride (bytes)
    size_t y_stride;
    int y_dtype;
    float *partials;      // [2][gridDim.x][consumer groups][d_model]
    const unsigned *keep_words;  // [L][chunks of 32 neurons] keep bits A_lj >= tau_l from keep_words_kernel, or null:
                                 // the scanner tests the score vectors itself
    WsCtrl *ctrl;
    int32_t *status;
    int d_model, d_ff, L;
    int act;
};

// Tracing build (-DCLADA_STACK_TRACE, off by default): every CTA records %globaltimer stamps per layer into a
// caller-provided device buffer [n_ctas][L][kTraceSlots] set with clada_stack_trace_buffer().  Slots: 0 layer
// start (x in registers), 1 rows consumed, 2 arrived at the barrier, 3 unused, 4 barrier passed,
// 5 column sums written, 6 producer's first copy of the layer, 7 its last, 8 ns the producer waited for free
// stages, 9 ns consumer thread 0 waited for full stages.
#ifdef CLADA_STACK_TRACE
constexpr int kTraceSlots = 10;
__device__ unsigned long long *g_stack_trace = nullptr;
__device__ __forceinline__ unsigned long long trace_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
#define STACK_TRACE(l, slot, value)                                                                   \
    do {                                                                                              \
        if (g_stack_trace) g_stack_trace[((size_t)blockIdx.x * p.L + (l)) * kTraceSlots + (slot)] = (value); \
    } while (0)
#else
#define STACK_TRACE(l, slot, value) \
    do {                            \
    } while (0)
#endif

__device__ __forceinline__ int stack_split_at(int n, int c, int n_ctas) {
    return (int)(((unsigned)n * (unsigned)c) / (unsigned)n_ctas);
}

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

constexpr int kEpiWarps = 2;
constexpr int kStackThreads = kConsumers + 64 + kEpiWarps * kWarp;  // consumers, producer, scanner, epilogue warps
constexpr int kScanWarp = kConsWarps + 1;
constexpr int kEpiWarp = kConsWarps + 2;  // first epilogue warp
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 2, %0;" ::"n"(kEpiWarps * kWarp) : "memory"); }
constexpr int kListBufs = 4;                    // kept lists are built up to four layers ahead

// Score test of one layer by ONE warp (the scanner): keep bits A_j >= tau, one ballot per 32-neuron chunk with
// coalesced loads (32 chunks = 1024 neurons per round, all loads of a round in flight together), the chunk words
// parked in keep[]; then the ranks again from the parked words, and this CTA's equal share [r0, r1) of the kept
// neurons, ascending, written to list[].  Returns the layer's kept count; *my_n = r1 - r0.
__device__ __forceinline__ int scan_share_list(const float *__restrict__ scores, const unsigned *__restrict__ words,
                                               const float tau, const int F, const int cta, const int n_ctas,
                                               int *list, unsigned *keep, int *my_n, const uint64_t keep_policy) {
    const int lane = threadIdx.x & 31;
    const int chunks = (F + kWarp - 1) / kWarp;
    const float kNoNeuron = __int_as_float(0x7fc00000);  // NaN: no threshold keeps a position past d_ff
    int n_act = 0;
    if (words) {  // the layer's keep words are there already (4 bytes per chunk instead of 128 bytes of scores)
        for (int q0 = 0; q0 < chunks; q0 += 4 * kWarp) {
            unsigned w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) w[u] = q0 + u * kWarp + lane < chunks ? __ldcg(words + q0 + u * kWarp + lane) : 0u;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (q0 + u * kWarp + lane < chunks) keep[q0 + u * kWarp + lane] = w[u];
                n_act += __popc(w[u]);
            }
        }
    } else
    for (int q0 = 0; q0 < chunks; q0 += kWarp) {
        const bool whole = q0 + kWarp <= chunks && (q0 + kWarp) * kWarp <= F;
        float v[kWarp];
        if (whole) {
            const float *src = scores + (size_t)q0 * kWarp + lane;
#pragma unroll
            for (int c = 0; c < kWarp; ++c) v[c] = ld_keep(src + c * kWarp, keep_policy);
        } else {
#pragma unroll
            for (int c = 0; c < kWarp; ++c) {
                const int j = (q0 + c) * kWarp + lane;
                v[c] = (q0 + c < chunks && j < F) ? ld_keep(scores + j, keep_policy) : kNoNeuron;
            }
        }
        unsigned mine = 0u;
#pragma unroll
        for (int c = 0; c < kWarp; ++c) {
            const unsigned w = __ballot_sync(0xffffffffu, v[c] >= tau);
            if (lane == c) mine = w;  // lane c keeps the word of chunk q0 + c
        }
        if (q0 + lane < chunks) keep[q0 + lane] = mine;
        n_act += __popc(mine);
    }
    n_act = warp_sum(n_act);
    __syncwarp();
    const int r0 = stack_split_at(n_act, cta, n_ctas);
    const int r1 = stack_split_at(n_act, cta + 1, n_ctas);
    int base = 0;
    for (int q0 = 0; q0 < chunks && base < r1; q0 += kWarp) {
        const unsigned w = q0 + lane < chunks ? keep[q0 + lane] : 0u;
        const int cnt = __popc(w);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < kWarp; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const int fr = base + incl - cnt;  // rank of this chunk's first kept neuron
        if (fr < r1 && fr + cnt > r0) {    // at most a few chunks hold the share: their lanes walk the bits
            unsigned rest = w;
            int rank = fr;
            while (rest) {
                const int b = __ffs(rest) - 1;
                rest &= rest - 1;
                if (rank >= r0 && rank < r1) list[rank - r0] = (q0 + lane) * kWarp + b;
                ++rank;
            }
        }
        base += __shfl_sync(0xffffffffu, incl, kWarp - 1);
    }
    *my_n = r1 - r0;
    return n_act;
}

template <typename T, int NV, bool GATED, int GROUPS>
__global__ void __launch_bounds__(kStackThreads, 1)
sparse_ffn_stack_kernel(const StackParams p, const __grid_constant__ StackLayers lay, const int n_stages,
                        const int list_cap) {
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = Pairs<T>::kPairs;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff, d = p.d_model, L = p.L;
    const int vpr = d / E;  // 16-byte vectors per row
    const uint32_t row_bytes = (uint32_t)vpr * 16u;
    constexpr uint32_t kRows = GATED ? 3u : 2u;
    const uint32_t stage_bytes = kRows * row_bytes;
    const uint32_t down_off = (kRows - 1u) * row_bytes;

    // dynamic shared memory: ring | full[kMaxStages] | empty[kMaxStages] | list-ready[4] | list-free[4] |
    // lists[4][list_cap] | keep words of the layer being scanned
    const uint32_t ring = smem_u32(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)n_stages * stage_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages);
    const uint32_t lready0 = smem_u32(bars + 2 * kMaxStages);             // scanner -> producer, consumers
    const uint32_t lfree0 = smem_u32(bars + 2 * kMaxStages + kListBufs);  // producer, consumers, epilogue -> scanner
    const uint32_t pdone = smem_u32(bars + 2 * kMaxStages + 2 * kListBufs);      // consumers -> epilogue: partial row stored
    const uint32_t bdone = smem_u32(bars + 2 * kMaxStages + 2 * kListBufs + 1);  // epilogue -> consumers: barrier passed
    int *s_list = reinterpret_cast<int *>(bars + 2 * kMaxStages + 2 * kListBufs + 2);
    unsigned *s_keep = reinterpret_cast<unsigned *>(s_list + kListBufs * list_cap);
    __shared__ int s_nact[kListBufs], s_myn[kListBufs];  // per list buffer: the layer's kept count, this CTA's share
    __shared__ int s_cur[2][3];                          // consumers' copy for the current layer (+ give-up flag)
    __shared__ int s_ecur[2][3];                         // the epilogue warps' copy
    __shared__ __align__(16) float s_dot[kDotFloats];

    pdl_launch_dependents();
    if (tid == kConsumers) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full0 + 8 * s, 1);            // the producer's expect_tx arrival
            mbar_init(empty0 + 8 * s, kConsWarps / GROUPS);  // one arrival per warp of the group that owns the stage
        }
        for (int k = 0; k < kListBufs; ++k) {
            mbar_init(lready0 + 8 * k, 1);  // the scanner
            mbar_init(lfree0 + 8 * k, 3);   // the producer, consumer thread 0 and the epilogue warp
        }
        mbar_init(pdone, kConsWarps);
        mbar_init(bdone, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();      // everything below may read what the previous kernel wrote
    __syncthreads();  // the mbarriers exist

    bool timed_out = false;

    if (warp == kScanWarp) {
        // ---- scanner: the kept list of every layer, up to four layers ahead of its use --------------------
        const uint64_t keep_policy = policy_evict_last();
        for (int l = 0; l < L; ++l) {
            const int k = l & (kListBufs - 1);
            // buffer k last held layer l - 4: the producer has issued its rows, the consumers have its counts
            if (l >= kListBufs && !mbar_wait(lfree0 + 8 * k, (uint32_t)((l >> 2) - 1) & 1u)) {
                timed_out = true;
                break;
            }
            const float tau = ld_keep(p.tau + (size_t)l * p.tau_stride, keep_policy);
            int my_n;
            const int n_act = scan_share_list(p.scores + (size_t)l * F,
                                              p.keep_words ? p.keep_words + (size_t)l * ((F + kWarp - 1) / kWarp) : nullptr,
                                              tau, F, cta, n_ctas, s_list + k * list_cap, s_keep, &my_n, keep_policy);
            if (lane == 0) {
                s_nact[k] = n_act;
                s_myn[k] = my_n;
            }
            __syncwarp();  // every lane's list entries are written before lane 0 announces them
            if (lane == 0) mbar_arrive(lready0 + 8 * k);
        }
        if (timed_out && lane == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }

    if (warp >= kEpiWarp) {
        // ---- epilogue warps: grid barrier and column sums of every layer, off the consumers' path ----------
        // Per layer that kept something (barrier number e): wait until this CTA's consumers have stored their
        // partial row, arrive at the device-wide count, wait for every CTA, tell the consumers (who may then
        // reuse the other partial buffer), and sum this CTA's slice of columns over all partial rows in CTA
        // order.  A layer that kept nothing gets its zeros from here.
        const int et = tid - kEpiWarp * kWarp, ew = warp - kEpiWarp;
        unsigned epoch = 0;
        const int ngroups = d / 4;
        for (int l = 0; l < L; ++l) {
            // the first epilogue thread takes the layer's kept count (and whether it gave up waiting) for all
            if (et == 0) {
                const int k = l & (kListBufs - 1);
                if (!timed_out && !mbar_wait(lready0 + 8 * k, (uint32_t)(l >> 2) & 1u)) timed_out = true;
                s_ecur[l & 1][0] = timed_out ? 0 : s_nact[k];
                s_ecur[l & 1][1] = timed_out ? 1 : 0;
                mbar_arrive(lfree0 + 8 * k);
            }
            epilogue_sync();
            const int n_act = s_ecur[l & 1][0];
            if (s_ecur[l & 1][1]) timed_out = true;
            char *yl = p.y + (size_t)l * p.y_stride;
            if (n_act == 0) {
                const int q0 = stack_split_at(ngroups, cta, n_ctas), q1 = stack_split_at(ngroups, cta + 1, n_ctas);
                for (int q = q0 + et; q < q1; q += kEpiWarps * kWarp) {
                    if (p.y_dtype == CLADA_F32)
                        reinterpret_cast<float4 *>(yl)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    else
                        reinterpret_cast<uint2 *>(yl)[q] = make_uint2(0u, 0u);
                }
                continue;
            }
            if (et == 0) {
                if (!timed_out && !mbar_wait(pdone, epoch & 1u)) timed_out = true;
                // release at device scope: the consumers' row (ordered before this by their arrivals on the
                // shared-memory barrier) is visible to whoever sees the count
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(&p.ctrl->arrive) : "memory");
                STACK_TRACE(l, 2, trace_now());
                const unsigned target = (epoch + 1u) * (unsigned)n_ctas;
                unsigned spins = 0, seen;
                for (;;) {
                    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(seen) : "l"(&p.ctrl->arrive) : "memory");
                    if (seen >= target) break;
                    if (timed_out || ++spins > kBarrierSpinLimit) {
                        timed_out = true;
                        break;
                    }
                }
                STACK_TRACE(l, 4, trace_now());
                s_ecur[l & 1][2] = timed_out ? 1 : 0;
                mbar_arrive(bdone);  // every CTA has arrived: all column sums of the layer before are done
            }
            epilogue_sync();
            if (s_ecur[l & 1][2]) timed_out = true;
            const int n_rows = n_ctas * GROUPS;  // one partial row per (CTA, consumer group)
            const float *part = p.partials + (size_t)(epoch & 1u) * n_rows * d;
            ++epoch;
            // columns in groups of 4 (float4), a warp per group: lane l adds partial rows l, l+32, ... in order
            // (five loads in flight at a time), then the 32 lane sums combine by butterfly.
            for (int q = cta + ew * n_ctas; q < ngroups; q += kEpiWarps * n_ctas) {
                float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int rb = 0; rb < n_rows; rb += 5 * kWarp) {
                    float4 v[5];
#pragma unroll
                    for (int u = 0; u < 5; ++u) {
                        const int r = rb + u * kWarp + lane;
                        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (r < n_rows) v[u] = __ldcg(reinterpret_cast<const float4 *>(part + (size_t)r * d) + q);
                    }
#pragma unroll
                    for (int u = 0; u < 5; ++u) {
                        s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w;
                    }
                }
                s.x = warp_sum(s.x); s.y = warp_sum(s.y); s.z = warp_sum(s.z); s.w = warp_sum(s.w);
                if (lane == 0) {
                    if (p.y_dtype == CLADA_F32)
                        reinterpret_cast<float4 *>(yl)[q] = s;
                    else
                        reinterpret_cast<uint2 *>(yl)[q] = pack4_16bit(p.y_dtype, s);
                }
            }
            if (et == 0) STACK_TRACE(l, 5, trace_now());
        }
        epilogue_sync();  // every epilogue warp has read its last partial rows
        if (et == 0) {
            if (timed_out) {
                if (p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
            } else {
                // The counters go back to zero for the next launch: the last CTA out resets them (every CTA
                // has then seen its last barrier complete).
                const unsigned left = atomicAdd(&p.ctrl->depart, 1u);
                if (left == (unsigned)n_ctas - 1u) {
                    p.ctrl->arrive = 0;
                    p.ctrl->depart = 0;
                    __threadfence();
                }
            }
        }
        return;
    }

    if (warp == kConsWarps) {
        // ---- producer -----------------------------------------------------------------------------
        if (lane == 0) {
            const uint64_t stream_policy = policy_evict_first();
            const uint64_t keep_policy = policy_evict_last();
            long long issued = 0;
            int s = 0;  // ring position and the parity of its current use, kept incrementally
            uint32_t par = 0;
            for (int l = 0; l < L && !timed_out; ++l) {
                const int k = l & (kListBufs - 1);
                if (!mbar_wait(lready0 + 8 * k, (uint32_t)(l >> 2) & 1u)) {  // layer l's list is in buffer k
                    timed_out = true;
                    break;
                }
                const int my_n = s_myn[k];
                if (s_nact[k] == 0 || my_n == 0) {  // nothing of this layer for this CTA
                    mbar_arrive(lfree0 + 8 * k);
                    continue;
                }
                const int *list = s_list + k * list_cap;
                const char *Wg = static_cast<const char *>(lay.w[l][0]);
                const char *Wu = static_cast<const char *>(lay.w[l][1]);
                const char *Wd = static_cast<const char *>(lay.w[l][2]);
#ifdef CLADA_STACK_TRACE
                unsigned long long waited = 0;
#endif
                for (int i = -1; i < my_n; ++i) {  // i = -1: the layer's x takes a stage of its own
#ifdef CLADA_STACK_TRACE
                    const unsigned long long w0 = trace_now();
#endif
                    if (!mbar_wait(empty0 + 8 * s, par ^ 1)) {  // a fresh barrier passes parity 1 at once
                        timed_out = true;
                        break;
                    }
#ifdef CLADA_STACK_TRACE
                    waited += trace_now() - w0;
                    if (i == -1) STACK_TRACE(l, 6, trace_now());
#endif
                    const uint32_t dst = ring + (uint32_t)s * stage_bytes, bar = full0 + 8 * s;
                    if (i < 0) {
                        mbar_expect_tx(bar, row_bytes);
                        bulk_load_row_hint(dst, p.x + (size_t)l * p.x_stride, row_bytes, bar, keep_policy);
                    } else {
                        const size_t off = (size_t)guard_row(list[i], p.d_ff, p.status) * row_bytes;
                        mbar_expect_tx(bar, stage_bytes);
                        bulk_load_row_hint(dst, Wg + off, row_bytes, bar, stream_policy);
                        if (GATED) bulk_load_row_hint(dst + row_bytes, Wu + off, row_bytes, bar, stream_policy);
                        bulk_load_row_hint(dst + down_off, Wd + off, row_bytes, bar, stream_policy);
                    }
                    ++issued;
                    if (++s == n_stages) {
                        s = 0;
                        par ^= 1;
                    }
                }
#ifdef CLADA_STACK_TRACE
                STACK_TRACE(l, 7, trace_now());
                STACK_TRACE(l, 8, waited);
#endif
                if (!timed_out) mbar_arrive(lfree0 + 8 * k);  // the list has been read to its end
            }
            // Never leave with copies in flight: the last use of every stage must have landed.
            const long long first = issued > n_stages ? issued - n_stages : 0;
            for (long long i = first; i < issued; ++i)
                if (!mbar_wait(full0 + 8 * (int)(i % n_stages), (uint32_t)(i / n_stages) & 1u)) timed_out = true;
            if (timed_out && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        }
        return;
    }

    // ---- consumers ------------------------------------------------------------------------------------
    constexpr int GT = kConsumers / GROUPS;  // threads per consumer group
    const int grp = tid / GT, gt = tid - grp * GT;
    bool vok[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) vok[i] = gt + i * GT < vpr;
    int cs = 0;  // ring position of the next stage to consume, and the parity of its use
    uint32_t cpar = 0;
    unsigned epoch = 0;  // grid barriers passed so far (layers that kept something)
    for (int l = 0; l < L; ++l) {
        // Thread 0 takes the layer's counts from the scanner's buffer and hands them (and whether it gave up
        // waiting) to the others, so that all consumers take the same path through the layer.
        if (tid == 0) {
            const int k = l & (kListBufs - 1);
            if (!timed_out && !mbar_wait(lready0 + 8 * k, (uint32_t)(l >> 2) & 1u)) timed_out = true;
            s_cur[l & 1][0] = timed_out ? 0 : s_nact[k];
            s_cur[l & 1][1] = timed_out ? 0 : s_myn[k];
            s_cur[l & 1][2] = timed_out ? 1 : 0;
            mbar_arrive(lfree0 + 8 * k);  // the consumers are done with this buffer
        }
        consumer_sync();
        const int n_act = s_cur[l & 1][0], my_n = s_cur[l & 1][1];
        if (s_cur[l & 1][2]) timed_out = true;
        if (n_act == 0) continue;  // nothing is kept (every CTA sees the same count): the epilogue warps write y = 0
        // x of this thread's columns, from the stage the producer filled ahead of the layer's rows
        float2 xr[NV][P];
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int e = 0; e < P; ++e) xr[i][e] = make_float2(0.f, 0.f);
        if (my_n > 0) {
            if (!timed_out && !mbar_wait(full0 + 8 * cs, cpar)) timed_out = true;
            const uint32_t xa = ring + (uint32_t)cs * stage_bytes;
#pragma unroll
            for (int i = 0; i < NV; ++i)
                if (vok[i]) Pairs<T>::unpack(lds128(xa + (uint32_t)(gt + i * GT) * 16u), xr[i]);
            if (GROUPS > 1) consumer_sync();  // both groups have read x; the first group's warps hand the stage back
            __syncwarp();
            if (lane == 0 && grp == 0) mbar_arrive(empty0 + 8 * cs);
            if (++cs == n_stages) {
                cs = 0;
                cpar ^= 1;
            }
        }
        float2 acc[NV][P];
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int e = 0; e < P; ++e) acc[i][e] = make_float2(0.f, 0.f);
#ifdef CLADA_STACK_TRACE
        unsigned long long cwait = 0;
        if (tid == 0) STACK_TRACE(l, 0, trace_now());
        consume_share<T, NV, GATED, GROUPS>(my_n, p.act, ring, stage_bytes, row_bytes, down_off, full0, empty0, n_stages,
                                            cs, cpar, xr, vok, acc, s_dot, timed_out, &cwait);
        if (tid == 0) {
            STACK_TRACE(l, 1, trace_now());
            STACK_TRACE(l, 9, cwait);
        }
#else
        consume_share<T, NV, GATED, GROUPS>(my_n, p.act, ring, stage_bytes, row_bytes, down_off, full0, empty0, n_stages,
                                            cs, cpar, xr, vok, acc, s_dot, timed_out);
#endif
        // Partial y of this consumer group, into the buffer of this barrier number.  The buffer was last read
        // for the column sums of the barrier two back; all of those are done once every CTA has passed the
        // barrier before this one, which the epilogue warps report.
        if (epoch >= 1u && !timed_out && !mbar_wait(bdone, (epoch - 1u) & 1u)) timed_out = true;
        float *mine = p.partials + (((size_t)(epoch & 1u) * n_ctas + cta) * GROUPS + grp) * d;
        ++epoch;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            if (!vok[i]) continue;
            float4 *dst = reinterpret_cast<float4 *>(mine + (size_t)(gt + i * GT) * E);
#pragma unroll
            for (int e = 0; e < P; e += 2)
                dst[e / 2] = make_float4(acc[i][e].x, acc[i][e].y, acc[i][e + 1].x, acc[i][e + 1].y);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(pdone);  // this warp's part of the row is stored: on to the next layer
    }
    if (timed_out && tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
}

// Ring stages and dynamic shared memory of a launch; n_stages < GS means the kernel cannot take the layer
// (a reduction group holds GS stages at once; the x stage is handed back before the group starts).
static void stack_smem_plan(const DeviceInfo &di, int d_model, int d_ff, int dtype, bool gated, int *n_stages,
                            int *list_cap, size_t *smem, size_t *budget) {
    const size_t stage_bytes = (gated ? 3 : 2) * (size_t)d_model * elem_size(dtype);
    *list_cap = d_ff / di.num_sms + 2;
    const size_t tail = (2 * kMaxStages + 2 * kListBufs + 2) * sizeof(uint64_t) + kListBufs * (size_t)*list_cap * sizeof(int) +
                        (size_t)((d_ff + 31) / 32) * sizeof(unsigned);
    *budget = (size_t)di.max_smem_optin - 2048;  // leave room for the static arrays
    int n = *budget > tail ? (int)((*budget - tail) / stage_bytes) : 0;
    if (n > kMaxStages) n = kMaxStages;
    *n_stages = n;
    *smem = (size_t)n * stage_bytes + tail;
}

template <typename T, int NV, bool GATED, int GROUPS>
static int launch_stack_variant(const StackParams &p, const StackLayers &lay, int dtype, cudaStream_t st) {
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_stack_kernel<T, NV, GATED, GROUPS>;
    int n_stages, list_cap;
    size_t smem, budget;
    stack_smem_plan(di, p.d_model, p.d_ff, dtype, GATED, &n_stages, &list_cap, &smem, &budget);
    if (n_stages < GS) return CLADA_ERR_UNSUPPORTED;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
        configured[di.device & 63] = true;
    }
    StackParams params = p;
    StackLayers layers = lay;
    int stages_arg = n_stages, cap_arg = list_cap;
    void *args[] = {&params, &layers, &stages_arg, &cap_arg};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(di.num_sms);  // one CTA per SM
    cfg.blockDim = dim3(kStackThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident: the grid barriers cannot starve
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    CLADA_CUDA_TRY(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kern), args));
    return CLADA_OK;
}

template <typename T>
static int launch_stack_typed(const StackParams &p, const StackLayers &lay, int dtype, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    const int vpr = p.d_model / E;
    const bool gated = act_is_gated(p.act);
    if (vpr <= kConsumers / 2)  // narrow rows: two consumer groups of 256 threads, one vector per thread
        return gated ? launch_stack_variant<T, 1, true, 2>(p, lay, dtype, st)
                     : launch_stack_variant<T, 1, false, 2>(p, lay, dtype, st);
    if (vpr <= kConsumers)
        return gated ? launch_stack_variant<T, 1, true, 1>(p, lay, dtype, st)
                     : launch_stack_variant<T, 1, false, 1>(p, lay, dtype, st);
    if (vpr <= 2 * kConsumers)  // wide rows: two vectors per thread
        return gated ? launch_stack_variant<T, 2, true, 1>(p, lay, dtype, st)
                     : launch_stack_variant<T, 2, false, 1>(p, lay, dtype, st);
    return CLADA_ERR_UNSUPPORTED;
}

bool ffn_stack_supported(const clada_layer *layers, int L, int B, size_t ws_bytes) {
    if (B != 1 || L < 2) return false;
    if (layers[0].d_ff > kStackMaxDff) return false;
    for (int l = 1; l < L; ++l)
        if (layers[l].activation != layers[0].activation) return false;
    DeviceInfo di;
    if (device_info(&di) != CLADA_OK) return false;
    int n_stages, list_cap;
    size_t smem, budget;
    stack_smem_plan(di, layers[0].d_model, layers[0].d_ff, layers[0].dtype, act_is_gated(layers[0].activation), &n_stages,
                    &list_cap, &smem, &budget);
    if (n_stages < GS) return false;
    const int vpr = layers[0].d_model / (layers[0].dtype == CLADA_F32 ? 4 : 8);
    return ws_bytes >= kWsCtrlBytes + 2 * (size_t)di.num_sms * ffn_groups(vpr) * layers[0].d_model * sizeof(float);
}

// One sequence through L validated layers of one shape, dtype and FFN form: launches of up to
// kMaxStackLayers layers each.  Strides in bytes (x, y) and elements (tau).
int launch_ffn_stack(const clada_layer *layers, int L, const void *x, size_t x_stride, const float *scores,
                     const float *tau, long long tau_stride, void *y, size_t y_stride, int y_dtype, void *ws,
                     size_t ws_bytes, int32_t *status, cudaStream_t st) {
    DeviceInfo di;
    int rc0 = device_info(&di);
    if (rc0 != CLADA_OK) return rc0;
    // Behind the partial rows, when the workspace has the room: the keep words of every layer of a launch, written
    // by one small kernel before it, so that the scanner warp reads 4 bytes per 32 neurons instead of their scores.
    const int vpr0 = layers[0].d_model / (layers[0].dtype == CLADA_F32 ? 4 : 8);
    const size_t words_at = kWsCtrlBytes + 2 * (size_t)di.num_sms * ffn_groups(vpr0) * layers[0].d_model * sizeof(float);
    const bool have_words =
        ws_bytes >= words_at + keep_words_bytes_of(L < kMaxStackLayers ? L : kMaxStackLayers, layers[0].d_ff);
    for (int l0 = 0; l0 < L; l0 += kMaxStackLayers) {
        const int n = L - l0 < kMaxStackLayers ? L - l0 : kMaxStackLayers;
        StackLayers lay = {};
        for (int l = 0; l < n; ++l) {
            lay.w[l][0] = layers[l0 + l].w_gate;
            lay.w[l][1] = layers[l0 + l].w_up;
            lay.w[l][2] = layers[l0 + l].w_down_t;
        }
        StackParams p;
        p.x = static_cast<const char *>(x) + (size_t)l0 * x_stride;
        p.x_stride = x_stride;
        p.scores = scores + (size_t)l0 * layers[0].d_ff;
        p.tau = tau + (size_t)l0 * tau_stride;
        p.tau_stride = tau_stride;
        p.y = static_cast<char *>(y) + (size_t)l0 * y_stride;
        p.y_stride = y_stride;
        p.y_dtype = y_dtype;
        p.partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
        p.keep_words = nullptr;
        if (have_words) {
            unsigned *words = reinterpret_cast<unsigned *>(static_cast<char *>(ws) + words_at);
            const int rcw = launch_keep_words(p.scores, n, layers[0].d_ff, p.tau, tau_stride, words, st);
            if (rcw != CLADA_OK) return rcw;
            p.keep_words = words;
        }
        p.ctrl = static_cast<WsCtrl *>(ws);
        p.status = status;
        p.d_model = layers[0].d_model;
        p.d_ff = layers[0].d_ff;
        p.L = n;
        p.act = layers[0].activation;
        const int rc = layers[0].dtype == CLADA_F32    ? launch_stack_typed<float>(p, lay, CLADA_F32, st)
                       : layers[0].dtype == CLADA_BF16 ? launch_stack_typed<__nv_bfloat16>(p, lay, CLADA_BF16, st)
                                                       : launch_stack_typed<__half>(p, lay, CLADA_F16, st);
        if (rc != CLADA_OK) return rc;
    }
    return CLADA_OK;
}

}  // namespace clada

#ifdef CLADA_STACK_TRACE
// Tracing build only: where the stack kernel writes its time stamps (NULL switches tracing off).
extern "C" int clada_stack_trace_buffer(unsigned long long *buf) {
    CLADA_CUDA_TRY(cudaMemcpyToSymbol(clada::g_stack_trace, &buf, sizeof buf));
    return CLADA_OK;
}
#endif
