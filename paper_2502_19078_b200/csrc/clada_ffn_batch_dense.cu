// Batched decode of up to 16 sequences with per-sequence masks in ONE pass over the layer (16-bit layers):
//   h[b, j] = keep(b, j) * z(w_gate_j . x_b, w_up_j . x_b),   y_b = sum_j h[b, j] * w_down_j,   keep(b, j) = (A_bj >= tau_b)
// (Algorithm 2's masked FFN for every sequence of the batch).  With eight or more sequences that cut 40-50 % each,
// the union of the kept sets is the whole layer, so the layer is streamed densely, every row once, and the masks
// only zero entries of h.  Both contractions run on the 5th-generation tensor cores with the weights as the A
// operand (128 TMEM lanes) and the sequences as the N = 16 columns:
//
//   phase 1   D1[neuron, b] = W_gate/up[neuron, :] . x_b          A = weight rows (K-major), B = x (K-major),
//             K = d_model in blocks of 64 columns, four interleaved K splits in separate TMEM columns (short
//             accumulation chains), summed by the epilogue in fp32.
//   h         one epilogue thread per neuron: gate / up of its 16 sequences from TMEM, neuron value, keep bits from
//             the score vectors, and h split exactly into three 16-bit parts (h = h1 + h2 + h3 to fp32 precision),
//             because the second contraction takes 16-bit operands and y is held to 1e-5.
//   phase 2   D2[column, (part, b)] = sum_j W_down_t[j, column] * h_part[b, j]   A = down rows as they lie in memory
//             (MN-major: columns contiguous), B = the three parts of h as 48 rows (K-major): ONE instruction of N = 48
//             per 16 neurons and 128 columns, the three column groups added by the epilogue.  (Layers so wide that 48
//             TMEM columns per tile do not fit issue three N = 16 instructions into one column group instead.)
//
// Work split: 4 consecutive CTAs form a group.  Member m of group g streams the gate / up rows of its own
// rows_blk neurons (phase 1), the four members exchange their parts of h through global memory (each writes its
// slice of the operand image, a byte counter per group in the control block, bounded wait; the producer keeps
// prefetching meanwhile), and in phase 2 member m streams column slice m (a quarter of d_model) of the down rows
// of all four members' neurons, column tile by column tile, so that a finished tile's partial output is stored
// while the next tile streams.  Every weight byte is read once, and a group writes ONE partial output
// [B, d_model] instead of one per CTA.  After a grid barrier all threads sum the groups' partials in group order
// and write y.
//
// One persistent CTA per SM, 192 threads: warp 0 TMA producer (64-column boxes of rows_blk rows, 128-byte swizzle,
// mbarrier ring), warp 1 TMEM allocation + MMA issue from one thread, warps 2-5 epilogues.  Every wait is bounded;
// on expiry the CTA raises CLADA_STATUS_TIMEOUT, drains its copies and frees its tensor memory.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "ffn_batch.cuh"
#include "ffn_common.cuh"
#include "tc_common.cuh"

namespace clada {

constexpr int kBdThreads = 192;
constexpr int kBdSeqs = 16;          // sequences per launch = N of every MMA
constexpr int kBdMembers = 4;        // CTAs per group = column slices of phase 2
constexpr int kBdKSplit = 4;         // interleaved K splits of phase 1
constexpr int kBdMaxStages = 8;
constexpr int kBdMaxRows = 128;      // neurons per CTA (TMEM lanes)
constexpr int kBdMaxTiles = 24;      // 128-column tiles per member: 24 * 16 TMEM columns
constexpr int kBdParts = 3;          // 16-bit parts of h
constexpr uint32_t kBdTmemCols = 512;
constexpr uint32_t kBdImgBlock = kBdParts * 2048;  // bytes of a 64-neuron block of the h image: 48 rows of 128 bytes
constexpr int kBdGroupWord0 = 8;     // group byte counters: control-block words 8..63
constexpr int kBdMaxGroups = 4 * (64 - kBdGroupWord0);
constexpr unsigned kBdGroupSpinLimit = 1u << 22;

// Opt-in timeline (-DCLADA_BD_TRACE): %globaltimer stamps per CTA, 64 slots, written by the thread that passes the point.
#ifdef CLADA_BD_TRACE
__device__ unsigned long long *g_bd_trace = nullptr;  // [n_ctas][64]
#define BD_TRACE(slot)                                                \
    do {                                                              \
        if (g_bd_trace) {                                             \
            unsigned long long t_;                                    \
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));     \
            g_bd_trace[(size_t)blockIdx.x * 64 + (slot)] = t_;        \
        }                                                             \
    } while (0)
#define BD_CLOCK(slot)                                                           \
    do {                                                                         \
        if (g_bd_trace) g_bd_trace[(size_t)blockIdx.x * 64 + (slot)] = clock64(); \
    } while (0)
#else
#define BD_TRACE(slot) \
    do {               \
    } while (0)
#define BD_CLOCK(slot) \
    do {               \
    } while (0)
#endif

struct BdParams {
    int d_model, d_ff, B;
    int rows_blk;        // neurons per CTA
    int rpad;            // rows_blk rounded up to 16 (K steps of phase 2)
    int n_groups;
    int n_stages;
    int n_tiles, tps;    // 128-column tiles of d_model; tiles per member
    int act, dtype;
    int wide;            // phase 2 with one N = 48 instruction per K step (48 TMEM columns per tile fit), else three of N = 16
    uint32_t idesc_p1, idesc_p2, idesc_p2w;
    const float *scores;  // [B, d_ff]
    const float *tau;
    long long tau_stride;
    void *y;
    size_t y_stride;
    int y_dtype;
    float *partials;      // [n_groups, B, d_model]
    unsigned char *himg;  // [n_groups] images of the phase-2 B operand: K blocks x (3 parts x 16 rows x 128 bytes)
    WsCtrl *ctrl;
    int32_t *status;
};

// 2-D tiled TMA load with an L2 eviction hint.
__device__ __forceinline__ void bd_tma_load(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], "
        "[%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(policy)
        : "memory");
}
// Shared-memory descriptor of an MN-major operand tile with 128-byte swizzle: 64 contiguous elements along M per
// 128-byte row, 8 K rows per 1024-byte atom; the next 8 K rows follow 1024 bytes on (stride byte offset), the next
// 64 elements along M lie lbo_bytes on (leading byte offset).
__device__ __forceinline__ uint64_t bd_smem_desc_mn(uint32_t addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Byte offset of element (row n of 48 = 16 part + sequence, k) in the K-major, 128-byte-swizzled image of the
// [48, K] operand: blocks of 64 k, six 8-row atoms of 1024 bytes per block, 16-byte chunks XORed with the row
// inside the atom.
__device__ __forceinline__ uint32_t bd_himg_off(int k, int n) {
    const int kb = k >> 6, kk = k & 63;
    return (uint32_t)kb * kBdImgBlock + (uint32_t)(n >> 3) * 1024u + (uint32_t)(n & 7) * 128u +
           (uint32_t)(((kk >> 3) ^ (n & 7)) << 4) + (uint32_t)(kk & 7) * 2u;
}
__device__ __forceinline__ uint16_t bd_to16(int dtype, float v, float &back) {
    if (dtype == CLADA_F16) {
        const __half h = __float2half_rn(v);
        back = __half2float(h);
        return __half_as_ushort(h);
    }
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    back = __bfloat162float(h);
    return __bfloat16_as_ushort(h);
}
// The MMAs of one phase-2 stage (up to 8 K steps of 16 neurons), issued back to back from descriptors computed
// beforehand: the issuing thread's own instructions between two MMAs are what limits their rate.
//   da: MN-major descriptor of the stage's first 16 rows (the next K step lies 2048 bytes on);
//   dhv: the K-major descriptors of the member's K steps in the h image, computed once per launch and member.
template <bool WIDE>
__device__ __forceinline__ void bd_issue_stage(uint32_t d_y, uint64_t da, const uint64_t (&dhv)[kBdMaxRows / 16], int ksteps,
                                               uint32_t acc, uint32_t idesc) {
#pragma unroll
    for (int k = 0; k < kBdMaxRows / 16; ++k) {
        if (k < ksteps) {
            if (WIDE) {
                tc_mma(d_y, da + 128 * k, dhv[k], k > 0 ? 1u : acc, idesc);
            } else {  // the parts' rows lie 2048 bytes apart
                tc_mma(d_y, da + 128 * k, dhv[k], k > 0 ? 1u : acc, idesc);
                tc_mma(d_y, da + 128 * k, dhv[k] + 128, 1u, idesc);
                tc_mma(d_y, da + 128 * k, dhv[k] + 256, 1u, idesc);
            }
        }
    }
}
// The K-major descriptors of a member's K steps in the h image: the next step lies 32 bytes on, after the fourth
// step of a 64-neuron block the next block follows.
__device__ __forceinline__ void bd_member_descs(uint64_t dh0, int mm, int ksteps, uint64_t (&dhv)[kBdMaxRows / 16]) {
#pragma unroll
    for (int k = 0; k < kBdMaxRows / 16; ++k) {
        const int kk16 = mm * ksteps + k;
        dhv[k] = dh0 + (uint64_t)(kk16 >> 2) * (kBdImgBlock >> 4) + (uint64_t)(kk16 & 3) * 2;
    }
}
__device__ __forceinline__ void bd_epi_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }

__global__ void __launch_bounds__(kBdThreads, 1)
sparse_ffn_batch_dense_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                              const __grid_constant__ CUtensorMap map_wu, const __grid_constant__ CUtensorMap map_wd,
                              const BdParams p) {
    extern __shared__ unsigned char bd_smem_raw[];
    const uint32_t smem0 = (tc_smem_u32(bd_smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t s_full[kBdMaxStages], s_empty[kBdMaxStages], s_p1_full, s_h_own, s_h_all,
        s_tile_full[kBdMaxTiles];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort, s_group_ok;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const int grp = cta / kBdMembers, mem = cta - grp * kBdMembers;
    const bool active = grp < p.n_groups;  // the CTAs behind the last whole group only join the barrier and the sums
    const bool gated = act_is_gated(p.act);
    const int n_kblocks = (p.d_model + kTcTileK - 1) / kTcTileK;
    const int n_stages = p.n_stages;
    const uint32_t box_bytes = (uint32_t)p.rows_blk * 128u;     // what one weight box delivers
    const uint32_t slot_bytes = (uint32_t)p.rpad * 128u;        // where the next box of a stage starts
    const uint32_t stage_bytes = 2u * slot_bytes + 2048u;       // gate | up | x   or   down columns 0-63 | 64-127
    const int kimg_blocks = (kBdMembers * p.rpad + 63) / 64;
    const uint32_t img_bytes = (uint32_t)kimg_blocks * kBdImgBlock;
    const uint32_t himg_s = smem0 + (uint32_t)n_stages * stage_bytes;  // the group's h image in shared memory
    const int t0 = mem * p.tps;
    const int nt = max(0, min(p.tps, p.n_tiles - t0));          // this member's column tiles in phase 2
    const int j0 = cta * p.rows_blk;                            // this CTA's first neuron

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            tc_mbar_init(tc_smem_u32(&s_full[s]), 1);
            tc_mbar_init(tc_smem_u32(&s_empty[s]), 1);
        }
        tc_mbar_init(tc_smem_u32(&s_p1_full), 1);
        tc_mbar_init(tc_smem_u32(&s_h_own), 128);
        tc_mbar_init(tc_smem_u32(&s_h_all), 128);
        for (int t = 0; t < kBdMaxTiles; ++t) tc_mbar_init(tc_smem_u32(&s_tile_full[t]), 1);
        s_abort = 0;
        s_group_ok = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Rows rows_blk .. rpad-1 of every box slot are never written by a copy but are read by the last K step of
    // phase 2 (against h = 0): they must hold finite values.
    if (p.rpad > p.rows_blk) {
        const int pad_vecs = (p.rpad - p.rows_blk) * 8;  // 16-byte vectors per slot
        for (int i = threadIdx.x; i < n_stages * 2 * pad_vecs; i += kBdThreads) {
            const int slot = i / pad_vecs, v = i - slot * pad_vecs;
            const uint32_t a = smem0 + (uint32_t)(slot >> 1) * stage_bytes + (uint32_t)(slot & 1) * slot_bytes + box_bytes +
                               (uint32_t)v * 16u;
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&s_tmem_base)),
                     "r"(kBdTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;
    pdl_launch_dependents();
    pdl_wait();  // x, the scores and the thresholds may come from the launch before
    if (threadIdx.x == 0) BD_TRACE(0);

    if (active && warp == 0) {
        // ---- TMA producer ----------------------------------------------------------------------
        if (lane == 0) {
            const uint64_t stream_policy = policy_evict_first(), keep_policy = policy_evict_last();
            int kc = 0, s = 0;
            uint32_t par = 0;
            bool ok = true;
            for (int kb = 0; kb < n_kblocks && ok; ++kb, ++kc) {  // phase 1: gate | up | x, one K block per stage
                if (!tc_mbar_wait(tc_smem_u32(&s_empty[s]), par ^ 1, abort_flag)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = tc_smem_u32(&s_full[s]);
                const uint32_t dst = smem0 + (uint32_t)s * stage_bytes;
                tc_mbar_expect_tx(bar, 2048u + (gated ? 2u : 1u) * box_bytes);
                bd_tma_load(dst + 2u * slot_bytes, &map_x, kb * kTcTileK, 0, bar, keep_policy);
                bd_tma_load(dst, &map_wg, kb * kTcTileK, j0, bar, stream_policy);
                if (gated) bd_tma_load(dst + slot_bytes, &map_wu, kb * kTcTileK, j0, bar, stream_policy);
                if (++s == n_stages) {
                    s = 0;
                    par ^= 1;
                }
            }
            BD_TRACE(14);
            // Phase 2, one column tile of one member's rows per stage: first this CTA's own rows for every tile (their
            // h is here before the group's exchange is over), then tile by tile the other three members' rows.
            auto issue_p2 = [&](int mm, int t) -> bool {
                if (!tc_mbar_wait(tc_smem_u32(&s_empty[s]), par ^ 1, abort_flag)) return false;
                const int rows0 = (grp * kBdMembers + mm) * p.rows_blk;
                const uint32_t bar = tc_smem_u32(&s_full[s]);
                const uint32_t dst = smem0 + (uint32_t)s * stage_bytes;
                tc_mbar_expect_tx(bar, 2u * box_bytes);
                bd_tma_load(dst, &map_wd, (t0 + t) * kTcTileM, rows0, bar, stream_policy);
                bd_tma_load(dst + slot_bytes, &map_wd, (t0 + t) * kTcTileM + 64, rows0, bar, stream_policy);
                ++kc;
                if (++s == n_stages) {
                    s = 0;
                    par ^= 1;
                }
                return true;
            };
            for (int t = 0; t < nt && ok; ++t) ok = issue_p2(mem, t);
            for (int t = 0; t < nt && ok; ++t)
                for (int mo = 0; mo < kBdMembers - 1 && ok; ++mo) ok = issue_p2(mo + (mo >= mem ? 1 : 0), t);
            BD_TRACE(15);
            if (!ok) *abort_flag = 1;
            for (int i = max(0, kc - n_stages); i < kc; ++i) {  // never leave with copies in flight
                int never = 0;
                if (!tc_mbar_wait(tc_smem_u32(&s_full[i % n_stages]), (i / n_stages) & 1, &never)) *abort_flag = 1;
            }
        }
    } else if (active && warp == 1) {
        // ---- MMA issuer ------------------------------------------------------------------------
        if (lane == 0) {
            int s = 0;
            uint32_t par = 0;
            bool ok = true;
            // One thread issues every MMA, so its instruction count per MMA bounds the rate (an MMA of N <= 48 takes
            // the tensor pipe ~44 cycles): descriptors are advanced by additions, never rebuilt.
            const uint64_t desc0 = tc_smem_desc(smem0);  // K-major descriptor of the ring's first byte
            const uint64_t stage16 = stage_bytes >> 4, slot16 = slot_bytes >> 4;
            uint64_t dstage = desc0;                     // descriptor of the current stage's first byte
            for (int kb = 0; kb < n_kblocks && ok; ++kb) {
                if (!tc_mbar_wait(tc_smem_u32(&s_full[s]), par, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                if (kb == 0) BD_TRACE(1);
                const uint64_t dg = dstage, du = dstage + slot16, dx = dstage + 2 * slot16;
                const uint32_t d_g = tmem_base + (uint32_t)(kb % kBdKSplit) * (2 * kBdSeqs);  // this K split's columns
                const uint32_t acc0 = kb >= kBdKSplit ? 1u : 0u;
#pragma unroll
                for (int k = 0; k < kTcTileK / 16; ++k) {
                    tc_mma(d_g, dg + 2 * k, dx + 2 * k, k > 0 ? 1u : acc0, p.idesc_p1);
                    if (gated) tc_mma(d_g + kBdSeqs, du + 2 * k, dx + 2 * k, k > 0 ? 1u : acc0, p.idesc_p1);
                }
                tc_commit(tc_smem_u32(&s_empty[s]));
                dstage += stage16;
                if (++s == n_stages) {
                    s = 0;
                    par ^= 1;
                    dstage = desc0;
                }
            }
            if (ok) tc_commit(tc_smem_u32(&s_p1_full));
            BD_TRACE(2);
            // Phase 2 writes over the phase-1 columns: the epilogue has read them before it lets s_h_own complete.
            // A: the stage's two boxes as one MN-major tile, 16 rows (2048 bytes) further per K step.  B: the h image,
            // 32 bytes further per K step and from the fourth step of a 64-neuron block on to the next block.
            const int ksteps = p.rpad / 16;
            const uint32_t tile_cols = p.wide ? kBdParts * kBdSeqs : kBdSeqs;
            const uint64_t dmn0 = bd_smem_desc_mn(smem0, slot_bytes);
            const uint64_t dh0 = tc_smem_desc(himg_s);
            uint64_t dstage2 = dmn0 + (uint64_t)s * stage16;
            auto run_p2 = [&](const uint64_t (&dhv)[kBdMaxRows / 16], int t, uint32_t acc) -> bool {  // the MMAs of one stage
                if (!tc_mbar_wait(tc_smem_u32(&s_full[s]), par, abort_flag)) return false;
                tc_fence_after();
                const uint32_t d_y = tmem_base + (uint32_t)t * tile_cols;
                if (p.wide)
                    bd_issue_stage<true>(d_y, dstage2, dhv, ksteps, acc, p.idesc_p2w);
                else
                    bd_issue_stage<false>(d_y, dstage2, dhv, ksteps, acc, p.idesc_p2);
                tc_commit(tc_smem_u32(&s_empty[s]));
                dstage2 += stage16;
                if (++s == n_stages) {
                    s = 0;
                    par ^= 1;
                    dstage2 = dmn0;
                }
                return true;
            };
            // the B descriptors of the four members' K steps stay in registers for the whole phase
            uint64_t dh_own[kBdMaxRows / 16], dh_oth[kBdMembers - 1][kBdMaxRows / 16];
            bd_member_descs(dh0, mem, ksteps, dh_own);
#pragma unroll
            for (int mo = 0; mo < kBdMembers - 1; ++mo) bd_member_descs(dh0, mo + (mo >= mem ? 1 : 0), ksteps, dh_oth[mo]);
            // this CTA's own part of h is in shared memory first; the other members' parts follow the exchange
            if (ok && !tc_mbar_wait(tc_smem_u32(&s_h_own), 0, abort_flag)) ok = false;
            tc_fence_after();
            BD_TRACE(3);
            for (int t = 0; t < nt && ok; ++t) ok = run_p2(dh_own, t, 0u);
            if (ok && !tc_mbar_wait(tc_smem_u32(&s_h_all), 0, abort_flag)) ok = false;
            tc_fence_after();
            for (int t = 0; t < nt && ok; ++t) {
#pragma unroll
                for (int mo = 0; mo < kBdMembers - 1; ++mo)
                    if (ok) ok = run_p2(dh_oth[mo], t, 1u);
                if (ok) tc_commit(tc_smem_u32(&s_tile_full[t]));  // this tile's partial output is complete
            }
            BD_TRACE(4);
            if (!ok) *abort_flag = 1;
        }
    } else if (active) {
        // ---- epilogue warps (2..5): warp w reads TMEM lanes 32 (w % 4) .. +31 ----------------------
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;           // this thread's neuron of the CTA (phase 1), column of a tile (phase 2)
        const int etid = threadIdx.x - 64;           // 0..127
        const int j = j0 + r;
        const bool row_ok = r < p.rows_blk && j < p.d_ff;
        unsigned keep = 0;                           // bit b: sequence b keeps neuron j
#pragma unroll
        for (int b = 0; b < kBdSeqs; ++b)
            if (b < p.B && row_ok && __ldg(p.scores + (size_t)b * p.d_ff + j) >= __ldg(p.tau + (size_t)b * p.tau_stride))
                keep |= 1u << b;
        bool ok = tc_mbar_wait(tc_smem_u32(&s_p1_full), 0, abort_flag);
        tc_fence_after();
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        if (etid == 0) BD_TRACE(5);
        if (ok) {
            float g[kBdSeqs], u[kBdSeqs];
#pragma unroll
            for (int b = 0; b < kBdSeqs; ++b) g[b] = u[b] = 0.f;
            const int n_splits = min(kBdKSplit, n_kblocks);
            for (int sp = 0; sp < n_splits; ++sp) {
                uint32_t rg[16], ru[16];
                tc_ld16(t_lane + (uint32_t)sp * (2 * kBdSeqs), rg);
                if (gated) tc_ld16(t_lane + (uint32_t)sp * (2 * kBdSeqs) + kBdSeqs, ru);
                tc_wait_ld();
#pragma unroll
                for (int b = 0; b < kBdSeqs; ++b) {
                    g[b] += __uint_as_float(rg[b]);
                    if (gated) u[b] += __uint_as_float(ru[b]);
                }
            }
            if (r < p.rpad) {  // rows rows_blk .. rpad-1 are the zero padding of the K steps
                const int k = mem * p.rpad + r;  // this CTA's slice of the image, written where phase 2 reads it
#pragma unroll
                for (int b = 0; b < kBdSeqs; ++b) {
                    float h = ((keep >> b) & 1u) ? neuron_value_f(p.act, g[b], u[b]) : 0.f;
#pragma unroll
                    for (int part = 0; part < kBdParts; ++part) {
                        float back;
                        const uint16_t bits = bd_to16(p.dtype, h, back);
                        h -= back;
                        asm volatile("st.shared.u16 [%0], %1;" ::"r"(himg_s + bd_himg_off(k, part * kBdSeqs + b)), "h"(bits)
                                     : "memory");
                    }
                }
            }
        }
        if (ok) {  // the MMA thread may start on this CTA's own down rows
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before();  // phase 2 writes over the TMEM columns this thread has read
            tc_mbar_arrive(tc_smem_u32(&s_h_own));
        }
        bd_epi_sync();
        unsigned char *img = p.himg + (size_t)grp * img_bytes;
        const int cpr = p.rpad / 8;                       // 16-byte chunks of a member's slice per image row
        const int n_chunks = kBdParts * kBdSeqs * cpr;
        if (ok) {  // the slice goes to global memory for the other three members
            for (int i = etid; i < n_chunks; i += 128) {
                const int n = i / cpr, c = i - n * cpr;
                const uint32_t off = bd_himg_off(mem * p.rpad + 8 * c, n);
                __stcg(reinterpret_cast<uint4 *>(img + off), lds128(himg_s + off));
            }
            __threadfence();
        }
        if (etid == 0) BD_TRACE(6);
        bd_epi_sync();
        // group exchange: one byte counter per group; every member adds 1 when its part of h is in global memory
        if (etid == 0) {
            unsigned *word = reinterpret_cast<unsigned *>(p.ctrl) + kBdGroupWord0 + (grp >> 2);
            const unsigned shift = 8u * (unsigned)(grp & 3);
            int gok = 0;
            if (ok && !*abort_flag) {
                asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(word), "r"(1u << shift) : "memory");
                for (unsigned spins = 0; spins < kBdGroupSpinLimit; ++spins) {
                    unsigned seen;
                    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(seen) : "l"(word) : "memory");
                    if (((seen >> shift) & 0xffu) >= (unsigned)kBdMembers) {
                        gok = 1;
                        break;
                    }
                }
            }
            s_group_ok = gok;
            BD_TRACE(7);
        }
        bd_epi_sync();
        ok = ok && s_group_ok != 0;
        if (ok) {
            for (int i = etid; i < (kBdMembers - 1) * n_chunks; i += 128) {  // the other members' slices
                const int mo = i / n_chunks, rem = i - mo * n_chunks;
                const int m2 = mo + (mo >= mem ? 1 : 0);
                const int n = rem / cpr, c = rem - n * cpr;
                const uint32_t off = bd_himg_off(m2 * p.rpad + 8 * c, n);
                const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(img + off));
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(himg_s + off), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                             : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_mbar_arrive(tc_smem_u32(&s_h_all));
            if (etid == 0) BD_TRACE(8);
            // ---- phase 2 epilogue: each column tile of the group's partial output as soon as it is complete ----------
            for (int t = 0; t < nt && ok; ++t) {
                ok = tc_mbar_wait(tc_smem_u32(&s_tile_full[t]), 0, abort_flag);
                tc_fence_after();
                if (t == 0 && etid == 0) BD_TRACE(9);
                if (!ok) break;
                uint32_t ry[16];
                float yv[kBdSeqs];
                if (p.wide) {  // the three parts' column groups, added in part order
                    uint32_t r2[16], r3[16];
                    tc_ld16(t_lane + (uint32_t)t * (kBdParts * kBdSeqs), ry);
                    tc_ld16(t_lane + (uint32_t)t * (kBdParts * kBdSeqs) + kBdSeqs, r2);
                    tc_ld16(t_lane + (uint32_t)t * (kBdParts * kBdSeqs) + 2 * kBdSeqs, r3);
                    tc_wait_ld();
#pragma unroll
                    for (int b = 0; b < kBdSeqs; ++b)
                        yv[b] = (__uint_as_float(ry[b]) + __uint_as_float(r2[b])) + __uint_as_float(r3[b]);
                } else {
                    tc_ld16(t_lane + (uint32_t)t * kBdSeqs, ry);
                    tc_wait_ld();
#pragma unroll
                    for (int b = 0; b < kBdSeqs; ++b) yv[b] = __uint_as_float(ry[b]);
                }
                const int i = (t0 + t) * kTcTileM + r;
                if (i < p.d_model) {
#pragma unroll
                    for (int b = 0; b < kBdSeqs; ++b)
                        if (b < p.B) p.partials[((size_t)grp * p.B + b) * p.d_model + i] = yv[b];
                }
            }
        }
        if (etid == 0) BD_TRACE(10);
        if (!ok) *abort_flag = 1;
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) BD_TRACE(11);
    if (threadIdx.x == 0 && s_abort && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kBdTmemCols) : "memory");
    }
    // ---- all groups' partial outputs are in global memory after the barrier: sum them in group order ----------
    if (!grid_barrier(p.ctrl, gridDim.x, 32)) {
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }
    if (threadIdx.x == 0) BD_TRACE(12);
    if (cta == 0 && threadIdx.x < 64 - kBdGroupWord0)  // every member has passed its group's counter: clear them
        reinterpret_cast<unsigned *>(p.ctrl)[kBdGroupWord0 + threadIdx.x] = 0u;
    const int d4 = p.d_model / 4;
    for (int it = cta * kBdThreads + threadIdx.x; it < p.B * d4; it += gridDim.x * kBdThreads) {
        const int b = it / d4, q = it - b * d4;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 *src = reinterpret_cast<const float4 *>(p.partials) + (size_t)b * d4 + q;
        for (int g0 = 0; g0 < p.n_groups; g0 += 8) {
            float4 v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
                v[e] = g0 + e < p.n_groups ? __ldcg(src + (size_t)(g0 + e) * p.B * d4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                s.x += v[e].x; s.y += v[e].y; s.z += v[e].z; s.w += v[e].w;
            }
        }
        char *yb = static_cast<char *>(p.y) + b * p.y_stride;
        if (p.y_dtype == CLADA_F32) {
            reinterpret_cast<float4 *>(yb)[q] = s;
        } else {
            reinterpret_cast<uint2 *>(yb)[q] = pack4_16bit(p.y_dtype, s);
        }
    }
    if (threadIdx.x == 0) BD_TRACE(13);
}

// ---- host side ------------------------------------------------------------------------------

struct BdPlan {
    int rows_blk, rpad, n_groups, n_tiles, tps, n_stages;
    size_t smem, partial_bytes, himg_bytes;
};

// The split of a layer over the device's CTAs, or false when this kernel does not take the layer.
static bool bd_plan(const clada_layer *layer, int B, const DeviceInfo &di, BdPlan *pl) {
    if (layer->dtype != CLADA_BF16 && layer->dtype != CLADA_F16) return false;
    if (B < 1 || B > kBdSeqs) return false;
    if (layer->d_model % 8 != 0 || layer->d_model > kMaxDModel) return false;
    pl->n_groups = di.num_sms / kBdMembers;
    if (pl->n_groups < 1 || pl->n_groups > kBdMaxGroups) return false;
    const int n_ctas = pl->n_groups * kBdMembers;
    pl->rows_blk = (layer->d_ff + n_ctas - 1) / n_ctas;
    if (pl->rows_blk > kBdMaxRows) return false;
    pl->rpad = (pl->rows_blk + 15) / 16 * 16;
    pl->n_tiles = (layer->d_model + kTcTileM - 1) / kTcTileM;
    pl->tps = (pl->n_tiles + kBdMembers - 1) / kBdMembers;
    if (pl->tps > kBdMaxTiles) return false;
    const size_t stage_bytes = 2 * (size_t)pl->rpad * 128 + 2048;
    const size_t kimg_blocks = ((size_t)kBdMembers * pl->rpad + 63) / 64;
    pl->himg_bytes = kimg_blocks * kBdImgBlock;
    const size_t budget = (size_t)di.max_smem_optin - 1024;  // static arrays: barriers and flags
    // behind the ring: the h image; at least 16 KB, because a phase-1 A tile is always 128 rows high and with few
    // neurons per CTA the tile of the last stage reaches past its own slot
    const size_t tail = std::max<size_t>(pl->himg_bytes, 16384);
    if (budget < 1024 + tail + 3 * stage_bytes) return false;
    pl->n_stages = (int)std::min<size_t>(kBdMaxStages, (budget - 1024 - tail) / stage_bytes);
    pl->smem = 1024 + (size_t)pl->n_stages * stage_bytes + tail;
    pl->partial_bytes = (size_t)pl->n_groups * B * layer->d_model * sizeof(float);
    return true;
}

bool ffn_batch_dense_supported(const clada_layer *layer, int B) {
    DeviceInfo di;
    BdPlan pl;
    return device_info(&di) == CLADA_OK && bd_plan(layer, B, di, &pl);
}

// Scratch behind the control block: the groups' partial outputs, then their h images.
size_t ffn_batch_dense_scratch_bytes(const clada_layer *layer, int B) {
    DeviceInfo di;
    BdPlan pl;
    if (device_info(&di) != CLADA_OK || !bd_plan(layer, B, di, &pl)) return 0;
    return ((pl.partial_bytes + 255) & ~(size_t)255) + (size_t)pl.n_groups * pl.himg_bytes;
}

int launch_ffn_batch_dense(const clada_layer *layer, int B, const void *x, const float *scores, const float *tau,
                           long long tau_stride, void *y, int y_dtype, void *ws, int32_t *status, cudaStream_t st) {
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    BdPlan pl;
    if (!bd_plan(layer, B, di, &pl)) return CLADA_ERR_UNSUPPORTED;
    EncodeTiledFn enc;
    rc = encode_fn(&enc);
    if (rc != CLADA_OK) return rc;
    const bool gated = act_is_gated(layer->activation);
    CUtensorMap map_x, map_wg, map_wu, map_wd;
    if ((rc = make_map(enc, &map_x, x, B, layer->d_model, layer->dtype, kBdSeqs)) != CLADA_OK) return rc;
    if ((rc = make_map(enc, &map_wg, layer->w_gate, layer->d_ff, layer->d_model, layer->dtype, pl.rows_blk)) != CLADA_OK)
        return rc;
    if ((rc = make_map(enc, &map_wu, gated ? layer->w_up : layer->w_gate, layer->d_ff, layer->d_model, layer->dtype,
                       pl.rows_blk)) != CLADA_OK)
        return rc;
    if ((rc = make_map(enc, &map_wd, layer->w_down_t, layer->d_ff, layer->d_model, layer->dtype, pl.rows_blk)) != CLADA_OK)
        return rc;
    BdParams p;
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.B = B;
    p.rows_blk = pl.rows_blk;
    p.rpad = pl.rpad;
    p.n_groups = pl.n_groups;
    p.n_stages = pl.n_stages;
    p.n_tiles = pl.n_tiles;
    p.tps = pl.tps;
    p.act = layer->activation;
    p.dtype = layer->dtype;
    p.idesc_p1 = tc_instr_desc(layer->dtype, kBdSeqs);
    p.idesc_p2 = tc_instr_desc(layer->dtype, kBdSeqs) | (1u << 15);  // A (the down rows) is MN-major
    p.idesc_p2w = tc_instr_desc(layer->dtype, kBdParts * kBdSeqs) | (1u << 15);
    p.wide = pl.tps * kBdParts * kBdSeqs <= (int)kBdTmemCols ? 1 : 0;
    p.scores = scores;
    p.tau = tau;
    p.tau_stride = tau_stride;
    p.y = y;
    p.y_stride = (size_t)layer->d_model * elem_size(y_dtype);
    p.y_dtype = y_dtype;
    p.partials = reinterpret_cast<float *>(static_cast<char *>(ws) + kWsCtrlBytes);
    p.himg = reinterpret_cast<unsigned char *>(static_cast<char *>(ws) + kWsCtrlBytes + ((pl.partial_bytes + 255) & ~(size_t)255));
    p.ctrl = static_cast<WsCtrl *>(ws);
    p.status = status;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(sparse_ffn_batch_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)((size_t)di.max_smem_optin - 1024)));
        configured[di.device & 63] = true;
    }
    void *args[] = {&map_x, &map_wg, &map_wu, &map_wd, &p};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(di.num_sms);
    cfg.blockDim = dim3(kBdThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident: the group waits and the grid barrier cannot starve
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    CLADA_CUDA_TRY(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(sparse_ffn_batch_dense_kernel), args));
    return CLADA_OK;
}

}  // namespace clada

#ifdef CLADA_BD_TRACE
extern "C" int clada_bd_trace_buffer(unsigned long long *buf) {
    CLADA_CUDA_TRY(cudaMemcpyToSymbol(clada::g_bd_trace, &buf, sizeof buf));
    return CLADA_OK;
}
#endif
