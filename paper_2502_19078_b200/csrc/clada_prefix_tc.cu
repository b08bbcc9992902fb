// Prefill statistics (Eq. neuron_activation) on the 5th-generation tensor cores, bf16 or fp16 inputs:
//   gate[t,j] = x_t . w_gate_j,  up[t,j] = x_t . w_up_j   (fp32 accumulator in tensor memory)
//   partial[tile, j] = sum_{t in tile} z[t,j]^2,  z = value of neuron j for token t in the layer's FFN form
// and, on request, the hidden activations z[t,j] themselves (the dense prefill FFN's first half).
//
// Tokens are the M dimension (128 per tile = the 128 TMEM lanes), d_model the K dimension, and the B operand is
// a tile of w_gate rows with the same neurons' w_up rows right behind it in shared memory: ONE instruction of
// N = 256 columns (gate | up) per 16-wide K step reads 12 KB of operands per MFLOP instead of the 16 KB two
// N = 128 instructions would, and the epilogue thread that owns token t finds gate and up of a neuron in its own
// lane.  The sum over a tile's tokens is then a sum over lanes: a halving butterfly per 16 neurons (16 shuffles),
// the four warps' results combined through shared memory in warp order (deterministic).
//
// One persistent CTA per SM, 320 threads:
//   warp 0      TMA producer: per 64-wide K block the token tile and the two weight tiles, 128-byte swizzle, into a
//               4-stage shared-memory ring (mbarrier full/empty);
//   warp 1      allocates 512 TMEM columns (two accumulators), issues tcgen05.mma (M128 N256 K16, kind::f16) from
//               one elected thread, commits stages and accumulators;
//   warps 2-9   epilogue (two warps per quarter of the TMEM lanes, alternate groups of 16 neurons): tcgen05.ld
//               32x32b.x16 of gate and up columns, neuron value, optional store of 16 consecutive neurons of the
//               thread's token, squares, butterfly; the second accumulator lets tile i+1's MMAs run under tile
//               i's epilogue, and eight warps halve what is exposed after a CTA's last tile.
// Work items are (128 neurons x 128 tokens), neuron tile major; a token tile never leaves its prompt and rows
// past the prompt's end count as zero.  The items left after the last full wave of CTAs are issued as two
// 64-neuron halves each (N = 128) when they then fit one wave, which halves that wave's time.
// Every wait is bounded; on expiry the CTA raises CLADA_STATUS_TIMEOUT, drains its copies and frees TMEM.
#include <cuda.h>
#include <math.h>

#include <algorithm>

#include "common.cuh"
#include "prefix_common.cuh"
#include "tc_common.cuh"

namespace clada {

constexpr int kTcMaxStages = 8;
constexpr int kTcThreads = 192;
constexpr int kTcEpiWarps = 8;   // prefix_tc_kernel: epilogue warps, a multiple of 4 (TMEM lane quarters); 12 and 16 measured the same
constexpr int kTcPfThreads = 64 + 32 * kTcEpiWarps;
constexpr uint32_t kTcTileBytes = kTcTileM * kTcTileK * 2;       // 16 KiB: a 128-row tile
constexpr uint32_t kTcRingBytes = 192 * 1024;                    // shared-memory ring of the statistics kernel
constexpr uint32_t kTcTmemCols = 512;                            // two accumulators of up to 256 columns

struct TcParams {
    int d_model, d_ff;
    int n_full;     // work items of 128 neurons x 128 tokens, neuron tile major: item = ntile * n_ttiles + ttile
    int n_half;     // the last (n_half / 2) such items are issued as two 64-neuron halves each, so that a last,
                    // partly filled wave of CTAs takes half the time
    int n_stages;   // ring depth
    uint32_t idesc_half;  // instruction descriptor of a 64-neuron item
    int n_ntiles;   // neuron tiles of 128
    int n_ttiles;   // token tiles over all prompts
    int t_group;    // token tiles per group (their rows, t_group * 128 * d_model elements, should stay in L2)
    float *partials;  // [n_ttiles, d_ff]
    int32_t *status;
    void *z_out;    // [T_total, d_ff] in the layer's element type, or null: the hidden activations themselves
    int dtype;      // clada_dtype of the layer (for z_out)
    uint32_t idesc; // instruction descriptor for the layer's element type
    int act;        // clada_activation; the non-gated form skips the w_up tiles and their MMAs
    SeqTable tab;
};

__global__ void __launch_bounds__(kTcPfThreads, 1)
prefix_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                 const __grid_constant__ CUtensorMap map_wu, const __grid_constant__ CUtensorMap map_wg_half,
                 const __grid_constant__ CUtensorMap map_wu_half, const TcParams p) {
    extern __shared__ unsigned char tc_smem_raw[];
    // stage tiles must sit on 1024-byte boundaries (the swizzle pattern is anchored to the address)
    const uint32_t smem0 = (tc_smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t s_full[kTcMaxStages], s_empty[kTcMaxStages], s_acc_full[2], s_acc_empty[2], s_epi[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ float s_col[2][4][kTcTileM];  // [tile parity][epilogue warp][neuron of the tile]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_items = p.n_full + p.n_half;
    const int n_kblocks = (p.d_model + kTcTileK - 1) / kTcTileK;
    const bool gated = act_is_gated(p.act);
    const uint32_t stage_bytes = kTcTileBytes + (gated ? 2u : 1u) * kTcTileBytes;  // ring stride: a full item's stage
    const int n_stages = p.n_stages;
    // item -> (neurons per tile, first neuron, token tile)
    // Items run in groups of t_group token tiles: within a group all neuron tiles follow one another, token tile
    // fastest, so the CTAs of a wave share weight tiles and the group's token rows (sized to stay in L2) are
    // re-read from L2, not from HBM, by every neuron tile.
    auto tile_of = [&](int f, int &ntile, int &ttile) {
        const int per_group = p.n_ntiles * p.t_group;
        int g = f / per_group;
        const int n_groups = (p.n_ttiles + p.t_group - 1) / p.t_group;
        if (g > n_groups - 1) g = n_groups - 1;
        const int gs = min(p.t_group, p.n_ttiles - g * p.t_group);  // the last group may be smaller
        const int rem = f - g * per_group;
        ntile = rem / gs;
        ttile = g * p.t_group + rem % gs;
    };
    auto decode = [&](int item, int &nt, int &j0, int &ttile) {
        int ntile;
        if (item < p.n_full) {
            nt = 128;
            tile_of(item, ntile, ttile);
            j0 = ntile * 128;
        } else {
            const int h = item - p.n_full;
            nt = 64;
            tile_of(p.n_full + (h >> 1), ntile, ttile);
            j0 = ntile * 128 + (h & 1) * 64;
        }
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            tc_mbar_init(tc_smem_u32(&s_full[s]), 1);
            tc_mbar_init(tc_smem_u32(&s_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            tc_mbar_init(tc_smem_u32(&s_acc_full[a]), 1);
            tc_mbar_init(tc_smem_u32(&s_acc_empty[a]), kTcEpiWarps);  // one arrival per epilogue warp
            tc_mbar_init(tc_smem_u32(&s_epi[a]), kTcEpiWarps);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // one warp allocates tensor memory and leaves the base address in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&s_tmem_base)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    if (warp == 0) {
        // ---- TMA producer ----------------------------------------------------------------------
        if (lane == 0) {
            int kc = 0;  // K blocks issued so far
            int s = 0;   // ring position and the parity of its current use
            uint32_t par = 0;
            bool ok = true;
            const uint32_t full0 = tc_smem_u32(&s_full[0]), empty0 = tc_smem_u32(&s_empty[0]);
            uint32_t full_s = full0, empty_s = empty0, dst_s = smem0;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                int nt, j0, ttile, b;
                decode(item, nt, j0, ttile);
                long long t0, t1;
                locate_tile(p.tab, ttile, kTcTileM, b, t0, t1);
                const uint32_t w_bytes = (uint32_t)nt * kTcTileK * 2u;  // one weight tile of this item
                const CUtensorMap *mg = nt == 128 ? &map_wg : &map_wg_half;
                const CUtensorMap *mu = nt == 128 ? &map_wu : &map_wu_half;
                const uint32_t tx_bytes = kTcTileBytes + (gated ? 2u : 1u) * w_bytes;
                const uint32_t up_off = kTcTileBytes + w_bytes;
                const int row0 = (int)t0;
                int c0 = 0;  // first column of the K block
                // like the MMA issuer, this thread's own instructions per K block count: nothing is recomputed
                for (int kb = 0; kb < n_kblocks; ++kb, ++kc, c0 += kTcTileK) {
                    if (!tc_mbar_wait(empty_s, par ^ 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_mbar_expect_tx(full_s, tx_bytes);
                    tc_tma_load(dst_s, &map_x, c0, row0, full_s);
                    tc_tma_load(dst_s + kTcTileBytes, mg, c0, j0, full_s);
                    if (gated) tc_tma_load(dst_s + up_off, mu, c0, j0, full_s);
                    dst_s += stage_bytes;
                    full_s += 8;
                    empty_s += 8;
                    if (++s == n_stages) {
                        s = 0;
                        par ^= 1;
                        dst_s = smem0;
                        full_s = full0;
                        empty_s = empty0;
                    }
                }
            }
            if (!ok) *abort_flag = 1;
            // never leave with copies in flight: the last armed use of every stage must have landed
            for (int i = max(0, kc - n_stages); i < kc; ++i) {
                int never = 0;  // these copies land by themselves: wait for them even after an abort
                if (!tc_mbar_wait(tc_smem_u32(&s_full[i % n_stages]), (i / n_stages) & 1, &never)) *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ------------------------------------------------------------------------
        if (lane == 0) {
            // One thread issues every MMA of the CTA, and its own instructions between two MMAs are what paces
            // them (a lone thread issues an instruction every ~5 cycles): nothing in the K loop is recomputed --
            // the stage's descriptors and barrier addresses advance by additions.
            int it = 0;
            int s = 0;
            uint32_t par = 0;
            bool ok = true;
            const uint64_t desc0 = tc_smem_desc(smem0);          // descriptor of the ring's first byte
            const uint64_t stage16 = stage_bytes >> 4, tile16 = kTcTileBytes >> 4;
            const uint32_t full0 = tc_smem_u32(&s_full[0]), empty0 = tc_smem_u32(&s_empty[0]);
            uint64_t dstage = desc0;
            uint32_t full_s = full0, empty_s = empty0;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
                const int a = it & 1;
                // the epilogue must have drained this accumulator (fresh barrier: parity 1 passes)
                if (!tc_mbar_wait(tc_smem_u32(&s_acc_empty[a]), ((it >> 1) & 1) ^ 1, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_acc = tmem_base + (uint32_t)a * 256u;
                const uint32_t idesc = item < p.n_full ? p.idesc : p.idesc_half;
                uint32_t acc = 0u;  // the item's first MMA overwrites the accumulator
                for (int kb = 0; kb < n_kblocks; ++kb) {
                    if (!tc_mbar_wait(full_s, par, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    // A = the token tile (128 rows), B = the w_gate rows with the w_up rows right behind them:
                    // one instruction of N = 2 nt columns (gate | up) per 16-wide K step (+32 bytes = 2 descriptor
                    // units inside the swizzled row)
                    const uint64_t dx = dstage, dw = dstage + tile16;
                    tc_mma(d_acc, dx, dw, acc, idesc);
                    tc_mma(d_acc, dx + 2, dw + 2, 1u, idesc);
                    tc_mma(d_acc, dx + 4, dw + 4, 1u, idesc);
                    tc_mma(d_acc, dx + 6, dw + 6, 1u, idesc);
                    acc = 1u;
                    tc_commit(empty_s);  // the stage is free once these MMAs have read it
                    dstage += stage16;
                    full_s += 8;
                    empty_s += 8;
                    if (++s == n_stages) {
                        s = 0;
                        par ^= 1;
                        dstage = desc0;
                        full_s = full0;
                        empty_s = empty0;
                    }
                }
                if (ok) tc_commit(tc_smem_u32(&s_acc_full[a]));  // accumulator complete
            }
            if (!ok) *abort_flag = 1;
        }
    } else {
        // ---- epilogue warps (2..9): warp w may touch TMEM lanes 32 (w % 4) .. +31 = 32 tokens; the two warps of a
        // lane quarter take alternate groups of 16 columns ------------
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;
        const bool b16 = lane & 16, b8 = lane & 8, b4 = lane & 4, b2 = lane & 2;
        const int my_val = (b16 ? 8 : 0) + (b8 ? 4 : 0) + (b4 ? 2 : 0) + (b2 ? 1 : 0);
        const int e = (warp - 2) * 32 + lane;  // 0..127: the neuron of the tile this thread finishes
        int it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int a = it & 1;
            int nt, jbase, ttile, b;
            decode(item, nt, jbase, ttile);
            long long t0, t1;
            locate_tile(p.tab, ttile, kTcTileM, b, t0, t1);
            const int row = quarter * 32 + lane;          // this thread's token within the tile
            const bool tok_ok = row < (int)(t1 - t0);     // rows past the prompt's end belong to nobody
            if (!tc_mbar_wait(tc_smem_u32(&s_acc_full[a]), (it >> 1) & 1, abort_flag)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)a * 256u;
            for (int c0 = 16 * col_half; c0 < nt; c0 += 4 * kTcEpiWarps) {
                uint32_t rg[16], ru[16];
                tc_ld16(t_acc + c0, rg);
                if (gated) {
                    tc_ld16(t_acc + nt + c0, ru);
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) ru[c] = 0u;
                }
                tc_wait_ld();
                float z[16], q[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    z[c] = tok_ok ? neuron_value_f(p.act, __uint_as_float(rg[c]), __uint_as_float(ru[c])) : 0.f;
                    q[c] = z[c] * z[c];
                }
                if (p.z_out && tok_ok) {  // 16 consecutive neurons of this token: two 16-byte stores
                    const int j0 = jbase + c0;
                    uint16_t *dst = static_cast<uint16_t *>(p.z_out) + (size_t)(t0 + row) * p.d_ff + j0;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (j0 + 8 * h + 8 > p.d_ff) continue;  // d_ff is a multiple of 8 when Z is asked for
                        const uint2 lo = pack4_16bit(p.dtype, make_float4(z[8 * h], z[8 * h + 1], z[8 * h + 2], z[8 * h + 3]));
                        const uint2 hi = pack4_16bit(p.dtype, make_float4(z[8 * h + 4], z[8 * h + 5], z[8 * h + 6], z[8 * h + 7]));
                        *reinterpret_cast<uint4 *>(dst + 8 * h) = make_uint4(lo.x, lo.y, hi.x, hi.y);
                    }
                }
                // Sum of z^2 over the warp's 32 tokens for each of the 16 neurons: a halving butterfly (16
                // shuffles) that leaves the total of neuron my_val on every lane.  Fixed order.
                float v8[8], v4[4], v2[2], v1;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    v8[i] = (b16 ? q[i + 8] : q[i]) + __shfl_xor_sync(0xffffffffu, b16 ? q[i] : q[i + 8], 16);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    v4[i] = (b8 ? v8[i + 4] : v8[i]) + __shfl_xor_sync(0xffffffffu, b8 ? v8[i] : v8[i + 4], 8);
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    v2[i] = (b4 ? v4[i + 2] : v4[i]) + __shfl_xor_sync(0xffffffffu, b4 ? v4[i] : v4[i + 2], 4);
                v1 = (b2 ? v2[1] : v2[0]) + __shfl_xor_sync(0xffffffffu, b2 ? v2[0] : v2[1], 2);
                v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
                if ((lane & 1) == 0) s_col[a][quarter][c0 + my_val] = v1;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(tc_smem_u32(&s_acc_empty[a]));  // the accumulator may be overwritten
            // the four warps' token groups, added in warp order; s_col alternates with the accumulator, so a
            // warp that runs ahead writes the other half while this one is still being read
            // (an mbarrier rather than a hardware barrier: its wait is bounded like every other one here)
            if (lane == 0) tc_mbar_arrive(tc_smem_u32(&s_epi[a]));
            if (!tc_mbar_wait(tc_smem_u32(&s_epi[a]), (it >> 1) & 1, abort_flag)) {
                ok = false;
                break;
            }
            const int j = jbase + e;
            if (col_half == 0 && e < nt && j < p.d_ff)
                p.partials[(size_t)ttile * p.d_ff + j] = ((s_col[a][0][e] + s_col[a][1][e]) + s_col[a][2][e]) + s_col[a][3][e];
        }
        if (!ok) *abort_flag = 1;
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && s_abort && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}


// ---- host side ------------------------------------------------------------------------------

int run_prefix_partials_tc(const clada_layer *layer, const void *X, const SeqTable &tab, long long T_total,
                           float *partials, int32_t *status, cudaStream_t st, void *z_out) {
    static bool configured[64] = {};
    int n_ttiles = 0;
    for (int b = 0; b < tab.B; ++b) n_ttiles += tiles_of(tab.off[b + 1] - tab.off[b], kTcTileM);
    if (n_ttiles == 0) return CLADA_OK;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    EncodeTiledFn enc;
    rc = encode_fn(&enc);
    if (rc != CLADA_OK) return rc;
    const bool gated = act_is_gated(layer->activation);
    CUtensorMap map_x, map_wg, map_wu, map_wg_half, map_wu_half;
    // without a gate projection the w_up maps are never used by the kernel: give them w_gate's address
    const void *wu = gated ? layer->w_up : layer->w_gate;
    if ((rc = make_map(enc, &map_x, X, T_total, layer->d_model, layer->dtype)) != CLADA_OK) return rc;
    if ((rc = make_map(enc, &map_wg, layer->w_gate, layer->d_ff, layer->d_model, layer->dtype, 128)) != CLADA_OK) return rc;
    if ((rc = make_map(enc, &map_wu, wu, layer->d_ff, layer->d_model, layer->dtype, 128)) != CLADA_OK) return rc;
    if ((rc = make_map(enc, &map_wg_half, layer->w_gate, layer->d_ff, layer->d_model, layer->dtype, 64)) != CLADA_OK) return rc;
    if ((rc = make_map(enc, &map_wu_half, wu, layer->d_ff, layer->d_model, layer->dtype, 64)) != CLADA_OK) return rc;
    TcParams p;
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.n_ntiles = (layer->d_ff + 127) / 128;
    p.n_ttiles = n_ttiles;
    {   // about 40 MB of token rows per group
        const long long tile_bytes = (long long)kTcTileM * layer->d_model * 2;
        p.t_group = (int)std::max<long long>(1, std::min<long long>(n_ttiles, (40ll << 20) / tile_bytes));
    }
    // The items left over after the last full wave of CTAs run as 64-neuron halves when they then still fit one
    // wave: that wave takes half the time.  (Halves read more bytes per flop, so only the tail is split.)
    const long long items = (long long)p.n_ntiles * n_ttiles;
    const long long rest = items % di.num_sms;
    const long long split = (items > di.num_sms && 2 * rest <= di.num_sms) ? rest : 0;
    p.n_full = (int)(items - split);
    p.n_half = (int)(2 * split);
    p.partials = partials;
    p.status = status;
    p.act = layer->activation;
    p.z_out = z_out;
    p.dtype = layer->dtype;
    p.idesc = tc_instr_desc(layer->dtype, gated ? 256 : 128);  // gate | up columns in one instruction
    p.idesc_half = tc_instr_desc(layer->dtype, gated ? 128 : 64);
    p.tab = tab;
    const uint32_t stage_bytes = kTcTileBytes + (gated ? 2u : 1u) * kTcTileBytes;
    p.n_stages = std::min<int>(kTcMaxStages, (int)(kTcRingBytes / stage_bytes));
    const size_t smem = (size_t)kTcRingBytes + 1024;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(prefix_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[di.device & 63] = true;
    }
    const int grid = (int)std::min<long long>((long long)p.n_full + p.n_half, di.num_sms);
    prefix_tc_kernel<<<grid, kTcPfThreads, smem, st>>>(map_x, map_wg, map_wu, map_wg_half, map_wu_half, p);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

// ---- down projection of the dense prefill FFN --------------------------------------------------
//   Y[t, i] = sum_j Z[t, j] * W_out[i, j]      (Z: hidden activations, W_out in the paper's [d_model, d_ff] layout)
// Both operands are K-major (d_ff contiguous), so the tiles, descriptors and the role split are those of
// the statistics kernel: tokens are the M dimension (TMEM lanes), output columns the N dimension, one
// accumulator per tile (256 output columns, or 128 for short prompts), two in flight.  The epilogue thread
// that owns token t writes its row of the tile.
// Short prompts have fewer tiles than the device has SMs, and a tile's time is its number of K blocks whatever
// its width: given scratch, the K dimension of every tile is then split among n_split CTAs, each writes its fp32
// partial tile to the scratch, and down_reduce_kernel adds the partials in split order and writes Y.

constexpr int kDnMaxStages = 6;
constexpr int kDnMaxSplit = 8;                        // CTAs per output tile along K, at most
constexpr uint32_t kDnTmemCols = 512;                 // two accumulators of up to 256 columns

struct DownParams {
    int d_model, d_ff;
    long long T;
    int n_ttiles, n_dtiles;
    int t_group;   // token tiles per group: a group's rows of Z stay in L2 while every output tile reads them
    int nd;        // output columns per tile: 256 (fewer bytes read per flop), or 128 when 256 would leave SMs idle
    int n_stages;
    int n_split;   // CTAs per tile along K (1: no split, Y is written directly)
    int kb_split;  // K blocks per split
    float *partials;  // [n_split, T, d_model] fp32 when n_split > 1
    void *y;
    int y_dtype;
    uint32_t idesc;
    int32_t *status;
};

__global__ void __launch_bounds__(kTcThreads, 1)
down_tc_kernel(const __grid_constant__ CUtensorMap map_z, const __grid_constant__ CUtensorMap map_w,
               const DownParams p) {
    extern __shared__ unsigned char tc_smem_raw[];
    const uint32_t smem0 = (tc_smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t s_full[kDnMaxStages], s_empty[kDnMaxStages], s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.n_ttiles * p.n_dtiles;
    const int n_items = n_tiles * p.n_split;  // item = split * n_tiles + tile: a wave's CTAs walk the same K range
    const int nd = p.nd, n_stages = p.n_stages;
    // items in groups of t_group token tiles; within a group output tile by output tile, token tile fastest
    auto tile_of = [&](int f, int &dtile, int &ttile) {
        const int per_group = p.n_dtiles * p.t_group;
        int g = f / per_group;
        const int n_groups = (p.n_ttiles + p.t_group - 1) / p.t_group;
        if (g > n_groups - 1) g = n_groups - 1;
        const int gs = min(p.t_group, p.n_ttiles - g * p.t_group);
        const int rem = f - g * per_group;
        dtile = rem / gs;
        ttile = g * p.t_group + rem % gs;
    };
    const uint32_t stage_bytes = kTcTileBytes + (uint32_t)nd * kTcTileK * 2u;  // Z tile | W_out tile
    const int n_kblocks = (p.d_ff + kTcTileK - 1) / kTcTileK;
    // K blocks [kb_lo, kb_hi) of an item (never empty: the host sees to that)
    auto k_range = [&](int item, int &tile, int &kb_lo, int &kb_hi) {
        const int sp = item / n_tiles;
        tile = item - sp * n_tiles;
        kb_lo = sp * p.kb_split;
        kb_hi = min(n_kblocks, kb_lo + p.kb_split);
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            tc_mbar_init(tc_smem_u32(&s_full[s]), 1);
            tc_mbar_init(tc_smem_u32(&s_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            tc_mbar_init(tc_smem_u32(&s_acc_full[a]), 1);
            tc_mbar_init(tc_smem_u32(&s_acc_empty[a]), 4);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&s_tmem_base)),
                     "r"(kDnTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    // items run token tile fastest, so the CTAs of a wave share the same W_out tiles in L2
    if (warp == 0) {
        if (lane == 0) {
            int kc = 0;
            int s = 0;  // ring position and the parity of its current use, kept incrementally
            uint32_t par = 0;
            bool ok = true;
            // nothing in the K loop is recomputed (see prefix_tc_kernel): addresses advance by additions
            const uint32_t full0 = tc_smem_u32(&s_full[0]), empty0 = tc_smem_u32(&s_empty[0]);
            uint32_t full_s = full0, empty_s = empty0, dst_s = smem0;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                int dtile, ttile, tile, kb_lo, kb_hi;
                k_range(item, tile, kb_lo, kb_hi);
                tile_of(tile, dtile, ttile);
                const int row_z = ttile * kTcTileM, row_w = dtile * nd;
                int c0 = kb_lo * kTcTileK;
                for (int kb = kb_lo; kb < kb_hi; ++kb, ++kc, c0 += kTcTileK) {
                    if (!tc_mbar_wait(empty_s, par ^ 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_mbar_expect_tx(full_s, stage_bytes);
                    tc_tma_load(dst_s, &map_z, c0, row_z, full_s);
                    tc_tma_load(dst_s + kTcTileBytes, &map_w, c0, row_w, full_s);
                    dst_s += stage_bytes;
                    full_s += 8;
                    empty_s += 8;
                    if (++s == n_stages) {
                        s = 0;
                        par ^= 1;
                        dst_s = smem0;
                        full_s = full0;
                        empty_s = empty0;
                    }
                }
            }
            if (!ok) *abort_flag = 1;
            for (int i = max(0, kc - n_stages); i < kc; ++i) {
                int never = 0;  // these copies land by themselves: wait for them even after an abort
                if (!tc_mbar_wait(tc_smem_u32(&s_full[i % n_stages]), (i / n_stages) & 1, &never)) *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int it = 0;
            int s = 0;
            uint32_t par = 0;
            bool ok = true;
            // descriptors and barrier addresses advance by additions (see prefix_tc_kernel's issuer)
            const uint64_t desc0 = tc_smem_desc(smem0);
            const uint64_t stage16 = stage_bytes >> 4, tile16 = kTcTileBytes >> 4;
            const uint32_t full0 = tc_smem_u32(&s_full[0]), empty0 = tc_smem_u32(&s_empty[0]);
            uint64_t dstage = desc0;
            uint32_t full_s = full0, empty_s = empty0;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
                const int a = it & 1;
                if (!tc_mbar_wait(tc_smem_u32(&s_acc_empty[a]), ((it >> 1) & 1) ^ 1, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_acc = tmem_base + (uint32_t)a * 256u;
                uint32_t acc = 0u;
                int tile, kb_lo, kb_hi;
                k_range(item, tile, kb_lo, kb_hi);
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!tc_mbar_wait(full_s, par, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t dz = dstage, dw = dstage + tile16;
                    tc_mma(d_acc, dz, dw, acc, p.idesc);
                    tc_mma(d_acc, dz + 2, dw + 2, 1u, p.idesc);
                    tc_mma(d_acc, dz + 4, dw + 4, 1u, p.idesc);
                    tc_mma(d_acc, dz + 6, dw + 6, 1u, p.idesc);
                    acc = 1u;
                    tc_commit(empty_s);
                    dstage += stage16;
                    full_s += 8;
                    empty_s += 8;
                    if (++s == n_stages) {
                        s = 0;
                        par ^= 1;
                        dstage = desc0;
                        full_s = full0;
                        empty_s = empty0;
                    }
                }
                if (ok) tc_commit(tc_smem_u32(&s_acc_full[a]));
            }
            if (!ok) *abort_flag = 1;
        }
    } else {
        const int quarter = warp & 3;
        int it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int a = it & 1;
            int dtile, ttile, tile, kb_lo, kb_hi;
            k_range(item, tile, kb_lo, kb_hi);
            tile_of(tile, dtile, ttile);
            // a split item's fp32 partial tile goes to its split's copy of the output, added up afterwards
            float *part = p.n_split > 1 ? p.partials + (size_t)(item / n_tiles) * (size_t)p.T * p.d_model : nullptr;
            if (!tc_mbar_wait(tc_smem_u32(&s_acc_full[a]), (it >> 1) & 1, abort_flag)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)a * 256u;
            const long long t = (long long)ttile * kTcTileM + quarter * 32 + lane;
            const int i0 = dtile * nd;
            const int ncols = min(nd, p.d_model - i0);  // a multiple of 8 (d_model is)
            for (int c0 = 0; c0 < ncols; c0 += 16) {           // uniform per warp
                uint32_t r[16];
                tc_ld16(t_acc + c0, r);
                tc_wait_ld();
                if (t < p.T) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {              // two groups of 8 columns
                        if (c0 + 8 * h >= ncols) continue;
                        const float4 lo = make_float4(__uint_as_float(r[8 * h]), __uint_as_float(r[8 * h + 1]),
                                                      __uint_as_float(r[8 * h + 2]), __uint_as_float(r[8 * h + 3]));
                        const float4 hi = make_float4(__uint_as_float(r[8 * h + 4]), __uint_as_float(r[8 * h + 5]),
                                                      __uint_as_float(r[8 * h + 6]), __uint_as_float(r[8 * h + 7]));
                        const size_t at = (size_t)t * p.d_model + i0 + c0 + 8 * h;
                        if (part) {
                            float4 *dst = reinterpret_cast<float4 *>(part + at);
                            dst[0] = lo;
                            dst[1] = hi;
                        } else if (p.y_dtype == CLADA_F32) {
                            float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(p.y) + at);
                            dst[0] = lo;
                            dst[1] = hi;
                        } else {
                            const uint2 a2 = pack4_16bit(p.y_dtype, lo), b2 = pack4_16bit(p.y_dtype, hi);
                            *reinterpret_cast<uint4 *>(static_cast<uint16_t *>(p.y) + at) = make_uint4(a2.x, a2.y, b2.x, b2.y);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(tc_smem_u32(&s_acc_empty[a]));
        }
        if (!ok) *abort_flag = 1;
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && s_abort && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kDnTmemCols) : "memory");
    }
}

// Y = the sum of the splits' fp32 partial outputs, in split order (fixed: results repeat bit for bit).
__global__ void __launch_bounds__(256)
down_reduce_kernel(const float4 *__restrict__ partials, int n_split, size_t n4, void *y, int y_dtype) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    pdl_wait();  // launched while the contraction still runs: its partial outputs are complete from here on
    if (i >= n4) return;
    float4 s = __ldcg(partials + i);
    for (int k = 1; k < n_split; ++k) {
        const float4 v = __ldcg(partials + (size_t)k * n4 + i);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    if (y_dtype == CLADA_F32)
        static_cast<float4 *>(y)[i] = s;
    else
        static_cast<uint2 *>(y)[i] = pack4_16bit(y_dtype, s);
}

// CTAs per tile along K for a prompt of T tokens: 1 unless tiles of 256 output columns leave at least half of the
// SMs without one; at most kDnMaxSplit, and no split may be empty.
static int down_split(const clada_layer *layer, long long T, int num_sms) {
    const long long tiles = ((T + kTcTileM - 1) / kTcTileM) * ((layer->d_model + 255) / 256);
    if (tiles <= 0 || 2 * tiles > num_sms) return 1;
    const int n_kblocks = (layer->d_ff + kTcTileK - 1) / kTcTileK;
    int n = (int)std::min<long long>(kDnMaxSplit, num_sms / tiles);
    while (n > 1 && (n - 1) * ((n_kblocks + n - 1) / n) >= n_kblocks) --n;
    return n;
}

size_t down_split_scratch_bytes(const clada_layer *layer, long long T, int num_sms) {
    const int n = down_split(layer, T, num_sms);
    return n > 1 ? (size_t)n * (size_t)T * layer->d_model * sizeof(float) : 0;
}

int run_down_tc(const clada_layer *layer, const void *w_down, const void *Z, long long T, void *Y, int y_dtype,
                void *scratch, size_t scratch_bytes, int32_t *status, cudaStream_t st) {
    static bool configured[64] = {};
    if (T <= 0) return CLADA_OK;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    EncodeTiledFn enc;
    rc = encode_fn(&enc);
    if (rc != CLADA_OK) return rc;
    CUtensorMap map_z, map_w;
    if ((rc = make_map(enc, &map_z, Z, T, layer->d_ff, layer->dtype)) != CLADA_OK) return rc;
    DownParams p;
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.T = T;
    p.n_ttiles = (int)((T + kTcTileM - 1) / kTcTileM);
    {   // about 40 MB of hidden-activation rows per group
        const long long tile_bytes = (long long)kTcTileM * layer->d_ff * 2;
        p.t_group = (int)std::max<long long>(1, std::min<long long>(p.n_ttiles, (40ll << 20) / tile_bytes));
    }
    // 256 output columns per tile unless that leaves SMs without a tile -- or, given scratch, with K split among
    // as many CTAs per tile as fit the device
    p.n_split = 1;
    {
        const size_t need = down_split_scratch_bytes(layer, T, di.num_sms);
        if (scratch && need > 0 && scratch_bytes >= need) p.n_split = down_split(layer, T, di.num_sms);
    }
    p.nd = p.n_split > 1 || (long long)p.n_ttiles * ((layer->d_model + 255) / 256) >= di.num_sms ? 256 : 128;
    p.n_dtiles = (layer->d_model + p.nd - 1) / p.nd;
    p.kb_split = (((layer->d_ff + kTcTileK - 1) / kTcTileK) + p.n_split - 1) / p.n_split;
    p.partials = static_cast<float *>(scratch);
    const uint32_t dn_stage = kTcTileBytes + (uint32_t)p.nd * kTcTileK * 2u;
    p.n_stages = std::min<int>(kDnMaxStages, (int)(kTcRingBytes / dn_stage));
    p.y = Y;
    p.y_dtype = y_dtype;
    p.idesc = tc_instr_desc(layer->dtype, p.nd);
    p.status = status;
    if ((rc = make_map(enc, &map_w, w_down, layer->d_model, layer->d_ff, layer->dtype, p.nd)) != CLADA_OK) return rc;
    const size_t smem = (size_t)kTcRingBytes + 1024;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(down_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[di.device & 63] = true;
    }
    const long long items = (long long)p.n_ttiles * p.n_dtiles * p.n_split;
    const int grid = (int)std::min<long long>(items, di.num_sms);
    down_tc_kernel<<<grid, kTcThreads, smem, st>>>(map_z, map_w, p);
    CLADA_CUDA_TRY(cudaGetLastError());
    if (p.n_split > 1) {
        const size_t n4 = (size_t)T * layer->d_model / 4;  // d_model is a multiple of 8
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((n4 + 255) / 256));
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // hide the launch latency
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        CLADA_CUDA_TRY(cudaLaunchKernelEx(&cfg, down_reduce_kernel, static_cast<const float4 *>(scratch), p.n_split, n4, Y,
                                          y_dtype));
    }
    return CLADA_OK;
}

}  // namespace clada
