// Prefill statistics (Eq. neuron_activation) on the 5th-generation tensor cores, bf16 inputs:
//   gate[j,t] = w_gate_j . x_t,  up[j,t] = w_up_j . x_t   (fp32 accumulators in tensor memory)
//   partial[tile, j] = sum_{t in tile} (silu(gate[j,t]) * up[j,t])^2
//
// Neurons are the M dimension (128 per tile = the 128 TMEM lanes), tokens the N dimension (128 per
// tile = 128 TMEM columns), d_model the K dimension.  The epilogue thread that owns lane j therefore
// walks its own row of both accumulators and adds z^2 over the tile's tokens serially in a register:
// no cross-lane reduction, no z ever written.  A token tile never leaves its prompt; columns beyond
// the prompt's end are skipped.
//
// One persistent CTA per SM, 192 threads:
//   warp 0      TMA producer: per 64-wide K block three 128 x 64 bf16 tiles (w_gate, w_up, X), 128-byte
//               swizzle, into a 4-stage shared-memory ring (mbarrier full/empty);
//   warp 1      allocates 512 TMEM columns (two accumulator pairs), issues tcgen05.mma (M128 N128 K16,
//               kind::f16) for gate and up from one elected thread, commits stages and accumulators;
//   warps 2-5   epilogue: tcgen05.ld 32x32b.x16 of both accumulators, silu * up, square, sum; the
//               second accumulator pair lets tile i+1's MMAs run under tile i's epilogue.
// Every wait is bounded; on expiry the CTA raises CLADA_STATUS_TIMEOUT, drains its copies and frees TMEM.
#include <cuda.h>
#include <math.h>

#include <algorithm>

#include "common.cuh"
#include "prefix_common.cuh"

namespace clada {

constexpr int kTcTileM = 128;   // neurons per tile (TMEM lanes)
constexpr int kTcTileN = 128;   // tokens per tile (TMEM columns per accumulator)
constexpr int kTcTileK = 64;    // K block: 64 bf16 = 128 bytes = one swizzle row
constexpr int kTcStages = 4;
constexpr int kTcThreads = 192;
constexpr uint32_t kTcTileBytes = kTcTileM * kTcTileK * 2;       // 16 KiB
constexpr uint32_t kTcStageBytes = 3 * kTcTileBytes;             // w_gate | w_up | X
constexpr uint32_t kTcTmemCols = 512;                            // 2 x (gate 128 + up 128)
constexpr unsigned kTcSpinLimit = 1u << 20;

struct TcParams {
    int d_model, d_ff;
    int n_ntiles;   // neuron tiles
    int n_ttiles;   // token tiles over all prompts
    float *partials;  // [n_ttiles, d_ff]
    int32_t *status;
    void *z_out;    // [T_total, d_ff] in the layer's element type, or null: the hidden activations themselves
    int dtype;      // clada_dtype of the layer (for z_out)
    uint32_t idesc; // instruction descriptor for the layer's element type
    int act;        // clada_activation; the non-gated form skips the w_up tiles and their MMAs
    SeqTable tab;
};

__device__ __forceinline__ uint32_t tc_smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void tc_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase of the given parity; false if it gave up or another role raised the
// abort flag.  Each try suspends for at most ~1 us (the hint), so the bound is about a second.
__device__ __forceinline__ bool tc_mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    for (unsigned i = 0; i < kTcSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(1000u)
            : "memory");
        if (ok) return true;
        if (*abort_flag) return false;
    }
    return false;
}
// 2-D tiled TMA load (no multicast): box {64 elements, 128 rows} at element c0 of row c1.
__device__ __forceinline__ void tc_tma_load(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart (stride byte offset), version 1 (sm_100).  Fields are in 16-byte units.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);  // start address
    d |= (uint64_t)1 << 16;                  // leading byte offset (unused with swizzle): 1
    d |= (uint64_t)(1024 >> 4) << 32;        // stride byte offset
    d |= (uint64_t)1 << 46;                  // descriptor version
    d |= (uint64_t)2 << 61;                  // SWIZZLE_128B
    return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B of one 16-bit type (format code 1 = bf16, 0 = fp16,
// the same for both operands), both K-major, N = 128, M = 128.
constexpr uint32_t kTcInstrDescF16 = (1u << 4) | ((uint32_t)(kTcTileN >> 3) << 17) | ((uint32_t)(kTcTileM >> 4) << 24);
constexpr uint32_t kTcInstrDescBf16 = kTcInstrDescF16 | (1u << 7) | (1u << 10);
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate,
                                       uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }


__global__ void __launch_bounds__(kTcThreads, 1)
prefix_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                 const __grid_constant__ CUtensorMap map_wu, const TcParams p) {
    extern __shared__ unsigned char tc_smem_raw[];
    // stage tiles must sit on 1024-byte boundaries (the swizzle pattern is anchored to the address)
    const uint32_t smem0 = (tc_smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t s_full[kTcStages], s_empty[kTcStages], s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_items = p.n_ntiles * p.n_ttiles;
    const int n_kblocks = (p.d_model + kTcTileK - 1) / kTcTileK;
    const bool gated = act_is_gated(p.act);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            tc_mbar_init(tc_smem_u32(&s_full[s]), 1);
            tc_mbar_init(tc_smem_u32(&s_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            tc_mbar_init(tc_smem_u32(&s_acc_full[a]), 1);
            tc_mbar_init(tc_smem_u32(&s_acc_empty[a]), 4);  // one arrival per epilogue warp
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
            int kc = 0;  // K blocks issued so far (ring position)
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int ntile = item / p.n_ttiles, ttile = item % p.n_ttiles;
                int b;
                long long t0, t1;
                locate_tile(p.tab, ttile, kTcTileN, b, t0, t1);
                for (int kb = 0; kb < n_kblocks; ++kb, ++kc) {
                    const int s = kc % kTcStages;
                    if (!tc_mbar_wait(tc_smem_u32(&s_empty[s]), ((kc / kTcStages) & 1) ^ 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t bar = tc_smem_u32(&s_full[s]);
                    const uint32_t dst = smem0 + (uint32_t)s * kTcStageBytes;
                    tc_mbar_expect_tx(bar, gated ? kTcStageBytes : 2 * kTcTileBytes);
                    tc_tma_load(dst, &map_wg, kb * kTcTileK, ntile * kTcTileM, bar);
                    if (gated) tc_tma_load(dst + kTcTileBytes, &map_wu, kb * kTcTileK, ntile * kTcTileM, bar);
                    tc_tma_load(dst + 2 * kTcTileBytes, &map_x, kb * kTcTileK, (int)t0, bar);
                }
            }
            if (!ok) *abort_flag = 1;
            // never leave with copies in flight: the last armed use of every stage must have landed
            for (int i = max(0, kc - kTcStages); i < kc; ++i)
                {
                int never = 0;  // these copies land by themselves: wait for them even after an abort
                if (!tc_mbar_wait(tc_smem_u32(&s_full[i % kTcStages]), (i / kTcStages) & 1, &never)) *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ------------------------------------------------------------------------
        if (lane == 0) {
            int kc = 0, it = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
                const int a = it & 1;
                // the epilogue must have drained this accumulator pair (fresh barrier: parity 1 passes)
                if (!tc_mbar_wait(tc_smem_u32(&s_acc_empty[a]), ((it >> 1) & 1) ^ 1, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_gate = tmem_base + (uint32_t)a * 256u, d_up = d_gate + 128u;
                for (int kb = 0; kb < n_kblocks; ++kb, ++kc) {
                    const int s = kc % kTcStages;
                    if (!tc_mbar_wait(tc_smem_u32(&s_full[s]), (kc / kTcStages) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t base = smem0 + (uint32_t)s * kTcStageBytes;
                    const uint64_t dg = tc_smem_desc(base), du = tc_smem_desc(base + kTcTileBytes),
                                   dx = tc_smem_desc(base + 2 * kTcTileBytes);
#pragma unroll
                    for (int k = 0; k < kTcTileK / 16; ++k) {
                        // advancing K by 16 bf16 = 32 bytes = 2 descriptor units inside the swizzled row
                        const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                        tc_mma(d_gate, dg + 2 * k, dx + 2 * k, acc, p.idesc);
                        if (gated) tc_mma(d_up, du + 2 * k, dx + 2 * k, acc, p.idesc);
                    }
                    tc_commit(tc_smem_u32(&s_empty[s]));  // the stage is free once these MMAs have read it
                }
                if (ok) tc_commit(tc_smem_u32(&s_acc_full[a]));  // accumulators complete
            }
            if (!ok) *abort_flag = 1;
        }
    } else {
        // ---- epilogue warps (2..5): warp w may touch TMEM lanes 32 (w % 4) .. +31 -------------------
        const int quarter = warp & 3;
        int it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int a = it & 1;
            const int ntile = item / p.n_ttiles, ttile = item % p.n_ttiles;
            int b;
            long long t0, t1;
            locate_tile(p.tab, ttile, kTcTileN, b, t0, t1);
            const int ncols = (int)(t1 - t0);
            if (!tc_mbar_wait(tc_smem_u32(&s_acc_full[a]), (it >> 1) & 1, abort_flag)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t t_gate = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)a * 256u;
            const uint32_t t_up = t_gate + 128u;
            float sum = 0.f;
            const int jrow = ntile * kTcTileM + quarter * 32 + lane;
            for (int c0 = 0; c0 < ncols; c0 += 16) {  // uniform per warp: ncols is
                uint32_t rg[16], ru[16];
                tc_ld16(t_gate + c0, rg);
                if (gated) {
                    tc_ld16(t_up + c0, ru);
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) ru[c] = 0u;
                }
                tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    if (c0 + c < ncols) {
                        const float z = neuron_value_f(p.act, __uint_as_float(rg[c]), __uint_as_float(ru[c]));
                        sum = fmaf(z, z, sum);
                        if (p.z_out && jrow < p.d_ff) {  // a warp writes 32 consecutive neurons of one token
                            const size_t at = (size_t)(t0 + c0 + c) * p.d_ff + jrow;
                            if (p.dtype == CLADA_BF16)
                                static_cast<__nv_bfloat16 *>(p.z_out)[at] = __float2bfloat16_rn(z);
                            else
                                static_cast<__half *>(p.z_out)[at] = __float2half_rn(z);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(tc_smem_u32(&s_acc_empty[a]));
            const int j = ntile * kTcTileM + quarter * 32 + lane;
            if (j < p.d_ff) p.partials[(size_t)ttile * p.d_ff + j] = sum;
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, fetched through the runtime (the library does not link libcuda).
static int encode_fn(EncodeTiledFn *out) {
    static EncodeTiledFn cached = nullptr;
    if (!cached) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        CLADA_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !fn) return CLADA_ERR_UNSUPPORTED;
        cached = reinterpret_cast<EncodeTiledFn>(fn);
    }
    *out = cached;
    return CLADA_OK;
}

// Row-major bf16 or fp16 matrix [rows, cols] as a 2-D tensor map with a {64, 128} box and 128-byte swizzle;
// out-of-range rows and columns read as zero.
static int make_map(EncodeTiledFn enc, CUtensorMap *map, const void *base, long long rows, int cols, int dtype) {
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcTileK, (cuuint32_t)kTcTileM};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType et = dtype == CLADA_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = enc(map, et, 2, const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
        return CLADA_ERR_CUDA;
    }
    return CLADA_OK;
}

int run_prefix_partials_tc(const clada_layer *layer, const void *X, const SeqTable &tab, long long T_total,
                           float *partials, int32_t *status, cudaStream_t st, void *z_out) {
    static bool configured[64] = {};
    int n_ttiles = 0;
    for (int b = 0; b < tab.B; ++b) n_ttiles += tiles_of(tab.off[b + 1] - tab.off[b], kTcTileN);
    if (n_ttiles == 0) return CLADA_OK;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    EncodeTiledFn enc;
    rc = encode_fn(&enc);
    if (rc != CLADA_OK) return rc;
    CUtensorMap map_x, map_wg, map_wu;
    if ((rc = make_map(enc, &map_x, X, T_total, layer->d_model, layer->dtype)) != CLADA_OK) return rc;
    if ((rc = make_map(enc, &map_wg, layer->w_gate, layer->d_ff, layer->d_model, layer->dtype)) != CLADA_OK) return rc;
    // without a gate projection the w_up map is never used by the kernel: give it w_gate's address
    const void *wu = act_is_gated(layer->activation) ? layer->w_up : layer->w_gate;
    if ((rc = make_map(enc, &map_wu, wu, layer->d_ff, layer->d_model, layer->dtype)) != CLADA_OK) return rc;
    TcParams p;
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.n_ntiles = (layer->d_ff + kTcTileM - 1) / kTcTileM;
    p.n_ttiles = n_ttiles;
    p.partials = partials;
    p.status = status;
    p.act = layer->activation;
    p.z_out = z_out;
    p.dtype = layer->dtype;
    p.idesc = layer->dtype == CLADA_F16 ? kTcInstrDescF16 : kTcInstrDescBf16;
    p.tab = tab;
    const size_t smem = (size_t)kTcStages * kTcStageBytes + 1024;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(prefix_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[di.device & 63] = true;
    }
    const long long items = (long long)p.n_ntiles * n_ttiles;
    const int grid = (int)std::min<long long>(items, di.num_sms);
    prefix_tc_kernel<<<grid, kTcThreads, smem, st>>>(map_x, map_wg, map_wu, p);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

// ---- down projection of the dense prefill FFN --------------------------------------------------
//   Y[t, i] = sum_j Z[t, j] * W_out[i, j]      (Z: hidden activations, W_out in the paper's [d_model, d_ff] layout)
// Both operands are K-major (d_ff contiguous), so the tiles, descriptors and the role split are those of
// the statistics kernel: tokens are the M dimension (TMEM lanes), output columns the N dimension, one
// accumulator per tile, two in flight.  The epilogue thread that owns token t writes its row of the tile.

constexpr int kDnStages = 6;
constexpr uint32_t kDnStageBytes = 2 * kTcTileBytes;  // Z tile | W_out tile
constexpr uint32_t kDnTmemCols = 256;                 // two 128-column accumulators

struct DownParams {
    int d_model, d_ff;
    long long T;
    int n_ttiles, n_dtiles;
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
    __shared__ __align__(8) uint64_t s_full[kDnStages], s_empty[kDnStages], s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_items = p.n_ttiles * p.n_dtiles;
    const int n_kblocks = (p.d_ff + kTcTileK - 1) / kTcTileK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDnStages; ++s) {
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
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int dtile = item / p.n_ttiles, ttile = item % p.n_ttiles;
                for (int kb = 0; kb < n_kblocks; ++kb, ++kc) {
                    const int s = kc % kDnStages;
                    if (!tc_mbar_wait(tc_smem_u32(&s_empty[s]), ((kc / kDnStages) & 1) ^ 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t bar = tc_smem_u32(&s_full[s]);
                    const uint32_t dst = smem0 + (uint32_t)s * kDnStageBytes;
                    tc_mbar_expect_tx(bar, kDnStageBytes);
                    tc_tma_load(dst, &map_z, kb * kTcTileK, ttile * kTcTileM, bar);
                    tc_tma_load(dst + kTcTileBytes, &map_w, kb * kTcTileK, dtile * kTcTileN, bar);
                }
            }
            if (!ok) *abort_flag = 1;
            for (int i = max(0, kc - kDnStages); i < kc; ++i) {
                int never = 0;  // these copies land by themselves: wait for them even after an abort
                if (!tc_mbar_wait(tc_smem_u32(&s_full[i % kDnStages]), (i / kDnStages) & 1, &never)) *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int kc = 0, it = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
                const int a = it & 1;
                if (!tc_mbar_wait(tc_smem_u32(&s_acc_empty[a]), ((it >> 1) & 1) ^ 1, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_acc = tmem_base + (uint32_t)a * 128u;
                for (int kb = 0; kb < n_kblocks; ++kb, ++kc) {
                    const int s = kc % kDnStages;
                    if (!tc_mbar_wait(tc_smem_u32(&s_full[s]), (kc / kDnStages) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t base = smem0 + (uint32_t)s * kDnStageBytes;
                    const uint64_t dz = tc_smem_desc(base), dw = tc_smem_desc(base + kTcTileBytes);
#pragma unroll
                    for (int k = 0; k < kTcTileK / 16; ++k)
                        tc_mma(d_acc, dz + 2 * k, dw + 2 * k, (kb > 0 || k > 0) ? 1u : 0u, p.idesc);
                    tc_commit(tc_smem_u32(&s_empty[s]));
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
            const int dtile = item / p.n_ttiles, ttile = item % p.n_ttiles;
            if (!tc_mbar_wait(tc_smem_u32(&s_acc_full[a]), (it >> 1) & 1, abort_flag)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)a * 128u;
            const long long t = (long long)ttile * kTcTileM + quarter * 32 + lane;
            const int i0 = dtile * kTcTileN;
            const int ncols = min(kTcTileN, p.d_model - i0);  // a multiple of 8 (d_model is)
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
                        if (p.y_dtype == CLADA_F32) {
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

int run_down_tc(const clada_layer *layer, const void *w_down, const void *Z, long long T, void *Y, int y_dtype,
                int32_t *status, cudaStream_t st) {
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
    if ((rc = make_map(enc, &map_w, w_down, layer->d_model, layer->d_ff, layer->dtype)) != CLADA_OK) return rc;
    DownParams p;
    p.d_model = layer->d_model;
    p.d_ff = layer->d_ff;
    p.T = T;
    p.n_ttiles = (int)((T + kTcTileM - 1) / kTcTileM);
    p.n_dtiles = (layer->d_model + kTcTileN - 1) / kTcTileN;
    p.y = Y;
    p.y_dtype = y_dtype;
    p.idesc = layer->dtype == CLADA_F16 ? kTcInstrDescF16 : kTcInstrDescBf16;
    p.status = status;
    const size_t smem = (size_t)kDnStages * kDnStageBytes + 1024;
    if (!configured[di.device & 63]) {
        CLADA_CUDA_TRY(cudaFuncSetAttribute(down_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[di.device & 63] = true;
    }
    const long long items = (long long)p.n_ttiles * p.n_dtiles;
    const int grid = (int)std::min<long long>(items, di.num_sms);
    down_tc_kernel<<<grid, kTcThreads, smem, st>>>(map_z, map_w, p);
    CLADA_CUDA_TRY(cudaGetLastError());
    return CLADA_OK;
}

}  // namespace clada
