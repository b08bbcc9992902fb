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
// the same 16-byte vectors of x are the A fragments.  The 16 warps' partial D tiles are summed through shared
// memory in warp order (fp32, round to nearest), the neuron values h are formed, zeroed for the sequences that
// cut the neuron, and the down rows are scaled into the per-thread partial y on the CUDA cores as before.
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

// NV: 16-byte vectors of a row per consumer thread (down projection); NPS: pairs of k-steps per warp, i.e.
// 16-byte vectors of x per lane (16 warps x NPS x 4 lanes of a quad cover a row of up to 64 NPS vectors).
template <typename T, int NV, int BT, int NPS>
__global__ void __launch_bounds__(kFfnThreads, 1)
sparse_ffn_batch_tc_kernel(const FfnBatchParams p, const int n_stages) {
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = Pairs<T>::kPairs;
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
    __shared__ __align__(16) float s_part[kConsWarps][BT][8];  // per warp: D rows of the tile's sequences
    __shared__ __align__(16) float s_h[GS][4];                 // neuron value per (neuron of the chunk, sequence)

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
    const int g = lane >> 2, t = lane & 3;
    bool vok[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) vok[i] = tid < kConsumers && tid + i * kConsumers < vpr;
    __syncthreads();  // thresholds are in shared memory

    const int my_n = batch_union_share<BT>(p, s_tau, s_bal, s_balb, s_list, s_keep, s_wtot, keep_policy);
    __syncthreads();  // list, keep bits and the mbarriers are ready

    // A fragments: lane (g, t) = (lane / 4, lane % 4) holds, for each of its warp's pairs of k-steps, the
    // 16-byte vector 4 * pair + t of sequence g's x (zero for g >= BT and past the row's end).  A warp's pairs
    // are warp, warp + 16, ...: consecutive warps read consecutive 64-byte pieces of x.  They are loaded after
    // the prologue, which needs the registers; the first rows are still on their way from HBM then.
    uint4 afrag[NPS];
#pragma unroll
    for (int j = 0; j < NPS; ++j) {
        const int v = 4 * (warp + kConsWarps * j) + t;
        afrag[j] = make_uint4(0u, 0u, 0u, 0u);
        if (tid < kConsumers && g < BT && v < vpr)
            afrag[j] = *(reinterpret_cast<const uint4 *>(static_cast<const char *>(p.x) + g * p.x_stride) + v);
    }

    bool timed_out = false;

    if (warp == kConsWarps) {
        // ---- producer (rows at a padded pitch) ---------------------------------------------------------
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
                const size_t off = (size_t)s_list[i] * row_bytes;
                const uint32_t dst = ring + (uint32_t)s * stage_bytes, bar = full0 + 8 * s;
                mbar_expect_tx(bar, n_rows * row_bytes);
                bulk_load_row_hint(dst, Wg + off, row_bytes, bar, stream_policy);
                if (gated) bulk_load_row_hint(dst + pitch, Wu + off, row_bytes, bar, stream_policy);
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
        int cs = 0;           // ring position of the chunk's first neuron, and the parity of its use
        uint32_t cpar = 0;
        // B rows of this lane: columns 0-3 of the B tile are the gate rows of the chunk's neurons 0-3, columns
        // 4-7 their up rows; lane (g, t) feeds column g.
        const int nb = g & 3;
        const uint32_t b_off = (g >= 4 ? pitch : 0u);
        for (int g0 = 0; g0 < my_n; g0 += GS) {
            const int nn = min(GS, my_n - g0);
            // the chunk's stages
            uint32_t st_addr[GS];
            int st_idx[GS];
            {
                int s = cs;
                uint32_t par = cpar;
#pragma unroll
                for (int q = 0; q < GS; ++q) {
                    st_idx[q] = s;
                    st_addr[q] = ring + (uint32_t)s * stage_bytes;
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
            // ---- gate | up of four neurons for all sequences: one chain of warp-level MMAs per accumulator ----
            float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
            {
                const bool row_ok = nb < nn && (g < 4 || gated);
                uint32_t brow = st_addr[0];
                if (nb == 1) brow = st_addr[1];
                if (nb == 2) brow = st_addr[2];
                if (nb == 3) brow = st_addr[3];
                brow += b_off;
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
            if (g < BT) *reinterpret_cast<float2 *>(&s_part[warp][g][2 * t]) = make_float2(d0[0] + d1[0], d0[1] + d1[1]);
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
            // ---- sum over the 16 warps (their K slices), neuron values ------------------------------------
            if (tid < BT * 32) {
                // value (b, n) = tid / 4: lane part = tid % 4 adds warps 4 part .. 4 part + 3, the quad finishes
                const int b = tid >> 5, n = (tid >> 2) & 7, part = tid & 3;
                float s4 = (s_part[4 * part][b][n] + s_part[4 * part + 1][b][n]) +
                           (s_part[4 * part + 2][b][n] + s_part[4 * part + 3][b][n]);
                s4 += __shfl_xor_sync(0xffffffffu, s4, 1);
                s4 += __shfl_xor_sync(0xffffffffu, s4, 2);
                const float up = __shfl_xor_sync(0xffffffffu, s4, 16);  // column n + 4: the same neuron's up row
                if (n < GS && part == 0) {
                    float h = 0.f;
                    if (n < nn && ((s_keep[g0 + n] >> b) & 1)) h = neuron_value_f(p.act, s4, up);
                    s_h[n][b] = h;  // not kept by sequence b (or past the share's end): no contribution
                }
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
            // ---- down rows scaled into the partial y ---------------------------------------------------------
#pragma unroll
            for (int q = 0; q < GS; ++q) {
                if (q >= nn) continue;
                const float4 h4 = *reinterpret_cast<const float4 *>(&s_h[q][0]);
                const float hb[4] = {h4.x, h4.y, h4.z, h4.w};
                float2 h2[BT];
#pragma unroll
                for (int b = 0; b < BT; ++b) h2[b] = make_float2(hb[b], hb[b]);
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    if (!vok[k]) continue;
                    float2 fd[P];
                    Pairs<T>::unpack(lds128(st_addr[q] + down_off + (uint32_t)(tid + k * kConsumers) * 16u), fd);
#pragma unroll
                    for (int b = 0; b < BT; ++b)
#pragma unroll
                        for (int e = 0; e < P; ++e) acc[b][k][e] = __ffma2_rn(h2[b], fd[e], acc[b][k][e]);
                }
            }
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int q = 0; q < GS; ++q)
                    if (q < nn) mbar_arrive(empty0 + 8 * st_idx[q]);
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

// ---- host side ------------------------------------------------------------------------------

template <typename T, int NV, int BT, int NPS>
static int launch_tc_variant(const FfnBatchParams &p, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerVec;
    static bool configured[64] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_batch_tc_kernel<T, NV, BT, NPS>;
    const size_t stage_bytes = (act_is_gated(p.act) ? 3 : 2) * ((size_t)(p.d_model / E) * 16 + kRowPad);
    const size_t chunks = (size_t)(p.d_ff + 31) / 32;
    const size_t tail = 2 * kMaxStages * sizeof(uint64_t) + (1 + BT) * chunks * sizeof(unsigned) +
                        2 * (size_t)(p.d_ff / di.num_sms + 2) * sizeof(int);
    const size_t budget = (size_t)di.max_smem_optin - 4096;  // leave room for the static arrays
    if (budget < tail + GS * stage_bytes) return CLADA_ERR_UNSUPPORTED;  // a chunk holds GS stages at once
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

// Rows of up to 512 vectors (d_model 4096) take 8 pairs of k-steps per warp and tiles of 4 or 2; rows of up to
// 640 vectors (d_model 5120) 10 pairs and tiles of 2 (two vectors of partial y per thread and sequence).
bool ffn_batch_tc_supported(const clada_layer *layer, int bt) {
    if (layer->dtype != CLADA_BF16 && layer->dtype != CLADA_F16) return false;
    const int vpr = layer->d_model / 8;
    if (bt == 4) return vpr <= kConsumers;
    if (bt == 2) return vpr <= 640;
    return false;
}

template <typename T>
static int launch_tc_typed(const FfnBatchParams &p, int bt, cudaStream_t st) {
    const int vpr = p.d_model / Elem<T>::kPerVec;
    if (bt == 4 && vpr <= kConsumers) return launch_tc_variant<T, 1, 4, 8>(p, st);
    if (bt == 2 && vpr <= kConsumers) return launch_tc_variant<T, 1, 2, 8>(p, st);
    if (bt == 2 && vpr <= 640) return launch_tc_variant<T, 2, 2, 10>(p, st);
    return CLADA_ERR_UNSUPPORTED;
}

int launch_ffn_batch_tc(const FfnBatchParams &p, int dtype, int bt, cudaStream_t st) {
    return dtype == CLADA_BF16 ? launch_tc_typed<__nv_bfloat16>(p, bt, st) : launch_tc_typed<__half>(p, bt, st);
}

}  // namespace clada
