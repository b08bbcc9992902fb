// Sparse gated FFN for one decode token per sequence (Algorithm 2, generation phase):
//   kept = { j : A_j >= tau_final },  y = sum_{j in kept} silu(w_gate_j . x) (w_up_j . x) w_down_t[j,:]
//
// One persistent cooperative kernel per (layer, sequence):
//   prologue  every CTA scans the F scores against tau (warp ballots), learns the number of kept
//             neurons and takes an equal share [r0, r1) of the kept list in ascending order;
//   stream    the CTA walks its share G neurons at a time.  Thread t owns the same 16-byte column
//             vectors of every row (x and the partial y for those columns live in registers), so the
//             three rows of a neuron are read with fully coalesced 128-bit loads.  The loads of the
//             next group's gate/up rows are issued before the current group's down rows are consumed,
//             which keeps HBM requests in flight across the CTA-wide dot-product reduction;
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

constexpr int kFfnMaxWarps = 8;
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

template <typename T, int NV, int G>
__global__ void __launch_bounds__(kFfnMaxWarps *kWarp, 2)
sparse_ffn_kernel(const FfnParams p) {
    constexpr int E = Elem<T>::kPerVec;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads >> 5;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int F = p.d_ff, d = p.d_model;
    const int vpr = d / E;  // 16-byte vectors per row

    // shared: kept list of this CTA (dynamic), per-warp scan totals, dot-product exchange
    int *s_list = reinterpret_cast<int *>(smem_raw);
    __shared__ int s_wtot[kFfnMaxWarps];
    __shared__ float s_dot[2][kFfnMaxWarps][2 * G];

    // ---- prologue: threshold test and this CTA's share of the kept list -------------------------
    const float tau = *p.tau;
    const int chunks = (F + kWarp - 1) / kWarp;
    const int per_warp = (chunks + nwarps - 1) / nwarps;
    const int c0 = warp * per_warp, c1 = min(chunks, c0 + per_warp);
    int n = 0;
    for (int c = c0; c < c1; ++c) {
        const int j = c * kWarp + lane;
        const bool keep = j < F && p.scores[j] >= tau;
        n += __popc(__ballot_sync(0xffffffffu, keep));
    }
    if (lane == 0) s_wtot[warp] = n;
    __syncthreads();
    int base = 0, n_act = 0;
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
        const bool keep = j < F && p.scores[j] >= tau;
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
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

    // ---- x and the partial y of this thread's columns, in registers -----------------------------
    float xr[NV][E], acc[NV][E];
    bool vok[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int v = tid + i * nthreads;
        vok[i] = v < vpr;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (vok[i]) q = *(reinterpret_cast<const uint4 *>(p.x) + v);
        Elem<T>::unpack(q, xr[i]);
#pragma unroll
        for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
    }
    __syncthreads();  // s_list complete

    const uint4 *Wg = reinterpret_cast<const uint4 *>(p.w_gate);
    const uint4 *Wu = reinterpret_cast<const uint4 *>(p.w_up);
    const uint4 *Wd = reinterpret_cast<const uint4 *>(p.w_down_t);

    uint4 qg[G][NV], qu[G][NV], qd[G][NV];
    int jn[G];  // neurons of the group whose gate/up rows are in flight

    auto issue_gate_up = [&](int g0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            jn[g] = (g0 + g < my_n) ? s_list[g0 + g] : -1;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                qg[g][i] = make_uint4(0, 0, 0, 0);
                qu[g][i] = make_uint4(0, 0, 0, 0);
                if (jn[g] >= 0 && vok[i]) {
                    const size_t off = (size_t)jn[g] * vpr + tid + i * nthreads;
                    qg[g][i] = ldg_stream(Wg + off);
                    qu[g][i] = ldg_stream(Wu + off);
                }
            }
        }
    };

    issue_gate_up(0);
    int buf = 0;
    for (int g0 = 0; g0 < my_n; g0 += G, buf ^= 1) {
        // partial dot products over this thread's columns
        float pd[2 * G];
        int jcur[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            jcur[g] = jn[g];
            float sg = 0.f, su = 0.f;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                float fg[E], fu[E];
                Elem<T>::unpack(qg[g][i], fg);
                Elem<T>::unpack(qu[g][i], fu);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    sg = fmaf(fg[e], xr[i][e], sg);
                    su = fmaf(fu[e], xr[i][e], su);
                }
            }
            pd[2 * g] = sg;
            pd[2 * g + 1] = su;
        }
        // down rows of the same neurons: issue now, consume after the reduction
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                qd[g][i] = make_uint4(0, 0, 0, 0);
                if (jcur[g] >= 0 && vok[i])
                    qd[g][i] = ldg_stream(Wd + (size_t)jcur[g] * vpr + tid + i * nthreads);
            }
        // CTA-wide sums in a fixed order: lanes by butterfly, then warps 0..nwarps-1
#pragma unroll
        for (int k = 0; k < 2 * G; ++k) pd[k] = warp_sum(pd[k]);
        if (lane == 0) {
#pragma unroll
            for (int k = 0; k < 2 * G; ++k) s_dot[buf][warp][k] = pd[k];
        }
        __syncthreads();
        // next group's gate/up rows go out before the FMAs below
        issue_gate_up(g0 + G);
        float h[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float sg = 0.f, su = 0.f;
            for (int w = 0; w < nwarps; ++w) {
                sg += s_dot[buf][w][2 * g];
                su += s_dot[buf][w][2 * g + 1];
            }
            h[g] = (jcur[g] >= 0) ? silu_f(sg) * su : 0.f;
        }
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                float fd[E];
                Elem<T>::unpack(qd[g][i], fd);
#pragma unroll
                for (int e = 0; e < E; ++e) acc[i][e] = fmaf(h[g], fd[e], acc[i][e]);
            }
    }

    // ---- epilogue: partial rows, grid barrier, deterministic column reduction -------------------
    float *mine = p.partials + (size_t)cta * d;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        if (!vok[i]) continue;
        float4 *dst = reinterpret_cast<float4 *>(mine + (size_t)(tid + i * nthreads) * E);
#pragma unroll
        for (int e = 0; e < E; e += 4)
            dst[e / 4] = make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
    }
    if (!grid_barrier(p.ctrl, (unsigned)n_ctas)) {
        if (tid == 0 && p.status) atomicOr(p.status, CLADA_STATUS_TIMEOUT);
        return;
    }
    // columns in groups of 4 (float4); a warp sums one group: lane l adds partial rows l, l+32, ...
    // in order, then the 32 lane sums combine by butterfly.
    const int ngroups = d / 4;
    for (int q = cta + warp * n_ctas; q < ngroups; q += n_ctas * nwarps) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
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
static int launch_variant(const FfnParams &p, int threads, cudaStream_t st) {
    static int cached_ctas[64][kFfnMaxWarps + 1] = {};
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != CLADA_OK) return rc;
    auto kern = sparse_ffn_kernel<T, NV, G>;
    // dynamic shared memory: the kept-list share of one CTA at the smallest grid we may use
    const size_t smem = ((size_t)(p.d_ff / di.num_sms + 2) * sizeof(int) + 15) & ~(size_t)15;
    int &per_sm = cached_ctas[di.device & 63][threads / kWarp];
    if (per_sm == 0) {
        int occ = 0;
        CLADA_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, threads, smem));
        if (occ < 1) return CLADA_ERR_UNSUPPORTED;
        per_sm = occ > 4 ? 4 : occ;
    }
    const int grid = di.num_sms * per_sm;
    FfnParams params = p;
    void *args[] = {&params};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(threads);
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
    // threads: enough to cover a row with at most 4 vectors each, a multiple of 32, at most 256
    if (vpr <= 128) return launch_variant<T, 1, 4>(p, ((vpr + 31) / 32) * 32, st);
    if (vpr <= 256) return launch_variant<T, 1, 4>(p, 256, st);
    if (vpr <= 512) return launch_variant<T, 2, 2>(p, 256, st);
    if (vpr <= 768) return launch_variant<T, 3, 1>(p, 256, st);
    if (vpr <= 1024) return launch_variant<T, 4, 1>(p, 256, st);
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
    const size_t need = kWsCtrlBytes + (size_t)di.num_sms * 4 * layer->d_model * sizeof(float);
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
