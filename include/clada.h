/*
 * clada.h -- C ABI of the B200 (sm_100a) CLADA sparse gated FFN decode path.
 *
 * The library realises the data-parallel hot path of "Cognitive-Load-Aware
 * Dynamic Activation" (Algorithm 2 of the paper):
 *
 *   prefill :  per-neuron activation magnitudes A_j over the prompt
 *              (Eq. neuron_activation) and the baseline neuron subset
 *              { j : A_j >= tau_base } (Eq. base_threshold, last line);
 *   per step:  surprisal s_t and entropy H_t of the previous step's
 *              vocabulary distribution (Eqs. surprisal, entropy);
 *              tau_final = tau_base * (1 + lambda I(s_t > tau_s) + gamma I(H_t > tau_H))
 *              (Eq. final_threshold);
 *              mask regeneration A_j >= tau_final and the gated FFN over the
 *              kept neurons only (Algorithm 2, generation phase).
 *
 * Conventions
 * -----------
 *  - Unless a parameter says "host", every pointer is a DEVICE pointer owned
 *    by the caller.  The library allocates no device memory; scratch comes
 *    from a caller-provided workspace (clada_workspace_bytes / clada_workspace_init).
 *  - Calls validate on the host, enqueue their kernels on `stream`
 *    (a cudaStream_t passed as void*, NULL = default stream) and return
 *    without synchronising.
 *  - Matrices are row-major and dense.  Weight rows and x / X rows must start
 *    on 16-byte boundaries and d_model must be a multiple of 8.
 *  - Return value: CLADA_OK, or a negative clada_error; on error nothing was
 *    enqueued.  Conditions only the device can see (token id out of range,
 *    non-finite logit, a bounded wait that expired) OR bits of clada_status
 *    into the optional device word `status`; kernels never trap.
 *  - Two calls may run concurrently only with distinct workspaces.
 */
#ifndef CLADA_H_
#define CLADA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { CLADA_F32 = 0, CLADA_BF16 = 1, CLADA_F16 = 2 } clada_dtype;

typedef enum {
    CLADA_OK = 0,
    CLADA_ERR_NULL = -1,      /* a required pointer is NULL */
    CLADA_ERR_SHAPE = -2,     /* a size is <= 0, d_model % 8 != 0, offsets not ascending, ... */
    CLADA_ERR_ALIGN = -3,     /* a row base is not 16-byte aligned */
    CLADA_ERR_DTYPE = -4,     /* unknown or unsupported clada_dtype */
    CLADA_ERR_WORKSPACE = -5, /* workspace missing, misaligned or too small */
    CLADA_ERR_CUDA = -6,      /* a CUDA runtime call failed: see clada_last_cuda_error() */
    CLADA_ERR_UNSUPPORTED = -7 /* sizes beyond what the kernels were built for */
} clada_error;

typedef enum {
    CLADA_STATUS_BAD_TOKEN = 1,        /* token_id outside [0, V): surprisal = NaN */
    CLADA_STATUS_NONFINITE_LOGIT = 2,  /* +inf or NaN logit: surprisal = entropy = NaN */
    CLADA_STATUS_TIMEOUT = 4,          /* a bounded device-side wait gave up; outputs invalid,
                                          re-initialise the workspace before reusing it */
    CLADA_STATUS_BAD_INDEX = 8         /* a nested-list level, count or neuron index was out of range (clamped) */
} clada_status;

/* FFN form of a layer: the value z of neuron j for a token x from g = w_gate_j . x
 * and u = w_up_j . x (Eq. neuron_activation with the sigma of the model family,
 * Section 4.1).  The non-gated form has no w_up (pass NULL) and streams one
 * row fewer per neuron; biases are not part of the equation and are not applied. */
typedef enum {
    CLADA_ACT_SILU_GATED = 0, /* z = silu(g) * u                      (LLaMA, Mistral) */
    CLADA_ACT_GELU_GATED = 1, /* z = gelu(g) * u, tanh form of GELU   (Gemma)          */
    CLADA_ACT_RELU = 2        /* z = max(g, 0)                        (OPT)            */
} clada_activation;

/* One FFN layer.  Neuron j owns row j of each matrix, so its three
 * vectors are contiguous: w_gate row j = W_in,j, w_up row j = V_in,j,
 * w_down_t row j = column j of the output projection W_out
 * (text under Eq. neuron_activation). */
typedef struct clada_layer {
    int32_t d_model;          /* multiple of 8; <= 8192 (bf16, fp16) or 4096 (fp32) */
    int32_t d_ff;
    int32_t dtype;            /* clada_dtype of the weights and of x / X */
    int32_t activation;       /* clada_activation; 0 = SiLU-gated */
    const void *w_gate;       /* [d_ff, d_model] */
    const void *w_up;         /* [d_ff, d_model]; NULL for CLADA_ACT_RELU */
    const void *w_down_t;     /* [d_ff, d_model] */
    const float *w_down_norm; /* [d_ff] ||W_out,j||_2 (clada_down_norms); needed by the prefix calls only */
} clada_layer;

int clada_version(void);
const char *clada_status_string(int code);
/* Text of the last CUDA error seen by this thread's calls ("" if none). Host. */
const char *clada_last_cuda_error(void);

/* Bytes of workspace that suffice for any call on this layer with B
 * sequences and T_total prefix tokens in all (T_total = 0 for decode-only use).
 * 0 on invalid arguments. */
size_t clada_workspace_bytes(const clada_layer *layer, int32_t B, int64_t T_total);

/* Zero the workspace's control words.  Once after allocation, and again after
 * a CLADA_STATUS_TIMEOUT.  ws must be 256-byte aligned. */
int clada_workspace_init(void *ws, size_t ws_bytes, void *stream);

/* Measuring aid (the paper has no counterpart): reads `bytes` of device memory
 * at buf once (16-byte aligned, 16-byte loads that do not allocate in L1, as the
 * decode kernel's) and xors everything into *sink (device) so the reads are
 * kept.  Timed by the caller, it gives the read-only streaming bandwidth of the
 * device, the ceiling for the sparse FFN's weight rows. */
int clada_stream_read_probe(const void *buf, size_t bytes, uint32_t *sink, void *stream);

/* Self-test of the bounded device-side waits (the paper has no counterpart).
 * Every wait inside the decode kernels -- for a ring stage's mbarrier, for the
 * grid barrier -- gives up after a bounded number of polls and reports
 * CLADA_STATUS_TIMEOUT instead of hanging.  This call makes both kinds of wait
 * run out on purpose, in a form that cannot hang: two small CTAs wait on a
 * shared-memory barrier that nobody arrives at, then meet at the workspace's
 * grid barrier, which is told to expect one CTA more than the grid has.
 *   poll_limit  polls per wait before giving up, 1 .. 2^20 (a few thousand is plenty)
 *   report      out [2] int32, device: report[0] = 1 if the mbarrier wait gave up,
 *               report[1] = 1 if the grid barrier gave up (both are expected)
 *   status      optional device word; CLADA_STATUS_TIMEOUT is or-ed into it
 * Afterwards the workspace's control words are left as a timed-out decode
 * kernel leaves them (non-zero): call clada_workspace_init before the next
 * decode on this workspace, exactly as after a real CLADA_STATUS_TIMEOUT. */
int clada_selftest_bounded_waits(void *ws, size_t ws_bytes, uint32_t poll_limit, int32_t *report,
                                 int32_t *status, void *stream);

/* out[j] = ||W_out,j||_2 = the l2 norm of row j of w_down_t, fp32.  Once per
 * layer; the second factor of Eq. neuron_activation. */
int clada_down_norms(const clada_layer *layer, float *out /*[d_ff]*/, void *stream);

/* Eq. neuron_activation over B prompts (B <= 128).
 *   X            [T_total, d_model], the layer's input hidden states of all
 *                prompts back to back, in the weights' dtype
 *   seq_offsets  HOST int64 [B+1], ascending; prompt b = rows
 *                [seq_offsets[b], seq_offsets[b+1]); an empty prompt scores 0
 *   scores       out [B, d_ff] fp32:
 *                A[b,j] = sqrt(sum_t z_tj^2) * w_down_norm[j],
 *                z_tj = silu(w_gate_j . x_t) * (w_up_j . x_t)
 * Products of the stored values are exact; accumulation is fp32. */
int clada_prefix_scores(const clada_layer *layer, const void *X, const int64_t *seq_offsets,
                        int32_t B, float *scores, void *ws, size_t ws_bytes,
                        int32_t *status, void *stream);

/* Guard band.  Every neuron whose fp32 score lies within rel_band (relative)
 * of tau_base[b] * guard_mults[g] for some g gets its score recomputed with
 * fp64 accumulation and stored back rounded to fp32, so that the later
 * comparisons A_j >= tau are taken on correctly rounded scores where it
 * matters.  guard_mults: HOST [n_guard] (the multipliers decode will apply,
 * e.g. 1, 1+lambda, 1+gamma, 1+lambda+gamma), n_guard <= 8.
 * The paper has no counterpart; it only removes rounding noise from the
 * comparison the paper defines. */
int clada_refine_scores(const clada_layer *layer, const void *X, const int64_t *seq_offsets,
                        int32_t B, const float *tau_base /*[B]*/, const float *guard_mults,
                        int32_t n_guard, float rel_band, float *scores /*[B,d_ff] in/out*/,
                        void *ws, size_t ws_bytes, int32_t *status, void *stream);

/* Eq. base_threshold, last line, and Algorithm 2's mask generation: neuron j
 * of sequence b is kept iff scores[b,j] >= tau[b*tau_stride] (equality keeps;
 * NaN scores are cut).
 *   mask  out [B, d_ff] u8 (1 = kept), may be NULL
 *   idx   out [B, d_ff] int32, the kept neurons of b ascending in
 *         idx[b*d_ff .. b*d_ff+count[b]); the rest is left untouched; may be NULL
 *   count out [B] int32, may be NULL */
int clada_select(const float *scores, int32_t B, int32_t d_ff, const float *tau,
                 int64_t tau_stride, uint8_t *mask, int32_t *idx, int32_t *count,
                 void *stream);

/* Prefill phase of Algorithm 2 in one call: clada_prefix_scores, then (if
 * n_guard > 0) clada_refine_scores with rel_band 1e-4, then clada_select
 * against tau_base.  tau_base == NULL stops after the scores (used to
 * calibrate a threshold first). */
int clada_prefix_select(const clada_layer *layer, const void *X, const int64_t *seq_offsets,
                        int32_t B, const float *tau_base /*[B] or NULL*/,
                        const float *guard_mults /*host, may be NULL*/, int32_t n_guard,
                        float *scores, uint8_t *mask, int32_t *idx, int32_t *count,
                        void *ws, size_t ws_bytes, int32_t *status, void *stream);

/* Harness helper standing in for the offline threshold search (which is an
 * input to this path): tau_base[b] = 0.5*a + 0.5*b in fp32, a and b the
 * k_cut-th and (k_cut+1)-th smallest of scores[b,:], k_cut = floor(rho*d_ff + 0.5),
 * i.e. the threshold that cuts exactly k_cut neurons.  k_cut = 0 gives 0,
 * k_cut = d_ff gives +inf.  Scores must be non-negative (they are norms). */
int clada_tau_from_sparsity(const float *scores, int32_t B, int32_t d_ff, float rho,
                            float *tau_base /*[B]*/, void *stream);

/* Offline error-controlled threshold search (Eq. base_threshold) on a set of
 * validation prompts:
 *   tau_base = the largest eps with  mean_x CETT(x; eps) <= bound   (the paper uses 0.2),
 *   CETT(x; eps) = || sum_{A_j(x) < eps} n_j(x) ||_F / || MLP(x) ||_F,
 * where sample x is prompt b of X (rows seq_offsets[b] .. seq_offsets[b+1]), A_j(x)
 * its score, n_j(x) neuron j's contribution to the FFN output over the prompt's
 * tokens and MLP(x) the dense output.  CETT(x; .) only changes at scores of x, so
 * the candidates are the scores of all samples; the smallest one always
 * qualifies (nothing cut).
 *   X, seq_offsets, B   as in clada_prefix_scores (seq_offsets on the HOST, B <= 128)
 *   tau_base   out [1] device;  mean_cett  out [1] device, the mean CETT at tau_base, may be NULL
 *   scores     out [B, d_ff] fp32 (CUDA-core accumulation for every dtype)
 *   ws         clada_cett_workspace_bytes() bytes, 256-byte aligned; d_ff <= 16384
 * Not on the decode path: run once per layer before serving. */
size_t clada_cett_workspace_bytes(const clada_layer *layer, const int64_t *seq_offsets, int32_t B);
int clada_cett_threshold_search(const clada_layer *layer, const void *X, const int64_t *seq_offsets,
                                int32_t B, float bound, float *tau_base, float *mean_cett,
                                float *scores, void *ws, size_t ws_bytes, int32_t *status,
                                void *stream);
/* After a search, sample `sample`'s curve from the same workspace:
 * cum_out [d_ff+1] fp64 device, cum_out[k] = || sum of the k lowest-scored neurons' outputs ||_F^2
 * (so CETT with k neurons cut = sqrt(cum_out[k] / cum_out[d_ff])); order_out [d_ff]
 * int32 device, the neurons in ascending score order (ties by index); may be NULL. */
int clada_cett_curve(const clada_layer *layer, const int64_t *seq_offsets, int32_t B, int32_t sample,
                     const void *ws, size_t ws_bytes, double *cum_out, int32_t *order_out,
                     void *stream);

/* Eqs. surprisal and entropy, natural log, for B vocabulary rows:
 *   P = softmax(logits[b,:]);  surprisal[b] = -log P[token_id[b]];
 *   entropy[b] = -sum_w P[w] log P[w]   (0 log 0 = 0: -inf logits allowed).
 *   logits     [B, V] with row stride row_stride elements, fp32, bf16 or fp16
 *   token_id   [B] int32
 * Out-of-range token -> surprisal NaN + CLADA_STATUS_BAD_TOKEN;
 * +inf / NaN logit -> both NaN + CLADA_STATUS_NONFINITE_LOGIT. */
int clada_cogload(const void *logits, int32_t logits_dtype, int32_t B, int64_t V,
                  int64_t row_stride, const int32_t *token_id, float *surprisal,
                  float *entropy, int32_t *status, void *stream);

/* Eq. final_threshold for B sequences and L layers, fp32, evaluated left to
 * right without fused multiply-add:
 *   m = 1; if (surprisal[b] > tau_s) m += lambda[l]; if (entropy[b] > tau_H) m += gamma[l];
 *   tau_final[b,l] = tau_base[b,l] * m
 * lambda, gamma: [L] signed per-layer coefficients (the paper picks 0.80, 0.12). */
int clada_adjust_threshold(const float *tau_base /*[B,L]*/, const float *lambda,
                           const float *gamma, float tau_s, float tau_H,
                           const float *surprisal /*[B]*/, const float *entropy /*[B]*/,
                           int32_t B, int32_t L, float *tau_final /*[B,L]*/, void *stream);

/* clada_cogload followed by clada_adjust_threshold in one launch (the two
 * per-step scalar stages of Algorithm 2's generation loop).  surprisal and
 * entropy are still written. */
int clada_cogload_adjust(const void *logits, int32_t logits_dtype, int32_t B, int64_t V,
                         int64_t row_stride, const int32_t *token_id,
                         const float *tau_base, const float *lambda, const float *gamma,
                         float tau_s, float tau_H, int32_t L, float *surprisal,
                         float *entropy, float *tau_final, int32_t *status, void *stream);

/* Algorithm 2, generation phase, one layer, one token per sequence:
 *   kept_b = { j : scores[b,j] >= tau_final[b*tau_stride] }
 *   y[b,:] = sum_{j in kept_b} silu(w_gate_j . x_b) * (w_up_j . x_b) * w_down_t[j,:]
 * Only the kept neurons' rows are read.  No bias, no rescaling.
 *   x        [B, d_model] in the layer's dtype
 *   y        out [B, d_model], y_dtype fp32, bf16 or fp16
 *   mask_out / idx_out / count_out: optional (NULL), as in clada_select
 * Accumulation is fp32 in a fixed order: results are bit-identical run to run.
 * A batch of a 16-bit layer with d_ff <= 128 x (SM count) runs 16 sequences at
 * a time through ONE dense pass over the layer while 3 or more are left (at 40-60 %
 * sparsity the union of that many kept sets is most of the layer; both contractions on
 * the tensor cores, the hidden activations carried exactly as three 16-bit
 * parts, each sequence's mask applied to its own activations: same 1e-5 as the
 * CUDA-core path).  What is left, and every batch of other layers, runs in tiles
 * of 4 or 2 sequences that read the union of their kept rows once, preceded by
 * one small launch that tests the tiled sequences' scores once.
 * The workspace (clada_workspace_bytes(layer, B, 0) bytes at least) must have
 * been initialised with clada_workspace_init; with a workspace too small for the
 * dense pass's scratch but large enough for tiles the call uses tiles. */
int clada_sparse_ffn_decode(const clada_layer *layer, const void *x, int32_t B,
                            const float *scores /*[B,d_ff]*/, const float *tau_final,
                            int64_t tau_stride, void *y, int32_t y_dtype,
                            uint8_t *mask_out, int32_t *idx_out, int32_t *count_out,
                            void *ws, size_t ws_bytes, int32_t *status, void *stream);

/* Algorithm 2's sparse forward pass over a stack of L layers for one decode
 * step: clada_sparse_ffn_decode for l = 0 .. L-1 in one call.
 *   layers     HOST array of L layers of one shape, dtype and FFN form
 *   x          [L, B, d_model]: the input hidden state of every layer (this path has
 *              no attention, residual or norm between FFNs, so each layer's input is given)
 *   scores     [L, B, d_ff]
 *   tau_final  [B, L] as clada_adjust_threshold writes it
 *   y          out [L, B, d_model]
 * All layers are validated before anything is enqueued.
 * One sequence (B = 1, L >= 2) runs all layers in ONE persistent launch (up to
 * 128 layers per launch): the weight stream does not stop at layer
 * boundaries, the outputs are bit for bit those of the per-layer call.  One
 * small launch before it tests every layer's scores against its threshold
 * (4 bytes per 32 neurons, kept behind the partial rows in the workspace).  This
 * needs the workspace clada_workspace_bytes(layer, 1, 0) gives; with a smaller
 * one, for a batch, or for rows too wide for a ring of four stages
 * (d_model 8192 in 16-bit types) the call runs the per-layer launches in a loop. */
int clada_sparse_ffn_decode_layers(const clada_layer *layers, int32_t L, const void *x, int32_t B,
                                   const float *scores, const float *tau_final, void *y,
                                   int32_t y_dtype, void *ws, size_t ws_bytes, int32_t *status,
                                   void *stream);

/* clada_sparse_ffn_decode for callers that cannot allocate device memory (the
 * paper has no counterpart; this is a deployment variant of the call above).
 * Think of a plug-in that runs inside another engine's execution step, where
 * the host engine owns and budgets all device memory and allocation calls are
 * forbidden there, or of a server whose memory plan is frozen after start-up.
 * Same arguments and results as clada_sparse_ffn_decode, minus the workspace:
 * the kernel's scratch is a fixed array inside the library (about 5 MiB, held
 * by every GPU that loads the library until the process exits).  The call
 * itself allocates nothing.
 *  - Limits: d_model <= 8192 and a device with at most 160 SMs; beyond that the
 *    call returns CLADA_ERR_UNSUPPORTED (clada_last_cuda_error() says why)
 *    and enqueues nothing.  Every refusal happens before the first enqueue.
 *  - Batches: the array holds 160 x 8192 fp32 partial outputs.  B >= 2 runs in
 *    the largest launches whose scratch fits: the dense pass of
 *    clada_sparse_ffn_decode (SMs / 4 x B x d_model fp32 values plus SMs / 4
 *    images of the hidden activations of up to 48 KB: on a 148-SM device 8
 *    sequences fit up to d_model 2048, at 4096 they do not), else
 *    the largest tiles of sequences (4, 2 or 1 per launch; one row per SM and
 *    sequence of a tile, together with the batch's keep bits, 4 bytes per
 *    sequence and 32 neurons: tiles of 4 up to d_model 2048, tiles of 2 up to
 *    d_model 4096, one sequence per launch above that).  Results per sequence
 *    are those of clada_sparse_ffn_decode; smaller launches only read the
 *    shared weight rows once per launch instead of once per larger one.
 *  - The first call on a device looks up the array's device address; make that
 *    first call outside any stream capture.
 *  - All calls share the one array and it keeps the previous call's contents;
 *    each call clears the control words it needs at zero, in stream order.
 *    Two calls whose kernels overlap on the GPU (different streams) race on
 *    the array: serialise them, or use the workspace variant. */
int clada_sparse_ffn_decode_static(const clada_layer *layer, const void *x, int32_t B,
                                   const float *scores /*[B,d_ff]*/, const float *tau_final,
                                   int64_t tau_stride, void *y, int32_t y_dtype,
                                   uint8_t *mask_out, int32_t *idx_out, int32_t *count_out,
                                   int32_t *status, void *stream);

/* ---- Dense prefill FFN with the statistics as a by-product, in chunks ----------
 *
 * Algorithm 2's prefill phase runs the prompt through the dense layer; the
 * paper's Limitations name the pre-filling phase of long prompts (over 2048
 * tokens) as a cost, and its long-context table reaches 32K-token prompts.  These three
 * calls take the statistics from the prefill FFN itself and let a prompt arrive
 * in chunks (chunked prefill):
 *
 * clada_prefix_accumulate: one chunk.  Arguments as clada_prefix_scores, but
 *   sumsq  in/out [B, d_ff] fp32, device: running sum over the tokens seen so
 *          far of z[t,j]^2 per (prompt, neuron); zero it before the first chunk.
 *          seq_offsets describe THIS chunk's rows of X (a prompt may have no
 *          rows in a chunk).
 *   Z      out [T_chunk, d_ff] in the layer's element type, device, or NULL:
 *          the hidden activations z[t,j] themselves, rounded once to the
 *          element type (bf16 / fp16 layers only; CLADA_ERR_UNSUPPORTED for
 *          fp32 layers with Z != NULL).  d_ff must then be a multiple of 8.
 *   w_down_norm is not needed.  Workspace as for clada_prefix_scores of the chunk.
 * clada_prefix_finish: scores[b,j] = sqrt(sumsq[b,j]) * w_down_norm[j] (fp32),
 *   the same last step as clada_prefix_scores.  The guard band
 *   (clada_refine_scores) needs the whole prompt's X; with chunks that are not
 *   kept it is skipped and the scores carry the fp32 accumulation error.
 * clada_prefill_down: Y [T, d_model] (y_dtype) = Z [T, d_ff] . w_down^T with
 *   w_down [d_model, d_ff] in the paper's layout (W_out, neuron j = column j;
 *   the decode path's w_down_t is its transpose), tensor cores, fp32
 *   accumulation.  bf16 / fp16 layers; d_ff a multiple of 8; all pointers
 *   16-byte aligned.  Together with Z from clada_prefix_accumulate this is the
 *   layer's dense prefill output.
 *   ws / ws_bytes: optional workspace (NULL, 0: none).  A short prompt has fewer
 *   output tiles than the device has SMs; with a workspace of
 *   clada_workspace_bytes(layer, 1, T) bytes the K dimension (d_ff) of each tile
 *   is then split among up to 8 CTAs, whose fp32 partial outputs are added in a
 *   fixed order (same result on every call; it differs from the unsplit sum only
 *   by fp32 rounding).  A workspace too small for that is not an error: the call
 *   runs unsplit.  CLADA_ERR_WORKSPACE: ws not 256-byte aligned or smaller than
 *   its control block. */
int clada_prefix_accumulate(const clada_layer *layer, const void *X, const int64_t *seq_offsets,
                            int32_t B, float *sumsq, void *Z, void *ws, size_t ws_bytes,
                            int32_t *status, void *stream);
int clada_prefix_finish(const clada_layer *layer, const float *sumsq, int32_t B, float *scores,
                        void *stream);
int clada_prefill_down(const clada_layer *layer, const void *w_down, const void *Z, int64_t T,
                       void *Y, int32_t y_dtype, void *ws, size_t ws_bytes, int32_t *status,
                       void *stream);

/* ---- Nested index lists: the masks of Eq. final_threshold in compressed form ----
 *
 * The paper names mask memory as a limitation and mask compression as future
 * work (Limitations; Conclusion).  Eq. final_threshold can only yield
 * tau_base * m, m in {1, 1+lambda, 1+gamma, (1+lambda)+gamma}, and a kept set
 * is { j : A_j >= tau }: all four kept sets of a sequence are leading parts of
 * one list, its neurons in descending order of score.
 *
 * clada_nested_build, once per (sequence, layer) after the prefix statistics:
 *   scores     [B, d_ff] fp32, device (clada_prefix_scores / clada_refine_scores)
 *   tau_base   sequence b reads tau_base[b * tau_stride], device
 *   lambda, gamma  the layer's coefficients (host values, signed)
 *   order  out [B, d_ff] int32, device: neurons by descending score, equal
 *              scores by ascending index; zero scores of either sign come after
 *              every positive one and NaN scores last of all, which is where
 *              the comparison A_j >= tau puts them
 *   counts out [B, 4] int32, device: counts[b][k] = |{ j : A_bj >= tau_k }|,
 *              tau_k = fl32(tau_base_b * m_k), m = {1, 1+lambda, 1+gamma,
 *              (1+lambda)+gamma} in fp32 -- bit for bit the thresholds that
 *              clada_adjust_threshold produces, so order[b][0 .. counts[b][k])
 *              is exactly the kept set clada_select would give at level k.
 *   d_ff <= 32768 (every CTA holds the score vector in shared memory); otherwise
 *   CLADA_ERR_UNSUPPORTED.  Nothing is allocated.
 *
 * clada_cogload_level, per decode step: clada_cogload plus
 *   level  out [B] int32, device: I(s > tau_s) + 2 I(H > tau_H), the same fp32
 *              comparisons as the indicators of Eq. final_threshold (a NaN
 *              surprisal compares false).
 *
 * clada_sparse_ffn_decode_nested, per decode step and layer: the sparse FFN over
 * order[b][0 .. counts[b][level[b]]).  Same x / y / workspace / status rules as
 * clada_sparse_ffn_decode (workspace of clada_workspace_bytes(layer, 1, 0) is
 * enough); sequences run one launch each.  The sum over the kept neurons runs
 * in list order split over the CTAs, so y agrees with clada_sparse_ffn_decode to
 * rounding (fp32 sums in another order), not bit for bit.  count_out [B] or
 * NULL receives the kept count.  A level outside 0..3, a count outside
 * [0, d_ff] or an index outside [0, d_ff) is clamped into range, so no access
 * leaves the layer, and CLADA_STATUS_BAD_INDEX is or-ed into *status. */
int clada_nested_build(const float *scores, int32_t B, int32_t d_ff, const float *tau_base,
                       int64_t tau_stride, float lambda, float gamma, int32_t *order,
                       int32_t *counts, void *stream);
int clada_cogload_level(const void *logits, int32_t logits_dtype, int32_t B, int64_t V,
                        int64_t row_stride, const int32_t *token_id, float tau_s, float tau_H,
                        float *surprisal, float *entropy, int32_t *level, int32_t *status,
                        void *stream);
int clada_sparse_ffn_decode_nested(const clada_layer *layer, const void *x, int32_t B,
                                   const int32_t *order /*[B,d_ff]*/, const int32_t *counts /*[B,4]*/,
                                   const int32_t *level /*[B]*/, void *y, int32_t y_dtype,
                                   int32_t *count_out, void *ws, size_t ws_bytes, int32_t *status,
                                   void *stream);

#ifdef __cplusplus
}
#endif
#endif /* CLADA_H_ */
