/*
 * CLADA oracle -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow CPU restatement of what the cognitive-load-aware sparse gated
 * FFN computes, written from the paper's definitions.  Every sum is a plain
 * loop in double precision in the order the definition states; there is no
 * blocking, fusion or reordering.  It shares no code with the CUDA library and
 * is only ever called by the tests, the smoke check and the CPU-baseline leg
 * of the benchmark.
 *
 * Weight layout here is the paper's own: W_in and V_in are [d_ff, d_model]
 * with neuron j in row j; W_out is [d_model, d_ff] with neuron j in COLUMN j
 * (Section 3.2.1, text under Eq. neuron_activation).
 *
 * Pins (tests/test_oracle_pins.py): entropy/surprisal closed forms, literal
 * Frobenius form of the score, brute-force selection on tiny layers, dense
 * FFN against an independent float64 matrix formulation, zero-sparsity
 * identity, CETT identity; the offline threshold search against the definition
 * evaluated through the per-token FFN routines, a closed form for orthogonal
 * neuron outputs, and brute force over all candidates; the GELU-gated and
 * non-gated ReLU forms against a library formulation, a worked two-neuron
 * example and the tanh formula typed out.  The whole of Algorithm 2 end to end has no
 * published trace: parity unpinned beyond those per-step pins.
 *
 * Element types: 0 = IEEE fp32, 1 = bfloat16 (uint16 bit patterns), 2 = IEEE
 * fp16, the type of the paper's latency runs (Efficiency Evaluation).  All widen
 * to double exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { OR_F32 = 0, OR_BF16 = 1, OR_F16 = 2 };

/* IEEE 754 binary16 from its bit pattern: 1 sign bit, 5 exponent bits (bias
 * 15), 10 fraction bits; exponent 0 is zero / subnormal (fraction * 2^-24),
 * exponent 31 is inf / NaN. */
static double half_bits_to_double(uint16_t h)
{
    const int sign = (h >> 15) & 1, ex = (h >> 10) & 0x1f, frac = h & 0x3ff;
    double v;
    if (ex == 0)
        v = ldexp((double)frac, -24);
    else if (ex == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)frac / 1024.0, ex - 15);
    return sign ? -v : v;
}

static double elem(const void *p, int dtype, size_t i)
{
    if (dtype == OR_F32)
        return (double)((const float *)p)[i];
    if (dtype == OR_F16)
        return half_bits_to_double(((const uint16_t *)p)[i]);
    uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* sigma of Eq. neuron_activation read as SiLU: g * logistic(g). */
static double silu(double g) { return g / (1.0 + exp(-g)); }

/* The FFN forms of the model families the paper evaluates (Section 4.1):
 *   OR_SILU_GATED  z = silu(g) * u                       (LLaMA, Mistral)
 *   OR_GELU_GATED  z = gelu(g) * u, tanh form of GELU    (Gemma)
 *   OR_RELU        z = max(g, 0), no V_in factor         (OPT)
 * with g = W_in,j . x and u = V_in,j . x.  The gated forms are Eq.
 * neuron_activation with that sigma; the non-gated one is the same equation
 * with the V_in factor absent, the only reading an FFN without a gate
 * projection admits.  Biases are not part of the equation and are left out. */
#define OR_PI 3.14159265358979323846
enum { OR_SILU_GATED = 0, OR_GELU_GATED = 1, OR_RELU = 2 };

static int is_gated(int act) { return act != OR_RELU; }

static double neuron_value(int act, double g, double u)
{
    switch (act) {
    case OR_GELU_GATED: {
        /* 0.5 g (1 + tanh(sqrt(2/pi) (g + 0.044715 g^3))) */
        double inner = sqrt(2.0 / OR_PI) * (g + 0.044715 * g * g * g);
        return 0.5 * g * (1.0 + tanh(inner)) * u;
    }
    case OR_RELU:
        return g > 0.0 ? g : 0.0;
    default:
        return silu(g) * u;
    }
}

/* The widening itself, exposed so that a test can check every bit pattern. */
void oracle_widen(int dtype, const void *p, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = elem(p, dtype, (size_t)i);
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ *
 * Eq. neuron_activation, factored form.
 *
 * For sequence b with prefix rows [off[b], off[b+1]) of X and neuron j:
 *   z_t = silu(W_in,j . x_t) * (V_in,j . x_t)
 *   A_j = || z_{:,j} (outer) W_out,j ||  =  sqrt(sum_t z_t^2) * sqrt(sum_i W_out[i,j]^2)
 * (the matrix inside the norm has rank one, so its Frobenius and spectral
 * norms are the same number).
 * scores: [B, d_ff] double.
 * ------------------------------------------------------------------ */
void oracle_neuron_scores(int dtype, const void *X, const int64_t *off, int B,
                          int d_model, int d_ff, const void *W_in,
                          const void *V_in, const void *W_out, double *scores, int act)
{
#pragma omp parallel for schedule(dynamic, 8)
    for (int j = 0; j < d_ff; ++j) {
        double wnorm2 = 0.0;
        for (int i = 0; i < d_model; ++i) {
            double w = elem(W_out, dtype, (size_t)i * d_ff + j);
            wnorm2 += w * w;
        }
        for (int b = 0; b < B; ++b) {
            double zz = 0.0;
            for (int64_t t = off[b]; t < off[b + 1]; ++t) {
                double g = 0.0, u = 0.0;
                for (int k = 0; k < d_model; ++k) {
                    double x = elem(X, dtype, (size_t)t * d_model + k);
                    g += elem(W_in, dtype, (size_t)j * d_model + k) * x;
                    if (is_gated(act))
                        u += elem(V_in, dtype, (size_t)j * d_model + k) * x;
                }
                double z = neuron_value(act, g, u);
                zz += z * z;
            }
            scores[(size_t)b * d_ff + j] = sqrt(zz) * sqrt(wnorm2);
        }
    }
}

/* Eq. neuron_activation, literal form for ONE sequence of T rows: build the
 * T x d_model matrix M[t,i] = z_t * W_out[i,j] and take its Frobenius norm.
 * Tiny sizes only (allocates T*d_model doubles per neuron). */
void oracle_neuron_scores_literal(int dtype, const void *X, int T, int d_model,
                                  int d_ff, const void *W_in, const void *V_in,
                                  const void *W_out, double *scores, int act)
{
    double *M = (double *)malloc((size_t)T * d_model * sizeof(double));
    for (int j = 0; j < d_ff; ++j) {
        for (int t = 0; t < T; ++t) {
            double g = 0.0, u = 0.0;
            for (int k = 0; k < d_model; ++k) {
                double x = elem(X, dtype, (size_t)t * d_model + k);
                g += elem(W_in, dtype, (size_t)j * d_model + k) * x;
                if (is_gated(act))
                    u += elem(V_in, dtype, (size_t)j * d_model + k) * x;
            }
            double z = neuron_value(act, g, u);
            for (int i = 0; i < d_model; ++i)
                M[(size_t)t * d_model + i] = z * elem(W_out, dtype, (size_t)i * d_ff + j);
        }
        double fro2 = 0.0;
        for (size_t q = 0; q < (size_t)T * d_model; ++q)
            fro2 += M[q] * M[q];
        scores[j] = sqrt(fro2);
    }
    free(M);
}

/* Eq. base_threshold, last line: S_cut = { j : A_j < eps }.  A neuron is kept
 * iff A_j >= tau (equality keeps).  idx lists the kept neurons ascending.
 * Returns the number kept. */
int oracle_select(const double *scores, int d_ff, double tau, uint8_t *mask,
                  int32_t *idx)
{
    int count = 0;
    for (int j = 0; j < d_ff; ++j) {
        int keep = !(scores[j] < tau);
        if (mask)
            mask[j] = (uint8_t)keep;
        if (keep) {
            if (idx)
                idx[count] = j;
            ++count;
        }
    }
    return count;
}

/* Eqs. surprisal and entropy for one vocabulary row of logits (natural log):
 *   P = softmax(logits); s = -log P[token]; H = -sum_w P[w] log P[w]
 * with 0 log 0 := 0, so a logit of -inf contributes nothing.
 * Returns 0, or 1 if token is outside [0, V) (then s = NaN). */
int oracle_cogload(int dtype, const void *logits, int64_t V, int64_t token,
                   double *surprisal, double *entropy)
{
    double m = -INFINITY;
    for (int64_t w = 0; w < V; ++w) {
        double l = elem(logits, dtype, (size_t)w);
        if (l > m)
            m = l;
    }
    double Z = 0.0;
    for (int64_t w = 0; w < V; ++w)
        Z += exp(elem(logits, dtype, (size_t)w) - m);
    double logZ = log(Z);
    double H = 0.0;
    for (int64_t w = 0; w < V; ++w) {
        double logp = elem(logits, dtype, (size_t)w) - m - logZ;
        if (logp > -INFINITY)
            H -= exp(logp) * logp;
    }
    *entropy = H;
    if (token < 0 || token >= V) {
        *surprisal = NAN;
        return 1;
    }
    *surprisal = -(elem(logits, dtype, (size_t)token) - m - logZ);
    return 0;
}

/* Eq. final_threshold for B sequences and L layers:
 *   tau_final[b,l] = tau_base[b,l] * (1 + lambda[l]*I(s_b > tau_s) + gamma[l]*I(H_b > tau_H)).
 * The multiplier and the product are taken in fp32, left to right, with no
 * fused multiply-add (this file is compiled with -ffp-contract=off), so the
 * result is a definite fp32 number.  The indicators compare in double. */
void oracle_adjust_threshold(const float *tau_base, const float *lambda,
                             const float *gamma, float tau_s, float tau_H,
                             const double *surprisal, const double *entropy,
                             int B, int L, float *tau_final)
{
    for (int b = 0; b < B; ++b) {
        int hi_s = surprisal[b] > (double)tau_s;
        int hi_H = entropy[b] > (double)tau_H;
        for (int l = 0; l < L; ++l) {
            volatile float mult = 1.0f;
            if (hi_s)
                mult = mult + lambda[l];
            if (hi_H)
                mult = mult + gamma[l];
            volatile float t = tau_base[(size_t)b * L + l] * mult;
            tau_final[(size_t)b * L + l] = t;
        }
    }
}

/* Algorithm 2, mask regeneration + sparse forward pass, one token x:
 *   mask_j = (A_j >= tau);   y = sum_{j kept, ascending} silu(W_in,j.x) (V_in,j.x) W_out[:,j]
 * No bias, no rescaling of the kept neurons.  mask_out may be NULL.
 * Returns the number of kept neurons. */
int oracle_sparse_ffn(int dtype, const void *x, int d_model, int d_ff,
                      const void *W_in, const void *V_in, const void *W_out,
                      const double *scores, double tau, double *y,
                      uint8_t *mask_out, int act)
{
    double *h = (double *)calloc((size_t)d_ff, sizeof(double));
    uint8_t *keep = (uint8_t *)malloc((size_t)d_ff);
    int count = 0;
    for (int j = 0; j < d_ff; ++j) {
        keep[j] = (uint8_t)!(scores[j] < tau);
        count += keep[j];
        if (mask_out)
            mask_out[j] = keep[j];
    }
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d_ff; ++j) {
        if (!keep[j])
            continue;
        double g = 0.0, u = 0.0;
        for (int k = 0; k < d_model; ++k) {
            double xv = elem(x, dtype, (size_t)k);
            g += elem(W_in, dtype, (size_t)j * d_model + k) * xv;
            if (is_gated(act))
                u += elem(V_in, dtype, (size_t)j * d_model + k) * xv;
        }
        h[j] = neuron_value(act, g, u);
    }
#pragma omp parallel for schedule(static)
    for (int i = 0; i < d_model; ++i) {
        double acc = 0.0;
        for (int j = 0; j < d_ff; ++j)
            if (keep[j])
                acc += h[j] * elem(W_out, dtype, (size_t)i * d_ff + j);
        y[i] = acc;
    }
    free(h);
    free(keep);
    return count;
}

/* The dense gated FFN, y = W_out (silu(W_in x) * (V_in x)): the
 * zero-sparsity reference the sparse pass must reduce to. */
void oracle_dense_ffn(int dtype, const void *x, int d_model, int d_ff,
                      const void *W_in, const void *V_in, const void *W_out,
                      double *y, int act)
{
    double *h = (double *)malloc((size_t)d_ff * sizeof(double));
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d_ff; ++j) {
        double g = 0.0, u = 0.0;
        for (int k = 0; k < d_model; ++k) {
            double xv = elem(x, dtype, (size_t)k);
            g += elem(W_in, dtype, (size_t)j * d_model + k) * xv;
            if (is_gated(act))
                u += elem(V_in, dtype, (size_t)j * d_model + k) * xv;
        }
        h[j] = neuron_value(act, g, u);
    }
#pragma omp parallel for schedule(static)
    for (int i = 0; i < d_model; ++i) {
        double acc = 0.0;
        for (int j = 0; j < d_ff; ++j)
            acc += h[j] * elem(W_out, dtype, (size_t)i * d_ff + j);
        y[i] = acc;
    }
    free(h);
}

/* ------------------------------------------------------------------ *
 * The dense prefill FFN whose by-product the statistics are (Algorithm 2,
 * prefill phase: the prompt runs through the dense layer).
 *
 * Half-precision models keep the hidden activation z in the storage type
 * between the two projections; round_z != 0 reproduces that: z is computed in
 * double, rounded to fp32 (the accumulator type) and then to the storage type,
 * both to nearest even, before the down projection.  round_z == 0 keeps z in
 * double (then Y[t] equals oracle_dense_ffn of row t).
 * ------------------------------------------------------------------ */

/* v rounded to nearest even in a binary format with p significand bits (hidden
 * bit included), minimum normal exponent emin and largest finite value vmax. */
static double round_to_format(double v, int p, int emin, double vmax)
{
    if (v == 0.0 || isnan(v) || isinf(v))
        return v;
    int e;
    (void)frexp(fabs(v), &e);            /* |v| = f * 2^e, f in [0.5, 1)  ->  exponent e - 1 */
    int ex = e - 1;
    if (ex < emin)
        ex = emin;                       /* subnormal range: fixed quantum */
    const double quantum = ldexp(1.0, ex - (p - 1));
    const double r = nearbyint(v / quantum) * quantum;   /* default rounding mode: ties to even */
    if (fabs(r) > vmax)
        return v > 0 ? INFINITY : -INFINITY;
    return r;
}

double oracle_round_storage(int dtype, double v)
{
    const double f = (double)(float)v;   /* the fp32 accumulator value */
    if (dtype == OR_BF16)
        return round_to_format(f, 8, -126, 3.3895313892515355e38);
    if (dtype == OR_F16)
        return round_to_format(f, 11, -14, 65504.0);
    return f;
}

/* Z[t, j] = value of neuron j for token t (rounded to the storage type if round_z). */
void oracle_prefill_hidden(int dtype, const void *X, int T, int d_model, int d_ff,
                           const void *W_in, const void *V_in, int act, int round_z, double *Z)
{
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d_ff; ++j) {
        for (int t = 0; t < T; ++t) {
            double g = 0.0, u = 0.0;
            for (int k = 0; k < d_model; ++k) {
                double x = elem(X, dtype, (size_t)t * d_model + k);
                g += elem(W_in, dtype, (size_t)j * d_model + k) * x;
                if (is_gated(act))
                    u += elem(V_in, dtype, (size_t)j * d_model + k) * x;
            }
            double z = neuron_value(act, g, u);
            Z[(size_t)t * d_ff + j] = round_z ? oracle_round_storage(dtype, z) : z;
        }
    }
}

/* Y[t, i] = sum_j Z[t, j] W_out[i, j]: the down projection of given hidden activations. */
void oracle_down_proj(int dtype, const double *Z, int T, int d_model, int d_ff, const void *W_out, double *Y)
{
#pragma omp parallel for schedule(static)
    for (int i = 0; i < d_model; ++i) {
        for (int t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int j = 0; j < d_ff; ++j)
                acc += Z[(size_t)t * d_ff + j] * elem(W_out, dtype, (size_t)i * d_ff + j);
            Y[(size_t)t * d_model + i] = acc;
        }
    }
}

/* Mask compression by nesting.  Eq. final_threshold can only produce
 * tau_base * {1, 1+lambda, 1+gamma, 1+lambda+gamma}, and the kept set of any
 * threshold is { j : A_j >= tau }, so every kept set is a leading part of ONE
 * list: the neurons in descending order of score (equal scores in ascending
 * index order).  order receives that list; counts[k] = |{ j : A_j >= taus[k] }|,
 * so the kept set at level k is order[0 .. counts[k]).  (The paper names mask
 * memory as a limitation and mask compression as future work; this is the
 * plain definition of the compressed form, not an algorithm of the paper.) */
typedef struct { double a; int32_t j; } or_rank;

static int cmp_rank_desc(const void *x, const void *y)
{
    const or_rank *p = (const or_rank *)x, *q = (const or_rank *)y;
    if (p->a > q->a) return -1;
    if (p->a < q->a) return 1;
    return (p->j > q->j) - (p->j < q->j);
}

void oracle_nested_lists(const double *scores, int d_ff, const double *taus, int n_levels,
                         int32_t *order, int32_t *counts)
{
    or_rank *r = (or_rank *)malloc((size_t)d_ff * sizeof(or_rank));
    for (int j = 0; j < d_ff; ++j) { r[j].a = scores[j]; r[j].j = j; }
    qsort(r, (size_t)d_ff, sizeof(or_rank), cmp_rank_desc);
    for (int j = 0; j < d_ff; ++j) order[j] = r[j].j;
    free(r);
    for (int k = 0; k < n_levels; ++k) {
        int c = 0;
        for (int j = 0; j < d_ff; ++j)
            c += !(scores[j] < taus[k]);
        counts[k] = c;
    }
}

/* Which of the four thresholds Eq. final_threshold yields for a token:
 * level = I(s > tau_s) + 2 I(H > tau_H). */
int oracle_load_level(double surprisal, double entropy, double tau_s, double tau_H)
{
    return (surprisal > tau_s ? 1 : 0) + (entropy > tau_H ? 2 : 0);
}

/* Harness helper (stands in for the offline threshold search, which is an
 * input to the path): the threshold that cuts exactly k_cut = floor(rho*F+0.5)
 * neurons of an fp32 score vector, placed midway between the k_cut-th and
 * (k_cut+1)-th smallest scores.  Midpoint taken in fp32 as 0.5f*a + 0.5f*b.
 * k_cut == 0 gives 0 (keep all); k_cut == F gives +inf (cut all). */
static int cmp_float(const void *a, const void *b)
{
    float x = *(const float *)a, y = *(const float *)b;
    return (x > y) - (x < y);
}

float oracle_tau_from_sparsity(const float *scores, int d_ff, double rho)
{
    int k_cut = (int)floor(rho * d_ff + 0.5);
    if (k_cut <= 0)
        return 0.0f;
    if (k_cut >= d_ff)
        return INFINITY;
    float *s = (float *)malloc((size_t)d_ff * sizeof(float));
    memcpy(s, scores, (size_t)d_ff * sizeof(float));
    qsort(s, (size_t)d_ff, sizeof(float), cmp_float);
    volatile float lo = 0.5f * s[k_cut - 1];
    volatile float hi = 0.5f * s[k_cut];
    volatile float mid = lo + hi;
    free(s);
    return mid;
}

/* ------------------------------------------------------------------ *
 * Layer-wise base threshold (Eq. base_threshold), offline search.
 *
 *   tau_base = argmax eps  s.t.  E_{x in D_val}[ CETT(x; eps) ] <= bound,
 *   CETT(x; eps) = || sum_{j in S_cut} n_j(x) ||_2 / || MLP(x) ||_2,   S_cut = { j : A_j(x) < eps }.
 *
 * A validation sample x is one sequence of T tokens; A_j(x) is its score of
 * Eq. neuron_activation; n_j(x) is neuron j's contribution to the FFN output over
 * all T tokens (a T x d_model matrix), MLP(x) the dense output, norms Frobenius.
 *
 * oracle_cett_curve: for ONE sample, cett[k] = CETT when exactly the k
 * lowest-scored neurons are cut, k = 0 .. d_ff (cett[0] = 0, cett[d_ff] = 1),
 * by accumulating the cut neurons' outputs in ascending score order (ties in
 * index order).  Also returns the scores and that order.
 * ------------------------------------------------------------------ */
typedef struct { double a; int j; } or_pair;
static int cmp_pair(const void *p, const void *q)
{
    const or_pair *x = (const or_pair *)p, *y = (const or_pair *)q;
    if (x->a < y->a) return -1;
    if (x->a > y->a) return 1;
    return (x->j > y->j) - (x->j < y->j);
}

void oracle_cett_curve(int dtype, const void *X, int T, int d_model, int d_ff,
                       const void *W_in, const void *V_in, const void *W_out,
                       double *scores, int32_t *order, double *cett, int act)
{
    double *z = (double *)malloc((size_t)T * d_ff * sizeof(double));      /* z[t, j] */
    double *cut = (double *)calloc((size_t)T * d_model, sizeof(double));  /* running sum of cut outputs */
    or_pair *pr = (or_pair *)malloc((size_t)d_ff * sizeof(or_pair));
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d_ff; ++j) {
        double wnorm2 = 0.0, zz = 0.0;
        for (int i = 0; i < d_model; ++i) {
            double w = elem(W_out, dtype, (size_t)i * d_ff + j);
            wnorm2 += w * w;
        }
        for (int t = 0; t < T; ++t) {
            double g = 0.0, u = 0.0;
            for (int k = 0; k < d_model; ++k) {
                double x = elem(X, dtype, (size_t)t * d_model + k);
                g += elem(W_in, dtype, (size_t)j * d_model + k) * x;
                if (is_gated(act))
                    u += elem(V_in, dtype, (size_t)j * d_model + k) * x;
            }
            double zt = neuron_value(act, g, u);
            z[(size_t)t * d_ff + j] = zt;
            zz += zt * zt;
        }
        scores[j] = sqrt(zz) * sqrt(wnorm2);
        pr[j].a = scores[j];
        pr[j].j = j;
    }
    qsort(pr, (size_t)d_ff, sizeof(or_pair), cmp_pair);
    cett[0] = 0.0;
    for (int k = 0; k < d_ff; ++k) {
        const int j = pr[k].j;
        order[k] = j;
        double norm2 = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : norm2)
        for (int t = 0; t < T; ++t) {
            const double zt = z[(size_t)t * d_ff + j];
            for (int i = 0; i < d_model; ++i) {
                double *c = &cut[(size_t)t * d_model + i];
                *c += zt * elem(W_out, dtype, (size_t)i * d_ff + j);
                norm2 += (*c) * (*c);
            }
        }
        cett[k + 1] = sqrt(norm2);  /* numerator; divided by the dense norm below */
    }
    const double dense = cett[d_ff];  /* all neurons cut = the dense output */
    for (int k = 1; k <= d_ff; ++k)
        cett[k] = dense > 0.0 ? cett[k] / dense : 0.0;
    free(z);
    free(cut);
    free(pr);
}

/* The search itself, given every sample's scores [B, d_ff] and curve [B, d_ff+1]:
 * CETT(x; eps) is constant between consecutive scores of x, so the candidates
 * are the scores of all samples; the answer is the largest candidate whose mean
 * CETT over the samples is within the bound.  The smallest score of all always
 * qualifies (nothing is cut).  mean_out receives the mean CETT at the answer. */
double oracle_threshold_search(const double *scores, const double *cett, int B, int d_ff,
                               double bound, double *mean_out)
{
    double *sorted = (double *)malloc((size_t)B * d_ff * sizeof(double));
    for (int b = 0; b < B; ++b) {
        or_pair *pr = (or_pair *)malloc((size_t)d_ff * sizeof(or_pair));
        for (int j = 0; j < d_ff; ++j) { pr[j].a = scores[(size_t)b * d_ff + j]; pr[j].j = j; }
        qsort(pr, (size_t)d_ff, sizeof(or_pair), cmp_pair);
        for (int j = 0; j < d_ff; ++j) sorted[(size_t)b * d_ff + j] = pr[j].a;
        free(pr);
    }
    double best = -1.0, best_mean = 0.0;
    for (size_t c = 0; c < (size_t)B * d_ff; ++c) {
        const double eps = scores[c];
        double mean = 0.0;
        for (int b = 0; b < B; ++b) {
            int k = 0;  /* neurons of sample b with score < eps */
            while (k < d_ff && sorted[(size_t)b * d_ff + k] < eps) ++k;
            mean += cett[(size_t)b * (d_ff + 1) + k];
        }
        mean /= B;
        if (mean <= bound && eps > best) { best = eps; best_mean = mean; }
    }
    if (mean_out) *mean_out = best_mean;
    free(sorted);
    return best;
}
