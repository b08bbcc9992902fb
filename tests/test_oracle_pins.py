"""Pins for the CPU oracle: closed forms, invariants, brute force and library routines.

Each test fixes the oracle to something other than itself, so that a dropped term, a wrong sign
or index, or a transposed operand in oracle/clada_oracle.c fails here.  No GPU involved.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_bits(a: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _layer(rng, d, F, T, dtype="f32"):
    Wg = (rng.standard_normal((F, d)) * 0.3).astype(np.float32)
    Wu = (rng.standard_normal((F, d)) * 0.3).astype(np.float32)
    Wd = (rng.standard_normal((d, F)) * 0.3).astype(np.float32)
    X = rng.standard_normal((T, d)).astype(np.float32)
    if dtype == "bf16":
        return tuple(_bf16_bits(a) for a in (X, Wg, Wu, Wd))
    return X, Wg, Wu, Wd


def _f64(a):
    return _bf16_to_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)


# ----------------------------------------------------------------------------------------------
# Cognitive load: Eqs. surprisal / entropy
# ----------------------------------------------------------------------------------------------

def _golden_ln_vocab():
    rows = {}
    with open(os.path.join(GOLDEN, "ln_vocab.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v, val = line.split()
            rows[int(v)] = float(val)
    return rows


@pytest.mark.parametrize("V", [2, 4096, 32000, 128256])
def test_entropy_uniform_is_ln_V(oracle, V):
    golden = _golden_ln_vocab()
    logits = np.full(V, 1.75, dtype=np.float32)
    s, H = oracle.cogload(logits, V // 3)
    assert abs(H - golden[V]) < 1e-10
    assert abs(s - golden[V]) < 1e-10
    assert abs(golden[V] - math.log(V)) < 1e-12


def test_entropy_one_hot_is_zero(oracle):
    logits = np.full(1000, -np.inf, dtype=np.float32)
    logits[417] = 3.25
    s, H = oracle.cogload(logits, 417)
    assert H == 0.0 and s == 0.0
    s_other, _ = oracle.cogload(logits, 3)
    assert s_other == np.inf


@pytest.mark.parametrize("a,V", [(5.0, 4096), (-2.0, 100), (12.0, 32000)])
def test_two_level_closed_form(oracle, a, V):
    logits = np.zeros(V, dtype=np.float32)
    logits[7] = a
    p = math.exp(a) / (math.exp(a) + V - 1)
    q = (1 - p) / (V - 1)
    H_ref = -p * math.log(p) - (V - 1) * q * math.log(q)
    s_peak, H = oracle.cogload(logits, 7)
    s_rest, _ = oracle.cogload(logits, 8)
    assert abs(H - H_ref) < 1e-10
    assert abs(s_peak + math.log(p)) < 1e-10
    assert abs(s_rest + math.log(q)) < 1e-10


def test_cogload_matches_library_log_softmax(oracle):
    rng = np.random.default_rng(3)
    for V in (17, 1000, 32000):
        logits = (rng.standard_normal(V) * 3).astype(np.float32)
        tok = int(rng.integers(V))
        lp = scipy.special.log_softmax(logits.astype(np.float64))
        s, H = oracle.cogload(logits, tok)
        assert abs(s + lp[tok]) < 1e-10
        assert abs(H + np.sum(np.exp(lp) * lp)) < 1e-10
        assert 0.0 <= H <= math.log(V) + 1e-12 and s >= 0.0


def test_cogload_shift_invariance_and_bf16(oracle):
    rng = np.random.default_rng(4)
    logits = (rng.standard_normal(5000) * 2).astype(np.float32)
    s0, H0 = oracle.cogload(logits, 11)
    s1, H1 = oracle.cogload(logits + np.float32(8.0), 11)
    assert abs(s0 - s1) < 1e-5 and abs(H0 - H1) < 1e-5   # the shift itself rounds in fp32
    bits = _bf16_bits(logits)
    lp = scipy.special.log_softmax(_bf16_to_f64(bits))
    s, H = oracle.cogload(bits, 11)
    assert abs(s + lp[11]) < 1e-10 and abs(H + np.sum(np.exp(lp) * lp)) < 1e-10


def test_cogload_token_out_of_range(oracle):
    logits = np.zeros(10, dtype=np.float32)
    s, H = oracle.cogload(logits, 10)
    assert math.isnan(s) and abs(H - math.log(10)) < 1e-12
    s, _ = oracle.cogload(logits, -1)
    assert math.isnan(s)


# ----------------------------------------------------------------------------------------------
# Neuron scores: Eq. neuron_activation
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_scores_literal_frobenius_equals_factored(oracle, dtype):
    rng = np.random.default_rng(0)
    X, Wg, Wu, Wd = _layer(rng, d=12, F=9, T=7, dtype=dtype)
    A = oracle.neuron_scores(X, [0, 7], Wg, Wu, Wd)[0]
    A_lit = oracle.neuron_scores_literal(X, Wg, Wu, Wd)
    np.testing.assert_allclose(A, A_lit, rtol=1e-12)


def test_scores_against_explicit_matrix_norms(oracle):
    """numpy builds the matrix [sigma(W_in,j x) * V_in,j x] W_out,j and takes library norms of it."""
    rng = np.random.default_rng(1)
    X, Wg, Wu, Wd = _layer(rng, d=10, F=6, T=5)
    A = oracle.neuron_scores(X, [0, 5], Wg, Wu, Wd)[0]
    X64, Wg64, Wu64, Wd64 = (a.astype(np.float64) for a in (X, Wg, Wu, Wd))
    for j in range(6):
        g = X64 @ Wg64[j]
        z = g * scipy.special.expit(g) * (X64 @ Wu64[j])
        M = np.outer(z, Wd64[:, j])            # column j of W_out, T x d_model
        assert abs(A[j] - np.linalg.norm(M, "fro")) < 1e-12 * max(1.0, A[j])
        assert abs(A[j] - np.linalg.norm(M, 2)) < 1e-10 * max(1.0, A[j])   # rank one: same number


def test_scores_single_token_special_case(oracle):
    rng = np.random.default_rng(2)
    X, Wg, Wu, Wd = _layer(rng, d=16, F=8, T=1)
    A = oracle.neuron_scores(X, [0, 1], Wg, Wu, Wd)[0]
    x = X[0].astype(np.float64)
    g = Wg.astype(np.float64) @ x
    z = g * scipy.special.expit(g) * (Wu.astype(np.float64) @ x)
    ref = np.abs(z) * np.linalg.norm(Wd.astype(np.float64), axis=0)
    np.testing.assert_allclose(A, ref, rtol=1e-12)


def test_scores_invariances(oracle):
    rng = np.random.default_rng(5)
    X, Wg, Wu, Wd = _layer(rng, d=8, F=11, T=12)
    A = oracle.neuron_scores(X, [0, 12], Wg, Wu, Wd)[0]
    # token order does not matter
    perm = rng.permutation(12)
    np.testing.assert_allclose(oracle.neuron_scores(X[perm], [0, 12], Wg, Wu, Wd)[0], A, rtol=1e-12)
    # squares add across token chunks; ragged offsets index the right rows
    parts = oracle.neuron_scores(X, [0, 5, 5, 12], Wg, Wu, Wd)
    assert np.all(parts[1] == 0.0)
    np.testing.assert_allclose(np.sqrt(parts[0] ** 2 + parts[2] ** 2), A, rtol=1e-12)
    # permuting neurons permutes scores
    q = rng.permutation(11)
    Aq = oracle.neuron_scores(X, [0, 12], Wg[q], Wu[q], Wd[:, q])[0]
    np.testing.assert_allclose(Aq, A[q], rtol=1e-12)
    # gate and up are not interchangeable (silu acts on the gate only)
    A_swapped = oracle.neuron_scores(X, [0, 12], Wu, Wg, Wd)[0]
    assert np.max(np.abs(A_swapped - A) / A) > 1e-3


def test_scores_tie_to_per_token_neuron_outputs(oracle):
    """sum_t ||n_j(x_t)||^2 = A_j^2, n_j(x_t) obtained from the sparse FFN with only neuron j kept."""
    rng = np.random.default_rng(6)
    X, Wg, Wu, Wd = _layer(rng, d=8, F=5, T=6)
    A = oracle.neuron_scores(X, [0, 6], Wg, Wu, Wd)[0]
    for j in range(5):
        only_j = np.zeros(5)
        only_j[j] = 1.0
        tot = 0.0
        for t in range(6):
            n_j, mask, cnt = oracle.sparse_ffn(X[t], Wg, Wu, Wd, only_j, 0.5)
            assert cnt == 1 and mask[j] == 1
            tot += float(np.sum(n_j ** 2))
        assert abs(math.sqrt(tot) - A[j]) < 1e-12 * max(1.0, A[j])


# ----------------------------------------------------------------------------------------------
# Selection: S_cut = { j : A_j < eps }
# ----------------------------------------------------------------------------------------------

def test_select_brute_force_tiny(oracle):
    rng = np.random.default_rng(7)
    for F in (1, 2, 7, 16):
        A = rng.random(F) + 0.1
        order = np.sort(A)
        cuts = [0.0, order[0]] + [0.5 * (order[i] + order[i + 1]) for i in range(F - 1)] + [order[-1], np.inf]
        prev = None
        for tau in cuts:
            mask, idx, count = oracle.select(A, tau)
            keep = [j for j in range(F) if A[j] >= tau]
            assert list(idx) == keep and count == len(keep)
            assert list(np.nonzero(mask)[0]) == keep
            if prev is not None:
                assert set(keep) <= prev          # nested as tau grows
            prev = set(keep)
        assert oracle.select(A, order[0])[2] == F          # tau <= min keeps all; equality keeps
        assert oracle.select(A, np.inf)[2] == 0


def test_select_rank_count(oracle):
    rng = np.random.default_rng(8)
    A = rng.random(16)
    order = np.sort(A)
    for r in range(15):
        tau = 0.5 * (order[r] + order[r + 1])
        assert oracle.select(A, tau)[2] == 16 - (r + 1)


def test_tau_from_sparsity_cuts_k(oracle):
    rng = np.random.default_rng(9)
    A = rng.random(1376).astype(np.float32)
    for rho in (0.0, 0.3, 0.4, 0.5, 0.6, 1.0):
        tau = oracle.tau_from_sparsity(A, rho)
        k_cut = int(math.floor(rho * 1376 + 0.5))
        assert oracle.select(A.astype(np.float64), float(tau))[2] == 1376 - k_cut


# ----------------------------------------------------------------------------------------------
# Threshold adjustment: Eq. final_threshold
# ----------------------------------------------------------------------------------------------

def test_adjust_four_cases(oracle):
    tb = np.array([[0.37, 1.5, 2.25]] * 4, dtype=np.float32)
    lam = np.full(3, 0.80, dtype=np.float32)
    gam = np.full(3, 0.12, dtype=np.float32)
    s = np.array([1.0, 3.0, 1.0, 3.0])
    H = np.array([1.0, 1.0, 5.0, 5.0])
    out = oracle.adjust_threshold(tb, lam, gam, 2.0, 4.0, s, H)
    one = np.float32(1.0)
    mults = [one, one + np.float32(0.80), one + np.float32(0.12),
             (one + np.float32(0.80)) + np.float32(0.12)]
    for b in range(4):
        np.testing.assert_array_equal(out[b], tb[b] * mults[b])
    # against the exact rationals 1, 1.8, 1.12, 1.92 to fp32 rounding
    np.testing.assert_allclose(out[:, 0].astype(np.float64) / 0.37,
                               [1.0, 1.8, 1.12, 1.92], rtol=3e-7)


def test_adjust_strict_and_signed(oracle):
    tb = np.array([[2.0]], dtype=np.float32)
    lam = np.array([0.80], dtype=np.float32)
    gam = np.array([0.12], dtype=np.float32)
    # equality does not trigger: I(s > tau_s)
    assert oracle.adjust_threshold(tb, lam, gam, 2.0, 4.0, [2.0], [4.0])[0, 0] == np.float32(2.0)
    # coefficients are signed inputs
    out = oracle.adjust_threshold(tb, -lam, -gam, 2.0, 4.0, [2.5], [4.5])
    assert out[0, 0] == np.float32(2.0) * ((np.float32(1.0) - np.float32(0.80)) - np.float32(0.12))
    # lambda = gamma = 0: thresholds unchanged
    z = np.zeros(1, dtype=np.float32)
    assert oracle.adjust_threshold(tb, z, z, 2.0, 4.0, [9.0], [9.0])[0, 0] == np.float32(2.0)
    # per-layer coefficients index by layer, thresholds by (sequence, layer)
    tb2 = np.array([[1.0, 2.0], [3.0, 4.0]], dtype=np.float32)
    lam2 = np.array([0.5, 0.25], dtype=np.float32)
    out = oracle.adjust_threshold(tb2, lam2, np.zeros(2, np.float32), 0.0, 0.0, [1.0, -1.0], [0.0, 0.0])
    np.testing.assert_array_equal(out, np.array([[1.5, 2.5], [3.0, 4.0]], dtype=np.float32))


# ----------------------------------------------------------------------------------------------
# FFN: Algorithm 2, sparse forward pass
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_dense_ffn_matches_matrix_formulation(oracle, dtype):
    rng = np.random.default_rng(10)
    X, Wg, Wu, Wd = _layer(rng, d=24, F=40, T=3, dtype=dtype)
    tX, tWg, tWu, tWd = (torch.from_numpy(_f64(a)) for a in (X, Wg, Wu, Wd))
    ref = (torch.nn.functional.silu(tX @ tWg.T) * (tX @ tWu.T)) @ tWd.T
    for t in range(3):
        y = oracle.dense_ffn(X[t], Wg, Wu, Wd)
        np.testing.assert_allclose(y, ref[t].numpy(), rtol=1e-11, atol=1e-13)


def test_zero_sparsity_is_dense_bit_for_bit(oracle):
    rng = np.random.default_rng(11)
    X, Wg, Wu, Wd = _layer(rng, d=16, F=30, T=4)
    A = oracle.neuron_scores(X, [0, 4], Wg, Wu, Wd)[0]
    for t in range(4):
        y_s, mask, cnt = oracle.sparse_ffn(X[t], Wg, Wu, Wd, A, A.min())
        assert cnt == 30 and mask.all()
        assert np.array_equal(y_s, oracle.dense_ffn(X[t], Wg, Wu, Wd))
    y_none, mask, cnt = oracle.sparse_ffn(X[0], Wg, Wu, Wd, A, np.inf)
    assert cnt == 0 and not mask.any() and np.all(y_none == 0.0)


def test_sparse_ffn_is_masked_matrix_product(oracle):
    rng = np.random.default_rng(12)
    X, Wg, Wu, Wd = _layer(rng, d=16, F=30, T=8)
    A = oracle.neuron_scores(X, [0, 8], Wg, Wu, Wd)[0]
    tau = float(np.median(A))
    keep = torch.from_numpy(A >= tau)
    tX, tWg, tWu, tWd = (torch.from_numpy(a.astype(np.float64)) for a in (X, Wg, Wu, Wd))
    h = torch.nn.functional.silu(tX @ tWg.T) * (tX @ tWu.T)
    ref = (h * keep) @ tWd.T
    for t in range(8):
        y, mask, cnt = oracle.sparse_ffn(X[t], Wg, Wu, Wd, A, tau)
        assert cnt == int(keep.sum()) and np.array_equal(mask.astype(bool), keep.numpy())
        np.testing.assert_allclose(y, ref[t].numpy(), rtol=1e-11, atol=1e-13)


def test_cett_identity_and_prefix_bound(oracle):
    """dense - sparse = sum of the cut neurons' outputs, so CETT = ||dense - sparse|| / ||dense||;
    over the prefix, ||Y_dense - Y_sparse||_F <= sum_{cut} A_j (triangle inequality)."""
    rng = np.random.default_rng(13)
    T, F = 6, 20
    X, Wg, Wu, Wd = _layer(rng, d=12, F=F, T=T)
    A = oracle.neuron_scores(X, [0, T], Wg, Wu, Wd)[0]
    tau = float(np.sort(A)[8] * 0.5 + np.sort(A)[9] * 0.5)
    cut = np.nonzero(A < tau)[0]
    assert len(cut) == 9
    diff_fro2 = 0.0
    for t in range(T):
        y_d = oracle.dense_ffn(X[t], Wg, Wu, Wd)
        y_s, _, _ = oracle.sparse_ffn(X[t], Wg, Wu, Wd, A, tau)
        n_cut = np.zeros(12)
        for j in cut:
            e = np.zeros(F)
            e[j] = 1.0
            n_cut += oracle.sparse_ffn(X[t], Wg, Wu, Wd, e, 0.5)[0]
        np.testing.assert_allclose(y_d - y_s, n_cut, rtol=1e-9, atol=1e-12)
        cett = np.linalg.norm(n_cut) / np.linalg.norm(y_d)
        assert abs(cett - np.linalg.norm(y_d - y_s) / np.linalg.norm(y_d)) < 1e-9
        diff_fro2 += float(np.sum((y_d - y_s) ** 2))
    assert math.sqrt(diff_fro2) <= float(np.sum(A[cut])) * (1 + 1e-12)


# ----------------------------------------------------------------------------------------------
# Offline threshold search: Eq. base_threshold
# ----------------------------------------------------------------------------------------------

def _cett_by_definition(oracle, X, Wg, Wu, Wd, A, eps):
    """||sum_{A_j < eps} n_j(x)||_F / ||MLP(x)||_F through the (separately pinned) per-token FFN routines."""
    num = den = 0.0
    for t in range(X.shape[0]):
        y_d = oracle.dense_ffn(X[t], Wg, Wu, Wd)
        y_s, _, _ = oracle.sparse_ffn(X[t], Wg, Wu, Wd, A, eps)     # keeps A_j >= eps
        num += float(np.sum((y_d - y_s) ** 2))
        den += float(np.sum(y_d ** 2))
    return math.sqrt(num / den)


def test_cett_curve_matches_definition(oracle):
    rng = np.random.default_rng(20)
    T, F = 5, 9
    X, Wg, Wu, Wd = _layer(rng, d=8, F=F, T=T)
    A, order, cett = oracle.cett_curve(X, Wg, Wu, Wd)
    np.testing.assert_allclose(A, oracle.neuron_scores(X, [0, T], Wg, Wu, Wd)[0], rtol=1e-12)
    assert list(order) == list(np.argsort(A, kind="stable"))
    assert cett[0] == 0.0 and abs(cett[F] - 1.0) < 1e-12
    a = np.sort(A)
    for k in range(F + 1):
        eps = a[0] * 0.5 if k == 0 else (np.inf if k == F else 0.5 * (a[k - 1] + a[k]))
        assert abs(cett[k] - _cett_by_definition(oracle, X, Wg, Wu, Wd, A, eps)) < 1e-10
    # at eps equal to a score that neuron is still kept (S_cut uses strict <)
    assert abs(cett[3] - _cett_by_definition(oracle, X, Wg, Wu, Wd, A, a[3])) < 1e-10


def test_cett_curve_orthogonal_outputs_closed_form(oracle):
    """W_out diagonal: the neurons' outputs are orthogonal, so ||sum_cut n_j||^2 = sum_cut A_j^2."""
    rng = np.random.default_rng(21)
    d = F = 7
    X, Wg, Wu, _ = _layer(rng, d=d, F=F, T=6)
    Wd = np.diag(rng.random(F) + 0.5).astype(np.float32)
    A, order, cett = oracle.cett_curve(X, Wg, Wu, Wd)
    a2 = np.sort(A) ** 2
    ref = np.sqrt(np.concatenate([[0.0], np.cumsum(a2)]) / np.sum(a2))
    np.testing.assert_allclose(cett, ref, rtol=1e-10, atol=1e-12)


def test_threshold_search_brute_force(oracle):
    rng = np.random.default_rng(22)
    B, F, d = 3, 6, 8
    Wg = (rng.standard_normal((F, d)) * 0.3).astype(np.float32)
    Wu = (rng.standard_normal((F, d)) * 0.3).astype(np.float32)
    Wd = (rng.standard_normal((d, F)) * 0.3).astype(np.float32)
    Xs = [rng.standard_normal((T, d)).astype(np.float32) for T in (4, 7, 5)]
    curves = [oracle.cett_curve(X, Wg, Wu, Wd) for X in Xs]
    scores = np.stack([c[0] for c in curves])
    cett = np.stack([c[2] for c in curves])
    for bound in (0.0, 0.05, 0.2, 0.5, 1.0):
        tau, mean = oracle.threshold_search(scores, cett, bound)
        best, best_mean = None, None
        for eps in np.sort(scores.ravel()):
            m = np.mean([_cett_by_definition(oracle, Xs[b], Wg, Wu, Wd, scores[b], eps) for b in range(B)])
            if m <= bound + 1e-12:
                best, best_mean = eps, m
        assert tau == best and abs(mean - best_mean) < 1e-10
    assert oracle.threshold_search(scores, cett, 0.0)[0] == scores.min()      # nothing may be cut
    assert oracle.threshold_search(scores, cett, 1.0)[0] == scores.max()      # everything but the top neuron
    # a looser bound never lowers the threshold
    taus = [oracle.threshold_search(scores, cett, b)[0] for b in (0.01, 0.1, 0.2, 0.4, 0.8)]
    assert all(x <= y for x, y in zip(taus, taus[1:]))


# ----------------------------------------------------------------------------------------------
# FFN forms of the other model families (Section 4.1): GELU-gated and non-gated ReLU
# ----------------------------------------------------------------------------------------------

def _torch_h(act, tX, tWg, tWu):
    """Library formulation of the per-neuron value for every token: [T, d_ff] float64."""
    g = tX @ tWg.T
    if act == 1:
        return torch.nn.functional.gelu(g, approximate="tanh") * (tX @ tWu.T)
    if act == 2:
        return torch.relu(g)
    return torch.nn.functional.silu(g) * (tX @ tWu.T)


@pytest.mark.parametrize("act", [1, 2])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_variant_dense_and_masked_ffn_match_library(oracle, act, dtype):
    rng = np.random.default_rng(30 + act)
    T, F = 5, 40
    X, Wg, Wu, Wd = _layer(rng, d=24, F=F, T=T, dtype=dtype)
    V = None if act == 2 else Wu
    tX, tWg, tWu, tWd = (torch.from_numpy(_f64(a)) for a in (X, Wg, Wu, Wd))
    h = _torch_h(act, tX, tWg, tWu)
    A = oracle.neuron_scores(X, [0, T], Wg, V, Wd, act=act)[0]
    # scores against explicit norms of the library's h and of W_out's columns
    ref_A = torch.linalg.norm(h, dim=0) * torch.linalg.norm(tWd, dim=0)
    np.testing.assert_allclose(A, ref_A.numpy(), rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(oracle.neuron_scores_literal(X, Wg, V, Wd, act=act), A, rtol=1e-11, atol=1e-14)
    tau = float(np.median(A))
    keep = torch.from_numpy(A >= tau)
    for t in range(T):
        np.testing.assert_allclose(oracle.dense_ffn(X[t], Wg, V, Wd, act=act), (h[t] @ tWd.T).numpy(),
                                   rtol=1e-11, atol=1e-13)
        y, mask, cnt = oracle.sparse_ffn(X[t], Wg, V, Wd, A, tau, act=act)
        assert cnt == int(keep.sum()) and np.array_equal(mask.astype(bool), keep.numpy())
        np.testing.assert_allclose(y, ((h[t] * keep) @ tWd.T).numpy(), rtol=1e-11, atol=1e-13)
        y0, _, c0 = oracle.sparse_ffn(X[t], Wg, V, Wd, A, 0.0, act=act)
        assert c0 == F and np.array_equal(y0, oracle.dense_ffn(X[t], Wg, V, Wd, act=act))


def test_relu_form_worked_example(oracle):
    """Two neurons reading +x0 and -x0: only the one whose pre-activation is positive contributes,
    and it contributes its pre-activation times its W_out column; V_in plays no part."""
    W_in = np.array([[1.0, 0.0], [-1.0, 0.0]], np.float32)
    W_out = np.array([[2.0, 5.0], [3.0, 7.0]], np.float32)       # columns are the neurons' outputs
    x = np.array([2.0, 3.0], np.float32)
    assert np.array_equal(oracle.dense_ffn(x, W_in, None, W_out, act=2), [4.0, 6.0])
    assert np.array_equal(oracle.dense_ffn(-x, W_in, None, W_out, act=2), [10.0, 14.0])
    X = np.stack([x, -x, 2 * x])
    A = oracle.neuron_scores(X, [0, 3], W_in, None, W_out, act=2)[0]
    np.testing.assert_allclose(A, [math.sqrt(4 + 16) * math.sqrt(13), 2.0 * math.sqrt(74)], rtol=1e-14)


def test_gelu_form_scalar_values(oracle):
    """One neuron, one input: y = gelu(g) * u.  Checked against the tanh formula typed out for a few
    points, and against the erf form of GELU, which the tanh form approximates to within 5e-4."""
    for g in (-3.0, -1.0, -0.25, 0.0, 0.5, 1.0, 2.5):
        W_in = np.array([[g]], np.float32)
        V_in = np.array([[1.5]], np.float32)
        W_out = np.array([[1.0]], np.float32)
        y = oracle.dense_ffn(np.array([1.0], np.float32), W_in, V_in, W_out, act=1)[0]
        tanh_form = 0.5 * g * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (g + 0.044715 * g ** 3))) * 1.5
        erf_form = 0.5 * g * (1.0 + math.erf(g / math.sqrt(2.0))) * 1.5
        assert abs(y - tanh_form) < 1e-15 and abs(y - erf_form) < 7.5e-4


@pytest.mark.parametrize("act", [1, 2])
def test_variant_cett_curve_matches_definition(oracle, act):
    rng = np.random.default_rng(40 + act)
    T, F = 5, 9
    X, Wg, Wu, Wd = _layer(rng, d=8, F=F, T=T)
    V = None if act == 2 else Wu
    A, order, cett = oracle.cett_curve(X, Wg, V, Wd, act=act)
    np.testing.assert_allclose(A, oracle.neuron_scores(X, [0, T], Wg, V, Wd, act=act)[0], rtol=1e-12)
    a = np.sort(A)
    for k in range(F + 1):
        eps = a[0] * 0.5 if k == 0 else (np.inf if k == F else 0.5 * (a[k - 1] + a[k]))
        num = den = 0.0
        for t in range(T):
            y_d = oracle.dense_ffn(X[t], Wg, V, Wd, act=act)
            y_s, _, _ = oracle.sparse_ffn(X[t], Wg, V, Wd, A, eps, act=act)
            num += float(np.sum((y_d - y_s) ** 2))
            den += float(np.sum(y_d ** 2))
        assert abs(cett[k] - math.sqrt(num / den)) < 1e-10


# ----------------------------------------------------------------------------------------------
# fp16 elements (the precision of the paper's latency runs)
# ----------------------------------------------------------------------------------------------

def test_fp16_and_bf16_widening_every_bit_pattern(oracle):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    halves = bits.view(np.float16)
    got = oracle.widen(halves)
    ref = halves.astype(np.float64)                       # numpy's own conversion
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok], ref[ok]) and np.array_equal(np.signbit(got[ok]), np.signbit(ref[ok]))
    got_b = oracle.widen(bits)                            # the same patterns read as bfloat16
    ref_b = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    okb = ~np.isnan(ref_b)
    assert np.array_equal(np.isnan(got_b), np.isnan(ref_b)) and np.array_equal(got_b[okb], ref_b[okb])
    # a few values typed out
    assert oracle.widen(np.array([0x3C00, 0xC000, 0x0001, 0x7BFF, 0x3555], np.uint16).view(np.float16)).tolist() == \
        [1.0, -2.0, 2.0 ** -24, 65504.0, 0.333251953125]


@pytest.mark.parametrize("act", [0, 1, 2])
def test_fp16_layer_matches_library_formulation(oracle, act):
    rng = np.random.default_rng(50 + act)
    T, F = 4, 36
    X, Wg, Wu, Wd = (a.astype(np.float16) for a in _layer(rng, d=16, F=F, T=T))
    V = None if act == 2 else Wu
    tX, tWg, tWu, tWd = (torch.from_numpy(a.astype(np.float64)) for a in (X, Wg, Wu, Wd))
    h = _torch_h(act, tX, tWg, tWu)
    A = oracle.neuron_scores(X, [0, T], Wg, V, Wd, act=act)[0]
    ref_A = torch.linalg.norm(h, dim=0) * torch.linalg.norm(tWd, dim=0)
    np.testing.assert_allclose(A, ref_A.numpy(), rtol=1e-11, atol=1e-14)
    for t in range(T):
        np.testing.assert_allclose(oracle.dense_ffn(X[t], Wg, V, Wd, act=act), (h[t] @ tWd.T).numpy(),
                                   rtol=1e-11, atol=1e-13)
    lg = (rng.standard_normal(300) * 3).astype(np.float16)
    s, H = oracle.cogload(lg, 7)
    lp = torch.log_softmax(torch.from_numpy(lg.astype(np.float64)), dim=0)
    assert abs(s + lp[7].item()) < 1e-12 and abs(H + float((lp.exp() * lp).sum())) < 1e-12


# ----------------------------------------------------------------------------------------------
# Nested index lists (the compressed form of the four masks)
# ----------------------------------------------------------------------------------------------

def test_nested_lists_equal_the_masks(oracle):
    rng = np.random.default_rng(60)
    for F in (1, 7, 64, 333):
        A = rng.random(F) + 0.5
        if F >= 7:
            A[3] = A[5] = A[1]                       # equal scores
        srt = np.sort(A)
        taus = np.array([0.0, srt[F // 2], A[min(1, F - 1)], 0.5 * (srt[0] + srt[-1]), srt[-1], np.inf, srt[-1] * (1 + 1e-12)])
        order, counts = oracle.nested_lists(A, taus)
        assert sorted(order.tolist()) == list(range(F))                      # a permutation
        a = A[order]
        assert np.all(a[:-1] >= a[1:])                                       # descending
        assert all(order[i] < order[i + 1] for i in range(F - 1) if a[i] == a[i + 1])   # ties by index
        for k, tau in enumerate(taus):
            mask, idx, cnt = oracle.select(A, tau)                           # the mask definition (pinned above)
            assert counts[k] == cnt
            assert sorted(order[:cnt].tolist()) == idx.tolist()
        # nesting: a higher threshold keeps a leading part of a lower one's list
        by_tau = np.argsort(taus)
        assert all(counts[by_tau[i]] >= counts[by_tau[i + 1]] for i in range(len(taus) - 1))


def test_load_level_indexes_the_four_thresholds(oracle):
    lam, gam = np.float32(0.80), np.float32(0.12)
    one = np.float32(1.0)
    mults = [one, one + lam, one + gam, (one + lam) + gam]                   # fp32, left to right
    tau_base = np.array([[0.731]], np.float32)
    tau_s, tau_H = 2.0, 3.0
    for s, H, level in [(1.0, 1.0, 0), (2.5, 1.0, 1), (1.0, 3.5, 2), (2.5, 3.5, 3),
                        (2.0, 3.0, 0), (float("nan"), 4.0, 2)]:             # strict >, NaN compares false
        assert oracle.load_level(s, H, tau_s, tau_H) == level
        tf = oracle.adjust_threshold(tau_base, [lam], [gam], tau_s, tau_H, [s], [H])
        assert tf[0, 0] == np.float32(tau_base[0, 0] * mults[level])
    # negative coefficients (the prose reading) index the same way
    tf = oracle.adjust_threshold(tau_base, [-0.3], [-0.1], tau_s, tau_H, [2.5], [3.5])
    assert oracle.load_level(2.5, 3.5, tau_s, tau_H) == 3
    assert tf[0, 0] == np.float32(tau_base[0, 0] * ((one + np.float32(-0.3)) + np.float32(-0.1)))


def test_nested_ffn_equals_thresholded_ffn(oracle):
    rng = np.random.default_rng(61)
    T, F = 6, 50
    X, Wg, Wu, Wd = _layer(rng, d=16, F=F, T=T)
    A = oracle.neuron_scores(X, [0, T], Wg, Wu, Wd)[0]
    tau_base = float(np.sort(A)[20])
    taus = np.array([np.float32(tau_base) * m for m in (1.0, 1.8, 1.12, 1.92)], dtype=np.float64)
    order, counts = oracle.nested_lists(A, taus)
    for k in range(4):
        y_tau, mask, cnt = oracle.sparse_ffn(X[0], Wg, Wu, Wd, A, taus[k])
        marks = np.zeros(F)
        marks[order[:counts[k]]] = 1.0                                       # keep exactly the listed neurons
        y_list, mask2, cnt2 = oracle.sparse_ffn(X[0], Wg, Wu, Wd, marks, 0.5)
        assert cnt == cnt2 == counts[k] and np.array_equal(mask, mask2) and np.array_equal(y_tau, y_list)


# ----------------------------------------------------------------------------------------------
# Dense prefill FFN (the pass the statistics are a by-product of)
# ----------------------------------------------------------------------------------------------

def test_round_storage_matches_library_casts(oracle):
    rng = np.random.default_rng(70)
    vals = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-9, 6, 2000),
                           [0.0, -0.0, 1.0, 65504.0, 65519.9, 65520.0, 7e4, 6.0e-8, 2.98e-8, 2.9e-8, 1e-45,
                            1.00390625, 1.001953125, 1.005859375, 3.4e38, 3.39e38, -2.5]])
    f32 = vals.astype(np.float32)
    ref16 = f32.astype(np.float16).astype(np.float64)                         # numpy: nearest even
    ref_b = torch.from_numpy(f32).to(torch.bfloat16).to(torch.float64).numpy()   # torch: nearest even
    with np.errstate(over="ignore"):
        for v, r16, rb in zip(vals, ref16, ref_b):
            assert oracle.round_storage(2, v) == r16, v
            assert oracle.round_storage(1, v) == rb, v
            assert oracle.round_storage(0, v) == float(np.float32(v))
    # ties go to even: 1 + 2^-8 is halfway between two bf16 values, 1 + 2^-11 between two fp16 values
    assert oracle.round_storage(1, 1.00390625) == 1.0 and oracle.round_storage(1, 1.01171875) == 1.015625
    assert oracle.round_storage(2, 1.00048828125) == 1.0 and oracle.round_storage(2, 1.00146484375) == 1.001953125


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("act", [0, 1, 2])
def test_prefill_ffn_matches_library_formulation(oracle, dtype, act):
    rng = np.random.default_rng(71 + act)
    T, F, d = 7, 33, 24
    X, Wg, Wu, Wd = _layer(rng, d=d, F=F, T=T, dtype="bf16" if dtype == "bf16" else "f32")
    if dtype == "f16":
        X, Wg, Wu, Wd = (a.astype(np.float16) for a in (X, Wg, Wu, Wd))
    V = None if act == 2 else Wu
    tX, tWg, tWu, tWd = (torch.from_numpy(_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)) for a in (X, Wg, Wu, Wd))
    h = _torch_h(act, tX, tWg, tWu)                                       # [T, F] float64
    # without rounding: row t is the (separately pinned) per-token dense FFN
    Z0 = oracle.prefill_hidden(X, Wg, V, act=act, round_z=False)
    np.testing.assert_allclose(Z0, h.numpy(), rtol=1e-11, atol=1e-14)
    Y0 = oracle.down_proj(Z0, Wd)
    for t in range(T):
        np.testing.assert_allclose(Y0[t], oracle.dense_ffn(X[t], Wg, V, Wd, act=act), rtol=1e-11, atol=1e-13)
    # with rounding: the library's own casts, float64 -> float32 -> storage type
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[dtype]
    h_r = h.to(torch.float32).to(tdt).to(torch.float64)
    Z = oracle.prefill_hidden(X, Wg, V, act=act, round_z=True)
    # the library's h differs from the oracle's in the last bits of float64, which can move a value across a
    # rounding boundary only where it sits on one: allow one such element
    assert np.sum(Z != h_r.numpy()) <= 1
    np.testing.assert_allclose(oracle.down_proj(h_r.numpy(), Wd), (h_r @ tWd.T).numpy(), rtol=1e-11, atol=1e-13)


def test_down_proj_worked_example(oracle):
    """Y[t, i] = sum_j Z[t, j] W_out[i, j]: a transposed or mis-indexed operand changes these numbers."""
    Z = np.array([[1.0, 2.0, 3.0], [0.0, -1.0, 0.5]])
    W_out = np.array([[1.0, 0.0, 2.0], [0.0, 1.0, -1.0]], np.float32)        # [d_model = 2, d_ff = 3]
    np.testing.assert_array_equal(oracle.down_proj(Z, W_out), [[7.0, -1.0], [1.0, -1.5]])
