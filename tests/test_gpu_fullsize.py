"""GPU parity at the full sizes of the five workloads, one layer at a time.

The oracle cannot redo a whole stack in fp64, so at full size it checks
  * prefix statistics on sampled neurons (their three weight vectors are cut out and handed to the oracle,
    which then scores exactly those neurons over the whole prompt);
  * the sparse FFN output on whole tokens, with scores drawn by the shared generator (both sides then take
    the same keep decisions by construction), for sampled sequences of a batch;
  * cognitive load and threshold adjustment on every row of a step;
and the complete chain at full width (prefix statistics of whole prompts -> calibrated threshold -> guard band ->
masks at the four threshold levels -> FFN outputs, the oracle scoring ALL neurons): on the Llama-2-7B-shaped layer
that the benchmark times (512 tokens), on a layer of the 32-layer stack (2048 tokens), on two sequences of the
batch of 8 (14336 neurons, 1024 tokens, tiles of 4 sequences) and on the shortest and the longest prompt of the
ragged batch of 16 (5120 x 13824, up to 4096 tokens, tiles of 2) -- each with the paper's coefficients and with a
small pair under which every level keeps thousands of neurons.
Inputs are drawn on the GPU by the shared generator and copied bit for bit to the oracle's side.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import compare_masks, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5
COG_TOL = 1e-4
SCORE_TOL = 2e-5   # bf16 layers: tensor-core accumulators truncate, scores come out ~1e-5 low at K = 4096-5120


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _layer_on_gpu(clada, w, layer_idx):
    weights = wl.layer_weights(w, layer_idx, "cuda")
    wdt = weights["w_down"].t().contiguous()
    layer = clada.Layer(weights["w_gate"], weights["w_up"], wdt)
    norms = torch.empty(w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_down_norms(layer, norms)
    layer.set_down_norm(norms)
    return layer, weights


def _oracle_rows(weights, rows):
    """(W_in, V_in, W_out) restricted to the sampled neurons, in the paper's layout."""
    r = torch.as_tensor(rows, device=weights["w_gate"].device)
    return (wl.to_numpy_bits(weights["w_gate"][r]), wl.to_numpy_bits(weights["w_up"][r]),
            wl.to_numpy_bits(weights["w_down"][:, r].contiguous()))


def _prefix_sampled(clada, oracle, w, layer_idx, seqs, n_sample=48):
    """GPU scores of a whole batch of prompts vs oracle scores of sampled neurons on the given sequences."""
    lengths = wl.prefix_lengths(w)
    off = wl.seq_offsets(lengths)
    layer, weights = _layer_on_gpu(clada, w, layer_idx)
    scale = wl.channel_scale(w, "cuda")
    X = torch.cat([wl.hidden_states(w, layer_idx, "prefix", b, n, "cuda", scale) for b, n in enumerate(lengths)])
    ws = clada.new_workspace(layer, len(lengths), off[-1])
    scores = torch.empty(len(lengths), w.d_ff, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_scores(layer, X, off, scores, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rng = np.random.default_rng(layer_idx)
    rows = np.sort(rng.choice(w.d_ff, size=n_sample, replace=False))
    rows[0], rows[-1] = 0, w.d_ff - 1                      # first and last neuron (tile edges)
    W_in, V_in, W_out = _oracle_rows(weights, rows)
    for b in seqs:
        Xb = wl.to_numpy_bits(X[off[b]:off[b + 1]])
        A_or = oracle.neuron_scores(Xb, [0, lengths[b]], W_in, V_in, W_out)[0]
        A = scores[b].cpu().numpy().astype(np.float64)[rows]
        assert np.max(np.abs(A - A_or) / A_or) <= SCORE_TOL, (w.name, layer_idx, b)
    return lengths


def _ffn_synthetic_scores(clada, oracle, w, layer_idx, seqs, n_steps=2, rho=0.4):
    """FFN output parity on whole tokens with generator-drawn scores (identical keep decisions)."""
    layer, weights = _layer_on_gpu(clada, w, layer_idx)
    W_in, V_in, W_out = (wl.to_numpy_bits(weights[k]) for k in ("w_gate", "w_up", "w_down"))
    B = w.batch
    g = torch.Generator(device="cuda").manual_seed(1000 + layer_idx)
    scores = torch.rand(B, w.d_ff, generator=g, device="cuda") + 0.5
    tau = torch.empty(B, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, rho, tau)
    scale = wl.channel_scale(w, "cuda")
    xs = torch.stack([wl.hidden_states(w, layer_idx, "decode", b, n_steps, "cuda", scale) for b in range(B)], dim=1)
    ws = clada.new_workspace(layer, B, 0)
    y = torch.empty(B, w.d_model, dtype=torch.float32, device="cuda")
    mask = torch.empty(B, w.d_ff, dtype=torch.uint8, device="cuda")
    count = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc = scores.cpu().numpy().astype(np.float64)
    tb = tau.cpu().numpy()
    for t in range(n_steps):
        clada.clada_sparse_ffn_decode(layer, xs[t].contiguous(), scores, tau, 1, y, ws, mask, None, count, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert all(int(count[b]) == w.d_ff - w.k_cut(rho) for b in range(B))
        for b in seqs:
            y_or, m_or, _ = oracle.sparse_ffn(wl.to_numpy_bits(xs[t, b]), W_in, V_in, W_out, sc[b], float(tb[b]))
            np.testing.assert_array_equal(mask[b].cpu().numpy(), m_or)
            assert rel_inf(y[b].cpu().numpy(), y_or) <= FFN_TOL_F32, (w.name, layer_idx, t, b)


def _cogload_all_rows(clada, oracle, w, n_steps=2):
    lam = torch.full((w.n_layers,), 0.80, device="cuda")
    gam = torch.full((w.n_layers,), 0.12, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(7)
    tau_base = torch.rand(w.batch, w.n_layers, generator=g, device="cuda") + 0.5
    for t in range(n_steps):
        logits = torch.stack([wl.decode_logits(w, b, t + 1, "cuda")[t] for b in range(w.batch)])
        tokens = torch.stack([wl.chosen_tokens(w, logits[b:b + 1], b)[0] for b in range(w.batch)]).contiguous()
        s = torch.empty(w.batch, device="cuda")
        h = torch.empty(w.batch, device="cuda")
        tf = torch.empty(w.batch, w.n_layers, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        so = [oracle.cogload(logits[b].cpu().numpy(), int(tokens[b])) for b in range(w.batch)]
        tau_s = wl.universal_threshold([a for a, _ in so])
        tau_H = wl.universal_threshold([b_ for _, b_ in so])
        clada.clada_cogload_adjust(logits, tokens, tau_base, lam, gam, tau_s, tau_H, s, h, tf, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for b in range(w.batch):
            assert abs(s[b].item() - so[b][0]) <= COG_TOL and abs(h[b].item() - so[b][1]) <= COG_TOL
        ref = oracle.adjust_threshold(tau_base.cpu().numpy(), lam.cpu().numpy(), gam.cpu().numpy(), tau_s, tau_H,
                                      [a for a, _ in so], [b_ for _, b_ in so])
        np.testing.assert_array_equal(tf.cpu().numpy(), ref)


def test_c2_full_chain(clada, oracle):
    """The benchmark's layer end to end: oracle scores of all 11008 neurons over the 512-token prompt."""
    w = wl.WORKLOADS["c2_llama2_7b_layer"]
    T = w.prefix_len[0]
    layer, weights = _layer_on_gpu(clada, w, 0)
    W_in, V_in, W_out = (wl.to_numpy_bits(weights[k]) for k in ("w_gate", "w_up", "w_down"))
    scale = wl.channel_scale(w, "cuda")
    X = wl.hidden_states(w, 0, "prefix", 0, T, "cuda", scale)
    xs = wl.hidden_states(w, 0, "decode", 0, 4, "cuda", scale)
    A_or = oracle.neuron_scores(wl.to_numpy_bits(X), [0, T], W_in, V_in, W_out)[0]
    ws = clada.new_workspace(layer, 1, T)
    scores = torch.empty(1, w.d_ff, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_scores(layer, X, [0, T], scores, ws, status)
    A = scores[0].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(A - A_or) / A_or) <= SCORE_TOL
    mults = [1.0, 1.8, 1.12, 1.92]
    for rho in w.sparsities:
        tau_base = torch.empty(1, dtype=torch.float32, device="cuda")
        clada.clada_tau_from_sparsity(scores, rho, tau_base)
        mask = torch.empty(1, w.d_ff, dtype=torch.uint8, device="cuda")
        idx = torch.empty(1, w.d_ff, dtype=torch.int32, device="cuda")
        count = torch.empty(1, dtype=torch.int32, device="cuda")
        clada.clada_prefix_select(layer, X, [0, T], tau_base, mults, scores, mask, idx, count, ws, status)
        tb = np.float32(tau_base.item())
        # tau_base was placed on the unrefined scores; the guard band then corrects the few scores next to it
        # (the tensor-core sums run ~8e-6 low), which can move a neuron across: the count is the oracle's under
        # the same threshold, within a neuron or two of the calibration target.
        excused, mismatched = compare_masks(mask[0].cpu().numpy(), A_or, float(tb))
        assert mismatched == 0
        assert abs(int(count[0]) - (w.d_ff - w.k_cut(rho))) <= 2
        if excused == 0:
            assert int(count[0]) == int(np.sum(A_or >= float(tb)))
        y = torch.empty(1, w.d_model, dtype=torch.float32, device="cuda")
        for t, m in enumerate(mults[:3]):
            tau_t = torch.tensor([tb * np.float32(m)], dtype=torch.float32, device="cuda")
            clada.clada_sparse_ffn_decode(layer, xs[t:t + 1], scores, tau_t, 1, y, ws, mask, None, count, status)
            torch.cuda.synchronize()
            tau_f = float(tau_t.item())
            excused, mismatched = compare_masks(mask[0].cpu().numpy(), A_or, tau_f)
            assert mismatched == 0
            if excused == 0:
                y_or, _, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs[t]), W_in, V_in, W_out, A_or, tau_f)
                assert int(count[0]) == n_or
                if n_or:
                    assert rel_inf(y[0].cpu().numpy(), y_or) <= FFN_TOL_F32
    assert int(status.item()) == 0


@pytest.mark.parametrize("layer_idx", [0, 31])
def test_c3_stack_layers(clada, oracle, layer_idx):
    w = wl.WORKLOADS["c3_llama2_7b_stack"]
    _prefix_sampled(clada, oracle, w, layer_idx, seqs=[0], n_sample=24)
    _ffn_synthetic_scores(clada, oracle, w, layer_idx, seqs=[0])


def test_c3_cogload(clada, oracle):
    _cogload_all_rows(clada, oracle, wl.WORKLOADS["c3_llama2_7b_stack"], n_steps=4)


def test_c4_batch8(clada, oracle):
    w = wl.WORKLOADS["c4_llama3_8b_b8"]
    _prefix_sampled(clada, oracle, w, 1, seqs=[0, 7], n_sample=24)
    _ffn_synthetic_scores(clada, oracle, w, 1, seqs=[0, 5], n_steps=1)
    _cogload_all_rows(clada, oracle, w, n_steps=1)


def test_c5_batch16_ragged(clada, oracle):
    w = wl.WORKLOADS["c5_13b_b16"]
    lengths = wl.prefix_lengths(w)
    shortest, longest = int(np.argmin(lengths)), int(np.argmax(lengths))
    assert min(lengths) >= 256 and max(lengths) <= 4096 and len(set(lengths)) > 8
    _prefix_sampled(clada, oracle, w, 2, seqs=[shortest, longest], n_sample=16)
    for rho in (0.30, 0.60):
        _ffn_synthetic_scores(clada, oracle, w, 2, seqs=[3], n_steps=1, rho=rho)
    _cogload_all_rows(clada, oracle, w, n_steps=1)


def _fp32_levels(lam, gam):
    """The four multipliers Eq. final_threshold can produce, formed as the adjustment forms them (fp32, left to
    right): level = I(s > tau_s) + 2 I(H > tau_H)."""
    one, lam, gam = np.float32(1.0), np.float32(lam), np.float32(gam)
    return [one, one + lam, one + gam, (one + lam) + gam]


def _full_chain(clada, oracle, w, layer_idx, seqs, rho, coeffs, n_tokens=1):
    """Prefix statistics -> calibrated threshold -> guard band -> the masks at the four threshold levels -> FFN
    outputs, on a whole batch of prompts at full width, compared with the oracle on the sequences `seqs`: the
    oracle scores ALL d_ff neurons of those prompts.  `coeffs` lists (lambda, gamma) pairs; each pair gets its own
    guard band and its own four levels.  Returns the numbers of excused neurons and of kept neurons seen."""
    lengths = wl.prefix_lengths(w)
    off = wl.seq_offsets(lengths)
    B, F = len(lengths), w.d_ff
    layer, weights = _layer_on_gpu(clada, w, layer_idx)
    W_in, V_in, W_out = (wl.to_numpy_bits(weights[k]) for k in ("w_gate", "w_up", "w_down"))
    scale = wl.channel_scale(w, "cuda")
    X = torch.cat([wl.hidden_states(w, layer_idx, "prefix", b, n, "cuda", scale) for b, n in enumerate(lengths)])
    xs = torch.stack([wl.hidden_states(w, layer_idx, "decode", b, n_tokens, "cuda", scale) for b in range(B)], dim=1)
    ws = clada.new_workspace(layer, B, off[-1])
    scores = torch.empty(B, F, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_scores(layer, X, off, scores, ws, status)
    tau_base = torch.empty(B, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, rho, tau_base)
    torch.cuda.synchronize()
    A_gpu = scores.cpu().numpy().astype(np.float64)
    A_or = {}
    for b in seqs:
        A_or[b] = oracle.neuron_scores(wl.to_numpy_bits(X[off[b]:off[b + 1]]), [0, lengths[b]], W_in, V_in, W_out)[0]
        assert np.max(np.abs(A_gpu[b] - A_or[b]) / A_or[b]) <= SCORE_TOL, (w.name, layer_idx, b)
    tb = tau_base.cpu().numpy()
    mask = torch.empty(B, F, dtype=torch.uint8, device="cuda")
    idx = torch.empty(B, F, dtype=torch.int32, device="cuda")
    count = torch.empty(B, dtype=torch.int32, device="cuda")
    y = torch.empty(B, w.d_model, dtype=torch.float32, device="cuda")
    excused_total, kept_seen = 0, []
    for lam, gam in coeffs:
        levels = _fp32_levels(lam, gam)
        clada.clada_prefix_select(layer, X, off, tau_base, [float(m) for m in levels], scores, mask, idx, count, ws,
                                  status)
        torch.cuda.synchronize()
        for b in seqs:   # baseline masks of the prefill phase
            e, m = compare_masks(mask[b].cpu().numpy(), A_or[b], float(tb[b]))
            assert m == 0, (w.name, layer_idx, b, "baseline")
            excused_total += e
            n = int(count[b])
            np.testing.assert_array_equal(idx[b, :n].cpu().numpy(), np.nonzero(mask[b].cpu().numpy())[0])
        for k, mult in enumerate(levels):
            tau_k = (tb * mult).astype(np.float32)           # one fp32 product, as the adjustment forms it
            t = k % n_tokens
            clada.clada_sparse_ffn_decode(layer, xs[t].contiguous(), scores, torch.from_numpy(tau_k).cuda(), 1, y, ws,
                                          mask, None, count, status)
            torch.cuda.synchronize()
            for b in seqs:
                m_gpu = mask[b].cpu().numpy()
                e, m = compare_masks(m_gpu, A_or[b], float(tau_k[b]))
                assert m == 0, (w.name, layer_idx, b, lam, gam, k)
                excused_total += e
                assert int(count[b]) == int(m_gpu.sum())
                kept_seen.append(int(count[b]))
                if e == 0:
                    y_or, _, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs[t, b]), W_in, V_in, W_out, A_or[b],
                                                      float(tau_k[b]))
                    assert n_or == int(count[b])
                    if n_or:
                        assert rel_inf(y[b].cpu().numpy(), y_or) <= FFN_TOL_F32, (w.name, layer_idx, b, lam, gam, k)
    assert int(status.item()) == 0
    print(f"{w.name} layer {layer_idx}: sequences {list(seqs)}, excused neurons {excused_total}, "
          f"kept counts {sorted(set(kept_seen))}")
    return excused_total, kept_seen


# The paper's coefficients (0.80 / 0.12), under which the raised thresholds cut nearly everything on these
# synthetic layers, and a small pair under which all four levels keep thousands of neurons.
CHAIN_COEFFS = [(0.80, 0.12), (0.02, 0.01)]


def test_c3_full_chain_2048_tokens(clada, oracle):
    """One layer of the 32-layer stack workload: all 11008 neurons scored by the oracle over the 2048-token prompt."""
    w = wl.WORKLOADS["c3_llama2_7b_stack"]
    _, kept = _full_chain(clada, oracle, w, 15, seqs=[0], rho=0.40, coeffs=CHAIN_COEFFS, n_tokens=2)
    assert max(kept) == w.d_ff - w.k_cut(0.40) or abs(max(kept) - (w.d_ff - w.k_cut(0.40))) <= 2
    assert sum(1 for k in kept if k > 1000) >= 5


def test_c4_full_chain_two_sequences_of_the_batch(clada, oracle):
    """Batch of 8 prompts of 1024 tokens on the 14336-neuron layer; the tile kernel's masks and outputs for two of
    its sequences (one from each tile of 4) against the oracle's scores of all neurons."""
    w = wl.WORKLOADS["c4_llama3_8b_b8"]
    _, kept = _full_chain(clada, oracle, w, 1, seqs=[1, 6], rho=0.40, coeffs=CHAIN_COEFFS)
    assert sum(1 for k in kept if k > 1000) >= 10


def test_c5_full_chain_shortest_and_longest_prompt(clada, oracle):
    """Batch of 16 ragged prompts on the 5120 x 13824 layer (tiles of 2 sequences): the shortest and the longest
    prompt (up to 4096 tokens) against the oracle's scores of all neurons."""
    w = wl.WORKLOADS["c5_13b_b16"]
    lengths = wl.prefix_lengths(w)
    shortest, longest = int(np.argmin(lengths)), int(np.argmax(lengths))
    _, kept = _full_chain(clada, oracle, w, 2, seqs=[shortest, longest], rho=0.30, coeffs=CHAIN_COEFFS)
    assert sum(1 for k in kept if k > 1000) >= 10


def test_c2_threshold_search_full_width(clada, oracle):
    """Offline threshold search on the full-width layer (11008 neurons, two short validation prompts):
    sampled points of the curve against the definition, and the optimality of the chosen threshold."""
    w = wl.WORKLOADS["c2_llama2_7b_layer"]
    layer, weights = _layer_on_gpu(clada, w, 0)
    W_in, V_in, W_out = (wl.to_numpy_bits(weights[k]) for k in ("w_gate", "w_up", "w_down"))
    scale = wl.channel_scale(w, "cuda")
    lengths = [16, 24]
    off = wl.seq_offsets(lengths)
    X = torch.cat([wl.hidden_states(w, 0, "prefix", b, n, "cuda", scale) for b, n in enumerate(lengths)])
    F, bound = w.d_ff, 0.2
    ws = torch.empty(clada.clada_cett_workspace_bytes(layer, off), dtype=torch.uint8, device="cuda")
    tau = torch.empty(1, device="cuda")
    mean = torch.empty(1, device="cuda")
    scores = torch.empty(2, F, device="cuda")
    clada.clada_cett_threshold_search(layer, X, off, bound, tau, mean, scores, ws)
    cums = []
    for b in range(2):
        cum = torch.empty(F + 1, dtype=torch.float64, device="cuda")
        clada.clada_cett_curve(layer, off, b, ws, cum)
        cums.append(cum.cpu().numpy())
    torch.cuda.synchronize()
    sc = scores.cpu().numpy()
    cett = [np.sqrt(c / c[F]) for c in cums]
    # the curve of sample 0 at three cut sizes, by the definition (dense minus sparse output over the prompt)
    X0 = wl.to_numpy_bits(X[:16])
    A0 = oracle.neuron_scores(X0, [0, 16], W_in, V_in, W_out)[0]
    a_sorted = np.sort(A0)
    for k in (F // 4, F // 2, (3 * F) // 4):
        eps = 0.5 * (a_sorted[k - 1] + a_sorted[k])
        num = den = 0.0
        for t in range(16):
            y_d = oracle.dense_ffn(X0[t], W_in, V_in, W_out)
            y_s, _, n_kept = oracle.sparse_ffn(X0[t], W_in, V_in, W_out, A0, eps)
            assert n_kept == F - k
            num += float(np.sum((y_d - y_s) ** 2))
            den += float(np.sum(y_d ** 2))
        assert abs(cett[0][k] - np.sqrt(num / den)) <= 1e-4
    # optimality on the GPU's own curves: tau is a score, feasible, and every larger candidate is infeasible
    t = np.float32(tau.item())
    assert np.any(sc == t) and mean.item() <= bound + 1e-6
    srt = [np.sort(sc[b]) for b in range(2)]
    def mean_at(eps):
        return np.mean([cett[b][np.searchsorted(srt[b], eps, side="left")] for b in range(2)])
    assert abs(mean_at(t) - mean.item()) <= 1e-5
    larger = np.sort(sc[sc > t])
    assert larger.size > 0
    assert all(mean_at(e) > bound - 1e-6 for e in larger[:64])
    assert mean_at(larger[0]) > bound - 1e-6
