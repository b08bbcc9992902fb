"""GPU parity of the nested index lists (compressed form of the four masks of Eq. final_threshold).

  * clada_nested_build: order and counts bit-exact against the oracle on the GPU's own fp32 scores
    (both sides compare the same fp32 numbers), and the listed sets equal to clada_select's masks;
  * clada_cogload_level: the level against the oracle's, and against the threshold clada_cogload_adjust yields;
  * clada_sparse_ffn_decode_nested: outputs against the oracle's thresholded FFN and against the
    score-scanning kernel, over all four levels, on small and full-width layers.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5
LAM, GAM = 0.80, 0.12


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _thresholds(tau_base, lam, gam):
    """The four fp32 thresholds as Eq. final_threshold forms them."""
    one, l, g = np.float32(1.0), np.float32(lam), np.float32(gam)
    mults = [one, one + l, one + g, (one + l) + g]
    return [np.float32(np.float32(tau_base) * m) for m in mults]


@pytest.mark.parametrize("F", [1, 2, 33, 1376, 4097, 11008, 16384, 28672])
@pytest.mark.parametrize("lam,gam", [(LAM, GAM), (-0.3, -0.1)])
def test_nested_build_bit_exact(clada, oracle, F, lam, gam):
    B = 3
    g = torch.Generator().manual_seed(F)
    scores = (torch.rand(B, F, generator=g) * 0.2 + 0.9).float()
    if F >= 33:
        scores[0, 5] = scores[0, 17] = scores[0, 2]          # equal scores
        scores[1, :] = scores[1, 0]                          # all equal
    tau_base = torch.tensor([[0.55, 7.0], [float(scores[1, 0]), 7.0], [0.93, 7.0]], dtype=torch.float32)  # stride 2
    if F >= 33:
        tau_base[0, 0] = scores[0, 2]                        # equality keeps
    order = torch.empty(B, F, dtype=torch.int32, device="cuda")
    counts = torch.empty(B, 4, dtype=torch.int32, device="cuda")
    clada.clada_nested_build(scores.cuda(), tau_base.cuda(), lam, gam, order, counts, tau_stride=2)
    torch.cuda.synchronize()
    mask = torch.empty(1, F, dtype=torch.uint8, device="cuda")
    for b in range(B):
        taus = _thresholds(tau_base[b, 0].item(), lam, gam)
        o_or, c_or = oracle.nested_lists(scores[b].numpy().astype(np.float64), np.array(taus, np.float64))
        np.testing.assert_array_equal(order[b].cpu().numpy(), o_or)
        np.testing.assert_array_equal(counts[b].cpu().numpy(), c_or)
        for k in range(4):                                   # the listed set is clada_select's mask
            clada.clada_select(scores[b:b + 1].cuda(), torch.tensor([taus[k]]).cuda(), 1, mask)
            listed = np.zeros(F, np.uint8)
            listed[order[b, :int(counts[b, k])].cpu().numpy()] = 1
            np.testing.assert_array_equal(mask[0].cpu().numpy(), listed)


@pytest.mark.parametrize("F", [200, 11008, 16384])
@pytest.mark.parametrize("B", [1, 40])
def test_nested_build_puts_non_numbers_where_the_selection_puts_them(clada, F, B):
    """A NaN score is cut by every threshold (A_j >= tau is false), a zero of either sign only by positive ones:
    the list must order them so that order[:counts[k]] is still exactly clada_select's kept set -- on both the
    rank-sort and the bitonic route (B = 40 wide sequences takes the latter)."""
    g = torch.Generator().manual_seed(F + B)
    scores = (torch.rand(B, F, generator=g) * 0.2 + 0.9).float()
    scores[0, 3] = float("nan")
    scores[0, F - 1] = float("nan")
    scores[0, 7] = -0.0
    scores[0, 9] = 0.0
    scores[-1, 0] = float("nan")
    tau_base = torch.full((B,), 0.95, dtype=torch.float32)
    order = torch.empty(B, F, dtype=torch.int32, device="cuda")
    counts = torch.empty(B, 4, dtype=torch.int32, device="cuda")
    sd = scores.cuda()
    clada.clada_nested_build(sd, tau_base.cuda(), LAM, GAM, order, counts)
    mask = torch.empty(1, F, dtype=torch.uint8, device="cuda")
    cnt = torch.empty(1, dtype=torch.int32, device="cuda")
    for b in (0, B - 1):
        o = order[b].cpu().numpy()
        assert sorted(o.tolist()) == list(range(F))                  # a permutation
        nan_idx = set(np.nonzero(np.isnan(scores[b].numpy()))[0].tolist())
        assert set(o[F - len(nan_idx):].tolist()) == nan_idx         # the NaNs come last
        for k, tau in enumerate(_thresholds(0.95, LAM, GAM)):
            clada.clada_select(sd[b:b + 1], torch.tensor([tau]).cuda(), 1, mask, None, cnt)
            n = int(counts[b, k])
            assert n == int(cnt.item())
            kept = np.zeros(F, dtype=np.uint8)
            kept[o[:n]] = 1
            np.testing.assert_array_equal(kept, mask[0].cpu().numpy())
    torch.cuda.synchronize()


def test_cogload_level_matches_adjustment(clada, oracle):
    w = wl.WORKLOADS["c2_llama2_7b_layer"]
    n = 16
    logits = wl.decode_logits(w, 0, n)
    tokens = wl.chosen_tokens(w, logits, 0).contiguous()
    so = [oracle.cogload(logits[t].numpy(), int(tokens[t])) for t in range(n)]
    tau_s = wl.universal_threshold([a for a, _ in so])
    tau_H = wl.universal_threshold([b for _, b in so])
    s = torch.empty(n, device="cuda")
    h = torch.empty(n, device="cuda")
    level = torch.empty(n, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_cogload_level(logits.cuda(), tokens.cuda(), tau_s, tau_H, s, h, level, status)
    tau_base = torch.full((n, 1), 0.731, device="cuda")
    lam = torch.tensor([LAM], device="cuda")
    gam = torch.tensor([GAM], device="cuda")
    tf = torch.empty(n, 1, device="cuda")
    s2 = torch.empty(n, device="cuda")
    h2 = torch.empty(n, device="cuda")
    clada.clada_cogload_adjust(logits.cuda(), tokens.cuda(), tau_base, lam, gam, tau_s, tau_H, s2, h2, tf, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(s, s2) and torch.equal(h, h2)
    taus = _thresholds(0.731, LAM, GAM)
    lv = level.cpu().numpy()
    assert set(lv.tolist()) == {0, 1, 2, 3}                  # the workload's tokens reach all four levels
    for t in range(n):
        assert lv[t] == oracle.load_level(so[t][0], so[t][1], tau_s, tau_H)
        assert np.float32(tf[t, 0].item()) == taus[lv[t]]
    # a token outside the vocabulary: surprisal NaN compares false, the entropy bit still counts
    bad = tokens.clone()
    bad[0] = w.vocab
    clada.clada_cogload_level(logits.cuda(), bad.cuda(), tau_s, tau_H, s, h, level, status)
    torch.cuda.synchronize()
    assert int(status.item()) & 1 and int(level[0]) == (2 if so[0][1] > tau_H else 0)


def _nested_case(clada, oracle, w, act=0, B=2, prefix=48, rho=0.4):
    weights = wl.layer_weights(w, 0)
    lengths = [prefix + 7 * b for b in range(B)]
    scale = wl.channel_scale(w)
    X = torch.cat([wl.hidden_states(w, 0, "prefix", b, n, "cpu", scale) for b, n in enumerate(lengths)])
    off = wl.seq_offsets(lengths)
    layer = gpu_layer(weights, clada, activation=act)
    ws = clada.new_workspace(layer, B, off[-1])
    scores = torch.empty(B, w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_prefix_scores(layer, X.cuda(), off, scores, ws)
    tau_base = torch.empty(B, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, rho, tau_base)
    # lambda, gamma small enough that the synthetic layer keeps a useful number of neurons at every level
    lam, gam = 0.02, 0.005
    one = np.float32(1.0)
    mults = [float(m) for m in (one, one + np.float32(lam), one + np.float32(gam), (one + np.float32(lam)) + np.float32(gam))]
    clada.clada_refine_scores(layer, X.cuda(), off, tau_base, mults, 1e-4, scores, ws)
    order = torch.empty(B, w.d_ff, dtype=torch.int32, device="cuda")
    counts = torch.empty(B, 4, dtype=torch.int32, device="cuda")
    clada.clada_nested_build(scores, tau_base, lam, gam, order, counts)
    W_in, V_in, W_out = oracle_weights(weights, act)
    sc = scores.cpu().numpy().astype(np.float64)              # the keep decisions are taken on these fp32 numbers
    xs = torch.stack([wl.hidden_states(w, 0, "decode", b, 4, "cpu", scale) for b in range(B)], dim=1)
    y = torch.empty(B, w.d_model, dtype=torch.float32, device="cuda")
    y_scan = torch.empty(B, w.d_model, dtype=torch.float32, device="cuda")
    kept = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tb = tau_base.cpu().numpy()
    worst = 0.0
    for t in range(4):
        level = torch.tensor([(t + b) % 4 for b in range(B)], dtype=torch.int32, device="cuda")
        clada.clada_sparse_ffn_decode_nested(layer, xs[t].cuda(), order, counts, level, y, ws, kept, status)
        taus = np.array([_thresholds(tb[b], lam, gam)[(t + b) % 4] for b in range(B)], np.float32)
        clada.clada_sparse_ffn_decode(layer, xs[t].cuda(), scores, torch.from_numpy(taus).cuda(), 1, y_scan, ws)
        torch.cuda.synchronize()
        for b in range(B):
            y_or, m_or, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs[t, b]), W_in, V_in, W_out, sc[b], float(taus[b]),
                                                 act=act)
            assert int(kept[b]) == n_or == int(counts[b, (t + b) % 4])
            worst = max(worst, rel_inf(y[b].cpu().numpy(), y_or))
            assert rel_inf(y[b].cpu().numpy(), y_scan[b].cpu().numpy().astype(np.float64)) <= FFN_TOL_F32
    assert int(status.item()) == 0
    return worst


@pytest.mark.parametrize("name,kw,act", [
    ("c1_small_f32", {}, 0),
    ("c2_llama2_7b_layer", {"d_model": 520, "d_ff": 777}, 0),
    ("c2_llama2_7b_layer", {"d_ff": 1200}, 1),
    ("v1_opt_2p7b_layer", {"d_ff": 900}, 2),
    ("c5_13b_b16", {"d_ff": 600, "dtype": "f16"}, 0),
])
def test_nested_decode_parity(clada, oracle, name, kw, act):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    assert _nested_case(clada, oracle, w, act=act) <= FFN_TOL_F32


def test_nested_decode_full_width_c2(clada, oracle):
    """The benchmark's layer at full width: generator-drawn scores, all four levels, whole tokens."""
    w = wl.WORKLOADS["c2_llama2_7b_layer"]
    weights = wl.layer_weights(w, 0, "cuda")
    layer = gpu_layer(weights, clada)
    g = torch.Generator(device="cuda").manual_seed(11)
    scores = torch.rand(1, w.d_ff, generator=g, device="cuda") + 0.5
    tau_base = torch.empty(1, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, 0.4, tau_base)
    order = torch.empty(1, w.d_ff, dtype=torch.int32, device="cuda")
    counts = torch.empty(1, 4, dtype=torch.int32, device="cuda")
    clada.clada_nested_build(scores, tau_base, 0.10, 0.03, order, counts)
    ws = clada.new_workspace(layer, 1, 0)
    xs = wl.hidden_states(w, 0, "decode", 0, 4, "cuda", wl.channel_scale(w, "cuda"))
    y = torch.empty(1, w.d_model, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Wf = oracle_weights(weights)
    sc = scores[0].cpu().numpy().astype(np.float64)
    taus = _thresholds(tau_base.item(), 0.10, 0.03)
    o_or, c_or = oracle.nested_lists(sc, np.array(taus, np.float64))
    np.testing.assert_array_equal(order[0].cpu().numpy(), o_or)
    np.testing.assert_array_equal(counts[0].cpu().numpy(), c_or)
    assert c_or[0] == w.d_ff - w.k_cut(0.4) and c_or[3] < c_or[1] < c_or[2] < c_or[0]
    for k in range(4):
        level = torch.tensor([k], dtype=torch.int32, device="cuda")
        clada.clada_sparse_ffn_decode_nested(layer, xs[k:k + 1].contiguous(), order, counts, level, y, ws, None, status)
        torch.cuda.synchronize()
        y_or, _, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs[k]), *Wf, sc, float(taus[k]))
        assert n_or == c_or[k]
        assert rel_inf(y[0].cpu().numpy(), y_or) <= FFN_TOL_F32
    assert int(status.item()) == 0


def test_nested_decode_bad_inputs_are_clamped_and_reported(clada):
    """Out-of-range level, count or index: no access leaves the layer, the status word says so."""
    w = wl.scaled(wl.WORKLOADS["c1_small_f32"], d_model=64, d_ff=96)
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    ws = clada.new_workspace(layer, 1, 0)
    x = wl.hidden_states(w, 0, "decode", 0, 1, "cpu", wl.channel_scale(w)).cuda()
    y = torch.empty(1, w.d_model, dtype=torch.float32, device="cuda")
    good_order = torch.arange(w.d_ff, dtype=torch.int32, device="cuda").view(1, -1)
    cases = [
        (good_order, [10, 10, 10, 10], 7),                   # level outside 0..3
        (good_order, [w.d_ff + 5, 0, 0, 0], 0),              # count beyond d_ff
        (good_order, [-3, 0, 0, 0], 0),                      # negative count
        (torch.full((1, w.d_ff), w.d_ff + 100, dtype=torch.int32, device="cuda"), [8, 8, 8, 8], 1),  # bad indices
    ]
    for order, counts, level in cases:
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        clada.clada_sparse_ffn_decode_nested(layer, x, order.contiguous(),
                                             torch.tensor([counts], dtype=torch.int32, device="cuda"),
                                             torch.tensor([level], dtype=torch.int32, device="cuda"), y, ws, None, status)
        torch.cuda.synchronize()
        assert int(status.item()) & 8
        assert torch.isfinite(y).all()
    # nothing kept at a level: y = 0
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_sparse_ffn_decode_nested(layer, x, good_order, torch.tensor([[5, 0, 5, 5]], dtype=torch.int32, device="cuda"),
                                         torch.tensor([1], dtype=torch.int32, device="cuda"), y, ws, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.all(y == 0)


def test_many_launches_share_one_workspace(clada):
    """Three hundred launches of every decode flavour back to back on ONE workspace (score scan, nested list,
    nothing kept, a tile of four sequences): the grid barrier's counters must be back at zero after each, the
    status word stays clear, and every flavour returns the same bits every time."""
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=1024, d_ff=2400)
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    B = 4
    g = torch.Generator().manual_seed(5)
    scores = (torch.rand(B, w.d_ff, generator=g) + 0.5).cuda()
    tau = torch.empty(B, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, 0.4, tau)
    tau_none = torch.full((B,), 10.0, device="cuda")
    order = torch.empty(B, w.d_ff, dtype=torch.int32, device="cuda")
    counts = torch.empty(B, 4, dtype=torch.int32, device="cuda")
    clada.clada_nested_build(scores, tau, 0.1, 0.03, order, counts)
    level = torch.tensor([0, 1, 2, 3], dtype=torch.int32, device="cuda")
    x = torch.stack([wl.hidden_states(w, 0, "decode", b, 1, "cpu", wl.channel_scale(w))[0] for b in range(B)]).cuda()
    ws = clada.new_workspace(layer, B, 0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = {k: torch.empty(B, w.d_model, dtype=torch.float32, device="cuda") for k in ("scan1", "nested", "none", "tile")}
    first = None
    for it in range(75):
        clada.clada_sparse_ffn_decode(layer, x[:1], scores[:1], tau[:1], 1, outs["scan1"][:1], ws, status=status)
        clada.clada_sparse_ffn_decode_nested(layer, x, order, counts, level, outs["nested"], ws, None, status)
        clada.clada_sparse_ffn_decode(layer, x[:1], scores[:1], tau_none[:1], 1, outs["none"][:1], ws, status=status)
        clada.clada_sparse_ffn_decode(layer, x, scores, tau, 1, outs["tile"], ws, status=status)
        if it == 0:
            torch.cuda.synchronize()
            first = {k: v.clone() for k, v in outs.items()}
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.all(outs["none"][:1] == 0)
    for k in outs:
        rows = slice(0, 1) if k in ("scan1", "none") else slice(0, B)
        assert torch.equal(outs[k][rows], first[k][rows]), k
    # the tile's first sequence and the single-sequence launch keep the same neurons
    assert torch.allclose(outs["tile"][0], outs["scan1"][0], rtol=0, atol=1e-5 * float(outs["scan1"][0].abs().max()))
    # the control words are back at zero
    assert int(ws[:16].view(torch.int32).abs().sum().item()) == 0
