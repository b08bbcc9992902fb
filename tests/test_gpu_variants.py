"""GPU parity of the other FFN forms among the evaluated families (Section 4.1): GELU-gated (activation 1)
and ReLU without a gate projection (activation 2).  Same calls, same tolerances as the SiLU-gated path:
prefix statistics (CUDA-core route for fp32, tensor-core route for bf16), guard band, masks, sparse FFN
per sequence and in tiles of sequences, offline threshold search; then the full widths of the OPT-2.7B-
and Gemma-2B-shaped layers on sampled neurons and whole tokens.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import compare_masks, gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5
SCORE_TOL_F32 = 2e-6
SCORE_TOL_BF16 = 2e-5   # tensor-core accumulators truncate


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _prompts(w, lengths, dev="cpu"):
    scale = wl.channel_scale(w, dev)
    xs = [wl.hidden_states(w, 0, "prefix", b, n, dev, scale) for b, n in enumerate(lengths)]
    return torch.cat(xs, dim=0)


@pytest.mark.parametrize("act", [1, 2])
@pytest.mark.parametrize("name,kw,lengths", [
    ("c1_small_f32", {"d_model": 72, "d_ff": 130}, [70, 0, 129, 1]),
    ("c1_small_f32", {}, [64]),
    ("c2_llama2_7b_layer", {"d_model": 256, "d_ff": 300}, [200, 65]),
    ("v1_opt_2p7b_layer", {"d_ff": 260}, [130]),
])
def test_variant_prefix_scores(clada, oracle, act, name, kw, lengths):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    weights = wl.layer_weights(w, 0)
    X = _prompts(w, lengths)
    off = wl.seq_offsets(lengths)
    layer = gpu_layer(weights, clada, activation=act)
    ws = clada.new_workspace(layer, len(lengths), off[-1])
    scores = torch.empty(len(lengths), w.d_ff, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_scores(layer, X.cuda(), off, scores, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    A_or = oracle.neuron_scores(wl.to_numpy_bits(X), off, *oracle_weights(weights, act), act=act)
    A = scores.cpu().numpy().astype(np.float64)
    tol = SCORE_TOL_F32 if w.dtype == "f32" else SCORE_TOL_BF16
    for b, n in enumerate(lengths):
        if n == 0:
            assert np.all(A[b] == 0.0)
            continue
        err = np.abs(A[b] - A_or[b])
        assert np.max(err) <= tol * np.max(A_or[b]), (b, n)
        if act == 2:
            # a neuron that never fires on the prompt scores exactly 0 on both sides
            np.testing.assert_array_equal(A[b] == 0.0, A_or[b] == 0.0)


def _ffn_case(clada, oracle, w, act, rho, n_steps, B=1, prefix=48):
    weights = wl.layer_weights(w, 0)
    lengths = [prefix + 5 * b for b in range(B)]
    X = _prompts(w, lengths)
    off = wl.seq_offsets(lengths)
    layer = gpu_layer(weights, clada, activation=act)
    ws = clada.new_workspace(layer, B, off[-1])
    scores = torch.empty(B, w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_prefix_scores(layer, X.cuda(), off, scores, ws)
    tau_base = torch.empty(B, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, rho, tau_base)
    mults = [1.0, 1.8, 1.12, 1.92]
    clada.clada_refine_scores(layer, X.cuda(), off, tau_base, mults, 1e-4, scores, ws)
    W_in, V_in, W_out = oracle_weights(weights, act)
    A_or = oracle.neuron_scores(wl.to_numpy_bits(X), off, W_in, V_in, W_out, act=act)
    scale = wl.channel_scale(w)
    xs = torch.stack([wl.hidden_states(w, 0, "decode", b, n_steps, "cpu", scale) for b in range(B)], dim=1)
    y = torch.empty(B, w.d_model, dtype=torch.float32, device="cuda")
    mask = torch.empty(B, w.d_ff, dtype=torch.uint8, device="cuda")
    count = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    worst, excused, mismatched, compared = 0.0, 0, 0, 0
    tb = tau_base.cpu().numpy()
    for t in range(n_steps):
        mult = np.float32(mults[t % 4])
        tau_t = torch.from_numpy(tb * mult).cuda()
        clada.clada_sparse_ffn_decode(layer, xs[t].cuda(), scores, tau_t, 1, y, ws, mask, None, count, status)
        torch.cuda.synchronize()
        for b in range(B):
            tau_b = float(tb[b] * mult)
            y_or, m_or, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs[t, b]), W_in, V_in, W_out, A_or[b], tau_b, act=act)
            m_gpu = mask[b].cpu().numpy()
            e, m = compare_masks(m_gpu, A_or[b], tau_b)
            excused += e
            mismatched += m
            assert int(count[b]) == int(m_gpu.sum())
            if e == 0 and m == 0:
                compared += 1
                worst = max(worst, rel_inf(y[b].cpu().numpy(), y_or))
    assert int(status.item()) == 0
    return worst, excused, mismatched, compared


@pytest.mark.parametrize("act", [1, 2])
@pytest.mark.parametrize("name,kw,B", [
    ("c1_small_f32", {}, 1),
    ("c1_small_f32", {"d_model": 1032, "d_ff": 300}, 1),
    ("c2_llama2_7b_layer", {"d_model": 520, "d_ff": 777}, 1),
    ("v1_opt_2p7b_layer", {"d_ff": 900}, 1),
    ("v2_gemma_2b_layer", {"d_ff": 1500}, 1),
    ("c5_13b_b16", {"d_ff": 600}, 1),          # two 16-byte vectors per consumer thread
    ("v1_opt_2p7b_layer", {"d_ff": 900}, 7),   # tiles of 4 + 2 + 1 sequences
    ("c5_13b_b16", {"d_ff": 700}, 5),
    ("c1_small_f32", {}, 6),
])
def test_variant_sparse_ffn(clada, oracle, act, name, kw, B):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    worst, excused, mismatched, compared = _ffn_case(clada, oracle, w, act, rho=0.4, n_steps=4, B=B)
    assert mismatched == 0 and excused <= 2
    assert compared >= 3 * B and worst <= FFN_TOL_F32, worst


@pytest.mark.parametrize("act", [1, 2])
def test_variant_threshold_search(clada, oracle, act):
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=128, d_ff=200)
    weights = wl.layer_weights(w, 0)
    lengths = [40, 23, 64]
    X = _prompts(w, lengths)
    off = wl.seq_offsets(lengths)
    layer = gpu_layer(weights, clada, activation=act)
    ws = torch.empty(clada.clada_cett_workspace_bytes(layer, off), dtype=torch.uint8, device="cuda")
    tau = torch.empty(1, dtype=torch.float32, device="cuda")
    mean = torch.empty(1, dtype=torch.float32, device="cuda")
    scores = torch.empty(len(lengths), w.d_ff, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_cett_threshold_search(layer, X.cuda(), off, 0.2, tau, mean, scores, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    W_in, V_in, W_out = oracle_weights(weights, act)
    curves = [oracle.cett_curve(wl.to_numpy_bits(X[off[b]:off[b + 1]]), W_in, V_in, W_out, act=act)
              for b in range(len(lengths))]
    A_or = np.stack([c[0] for c in curves])
    cett = np.stack([c[2] for c in curves])
    tau_or, mean_or = oracle.threshold_search(A_or, cett, 0.2)
    # the answer is one of the scores; the GPU's copy of that score differs by fp32 accumulation only
    assert abs(tau.item() - tau_or) <= 1e-5 * tau_or
    assert abs(mean.item() - mean_or) <= 1e-4


def _full_width(clada, oracle, name, n_sample=40):
    """Full-width layer: prefix statistics on sampled neurons, FFN outputs on whole tokens."""
    w = wl.WORKLOADS[name]
    act = w.activation
    T = 256
    weights = wl.layer_weights(w, 0, "cuda")
    layer = gpu_layer(weights, clada, activation=act)
    scale = wl.channel_scale(w, "cuda")
    X = wl.hidden_states(w, 0, "prefix", 0, T, "cuda", scale)
    ws = clada.new_workspace(layer, 1, T)
    scores = torch.empty(1, w.d_ff, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_scores(layer, X, [0, T], scores, ws, status)
    torch.cuda.synchronize()
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(w.d_ff, size=n_sample, replace=False))
    rows[0], rows[-1] = 0, w.d_ff - 1
    r = torch.as_tensor(rows, device="cuda")
    W_in = wl.to_numpy_bits(weights["w_gate"][r])
    V_in = None if act == 2 else wl.to_numpy_bits(weights["w_up"][r])
    W_out = wl.to_numpy_bits(weights["w_down"][:, r].contiguous())
    A_or = oracle.neuron_scores(wl.to_numpy_bits(X), [0, T], W_in, V_in, W_out, act=act)[0]
    A = scores[0].cpu().numpy().astype(np.float64)[rows]
    assert np.max(np.abs(A - A_or)) <= SCORE_TOL_BF16 * np.max(A_or)
    # FFN on whole tokens with generator-drawn scores: identical keep decisions on both sides
    g = torch.Generator(device="cuda").manual_seed(77)
    syn = torch.rand(1, w.d_ff, generator=g, device="cuda") + 0.5
    tau = torch.empty(1, dtype=torch.float32, device="cuda")
    xs = wl.hidden_states(w, 0, "decode", 0, 2, "cuda", scale)
    y = torch.empty(1, w.d_model, dtype=torch.float32, device="cuda")
    mask = torch.empty(1, w.d_ff, dtype=torch.uint8, device="cuda")
    count = torch.empty(1, dtype=torch.int32, device="cuda")
    Wf = oracle_weights(weights, act)
    for t, rho in enumerate((0.4, 0.5)):
        clada.clada_tau_from_sparsity(syn, rho, tau)
        clada.clada_sparse_ffn_decode(layer, xs[t:t + 1].contiguous(), syn, tau, 1, y, ws, mask, None, count, status)
        torch.cuda.synchronize()
        assert int(count[0]) == w.d_ff - w.k_cut(rho)
        y_or, m_or, _ = oracle.sparse_ffn(wl.to_numpy_bits(xs[t]), *Wf, syn[0].cpu().numpy().astype(np.float64),
                                          float(tau.item()), act=act)
        np.testing.assert_array_equal(mask[0].cpu().numpy(), m_or)
        assert rel_inf(y[0].cpu().numpy(), y_or) <= FFN_TOL_F32
    assert int(status.item()) == 0


def test_opt_shaped_layer_full_width(clada, oracle):
    _full_width(clada, oracle, "v1_opt_2p7b_layer")


def test_gemma_shaped_layer_full_width(clada, oracle):
    _full_width(clada, oracle, "v2_gemma_2b_layer")


def test_variant_layer_validation(clada):
    """The non-gated form takes no w_up; an unknown activation code is refused by the library."""
    w = wl.scaled(wl.WORKLOADS["c1_small_f32"], d_model=64, d_ff=96)
    weights = wl.layer_weights(w, 0, "cuda")
    wdt = weights["w_down"].t().contiguous()
    with pytest.raises(clada.CladaError):
        clada.Layer(weights["w_gate"], weights["w_up"], wdt, activation=clada.ACT_RELU)
    with pytest.raises(clada.CladaError):
        clada.Layer(weights["w_gate"], None, wdt, activation=clada.ACT_GELU_GATED)
    layer = clada.Layer(weights["w_gate"], weights["w_up"], wdt)
    layer.c.activation = 9
    norms = torch.empty(w.d_ff, dtype=torch.float32, device="cuda")
    with pytest.raises(clada.CladaError):
        clada.clada_down_norms(layer, norms)


# ---- fp16 weights and activations (the precision of the paper's latency runs) -------------------------

@pytest.mark.parametrize("act", [0, 1, 2])
@pytest.mark.parametrize("name,kw,lengths", [
    ("c2_llama2_7b_layer", {"d_model": 256, "d_ff": 300}, [200, 0, 65, 1]),
    ("c2_llama2_7b_layer", {"d_ff": 200}, [300]),
])
def test_fp16_prefix_scores(clada, oracle, act, name, kw, lengths):
    test_variant_prefix_scores(clada, oracle, act, name, dict(kw, dtype="f16"), lengths)


@pytest.mark.parametrize("act", [0, 1, 2])
@pytest.mark.parametrize("name,kw,B", [
    ("c2_llama2_7b_layer", {"d_model": 520, "d_ff": 777}, 1),
    ("c2_llama2_7b_layer", {"d_ff": 1200}, 1),
    ("c5_13b_b16", {"d_ff": 600}, 1),
    ("c4_llama3_8b_b8", {"d_model": 1024, "d_ff": 1800}, 7),
    ("c5_13b_b16", {"d_ff": 700}, 5),
])
def test_fp16_sparse_ffn(clada, oracle, act, name, kw, B):
    w = wl.scaled(wl.WORKLOADS[name], dtype="f16", **kw)
    worst, excused, mismatched, compared = _ffn_case(clada, oracle, w, act, rho=0.4, n_steps=4, B=B)
    assert mismatched == 0 and excused <= 2
    assert compared >= 3 * B and worst <= FFN_TOL_F32, worst


def test_fp16_output_and_logits(clada, oracle):
    """y written as fp16 (rounded once from the fp32 sums), and surprisal / entropy from fp16 logits."""
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], dtype="f16", d_model=512, d_ff=640)
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    g = torch.Generator().manual_seed(3)
    scores = (torch.rand(1, w.d_ff, generator=g) + 0.5).cuda()
    tau = torch.empty(1, dtype=torch.float32, device="cuda")
    clada.clada_tau_from_sparsity(scores, 0.4, tau)
    x = wl.hidden_states(w, 0, "decode", 0, 1, "cpu", wl.channel_scale(w))
    ws = clada.new_workspace(layer, 1, 0)
    y32 = torch.empty(1, w.d_model, dtype=torch.float32, device="cuda")
    y16 = torch.empty(1, w.d_model, dtype=torch.float16, device="cuda")
    clada.clada_sparse_ffn_decode(layer, x.cuda(), scores, tau, 1, y32, ws)
    clada.clada_sparse_ffn_decode(layer, x.cuda(), scores, tau, 1, y16, ws)
    torch.cuda.synchronize()
    assert torch.equal(y16, y32.to(torch.float16))            # same sums, one rounding to nearest even
    y_or, _, _ = oracle.sparse_ffn(wl.to_numpy_bits(x[0]), *oracle_weights(weights),
                                   scores[0].cpu().numpy().astype(np.float64), float(tau.item()))
    assert rel_inf(y32[0].cpu().numpy(), y_or) <= FFN_TOL_F32
    V = 50272
    logits = (torch.randn(3, V, generator=g) * 3).to(torch.float16)
    tokens = torch.tensor([0, V - 1, 12345], dtype=torch.int32)
    s = torch.empty(3, device="cuda")
    h = torch.empty(3, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_cogload(logits.cuda(), tokens.cuda(), s, h, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for b in range(3):
        so, ho = oracle.cogload(logits[b].numpy(), int(tokens[b]))
        assert abs(s[b].item() - so) <= 1e-4 and abs(h[b].item() - ho) <= 1e-4


def test_fp16_threshold_search(clada, oracle):
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], dtype="f16", d_model=128, d_ff=200)
    weights = wl.layer_weights(w, 0)
    lengths = [40, 23]
    X = _prompts(w, lengths)
    off = wl.seq_offsets(lengths)
    layer = gpu_layer(weights, clada)
    ws = torch.empty(clada.clada_cett_workspace_bytes(layer, off), dtype=torch.uint8, device="cuda")
    tau = torch.empty(1, dtype=torch.float32, device="cuda")
    mean = torch.empty(1, dtype=torch.float32, device="cuda")
    scores = torch.empty(len(lengths), w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_cett_threshold_search(layer, X.cuda(), off, 0.2, tau, mean, scores, ws)
    torch.cuda.synchronize()
    W_in, V_in, W_out = oracle_weights(weights)
    curves = [oracle.cett_curve(wl.to_numpy_bits(X[off[b]:off[b + 1]]), W_in, V_in, W_out) for b in range(2)]
    tau_or, mean_or = oracle.threshold_search(np.stack([c[0] for c in curves]), np.stack([c[2] for c in curves]), 0.2)
    assert abs(tau.item() - tau_or) <= 1e-5 * tau_or and abs(mean.item() - mean_or) <= 1e-4
