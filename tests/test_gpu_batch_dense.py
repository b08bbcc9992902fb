"""GPU parity of the dense pass of batched decode: 3-16 sequences of a 16-bit layer go through the layer in one
launch (tensor cores, per-sequence masks applied to the hidden activations), every sequence compared with the
oracle's masked FFN for its own scores and threshold.  Same tolerances as the other FFN parity tests.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5
FFN_TOL_16_OUT = 2e-2


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _case(clada, oracle, name, kw, B, act=0, y_dtypes=(torch.float32,), seed=0, outputs=False):
    w = wl.scaled(wl.WORKLOADS[name], batch=B, **kw)
    d, F = w.d_model, w.d_ff
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada, activation=act)
    W_in, V_in, W_out = oracle_weights(weights, act)
    rng = np.random.default_rng(seed + 1000 * B + d + F)
    scores = (rng.random((B, F)) + 0.5).astype(np.float32)
    taus = (0.7 + 0.6 * rng.random(B)).astype(np.float32)
    taus[1] = np.inf          # keeps nothing
    taus[2] = 0.0             # keeps everything
    xs = torch.stack([wl.hidden_states(w, 0, "decode", b, 1)[0] for b in range(B)])
    ws = clada.new_workspace(layer, B, 0)
    sc_d, tau_d = torch.from_numpy(scores).cuda(), torch.from_numpy(taus).cuda()
    expected = [oracle.sparse_ffn(wl.to_numpy_bits(xs[b]), W_in, V_in, W_out, scores[b].astype(np.float64),
                                  float(taus[b]), act=act) for b in range(B)]
    for y_dtype in y_dtypes:
        tol = FFN_TOL_F32 if y_dtype == torch.float32 else FFN_TOL_16_OUT
        y = torch.full((B, d), float("nan"), dtype=y_dtype, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if outputs:
            mask = torch.empty(B, F, dtype=torch.uint8, device="cuda")
            idx = torch.full((B, F), -1, dtype=torch.int32, device="cuda")
            count = torch.empty(B, dtype=torch.int32, device="cuda")
            clada.clada_sparse_ffn_decode(layer, xs.cuda(), sc_d, tau_d, 1, y, ws, mask, idx, count, status)
        else:
            clada.clada_sparse_ffn_decode(layer, xs.cuda(), sc_d, tau_d, 1, y, ws, None, None, None, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        worst = 0.0
        for b in range(B):
            y_or, m_or, n_or = expected[b]
            if outputs:
                assert int(count[b]) == n_or
                np.testing.assert_array_equal(mask[b].cpu().numpy(), m_or)
            got = y[b].float().cpu().numpy()
            assert np.all(np.isfinite(got)), b
            if n_or == 0:
                assert np.all(got == 0), b
            else:
                err = rel_inf(got, y_or)
                worst = max(worst, err)
                assert err <= tol, (b, y_dtype, err)
        # the same call again gives the same bits (fixed summation orders, counters back at zero)
        y2 = torch.empty_like(y)
        clada.clada_sparse_ffn_decode(layer, xs.cuda(), sc_d, tau_d, 1, y2, ws, None, None, None, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and torch.equal(y, y2)
    return worst


@pytest.mark.parametrize("name,kw,B", [
    ("c4_llama3_8b_b8", {"d_model": 1024, "d_ff": 1800}, 8),      # 13 neurons per CTA, 8 column tiles
    ("c5_13b_b16", {"d_model": 5120, "d_ff": 700}, 16),           # 40 column tiles, 10 per member
    ("c2_llama2_7b_layer", {"d_model": 520, "d_ff": 777}, 5),     # d_model not a multiple of 64: ragged K block, ragged tile
    ("c2_llama2_7b_layer", {"d_model": 64, "d_ff": 100}, 6),      # fewer neurons than CTAs, one column tile
    ("c4_llama3_8b_b8", {"d_model": 2048, "d_ff": 9000}, 9),      # 61 neurons per CTA: three padded rows per box
    ("c4_llama3_8b_b8", {"d_model": 256, "d_ff": 18900}, 7),      # 128 neurons per CTA, the most a launch takes
    ("c5_13b_b16", {"d_model": 8192, "d_ff": 600}, 6),            # 16 column tiles per member: three N = 16 instructions per K step
    ("c4_llama3_8b_b8", {"d_model": 4096, "d_ff": 1000}, 4),      # the smallest batches that take the dense pass
    ("c2_llama2_7b_layer", {"d_model": 1024, "d_ff": 900}, 3),
    ("c2_llama2_7b_layer", {"d_model": 8, "d_ff": 5}, 5),         # one K block of 8 columns, members 1-3 without a column tile
    ("c2_llama2_7b_layer", {"d_model": 72, "d_ff": 130}, 16),     # one neuron per CTA, ragged everything
])
def test_dense_pass_matches_oracle(clada, oracle, name, kw, B):
    _case(clada, oracle, name, kw, B, y_dtypes=(torch.float32, torch.bfloat16), outputs=(B == 8))


@pytest.mark.parametrize("B", [17, 18, 20, 33])
def test_batches_beyond_sixteen_sequences(clada, oracle, B):
    """16 sequences per dense launch; what is left over runs densely too (3 or more), as a tile of two, or singly."""
    _case(clada, oracle, "c2_llama2_7b_layer", {"d_model": 1024, "d_ff": 1500}, B, outputs=True)


@pytest.mark.parametrize("act", [1, 2])
def test_dense_pass_other_ffn_forms(clada, oracle, act):
    _case(clada, oracle, "v1_opt_2p7b_layer", {"d_ff": 1300}, 8, act=act)


def test_dense_pass_fp16_layer(clada, oracle):
    _case(clada, oracle, "c5_13b_b16", {"d_model": 1024, "d_ff": 2100, "dtype": "f16"}, 12,
          y_dtypes=(torch.float32, torch.float16))


@pytest.mark.parametrize("name,picks", [("c5_13b_b16", (2, 7, 15)), ("c4_llama3_8b_b8", (0, 2, 5))])
def test_dense_pass_full_width_sampled(clada, oracle, name, picks):
    """The batched workloads' own widths and batch sizes (c5: d_model 5120, d_ff 13824, 16 sequences; c4: 4096,
    14336, 8) in the launch configuration the benchmark times: three sequences checked against the oracle (among
    them one that keeps all), and the one that keeps nothing is zero."""
    w = wl.WORKLOADS[name]
    B, d, F = w.batch, w.d_model, w.d_ff
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    W_in, V_in, W_out = oracle_weights(weights)
    rng = np.random.default_rng(5)
    scores = (rng.random((B, F)) + 0.5).astype(np.float32)
    taus = np.full(B, 0.9, dtype=np.float32)
    taus[1], taus[2] = np.inf, 0.0
    xs = torch.stack([wl.hidden_states(w, 0, "decode", b, 1)[0] for b in range(B)])
    ws = clada.new_workspace(layer, B, 0)
    y = torch.empty(B, d, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_sparse_ffn_decode(layer, xs.cuda(), torch.from_numpy(scores).cuda(), torch.from_numpy(taus).cuda(), 1,
                                  y, ws, None, None, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((y[1] == 0).all())
    for b in picks:
        y_or, _, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs[b]), W_in, V_in, W_out, scores[b].astype(np.float64),
                                          float(taus[b]))
        assert n_or > 0 and rel_inf(y[b].cpu().numpy(), y_or) <= FFN_TOL_F32, b


def test_stack_call_with_a_batch_runs_dense_passes(clada, oracle):
    """clada_sparse_ffn_decode_layers with 6 sequences: every layer takes the dense pass with tau_final read at
    stride L; same bits as the per-layer calls, and one (layer, sequence) checked against the oracle."""
    L, B = 3, 6
    w = wl.scaled(wl.WORKLOADS["c3_llama2_7b_stack"], d_model=1024, d_ff=1100, batch=B)
    weights = [wl.layer_weights(w, l) for l in range(L)]
    layers = [gpu_layer(wt, clada) for wt in weights]
    stack = clada.LayerStack(layers)
    ws = clada.new_workspace(layers[0], B, 0)
    g = torch.Generator(device="cuda").manual_seed(3)
    scores = torch.rand(L, B, w.d_ff, generator=g, device="cuda") + 0.5
    tau = torch.rand(B, L, generator=g, device="cuda") * 0.5 + 0.75
    x_h = torch.stack([torch.stack([wl.hidden_states(w, l, "decode", b, 1)[0] for b in range(B)]) for l in range(L)])
    x = x_h.cuda()
    y_stack = torch.empty(L, B, w.d_model, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_sparse_ffn_decode_layers(stack, x, scores, tau, y_stack, ws, status)
    y_ref = torch.empty_like(y_stack)
    for l in range(L):
        clada.clada_sparse_ffn_decode(layers[l], x[l], scores[l], tau[:, l], L, y_ref[l], ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(y_stack, y_ref)
    l, b = 2, 4
    W_in, V_in, W_out = oracle_weights(weights[l])
    y_or, _, n_or = oracle.sparse_ffn(wl.to_numpy_bits(x_h[l, b]), W_in, V_in, W_out,
                                      scores[l, b].cpu().numpy().astype(np.float64), float(tau[b, l].item()))
    assert n_or > 0 and rel_inf(y_stack[l, b].cpu().numpy(), y_or) <= FFN_TOL_F32
