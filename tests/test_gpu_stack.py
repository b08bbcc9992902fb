"""The persistent stack kernel (one sequence through all layers in one launch) behind
clada_sparse_ffn_decode_layers: against the oracle layer by layer, and bit for bit against the per-layer
call, whose shares, reduction groups and summation order it keeps.  Cases cover layers that keep nothing or
everything, stacks of two layers and of more than one launch's worth, rows of two vectors per thread, the
non-gated form, every element type, repeated calls on one workspace and mixing with per-layer calls.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5
FFN_TOL_16BIT_OUT = 2e-2


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _stack_case(clada, name, d, F, L, act=0, seed=0, tau_lo=0.75, tau_hi=1.25):
    w = wl.scaled(wl.WORKLOADS[name], d_model=d, d_ff=F)
    weights = [wl.layer_weights(w, l) for l in range(L)]
    layers = [gpu_layer(wt, clada, activation=act) for wt in weights]
    g = torch.Generator().manual_seed(seed + 13 * L + F)
    scores = torch.rand(L, 1, F, generator=g) + 0.5
    tau = torch.rand(1, L, generator=g) * (tau_hi - tau_lo) + tau_lo
    x = torch.stack([wl.hidden_states(w, l, "decode", 0, 1) for l in range(L)])      # [L, 1, d]
    return w, weights, layers, scores, tau, x


def _run_both(clada, layers, x, scores, tau, y_dtype=torch.float32, ws=None):
    L, d = len(layers), layers[0].d_model
    stack = clada.LayerStack(layers)
    if ws is None:
        ws = clada.new_workspace(layers[0], 1, 0)
    xd, sd, td = x.cuda(), scores.cuda(), tau.cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_stack = torch.full((L, 1, d), float("nan"), dtype=y_dtype, device="cuda")
    clada.clada_sparse_ffn_decode_layers(stack, xd, sd, td, y_stack, ws, status)
    y_ref = torch.empty_like(y_stack)
    for l in range(L):
        clada.clada_sparse_ffn_decode(layers[l], xd[l], sd[l], td[:, l], L, y_ref[l], ws, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return y_stack, y_ref, ws


def _check_oracle(oracle, weights, x, scores, tau, y_stack, act=0, tol=FFN_TOL_F32, layers_to_check=None):
    L = len(weights)
    for l in (layers_to_check if layers_to_check is not None else range(L)):
        W_in, V_in, W_out = oracle_weights(weights[l], act)
        y_or, _, n = oracle.sparse_ffn(wl.to_numpy_bits(x[l, 0]), W_in, V_in, W_out,
                                       scores[l, 0].numpy().astype(np.float64), float(tau[0, l]), act=act)
        yg = y_stack[l, 0].float().cpu().numpy()
        if n == 0:
            assert not yg.any()
        else:
            assert rel_inf(yg, y_or) <= tol, (l, n)


@pytest.mark.parametrize("name,d,F,L", [
    ("c2_llama2_7b_layer", 1024, 900, 3),
    ("c2_llama2_7b_layer", 4096, 1200, 2),
    ("c2_llama2_7b_layer", 4096, 700, 5),
    ("c5_13b_b16", 5120, 800, 4),             # two 16-byte vectors per consumer thread
    ("c2_llama2_7b_layer", 8192, 300, 3),
    ("c1_small_f32", 512, 1376, 4),           # fp32 weights
    ("c2_llama2_7b_layer", 64, 100, 7),       # fewer kept neurons than CTAs: most shares are empty
    ("c2_llama2_7b_layer", 520, 20001, 3),    # two score-test batches, ragged last chunk
])
def test_stack_kernel_matches_oracle_and_per_layer_calls(clada, oracle, name, d, F, L):
    w, weights, layers, scores, tau, x = _stack_case(clada, name, d, F, L)
    y_stack, y_ref, _ = _run_both(clada, layers, x, scores, tau)
    assert torch.equal(y_stack, y_ref)          # same shares, same groups, same order: the same bits
    _check_oracle(oracle, weights, x, scores, tau, y_stack)


def test_stack_kernel_empty_and_full_layers(clada, oracle):
    """Layers that keep nothing (their y is zero and they take no grid barrier) between layers that keep
    everything or a part, in every position of the stack."""
    L = 8
    w, weights, layers, scores, tau, x = _stack_case(clada, "c2_llama2_7b_layer", 1024, 640, L)
    inf = float("inf")
    for pattern in ([inf, 1.0, inf, inf, 0.0, 1.0, 0.9, inf], [1.0, inf, 0.0, 1.1, inf, inf, inf, 1.0],
                    [inf] * 8, [0.0] * 8):
        tau = torch.tensor([pattern], dtype=torch.float32)
        y_stack, y_ref, _ = _run_both(clada, layers, x, scores, tau)
        assert torch.equal(y_stack, y_ref)
        _check_oracle(oracle, weights, x, scores, tau, y_stack)


def test_stack_kernel_more_layers_than_one_launch(clada, oracle):
    """130 small layers: the call splits into launches of at most 128 layers."""
    L = 130
    w, weights, layers, scores, tau, x = _stack_case(clada, "c2_llama2_7b_layer", 64, 96, L)
    y_stack, y_ref, _ = _run_both(clada, layers, x, scores, tau)
    assert torch.equal(y_stack, y_ref)
    _check_oracle(oracle, weights, x, scores, tau, y_stack, layers_to_check=[0, 1, 63, 127, 128, 129])


@pytest.mark.parametrize("act", [1, 2])
def test_stack_kernel_other_ffn_forms(clada, oracle, act):
    w, weights, layers, scores, tau, x = _stack_case(clada, "c2_llama2_7b_layer", 2048, 500, 3, act=act)
    y_stack, y_ref, _ = _run_both(clada, layers, x, scores, tau)
    assert torch.equal(y_stack, y_ref)
    _check_oracle(oracle, weights, x, scores, tau, y_stack, act=act)


@pytest.mark.parametrize("wdtype,ydtype", [(torch.float16, torch.float32), (torch.bfloat16, torch.bfloat16),
                                           (torch.float16, torch.float16)])
def test_stack_kernel_element_types(clada, oracle, wdtype, ydtype):
    L, d, F = 3, 1024, 700
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=d, d_ff=F)
    weights = [{k: v.to(wdtype) for k, v in wl.layer_weights(w, l).items()} for l in range(L)]
    layers = [gpu_layer(wt, clada) for wt in weights]
    g = torch.Generator().manual_seed(5)
    scores = torch.rand(L, 1, F, generator=g) + 0.5
    tau = torch.rand(1, L, generator=g) * 0.5 + 0.75
    x = torch.stack([wl.hidden_states(w, l, "decode", 0, 1) for l in range(L)]).to(wdtype)
    y_stack, y_ref, _ = _run_both(clada, layers, x, scores, tau, y_dtype=ydtype)
    assert torch.equal(y_stack, y_ref)
    _check_oracle(oracle, weights, x, scores, tau, y_stack,
                  tol=FFN_TOL_F32 if ydtype == torch.float32 else FFN_TOL_16BIT_OUT)


def test_stack_kernel_repeats_on_one_workspace(clada):
    """Forty stack calls and per-layer calls interleaved on one workspace: the barrier counters return to zero
    after every launch, and the outputs repeat bit for bit."""
    L = 6
    w, weights, layers, scores, tau, x = _stack_case(clada, "c2_llama2_7b_layer", 2048, 800, L)
    y0, y_ref, ws = _run_both(clada, layers, x, scores, tau)
    for _ in range(20):
        y1, y_ref1, _ = _run_both(clada, layers, x, scores, tau, ws=ws)
        assert torch.equal(y1, y0) and torch.equal(y_ref1, y_ref)
    ctrl = ws[:8].view(torch.int32).cpu().tolist()
    assert ctrl == [0, 0]


def test_stack_call_falls_back_to_the_loop(clada):
    """A batch, or a workspace too small for the stack launch's double-buffered partial rows, takes the per-layer
    loop: same results."""
    L, d, F = 3, 1024, 600
    w, weights, layers, scores, tau, x = _stack_case(clada, "c2_llama2_7b_layer", d, F, L)
    stack = clada.LayerStack(layers)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    small = torch.zeros(256 + sms * 2 * d * 4, dtype=torch.uint8, device="cuda")  # room for one layer's rows only
    y_small = torch.empty(L, 1, d, device="cuda")
    clada.clada_sparse_ffn_decode_layers(stack, x.cuda(), scores.cuda(), tau.cuda(), y_small, small)
    y_stack, y_ref, _ = _run_both(clada, layers, x, scores, tau)
    torch.cuda.synchronize()
    assert torch.equal(y_small, y_ref) and torch.equal(y_stack, y_ref)


def test_stack_kernel_full_size_layers(clada, oracle):
    """Three layers of the Llama-2-7B-shaped stack at full width (40 % sparsity, scores drawn by the shared
    generator), four decode tokens, against the oracle."""
    w = wl.WORKLOADS["c3_llama2_7b_stack"]
    idxs = [0, 15, 31]
    weights = [wl.layer_weights(w, l, "cuda") for l in idxs]
    layers = []
    for wt in weights:
        layers.append(clada.Layer(wt["w_gate"], wt["w_up"], wt["w_down"].t().contiguous()))
    stack = clada.LayerStack(layers)
    L, F, d = len(idxs), w.d_ff, w.d_model
    g = torch.Generator(device="cuda").manual_seed(2024)
    scores = torch.rand(L, 1, F, generator=g, device="cuda") + 0.5
    tau = torch.empty(1, L, device="cuda")
    for l in range(L):
        clada.clada_tau_from_sparsity(scores[l], 0.4, tau[:, l])
    scale = wl.channel_scale(w, "cuda")
    xs = torch.stack([wl.hidden_states(w, l, "decode", 0, 4, "cuda", scale) for l in idxs], dim=1).unsqueeze(2)
    ws = clada.new_workspace(layers[0], 1, 0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ys = torch.empty(4, L, 1, d, device="cuda")
    for t in range(4):
        clada.clada_sparse_ffn_decode_layers(stack, xs[t].contiguous(), scores, tau, ys[t], ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sc, tb = scores.cpu().numpy().astype(np.float64), tau.cpu().numpy()
    for i, l in enumerate(idxs):
        W_in, V_in, W_out = (wl.to_numpy_bits(weights[i][k]) for k in ("w_gate", "w_up", "w_down"))
        for t in range(4):
            y_or, _, n = oracle.sparse_ffn(wl.to_numpy_bits(xs[t, i, 0]), W_in, V_in, W_out, sc[i, 0], float(tb[0, i]))
            assert n == F - w.k_cut(0.4)
            assert rel_inf(ys[t, i, 0].cpu().numpy(), y_or) <= FFN_TOL_F32, (l, t)


@pytest.mark.parametrize("name,d,F", [("v2_gemma_2b_layer", 2048, 16384),      # two consumer groups, ring of 16 stages
                                      ("c2_llama2_7b_layer", 4096, 11008),     # one group, ring of 9 stages
                                      ("c5_13b_b16", 5120, 13824)])            # two vectors per thread, 7 stages
def test_many_launches_back_to_back_at_full_width(clada, name, d, F):
    """Hundreds of launches queued without a host synchronisation, each CTA's share several times the ring's
    depth: every launch must give the bits of a launch that ran alone, and no bounded wait may expire.  (Bulk
    copies complete out of order; a consumer group that moved past a stage before its copy had landed would
    take the next use's parity for granted -- this is the case that catches it.)"""
    w = wl.scaled(wl.WORKLOADS[name], d_model=d, d_ff=F)
    L = 4
    layers = []
    for l in range(L):
        wt = wl.layer_weights(w, l, "cuda")
        layers.append(clada.Layer(wt["w_gate"], wt["w_up"] if w.activation != 2 else None,
                                  wt["w_down"].t().contiguous(), activation=w.activation))
    stack = clada.LayerStack(layers)
    g = torch.Generator(device="cuda").manual_seed(F)
    scores = torch.rand(L, 1, F, generator=g, device="cuda") + 0.5
    tau = torch.empty(1, L, device="cuda")
    for l in range(L):
        clada.clada_tau_from_sparsity(scores[l], 0.4, tau[:, l])
    scale = wl.channel_scale(w, "cuda")
    x = torch.stack([wl.hidden_states(w, l, "decode", 0, 1, "cuda", scale) for l in range(L)])   # [L, 1, d]
    ws = clada.new_workspace(layers[0], 1, 0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_alone = torch.empty(L, 1, d, device="cuda")
    for l in range(L):
        clada.clada_sparse_ffn_decode(layers[l], x[l], scores[l], tau[:, l], L, y_alone[l], ws, status=status)
        torch.cuda.synchronize()
    n_rep = 48
    y_loop = torch.empty(n_rep, L, 1, d, device="cuda")
    y_stack = torch.empty(n_rep, L, 1, d, device="cuda")
    for r in range(n_rep):
        for l in range(L):
            clada.clada_sparse_ffn_decode(layers[l], x[l], scores[l], tau[:, l], L, y_loop[r, l], ws, status=status)
    for r in range(n_rep):
        clada.clada_sparse_ffn_decode_layers(stack, x, scores, tau, y_stack[r], ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert float(y_alone.abs().max()) > 0
    assert torch.equal(y_loop, y_alone.expand(n_rep, L, 1, d))
    assert torch.equal(y_stack, y_alone.expand(n_rep, L, 1, d))
