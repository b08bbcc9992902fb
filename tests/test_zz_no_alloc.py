"""The decode entry point that allocates nothing, against the workspace entry point and the oracle.

Some users of this library run where device allocation is off limits: inside another engine's
execution step that owns all device memory, or in a server whose memory plan was frozen at start-up.
clada_sparse_ffn_decode_static serves them with scratch that lives inside the library.  This file
checks, through the C ABI, that it gives the same outputs as clada_sparse_ffn_decode, on two calls
in a row (the second call meets the scratch as the first one left it).  It is collected last, so a
run that stops at the first failure has already run everything else; it also passes on its own in a
fresh process, where its first call is the one that looks up the scratch address.

The workspace entry is itself checked against the oracle elsewhere (tests/test_gpu_parity.py); the batch
cases here check both entries against the oracle as well, because the fixed array can force the static entry
into smaller launches than the workspace entry takes (tiles instead of the dense pass, or smaller tiles: other
CTA shares, so other rounding).
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5      # the tolerance the other FFN parity tests use for fp32 outputs
FFN_TOL_BF16_OUT = 2e-2


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _run(clada, entry, layer, x, scores, tau, y_dtype, ws):
    B, F = scores.shape
    y = torch.empty(B, layer.d_model, dtype=y_dtype, device="cuda")
    mask = torch.empty(B, F, dtype=torch.uint8, device="cuda")
    idx = torch.full((B, F), -1, dtype=torch.int32, device="cuda")
    count = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if entry == "workspace":
        clada.clada_sparse_ffn_decode(layer, x, scores, tau, 1, y, ws, mask, idx, count, status)
    else:
        clada.clada_sparse_ffn_decode_static(layer, x, scores, tau, 1, y, mask, idx, count, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return y.float().cpu().numpy(), mask.cpu().numpy(), idx.cpu().numpy(), count.cpu().numpy()


@pytest.mark.parametrize("name,d,F,B,y_dtype", [
    ("c2_llama2_7b_layer", 1024, 1500, 2, torch.float32),      # tiles of 2 in both entries
    ("c1_small_f32", 512, 1376, 2, torch.float32),
    ("c2_llama2_7b_layer", 4096, 900, 2, torch.bfloat16),
    ("c2_llama2_7b_layer", 4096, 900, 1, torch.float32),       # the single-sequence kernel on the array
    ("c2_llama2_7b_layer", 4096, 900, 3, torch.float32),       # three sequences: one dense pass in both entries
    ("c2_llama2_7b_layer", 4096, 900, 4, torch.float32),
    ("c2_llama2_7b_layer", 4096, 900, 8, torch.float32),       # the Llama-3-8B workload's batch
    ("c5_13b_b16", 5120, 700, 2, torch.float32),               # wider than a tile of 2 fits: one sequence per launch
    ("c2_llama2_7b_layer", 2048, 1200, 5, torch.float32),      # narrow enough for tiles of 4 on the array
])
def test_static_scratch_entry_matches_workspace_entry_and_oracle(clada, oracle, name, d, F, B, y_dtype):
    w = wl.scaled(wl.WORKLOADS[name], d_model=d, d_ff=F)
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    W_in, V_in, W_out = oracle_weights(weights)
    ws = clada.new_workspace(layer, B, 0)
    rng = np.random.default_rng(d + F + B)
    scores_h = (rng.random((B, F)) + 0.5).astype(np.float32)
    scores = torch.from_numpy(scores_h).cuda()
    xs_h = torch.stack([wl.hidden_states(w, 0, "decode", b, 2) for b in range(B)], dim=1)   # [2 calls, B, d]
    xs = xs_h.cuda()
    tol = FFN_TOL_F32 if y_dtype == torch.float32 else FFN_TOL_BF16_OUT
    for call, tau_val in enumerate((0.9, 1.2)):          # two calls in a row, different kept sets
        tau = torch.full((B,), tau_val, dtype=torch.float32, device="cuda")
        y_ws, m_ws, i_ws, c_ws = _run(clada, "workspace", layer, xs[call], scores, tau, y_dtype, ws)
        y_st, m_st, i_st, c_st = _run(clada, "static", layer, xs[call], scores, tau, y_dtype, ws)
        np.testing.assert_array_equal(m_st, m_ws)
        np.testing.assert_array_equal(i_st, i_ws)
        np.testing.assert_array_equal(c_st, c_ws)
        assert 0 < int(c_ws[0]) < F
        for b in range(B):
            y_or, m_or, n_or = oracle.sparse_ffn(wl.to_numpy_bits(xs_h[call, b]), W_in, V_in, W_out,
                                                 scores_h[b].astype(np.float64), float(np.float32(tau_val)))
            np.testing.assert_array_equal(m_st[b], m_or)
            assert int(c_st[b]) == n_or
            assert rel_inf(y_st[b], y_or) <= tol
            assert rel_inf(y_ws[b], y_or) <= tol


def test_static_scratch_entry_after_other_batch_sizes(clada, oracle):
    """Calls of different batch sizes back to back on the one array, and a call that meets control words a
    failed predecessor left non-zero: every call clears the words it needs, so each result stands alone."""
    d, F = 4096, 640
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=d, d_ff=F)
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    W_in, V_in, W_out = oracle_weights(weights)
    rng = np.random.default_rng(7)
    ws = clada.new_workspace(layer, 8, 0)
    for B in (8, 1, 3, 2, 1):
        scores_h = (rng.random((B, F)) + 0.5).astype(np.float32)
        x_h = torch.stack([wl.hidden_states(w, 0, "decode", 10 + b, 1)[0] for b in range(B)])
        tau = torch.full((B,), 1.0, dtype=torch.float32, device="cuda")
        y_st, m_st, _, c_st = _run(clada, "static", layer, x_h.cuda(), torch.from_numpy(scores_h).cuda(), tau,
                                   torch.float32, ws)
        y_ws, m_ws, _, _ = _run(clada, "workspace", layer, x_h.cuda(), torch.from_numpy(scores_h).cuda(), tau,
                                torch.float32, ws)      # a workspace call in between changes nothing for the next
        np.testing.assert_array_equal(m_st, m_ws)
        for b in range(B):
            y_or, m_or, _ = oracle.sparse_ffn(wl.to_numpy_bits(x_h[b]), W_in, V_in, W_out,
                                              scores_h[b].astype(np.float64), 1.0)
            np.testing.assert_array_equal(m_st[b], m_or)
            assert rel_inf(y_st[b], y_or) <= FFN_TOL_F32


def test_static_scratch_entry_rejects_oversized_layers(clada):
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=64, d_ff=40)
    layer = gpu_layer(wl.layer_weights(w, 0), clada)
    layer.c.d_model = 8192 + 8          # pretend: beyond the built-in scratch; nothing is enqueued
    x = torch.zeros(1, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(clada.CladaError, match="beyond"):
        clada.clada_sparse_ffn_decode_static(layer, x, torch.ones(1, 40, device="cuda"),
                                             torch.ones(1, device="cuda"), 1, torch.empty(1, 64, device="cuda"))
    layer.c.d_model = 64
    torch.cuda.synchronize()


def test_static_scratch_entry_refuses_before_enqueueing(clada):
    """A refused call leaves nothing in the stream: a NULL output, a bad batch size and a misaligned x are all
    turned away on the host, and the stream is idle afterwards."""
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=64, d_ff=40)
    layer = gpu_layer(wl.layer_weights(w, 0), clada)
    lib = clada.load()
    x = torch.zeros(2, 64, dtype=torch.bfloat16, device="cuda")
    sc = torch.ones(2, 40, device="cuda")
    tau = torch.ones(2, device="cuda")
    y = torch.empty(2, 64, device="cuda")
    torch.cuda.synchronize()
    st = torch.cuda.current_stream()
    ERR_NULL, ERR_SHAPE, ERR_ALIGN = -1, -2, -3          # clada_error of include/clada.h
    cases = [
        (x.data_ptr(), 2, sc.data_ptr(), tau.data_ptr(), 0, ERR_NULL),                 # y == NULL
        (x.data_ptr(), 0, sc.data_ptr(), tau.data_ptr(), y.data_ptr(), ERR_SHAPE),     # B == 0
        (x.data_ptr() + 2, 1, sc.data_ptr(), tau.data_ptr(), y.data_ptr(), ERR_ALIGN),
    ]
    for xp, B, sp, tp, yp, want in cases:
        rc = lib.clada_sparse_ffn_decode_static(layer.ref, xp, B, sp, tp, 1, yp, 0, None, None, None, None,
                                                st.cuda_stream)
        assert rc == want
        assert st.query()          # nothing was enqueued
