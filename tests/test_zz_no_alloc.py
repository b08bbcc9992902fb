"""The decode entry point that allocates nothing, against the workspace entry point.

Some users of this library run where device allocation is off limits: inside another engine's
execution step that owns all device memory, or in a server whose memory plan was frozen at start-up.
clada_sparse_ffn_decode_static serves them with scratch that lives inside the library.  This file
checks, through the C ABI, that it gives the same outputs as clada_sparse_ffn_decode, on two calls
in a row (the second call meets the scratch as the first one left it).  It is collected last, so a
run that stops at the first failure has already run everything else; it also passes on its own in a
fresh process, where its first call is the one that looks up the scratch address.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5      # the tolerance the other FFN parity tests use for fp32 outputs
FFN_TOL_BF16_OUT = 2e-2


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


@pytest.mark.parametrize("name,d,F,y_dtype", [
    ("c2_llama2_7b_layer", 1024, 1500, torch.float32),
    ("c1_small_f32", 512, 1376, torch.float32),
    ("c2_llama2_7b_layer", 4096, 900, torch.bfloat16),
])
def test_static_scratch_entry_matches_workspace_entry(clada, name, d, F, y_dtype):
    w = wl.scaled(wl.WORKLOADS[name], d_model=d, d_ff=F)
    layer = gpu_layer(wl.layer_weights(w, 0), clada)
    ws = clada.new_workspace(layer, 2, 0)
    B = 2
    rng = np.random.default_rng(d + F)
    scores = torch.from_numpy((rng.random((B, F)) + 0.5).astype(np.float32)).cuda()
    xs = torch.stack([wl.hidden_states(w, 0, "decode", b, 2) for b in range(B)], dim=1).cuda()   # [2 calls, B, d]
    tol = FFN_TOL_F32 if y_dtype == torch.float32 else FFN_TOL_BF16_OUT
    for call, tau_val in enumerate((0.9, 1.2)):          # two calls in a row, different kept sets
        tau = torch.full((B,), tau_val, dtype=torch.float32, device="cuda")
        outs = []
        for entry in ("workspace", "static"):
            y = torch.empty(B, d, dtype=y_dtype, device="cuda")
            mask = torch.empty(B, F, dtype=torch.uint8, device="cuda")
            idx = torch.full((B, F), -1, dtype=torch.int32, device="cuda")
            count = torch.empty(B, dtype=torch.int32, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            if entry == "workspace":
                clada.clada_sparse_ffn_decode(layer, xs[call], scores, tau, 1, y, ws, mask, idx, count, status)
            else:
                clada.clada_sparse_ffn_decode_static(layer, xs[call], scores, tau, 1, y, mask, idx, count, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            outs.append((y.float().cpu().numpy(), mask.cpu().numpy(), idx.cpu().numpy(), count.cpu().numpy()))
        (y_ws, m_ws, i_ws, c_ws), (y_st, m_st, i_st, c_st) = outs
        np.testing.assert_array_equal(m_st, m_ws)
        np.testing.assert_array_equal(i_st, i_ws)
        np.testing.assert_array_equal(c_st, c_ws)
        assert 0 < int(c_ws[0]) < F
        for b in range(B):
            assert rel_inf(y_st[b], y_ws[b].astype(np.float64)) <= tol


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
