"""The bounded device-side waits, made to run out in the harmless form: clada_selftest_bounded_waits waits on a
shared-memory barrier nobody arrives at and on a grid barrier told to expect one CTA too many, with a small poll
limit.  The kernel must return, report both give-ups and raise CLADA_STATUS_TIMEOUT; the workspace's control
words are then dirty, and after clada_workspace_init ordinary decodes on the same workspace (per-layer launch,
tile of sequences, persistent stack launch) match the oracle again.  Nothing here faults, traps or waits
without a bound.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

FFN_TOL_F32 = 1e-5


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def test_bounded_waits_give_up_and_the_workspace_recovers(clada, oracle):
    L, B, d, F = 3, 2, 1024, 700
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=d, d_ff=F)
    weights = [wl.layer_weights(w, l) for l in range(L)]
    layers = [gpu_layer(wt, clada) for wt in weights]
    ws = clada.new_workspace(layers[0], B, 0)
    report = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for limit in (64, 3000):
        clada.clada_workspace_init(ws)
        report.fill_(-1)
        status.zero_()
        clada.clada_selftest_bounded_waits(ws, limit, report, status)
        torch.cuda.synchronize()                       # the kernel returned: no wait was unbounded
        assert report.cpu().tolist() == [1, 1]         # both waits gave up
        assert int(status.item()) & clada.STATUS_TIMEOUT
        ctrl = ws[:8].view(torch.int32).cpu().tolist()
        assert ctrl[0] != 0                            # the barrier counters are dirty, as after a real time-out
    # recovery as the header prescribes: re-initialise the workspace, then carry on
    clada.clada_workspace_init(ws)
    status.zero_()
    g = torch.Generator().manual_seed(3)
    scores = torch.rand(L, B, F, generator=g) + 0.5
    tau = torch.rand(B, L, generator=g) * 0.4 + 0.8
    x = torch.stack([torch.stack([wl.hidden_states(w, l, "decode", b, 1)[0] for b in range(B)]) for l in range(L)])
    xd, sd, td = x.cuda(), scores.cuda(), tau.cuda()
    y = torch.empty(L, B, d, device="cuda")
    for l in range(L):                                 # a tile of two sequences per layer
        clada.clada_sparse_ffn_decode(layers[l], xd[l], sd[l], td[:, l], L, y[l], ws, status=status)
    y1 = torch.empty(L, 1, d, device="cuda")           # one sequence: per-layer launches, then the stack launch
    for l in range(L):
        clada.clada_sparse_ffn_decode(layers[l], xd[l, :1], sd[l, :1], td[:1, l], L, y1[l], ws, status=status)
    ys = torch.empty(L, 1, d, device="cuda")
    clada.clada_sparse_ffn_decode_layers(clada.LayerStack(layers), xd[:, :1].contiguous(), sd[:, :1].contiguous(),
                                         td[:1].contiguous(), ys, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(ys, y1)
    for l in range(L):
        W_in, V_in, W_out = oracle_weights(weights[l])
        for b in range(B):
            y_or, _, n = oracle.sparse_ffn(wl.to_numpy_bits(x[l, b]), W_in, V_in, W_out,
                                           scores[l, b].numpy().astype(np.float64), float(tau[b, l]))
            assert 0 < n < F
            assert rel_inf(y[l, b].cpu().numpy(), y_or) <= FFN_TOL_F32
            if b == 0:
                assert rel_inf(y1[l, 0].cpu().numpy(), y_or) <= FFN_TOL_F32


def test_selftest_refuses_bad_arguments(clada):
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    report = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(clada.CladaError):
        clada.clada_selftest_bounded_waits(ws, 0, report)             # no polls at all
    with pytest.raises(clada.CladaError):
        clada.clada_selftest_bounded_waits(ws, (1 << 20) + 1, report)  # longer than the documented bound
    with pytest.raises(clada.CladaError):
        clada.clada_selftest_bounded_waits(ws[:64], 100, report)      # no room for the control words
    torch.cuda.synchronize()
