"""GPU parity of the dense prefill FFN with the statistics as a by-product, in chunks.

  * hidden activations Z against the oracle's (equal up to one unit in the last place of the storage type on
    the few elements where the fp32 value sits next to a rounding boundary);
  * Y = Z W_out^T against the oracle's down projection OF THE GPU'S OWN Z (isolates the second contraction:
    fp32 tensor-core accumulation only), and against the oracle's whole dense FFN (adds the rounding flips);
  * chunked accumulation of the statistics against the oracle's scores over the whole prompts.
"""
import numpy as np
import pytest
import torch

from paper_2502_19078_b200 import workloads as wl
from tests._util import gpu_layer, oracle_weights, rel_inf

pytestmark = pytest.mark.gpu

SCORE_TOL = 2e-5
DOWN_TOL = 3e-5      # fp32 tensor-core accumulation over d_ff terms, relative to the largest output
FFN_TOL = 2e-3       # plus the storage-type rounding of z taken on fp32 instead of fp64 values: a value near a
                     # rounding boundary of the 16-bit type may land on the other side, one ulp of z (2^-8 relative for bf16)


@pytest.fixture(scope="module")
def clada():
    from paper_2502_19078_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _widen(t):
    return t.to(torch.float64).cpu().numpy()


def _ulp(v, dtype):
    """Spacing of the storage type at |v| (normal range)."""
    p = 8 if dtype == "bf16" else 11
    e = np.floor(np.log2(np.maximum(np.abs(v), 1e-30)))
    return 2.0 ** (e - (p - 1))


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("act", [0, 1, 2])
@pytest.mark.parametrize("d,F,lengths", [(256, 304, [200, 0, 65, 1]), (520, 136, [130])])
def test_prefill_ffn_parity(clada, oracle, dtype, act, d, F, lengths):
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=d, d_ff=F, dtype=dtype)
    weights = wl.layer_weights(w, 0)
    scale = wl.channel_scale(w)
    X = torch.cat([wl.hidden_states(w, 0, "prefix", b, n, "cpu", scale) for b, n in enumerate(lengths)])
    off = wl.seq_offsets(lengths)
    T = off[-1]
    layer = gpu_layer(weights, clada, activation=act)
    ws = clada.new_workspace(layer, len(lengths), T)
    sumsq = torch.zeros(len(lengths), F, dtype=torch.float32, device="cuda")
    Z = torch.full((T, F), float("nan"), dtype=w.torch_dtype, device="cuda")
    Y = torch.full((T, d), float("nan"), dtype=torch.float32, device="cuda")
    scores = torch.empty(len(lengths), F, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_accumulate(layer, X.cuda(), off, sumsq, ws, Z, status)
    clada.clada_prefix_finish(layer, sumsq, scores)
    # with the workspace these few tiles are split along K (five CTAs per tile at d_ff 304, three at 136)
    clada.clada_prefill_down(layer, weights["w_down"].cuda().contiguous(), Z, Y, status, ws=ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    W_in, V_in, W_out = oracle_weights(weights, act)
    Xn = wl.to_numpy_bits(X)
    # statistics
    A_or = oracle.neuron_scores(Xn, off, W_in, V_in, W_out, act=act)
    A = scores.cpu().numpy().astype(np.float64)
    for b, n in enumerate(lengths):
        if n == 0:
            assert np.all(A[b] == 0.0)
        else:
            assert np.max(np.abs(A[b] - A_or[b])) <= SCORE_TOL * np.max(A_or[b])
    # hidden activations
    Z_or = oracle.prefill_hidden(Xn, W_in, V_in, act=act, round_z=True)
    Zg = _widen(Z)
    assert np.isfinite(Zg).all()
    diff = np.abs(Zg - Z_or)
    # the fp32 value differs from the fp64 one by ~1e-5 relative (plus the absolute error of a cancelling
    # dot product), so it may fall on the other side of a rounding boundary: one unit, on few elements
    gmax = np.max(np.abs(Z_or))
    assert np.all(diff <= _ulp(Z_or, dtype) * 1.0001 + 2e-5 * gmax)
    assert np.mean(diff > 0) <= 0.03
    # down projection of the GPU's own Z
    Y_own = oracle.down_proj(Zg, W_out)
    Yg = Y.cpu().numpy().astype(np.float64)
    assert np.isfinite(Yg).all()
    assert rel_inf(Yg, Y_own) <= DOWN_TOL
    # the whole dense FFN
    Y_or = oracle.down_proj(Z_or, W_out)
    assert rel_inf(Yg, Y_or) <= FFN_TOL


def test_prefill_output_types_and_ragged_columns(clada, oracle):
    """Y in bf16 / fp16, a d_model that is not a multiple of the 128-column tile, T not a multiple of 128."""
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=200, d_ff=264)
    weights = wl.layer_weights(w, 0)
    T = 150
    X = wl.hidden_states(w, 0, "prefix", 0, T, "cpu", wl.channel_scale(w))
    layer = gpu_layer(weights, clada)
    ws = clada.new_workspace(layer, 1, T)
    sumsq = torch.zeros(1, w.d_ff, dtype=torch.float32, device="cuda")
    Z = torch.empty(T, w.d_ff, dtype=torch.bfloat16, device="cuda")
    clada.clada_prefix_accumulate(layer, X.cuda(), [0, T], sumsq, ws, Z)
    wd = weights["w_down"].cuda().contiguous()
    Y32 = torch.empty(T, w.d_model, dtype=torch.float32, device="cuda")
    clada.clada_prefill_down(layer, wd, Z, Y32)
    for dt in (torch.bfloat16, torch.float16):
        Y16 = torch.full((T + 3, w.d_model), 7.0, dtype=dt, device="cuda")      # rows past T must stay untouched
        clada.clada_prefill_down(layer, wd, Z, Y16[:T])
        torch.cuda.synchronize()
        assert torch.equal(Y16[:T], Y32.to(dt)) and torch.all(Y16[T:] == 7.0)
    Y_own = oracle.down_proj(_widen(Z), oracle_weights(weights)[2])
    assert rel_inf(Y32.cpu().numpy().astype(np.float64), Y_own) <= DOWN_TOL


@pytest.mark.parametrize("d,F,T", [(512, 1000, 300),     # 6 tiles x 8 splits of 2 K blocks, the last one ragged
                                   (1024, 4160, 128),    # 4 tiles x 8 splits of 9 K blocks (the last: 2)
                                   (2048, 704, 600)])    # 40 tiles x 3 splits of 4 K blocks (the last: 3)
def test_prefill_down_split_along_k(clada, oracle, d, F, T):
    """A short prompt's down projection with a workspace: every output tile's K range is split among several CTAs
    and their fp32 partial outputs are added in a fixed order.  Against the oracle's projection of the same Z,
    against the unsplit call (fp32 rounding apart), bit-identical on repetition, in fp32 and bf16 outputs, and
    rows past T stay untouched."""
    w = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=d, d_ff=F)
    weights = wl.layer_weights(w, 0)
    layer = gpu_layer(weights, clada)
    g = torch.Generator().manual_seed(11)
    Z = (torch.randn(T, F, generator=g) * 0.5).to(torch.bfloat16).cuda()
    wd = weights["w_down"].cuda().contiguous()
    ws = clada.new_workspace(layer, 1, T)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y_plain = torch.empty(T, d, dtype=torch.float32, device="cuda")
    clada.clada_prefill_down(layer, wd, Z, Y_plain, status)
    Y_split = torch.full((T + 2, d), 7.0, dtype=torch.float32, device="cuda")
    clada.clada_prefill_down(layer, wd, Z, Y_split[:T], status, ws=ws)
    Y_again = torch.empty(T, d, dtype=torch.float32, device="cuda")
    clada.clada_prefill_down(layer, wd, Z, Y_again, status, ws=ws)
    Y16 = torch.full((T + 2, d), 7.0, dtype=torch.bfloat16, device="cuda")
    clada.clada_prefill_down(layer, wd, Z, Y16[:T], status, ws=ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(Y_split[:T], Y_again) and torch.all(Y_split[T:] == 7.0) and torch.all(Y16[T:] == 7.0)
    assert torch.equal(Y16[:T], Y_split[:T].to(torch.bfloat16))
    Y_own = oracle.down_proj(_widen(Z), oracle_weights(weights)[2])
    assert rel_inf(Y_split[:T].cpu().numpy().astype(np.float64), Y_own) <= DOWN_TOL
    assert rel_inf(Y_plain.cpu().numpy().astype(np.float64), Y_own) <= DOWN_TOL
    assert not torch.equal(Y_plain, Y_split[:T]) or F <= 64      # the split really ran (another summation order)
    # the workspace's control block is left as it was: a decode on it still works
    x = wl.hidden_states(w, 0, "decode", 0, 1)[0].cuda()
    y = torch.empty(1, d, device="cuda")
    clada.clada_sparse_ffn_decode(layer, x[None], torch.ones(1, F, device="cuda"), torch.zeros(1, device="cuda"), 1, y, ws,
                                  None, None, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and bool(torch.isfinite(y).all())


@pytest.mark.parametrize("name,kw", [("c2_llama2_7b_layer", {"d_model": 256, "d_ff": 300}),
                                     ("c1_small_f32", {"d_model": 72, "d_ff": 130})])
def test_chunked_statistics_equal_whole_prompt(clada, oracle, name, kw):
    """Three prompts fed in four chunks of uneven size (a prompt may be absent from a chunk)."""
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    weights = wl.layer_weights(w, 0)
    lengths = [300, 37, 150]
    scale = wl.channel_scale(w)
    Xs = [wl.hidden_states(w, 0, "prefix", b, n, "cpu", scale) for b, n in enumerate(lengths)]
    layer = gpu_layer(weights, clada)
    cuts = [[0, 100, 130, 300, 300], [0, 37, 37, 37, 37], [0, 0, 64, 64, 150]]   # per prompt: chunk boundaries
    sumsq = torch.zeros(3, w.d_ff, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for c in range(4):
        parts = [Xs[b][cuts[b][c]:cuts[b][c + 1]] for b in range(3)]
        off = wl.seq_offsets([p.shape[0] for p in parts])
        Xc = torch.cat(parts).cuda() if off[-1] > 0 else torch.empty(8, w.d_model, dtype=w.torch_dtype, device="cuda")
        ws = clada.new_workspace(layer, 3, max(off[-1], 1))
        clada.clada_prefix_accumulate(layer, Xc, off, sumsq, ws, None, status)
    scores = torch.empty(3, w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_prefix_finish(layer, sumsq, scores)
    whole = torch.empty(3, w.d_ff, dtype=torch.float32, device="cuda")
    off_all = wl.seq_offsets(lengths)
    ws = clada.new_workspace(layer, 3, off_all[-1])
    clada.clada_prefix_scores(layer, torch.cat(Xs).cuda(), off_all, whole, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    A_or = oracle.neuron_scores(wl.to_numpy_bits(torch.cat(Xs)), off_all, *oracle_weights(weights))
    A = scores.cpu().numpy().astype(np.float64)
    tol = 2e-6 if w.dtype == "f32" else SCORE_TOL
    for b in range(3):
        assert np.max(np.abs(A[b] - A_or[b])) <= tol * np.max(A_or[b])
    # and against the one-call route: the same tile sums added in another order
    assert torch.allclose(scores, whole, rtol=2e-6, atol=0)


@pytest.mark.parametrize("T", [512, 2048])
def test_prefill_full_width_c2(clada, oracle, T):
    """The benchmark's layer at full width: sampled rows of Z and Y against the oracle.  2048 tokens run the down
    projection in 256-column tiles; 512 tokens too, given the workspace, with every tile's K range split between
    two CTAs (and in 128-column tiles, unsplit, without the workspace: both are checked)."""
    w = wl.WORKLOADS["c2_llama2_7b_layer"]
    weights = wl.layer_weights(w, 0, "cuda")
    layer = gpu_layer(weights, clada)
    X = wl.hidden_states(w, 0, "prefix", 0, T, "cuda", wl.channel_scale(w, "cuda"))
    ws = clada.new_workspace(layer, 1, T)
    sumsq = torch.zeros(1, w.d_ff, dtype=torch.float32, device="cuda")
    Z = torch.empty(T, w.d_ff, dtype=torch.bfloat16, device="cuda")
    Y = torch.empty(T, w.d_model, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    clada.clada_prefix_accumulate(layer, X, [0, T], sumsq, ws, Z, status)
    clada.clada_prefill_down(layer, weights["w_down"].contiguous(), Z, Y, status, ws=ws)
    Y_plain = torch.empty_like(Y)
    clada.clada_prefill_down(layer, weights["w_down"].contiguous(), Z, Y_plain, status)
    scores = torch.empty(1, w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_prefix_finish(layer, sumsq, scores)
    whole = torch.empty(1, w.d_ff, dtype=torch.float32, device="cuda")
    clada.clada_prefix_scores(layer, X, [0, T], whole, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(scores, whole)      # one chunk: the very same sums
    rows = [0, 127, 128, 300, T - 1]
    W_in, V_in, W_out = oracle_weights(weights)
    Xn = wl.to_numpy_bits(X[rows])
    Z_or = oracle.prefill_hidden(Xn, W_in, V_in, round_z=True)
    Zg = _widen(Z[rows])
    diff = np.abs(Zg - Z_or)
    assert np.all(diff <= _ulp(Z_or, "bf16") * 1.0001 + 2e-5 * np.max(np.abs(Z_or))) and np.mean(diff > 0) <= 0.03
    Y_own = oracle.down_proj(Zg, W_out)
    for Yt in (Y, Y_plain):
        Yg = Yt[rows].cpu().numpy().astype(np.float64)
        assert rel_inf(Yg, Y_own) <= DOWN_TOL
        assert rel_inf(Yg, oracle.down_proj(Z_or, W_out)) <= FFN_TOL
    assert torch.equal(Y, Y_plain) == (T == 2048)      # enough tiles for every SM: the workspace changes nothing


def test_new_entry_points_refuse_what_they_cannot_do(clada):
    """Host-side checks: nothing is launched, the context stays usable."""
    w32 = wl.scaled(wl.WORKLOADS["c1_small_f32"], d_model=64, d_ff=96)
    l32 = gpu_layer(wl.layer_weights(w32, 0), clada)
    ws = clada.new_workspace(l32, 1, 16)
    X = torch.zeros(16, 64, device="cuda")
    sumsq = torch.zeros(1, 96, device="cuda")
    Z32 = torch.empty(16, 96, device="cuda")
    with pytest.raises(clada.CladaError, match="support"):          # hidden activations: 16-bit layers only
        clada.clada_prefix_accumulate(l32, X, [0, 16], sumsq, ws, Z32)
    with pytest.raises(clada.CladaError, match="support"):
        clada.clada_prefill_down(l32, torch.zeros(64, 96, device="cuda"), Z32, torch.empty(16, 64, device="cuda"))
    clada.clada_prefix_accumulate(l32, X, [0, 16], sumsq, ws, None)      # statistics alone work for fp32
    wb = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=64, d_ff=100)   # d_ff % 8 != 0
    lb = gpu_layer(wl.layer_weights(wb, 0), clada)
    wsb = clada.new_workspace(lb, 1, 16)
    Xb = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    Zb = torch.empty(16, 100, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(clada.CladaError, match="shape"):
        clada.clada_prefix_accumulate(lb, Xb, [0, 16], torch.zeros(1, 100, device="cuda"), wsb, Zb)
    with pytest.raises(clada.CladaError, match="shape"):
        clada.clada_prefill_down(lb, torch.zeros(64, 100, dtype=torch.bfloat16, device="cuda"), Zb,
                                 torch.empty(16, 64, device="cuda"))
    w8 = wl.scaled(wl.WORKLOADS["c2_llama2_7b_layer"], d_model=64, d_ff=104)
    l8 = gpu_layer(wl.layer_weights(w8, 0), clada)
    ws8 = clada.new_workspace(l8, 1, 16)
    Z8 = torch.zeros(16, 104, dtype=torch.bfloat16, device="cuda")
    wd8 = torch.zeros(64, 104, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(clada.CladaError, match="workspace"):             # a workspace off its 256-byte boundary
        clada.clada_prefill_down(l8, wd8, Z8, torch.empty(16, 64, device="cuda"), ws=ws8[16:])
    with pytest.raises(clada.CladaError, match="workspace"):             # smaller than its control block
        clada.clada_prefill_down(l8, wd8, Z8, torch.empty(16, 64, device="cuda"), ws=ws8[:128])
    Y8 = torch.full((16, 64), 5.0, device="cuda")
    clada.clada_prefill_down(l8, wd8, Z8, Y8, ws=ws8[:256])               # too small to split: runs unsplit
    torch.cuda.synchronize()
    assert bool((Y8 == 0).all())
    big = torch.ones(1, 32769, device="cuda")                             # the list build holds 32768 scores per CTA
    with pytest.raises(clada.CladaError, match="support"):
        clada.clada_nested_build(big, torch.ones(1, device="cuda"), 0.8, 0.12,
                                 torch.empty(1, 32769, dtype=torch.int32, device="cuda"),
                                 torch.empty(1, 4, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
