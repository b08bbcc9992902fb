"""ctypes front end of the CLADA CPU oracle (TEST INFRASTRUCTURE, not the product).

Loads ``libclada_oracle.so`` built from ``clada_oracle.c`` in this folder (``build()``
compiles it with gcc).  Arrays are numpy; bf16 tensors travel as uint16 bit patterns.
Nothing here imports the CUDA package, and the CUDA package never imports this.
Weight layout is the paper's: W_in, V_in are [d_ff, d_model]; W_out is [d_model, d_ff].
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "clada_oracle.c")
_LIB = os.path.join(_HERE, "libclada_oracle.so")

F32, BF16, F16 = 0, 1, 2
# FFN forms (Section 4.1 model families): z = silu(g)*u, z = gelu_tanh(g)*u, z = relu(g) without V_in
SILU_GATED, GELU_GATED, RELU = 0, 1, 2
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP for the row loops, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        vp, i32, i64, dbl, f32 = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64,
                                  ctypes.c_double, ctypes.c_float)
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_widen.argtypes = [i32, vp, i64, vp]
        L.oracle_widen.restype = None
        L.oracle_neuron_scores.argtypes = [i32, vp, vp, i32, i32, i32, vp, vp, vp, vp, i32]
        L.oracle_neuron_scores.restype = None
        L.oracle_neuron_scores_literal.argtypes = [i32, vp, i32, i32, i32, vp, vp, vp, vp, i32]
        L.oracle_neuron_scores_literal.restype = None
        L.oracle_select.argtypes = [vp, i32, dbl, vp, vp]
        L.oracle_select.restype = ctypes.c_int
        L.oracle_cogload.argtypes = [i32, vp, i64, i64, vp, vp]
        L.oracle_cogload.restype = ctypes.c_int
        L.oracle_adjust_threshold.argtypes = [vp, vp, vp, f32, f32, vp, vp, i32, i32, vp]
        L.oracle_adjust_threshold.restype = None
        L.oracle_sparse_ffn.argtypes = [i32, vp, i32, i32, vp, vp, vp, vp, dbl, vp, vp, i32]
        L.oracle_sparse_ffn.restype = ctypes.c_int
        L.oracle_dense_ffn.argtypes = [i32, vp, i32, i32, vp, vp, vp, vp, i32]
        L.oracle_dense_ffn.restype = None
        L.oracle_cett_curve.argtypes = [i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, i32]
        L.oracle_cett_curve.restype = None
        L.oracle_threshold_search.argtypes = [vp, vp, i32, i32, dbl, vp]
        L.oracle_threshold_search.restype = dbl
        L.oracle_round_storage.argtypes = [i32, dbl]
        L.oracle_round_storage.restype = dbl
        L.oracle_prefill_hidden.argtypes = [i32, vp, i32, i32, i32, vp, vp, i32, i32, vp]
        L.oracle_prefill_hidden.restype = None
        L.oracle_down_proj.argtypes = [i32, vp, i32, i32, i32, vp, vp]
        L.oracle_down_proj.restype = None
        L.oracle_nested_lists.argtypes = [vp, i32, vp, i32, vp, vp]
        L.oracle_nested_lists.restype = None
        L.oracle_load_level.argtypes = [dbl, dbl, dbl, dbl]
        L.oracle_load_level.restype = ctypes.c_int
        L.oracle_tau_from_sparsity.argtypes = [vp, i32, dbl]
        L.oracle_tau_from_sparsity.restype = f32
        _lib = L
    return _lib


def widen(a: np.ndarray) -> np.ndarray:
    """The oracle's own element widening to float64 (for the pin that checks every 16-bit pattern)."""
    a = np.ascontiguousarray(a)
    out = np.empty(a.size, dtype=np.float64)
    lib().oracle_widen(_dt(a), _p(a), a.size, _p(out))
    return out.reshape(a.shape)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _dt(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float16:
        return F16
    raise TypeError(f"oracle takes float32, float16 or uint16 (bf16 bits) arrays, got {a.dtype}")


def _c(a: np.ndarray, dtype=None) -> np.ndarray:
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _check_weights(X, W_in, V_in, W_out, act=SILU_GATED):
    d_ff, d_model = W_in.shape
    if act == RELU:
        assert V_in is None, "the non-gated form has no V_in"
    else:
        assert V_in.shape == (d_ff, d_model), "V_in must be [d_ff, d_model]"
        assert V_in.dtype == W_in.dtype
    assert W_out.shape == (d_model, d_ff), "W_out must be [d_model, d_ff] (neuron j = column j)"
    assert X.shape[-1] == d_model
    assert X.dtype == W_in.dtype == W_out.dtype
    return d_model, d_ff


def _pv(V_in):
    return None if V_in is None else _p(V_in)


def neuron_scores(X, seq_offsets, W_in, V_in, W_out, act=SILU_GATED) -> np.ndarray:
    """A[b, j] of Eq. neuron_activation for each prefix b = rows seq_offsets[b]:seq_offsets[b+1] of X."""
    X, W_in, W_out = _c(X), _c(W_in), _c(W_out)
    V_in = None if V_in is None else _c(V_in)
    d_model, d_ff = _check_weights(X, W_in, V_in, W_out, act)
    off = _c(np.asarray(seq_offsets), np.int64)
    B = off.size - 1
    assert off[0] >= 0 and off[-1] <= X.shape[0] and np.all(np.diff(off) >= 0)
    out = np.empty((B, d_ff), dtype=np.float64)
    lib().oracle_neuron_scores(_dt(X), _p(X), _p(off), B, d_model, d_ff,
                               _p(W_in), _pv(V_in), _p(W_out), _p(out), int(act))
    return out


def neuron_scores_literal(X, W_in, V_in, W_out, act=SILU_GATED) -> np.ndarray:
    """Same quantity for one prefix X [T, d_model], by the Frobenius norm of the explicit T x d_model matrix."""
    X, W_in, W_out = _c(X), _c(W_in), _c(W_out)
    V_in = None if V_in is None else _c(V_in)
    d_model, d_ff = _check_weights(X, W_in, V_in, W_out, act)
    out = np.empty(d_ff, dtype=np.float64)
    lib().oracle_neuron_scores_literal(_dt(X), _p(X), X.shape[0], d_model, d_ff,
                                       _p(W_in), _pv(V_in), _p(W_out), _p(out), int(act))
    return out


def select(scores, tau):
    """(mask u8 [d_ff], idx int32 [count] ascending, count) with neuron j kept iff scores[j] >= tau."""
    scores = _c(scores, np.float64)
    d_ff = scores.size
    mask = np.empty(d_ff, dtype=np.uint8)
    idx = np.empty(d_ff, dtype=np.int32)
    count = lib().oracle_select(_p(scores), d_ff, float(tau), _p(mask), _p(idx))
    return mask, idx[:count].copy(), int(count)


def cogload(logits, token_id):
    """(surprisal, entropy) in nats of softmax(logits) for one vocabulary row; token out of range -> s = nan."""
    logits = _c(logits)
    assert logits.ndim == 1
    s = ctypes.c_double()
    h = ctypes.c_double()
    lib().oracle_cogload(_dt(logits), _p(logits), logits.size, int(token_id),
                         ctypes.byref(s), ctypes.byref(h))
    return s.value, h.value


def adjust_threshold(tau_base, lam, gam, tau_s, tau_H, surprisal, entropy) -> np.ndarray:
    """tau_final [B, L] fp32 of Eq. final_threshold."""
    tau_base = _c(tau_base, np.float32)
    B, L = tau_base.shape
    lam, gam = _c(lam, np.float32), _c(gam, np.float32)
    s, h = _c(surprisal, np.float64), _c(entropy, np.float64)
    assert lam.size == L and gam.size == L and s.size == B and h.size == B
    out = np.empty((B, L), dtype=np.float32)
    lib().oracle_adjust_threshold(_p(tau_base), _p(lam), _p(gam), float(np.float32(tau_s)), float(np.float32(tau_H)),
                                  _p(s), _p(h), B, L, _p(out))
    return out


def sparse_ffn(x, W_in, V_in, W_out, scores, tau, act=SILU_GATED):
    """(y [d_model] float64, mask u8 [d_ff], count) of the masked gated FFN for one token x."""
    x, W_in, W_out = _c(x), _c(W_in), _c(W_out)
    V_in = None if V_in is None else _c(V_in)
    d_model, d_ff = _check_weights(x, W_in, V_in, W_out, act)
    scores = _c(scores, np.float64)
    assert scores.size == d_ff and x.size == d_model
    y = np.empty(d_model, dtype=np.float64)
    mask = np.empty(d_ff, dtype=np.uint8)
    count = lib().oracle_sparse_ffn(_dt(x), _p(x), d_model, d_ff, _p(W_in), _pv(V_in), _p(W_out),
                                    _p(scores), float(tau), _p(y), _p(mask), int(act))
    return y, mask, int(count)


def dense_ffn(x, W_in, V_in, W_out, act=SILU_GATED) -> np.ndarray:
    x, W_in, W_out = _c(x), _c(W_in), _c(W_out)
    V_in = None if V_in is None else _c(V_in)
    d_model, d_ff = _check_weights(x, W_in, V_in, W_out, act)
    y = np.empty(d_model, dtype=np.float64)
    lib().oracle_dense_ffn(_dt(x), _p(x), d_model, d_ff, _p(W_in), _pv(V_in), _p(W_out), _p(y), int(act))
    return y


def tau_from_sparsity(scores_f32, rho) -> np.float32:
    """Harness helper: fp32 midpoint threshold that cuts floor(rho*F + 0.5) neurons of an fp32 score vector."""
    s = _c(scores_f32, np.float32)
    return np.float32(lib().oracle_tau_from_sparsity(_p(s), s.size, float(rho)))


def cett_curve(X, W_in, V_in, W_out, act=SILU_GATED):
    """For one validation sample X [T, d_model]: (scores [d_ff], order int32 [d_ff] ascending by score,
    cett [d_ff + 1]) with cett[k] = CETT of Eq. base_threshold when the k lowest-scored neurons are cut."""
    X, W_in, W_out = _c(X), _c(W_in), _c(W_out)
    V_in = None if V_in is None else _c(V_in)
    d_model, d_ff = _check_weights(X, W_in, V_in, W_out, act)
    scores = np.empty(d_ff, dtype=np.float64)
    order = np.empty(d_ff, dtype=np.int32)
    cett = np.empty(d_ff + 1, dtype=np.float64)
    lib().oracle_cett_curve(_dt(X), _p(X), X.shape[0], d_model, d_ff, _p(W_in), _pv(V_in), _p(W_out),
                            _p(scores), _p(order), _p(cett), int(act))
    return scores, order, cett


def threshold_search(scores, cett, bound=0.2):
    """(tau_base, mean CETT at tau_base): the largest score value eps over all samples with
    mean_x CETT(x; eps) <= bound (Eq. base_threshold).  scores [B, d_ff], cett [B, d_ff + 1]."""
    scores, cett = _c(scores, np.float64), _c(cett, np.float64)
    B, d_ff = scores.shape
    assert cett.shape == (B, d_ff + 1)
    mean = ctypes.c_double()
    tau = lib().oracle_threshold_search(_p(scores), _p(cett), B, d_ff, float(bound), ctypes.byref(mean))
    return float(tau), mean.value


def nested_lists(scores, taus):
    """(order int32 [d_ff], counts int32 [len(taus)]): neurons by descending score (ties by ascending index) and,
    per threshold, how many of them satisfy A_j >= tau -- the kept set at level k is order[:counts[k]]."""
    scores, taus = _c(scores, np.float64), _c(taus, np.float64)
    order = np.empty(scores.size, dtype=np.int32)
    counts = np.empty(taus.size, dtype=np.int32)
    lib().oracle_nested_lists(_p(scores), scores.size, _p(taus), taus.size, _p(order), _p(counts))
    return order, counts


def load_level(surprisal, entropy, tau_s, tau_H) -> int:
    """I(s > tau_s) + 2 I(H > tau_H): the index of the threshold Eq. final_threshold yields."""
    return int(lib().oracle_load_level(float(surprisal), float(entropy), float(np.float32(tau_s)),
                                       float(np.float32(tau_H))))


def round_storage(dtype_code: int, v: float) -> float:
    """v rounded to fp32 and then to the storage type (F32 / BF16 / F16), both to nearest even."""
    return float(lib().oracle_round_storage(int(dtype_code), float(v)))


def prefill_hidden(X, W_in, V_in, act=SILU_GATED, round_z=True) -> np.ndarray:
    """Z [T, d_ff] float64: every neuron's value for every prompt token, rounded to the storage type of X
    (as half-precision models keep it between the two projections) unless round_z is False."""
    X, W_in = _c(X), _c(W_in)
    V_in = None if V_in is None else _c(V_in)
    d_ff, d_model = W_in.shape
    assert X.shape[1] == d_model and X.dtype == W_in.dtype
    Z = np.empty((X.shape[0], d_ff), dtype=np.float64)
    lib().oracle_prefill_hidden(_dt(X), _p(X), X.shape[0], d_model, d_ff, _p(W_in), _pv(V_in), int(act),
                                1 if round_z else 0, _p(Z))
    return Z


def down_proj(Z, W_out) -> np.ndarray:
    """Y [T, d_model] float64 = Z W_out^T for hidden activations Z [T, d_ff] (float64) and W_out [d_model, d_ff]."""
    Z, W_out = _c(Z, np.float64), _c(W_out)
    d_model, d_ff = W_out.shape
    assert Z.shape[1] == d_ff
    Y = np.empty((Z.shape[0], d_model), dtype=np.float64)
    lib().oracle_down_proj(_dt(W_out), _p(Z), Z.shape[0], d_model, d_ff, _p(W_out), _p(Y))
    return Y
