"""Thin ctypes binding of ``libclada.so``: the same call names as ``include/clada.h``.

Argument marshalling only -- every step of the path runs in the CUDA library.  Tensors are
torch CUDA tensors (torch provides device memory and streams, nothing else); each wrapper checks
dtype / contiguity, passes raw pointers and raises ``CladaError`` on a negative return code.
There is no fallback: if the shared library is missing or cannot be loaded, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("CLADA_LIB") or os.path.join(_HERE, "libclada.so")   # CLADA_LIB: another build of the library

CLADA_F32, CLADA_BF16, CLADA_F16 = 0, 1, 2
STATUS_BAD_TOKEN, STATUS_NONFINITE_LOGIT, STATUS_TIMEOUT = 1, 2, 4

_INT_RETURNING = [
    "clada_workspace_init", "clada_down_norms", "clada_prefix_scores", "clada_refine_scores",
    "clada_select", "clada_prefix_select", "clada_tau_from_sparsity", "clada_cogload",
    "clada_adjust_threshold", "clada_cogload_adjust", "clada_sparse_ffn_decode",
    "clada_sparse_ffn_decode_static", "clada_sparse_ffn_decode_layers", "clada_selftest_bounded_waits", "clada_cett_threshold_search",
    "clada_cett_curve",
]


class CladaError(RuntimeError):
    pass


class _CLayer(ctypes.Structure):
    _fields_ = [("d_model", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("activation", ctypes.c_int32), ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p),
                ("w_down_t", ctypes.c_void_p), ("w_down_norm", ctypes.c_void_p)]


_lib = None


def load() -> ctypes.CDLL:
    """Load libclada.so (built in-tree by ``build.build()``); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise CladaError(f"{LIB_PATH} not found: build it with "
                         f"`python -m paper_2502_19078_b200.build` (there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    lp = ctypes.POINTER(_CLayer)
    L.clada_version.restype = ctypes.c_int
    L.clada_status_string.argtypes = [ctypes.c_int]
    L.clada_status_string.restype = ctypes.c_char_p
    L.clada_last_cuda_error.restype = ctypes.c_char_p
    L.clada_workspace_bytes.argtypes = [lp, i32, i64]
    L.clada_workspace_bytes.restype = sz
    L.clada_workspace_init.argtypes = [vp, sz, vp]
    L.clada_selftest_bounded_waits.argtypes = [vp, sz, ctypes.c_uint32, vp, vp, vp]
    L.clada_down_norms.argtypes = [lp, vp, vp]
    L.clada_prefix_scores.argtypes = [lp, vp, vp, i32, vp, vp, sz, vp, vp]
    L.clada_refine_scores.argtypes = [lp, vp, vp, i32, vp, vp, i32, f32, vp, vp, sz, vp, vp]
    L.clada_select.argtypes = [vp, i32, i32, vp, i64, vp, vp, vp, vp]
    L.clada_prefix_select.argtypes = [lp, vp, vp, i32, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
    L.clada_tau_from_sparsity.argtypes = [vp, i32, i32, f32, vp, vp]
    L.clada_cogload.argtypes = [vp, i32, i32, i64, i64, vp, vp, vp, vp, vp]
    L.clada_adjust_threshold.argtypes = [vp, vp, vp, f32, f32, vp, vp, i32, i32, vp, vp]
    L.clada_cogload_adjust.argtypes = [vp, i32, i32, i64, i64, vp, vp, vp, vp, f32, f32, i32, vp, vp, vp, vp, vp]
    L.clada_sparse_ffn_decode.argtypes = [lp, vp, i32, vp, vp, i64, vp, i32, vp, vp, vp, vp, sz, vp, vp]
    L.clada_sparse_ffn_decode_static.argtypes = [lp, vp, i32, vp, vp, i64, vp, i32, vp, vp, vp, vp, vp]
    L.clada_sparse_ffn_decode_layers.argtypes = [vp, i32, vp, i32, vp, vp, vp, i32, vp, sz, vp, vp]
    L.clada_stream_read_probe.argtypes = [vp, sz, vp, vp]
    L.clada_prefix_accumulate.argtypes = [lp, vp, vp, i32, vp, vp, vp, sz, vp, vp]
    L.clada_prefix_finish.argtypes = [lp, vp, i32, vp, vp]
    L.clada_prefill_down.argtypes = [lp, vp, vp, i64, vp, i32, vp, sz, vp, vp]
    L.clada_nested_build.argtypes = [vp, i32, i32, vp, i64, f32, f32, vp, vp, vp]
    L.clada_cogload_level.argtypes = [vp, i32, i32, i64, i64, vp, f32, f32, vp, vp, vp, vp, vp]
    L.clada_sparse_ffn_decode_nested.argtypes = [lp, vp, i32, vp, vp, vp, vp, i32, vp, vp, sz, vp, vp]
    L.clada_cett_workspace_bytes.argtypes = [lp, vp, i32]
    L.clada_cett_workspace_bytes.restype = sz
    L.clada_cett_threshold_search.argtypes = [lp, vp, vp, i32, f32, vp, vp, vp, vp, sz, vp, vp]
    L.clada_cett_curve.argtypes = [lp, vp, i32, i32, vp, sz, vp, vp, vp]
    for name in _INT_RETURNING:
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def _check(rc: int, what: str) -> None:
    if rc != 0:
        L = load()
        msg = L.clada_status_string(rc).decode()
        if rc == -6:
            msg += ": " + L.clada_last_cuda_error().decode()
        raise CladaError(f"{what} failed ({rc}): {msg}")


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return CLADA_F32
    if t == torch.bfloat16:
        return CLADA_BF16
    if t == torch.float16:
        return CLADA_F16
    raise CladaError(f"unsupported dtype {t}")


def _ptr(t: Optional[torch.Tensor], dtype=None, name="tensor") -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise CladaError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise CladaError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise CladaError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# clada_activation of include/clada.h
ACT_SILU_GATED, ACT_GELU_GATED, ACT_RELU = 0, 1, 2


class Layer:
    """One FFN layer in the library's neuron-major layout (keeps the tensors alive).
    ``activation`` is a clada_activation; the non-gated ReLU form takes ``w_up=None``."""

    def __init__(self, w_gate: torch.Tensor, w_up: Optional[torch.Tensor], w_down_t: torch.Tensor,
                 w_down_norm: Optional[torch.Tensor] = None, activation: int = ACT_SILU_GATED):
        d_ff, d_model = w_gate.shape
        if activation == ACT_RELU:
            if w_up is not None:
                raise CladaError("the non-gated form has no w_up")
        elif w_up is None or w_up.shape != (d_ff, d_model) or w_up.dtype != w_gate.dtype:
            raise CladaError("w_up must be [d_ff, d_model] of the weights' dtype")
        if w_down_t.shape != (d_ff, d_model):
            raise CladaError("w_gate, w_up, w_down_t must all be [d_ff, d_model]")
        if w_gate.dtype != w_down_t.dtype:
            raise CladaError("weights must share one dtype")
        self.d_model, self.d_ff = int(d_model), int(d_ff)
        self.dtype = w_gate.dtype
        self.activation = int(activation)
        self.w_gate, self.w_up, self.w_down_t = w_gate, w_up, w_down_t
        self.w_down_norm = w_down_norm
        self.c = _CLayer(self.d_model, self.d_ff, _dtype_code(self.dtype), self.activation,
                         _ptr(w_gate, name="w_gate"), _ptr(w_up, name="w_up"),
                         _ptr(w_down_t, name="w_down_t"),
                         _ptr(w_down_norm, torch.float32, "w_down_norm"))

    def set_down_norm(self, w_down_norm: torch.Tensor) -> None:
        self.w_down_norm = w_down_norm
        self.c.w_down_norm = _ptr(w_down_norm, torch.float32, "w_down_norm")

    @property
    def ref(self):
        return ctypes.byref(self.c)


def _offsets(seq_offsets: Sequence[int]):
    arr = (ctypes.c_int64 * len(seq_offsets))(*[int(v) for v in seq_offsets])
    return arr, len(seq_offsets) - 1


def _floats(vals):
    arr = (ctypes.c_float * len(vals))(*[float(v) for v in vals])
    return arr


def clada_version() -> int:
    return int(load().clada_version())


def clada_workspace_bytes(layer: Layer, B: int, T_total: int) -> int:
    n = int(load().clada_workspace_bytes(layer.ref, B, T_total))
    if n == 0:
        raise CladaError("clada_workspace_bytes: invalid arguments")
    return n


def clada_workspace_init(ws: torch.Tensor, stream=None) -> None:
    _check(load().clada_workspace_init(_ptr(ws, torch.uint8, "ws"), ws.numel(), _stream(stream)),
           "clada_workspace_init")


def new_workspace(layer: Layer, B: int, T_total: int, stream=None) -> torch.Tensor:
    """Allocate (through torch) and initialise a workspace for this layer shape."""
    ws = torch.empty(clada_workspace_bytes(layer, B, T_total), dtype=torch.uint8, device=layer.w_gate.device)
    clada_workspace_init(ws, stream)
    return ws


def clada_selftest_bounded_waits(ws, poll_limit: int, report, status=None, stream=None) -> None:
    _check(load().clada_selftest_bounded_waits(_ptr(ws, torch.uint8, "ws"), ws.numel(), int(poll_limit),
                                               _ptr(report, torch.int32, "report"), _ptr(status, torch.int32, "status"),
                                               _stream(stream)), "clada_selftest_bounded_waits")


def clada_down_norms(layer: Layer, out: torch.Tensor, stream=None) -> None:
    _check(load().clada_down_norms(layer.ref, _ptr(out, torch.float32, "out"), _stream(stream)),
           "clada_down_norms")


def clada_prefix_scores(layer: Layer, X, seq_offsets, scores, ws, status=None, stream=None) -> None:
    off, B = _offsets(seq_offsets)
    _check(load().clada_prefix_scores(layer.ref, _ptr(X, layer.dtype, "X"), ctypes.addressof(off), B,
                                      _ptr(scores, torch.float32, "scores"), _ptr(ws, torch.uint8, "ws"),
                                      ws.numel(), _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_prefix_scores")


def clada_refine_scores(layer: Layer, X, seq_offsets, tau_base, guard_mults, rel_band, scores, ws,
                        status=None, stream=None) -> None:
    off, B = _offsets(seq_offsets)
    gm = _floats(guard_mults)
    _check(load().clada_refine_scores(layer.ref, _ptr(X, layer.dtype, "X"), ctypes.addressof(off), B,
                                      _ptr(tau_base, torch.float32, "tau_base"), ctypes.addressof(gm),
                                      len(guard_mults), float(rel_band),
                                      _ptr(scores, torch.float32, "scores"), _ptr(ws, torch.uint8, "ws"),
                                      ws.numel(), _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_refine_scores")


def clada_select(scores, tau, tau_stride=1, mask=None, idx=None, count=None, stream=None) -> None:
    B, d_ff = scores.shape
    _check(load().clada_select(_ptr(scores, torch.float32, "scores"), B, d_ff, _ptr(tau, torch.float32, "tau"),
                               tau_stride, _ptr(mask, torch.uint8, "mask"), _ptr(idx, torch.int32, "idx"),
                               _ptr(count, torch.int32, "count"), _stream(stream)), "clada_select")


def clada_prefix_select(layer: Layer, X, seq_offsets, tau_base, guard_mults, scores, mask, idx, count, ws,
                        status=None, stream=None) -> None:
    off, B = _offsets(seq_offsets)
    gm, gm_ptr, n_guard = None, None, 0
    if guard_mults is not None and len(guard_mults) > 0:
        gm = _floats(guard_mults)
        gm_ptr, n_guard = ctypes.addressof(gm), len(guard_mults)
    _check(load().clada_prefix_select(layer.ref, _ptr(X, layer.dtype, "X"), ctypes.addressof(off), B,
                                      _ptr(tau_base, torch.float32, "tau_base"), gm_ptr, n_guard,
                                      _ptr(scores, torch.float32, "scores"), _ptr(mask, torch.uint8, "mask"),
                                      _ptr(idx, torch.int32, "idx"), _ptr(count, torch.int32, "count"),
                                      _ptr(ws, torch.uint8, "ws"), ws.numel(),
                                      _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_prefix_select")


def clada_tau_from_sparsity(scores, rho, tau_base, stream=None) -> None:
    B, d_ff = scores.shape
    _check(load().clada_tau_from_sparsity(_ptr(scores, torch.float32, "scores"), B, d_ff, float(rho),
                                          _ptr(tau_base, torch.float32, "tau_base"), _stream(stream)),
           "clada_tau_from_sparsity")


def _logits_args(logits):
    if not logits.is_cuda or logits.dim() != 2 or logits.stride(1) != 1:
        raise CladaError("logits must be a 2-D CUDA tensor with contiguous rows")
    B, V = logits.shape
    return logits.data_ptr(), _dtype_code(logits.dtype), B, V, logits.stride(0)


def clada_cogload(logits, token_id, surprisal, entropy, status=None, stream=None) -> None:
    _check(load().clada_cogload(*_logits_args(logits), _ptr(token_id, torch.int32, "token_id"),
                                _ptr(surprisal, torch.float32, "surprisal"),
                                _ptr(entropy, torch.float32, "entropy"),
                                _ptr(status, torch.int32, "status"), _stream(stream)), "clada_cogload")


def clada_adjust_threshold(tau_base, lam, gam, tau_s, tau_H, surprisal, entropy, tau_final, stream=None) -> None:
    B, L = tau_base.shape
    _check(load().clada_adjust_threshold(_ptr(tau_base, torch.float32, "tau_base"), _ptr(lam, torch.float32, "lambda"),
                                         _ptr(gam, torch.float32, "gamma"), float(tau_s), float(tau_H),
                                         _ptr(surprisal, torch.float32, "surprisal"),
                                         _ptr(entropy, torch.float32, "entropy"), B, L,
                                         _ptr(tau_final, torch.float32, "tau_final"), _stream(stream)),
           "clada_adjust_threshold")


def clada_cogload_adjust(logits, token_id, tau_base, lam, gam, tau_s, tau_H, surprisal, entropy, tau_final,
                         status=None, stream=None) -> None:
    L = tau_base.shape[1]
    _check(load().clada_cogload_adjust(*_logits_args(logits), _ptr(token_id, torch.int32, "token_id"),
                                       _ptr(tau_base, torch.float32, "tau_base"),
                                       _ptr(lam, torch.float32, "lambda"), _ptr(gam, torch.float32, "gamma"),
                                       float(tau_s), float(tau_H), L,
                                       _ptr(surprisal, torch.float32, "surprisal"),
                                       _ptr(entropy, torch.float32, "entropy"),
                                       _ptr(tau_final, torch.float32, "tau_final"),
                                       _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_cogload_adjust")


def clada_sparse_ffn_decode(layer: Layer, x, scores, tau_final, tau_stride, y, ws, mask_out=None, idx_out=None,
                            count_out=None, status=None, stream=None) -> None:
    """tau_final may be a view into a larger [B, L] array: pass the element for (b=0, this layer) and
    tau_stride = L."""
    B = x.shape[0]
    if not tau_final.is_cuda or tau_final.dtype != torch.float32:
        raise CladaError("tau_final must be a CUDA float32 tensor")
    _check(load().clada_sparse_ffn_decode(layer.ref, _ptr(x, layer.dtype, "x"), B,
                                          _ptr(scores, torch.float32, "scores"), tau_final.data_ptr(),
                                          int(tau_stride), _ptr(y, name="y"), _dtype_code(y.dtype),
                                          _ptr(mask_out, torch.uint8, "mask_out"),
                                          _ptr(idx_out, torch.int32, "idx_out"),
                                          _ptr(count_out, torch.int32, "count_out"),
                                          _ptr(ws, torch.uint8, "ws"), ws.numel(),
                                          _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_sparse_ffn_decode")


def clada_sparse_ffn_decode_static(layer: Layer, x, scores, tau_final, tau_stride, y, mask_out=None, idx_out=None,
                                   count_out=None, status=None, stream=None) -> None:
    """clada_sparse_ffn_decode without a workspace argument: the scratch is a fixed array inside the
    library, for callers that are not allowed to allocate device memory.  Calls share that array, so
    do not let two of them overlap on the GPU."""
    B = x.shape[0]
    if not tau_final.is_cuda or tau_final.dtype != torch.float32:
        raise CladaError("tau_final must be a CUDA float32 tensor")
    _check(load().clada_sparse_ffn_decode_static(layer.ref, _ptr(x, layer.dtype, "x"), B,
                                                 _ptr(scores, torch.float32, "scores"), tau_final.data_ptr(),
                                                 int(tau_stride), _ptr(y, name="y"), _dtype_code(y.dtype),
                                                 _ptr(mask_out, torch.uint8, "mask_out"),
                                                 _ptr(idx_out, torch.int32, "idx_out"),
                                                 _ptr(count_out, torch.int32, "count_out"),
                                                 _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_sparse_ffn_decode_static")


class LayerStack:
    """L layers of one shape as the contiguous host array clada_sparse_ffn_decode_layers takes."""

    def __init__(self, layers):
        self.layers = list(layers)
        self.array = (_CLayer * len(self.layers))(*[l.c for l in self.layers])

    def __len__(self):
        return len(self.layers)


def clada_sparse_ffn_decode_layers(stack: LayerStack, x, scores, tau_final, y, ws, status=None, stream=None) -> None:
    """x [L, B, d], scores [L, B, F], tau_final [B, L], y [L, B, d]."""
    L, B = x.shape[0], x.shape[1]
    if L != len(stack):
        raise CladaError("x must have one [B, d_model] slab per layer")
    _check(load().clada_sparse_ffn_decode_layers(ctypes.addressof(stack.array), L, _ptr(x, stack.layers[0].dtype, "x"), B,
                                                 _ptr(scores, torch.float32, "scores"),
                                                 _ptr(tau_final, torch.float32, "tau_final"), _ptr(y, name="y"),
                                                 _dtype_code(y.dtype), _ptr(ws, torch.uint8, "ws"), ws.numel(),
                                                 _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_sparse_ffn_decode_layers")


def clada_cett_workspace_bytes(layer: Layer, seq_offsets) -> int:
    off, B = _offsets(seq_offsets)
    n = int(load().clada_cett_workspace_bytes(layer.ref, ctypes.addressof(off), B))
    if n == 0:
        raise CladaError("clada_cett_workspace_bytes: invalid arguments")
    return n


def clada_cett_threshold_search(layer: Layer, X, seq_offsets, bound, tau_base, mean_cett, scores, ws, status=None,
                                stream=None) -> None:
    off, B = _offsets(seq_offsets)
    _check(load().clada_cett_threshold_search(layer.ref, _ptr(X, layer.dtype, "X"), ctypes.addressof(off), B,
                                              float(bound), _ptr(tau_base, torch.float32, "tau_base"),
                                              _ptr(mean_cett, torch.float32, "mean_cett"),
                                              _ptr(scores, torch.float32, "scores"), _ptr(ws, torch.uint8, "ws"),
                                              ws.numel(), _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_cett_threshold_search")


def clada_cett_curve(layer: Layer, seq_offsets, sample, ws, cum_out, order_out=None, stream=None) -> None:
    off, B = _offsets(seq_offsets)
    _check(load().clada_cett_curve(layer.ref, ctypes.addressof(off), B, int(sample), _ptr(ws, torch.uint8, "ws"),
                                   ws.numel(), _ptr(cum_out, torch.float64, "cum_out"),
                                   _ptr(order_out, torch.int32, "order_out"), _stream(stream)), "clada_cett_curve")


def clada_nested_build(scores, tau_base, lam, gam, order, counts, tau_stride=1, stream=None) -> None:
    """scores [B, F] fp32, tau_base (sequence b at b * tau_stride) -> order [B, F] int32, counts [B, 4] int32."""
    B, F = scores.shape
    _check(load().clada_nested_build(_ptr(scores, torch.float32, "scores"), B, F,
                                     _ptr(tau_base, torch.float32, "tau_base"), int(tau_stride), float(lam),
                                     float(gam), _ptr(order, torch.int32, "order"),
                                     _ptr(counts, torch.int32, "counts"), _stream(stream)), "clada_nested_build")


def clada_cogload_level(logits, token_id, tau_s, tau_H, surprisal, entropy, level, status=None, stream=None) -> None:
    _check(load().clada_cogload_level(*_logits_args(logits), _ptr(token_id, torch.int32, "token_id"),
                                      float(tau_s), float(tau_H), _ptr(surprisal, torch.float32, "surprisal"),
                                      _ptr(entropy, torch.float32, "entropy"), _ptr(level, torch.int32, "level"),
                                      _ptr(status, torch.int32, "status"), _stream(stream)), "clada_cogload_level")


def clada_sparse_ffn_decode_nested(layer: Layer, x, order, counts, level, y, ws, count=None, status=None,
                                   stream=None) -> None:
    """x [B, d], order [B, F], counts [B, 4], level [B] -> y [B, d] over order[b][:counts[b][level[b]]]."""
    B = x.shape[0] if x.dim() == 2 else 1
    _check(load().clada_sparse_ffn_decode_nested(layer.ref, _ptr(x, layer.dtype, "x"), B,
                                                 _ptr(order, torch.int32, "order"),
                                                 _ptr(counts, torch.int32, "counts"),
                                                 _ptr(level, torch.int32, "level"), _ptr(y, name="y"),
                                                 _dtype_code(y.dtype), _ptr(count, torch.int32, "count"),
                                                 _ptr(ws, torch.uint8, "ws"), ws.numel(),
                                                 _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_sparse_ffn_decode_nested")


def clada_prefix_accumulate(layer: Layer, X, seq_offsets, sumsq, ws, Z=None, status=None, stream=None) -> None:
    """One chunk of prompts: sumsq [B, F] += sum_t z^2; Z [T_chunk, F] (layer dtype) receives the hidden activations."""
    off, B = _offsets(seq_offsets)
    _check(load().clada_prefix_accumulate(layer.ref, _ptr(X, layer.dtype, "X"), ctypes.addressof(off), B,
                                          _ptr(sumsq, torch.float32, "sumsq"), _ptr(Z, layer.dtype, "Z"),
                                          _ptr(ws, torch.uint8, "ws"), ws.numel(),
                                          _ptr(status, torch.int32, "status"), _stream(stream)),
           "clada_prefix_accumulate")


def clada_prefix_finish(layer: Layer, sumsq, scores, stream=None) -> None:
    _check(load().clada_prefix_finish(layer.ref, _ptr(sumsq, torch.float32, "sumsq"), sumsq.shape[0],
                                      _ptr(scores, torch.float32, "scores"), _stream(stream)), "clada_prefix_finish")


def clada_prefill_down(layer: Layer, w_down, Z, Y, status=None, stream=None, ws=None) -> None:
    """Y [T, d_model] = Z [T, d_ff] w_down^T, w_down [d_model, d_ff] in the paper's layout; ws: optional workspace."""
    _check(load().clada_prefill_down(layer.ref, _ptr(w_down, layer.dtype, "w_down"), _ptr(Z, layer.dtype, "Z"),
                                     Z.shape[0], _ptr(Y, name="Y"), _dtype_code(Y.dtype),
                                     _ptr(ws, torch.uint8, "ws"), ws.numel() if ws is not None else 0,
                                     _ptr(status, torch.int32, "status"), _stream(stream)), "clada_prefill_down")


def clada_stream_read_probe(buf: torch.Tensor, sink: torch.Tensor, stream=None) -> None:
    """Read `buf` once with streaming 16-byte loads (a measuring aid); `sink` is one int32 on the device."""
    _check(load().clada_stream_read_probe(_ptr(buf, name="buf"), buf.numel() * buf.element_size(),
                                          _ptr(sink, torch.int32, "sink"), _stream(stream)),
           "clada_stream_read_probe")
