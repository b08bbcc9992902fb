"""Seeded synthetic inputs for the CLADA sparse-FFN path.

This module only DRAWS inputs (weights, hidden states, vocabulary logits, chosen tokens,
prefix lengths) and fixes the workload shapes.  It holds none of the method's arithmetic:
no softmax, no SiLU, no thresholds.  Both the CUDA library's tests/benchmark and the CPU
oracle's tests take their inputs from here, so that the two sides see the same bits.

Shapes follow the FFN dimensions of the models the paper evaluates (LLaMA-2-7B 4096x11008,
LLaMA-3-8B 4096x14336, a 13B shape 5120x13824, OPT-2.7B 2560x10240, Gemma-2B 2048x16384; Section 4.1) and its prompt / generation
lengths (Section 4.2, long-context table).  The paper's trained weights and datasets are
replaced by these draws:

* weights  ~ N(0, 0.02^2), cast to the workload dtype; W_out is produced in the paper's
  [d_model, d_ff] layout.
* hidden states x = g * c, g ~ N(0,1) iid, c in R^d one lognormal(0, 0.5) vector per
  workload shared by all tokens, sequences and layers.
* logits per decode step, one recipe per workload (Gaussian, Gaussian + planted peak,
  temperature mixture).
* chosen token: the arg-max logit on even steps, a seeded uniform id on odd steps.

A tensor is identified by (workload, layer, name, sequence); its seed is a CRC of that
tuple, so any slice can be regenerated alone.  Draws on "cpu" and on "cuda" differ (two RNG
implementations): a test picks one device, draws there, and copies to the other side.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, List, Tuple

import torch

BASE_SEED = 0


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    d_model: int
    d_ff: int
    dtype: str               # "f32" | "bf16" | "f16": weights and hidden states
    n_layers: int
    batch: int
    prefix_len: Tuple[int, int]   # (lo, hi): every prefix has lo tokens if lo == hi, else U{lo..hi}
    n_decode: int
    vocab: int
    logit_recipe: str        # "gauss2" | "gauss3_peak" | "temp_mix" | "gauss3"
    sparsities: Tuple[float, ...]
    activation: int = 0      # FFN form: 0 SiLU-gated, 1 GELU-gated, 2 ReLU without a gate projection

    @property
    def torch_dtype(self) -> torch.dtype:
        return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def k_cut(self, rho: float) -> int:
        """Neurons cut at baseline sparsity rho."""
        return int(rho * self.d_ff + 0.5)


WORKLOADS: Dict[str, Workload] = {
    w.name: w for w in [
        Workload("c1_small_f32", 512, 1376, "f32", 1, 1, (64, 64), 16, 4096, "gauss2", (0.40,)),
        Workload("c2_llama2_7b_layer", 4096, 11008, "bf16", 1, 1, (512, 512), 128, 32000,
                 "gauss3_peak", (0.40, 0.50)),
        Workload("c3_llama2_7b_stack", 4096, 11008, "bf16", 32, 1, (2048, 2048), 256, 32000,
                 "temp_mix", (0.40,)),
        Workload("c4_llama3_8b_b8", 4096, 14336, "bf16", 32, 8, (1024, 1024), 256, 128256,
                 "gauss3", (0.40,)),
        Workload("c5_13b_b16", 5120, 13824, "bf16", 40, 16, (256, 4096), 512, 32000,
                 "gauss3", (0.30, 0.40, 0.50, 0.60)),
        # the other FFN forms among the evaluated families: OPT-2.7B (ReLU, no gate) and Gemma-2B (GELU-gated)
        Workload("v1_opt_2p7b_layer", 2560, 10240, "bf16", 1, 1, (512, 512), 128, 50272, "gauss3_peak",
                 (0.40, 0.50), activation=2),
        Workload("v2_gemma_2b_layer", 2048, 16384, "bf16", 1, 1, (512, 512), 128, 256000, "gauss3_peak",
                 (0.40, 0.50), activation=1),
    ]
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (tests shrink sizes this way)."""
    return dataclasses.replace(w, **kw)


def _seed(w: Workload, layer: int, name: str, seq: int = 0) -> int:
    key = f"{BASE_SEED}/{w.name}/{layer}/{name}/{seq}".encode()
    return zlib.crc32(key) & 0x7FFFFFFF


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn(shape, device, seed) -> torch.Tensor:
    return torch.randn(shape, generator=_gen(device, seed), device=device, dtype=torch.float32)


def channel_scale(w: Workload, device="cpu") -> torch.Tensor:
    """c in R^d, lognormal(0, 0.5), one per workload."""
    return torch.exp(0.5 * _randn((w.d_model,), device, _seed(w, -1, "channel_scale")))


def layer_weights(w: Workload, layer: int, device="cpu") -> Dict[str, torch.Tensor]:
    """W_in (gate) [F,d], V_in (up) [F,d], W_out (down) [d,F]: N(0, 0.02^2) in the workload dtype."""
    out = {}
    for name, shape in (("w_gate", (w.d_ff, w.d_model)), ("w_up", (w.d_ff, w.d_model)),
                        ("w_down", (w.d_model, w.d_ff))):
        t = _randn(shape, device, _seed(w, layer, name))
        out[name] = (t * 0.02).to(w.torch_dtype)
    return out


def prefix_lengths(w: Workload) -> List[int]:
    lo, hi = w.prefix_len
    if lo == hi:
        return [lo] * w.batch
    g = _gen("cpu", _seed(w, -1, "prefix_lengths"))
    return [int(v) for v in torch.randint(lo, hi + 1, (w.batch,), generator=g)]


def seq_offsets(lengths: List[int]) -> List[int]:
    off = [0]
    for n in lengths:
        off.append(off[-1] + int(n))
    return off


def hidden_states(w: Workload, layer: int, kind: str, seq: int, n: int, device="cpu",
                  scale: torch.Tensor | None = None) -> torch.Tensor:
    """[n, d] hidden states of one sequence at one layer; kind = "prefix" | "decode"."""
    if scale is None:
        scale = channel_scale(w, device)
    g = _randn((n, w.d_model), device, _seed(w, layer, kind, seq))
    return (g * scale).to(w.torch_dtype)


def decode_logits(w: Workload, seq: int, n: int | None = None, device="cpu") -> torch.Tensor:
    """[n, V] fp32 vocabulary logits of the steps BEFORE each decode step (step t reads row t)."""
    n = w.n_decode if n is None else n
    V = w.vocab
    r = w.logit_recipe
    seed = _seed(w, -1, "logits", seq)
    if r == "gauss2":
        return 2.0 * _randn((n, V), device, seed)
    if r == "gauss3":
        return 3.0 * _randn((n, V), device, seed)
    if r == "gauss3_peak":
        l = 3.0 * _randn((n, V), device, seed)
        g = _gen("cpu", seed + 1)
        where = torch.randint(0, V, (n,), generator=g)
        height = 6.0 + 8.0 * torch.rand((n,), generator=g)
        rows = torch.arange(n, device=device)
        l[rows, where.to(device)] += height.to(device)
        return l
    if r == "temp_mix":
        l = 3.0 * _randn((n, V), device, seed)
        g = _gen("cpu", seed + 1)
        peaked = torch.rand((n,), generator=g) < 0.5
        temp = torch.where(peaked, torch.tensor(0.5), torch.tensor(2.0))
        return l / temp.to(device)[:, None]
    raise ValueError(r)


def chosen_tokens(w: Workload, logits: torch.Tensor, seq: int) -> torch.Tensor:
    """int32 [n]: the arg-max id on even steps, a seeded uniform id on odd steps."""
    n, V = logits.shape
    g = _gen("cpu", _seed(w, -1, "tokens", seq))
    uni = torch.randint(0, V, (n,), generator=g).to(logits.device)
    top = torch.argmax(logits, dim=1)
    even = (torch.arange(n, device=logits.device) % 2) == 0
    return torch.where(even, top, uni).to(torch.int32)


def universal_threshold(values, margin: float = 1e-3) -> float:
    """A cut-off for the 'universal' tau_s / tau_H the paper leaves unspecified: the midpoint of the two
    middle order statistics of the workload's own per-step values, moved up past the next gaps until no
    value lies within `margin` of it (so a rounding difference cannot flip an indicator)."""
    v = sorted(float(a) for a in values)
    n = len(v)
    if n == 0:
        return 0.0
    if n == 1:
        return v[0] + 1.0
    for k in range(n // 2, n):
        lo, hi = v[k - 1], v[k]
        if hi - lo > 2.0 * margin:
            return 0.5 * (lo + hi)
    return v[-1] + 1.0


def to_numpy_bits(t: torch.Tensor):
    """numpy view the oracle takes: float32 and float16 as is, bfloat16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
