"""Shared helpers of the GPU parity tests: move one seeded draw to both sides, compare masks."""
from __future__ import annotations

import numpy as np
import torch

from paper_2502_19078_b200 import workloads as wl


def gpu_layer(weights, binding, dev="cuda", activation=0):
    """binding.Layer (neuron-major, on the GPU) from a workloads.layer_weights() draw, norms included.
    The non-gated form (activation 2) leaves the drawn w_up out."""
    wg = weights["w_gate"].to(dev).contiguous()
    wu = None if activation == 2 else weights["w_up"].to(dev).contiguous()
    wdt = weights["w_down"].to(dev).t().contiguous()      # row j = column j of W_out
    layer = binding.Layer(wg, wu, wdt, activation=activation)
    norms = torch.empty(layer.d_ff, dtype=torch.float32, device=dev)
    binding.clada_down_norms(layer, norms)
    layer.set_down_norm(norms)
    return layer


def oracle_weights(weights, activation=0):
    """(W_in, V_in, W_out) numpy arrays in the paper's layout for the oracle (V_in None when non-gated)."""
    return (wl.to_numpy_bits(weights["w_gate"]),
            None if activation == 2 else wl.to_numpy_bits(weights["w_up"]),
            wl.to_numpy_bits(weights["w_down"]))


def compare_masks(mask_gpu: np.ndarray, scores_oracle: np.ndarray, tau: float, rel=1e-6):
    """Masks must agree bit for bit except where the oracle's score lies within `rel` of tau.
    Returns (n_excused, n_mismatched)."""
    mask_or = scores_oracle >= tau
    diff = np.nonzero(mask_or != mask_gpu.astype(bool))[0]
    if diff.size == 0:
        return 0, 0
    near = np.abs(scores_oracle[diff] - tau) <= rel * abs(tau)
    return int(near.sum()), int((~near).sum())


def rel_inf(a: np.ndarray, ref: np.ndarray) -> float:
    denom = float(np.max(np.abs(ref)))
    if denom == 0.0:
        return float(np.max(np.abs(a)))
    return float(np.max(np.abs(a.astype(np.float64) - ref)) / denom)
