#!/usr/bin/env python
"""Benchmark of the CLADA sparse-FFN hot path on the Llama-2-7B-shaped layer workload.

One step = one pass of the whole path over one batch of synthetic input:
    prefill statistics of the 512-token prompt (once), then for each baseline sparsity (40 %, 50 %):
    guard-band refinement + baseline selection, then 128 decode tokens, each
    cogload+threshold adjustment (one launch) and the sparse gated FFN (one launch).
The layer exists in several identical copies at different addresses and decode step t reads copy
t mod n, so that no step can be served from L2 (one copy's kept rows are 135-162 MB, L2 is 126 MB).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-graph] [--workload NAME] [--no-info]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
Beside the step's throughput the line carries the FFN kernels timed alone (the per-layer launch the step uses, and
the persistent launch that takes a whole stack of layers), each as the median of several samples taken while the
clocks are being recorded, and -- unless --no-info -- the same figures on the other workloads' layers.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2502_19078_b200 import sharding  # noqa: E402
from paper_2502_19078_b200 import workloads as wl  # noqa: E402

WORKLOAD = "c2_llama2_7b_layer"
METRIC = "sparse_ffn_decode_tokens_per_s"
LAMBDA, GAMMA = 0.80, 0.12
N_COPIES = 4
STACK_PASSES = 32      # layer passes per persistent launch in the single-layer workloads' stack measurement
PROFILES = os.path.join(ROOT, "profiles")
CSRC = os.path.join(ROOT, "paper_2502_19078_b200", "csrc")
# sources a kernel's code comes from: the DRAM traffic on record for it counts only while these are unchanged
from paper_2502_19078_b200.ncu_summary import KERNEL_SOURCES, sources_hash  # noqa: E402  (one list for both sides)


def recorded_traffic(kernel: str, workload: str):
    """DRAM read + write bytes per launch (or per layer pass) of `kernel` from the ncu capture on record under
    profiles/ (written by paper_2502_19078_b200.ncu_summary), or None when there is no record for this workload
    or the kernel's sources have changed since the counters were taken."""
    for name in (f"traffic_{kernel}_{workload}.txt", f"traffic_{kernel}.txt"):
        try:
            rec = {}
            with open(os.path.join(PROFILES, name)) as f:
                for line in f:
                    if ":" in line and not line.startswith("#"):
                        k, v = line.split(":", 1)
                        rec[k.strip()] = v.strip()
            if rec.get("workload") == workload and rec.get("sources_sha256") == sources_hash(kernel):
                return float(rec["dram_bytes_per_unit"])
        except Exception:
            pass
    return None


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi sampling of SM clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [c.strip() for c in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------

class Job:
    """Device-resident state of one workload instance and the launch sequence of one step."""

    def __init__(self, clada, w, dev, rank: int):
        self.clada, self.w, self.dev = clada, w, dev
        T = w.prefix_len[0]
        self.T, self.N = T, w.n_decode
        weights = wl.layer_weights(w, 0, dev)
        wdt = weights["w_down"].t().contiguous()
        del weights["w_down"]
        self.layers = []
        for c in range(N_COPIES):
            gated = w.activation != clada.ACT_RELU
            wu = weights["w_up"] if gated else None
            if c == 0:
                lay = clada.Layer(weights["w_gate"], wu, wdt, activation=w.activation)
            else:
                lay = clada.Layer(weights["w_gate"].clone(), wu.clone() if gated else None, wdt.clone(),
                                  activation=w.activation)
            self.layers.append(lay)
        norms = torch.empty(w.d_ff, dtype=torch.float32, device=dev)
        clada.clada_down_norms(self.layers[0], norms)
        for lay in self.layers:
            lay.set_down_norm(norms)
        scale = wl.channel_scale(w, dev)
        # a rank's sequence differs from the other ranks' (independent jobs, no exchange)
        self.X = wl.hidden_states(w, 0, "prefix", rank, T, dev, scale)
        self.xs = wl.hidden_states(w, 0, "decode", rank, self.N, dev, scale)
        self.logits = wl.decode_logits(w, rank, self.N, dev)
        self.tokens = wl.chosen_tokens(w, self.logits, rank).contiguous()
        self.off = [0, T]
        self.ws = clada.new_workspace(self.layers[0], 1, T)
        f32 = dict(dtype=torch.float32, device=dev)
        self.scores = torch.empty(1, w.d_ff, **f32)
        self.mask = torch.empty(1, w.d_ff, dtype=torch.uint8, device=dev)
        self.idx = torch.empty(1, w.d_ff, dtype=torch.int32, device=dev)
        self.count = torch.empty(1, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.lam = torch.full((1,), LAMBDA, **f32)
        self.gam = torch.full((1,), GAMMA, **f32)
        self.zero = torch.zeros(1, **f32)
        self.s = torch.empty(self.N, **f32)
        self.h = torch.empty(self.N, **f32)
        self.tau_final = torch.empty(1, 1, **f32)
        self.y = torch.empty(len(w.sparsities), self.N, w.d_model, **f32)
        # the persistent stack launch on this layer: STACK_PASSES layer passes over the rotating copies
        self.stack = clada.LayerStack([self.layers[i % N_COPIES] for i in range(STACK_PASSES)])
        self.stack_scores = torch.empty(STACK_PASSES, 1, w.d_ff, **f32)
        self.stack_tau = torch.empty(1, STACK_PASSES, **f32)
        self.guard = [1.0, 1.0 + LAMBDA, 1.0 + GAMMA, 1.0 + LAMBDA + GAMMA]
        # calibration (stands in for the offline threshold search; not part of a step)
        clada.clada_prefix_scores(self.layers[0], self.X, self.off, self.scores, self.ws)
        self.tau_base = []
        for rho in w.sparsities:
            t = torch.empty(1, 1, **f32)
            clada.clada_tau_from_sparsity(self.scores, rho, t.view(1))
            self.tau_base.append(t)
        clada.clada_cogload(self.logits, self.tokens, self.s, self.h)
        torch.cuda.synchronize()
        self.tau_s = wl.universal_threshold(self.s.tolist())
        self.tau_H = wl.universal_threshold(self.h.tolist())
        self.counts = {}
        # nested index lists (the masks' compressed form): per sparsity one list + four counts
        i32 = dict(dtype=torch.int32, device=dev)
        self.order = torch.empty(len(w.sparsities), 1, w.d_ff, **i32)
        self.ncounts = torch.empty(len(w.sparsities), 1, 4, **i32)
        self.level = torch.zeros(1, **i32)

    def step_nested(self):
        """The same step with the kept sets held as nested index lists: the selection builds one list and
        four counts per sparsity, a decode token takes its load level and the FFN reads the list's head."""
        c, w = self.clada, self.w
        L0 = self.layers[0]
        c.clada_prefix_scores(L0, self.X, self.off, self.scores, self.ws, self.status)
        for r, rho in enumerate(w.sparsities):
            tb = self.tau_base[r]
            c.clada_refine_scores(L0, self.X, self.off, tb.view(1), self.guard, 1e-4, self.scores, self.ws, self.status)
            c.clada_nested_build(self.scores, tb.view(1), LAMBDA, GAMMA, self.order[r], self.ncounts[r])
            for t in range(self.N):
                c.clada_cogload_level(self.logits[t:t + 1], self.tokens[t:t + 1], self.tau_s, self.tau_H,
                                      self.s[t:t + 1], self.h[t:t + 1], self.level, self.status)
                c.clada_sparse_ffn_decode_nested(self.layers[t % N_COPIES], self.xs[t:t + 1], self.order[r],
                                                 self.ncounts[r], self.level, self.y[r, t:t + 1], self.ws,
                                                 status=self.status)

    def ffn_only_loop_nested(self):
        """Nested-list FFN launches at the baseline level back to back (call after step_nested)."""
        self.level.zero_()
        for t in range(self.N):
            self.clada.clada_sparse_ffn_decode_nested(self.layers[t % N_COPIES], self.xs[t:t + 1], self.order[0],
                                                      self.ncounts[0], self.level, self.y[0, t:t + 1], self.ws)

    def step(self, adapt: bool = True):
        """One pass of the whole path.  adapt=False runs it with lambda = gamma = 0 (the paper's ablation row
        without semantic adaptation): every token then decodes at the configured baseline sparsity."""
        c, w = self.clada, self.w
        L0 = self.layers[0]
        lam, gam = (self.lam, self.gam) if adapt else (self.zero, self.zero)
        c.clada_prefix_scores(L0, self.X, self.off, self.scores, self.ws, self.status)
        for r, rho in enumerate(w.sparsities):
            tb = self.tau_base[r]
            c.clada_refine_scores(L0, self.X, self.off, tb.view(1), self.guard, 1e-4, self.scores, self.ws, self.status)
            c.clada_select(self.scores, tb.view(1), 1, self.mask, self.idx, self.count)
            for t in range(self.N):
                c.clada_cogload_adjust(self.logits[t:t + 1], self.tokens[t:t + 1], tb, lam, gam,
                                       self.tau_s, self.tau_H, self.s[t:t + 1], self.h[t:t + 1], self.tau_final,
                                       self.status)
                c.clada_sparse_ffn_decode(self.layers[t % N_COPIES], self.xs[t:t + 1], self.scores, self.tau_final, 1,
                                          self.y[r, t:t + 1], self.ws, status=self.status)

    @property
    def launches_per_step(self) -> int:
        # prefix (2) + per sparsity: guard band (candidates, refine, finish), select, N x (cogload, FFN)
        return 2 + len(self.w.sparsities) * (4 + 2 * self.N)

    def tokens_per_step(self) -> int:
        return len(self.w.sparsities) * self.N

    def kept_per_token(self):
        """Average number of kept neurons per decode token over the step (for algorithmic bytes)."""
        c = self.clada
        cnt = torch.empty(1, dtype=torch.int32, device=self.dev)
        tot = 0
        for r in range(len(self.w.sparsities)):
            tb = self.tau_base[r]
            for t in range(self.N):
                c.clada_cogload_adjust(self.logits[t:t + 1], self.tokens[t:t + 1], tb, self.lam, self.gam,
                                       self.tau_s, self.tau_H, self.s[t:t + 1], self.h[t:t + 1], self.tau_final)
                c.clada_select(self.scores, self.tau_final.view(1), 1, None, None, cnt)
                tot += int(cnt.item())
        return tot / self.tokens_per_step()

    ffn_launches_per_loop = property(lambda self: self.N)
    # two contractions per (token, neuron) with a gate projection, one without
    prefix_flop = property(lambda self: (2.0 if self.w.activation == 2 else 4.0) * self.T * self.w.d_model * self.w.d_ff)
    l2_note = f"inputs larger than L2: {N_COPIES} rotating copies of the layer"
    step_note = "prefix statistics + per sparsity (guard band, select, 128 x (cogload+adjust, sparse FFN))"

    def prefix_once(self):
        self.clada.clada_prefix_scores(self.layers[0], self.X, self.off, self.scores, self.ws, self.status)

    def prefill_prepare(self) -> bool:
        """Buffers of the dense prefill FFN of the prompt (16-bit layers): hidden activations Z, output Y, the running
        sums of squares, and the down projection in the paper's [d_model, d_ff] layout."""
        if self.w.dtype == "f32":
            return False
        L0 = self.layers[0]
        self.pf_w_down = L0.w_down_t.t().contiguous()
        self.pf_sumsq = torch.zeros(1, self.w.d_ff, dtype=torch.float32, device=self.dev)
        self.pf_Z = torch.empty(self.T, self.w.d_ff, dtype=self.w.torch_dtype, device=self.dev)
        self.pf_Y = torch.empty(self.T, self.w.d_model, dtype=self.w.torch_dtype, device=self.dev)
        return True

    def prefill_statistics_once(self):
        self.clada.clada_prefix_accumulate(self.layers[0], self.X, self.off, self.pf_sumsq, self.ws, self.pf_Z, self.status)

    def prefill_down_once(self):
        self.clada.clada_prefill_down(self.layers[0], self.pf_w_down, self.pf_Z, self.pf_Y, self.status, ws=self.ws)

    def io_tensors(self):
        return [self.X, self.xs, self.logits, self.tokens], self.y

    def ffn_only_loop(self, r: int = 0):
        """The FFN launches of one sparsity level at its baseline threshold back to back (for the kernel's
        own duration)."""
        for t in range(self.N):
            self.clada.clada_sparse_ffn_decode(self.layers[t % N_COPIES], self.xs[t:t + 1], self.scores,
                                               self.tau_base[r], 1, self.y[0, t:t + 1], self.ws)

    stack_passes_per_loop = property(lambda self: (self.N // STACK_PASSES) * STACK_PASSES)

    def stack_prepare(self, r: int = 0):
        self.stack_scores.copy_(self.scores.expand(STACK_PASSES, 1, -1))
        self.stack_tau.copy_(self.tau_base[r].expand(1, STACK_PASSES))

    def ffn_stack_loop(self):
        """The same layer passes (token t on copy t mod n, baseline threshold) through the persistent stack
        launch: STACK_PASSES passes per launch (call stack_prepare first)."""
        for t0 in range(0, self.stack_passes_per_loop, STACK_PASSES):
            self.clada.clada_sparse_ffn_decode_layers(self.stack, self.xs[t0:t0 + STACK_PASSES].unsqueeze(1),
                                                      self.stack_scores, self.stack_tau,
                                                      self.y[0, t0:t0 + STACK_PASSES].unsqueeze(1), self.ws)


class StackJob:
    """A whole FFN stack (workload c3: 32 Llama-2-7B-shaped layers, one sequence): per token one
    cogload+adjust launch for all layers, then the native per-layer loop of the library."""

    def __init__(self, clada, w, dev, rank: int):
        self.clada, self.w, self.dev = clada, w, dev
        L, T = w.n_layers, w.prefix_len[0]
        self.L, self.T, self.N = L, T, w.n_decode
        scale = wl.channel_scale(w, dev)
        f32 = dict(dtype=torch.float32, device=dev)
        self.layers, Xs, xs = [], [], []
        for l in range(L):
            wt = wl.layer_weights(w, l, dev)
            lay = clada.Layer(wt["w_gate"], wt["w_up"], wt["w_down"].t().contiguous())
            norms = torch.empty(w.d_ff, **f32)
            clada.clada_down_norms(lay, norms)
            lay.set_down_norm(norms)
            self.layers.append(lay)
            Xs.append(wl.hidden_states(w, l, "prefix", rank, T, dev, scale))
            xs.append(wl.hidden_states(w, l, "decode", rank, self.N, dev, scale))
        self.stack = clada.LayerStack(self.layers)
        self.X = torch.stack(Xs)                                   # [L, T, d]
        self.xs = torch.stack(xs, dim=1).unsqueeze(2).contiguous()  # [N, L, 1, d]
        self.logits = wl.decode_logits(w, rank, self.N, dev)
        self.tokens = wl.chosen_tokens(w, self.logits, rank).contiguous()
        self.off = [0, T]
        self.ws = clada.new_workspace(self.layers[0], 1, T)
        self.scores = torch.empty(L, 1, w.d_ff, **f32)
        self.mask = torch.empty(1, w.d_ff, dtype=torch.uint8, device=dev)
        self.idx = torch.empty(1, w.d_ff, dtype=torch.int32, device=dev)
        self.count = torch.empty(1, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.lam = torch.full((L,), LAMBDA, **f32)
        self.gam = torch.full((L,), GAMMA, **f32)
        self.s = torch.empty(self.N, **f32)
        self.h = torch.empty(self.N, **f32)
        self.tau_final = torch.empty(1, L, **f32)
        self.tau_base = torch.empty(1, L, **f32)
        self.y = torch.empty(self.N, L, 1, w.d_model, **f32)
        self.guard = [1.0, 1.0 + LAMBDA, 1.0 + GAMMA, 1.0 + LAMBDA + GAMMA]
        self.rho = w.sparsities[0]
        for l in range(L):   # calibration, outside the step
            clada.clada_prefix_scores(self.layers[l], self.X[l], self.off, self.scores[l], self.ws)
            clada.clada_tau_from_sparsity(self.scores[l], self.rho, self.tau_base[:, l])
        clada.clada_cogload(self.logits, self.tokens, self.s, self.h)
        torch.cuda.synchronize()
        self.tau_s = wl.universal_threshold(self.s.tolist())
        self.tau_H = wl.universal_threshold(self.h.tolist())

    ffn_launches_per_loop = property(lambda self: self.L * 8)
    prefix_flop = property(lambda self: 4.0 * self.T * self.w.d_model * self.w.d_ff)
    l2_note = "inputs larger than L2: 32 layers, 8.7 GB of weights per token"
    step_note = "per layer: prefix statistics, guard band, select; then 256 x (cogload+adjust for 32 layers, 32 sparse FFNs)"

    def step(self):
        c = self.clada
        for l in range(self.L):
            c.clada_prefix_select(self.layers[l], self.X[l], self.off, self.tau_base[:, l].contiguous(), self.guard,
                                  self.scores[l], self.mask, self.idx, self.count, self.ws, self.status)
        for t in range(self.N):
            c.clada_cogload_adjust(self.logits[t:t + 1], self.tokens[t:t + 1], self.tau_base, self.lam, self.gam,
                                   self.tau_s, self.tau_H, self.s[t:t + 1], self.h[t:t + 1], self.tau_final, self.status)
            c.clada_sparse_ffn_decode_layers(self.stack, self.xs[t], self.scores, self.tau_final, self.y[t], self.ws,
                                             self.status)

    @property
    def launches_per_step(self) -> int:
        return self.L * 7 + self.N * 2      # per token: cogload+adjust, one persistent FFN launch

    def tokens_per_step(self) -> int:
        return self.N

    def kept_per_token(self):
        """Average kept neurons per (token, layer) over the step."""
        c = self.clada
        cnt = torch.empty(1, dtype=torch.int32, device=self.dev)
        tot, n = 0, 0
        for t in range(0, self.N, 8):
            c.clada_cogload_adjust(self.logits[t:t + 1], self.tokens[t:t + 1], self.tau_base, self.lam, self.gam,
                                   self.tau_s, self.tau_H, self.s[t:t + 1], self.h[t:t + 1], self.tau_final)
            for l in (0, self.L // 2, self.L - 1):
                c.clada_select(self.scores[l], self.tau_final[:, l].contiguous(), 1, None, None, cnt)
                tot += int(cnt.item())
                n += 1
        return tot / n

    def prefix_once(self):
        self.clada.clada_prefix_scores(self.layers[0], self.X[0], self.off, self.scores[0], self.ws, self.status)

    def io_tensors(self):
        return [self.X, self.xs, self.logits, self.tokens], self.y

    ffn_kernel = "sparse_ffn_stack_kernel (one launch = all layers of a token)"

    def ffn_only_loop(self):
        """Eight tokens x 32 layers at the baseline thresholds: one persistent launch per token."""
        for t in range(8):
            self.clada.clada_sparse_ffn_decode_layers(self.stack, self.xs[t], self.scores, self.tau_base, self.y[t], self.ws)

    def ffn_per_layer_loop(self):
        """The same passes as one launch per layer."""
        for t in range(8):
            for l in range(self.L):
                self.clada.clada_sparse_ffn_decode(self.layers[l], self.xs[t, l], self.scores[l], self.tau_base[:, l],
                                                   self.L, self.y[t, l], self.ws)


class BatchJob:
    """One layer of a batched workload (c4: 8 sequences, c5: 16, each with its own prompt, scores, threshold and
    mask): prefix statistics of all prompts, then N decode steps of (cogload+adjust for the batch, sparse FFN for
    the batch: one dense pass over the layer per 16 sequences).  Informational: the metric's workload is the
    single-sequence layer."""
    layers_run = 1
    N_DECODE = 32      # decode steps per timed step (the workloads' 256-512 would only repeat these)
    N_LOGITS = 8       # distinct logit rows per sequence, cycled

    def __init__(self, clada, w, dev, rank: int):
        self.clada, self.w, self.dev = clada, w, dev
        B = self.B = w.batch
        self.N = self.N_DECODE
        lengths = wl.prefix_lengths(w)
        self.off = wl.seq_offsets(lengths)
        self.T = self.off[-1]
        weights = wl.layer_weights(w, 0, dev)
        self.layer = clada.Layer(weights["w_gate"], weights["w_up"], weights["w_down"].t().contiguous(),
                                 activation=w.activation)
        norms = torch.empty(w.d_ff, dtype=torch.float32, device=dev)
        clada.clada_down_norms(self.layer, norms)
        self.layer.set_down_norm(norms)
        scale = wl.channel_scale(w, dev)
        seq0 = rank * B    # a rank's sequences differ from the other ranks'
        self.X = torch.cat([wl.hidden_states(w, 0, "prefix", seq0 + b, n, dev, scale) for b, n in enumerate(lengths)])
        self.xs = torch.stack([wl.hidden_states(w, 0, "decode", seq0 + b, self.N, dev, scale) for b in range(B)],
                              dim=1).contiguous()                                        # [N, B, d]
        lg = [wl.decode_logits(w, seq0 + b, self.N_LOGITS, dev) for b in range(B)]
        self.logits = torch.stack(lg, dim=1).contiguous()                               # [N_LOGITS, B, V]
        self.tokens = torch.stack([wl.chosen_tokens(w, lg[b], seq0 + b) for b in range(B)], dim=1).contiguous()
        f32 = dict(dtype=torch.float32, device=dev)
        self.ws = clada.new_workspace(self.layer, B, self.T)
        self.scores = torch.empty(B, w.d_ff, **f32)
        self.mask = torch.empty(B, w.d_ff, dtype=torch.uint8, device=dev)
        self.idx = torch.empty(B, w.d_ff, dtype=torch.int32, device=dev)
        self.count = torch.empty(B, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.lam = torch.full((1,), LAMBDA, **f32)
        self.gam = torch.full((1,), GAMMA, **f32)
        self.s = torch.empty(self.N_LOGITS, B, **f32)
        self.h = torch.empty(self.N_LOGITS, B, **f32)
        self.tau_final = torch.empty(B, 1, **f32)
        self.tau_base = torch.empty(B, 1, **f32)
        self.y = torch.empty(self.N, B, w.d_model, **f32)
        self.guard = [1.0, 1.0 + LAMBDA, 1.0 + GAMMA, 1.0 + LAMBDA + GAMMA]
        self.rho = w.sparsities[0]
        clada.clada_prefix_scores(self.layer, self.X, self.off, self.scores, self.ws)
        clada.clada_tau_from_sparsity(self.scores, self.rho, self.tau_base.view(B))
        clada.clada_cogload(self.logits.view(-1, w.vocab), self.tokens.view(-1), self.s.view(-1), self.h.view(-1))
        clada.clada_select(self.scores, self.tau_base.view(B), 1, self.mask, None, self.count)
        torch.cuda.synchronize()
        self.tau_s = wl.universal_threshold(self.s.flatten().tolist())
        self.tau_H = wl.universal_threshold(self.h.flatten().tolist())
        # Rows one layer-step at the baseline thresholds has to read: per launch, the union of the kept sets of the
        # launch's sequences (the library takes 16 sequences per dense pass from 3 sequences on -- the pass reads
        # every row of the layer, its union or not -- and tiles of 4 or 2 below that).
        tile = 4 if w.d_model * w.elem_bytes <= 8192 else 2
        self.launch_sizes, rest = [], B
        while rest > 0:
            n = min(rest, 16) if rest >= 3 and w.dtype != "f32" else min(rest, tile)
            self.launch_sizes.append(n)
            rest -= n
        m = self.mask.bool()
        self.union_rows, b0 = 0, 0
        for n in self.launch_sizes:
            self.union_rows += int(m[b0:b0 + n].any(dim=0).sum())
            b0 += n
        self.dense = max(self.launch_sizes) > 4

    traffic_kernel = property(lambda self: "sparse_ffn_batch_dense_kernel" if self.dense else "sparse_ffn_batch_tc_kernel")
    ffn_kernel = property(lambda self: "sparse_ffn_batch_dense_kernel (one call = one dense pass per 16 sequences)"
                          if self.dense else
                          "sparse_ffn_batch_tc_kernel (one call = keep words of the batch + all its tiles)")
    step_note = property(lambda self: f"prefix statistics, guard band, select for {self.B} prompts; then {self.N} x "
                                      f"(cogload+adjust for the batch, sparse FFN for the batch in launches of "
                                      f"{self.launch_sizes} sequences)")
    l2_note = ("inputs larger than L2: every layer-step streams the layer (dense pass) or the union of its tiles' "
               "kept rows (see bytes_per_launch)")
    ffn_launches_per_loop = property(lambda self: self.N)
    prefix_flop = property(lambda self: (2.0 if self.w.activation == 2 else 4.0) * self.T * self.w.d_model * self.w.d_ff)

    @property
    def ffn_bytes_per_launch(self):
        w, eb = self.w, self.w.elem_bytes
        return self.union_rows * 3 * w.d_model * eb + self.B * (w.d_ff * 4 + w.d_model * eb + w.d_model * 4)

    def step(self):
        c, B = self.clada, self.B
        c.clada_prefix_select(self.layer, self.X, self.off, self.tau_base.view(B), self.guard, self.scores, self.mask,
                              self.idx, self.count, self.ws, self.status)
        for t in range(self.N):
            r = t % self.N_LOGITS
            c.clada_cogload_adjust(self.logits[r], self.tokens[r], self.tau_base, self.lam, self.gam, self.tau_s,
                                   self.tau_H, self.s[r], self.h[r], self.tau_final, self.status)
            c.clada_sparse_ffn_decode(self.layer, self.xs[t], self.scores, self.tau_final.view(B), 1, self.y[t],
                                      self.ws, status=self.status)

    @property
    def launches_per_step(self) -> int:
        keep_words = 0 if all(n > 4 or n == 1 for n in self.launch_sizes) else 1
        return 7 + self.N * (1 + keep_words + len(self.launch_sizes))      # cogload+adjust, keep words, the FFN launches

    def tokens_per_step(self) -> int:
        return self.B * self.N

    def kept_per_token(self):
        c, B = self.clada, self.B
        tot = 0
        for r in range(self.N_LOGITS):
            c.clada_cogload_adjust(self.logits[r], self.tokens[r], self.tau_base, self.lam, self.gam, self.tau_s,
                                   self.tau_H, self.s[r], self.h[r], self.tau_final)
            c.clada_select(self.scores, self.tau_final.view(B), 1, None, None, self.count)
            tot += int(self.count.sum().item())
        return tot / (self.N_LOGITS * B)

    def prefix_once(self):
        self.clada.clada_prefix_scores(self.layer, self.X, self.off, self.scores, self.ws, self.status)

    def io_tensors(self):
        return [self.X, self.xs, self.logits, self.tokens], self.y

    def ffn_only_loop(self):
        for t in range(self.N):
            self.clada.clada_sparse_ffn_decode(self.layer, self.xs[t], self.scores, self.tau_base.view(self.B), 1,
                                               self.y[t], self.ws)


FFN_INNER = 12      # replays per sample of an FFN-only loop (a sample lasts 40-60 ms)
FFN_REPEATS = 7     # samples per figure


def _graphed(fn, stream, use_graph):
    """fn run once to warm up, then (with use_graph) captured; returns the callable to time."""
    fn()
    if not use_graph:
        return fn
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        fn()
    g.replay()
    return g.replay


def _median_ms(run, inner=1, repeats=None):
    """Median over `repeats` samples of the device time of one run (each sample times `inner` runs)."""
    repeats = FFN_REPEATS if repeats is None else repeats
    samples = sorted(_timed(run, inner, lambda: None) / inner for _ in range(repeats))
    return samples[len(samples) // 2]


def _timed(fn, steps, dist_barrier):
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist_barrier()
    torch.cuda.synchronize()
    start.record()
    for _ in range(steps):
        fn()
    end.record()
    torch.cuda.synchronize()
    dist_barrier()
    return start.elapsed_time(end)


def other_workloads_info(clada, dev, stream, use_graph, peak, read_gbs):
    """FFN-only figures on the other workloads' layers, for information: the 32-layer stack (eight tokens, one
    persistent launch per token, and the same passes as one launch per layer) and one layer of each batched
    workload (the batch's call = one dense pass per 16 sequences; bytes = the union of the kept rows of each
    launch's sequences, which the pass reads along with the few rows nobody keeps)."""
    out = {}
    for name in ("c3_llama2_7b_stack", "c4_llama3_8b_b8", "c5_13b_b16"):
        w = wl.WORKLOADS[name]
        job = (BatchJob if w.batch > 1 else StackJob)(clada, w, dev, 0)
        t_ms = _median_ms(_graphed(job.ffn_only_loop, stream, use_graph), inner=3) / job.ffn_launches_per_loop
        kept = w.d_ff - w.k_cut(w.sparsities[0])
        if w.batch > 1:
            nbytes = job.ffn_bytes_per_launch
            rec = {"kernel": job.ffn_kernel, "layers_run": 1, "batch": w.batch, "sequences_per_launch": job.launch_sizes,
                   "sparsity": w.sparsities[0], "us_per_batch_call": t_ms * 1e3, "bytes_per_batch_call": nbytes,
                   "union_rows": job.union_rows, "traffic": recorded_traffic(job.traffic_kernel, name)}
        else:
            nbytes = kept * 3 * w.d_model * w.elem_bytes + w.d_ff * 4 + w.d_model * w.elem_bytes + w.d_model * 4
            t_layer = _median_ms(_graphed(job.ffn_per_layer_loop, stream, use_graph), inner=3) / job.ffn_launches_per_loop
            rec = {"kernel": "sparse_ffn_stack_kernel", "layers": job.L, "sparsity": w.sparsities[0], "kept_neurons": kept,
                   "us_per_layer_pass": t_ms * 1e3, "bytes_per_layer_pass": nbytes,
                   "ffn_only_tokens_per_s": 1.0 / (t_ms * 1e-3 * job.L),
                   "per_layer_launch": {"kernel": "sparse_ffn_kernel", "us_per_launch": t_layer * 1e3,
                                        "achieved": nbytes / (t_layer * 1e-3) / 1e9,
                                        "frac": nbytes / (t_layer * 1e-3) / 1e9 / peak}}
        gbs = nbytes / (t_ms * 1e-3) / 1e9
        rec.update({"achieved": gbs, "unit": "GB/s", "frac": gbs / peak, "frac_of_read_only_stream": gbs / read_gbs,
                    "device_status_word": int(job.status.item())})
        out[name] = rec
        del job
        torch.cuda.empty_cache()
    return out


def run_ours(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()

    from paper_2502_19078_b200 import binding as clada
    from paper_2502_19078_b200 import build
    if rank == 0:
        build.build()
    barrier()
    clada.load()
    w = wl.WORKLOADS[args.workload]
    if args.batch:
        w = wl.scaled(w, batch=args.batch)
    job = (BatchJob if w.batch > 1 else StackJob if w.n_layers > 1 else Job)(clada, w, dev, rank)

    stream = torch.cuda.Stream()
    graph = None
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3) if not args.graph else 1):
            job.step()
        stream.synchronize()
        if args.graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                job.step()
            run = graph.replay
            for _ in range(max(args.warmup, 3)):
                run()
        else:
            run = job.step
        stream.synchronize()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        ms = _timed(run, args.steps, barrier)
        clocks = sampler.stop() if rank == 0 else None

        # the step without semantic adaptation (lambda = gamma = 0): every token at the configured sparsity
        base_ms = None
        if isinstance(job, Job):
            base_run = _graphed(lambda: job.step(adapt=False), stream, args.graph)
            for _ in range(2):
                base_run()
            base_ms = _timed(base_run, args.steps, barrier)

        # the prefix statistics alone (tensor-core contraction), for its own roofline line; taken before the long
        # streaming loops below, which leave the GPU at its power cap (the bf16 peak is a burst figure too)
        pf = job.prefix_once
        pf()
        prefix_ms = _timed(pf, 10, lambda: None) / 10
        # the dense prefill FFN of the same prompt: statistics pass that also writes the hidden activations, then
        # the down projection (both tensor-core contractions; for their own roofline lines)
        prefill = None
        if hasattr(job, "prefill_prepare") and job.prefill_prepare():
            job.prefill_statistics_once()
            job.prefill_down_once()
            stat_ms = _timed(job.prefill_statistics_once, 10, lambda: None) / 10
            down_ms = _timed(job.prefill_down_once, 10, lambda: None) / 10
            down_flop = 2.0 * job.T * w.d_model * w.d_ff
            prefill = {"bound": "tensor", "peak": None, "unit": "TFLOP/s", "tokens": job.T,
                       "statistics_and_hidden": {"kernel": "prefix_tc_kernel writing Z (clada_prefix_accumulate)", "ms": stat_ms,
                                                 "flop": job.prefix_flop},
                       "down_projection": {"kernel": "down_tc_kernel, K split with the workspace (+ down_reduce_kernel)"
                                                     " (clada_prefill_down)", "ms": down_ms, "flop": down_flop}}

        # The FFN kernels alone, for the roofline: the same launches back to back at the baseline threshold,
        # median of several samples, all inside one recorded window of the clocks.
        roof_sampler = ClockSampler(local)
        if rank == 0:
            roof_sampler.start()
        n_sp = len(w.sparsities) if isinstance(job, Job) else 1
        ffn_ms, stack_ms = [], []
        for r in range(n_sp):
            fr = _graphed((lambda rr: (lambda: job.ffn_only_loop(rr)))(r) if isinstance(job, Job) else job.ffn_only_loop,
                          stream, args.graph)
            ffn_ms.append(_median_ms(fr, inner=FFN_INNER) / job.ffn_launches_per_loop)
            if hasattr(job, "ffn_stack_loop"):
                job.stack_prepare(r)
                sr = _graphed(job.ffn_stack_loop, stream, args.graph)
                stack_ms.append(_median_ms(sr, inner=FFN_INNER) / job.stack_passes_per_loop)
        per_layer_ms = None
        if hasattr(job, "ffn_per_layer_loop"):
            pr = _graphed(job.ffn_per_layer_loop, stream, args.graph)
            per_layer_ms = _median_ms(pr, inner=FFN_INNER) / job.ffn_launches_per_loop
        roof_clocks = roof_sampler.stop() if rank == 0 else None
        # read-only streaming bandwidth of this machine (the peak file's figure is a read + write copy)
        probe = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
        probe.zero_()
        sink = torch.zeros(1, dtype=torch.int32, device=dev)
        rd = lambda: clada.clada_stream_read_probe(probe, sink)
        rd()
        read_gbs = probe.numel() / (_timed(rd, 10, lambda: None) / 10 * 1e-3) / 1e9
        del probe
        kept = job.kept_per_token()
        kept_base = w.d_ff - w.k_cut(w.sparsities[0])

        # end to end: inputs start in pinned host memory, outputs end there
        dev_in, dev_out = job.io_tensors()
        host_in = [t.cpu().pin_memory() for t in dev_in]
        hy = torch.empty(dev_out.shape, dtype=dev_out.dtype).pin_memory()

        # Pipelined across steps: the inputs of step i+1 cross PCIe (copy stream, into staging buffers on the device)
        # while step i computes; a step waits for its own inputs, moves them from staging into the tensors the
        # launches read (device-to-device), runs, and reads its result back.  Every step's inputs and result
        # travel inside the timed region; a run of K steps issues K+1 input copies (the last one for nobody).
        copy_stream = torch.cuda.Stream(device=dev)
        staging = [torch.empty_like(t) for t in dev_in]
        h2d_done, staging_free = torch.cuda.Event(), torch.cuda.Event()
        e2e_state = {"primed": False}

        def start_h2d():
            copy_stream.wait_event(staging_free)
            with torch.cuda.stream(copy_stream):
                for st_, ht in zip(staging, host_in):
                    st_.copy_(ht, non_blocking=True)
                h2d_done.record(copy_stream)

        def e2e_step():
            cur = torch.cuda.current_stream()
            if not e2e_state["primed"]:      # the first step of a run: its own copy, nothing to overlap with
                staging_free.record(cur)
                start_h2d()
                e2e_state["primed"] = True
            cur.wait_event(h2d_done)
            for dt, st_ in zip(dev_in, staging):
                dt.copy_(st_, non_blocking=True)
            staging_free.record(cur)
            start_h2d()
            run()
            hy.copy_(dev_out, non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        e2e_state["primed"] = False          # the timed run starts with nothing in flight
        e2e_ms = _timed(e2e_step, args.steps, barrier)
        torch.cuda.synchronize()

        # the same step over nested index lists, reported beside the headline (not in place of it)
        nested_ms = nested_ffn_ms = None
        if hasattr(job, "step_nested"):
            job.step_nested()
            n_run = job.step_nested
            nf_run = job.ffn_only_loop_nested
            if args.graph:
                n_graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(n_graph, stream=stream):
                    job.step_nested()
                n_run = n_graph.replay
            for _ in range(3):
                n_run()
            nested_ms = _timed(n_run, args.steps, barrier)
            job.ffn_only_loop_nested()
            if args.graph:
                nf_graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(nf_graph, stream=stream):
                    job.ffn_only_loop_nested()
                nf_run = nf_graph.replay
            nf_run()
            nested_ffn_ms = _median_ms(nf_run, inner=FFN_INNER) / job.ffn_launches_per_loop
        status = int(job.status.item())
        info = None
        if rank == 0 and world == 1 and w.name == WORKLOAD and args.info:
            info = other_workloads_info(clada, dev, stream, args.graph, _peaks()[0], read_gbs)

    # every rank ran its own sequence; the job's rate is all ranks' tokens over the slowest rank's time
    tokens_rank = job.tokens_per_step() * args.steps
    value, ms = sharding.whole_job_rate(tokens_rank, ms, dev)
    e2e_value, e2e_ms = sharding.whole_job_rate(tokens_rank, e2e_ms, dev)
    nested_value = None
    if nested_ms is not None:
        nested_value, nested_ms = sharding.whole_job_rate(tokens_rank, nested_ms, dev)
    base_value = None
    if base_ms is not None:
        base_value, base_ms = sharding.whole_job_rate(tokens_rank, base_ms, dev)

    peak, peak_kind = _peaks()
    prefix_flop = job.prefix_flop
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            bf16_peak = float(json.load(f)["bf16_tflops"])
        bf16_kind = "measured (burst)"
    except Exception:
        bf16_peak, bf16_kind = 1590.0, "fallback"
    eb = w.elem_bytes
    # algorithmic bytes of one FFN layer pass: three rows per kept neuron (two without a gate projection)
    # + scores + x in + y out
    rows = 2 if w.activation == 2 else 3

    def pass_bytes(kept_neurons):
        return kept_neurons * rows * w.d_model * eb + w.d_ff * 4 + w.d_model * eb + w.d_model * 4

    def figures(nbytes, t_ms):
        gbs = nbytes / (t_ms * 1e-3) / 1e9
        return {"achieved": gbs, "frac": gbs / peak, "frac_of_read_only_stream": gbs / read_gbs}

    ffn_bytes = job.ffn_bytes_per_launch if hasattr(job, "ffn_bytes_per_launch") else pass_bytes(kept_base)
    sample_note = f"median of {FFN_REPEATS} samples of {FFN_INNER} replays of the loop's CUDA graph, clocks recorded over all of them"
    per_launch = {"kernel": "sparse_ffn_kernel", "call": "clada_sparse_ffn_decode: one launch per layer pass",
                  **figures(ffn_bytes, ffn_ms[0]), "bytes_per_launch": ffn_bytes, "us_per_launch": ffn_ms[0] * 1e3,
                  "kept_neurons": kept_base,
                  "traffic": recorded_traffic(getattr(job, "traffic_kernel", "sparse_ffn_kernel"), w.name)}
    if isinstance(job, Job):
        per_launch["by_sparsity"] = [
            {"sparsity": w.sparsities[r], "kept_neurons": w.d_ff - w.k_cut(w.sparsities[r]), "us_per_launch": t * 1e3,
             **figures(pass_bytes(w.d_ff - w.k_cut(w.sparsities[r])), t)} for r, t in enumerate(ffn_ms)]
    common = {"bound": "hbm", "peak": peak, "unit": "GB/s", "peak_kind": peak_kind, "read_only_stream_gbs": read_gbs,
              "samples": sample_note, "clocks": roof_clocks}
    if stack_ms:
        # The persistent launch that takes a whole stack of layers is the library's decode path for a model's
        # layers; on this one-layer workload it runs STACK_PASSES passes per launch over the rotating copies.
        # The timed step itself launches per layer (its figures: per_layer_launch).
        roofline = {**common, "kernel": "sparse_ffn_stack_kernel",
                    "call": f"clada_sparse_ffn_decode_layers: one persistent launch per {STACK_PASSES} layer passes "
                            f"(the same passes as per_layer_launch: token t on copy t mod {N_COPIES})",
                    **figures(pass_bytes(kept_base), stack_ms[0]), "bytes_per_launch": pass_bytes(kept_base) * STACK_PASSES,
                    "bytes_per_layer_pass": pass_bytes(kept_base), "us_per_layer_pass": stack_ms[0] * 1e3,
                    "us_per_launch": stack_ms[0] * 1e3 * STACK_PASSES, "kept_neurons": kept_base,
                    "traffic": (lambda t: None if t is None else t * STACK_PASSES)(
                        recorded_traffic("sparse_ffn_stack_kernel", w.name)),
                    "by_sparsity": [
                        {"sparsity": w.sparsities[r], "kept_neurons": w.d_ff - w.k_cut(w.sparsities[r]),
                         "us_per_layer_pass": t * 1e3, **figures(pass_bytes(w.d_ff - w.k_cut(w.sparsities[r])), t)}
                        for r, t in enumerate(stack_ms)],
                    "per_layer_launch": per_launch}
    elif isinstance(job, StackJob):
        roofline = {**common, "kernel": "sparse_ffn_stack_kernel",
                    "call": "clada_sparse_ffn_decode_layers: one persistent launch per token (all layers)",
                    **figures(ffn_bytes, ffn_ms[0]), "bytes_per_launch": ffn_bytes * job.L, "bytes_per_layer_pass": ffn_bytes,
                    "us_per_layer_pass": ffn_ms[0] * 1e3, "us_per_launch": ffn_ms[0] * 1e3 * job.L, "kept_neurons": kept_base,
                    "traffic": None,
                    "per_layer_launch": {"kernel": "sparse_ffn_kernel", "call": "clada_sparse_ffn_decode per layer",
                                         **figures(ffn_bytes, per_layer_ms), "us_per_launch": per_layer_ms * 1e3}}
    else:
        roofline = {**common, **per_launch, "kernel": getattr(job, "ffn_kernel", "sparse_ffn_kernel")}
    h2d = sum(x.numel() * x.element_size() for x in host_in)
    d2h = hy.numel() * hy.element_size()

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "d_model": w.d_model, "d_ff": w.d_ff, "layers": getattr(job, "layers_run", w.n_layers), "prefix_tokens": job.T,
                   "decode_tokens_per_sparsity": job.N, "sparsities": list(w.sparsities), "batch": w.batch,
                   "l2": job.l2_note, "cuda_graph": bool(args.graph), "avg_kept_neurons_per_token": kept,
                   "lambda": LAMBDA, "gamma": GAMMA, "step": job.step_note},
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipelined": "inputs of step i+1 are copied (pinned host -> device staging) while step i computes"},
        "gpu_launches": job.launches_per_step * args.steps,
        "roofline": roofline,
        "prefix_roofline": {"bound": "tensor", "kernel": "prefix_tc_kernel (+finalize)", "ms": prefix_ms,
                            "achieved": prefix_flop / (prefix_ms * 1e-3) / 1e12, "peak": bf16_peak, "unit": "TFLOP/s",
                            "frac": prefix_flop / (prefix_ms * 1e-3) / 1e12 / bf16_peak, "peak_kind": bf16_kind,
                            "flop": prefix_flop},
        "clocks": clocks, "device_status_word": status,
    }
    if prefill is not None:
        prefill["peak"], prefill["peak_kind"] = bf16_peak, bf16_kind
        for part in ("statistics_and_hidden", "down_projection"):
            rec = prefill[part]
            rec["achieved"] = rec["flop"] / (rec["ms"] * 1e-3) / 1e12
            rec["frac"] = rec["achieved"] / bf16_peak
        line["prefill_roofline"] = prefill
    if base_value is not None:
        # lambda = gamma = 0 (the paper's ablation without semantic adaptation): the same step with every token
        # at the configured baseline sparsities, i.e. the kept sets the roofline figures are taken on
        line["value_baseline_only"] = {"value": base_value, "unit": "tokens/s", "ms_per_step": base_ms / args.steps,
                                       "kept_neurons_per_token": [w.d_ff - w.k_cut(r) for r in w.sparsities],
                                       "lambda": 0.0, "gamma": 0.0}
    if info:
        line["other_workloads"] = info
    if nested_value is not None:
        # list entries instead of the score vector: 4 bytes per kept neuron
        nb = kept_base * rows * w.d_model * eb + kept_base * 4 + w.d_model * eb + w.d_model * 4
        line["nested_lists"] = {
            "value": nested_value, "unit": "tokens/s", "ms_per_step": nested_ms / args.steps,
            "step": "prefix statistics + per sparsity (guard band, nested lists, 128 x (cogload+level, sparse FFN "
                    "over the list's head))",
            "ffn_us_per_launch": nested_ffn_ms * 1e3, "ffn_bytes_per_launch": nb,
            "ffn_achieved_gbs": nb / (nested_ffn_ms * 1e-3) / 1e9, "ffn_frac": nb / (nested_ffn_ms * 1e-3) / 1e9 / peak}
    if rank == 0:
        if world == 1 and w.name == WORKLOAD:
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (baseline, not a target)
# ------------------------------------------------------------------------------------------------

_ORACLE_WEIGHTS = {}


def oracle_sample(w, n_prefix, n_tokens):
    """Times the oracle, as it stands, on a bounded sample of the workload: the statistics of the first
    n_prefix prompt tokens, then the first n_tokens decode tokens (cogload, adjustment, sparse FFN) per
    sparsity.  The whole-step rate charges the prefix pro rata: a full step is T prompt tokens and N decode
    tokens per sparsity, the sample's share of the prompt cost is (n_tokens / N) of (T / n_prefix) x measured."""
    import numpy as np
    from oracle import clada_oracle as orc
    orc.build()
    if w.name not in _ORACLE_WEIGHTS:
        weights = wl.layer_weights(w, 0)
        _ORACLE_WEIGHTS[w.name] = tuple(wl.to_numpy_bits(weights[k]) for k in ("w_gate", "w_up", "w_down"))
    W_in, V_in, W_out = _ORACLE_WEIGHTS[w.name]
    act = w.activation
    if act == 2:
        V_in = None
    scale = wl.channel_scale(w)
    T, N = w.prefix_len[0], w.n_decode
    X = wl.to_numpy_bits(wl.hidden_states(w, 0, "prefix", 0, n_prefix, "cpu", scale))
    xs = wl.to_numpy_bits(wl.hidden_states(w, 0, "decode", 0, n_tokens, "cpu", scale))
    logits = wl.decode_logits(w, 0, n_tokens)
    tokens = wl.chosen_tokens(w, logits, 0)
    t0 = time.perf_counter()
    A = orc.neuron_scores(X, [0, n_prefix], W_in, V_in, W_out, act=act)[0]
    t_prefix = time.perf_counter() - t0
    t1 = time.perf_counter()
    sh = [orc.cogload(logits[t].numpy(), int(tokens[t])) for t in range(n_tokens)]
    t_cog = time.perf_counter() - t1
    tau_s = wl.universal_threshold([a for a, _ in sh])
    tau_H = wl.universal_threshold([b for _, b in sh])
    t2 = time.perf_counter()
    n_done = 0
    for rho in w.sparsities:
        tau_base = orc.tau_from_sparsity(A.astype(np.float32), rho)
        for t in range(n_tokens):
            tf = orc.adjust_threshold(np.array([[tau_base]], np.float32), [LAMBDA], [GAMMA], tau_s, tau_H,
                                      [sh[t][0]], [sh[t][1]])
            orc.sparse_ffn(xs[t], W_in, V_in, W_out, A, float(tf[0, 0]), act=act)
            n_done += 1
    t_decode = time.perf_counter() - t2 + t_cog * len(w.sparsities)
    step_s = t_decode + t_prefix * (T / n_prefix) * (n_tokens / N)
    return {"tokens": n_done, "decode_s": t_decode, "prefix_tokens": n_prefix, "prefix_s": t_prefix,
            "step_s": step_s, "cores": orc.num_threads()}


def _sample_text(r, w):
    return (f"{r['tokens']} decode tokens ({r['tokens'] // len(w.sparsities)} per sparsity) of the full-size layer "
            f"(cogload + adjustment + sparse FFN: {r['decode_s']:.1f} s) plus the prompt statistics of "
            f"{r['prefix_tokens']} of {w.prefix_len[0]} prompt tokens ({r['prefix_s']:.1f} s, charged pro rata)")


def cpu_baseline(w):
    r = oracle_sample(w, n_prefix=w.prefix_len[0], n_tokens=w.n_decode)   # the whole step: ~5-10 s of CPU work
    return {"value": r["tokens"] / r["step_s"], "unit": "tokens/s", "cores": r["cores"], "kind": "oracle",
            "sample": _sample_text(r, w)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.WORKLOADS[WORKLOAD]
    for _ in range(min(args.warmup, 1)):
        oracle_sample(w, n_prefix=4, n_tokens=2)
    tot_tokens, tot_s, last = 0, 0.0, None
    for _ in range(args.steps):
        last = oracle_sample(w, n_prefix=64, n_tokens=16)
        tot_tokens += last["tokens"]
        tot_s += last["step_s"]
    value = tot_tokens / tot_s
    sample = "per step " + _sample_text(last, w)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": min(args.warmup, 1),
        "ms_per_step": 1e3 * tot_s / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": last["cores"], "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", dest="graph", action="store_false")
    ap.add_argument("--no-info", dest="info", action="store_false",
                    help="leave out the informational figures on the other workloads' layers")
    ap.add_argument("--batch", type=int, default=0,
                    help="sequences per batch for the batched workloads instead of the workload's own (e.g. 2: the tile kernel)")
    ap.add_argument("--quick", action="store_true",
                    help="for profiler captures: one replay per sample of the FFN-only loops and no informational "
                         "workloads (the figures of such a run are not bench values)")
    ap.add_argument("--workload", default=WORKLOAD, choices=[WORKLOAD, "c3_llama2_7b_stack", "c4_llama3_8b_b8", "c5_13b_b16", "v1_opt_2p7b_layer",
                             "v2_gemma_2b_layer"],
                    help="the metric's workload (default); the 32-layer stack or the OPT- / Gemma-shaped "
                         "layers (other FFN forms) for information")
    args = ap.parse_args()
    if args.quick:
        global FFN_INNER, FFN_REPEATS
        FFN_INNER, FFN_REPEATS, args.info = 1, 1, False
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and not sharding.under_launcher():
        # started by hand rather than by torchrun: become the launcher of one rank per GPU
        try:
            rc = sharding.launch_ranks(args.gpus, [os.path.abspath(__file__)] + sys.argv[1:],
                                       devices_available=torch.cuda.device_count())
        except ValueError as e:
            sys.exit(f"bench.py: {e}")
        sys.exit(rc)
    else:
        run_ours(args)      # one rank; the world size is the launcher's (RANK / WORLD_SIZE)


if __name__ == "__main__":
    main()
