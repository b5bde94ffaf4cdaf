"""Drives a synthetic workload through the library: generate -> upload -> compress -> probe -> commit -> decode.

Used by the GPU tests, the smoke check and the benchmark.  Everything numerical happens inside libfdkv; this
module only moves seeded inputs to the device and calls the binding.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synth


def to_device(x: np.ndarray, dtype: str, device) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(device)
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def make_context(w: synth.Workload, max_tail: int | None = None, arena_bytes: int | None = None,
                 device="cuda:0", max_fold: int = 0, row_format: int = 0) -> B.Context:
    cfg = B.Config(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, w.T,
                   max_tail if max_tail is not None else max(w.n_steps, 1), B.BF16 if w.dtype == "bf16" else B.F32,
                   w.keep_num, w.keep_den, w.residual_rule, w.block_size, max_fold, row_format or w.row_format)
    return B.Context(cfg, device=device, arena_bytes=arena_bytes)


class Prefilled:
    """One workload with every sequence compressed, routed and committed."""

    def __init__(self, w: synth.Workload, ctx: B.Context | None = None, max_tail: int | None = None,
                 arena_bytes: int | None = None, device="cuda:0", max_fold: int = 0, row_format: int = 0):
        self.w = w
        self.device = torch.device(device)
        self.ctx = ctx or make_context(w, max_tail, arena_bytes, device, max_fold, row_format)
        self.scores = {}
        self.probe_modes = {}
        self._inputs = {}  # the library reads exact-mode rows at commit: keep the uploads alive until then

    def upload_pair(self, seq: int, pair: int):
        """Device tensors k0.., v0.. of one depth block (a pair, or four layers)."""
        kv = synth.layer_block_kv(self.w, seq, pair) if self.w.block_size == 4 else synth.layer_pair_kv(self.w, seq, pair)
        return {n: to_device(a, self.w.dtype, self.device) for n, a in kv.items()}

    def upload_probe_q(self, seq: int):
        return [to_device(synth.probe_q(self.w, seq, l), self.w.dtype, self.device) for l in range(self.w.n_layers)]

    def compress(self, seq: int, keep_inputs: bool = True):
        """Uploads and compresses every pair of a sequence; returns the per-layer device tensors."""
        w = self.w
        k_layers, v_layers = [None] * w.n_layers, [None] * w.n_layers
        nb = w.block_size
        for p in range(w.n_blocks):
            t = self.upload_pair(seq, p)
            for l in range(nb):
                k_layers[nb * p + l], v_layers[nb * p + l] = t[f"k{l}"], t[f"v{l}"]
            self.ctx.compress_prefill(seq, p, p + 1, w.T, k_layers, v_layers)
        self._inputs[seq] = (k_layers, v_layers)
        return k_layers, v_layers

    def commit(self, seq: int):
        self.ctx.commit(seq)
        self._inputs.pop(seq, None)

    def probe(self, seq: int, lam: float):
        q_layers = self.upload_probe_q(seq)
        modes, scores = self.ctx.probe(seq, 0, self.w.n_blocks, q_layers, synth.probe_positions(self.w), lam)
        torch.cuda.synchronize()
        self.scores[seq] = scores.cpu().numpy().astype(np.float64)
        self.probe_modes[seq] = modes.cpu().numpy()
        return self.probe_modes[seq], self.scores[seq]

    def prefill(self, seq: int, modes="quota", lam: float = 0.0):
        """modes: 'probe' (the rule at lam), 'quota' (benchmark mix from the probe's scores) or an int array."""
        self.compress(seq)
        if isinstance(modes, str):
            pm, sc = self.probe(seq, lam)
            if modes == "quota":
                self.ctx.set_modes(seq, synth.quota_modes(sc[..., 0]))
            elif modes != "probe":
                raise ValueError(modes)
        else:
            if self.w.residual_rule == 1:
                self.probe(seq, lam)  # the token rule chooses its sets inside the probe
            self.ctx.set_modes(seq, np.asarray(modes, dtype=np.int32))
        self.commit(seq)
        return self.ctx.get_modes(seq).numpy()

    # ---- decode-side inputs ----
    def decode_q(self, layer: int, step: int) -> torch.Tensor:
        w = self.w
        q = np.stack([synth.decode_q(w, b, layer)[step] for b in range(w.batch)])
        return to_device(q, w.dtype, self.device)

    def new_rows(self, layer: int, step: int):
        """k_new, v_new [batch, Hkv, d] of one layer and step."""
        w = self.w
        k = np.empty((w.batch, w.n_kv_heads, w.head_dim), np.float32)
        v = np.empty_like(k)
        nb = w.block_size
        rows = synth.block_tail_rows if nb == 4 else synth.tail_rows
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                k[b, h] = rows(w, b, layer // nb, h, False)[layer % nb][step]
                v[b, h] = rows(w, b, layer // nb, h, True)[layer % nb][step]
        return to_device(k, w.dtype, self.device), to_device(v, w.dtype, self.device)
