"""Helpers of the GPU parity tests: run the library and the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import fdkv_ref as R
from paper_2607_06519_b200 import synth

TOL = {"f32": 1e-3, "bf16": 2e-2}  # max|delta| / max|ref| per output vector (float32 accumulation)


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def bits(t: torch.Tensor) -> np.ndarray:
    """Bit patterns of a device tensor, widened to float32 patterns for bf16."""
    return f32(t).view(np.uint32)


def oracle_unit(w: synth.Workload, seq: int, pair: int, h: int) -> R.Unit:
    k0, k1 = synth.unit_tensor(w, seq, pair, h, False)
    v0, v1 = synth.unit_tensor(w, seq, pair, h, True)
    return R.Unit(k0, k1, v0, v1, w.dtype == "bf16", w.keep_num, w.keep_den)


def check_compression(ctx, w, seq, pair, h, unit: R.Unit | None = None):
    """Stored Z0 and both residual lists of one unit must equal the oracle's bit for bit."""
    u = unit or oracle_unit(w, seq, pair, h)
    for is_v, name in ((0, "k"), (1, "v")):
        z0 = ctx.get_shared(seq, pair, h, is_v, w.T)
        assert np.array_equal(bits(z0), u.z0[name].view(np.uint32)), f"z0 {name} pair {pair} head {h}"
        idx, val = ctx.get_residual(seq, pair, h, is_v)
        assert idx.numel() == u.k_keep
        got = idx.cpu().numpy()
        assert np.array_equal(got, u.kept[name]), f"indices {name} pair {pair} head {h}"
        want_val = u.z1[name].ravel()[u.kept[name]]
        assert np.array_equal(bits(val), want_val.view(np.uint32)), f"values {name} pair {pair} head {h}"
    return u


def vector_errors(got: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """max_c |got - ref| / max_c |ref| per output vector (last axis = channels)."""
    num = np.max(np.abs(got.astype(np.float64) - ref), axis=-1)
    den = np.max(np.abs(ref), axis=-1)
    return num / den


def oracle_layer_out(units, modes_row, w, layer, q_layer: np.ndarray) -> np.ndarray:
    """units: dict h -> R.Unit (tails already appended); q_layer [Hq, d] -> [Hq, d] float64."""
    out = np.zeros((w.n_q_heads, w.head_dim))
    G = w.group
    for h, u in units.items():
        out[h * G:(h + 1) * G] = u.attend(int(modes_row[h]), layer & 1, q_layer[h * G:(h + 1) * G])
    return out
