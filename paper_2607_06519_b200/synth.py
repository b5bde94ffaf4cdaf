"""Seeded synthetic K/V/Q generator shared by the tests, the benchmark and the smoke check.

This module only draws inputs.  It contains none of the method's arithmetic (no depth
transform, no selection, no probe, no attention) and imports neither the CUDA binding nor the
CPU oracle, so both sides can be fed from it without sharing any code of their own.

Recipe (stands in for the long-context prompts the paper evaluates on; Section "Experiments"):
every KV head of a layer pair gets a per-channel scale ``sigma = exp(N(0,1))`` (a few
high-magnitude channels), a layer-0 tensor ``x0 = u0 * sigma`` and a correlated layer-1 tensor
``x1 = (rho*u0 + sqrt(1-rho^2) * m * n1) * sigma`` where ``m`` is 8 on a few planted "needle"
tokens and 1 elsewhere (rare tokens with a large layer-specific deviation).  All arithmetic is
float32; for bf16 workloads every tensor is rounded to nearest-even bf16 and returned as
float32 holding exactly representable values.

One independent Philox stream per purpose keeps any slice reproducible without generating the
rest: ``key = (seed, seq<<48 | a<<32 | b<<16 | tag)``.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
import os

import numpy as np

TAG_K, TAG_V, TAG_NEEDLE, TAG_PROBE_Q, TAG_DECODE_Q, TAG_TAIL_K, TAG_TAIL_V, TAG_RHO = range(8)
TAG_BLOCK_K, TAG_BLOCK_V, TAG_BLOCK_TAIL_K, TAG_BLOCK_TAIL_V = range(8, 12)  # four-layer blocks


@dataclass(frozen=True)
class Workload:
    """Shape and recipe parameters of one synthetic workload."""

    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    T: int
    dtype: str  # "f32" or "bf16"
    keep_num: int
    keep_den: int
    n_needles: int
    W: int
    seed: int
    fixed_rho: float | None = None
    n_steps: int = 1
    seq_seeds: tuple | None = None  # per-sequence seed override (batched workload)
    residual_rule: int = 0  # 0: largest-magnitude entries; 1: probe-scored tokens (the paper's rule)
    block_size: int = 2  # layers per depth block (2 or 4)
    row_format: int = 0  # 0: committed rows in the storage type; 1: 8-bit rows with per-channel scales

    @property
    def n_pairs(self) -> int:
        return self.n_layers // 2

    @property
    def n_blocks(self) -> int:
        return self.n_layers // self.block_size

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def k_tok(self) -> int:
        return (self.T * self.keep_num) // self.keep_den

    @property
    def k_keep(self) -> int:
        return (self.T * self.head_dim * self.keep_num) // self.keep_den

    def seed_of(self, seq: int) -> int:
        return self.seq_seeds[seq] if self.seq_seeds is not None else self.seed

    def scaled(self, **kw) -> "Workload":
        d = dict(self.__dict__)
        d.update(kw)
        return Workload(**d)


def _llama(name, batch, T, keep_den, n_needles, seed, n_steps=1, seq_seeds=None):
    return Workload(name=name, n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, batch=batch,
                    T=T, dtype="bf16", keep_num=1, keep_den=keep_den, n_needles=n_needles, W=64,
                    seed=seed, n_steps=n_steps, seq_seeds=seq_seeds)


WORKLOADS = {
    # tiny correctness case
    "tiny": Workload(name="tiny", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, batch=1, T=512,
                     dtype="f32", keep_num=1, keep_den=8, n_needles=8, W=32, seed=0, fixed_rho=0.9),
    # Llama-3-8B-shaped single decode step at 32k (also the prefill compression + probe workload)
    "decode32k": _llama("decode32k", 1, 32768, 16, 64, 2),
    # batched decode, 8 sequences x 32k, 128 steps appending to the exact tail
    "batch8": _llama("batch8", 8, 32768, 16, 64, 3, n_steps=128,
                     seq_seeds=tuple(3 * 1000 + b for b in range(8))),
    # long context
    "decode128k": _llama("decode128k", 1, 131072, 32, 256, 4),
    "prefill32k": _llama("prefill32k", 1, 32768, 16, 64, 2),
}
# reduced-depth variants of the 32k / 128k workloads (4 layers): same kernels and per-launch sizes, a few GB on the
# device; used for profiler captures and quick checks
WORKLOADS["decode32k_4l"] = WORKLOADS["decode32k"].scaled(n_layers=4, name="decode32k_4l")
WORKLOADS["decode128k_4l"] = WORKLOADS["decode128k"].scaled(n_layers=4, name="decode128k_4l")
# the same 32k workload with the paper's token-granular residual (probe-scored tokens keep whole rows)
# the 32k workload while it generates: every step appends one token to every layer's exact tail (stream launches)
WORKLOADS["decode32k_gen"] = WORKLOADS["decode32k"].scaled(n_steps=64, name="decode32k_gen")
WORKLOADS["decode32k_tok"] = WORKLOADS["decode32k"].scaled(residual_rule=1, name="decode32k_tok")
WORKLOADS["decode32k_tok_4l"] = WORKLOADS["decode32k_tok"].scaled(n_layers=4, name="decode32k_tok_4l")
# depth blocks of four layers (the paper's default block size): tiny correctness case and the 32k shape
# the 32k workload with the committed rows stored as 8-bit floats
WORKLOADS["decode32k_fp8"] = WORKLOADS["decode32k"].scaled(row_format=1, name="decode32k_fp8")
WORKLOADS["decode32k_fp8_4l"] = WORKLOADS["decode32k_fp8"].scaled(n_layers=4, name="decode32k_fp8_4l")
WORKLOADS["decode128k_fp8"] = WORKLOADS["decode128k"].scaled(row_format=1, name="decode128k_fp8")
WORKLOADS["tiny_b4"] = WORKLOADS["tiny"].scaled(n_layers=4, block_size=4, name="tiny_b4")
WORKLOADS["decode32k_b4"] = WORKLOADS["decode32k"].scaled(block_size=4, name="decode32k_b4")
# the paper's default pairing: blocks of four layers with probe-scored tokens
WORKLOADS["decode32k_b4_tok"] = WORKLOADS["decode32k"].scaled(block_size=4, residual_rule=1, name="decode32k_b4_tok")
WORKLOADS["decode32k_b4_8l"] = WORKLOADS["decode32k"].scaled(n_layers=8, block_size=4, name="decode32k_b4_8l")


def rng(seed: int, seq: int, a: int, b: int, tag: int) -> np.random.Generator:
    lo = (int(seq) << 48) | (int(a) << 32) | (int(b) << 16) | int(tag)
    return np.random.Generator(np.random.Philox(key=np.array([int(seed), lo], dtype=np.uint64)))


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest-even bf16 and return them as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rs(x: np.ndarray, dtype: str) -> np.ndarray:
    return round_bf16(x) if dtype == "bf16" else np.ascontiguousarray(x, dtype=np.float32)


def rho_of(w: Workload, seq: int, pair: int) -> float:
    if w.fixed_rho is not None:
        return float(w.fixed_rho)
    return float(rng(w.seed_of(seq), seq, pair, 0xFFFF, TAG_RHO).uniform(0.7, 0.95))


def needle_positions(w: Workload, seq: int, pair: int, h: int) -> np.ndarray:
    r = rng(w.seed_of(seq), seq, pair, h, TAG_NEEDLE)
    return np.sort(r.choice(w.T, w.n_needles, replace=False))


def unit_sigma(w: Workload, seq: int, pair: int, h: int, is_v: bool) -> np.ndarray:
    r = rng(w.seed_of(seq), seq, pair, h, TAG_V if is_v else TAG_K)
    return np.exp(r.standard_normal(w.head_dim)).astype(np.float32)


def unit_tensor(w: Workload, seq: int, pair: int, h: int, is_v: bool):
    """(x0, x1): the [T, d] K (or V) tensors of layers 2*pair and 2*pair+1 for KV head h."""
    T, d = w.T, w.head_dim
    r = rng(w.seed_of(seq), seq, pair, h, TAG_V if is_v else TAG_K)
    sigma = np.exp(r.standard_normal(d)).astype(np.float32)
    u0 = r.standard_normal((T, d), dtype=np.float32)
    n1 = r.standard_normal((T, d), dtype=np.float32)
    rho = rho_of(w, seq, pair)
    rho32 = np.float32(rho)
    beta32 = np.float32(np.sqrt(1.0 - rho * rho))
    m = np.ones((T, 1), dtype=np.float32)
    m[needle_positions(w, seq, pair, h), 0] = np.float32(8.0)
    x0 = _rs(u0 * sigma, w.dtype)
    n1 *= m
    n1 *= beta32
    u0 *= rho32
    u0 += n1
    u0 *= sigma
    x1 = _rs(u0, w.dtype)
    return x0, x1


def block_tensor(w: Workload, seq: int, blk: int, h: int, is_v: bool):
    """[x0, x1, x2, x3]: the [T, d] K (or V) tensors of the four layers of block `blk` for KV head h.

    A first-order chain in unit-variance space: u_0 ~ N(0,1), u_l = rho u_{l-1} + sqrt(1-rho^2) m n_l, each layer
    scaled by the head's per-channel sigma; m is 8 on the planted needle tokens."""
    T, d = w.T, w.head_dim
    r = rng(w.seed_of(seq), seq, blk, h, TAG_BLOCK_V if is_v else TAG_BLOCK_K)
    sigma = np.exp(r.standard_normal(d)).astype(np.float32)
    u = r.standard_normal((T, d), dtype=np.float32)
    rho = rho_of(w, seq, blk)
    rho32 = np.float32(rho)
    beta32 = np.float32(np.sqrt(1.0 - rho * rho))
    m = np.ones((T, 1), dtype=np.float32)
    m[needle_positions(w, seq, blk, h), 0] = np.float32(8.0)
    out = [_rs(u * sigma, w.dtype)]
    for _ in range(3):
        n = r.standard_normal((T, d), dtype=np.float32)
        n *= m
        n *= beta32
        u = u * rho32
        u += n
        out.append(_rs(u * sigma, w.dtype))
    return out


def block_sigma(w: Workload, seq: int, blk: int, h: int, is_v: bool) -> np.ndarray:
    r = rng(w.seed_of(seq), seq, blk, h, TAG_BLOCK_V if is_v else TAG_BLOCK_K)
    return np.exp(r.standard_normal(w.head_dim)).astype(np.float32)


def block_tail_rows(w: Workload, seq: int, blk: int, h: int, is_v: bool):
    """[x0_new .. x3_new]: [n_steps, d] generated-token rows for the four layers of a block (same chain, m = 1)."""
    sigma = block_sigma(w, seq, blk, h, is_v)
    r = rng(w.seed_of(seq), seq, blk, h, TAG_BLOCK_TAIL_V if is_v else TAG_BLOCK_TAIL_K)
    rho = rho_of(w, seq, blk)
    rho32 = np.float32(rho)
    beta32 = np.float32(np.sqrt(1.0 - rho * rho))
    u = r.standard_normal((w.n_steps, w.head_dim), dtype=np.float32)
    out = [_rs(u * sigma, w.dtype)]
    for _ in range(3):
        n = r.standard_normal((w.n_steps, w.head_dim), dtype=np.float32)
        u = rho32 * u + beta32 * n
        out.append(_rs(u * sigma, w.dtype))
    return out


def layer_block_kv(w: Workload, seq: int, blk: int, threads: int | None = None):
    """K and V of the four layers of a block in model layout: dict k0..k3, v0..v3, each [T, Hkv, d] float32."""
    T, H, d = w.T, w.n_kv_heads, w.head_dim
    out = {f"{n}{l}": np.empty((T, H, d), dtype=np.float32) for n in ("k", "v") for l in range(4)}

    def fill(job):
        h, is_v = job
        xs = block_tensor(w, seq, blk, h, is_v)
        for l in range(4):
            out[f"{'v' if is_v else 'k'}{l}"][:, h, :] = xs[l]

    jobs = [(h, is_v) for h in range(H) for is_v in (False, True)]
    n = threads or min(len(jobs), os.cpu_count() or 1)
    if n <= 1:
        for j in jobs:
            fill(j)
    else:
        with ThreadPoolExecutor(n) as ex:
            list(ex.map(fill, jobs))
    return out


def probe_q(w: Workload, seq: int, layer: int) -> np.ndarray:
    """[W, Hq, d] probe queries of one layer (the last W prompt positions)."""
    r = rng(w.seed_of(seq), seq, layer, 0xFFFF, TAG_PROBE_Q)
    return _rs(r.standard_normal((w.W, w.n_q_heads, w.head_dim), dtype=np.float32), w.dtype)


def probe_positions(w: Workload) -> np.ndarray:
    return np.arange(w.T - w.W, w.T, dtype=np.int32)


def decode_q(w: Workload, seq: int, layer: int) -> np.ndarray:
    """[n_steps, Hq, d] decode queries of one layer; row j is the query of step j."""
    r = rng(w.seed_of(seq), seq, layer, 0xFFFE, TAG_DECODE_Q)
    return _rs(r.standard_normal((w.n_steps, w.n_q_heads, w.head_dim), dtype=np.float32), w.dtype)


def tail_rows(w: Workload, seq: int, pair: int, h: int, is_v: bool):
    """(x0_new, x1_new): [n_steps, d] generated-token rows for layers 2*pair and 2*pair+1."""
    sigma = unit_sigma(w, seq, pair, h, is_v)
    r = rng(w.seed_of(seq), seq, pair, h, TAG_TAIL_V if is_v else TAG_TAIL_K)
    u0 = r.standard_normal((w.n_steps, w.head_dim), dtype=np.float32)
    n1 = r.standard_normal((w.n_steps, w.head_dim), dtype=np.float32)
    rho = rho_of(w, seq, pair)
    rho32 = np.float32(rho)
    beta32 = np.float32(np.sqrt(1.0 - rho * rho))
    x0 = _rs(u0 * sigma, w.dtype)
    x1 = _rs((rho32 * u0 + beta32 * n1) * sigma, w.dtype)
    return x0, x1


def layer_pair_kv(w: Workload, seq: int, pair: int, threads: int | None = None):
    """K and V of both layers of a pair in model layout: dict with k0,k1,v0,v1, each [T, Hkv, d] float32."""
    T, H, d = w.T, w.n_kv_heads, w.head_dim
    out = {n: np.empty((T, H, d), dtype=np.float32) for n in ("k0", "k1", "v0", "v1")}

    def fill(job):
        h, is_v = job
        x0, x1 = unit_tensor(w, seq, pair, h, is_v)
        out["v0" if is_v else "k0"][:, h, :] = x0
        out["v1" if is_v else "k1"][:, h, :] = x1

    jobs = [(h, is_v) for h in range(H) for is_v in (False, True)]
    n = threads or min(len(jobs), os.cpu_count() or 1)
    if n <= 1:
        for j in jobs:
            fill(j)
    else:
        with ThreadPoolExecutor(n) as ex:
            list(ex.map(fill, jobs))
    return out


def quota_modes(e_shared: np.ndarray, frac_shared: float = 0.5, frac_exact: float = 0.15) -> np.ndarray:
    """Benchmark policy (not part of the method): fix the mode mix from the probe's own scores.

    Units are ranked by their shared-mode probe error (ties by unit index); the lowest half become
    shared, the highest 15 % exact, the rest residual.  Returns int32 modes (0 shared, 1 residual, 2 exact).
    """
    e = np.asarray(e_shared, dtype=np.float64).ravel()
    n = e.size
    order = np.lexsort((np.arange(n), e))
    n_sh = int(round(n * frac_shared))
    n_ex = int(round(n * frac_exact))
    modes = np.ones(n, dtype=np.int32)
    modes[order[:n_sh]] = 0
    if n_ex:
        modes[order[n - n_ex:]] = 2
    return modes.reshape(np.shape(e_shared))
