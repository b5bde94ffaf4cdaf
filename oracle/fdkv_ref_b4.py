"""CPU oracle for depth blocks of four layers (B = 4 in Eq. 1) -- TEST INFRASTRUCTURE, not part of the product.

Plain numpy restatement, one step per function, float64 after the stored values.  Only the tests, the smoke check
and the benchmark's CPU-baseline leg may import it; the CUDA library shares no code with it.

What is computed (Method section, Eq. 1-3, with B = 4):

* Eq. 1: Z = F_4 X with F_4 the orthonormal DCT-II.  Its first row is (1/2, 1/2, 1/2, 1/2), so the shared
  low-frequency coefficient is Z0 = (x0 + x1 + x2 + x3) / 2 and its contribution to every layer is Z0 / 2 (the block
  mean).  Because F_4 is orthonormal, the three high-frequency coefficients of a position contribute
  sum_{j>=1} F_4[j][l] Z_j = x_l - mean(x) to layer l: the deviation from the block mean.
* Stored values ("normative" arithmetic, float32, no fused multiply-add):
      s   = (x0 + x1) + (x2 + x3)
      z0  = rs(0.5 * s)                       rs = round to the storage type (float32: identity, bf16: nearest even)
      dev_l = rs(x_l - 0.5 * z0)              l = 0..3: the high-frequency part of layer l in layer space
      e   = (dev_0^2 + dev_1^2) + (dev_2^2 + dev_3^2)      the position's high-frequency energy (Parseval: the sum
                                              of its three squared high-frequency coefficients)
  The library keeps, per kept position, the four layer-space values dev_l instead of the three coefficients
  Z_1..Z_3 (they span the same three dimensions: sum_l dev_l = 0 up to rounding), so that a decode call for layer l
  reads one value per kept position.
* Eq. 3 (entry form): the three high-frequency groups share one kept set per tensor: the k positions with the
  largest energy e, ties to the lowest flat index; k = floor(T d num / den).
* Candidates: shared = z0 / 2; residual = z0 / 2 + dev_l on the kept positions; exact = x_l.
* Eq. 2: mean over the block's four layers, the group's query heads and the probe queries of the causal squared
  logit error of the key candidate.

Pins: tests/test_oracle_pins_b4.py (scipy's orthonormal DCT-II, Parseval, round trip with everything kept, brute
force on tiny inputs, reduction to a dense numpy evaluation of Eq. 1-3).  Unpinned by the paper (this build's
reading): the energy as the shared selection key, Omega = bytes / bytes(exact) with four values and one index per
kept position, the scale of lambda.
"""
from __future__ import annotations

import numpy as np

from . import fdkv_ref as R

SHARED, RESIDUAL, EXACT = 0, 1, 2
B = 4


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def round_bf16(a):
    """float32 -> nearest-even bf16, returned as float32 (finite inputs)."""
    u = _f32(a).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def dct4_matrix() -> np.ndarray:
    """Orthonormal DCT-II of size 4, float64: F[j][l] = a_j cos(pi (2 l + 1) j / 8), a_0 = 1/2, a_j = 1/sqrt 2."""
    F = np.empty((4, 4), dtype=np.float64)
    for j in range(4):
        a = 0.5 if j == 0 else np.sqrt(0.5)
        for l in range(4):
            F[j, l] = a * np.cos(np.pi * (2 * l + 1) * j / 8.0)
    return F


def depth_split4(x, bf16: bool):
    """x: four [T, d] arrays (layers of the block).  Returns z0, dev (list of 4), energy; all float32 arrays."""
    x = [_f32(a) for a in x]
    rs = round_bf16 if bf16 else (lambda a: a)
    s = (x[0] + x[1]) + (x[2] + x[3])            # float32 adds in this order
    z0 = rs(np.float32(0.5) * s)
    half = np.float32(0.5) * z0                  # exact
    dev = [rs(x[l] - half) for l in range(4)]
    sq = [d * d for d in dev]                    # float32 products, rounded
    energy = (sq[0] + sq[1]) + (sq[2] + sq[3])
    return z0, dev, energy


def reconstruct4(z0, dev_l, kept_idx, mode: int, x_exact) -> np.ndarray:
    """Candidate rows of one layer, float64."""
    if mode == EXACT:
        return np.asarray(x_exact, dtype=np.float64).copy()
    out = 0.5 * np.asarray(z0, dtype=np.float64)
    if mode == RESIDUAL and len(kept_idx):
        flat = out.reshape(-1)
        flat[np.asarray(kept_idx, dtype=np.int64)] += np.asarray(dev_l, dtype=np.float64).reshape(-1)[kept_idx]
    return out


def probe_error4(dev_k, kept_idx, q, group: int, h: int, pos):
    """Eq. 2's error term for the shared and the residual candidate of one (block, KV head).

    dev_k: the four layers' key deviations [T, d]; q: the four layers' probe queries [W, Hq, d]; pos: [W] probe
    positions (a query sees keys t <= its position).  Returns (e_shared, e_residual)."""
    T, d = dev_k[0].shape
    pos = np.asarray(pos, dtype=np.int64)
    W = len(pos)
    causal = np.arange(T)[None, :] <= pos[:, None]                      # [W, T]
    keep = np.zeros(T * d, dtype=bool)
    keep[np.asarray(kept_idx, dtype=np.int64)] = True
    tot = np.zeros(2, dtype=np.float64)
    for l in range(4):
        full = np.asarray(dev_k[l], dtype=np.float64)                   # what the shared candidate misses
        drop = np.where(keep.reshape(T, d), 0.0, full)                  # what the residual candidate misses
        for g in range(group):
            ql = np.asarray(q[l], dtype=np.float64)[:, h * group + g, :]  # [W, d]
            for cand, miss in enumerate((full, drop)):
                logit_err = (ql @ miss.T) / np.sqrt(float(d))           # [W, T]
                tot[cand] += np.sum(np.where(causal, logit_err, 0.0) ** 2)
    tot /= 4.0 * group * W
    return float(tot[0]), float(tot[1])


def token_scores4(dev_k, q, group: int, h: int, pos) -> np.ndarray:
    """The token score between Eq. 2 and Eq. 3 for a block of four: s_t = max over the block's layers l, the group's
    query heads and the probe queries that can see token t of |Q_l . (K_l[t] - Khat_l^shared[t])|, where the shared-depth
    candidate misses exactly layer l's deviation from the block mean: K_l - Khat_l^shared = dev_l.  No 1/sqrt(d): the
    printed score has none.  dev_k: the four layers' stored key deviations [T, d]; q: their probe queries [W, Hq, d]."""
    T = dev_k[0].shape[0]
    pos = np.asarray(pos, dtype=np.int64)
    visible = np.arange(T)[None, :] <= pos[:, None]                   # [W, T]
    best = np.zeros(T, dtype=np.float64)
    for l in range(4):
        miss = np.asarray(dev_k[l], dtype=np.float64)
        for g in range(group):
            ql = np.asarray(q[l], dtype=np.float64)[:, h * group + g, :]
            s = np.abs(ql @ miss.T)                                     # [W, T]
            best = np.maximum(best, np.where(visible, s, 0.0).max(axis=0))
    return best


def omega4_tokens(T: int, d: int, e_bytes: int, k_tok: int) -> np.ndarray:
    """Normalised memory cost under the token rule: a kept token stores the four layers' deviation rows of K and of V
    and one int32 token index."""
    shared = 2.0 * T * d * e_bytes
    residual = shared + 2.0 * 4.0 * k_tok * d * e_bytes + 4.0 * k_tok
    exact = 2.0 * 4.0 * T * d * e_bytes
    return np.array([shared / exact, residual / exact, 1.0], dtype=np.float64)


def omega4(T: int, d: int, e_bytes: int, k: int) -> np.ndarray:
    """Normalised memory cost of the three modes for one (block, KV head), K and V together."""
    shared = 2.0 * T * d * e_bytes
    residual = shared + 2.0 * k * (4.0 * e_bytes + 4.0)  # four layer values and one int32 index per kept position
    exact = 2.0 * 4.0 * T * d * e_bytes
    return np.array([shared / exact, residual / exact, 1.0], dtype=np.float64)


class Unit4:
    """Compressed state of one (block of four layers, KV head): shared coefficient, deviations, kept sets, tails."""

    def __init__(self, k_layers, v_layers, bf16: bool, keep_num: int, keep_den: int, select: bool = True):
        self.x = {"k": [_f32(a) for a in k_layers], "v": [_f32(a) for a in v_layers]}
        self.T, self.d = self.x["k"][0].shape
        self.bf16 = bf16
        self.k_keep = R.keep_count(self.T, self.d, keep_num, keep_den)
        self.k_tok = (self.T * keep_num) // keep_den
        self.z0, self.dev, self.energy, self.kept = {}, {}, {}, {}
        for name in ("k", "v"):
            self.z0[name], self.dev[name], self.energy[name] = depth_split4(self.x[name], bf16)
            if select:  # entry form: the positions of largest high-frequency energy, K and V independently
                self.kept[name] = R.select_entries(self.energy[name], self.k_keep)
        self.tail = {(n, l): [] for n in ("k", "v") for l in range(4)}

    def use_tokens(self, tokens):
        """Token rule (Eq. 3 with one indicator per token): the listed tokens keep every high-frequency value of K and of
        V, in all four layers."""
        self.tokens = np.asarray(tokens, dtype=np.int32)
        ent = R.token_entries(self.tokens, self.d)
        self.kept = {"k": ent, "v": ent}

    def append(self, layer_in_block: int, k_row, v_row):
        self.tail[("k", layer_in_block)].append(_f32(k_row))
        self.tail[("v", layer_in_block)].append(_f32(v_row))

    def fold(self, n: int, keep_num: int, keep_den: int):
        """Periodic refresh for a block of four: the first n generated tokens of the four layers leave the exact tails
        and join the compressed form under the unit's mode; the chunk keeps its own floor(n d num / den) positions of
        largest high-frequency energy per tensor."""
        for name in ("k", "v"):
            tails = [self.tail[(name, l)] for l in range(4)]
            assert all(len(t) >= n for t in tails)
            xc = [np.stack(t[:n]) for t in tails]
            z0c, devc, ec = depth_split4(xc, self.bf16)
            keptc = R.select_entries(ec, R.keep_count(n, self.d, keep_num, keep_den))
            self.kept[name] = np.concatenate([self.kept[name], keptc + np.int32(self.T * self.d)]).astype(np.int32)
            self.x[name] = [np.concatenate([self.x[name][l], xc[l]]) for l in range(4)]
            self.z0[name] = np.concatenate([self.z0[name], z0c])
            self.dev[name] = [np.concatenate([self.dev[name][l], devc[l]]) for l in range(4)]
            self.energy[name] = np.concatenate([self.energy[name], ec])
            for l in range(4):
                self.tail[(name, l)] = tails[l][n:]
        self.T += n
        self.k_keep = self.kept["k"].size

    def rows(self, name: str, mode: int, layer_in_block: int) -> np.ndarray:
        pre = reconstruct4(self.z0[name], self.dev[name][layer_in_block], self.kept[name], mode,
                           self.x[name][layer_in_block])
        tail = self.tail[(name, layer_in_block)]
        if tail:
            pre = np.concatenate([pre, np.stack(tail).astype(np.float64)], axis=0)
        return pre

    def attend(self, mode: int, layer_in_block: int, q_heads) -> np.ndarray:
        kh = self.rows("k", mode, layer_in_block)
        vh = self.rows("v", mode, layer_in_block)
        return np.stack([R.attention(kh, vh, q) for q in _f32(q_heads)])
