"""numpy front end of the CPU oracle (test infrastructure; see fdkv_oracle.c for what each step follows).

Per-unit helpers mirror the steps of the method; `Cache` strings them together for one sequence so that the
tests can ask for "the attention output of layer l, query head i under these modes".  Nothing here is used by
the CUDA library, and nothing here uses it.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_i64 = C.c_int64

_lib.fdkv_ref_threads.restype = C.c_int
_lib.fdkv_ref_depth_split.argtypes = [_f32p, _f32p, _i64, C.c_int, _f32p, _f32p]
_lib.fdkv_ref_depth_split_f64.argtypes = [_f64p, _f64p, _i64, _f64p, _f64p]
_lib.fdkv_ref_depth_merge_f64.argtypes = [_f64p, _f64p, _i64, _f64p, _f64p]
_lib.fdkv_ref_select_entries.argtypes = [_f32p, _i64, _i64, _i32p]
_lib.fdkv_ref_select_entries.restype = _i64
_lib.fdkv_ref_reconstruct.argtypes = [_f32p, _f32p, _i32p, _i64, _i64, C.c_int, C.c_int, _f32p, _f64p]
_lib.fdkv_ref_probe_error.argtypes = [_f32p, _i32p, _i64, _i64, _i64, _f32p, _f32p, _i64, _i64, _i64, _i32p, _i64, _f64p]
_lib.fdkv_ref_omega.argtypes = [_i64, _i64, _i64, _i64, _f64p]
_lib.fdkv_ref_omega_tokens.argtypes = [_i64, _i64, _i64, _i64, _f64p]
_lib.fdkv_ref_mode.argtypes = [C.c_double, C.c_double, _f64p, C.c_double, _f64p, C.POINTER(C.c_double)]
_lib.fdkv_ref_mode.restype = C.c_int
_lib.fdkv_ref_route_budget.argtypes = [_f64p, _f64p, _i64, _f64p, C.c_double, C.c_double, C.c_double, C.c_double, _i64,
                                          C.POINTER(C.c_double), C.POINTER(C.c_double), _i32p]
_lib.fdkv_ref_route_budget.restype = C.c_int
_lib.fdkv_ref_attention.argtypes = [_f64p, _f64p, _i64, _i64, _f32p, _f64p]
_lib.fdkv_ref_token_scores.argtypes = [_f32p, _i64, _i64, _f32p, _f32p, _i64, _i64, _i64, _i32p, _i64, _f64p]
_lib.fdkv_ref_select_tokens.argtypes = [_f64p, _i64, _i64, _i32p]
_lib.fdkv_ref_select_tokens.restype = _i64

SHARED, RESIDUAL, EXACT = 0, 1, 2


def threads() -> int:
    return int(_lib.fdkv_ref_threads())


def _c32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def depth_split(x0, x1, bf16: bool):
    x0, x1 = _c32(x0), _c32(x1)
    z0, z1 = np.empty_like(x0), np.empty_like(x1)
    _lib.fdkv_ref_depth_split(x0, x1, x0.size, int(bf16), z0, z1)
    return z0, z1


def depth_split_f64(x0, x1):
    x0 = np.ascontiguousarray(x0, dtype=np.float64)
    x1 = np.ascontiguousarray(x1, dtype=np.float64)
    z0, z1 = np.empty_like(x0), np.empty_like(x1)
    _lib.fdkv_ref_depth_split_f64(x0, x1, x0.size, z0, z1)
    return z0, z1


def depth_merge_f64(z0, z1):
    z0 = np.ascontiguousarray(z0, dtype=np.float64)
    z1 = np.ascontiguousarray(z1, dtype=np.float64)
    x0, x1 = np.empty_like(z0), np.empty_like(z1)
    _lib.fdkv_ref_depth_merge_f64(z0, z1, z0.size, x0, x1)
    return x0, x1


def keep_count(T: int, d: int, num: int, den: int) -> int:
    return (T * d * num) // den


def select_entries(z1, k: int) -> np.ndarray:
    z1 = _c32(z1)
    k = max(0, min(int(k), z1.size))
    idx = np.empty(max(k, 1), dtype=np.int32)
    n = _lib.fdkv_ref_select_entries(z1.ravel(), z1.size, k, idx)
    assert n == k
    return idx[:k]


def reconstruct(z0, z1, kept_idx, mode: int, layer_in_pair: int, x_exact) -> np.ndarray:
    z0, z1, x_exact = _c32(z0), _c32(z1), _c32(x_exact)
    kept = np.ascontiguousarray(kept_idx, dtype=np.int32)
    out = np.empty(z0.shape, dtype=np.float64)
    _lib.fdkv_ref_reconstruct(z0.ravel(), z1.ravel(), kept if kept.size else np.zeros(1, np.int32), kept.size,
                              z0.size, int(mode), int(layer_in_pair), x_exact.ravel(), out.reshape(-1))
    return out


def probe_error(z1k, kept_idx, q0, q1, group: int, h: int, pos):
    z1k, q0, q1 = _c32(z1k), _c32(q0), _c32(q1)
    T, d = z1k.shape
    W, Hq, _ = q0.shape
    kept = np.ascontiguousarray(kept_idx, dtype=np.int32)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    e = np.zeros(2, dtype=np.float64)
    _lib.fdkv_ref_probe_error(z1k, kept if kept.size else np.zeros(1, np.int32), kept.size, T, d, q0, q1, Hq,
                              group, h, pos, W, e)
    return float(e[0]), float(e[1])


def omega(T: int, d: int, e_bytes: int, k: int) -> np.ndarray:
    om = np.zeros(3, dtype=np.float64)
    _lib.fdkv_ref_omega(T, d, e_bytes, k, om)
    return om


def omega_tokens(T: int, d: int, e_bytes: int, k_tok: int) -> np.ndarray:
    om = np.zeros(3, dtype=np.float64)
    _lib.fdkv_ref_omega_tokens(T, d, e_bytes, k_tok, om)
    return om


def token_entries(tokens, d: int) -> np.ndarray:
    """Flat entry indices t*d + ch of every channel of the given tokens (ascending when the tokens are)."""
    t = np.asarray(tokens, dtype=np.int64)
    return (t[:, None] * d + np.arange(d, dtype=np.int64)[None, :]).reshape(-1).astype(np.int32)


def mode_rule(e_shared: float, e_residual: float, om, lam: float):
    loss = np.zeros(3, dtype=np.float64)
    margin = C.c_double(0.0)
    m = _lib.fdkv_ref_mode(float(e_shared), float(e_residual), np.ascontiguousarray(om, dtype=np.float64),
                           float(lam), loss, C.byref(margin))
    return int(m), loss, float(margin.value)


def route_budget(e_shared, e_residual, om, bytes_exact_unit: float, budget_bytes: float, lam_lo: float = 1e-9,
                 ratio: float = 1.0 + 2.0 ** -12, max_steps: int = 400000):
    """Plain scan: lambda = 0, lam_lo, lam_lo * ratio, ... until the routing fits the budget.
    Returns (fits, lambda, modes, previous grid value): the true threshold lies in (previous, lambda]."""
    e_sh = np.ascontiguousarray(e_shared, dtype=np.float64).ravel()
    e_rs = np.ascontiguousarray(e_residual, dtype=np.float64).ravel()
    modes = np.zeros(e_sh.size, dtype=np.int32)
    lam, prev = C.c_double(0.0), C.c_double(0.0)
    fits = _lib.fdkv_ref_route_budget(e_sh, e_rs, e_sh.size, np.ascontiguousarray(om, dtype=np.float64), float(bytes_exact_unit),
                                      float(budget_bytes), float(lam_lo), float(ratio), int(max_steps), C.byref(lam),
                                      C.byref(prev), modes)
    return bool(fits), float(lam.value), modes, float(prev.value)


def attention(khat, vhat, q) -> np.ndarray:
    khat = np.ascontiguousarray(khat, dtype=np.float64)
    vhat = np.ascontiguousarray(vhat, dtype=np.float64)
    q = _c32(q)
    n, d = khat.shape
    out = np.empty(d, dtype=np.float64)
    _lib.fdkv_ref_attention(khat, vhat, n, d, q, out)
    return out


def token_scores(z1k, q0, q1, group: int, h: int, pos) -> np.ndarray:
    z1k, q0, q1 = _c32(z1k), _c32(q0), _c32(q1)
    T, d = z1k.shape
    W, Hq, _ = q0.shape
    s = np.empty(T, dtype=np.float64)
    _lib.fdkv_ref_token_scores(z1k, T, d, q0, q1, Hq, group, h, np.ascontiguousarray(pos, dtype=np.int32), W, s)
    return s


def select_tokens(s, k_tok: int) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float64)
    k_tok = max(0, min(int(k_tok), s.size))
    out = np.empty(max(k_tok, 1), dtype=np.int32)
    _lib.fdkv_ref_select_tokens(s, s.size, k_tok, out)
    return out[:k_tok]


class Unit:
    """Compressed state of one (pair, KV head): coefficients, kept sets, originals, and the exact tails.

    Entry rule (default): K and V each keep their k largest-magnitude Z1 entries.  Token rule (`tokens` given, or
    chosen later with `use_tokens`): the listed tokens keep every Z1 coefficient of K and of V.
    """

    def __init__(self, k0, k1, v0, v1, bf16: bool, keep_num: int, keep_den: int, tokens=None, select: bool = True):
        self.x = {"k": (_c32(k0), _c32(k1)), "v": (_c32(v0), _c32(v1))}
        self.T, self.d = self.x["k"][0].shape
        self.bf16 = bf16
        self.k_keep = keep_count(self.T, self.d, keep_num, keep_den)
        self.k_tok = (self.T * keep_num) // keep_den
        self.z0, self.z1, self.kept = {}, {}, {}
        for name in ("k", "v"):
            self.z0[name], self.z1[name] = depth_split(self.x[name][0], self.x[name][1], bf16)
            if tokens is None and select:
                self.kept[name] = select_entries(self.z1[name], self.k_keep)
        self.tail = {("k", 0): [], ("k", 1): [], ("v", 0): [], ("v", 1): []}
        if tokens is not None:
            self.use_tokens(tokens)

    def use_tokens(self, tokens):
        """Token rule: the same token set for K and V, all d coefficients of each."""
        self.tokens = np.asarray(tokens, dtype=np.int32)
        ent = token_entries(self.tokens, self.d)
        self.kept = {"k": ent, "v": ent}

    def append(self, layer_in_pair: int, k_row, v_row):
        self.tail[("k", layer_in_pair)].append(_c32(k_row))
        self.tail[("v", layer_in_pair)].append(_c32(v_row))

    def fold(self, n: int, keep_num: int, keep_den: int):
        """Periodic refresh (Method, last paragraph: routing is decided once; the cache may be refreshed every fixed
        number of tokens): the first n generated tokens of both layers leave the exact tail and join the compressed
        form under the unit's mode.  The chunk is transformed by Eq. 1 and keeps its own k = floor(n d num / den)
        largest-magnitude Z1 entries per tensor (Eq. 3 applied to the chunk); its originals stay available to the
        exact mode.  Entry rule only."""
        assert not hasattr(self, "tokens")
        for name in ("k", "v"):
            t0, t1 = self.tail[(name, 0)], self.tail[(name, 1)]
            assert len(t0) >= n and len(t1) >= n
            x0c, x1c = np.stack(t0[:n]), np.stack(t1[:n])
            z0c, z1c = depth_split(x0c, x1c, self.bf16)
            keptc = select_entries(z1c, keep_count(n, self.d, keep_num, keep_den))
            self.kept[name] = np.concatenate([self.kept[name], keptc + np.int32(self.T * self.d)]).astype(np.int32)
            self.x[name] = (np.concatenate([self.x[name][0], x0c]), np.concatenate([self.x[name][1], x1c]))
            self.z0[name] = np.concatenate([self.z0[name], z0c])
            self.z1[name] = np.concatenate([self.z1[name], z1c])
            self.tail[(name, 0)], self.tail[(name, 1)] = t0[n:], t1[n:]
        self.T += n
        self.k_keep = self.kept["k"].size

    def rows(self, name: str, mode: int, layer_in_pair: int) -> np.ndarray:
        pre = reconstruct(self.z0[name], self.z1[name], self.kept[name], mode, layer_in_pair,
                          self.x[name][layer_in_pair])
        tail = self.tail[(name, layer_in_pair)]
        if tail:
            pre = np.concatenate([pre, np.stack(tail).astype(np.float64)], axis=0)
        return pre

    def attend(self, mode: int, layer_in_pair: int, q_heads) -> np.ndarray:
        """q_heads: [G, d] queries of the group that reads this KV head -> [G, d] float64 outputs."""
        kh = self.rows("k", mode, layer_in_pair)
        vh = self.rows("v", mode, layer_in_pair)
        return np.stack([attention(kh, vh, q) for q in _c32(q_heads)])
