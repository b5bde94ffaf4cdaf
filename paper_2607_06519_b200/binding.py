"""Thin ctypes binding over libfdkv.so: argument marshalling only, every step runs in the CUDA kernels.

torch is used for device memory and streams.  Importing this module loads the shared library and raises if
it is missing; there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FDKV_LIB_PATH", os.path.join(_HERE, "libfdkv.so"))  # override: A/B runs of two builds

F32, BF16 = 0, 1
SHARED, RESIDUAL, EXACT = 0, 1, 2
RESIDUAL_ENTRIES, RESIDUAL_TOKENS = 0, 1
_STATUS = ["ok", "invalid argument", "unsupported", "arena full", "workspace too small", "state", "cuda error",
           "device timeout", "device check failed", "too large for the built-in scratch"]
NOALLOC_MAX_ELEMS = 1 << 20


class FdkvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = _STATUS[code] if 0 <= code < len(_STATUS) else str(code)
        super().__init__(f"{where}: fdkv status {code} ({name})")


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "max_batch", "max_prefill",
                                         "max_tail", "dtype", "keep_num", "keep_den", "residual_rule", "block_size", "max_fold", "row_format")]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_06519_b200.build` "
                          "(nvcc, sm_100a); this package has no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    P = C.POINTER
    sig = {
        "fdkv_sizes": [P(_Config), P(sz), P(sz)],
        "fdkv_create": [P(_Config), vp, sz, vp, sz, P(vp)],
        "fdkv_reset": [vp],
        "fdkv_compress_prefill": [vp, i32, i32, i32, i32, P(vp), P(vp), i64, i64, vp],
        "fdkv_probe": [vp, i32, i32, i32, P(vp), P(i32), i32, C.c_double, vp, vp, vp],
        "fdkv_set_modes": [vp, i32, P(i32)],
        "fdkv_route_budget": [vp, i32, sz, P(C.c_double), P(i32), vp],
        "fdkv_commit": [vp, i32, vp],
        "fdkv_decode_attn": [vp, i32, i32, vp, vp, vp, vp, i32, vp],
        "fdkv_decode_attn_host": [vp, i32, i32, vp, vp, vp, vp, i32, vp],
        "fdkv_decode_step_host": [vp, i32, vp, vp, vp, vp, i32, vp],
        "fdkv_set_tail_len": [vp, i32, i32, vp],
        "fdkv_fold_tail": [vp, i32, i32, vp],
        "fdkv_get_rows_e4m3": [vp, i32, i32, i32, i32, vp, vp, vp],
        "fdkv_get_shared": [vp, i32, i32, i32, i32, vp, vp],
        "fdkv_get_residual": [vp, i32, i32, i32, i32, vp, vp, P(i32), vp],
        "fdkv_get_modes": [vp, i32, P(i32)],
        "fdkv_get_token_set": [vp, i32, i32, i32, vp, vp, P(i32), vp],
        "fdkv_footprint": [vp, i32, P(sz), P(sz)],
        "fdkv_decode_bytes": [vp, i32, i32, P(sz)],
        "fdkv_plan_decode": [i32, i32, P(i32), P(i32), i32, i32, i32, i32, i32, P(C.c_uint32), P(i32), P(i32)],
        "fdkv_device_status": [vp],
        "fdkv_compress_unit_noalloc": [vp, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, P(i32), vp],
        "fdkv_test_wait_expiry": [vp, i32, vp],
        "fdkv_test_clear_device_status": [vp, vp],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.fdkv_destroy.argtypes = [vp]
    lib.fdkv_destroy.restype = None
    lib.fdkv_last_cuda_error.restype = C.c_int32
    lib.fdkv_status_str.argtypes = [C.c_int]
    lib.fdkv_status_str.restype = C.c_char_p
    lib.fdkv_launch_count.restype = C.c_int64
    lib.fdkv_kernel_launch_count.argtypes = [C.c_int32]
    lib.fdkv_kernel_launch_count.restype = C.c_int64
    return lib


_lib = _load()


def launch_count() -> int:
    return int(_lib.fdkv_launch_count())


KERNEL_PROBE_TC, KERNEL_PROBE_PORTABLE, KERNEL_DECODE_FAST, KERNEL_DECODE_PORTABLE, KERNEL_TOKEN_SCORE = range(5)


def kernel_launch_count(kernel: int) -> int:
    """Launches of one of the kernels that exist in a portable and an sm_100a form (fdkv_kernel_id)."""
    return int(_lib.fdkv_kernel_launch_count(kernel))


def last_cuda_error() -> int:
    return int(_lib.fdkv_last_cuda_error())


@dataclass
class Config:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    max_batch: int
    max_prefill: int
    max_tail: int
    dtype: int
    keep_num: int
    keep_den: int
    residual_rule: int = 0  # 0: largest-magnitude entries; 1: the paper's probe-scored tokens
    block_size: int = 2  # layers per depth block (B of Eq. 1): 2 or 4; "pair" arguments then index blocks
    max_fold: int = 0  # generated tokens fold_tail may move into the compressed form per sequence
    row_format: int = 0  # 0: committed rows keep the storage type; 1: e4m3 codes with per-channel scales

    def c(self) -> _Config:
        return _Config(*(int(getattr(self, f[0])) for f in _Config._fields_))


def sizes(cfg: Config):
    a, w = C.c_size_t(0), C.c_size_t(0)
    st = _lib.fdkv_sizes(C.byref(cfg.c()), C.byref(a), C.byref(w))
    if st:
        raise FdkvError(st, "fdkv_sizes")
    return a.value, w.value


def _check(st: int, where: str):
    if st:
        raise FdkvError(st, where)


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def plan_decode(T, modes, n_kv_heads: int, keep_num: int, keep_den: int, n_ctas: int, residual_rule: int = 0, row_format: int = 0):
    """fdkv_plan_decode (host only): T = prefill length per sequence, modes = [batch][n_kv_heads] of the layer's units.
    Returns (ranges, parts): ranges[c] = ((unit, slice) begin, (unit, slice) end) of thread block c, parts[u] = split-K
    parts of unit u."""
    batch = len(T)
    t_arr = (C.c_int32 * batch)(*[int(t) for t in T])
    flat = [int(m) for row in modes for m in row]
    if len(flat) != batch * n_kv_heads:
        raise ValueError("modes must be [batch][n_kv_heads]")
    m_arr = (C.c_int32 * len(flat))(*flat)
    start = (C.c_uint32 * (n_ctas + 1))()
    used = C.c_int32(0)
    parts = (C.c_int32 * len(flat))()
    _check(_lib.fdkv_plan_decode(batch, n_kv_heads, t_arr, m_arr, keep_num, keep_den, residual_rule, row_format, n_ctas, start,
                                 C.byref(used), parts), "fdkv_plan_decode")
    pts = [(int(v) >> 20, int(v) & 0xFFFFF) for v in start[:used.value + 1]]
    return [(pts[c], pts[c + 1]) for c in range(used.value)], list(parts)


def compress_unit_noalloc(x0, x1, keep_num: int, keep_den: int, z0_out, idx_out, val_out, stream=None) -> int:
    """Allocation-free compression of one [T, d] pair into caller-owned outputs (no context, no workspace).

    For callers that may not allocate device memory: the scratch is a static array inside the library.  The
    outputs must already exist (z0_out [T, d], idx_out int32 [k], val_out [k]); returns k.  Calls on one device
    share the scratch, so do not overlap them on different streams.
    """
    T, d = x0.shape
    dtype = BF16 if x0.dtype == torch.bfloat16 else F32
    cnt = C.c_int32(0)
    _check(_lib.fdkv_compress_unit_noalloc(_ptr(x0), _ptr(x1), x0.stride(0), T, d, dtype, keep_num, keep_den, _ptr(z0_out),
                                           _ptr(idx_out), _ptr(val_out), C.byref(cnt), _stream(stream)),
           "fdkv_compress_unit_noalloc")
    return int(cnt.value)


class Context:
    """One fdkv context over torch-owned device memory."""

    def __init__(self, cfg: Config, device="cuda:0", arena_bytes: int | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("fdkv needs a CUDA device; there is no CPU path")
        self.cfg = cfg
        self.device = torch.device(device)
        self.tdtype = torch.bfloat16 if cfg.dtype == BF16 else torch.float32
        worst, work = sizes(cfg)
        self.arena_bytes = int(arena_bytes if arena_bytes is not None else worst)
        with torch.cuda.device(self.device):
            self.arena = torch.empty(self.arena_bytes, dtype=torch.uint8, device=self.device)
            self.work = torch.empty(work, dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            torch.cuda.synchronize()
            _check(_lib.fdkv_create(C.byref(cfg.c()), self.arena.data_ptr(), self.arena_bytes, self.work.data_ptr(), work,
                                    C.byref(h)), "fdkv_create")
        self.h = h
        self.block_size = cfg.block_size or 2
        self.n_pairs = cfg.n_layers // self.block_size  # depth blocks (pairs when the block size is 2)

    def close(self):
        if getattr(self, "h", None):
            _lib.fdkv_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        _check(_lib.fdkv_reset(self.h), "fdkv_reset")

    def compress_prefill(self, seq, pair_begin, pair_end, T, k_layers, v_layers, stream=None):
        """k_layers / v_layers: per-layer tensors [T, n_kv_heads, head_dim] (None outside the pair range)."""
        L = self.cfg.n_layers
        ref = k_layers[2 * pair_begin]
        kp = (C.c_void_p * L)(*[None if t is None else t.data_ptr() for t in k_layers])
        vp = (C.c_void_p * L)(*[None if t is None else t.data_ptr() for t in v_layers])
        for t in list(k_layers) + list(v_layers):
            if t is not None and (t.stride() != ref.stride() or t.dtype != self.tdtype or t.stride(2) != 1):
                raise ValueError("all K/V layers must share one [T, Hkv, d] strided layout and the context dtype")
        _check(_lib.fdkv_compress_prefill(self.h, seq, pair_begin, pair_end, T, kp, vp, ref.stride(0), ref.stride(1),
                                          _stream(stream)), "fdkv_compress_prefill")

    def probe(self, seq, pair_begin, pair_end, q_layers, probe_pos, lam, stream=None):
        """q_layers: per-layer contiguous [W, n_q_heads, head_dim]; returns (modes int32 [pairs, Hkv], scores f32 [pairs, Hkv, 2])."""
        L = self.cfg.n_layers
        W = len(probe_pos)
        qp = (C.c_void_p * L)(*[None if t is None else t.data_ptr() for t in q_layers])
        pos = (C.c_int32 * W)(*[int(p) for p in probe_pos])
        n = (pair_end - pair_begin) * self.cfg.n_kv_heads
        modes = torch.empty(n, dtype=torch.int32, device=self.device)
        scores = torch.empty(n * 2, dtype=torch.float32, device=self.device)
        _check(_lib.fdkv_probe(self.h, seq, pair_begin, pair_end, qp, pos, W, float(lam), _ptr(modes), _ptr(scores),
                               _stream(stream)), "fdkv_probe")
        return modes.view(pair_end - pair_begin, -1), scores.view(pair_end - pair_begin, -1, 2)

    def set_modes(self, seq, modes):
        flat = [int(m) for m in torch.as_tensor(modes).reshape(-1).tolist()]
        arr = (C.c_int32 * len(flat))(*flat)
        if len(flat) != self.n_pairs * self.cfg.n_kv_heads:
            raise ValueError("modes must have n_pairs * n_kv_heads entries")
        _check(_lib.fdkv_set_modes(self.h, seq, arr), "fdkv_set_modes")

    def route_budget(self, seq, budget_bytes, stream=None):
        """Smallest lambda whose routing fits the byte budget: (fits, lambda, modes int32 [pairs, Hkv]); sets the modes."""
        n = self.n_pairs * self.cfg.n_kv_heads
        lam = C.c_double(0.0)
        arr = (C.c_int32 * n)()
        st = _lib.fdkv_route_budget(self.h, seq, int(budget_bytes), C.byref(lam), arr, _stream(stream))
        if st not in (0, 3):
            raise FdkvError(st, "fdkv_route_budget")
        return st == 0, float(lam.value), torch.tensor(list(arr), dtype=torch.int32).view(self.n_pairs, -1)

    def commit(self, seq, stream=None):
        _check(_lib.fdkv_commit(self.h, seq, _stream(stream)), "fdkv_commit")

    def decode_attn(self, layer, q, k_new=None, v_new=None, out=None, out_dtype=None, stream=None):
        """q: [batch, n_q_heads, d]; returns out [batch, n_q_heads, d]."""
        batch = q.shape[0]
        od = self.cfg.dtype if out_dtype is None else out_dtype
        if out is None:
            out = torch.empty(q.shape, dtype=torch.bfloat16 if od == BF16 else torch.float32, device=self.device)
        _check(_lib.fdkv_decode_attn(self.h, layer, batch, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), od,
                                     _stream(stream)), "fdkv_decode_attn")
        return out

    def decode_attn_host(self, layer, q, k_new, v_new, out, out_dtype, stream=None):
        """Same with host (ideally pinned) tensors; synchronous."""
        _check(_lib.fdkv_decode_attn_host(self.h, layer, q.shape[0], _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                          out_dtype, _stream(stream)), "fdkv_decode_attn_host")
        return out

    def decode_step_host(self, q, k_new, v_new, out, out_dtype, stream=None):
        """All layers of one step with host (ideally pinned) tensors: q, out [L, batch, Hq, d]; k_new, v_new
        [L, batch, Hkv, d] or None.  One copy in, L layer calls, one copy out; synchronous."""
        _check(_lib.fdkv_decode_step_host(self.h, q.shape[1], _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), out_dtype,
                                          _stream(stream)), "fdkv_decode_step_host")
        return out

    def set_tail_len(self, seq, n, stream=None):
        _check(_lib.fdkv_set_tail_len(self.h, seq, n, _stream(stream)), "fdkv_set_tail_len")

    def fold_tail(self, seq, n, stream=None):
        """Moves the first n generated tokens of every layer from the exact tails into the compressed form."""
        _check(_lib.fdkv_fold_tail(self.h, seq, n, _stream(stream)), "fdkv_fold_tail")

    def get_rows_e4m3(self, seq, layer, kv_head, is_v, T, stream=None):
        """8-bit row streams: (codes uint8 [T, d], scales float32 [d]) of a committed layer's K or V rows."""
        codes = torch.empty((T, self.cfg.head_dim), dtype=torch.uint8, device=self.device)
        scale = torch.empty(self.cfg.head_dim, dtype=torch.float32, device=self.device)
        _check(_lib.fdkv_get_rows_e4m3(self.h, seq, layer, kv_head, int(is_v), _ptr(codes), _ptr(scale), _stream(stream)),
               "fdkv_get_rows_e4m3")
        return codes, scale

    def get_shared(self, seq, pair, kv_head, is_v, T, stream=None):
        out = torch.empty((T, self.cfg.head_dim), dtype=self.tdtype, device=self.device)
        _check(_lib.fdkv_get_shared(self.h, seq, pair, kv_head, int(is_v), _ptr(out), _stream(stream)), "fdkv_get_shared")
        return out

    def get_residual(self, seq, pair, kv_head, is_v, stream=None):
        cnt = C.c_int32(0)
        _check(_lib.fdkv_get_residual(self.h, seq, pair, kv_head, int(is_v), None, None, C.byref(cnt), _stream(stream)),
               "fdkv_get_residual")
        k = cnt.value
        idx = torch.empty(k, dtype=torch.int32, device=self.device)
        # a block of four layers keeps four values per position: [4, k]
        val = torch.empty((4, k) if self.block_size == 4 else (k,), dtype=self.tdtype, device=self.device)
        _check(_lib.fdkv_get_residual(self.h, seq, pair, kv_head, int(is_v), _ptr(idx), _ptr(val), C.byref(cnt),
                                      _stream(stream)), "fdkv_get_residual")
        return idx, val

    def get_token_set(self, seq, pair, kv_head, T, stream=None):
        """Token rule: (selected tokens int32 [k_tok] ascending, scores float32 [T]) of a staged, probed unit."""
        cnt = C.c_int32(0)
        _check(_lib.fdkv_get_token_set(self.h, seq, pair, kv_head, None, None, C.byref(cnt), _stream(stream)), "fdkv_get_token_set")
        tok = torch.empty(cnt.value, dtype=torch.int32, device=self.device)
        score = torch.empty(T, dtype=torch.float32, device=self.device)
        _check(_lib.fdkv_get_token_set(self.h, seq, pair, kv_head, _ptr(tok), _ptr(score), C.byref(cnt), _stream(stream)),
               "fdkv_get_token_set")
        return tok, score

    def get_modes(self, seq):
        n = self.n_pairs * self.cfg.n_kv_heads
        arr = (C.c_int32 * n)()
        _check(_lib.fdkv_get_modes(self.h, seq, arr), "fdkv_get_modes")
        return torch.tensor(list(arr), dtype=torch.int32).view(self.n_pairs, -1)

    def footprint(self, seq):
        by = (C.c_size_t * 3)()
        ex = C.c_size_t(0)
        _check(_lib.fdkv_footprint(self.h, seq, by, C.byref(ex)), "fdkv_footprint")
        return list(by), ex.value

    def decode_bytes(self, layer, batch):
        b = C.c_size_t(0)
        _check(_lib.fdkv_decode_bytes(self.h, layer, batch, C.byref(b)), "fdkv_decode_bytes")
        return b.value

    def device_status(self):
        return int(_lib.fdkv_device_status(self.h))

    # ---- test hooks (include/fdkv_testing.h) ----
    def test_wait_expiry(self, poll_cap: int, stream=None):
        """Runs a bounded device-side wait that nobody satisfies; device_status() then reports the timeout (7)."""
        _check(_lib.fdkv_test_wait_expiry(self.h, int(poll_cap), _stream(stream)), "fdkv_test_wait_expiry")

    def test_clear_device_status(self, stream=None):
        _check(_lib.fdkv_test_clear_device_status(self.h, _stream(stream)), "fdkv_test_clear_device_status")
