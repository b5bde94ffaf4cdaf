"""CPU oracle for 8-bit row streams (the composition with quantisation the Method section mentions after Eq. 3 and
the Limitations paragraph repeats) -- TEST INFRASTRUCTURE, not part of the product.

The paper only says that the stored coefficients can be quantised with an existing scheme; it fixes none.  This
build's reading: the dense row streams of a committed unit (the shared coefficient rows Z0 of shared / residual
units, the original rows of exact units) are stored as 8-bit floats (4 exponent bits, bias 7, 3 mantissa bits, no
infinities, largest finite value 448), with one float32 scale per channel of each stored tensor:

    amax_c  = max_t |R[t, c]|                       over the tensor's T rows (float32)
    scale_c = amax_c / 448  (float32 division), 1 if amax_c = 0
    code    = e4m3( R[t, c] / scale_c )             float32 division, round to nearest even, saturating at 448
    value   = decode(code) * scale_c                what attention sees

The sparse residual values and the generated-token tails stay in the storage type.  Everything after the codes is
float64 here.  Pins: tests/test_oracle_pins_fp8.py (torch's float8_e4m3fn cast, all 256 codes, error bounds).
Unpinned by the paper: the whole scheme (format, per-channel scales, what is quantised).
"""
from __future__ import annotations

import numpy as np

from . import fdkv_ref as R

E4M3_MAX = np.float32(448.0)


def e4m3_decode(codes) -> np.ndarray:
    """uint8 codes -> float32 values (code 0x7F / 0xFF, the format's NaN, never occurs here)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int32)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    normal = (1.0 + m / 8.0) * np.exp2(e.astype(np.float64) - 7.0)
    sub = (m / 8.0) * np.exp2(-6.0)
    return (sign * np.where(e > 0, normal, sub)).astype(np.float32)


def e4m3_encode(x) -> np.ndarray:
    """float32 -> nearest e4m3 code, ties to even, saturating at +-448 (finite inputs)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    a = np.minimum(np.abs(x).astype(np.float64), 448.0)
    # exponent of the value, clamped to the subnormal range: spacing of representable numbers is 2^(e-3)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, -6.0, 8.0)
    step = np.exp2(e - 3.0)
    q = np.rint(a / step)                # numpy rounds half to even
    v = q * step                         # may have carried into the next binade: still representable or 448-capped
    v = np.minimum(v, 448.0)
    # encode v
    with np.errstate(divide="ignore"):
        ev = np.floor(np.log2(np.where(v > 0, v, 1.0)))
    is_sub = v < np.exp2(-6.0)
    exp_field = np.where(is_sub, 0, ev + 7).astype(np.int32)
    man = np.where(is_sub, np.rint(v / np.exp2(-9.0)), np.rint((v / np.exp2(ev) - 1.0) * 8.0)).astype(np.int32)
    code = (exp_field << 3) | man
    code = np.where(np.signbit(x), code | 0x80, code)
    return code.astype(np.uint8)


def quantise_rows(rows):
    """rows [T, d] float32 (values of the storage type) -> (codes uint8 [T, d], scale float32 [d])."""
    r = np.ascontiguousarray(rows, dtype=np.float32)
    amax = np.max(np.abs(r), axis=0).astype(np.float32)
    scale = np.where(amax > 0, amax / E4M3_MAX, np.float32(1.0)).astype(np.float32)   # float32 division
    codes = e4m3_encode((r / scale[None, :]).astype(np.float32))                      # float32 division
    return codes, scale


def dequantise_rows(codes, scale) -> np.ndarray:
    return e4m3_decode(codes).astype(np.float64) * np.asarray(scale, dtype=np.float64)[None, :]


class UnitFp8(R.Unit):
    """A pair unit (entry rule) whose committed row streams are 8-bit: Z0 of K and V, and the four exact tensors."""

    def __init__(self, k0, k1, v0, v1, bf16: bool, keep_num: int, keep_den: int):
        super().__init__(k0, k1, v0, v1, bf16, keep_num, keep_den)
        self.q_z0, self.q_x = {}, {}
        for name in ("k", "v"):
            self.q_z0[name] = quantise_rows(self.z0[name])
            self.q_x[name] = tuple(quantise_rows(self.x[name][l]) for l in range(2))

    def rows(self, name: str, mode: int, layer_in_pair: int) -> np.ndarray:
        if mode == R.EXACT:
            pre = dequantise_rows(*self.q_x[name][layer_in_pair])
        else:
            pre = dequantise_rows(*self.q_z0[name])
            if mode == R.RESIDUAL and self.kept[name].size:
                s = 1.0 if layer_in_pair == 0 else -1.0
                idx = self.kept[name].astype(np.int64)
                flat = pre.reshape(-1)
                flat[idx] += s * self.z1[name].reshape(-1)[idx].astype(np.float64)
            pre = pre * np.sqrt(0.5)
        tail = self.tail[(name, layer_in_pair)]
        if tail:
            pre = np.concatenate([pre, np.stack(tail).astype(np.float64)], axis=0)
        return pre


class Unit4Fp8:
    """A block-of-four unit (see fdkv_ref_b4.Unit4) whose committed row streams are 8-bit."""

    def __init__(self, k_layers, v_layers, bf16: bool, keep_num: int, keep_den: int):
        from . import fdkv_ref_b4 as R4
        self.u = R4.Unit4(k_layers, v_layers, bf16, keep_num, keep_den)
        self.q_z0 = {n: quantise_rows(self.u.z0[n]) for n in ("k", "v")}
        self.q_x = {n: [quantise_rows(self.u.x[n][l]) for l in range(4)] for n in ("k", "v")}

    def append(self, layer_in_block: int, k_row, v_row):
        self.u.append(layer_in_block, k_row, v_row)

    def rows(self, name: str, mode: int, layer_in_block: int) -> np.ndarray:
        u = self.u
        if mode == R.EXACT:
            pre = dequantise_rows(*self.q_x[name][layer_in_block])
        else:
            pre = 0.5 * dequantise_rows(*self.q_z0[name])
            if mode == R.RESIDUAL and u.kept[name].size:
                idx = u.kept[name].astype(np.int64)
                pre.reshape(-1)[idx] += u.dev[name][layer_in_block].reshape(-1)[idx].astype(np.float64)
        tail = u.tail[(name, layer_in_block)]
        if tail:
            pre = np.concatenate([pre, np.stack(tail).astype(np.float64)], axis=0)
        return pre

    def attend(self, mode: int, layer_in_block: int, q_heads) -> np.ndarray:
        kh = self.rows("k", mode, layer_in_block)
        vh = self.rows("v", mode, layer_in_block)
        return np.stack([R.attention(kh, vh, q) for q in np.ascontiguousarray(q_heads, dtype=np.float32)])
