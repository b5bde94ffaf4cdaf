"""Pins of the 8-bit row-stream oracle (oracle/fdkv_ref_fp8.py): the e4m3 codec against torch's float8_e4m3fn cast and
against the format's definition (all 256 codes), the per-channel scale rule, the error bound of a quantised row, and
the reduction of the quantised unit to the plain one when the rows are exactly representable."""
import numpy as np
import pytest
import torch

from oracle import fdkv_ref as R
from oracle import fdkv_ref_fp8 as R8
from paper_2607_06519_b200 import synth


def test_decode_follows_the_format_definition():
    codes = np.arange(256, dtype=np.uint8)
    ok = (codes & 0x7F) != 0x7F  # the two NaN patterns
    want = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy()
    got = R8.e4m3_decode(codes)
    assert np.array_equal(got[ok], want[ok])
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6 and got[0x38] == 1.0


def test_encode_is_the_inverse_on_codes_and_matches_torch_in_range():
    codes = np.arange(256, dtype=np.uint8)
    ok = (codes & 0x7F) != 0x7F
    vals = R8.e4m3_decode(codes[ok])
    back = R8.e4m3_encode(vals)
    assert np.array_equal(back[vals != 0], codes[ok][vals != 0])  # +-0 both decode to 0
    g = np.random.default_rng(0)
    x = np.concatenate([g.uniform(-448, 448, 20000), g.standard_normal(20000) * 0.01, g.standard_normal(20000) * 5,
                        np.array([0.0, 448.0, -448.0, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -9, 17.0, 18.0, 19.0, 1.0625, 1.1875])]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = R8.e4m3_encode(x)
    nz = R8.e4m3_decode(got) != 0  # torch keeps the sign of values that round to zero; only magnitudes matter there
    assert np.array_equal(got[nz], want[nz])
    assert np.all(R8.e4m3_decode(want[~nz]) == 0)
    # ties go to the even mantissa: 17 -> 16 (mantissa 0), 19 -> 20 (mantissa 2), 1.0625 -> 1.0, 1.1875 -> 1.25
    assert R8.e4m3_decode(R8.e4m3_encode(np.float32([17.0, 19.0, 1.0625, 1.1875]))).tolist() == [16.0, 20.0, 1.0, 1.25]
    # saturation
    assert R8.e4m3_decode(R8.e4m3_encode(np.float32([1e6, -1e6, 460.0]))).tolist() == [448.0, -448.0, 448.0]


def test_quantised_rows_scale_rule_and_error_bound():
    g = np.random.default_rng(1)
    rows = synth.round_bf16((g.standard_normal((300, 16)) * np.exp(g.standard_normal(16))).astype(np.float32))
    rows[:, 5] = 0
    codes, scale = R8.quantise_rows(rows)
    amax = np.abs(rows).max(axis=0)
    assert scale[5] == 1.0 and np.all(codes[:, 5] & 0x7F == 0)
    np.testing.assert_array_equal(scale[amax > 0], (amax[amax > 0] / np.float32(448.0)).astype(np.float32))
    dq = R8.dequantise_rows(codes, scale)
    # the largest entry of every channel is hit exactly (up to the rounding of the scale); the rest within half a step
    top = np.abs(dq).max(axis=0)
    np.testing.assert_allclose(top[amax > 0], amax[amax > 0], rtol=2e-7)
    err = np.abs(dq - rows)
    bound = np.maximum(np.abs(rows) * 2.0 ** -4, scale[None, :] * 2.0 ** -10) * (1 + 1e-6)
    assert np.all(err <= bound)


def test_unit_with_representable_rows_equals_the_plain_unit():
    # rows that are small integers times a power of two quantise without error when the channel maximum is 7 * 2^k
    g = np.random.default_rng(2)
    T, d = 64, 8
    mk = lambda: (g.integers(-7, 8, (T, d)) * 2.0).astype(np.float32)
    k0 = mk(); k0[0, :] = 14.0
    u8 = R8.UnitFp8(k0, k0.copy(), mk(), mk(), True, 1, 4)  # equal K layers: z1 = 0, z0 = sqrt2 * k0 rounded to bf16
    u = R.Unit(u8.x["k"][0], u8.x["k"][1], u8.x["v"][0], u8.x["v"][1], True, 1, 4)
    q = g.standard_normal((2, d)).astype(np.float32)
    # exact mode: the original rows (integers up to 14 with channel maximum 14 -> codes exact)
    np.testing.assert_allclose(u8.rows("k", R.EXACT, 0), u.rows("k", R.EXACT, 0), rtol=1e-6)
    # general data: within the format's relative step of the plain unit
    k0 = g.standard_normal((T, d)).astype(np.float32); k1 = (k0 + 0.1 * g.standard_normal((T, d))).astype(np.float32)
    u8 = R8.UnitFp8(k0, k1, k1, k0, False, 1, 4)
    u = R.Unit(k0, k1, k1, k0, False, 1, 4)
    for mode in (R.SHARED, R.RESIDUAL, R.EXACT):
        a, b = u8.rows("k", mode, 1), u.rows("k", mode, 1)
        assert np.abs(a - b).max() <= 2.0 ** -4 * np.abs(b).max() * 1.5
        out8, out = u8.attend(mode, 1, q), u.attend(mode, 1, q)
        assert np.abs(out8 - out).max() <= 0.2 * np.abs(out).max()
