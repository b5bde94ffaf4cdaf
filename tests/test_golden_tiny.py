"""The stored golden values of the tiny workload (written by tests/golden/make_golden.py from the oracle alone)
are re-derived here by the dense numpy float64 brute force, which shares no code with the oracle."""
import json
import os

import numpy as np
import pytest

import brute_force as bf
from paper_2607_06519_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bruteforce_reproduces_golden(dtype):
    g = json.load(open(os.path.join(HERE, "golden", f"tiny_{dtype}.json")))
    w = synth.WORKLOADS["tiny"].scaled(dtype=dtype)
    bf16 = dtype == "bf16"
    pos = synth.probe_positions(w)
    pq = (synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1))
    e = 2 if bf16 else 4
    Td = w.T * w.head_dim
    omega = [0.5, (2 * Td * e + 2 * w.k_keep * (e + 4)) / (4 * Td * e), 1.0]
    np.testing.assert_allclose(g["omega"], omega, rtol=1e-15)
    for h, rec in enumerate(g["heads"]):
        assert rec["needles"] == synth.needle_positions(w, 0, 0, h).tolist()
        k0, k1 = synth.unit_tensor(w, 0, 0, h, False)
        v0, v1 = synth.unit_tensor(w, 0, 0, h, True)
        z0k, z1k = bf.stored_coefficients(k0, k1, bf16)
        z0v, z1v = bf.stored_coefficients(v0, v1, bf16)
        masks = {}
        for name, z0, z1 in (("k", z0k, z1k), ("v", z0v, z1v)):
            m = bf.kept_mask(z1, w.k_keep)
            masks[name] = m
            idx = np.flatnonzero(m.ravel())
            assert idx[:6].tolist() == rec[name]["idx_head"]
            assert int(idx.sum()) == rec[name]["idx_sum"]
            keys = z1.ravel().view(np.uint32) & 0x7FFFFFFF
            assert int(keys[idx].min()) == rec[name]["tau_key"]
            assert int((keys > rec[name]["tau_key"]).sum()) == rec[name]["n_gt"]
            assert int((keys == rec[name]["tau_key"]).sum()) == rec[name]["n_eq"]
            assert float(z1.ravel()[idx].astype(np.float64).sum()) == pytest.approx(rec[name]["val_sum"], rel=1e-12)
            assert float(z0.astype(np.float64).sum()) == pytest.approx(rec[name]["z0_sum"], rel=1e-12)
        e_sh, e_rs = bf.probe_errors(z0k, z1k, masks["k"], pq, w.group, h, pos)
        assert e_sh == pytest.approx(rec["e_shared"], rel=1e-9)
        assert e_rs == pytest.approx(rec["e_residual"], rel=1e-9)
        for lam, mode in zip(g["lambdas"], rec["modes"]):
            L = [e_sh + lam * omega[0], e_rs + lam * omega[1], lam * omega[2]]
            assert int(np.argmin(L)) == mode
        Kc = bf.candidates(z0k, z1k, masks["k"], (k0, k1))
        Vc = bf.candidates(z0v, z1v, masks["v"], (v0, v1))
        for layer in range(2):
            q = synth.decode_q(w, 0, layer)[0][h * w.group:(h + 1) * w.group]
            for mode, mname in enumerate(("shared", "residual", "exact")):
                o = np.stack([bf.attention(Kc[mode][layer], Vc[mode][layer], qq) for qq in q])
                ref = rec["decode"][f"l{layer}_{mname}"]
                np.testing.assert_allclose(o[:, :3], ref["first3"], rtol=1e-9, atol=1e-12)
                assert float(np.abs(o).max()) == pytest.approx(ref["max_abs"], rel=1e-9)
        s = bf.token_scores(z0k, z1k, pq, w.group, h, pos)
        order = np.lexsort((np.arange(w.T), -s))
        tok = np.sort(order[: w.T // 8])
        assert tok[:8].tolist() == rec["token_rule"]["tok_head"]
        assert int(tok.sum()) == rec["token_rule"]["tok_sum"]


def test_golden_shows_the_needle_effect():
    """Layer 1, query head 0 of the tiny case: a planted needle dominates; the shared cache misses it and the
    sparse residual recovers the exact output (the paper's motivating claim, Introduction and Method)."""
    g = json.load(open(os.path.join(HERE, "golden", "tiny_f32.json")))
    d = g["heads"][0]["decode"]
    ex, rs, sh = (d[f"l1_{m}"]["first3"][0][1] for m in ("exact", "residual", "shared"))
    assert abs(rs - ex) < 0.01 * abs(ex)
    assert abs(sh - ex) > 0.5 * abs(ex)
