"""Pins of the four-layer-block oracle (oracle/fdkv_ref_b4.py) against what the paper and the mathematics fix.

Eq. 1 with B = 4 is the orthonormal DCT-II: pinned to scipy's implementation, to Parseval and to the round trip.
The layer-space form the oracle stores (block mean + per-layer deviation) is pinned to the coefficient form.
Selection, reconstruction, Eq. 2 and attention are pinned by brute force on tiny inputs and by reductions: a block
whose layers 2, 3 repeat layers 0, 1 must reproduce the two-layer oracle; four equal layers make the shared
candidate exact.
"""
import itertools

import numpy as np
import pytest
import scipy.fft

from oracle import fdkv_ref as R
from oracle import fdkv_ref_b4 as R4
from paper_2607_06519_b200 import synth


def _rand_layers(seed, T=24, d=8, scale=1.0):
    g = np.random.default_rng(seed)
    return [(g.standard_normal((T, d)) * scale).astype(np.float32) for _ in range(4)]


def test_dct4_is_scipys_orthonormal_dct2():
    F = R4.dct4_matrix()
    ref = scipy.fft.dct(np.eye(4), type=2, norm="ortho", axis=0)  # column l = transform of unit vector e_l
    np.testing.assert_allclose(F, ref, atol=1e-15)
    np.testing.assert_allclose(F @ F.T, np.eye(4), atol=1e-15)
    np.testing.assert_allclose(F[0], 0.5)


def test_layer_space_form_equals_coefficient_form():
    # Z0 / 2 is the block mean and sum_{j>=1} F[j][l] Z_j is the deviation of layer l from it (Eq. 1, B = 4)
    F = R4.dct4_matrix()
    x = np.stack([a.astype(np.float64) for a in _rand_layers(1)])  # [4, T, d]
    Z = np.einsum("jl,ltd->jtd", F, x)
    mean = x.mean(axis=0)
    np.testing.assert_allclose(0.5 * Z[0], mean, atol=1e-14)
    for l in range(4):
        hf = sum(F[j, l] * Z[j] for j in range(1, 4))
        np.testing.assert_allclose(hf, x[l] - mean, atol=1e-14)
    # Parseval on the high-frequency part: the selection key
    np.testing.assert_allclose((Z[1:] ** 2).sum(axis=0), ((x - mean) ** 2).sum(axis=0), rtol=1e-12)
    # full inverse
    np.testing.assert_allclose(np.einsum("jl,jtd->ltd", F, Z), x, atol=1e-14)


@pytest.mark.parametrize("bf16", [False, True])
def test_stored_values_follow_the_stated_arithmetic(bf16):
    x = _rand_layers(2, scale=3.0)
    if bf16:
        x = [synth.round_bf16(a) for a in x]
    z0, dev, energy = R4.depth_split4(x, bf16)
    rs = synth.round_bf16 if bf16 else (lambda a: a)
    # element by element, written out again with python floats rounded through float32
    f = np.float32
    for t, c in itertools.product(range(0, 24, 5), range(8)):
        s = f(f(x[0][t, c] + x[1][t, c]) + f(x[2][t, c] + x[3][t, c]))
        z = rs(np.array([f(0.5) * s], dtype=np.float32))[0]
        assert z0[t, c] == z
        e = []
        for l in range(4):
            dv = rs(np.array([f(x[l][t, c] - f(0.5) * z)], dtype=np.float32))[0]
            assert dev[l][t, c] == dv
            e.append(f(dv * dv))
        assert energy[t, c] == f(f(e[0] + e[1]) + f(e[2] + e[3]))
    # against float64 within the storage rounding
    x64 = np.stack([a.astype(np.float64) for a in x])
    tol = 2.0 ** -8 if bf16 else 2.0 ** -22
    np.testing.assert_allclose(z0, 0.5 * x64.sum(axis=0), rtol=tol, atol=tol * np.abs(x64).max())
    for l in range(4):
        np.testing.assert_allclose(dev[l], x64[l] - 0.5 * z0.astype(np.float64), rtol=tol, atol=1e-30)
    if bf16:
        for a in [z0] + dev:
            assert np.array_equal(synth.round_bf16(a), a)
    # the selection key is the energy of the three high-frequency DCT coefficients (Eq. 1 with B = 4, Parseval), kept
    # in float32: against scipy's transform of the inputs it is off only by the storage rounding of the deviations
    Z = scipy.fft.dct(x64, type=2, norm="ortho", axis=0)
    hf = (Z[1:] ** 2).sum(axis=0)
    np.testing.assert_allclose(energy, hf, rtol=8 * tol, atol=8 * tol * hf.max())
    assert energy.dtype == np.float32
    if bf16:  # not rounded to the storage type: the key keeps its float32 mantissa
        assert not np.array_equal(synth.round_bf16(energy), energy)


def test_selection_is_top_k_energy_with_lowest_index_ties():
    x = _rand_layers(3, T=16, d=8)
    x[2][3] = x[2][5]  # make some equal energies likely
    _, _, energy = R4.depth_split4(x, False)
    e = energy.reshape(-1).copy()
    e[10] = e[40] = e[41] = e[7]  # forced ties
    for k in (0, 1, 5, 37, e.size):
        got = R.select_entries(e.reshape(energy.shape), k)
        order = np.lexsort((np.arange(e.size), -e.astype(np.float64)))
        want = np.sort(order[:k])
        assert np.array_equal(got, want)


def test_reconstruction_special_cases():
    x = _rand_layers(4)
    z0, dev, energy = R4.depth_split4(x, False)
    n = energy.size
    all_idx = np.arange(n, dtype=np.int32)
    none = np.zeros(0, dtype=np.int32)
    for l in range(4):
        full = R4.reconstruct4(z0, dev[l], all_idx, R4.RESIDUAL, x[l])
        np.testing.assert_allclose(full, x[l], rtol=0, atol=4 * np.finfo(np.float32).eps * np.abs(np.stack(x)).max())
        sh = R4.reconstruct4(z0, dev[l], none, R4.SHARED, x[l])
        np.testing.assert_array_equal(sh, 0.5 * z0.astype(np.float64))
        np.testing.assert_array_equal(R4.reconstruct4(z0, dev[l], none, R4.RESIDUAL, x[l]), sh)
        np.testing.assert_array_equal(R4.reconstruct4(z0, dev[l], all_idx, R4.EXACT, x[l]), x[l].astype(np.float64))
    # a kept position is restored, a dropped one is the block mean
    kept = np.array([3, 17], dtype=np.int32)
    r = R4.reconstruct4(z0, dev[1], kept, R4.RESIDUAL, x[1]).reshape(-1)
    assert r[3] == 0.5 * float(z0.reshape(-1)[3]) + float(dev[1].reshape(-1)[3])
    assert r[4] == 0.5 * float(z0.reshape(-1)[4])


def _probe_brute(dev, kept, q, group, h, pos):
    T, d = dev[0].shape
    keep = set(int(i) for i in kept)
    tot = [0.0, 0.0]
    for l in range(4):
        for g in range(group):
            for wi, p in enumerate(pos):
                for t in range(int(p) + 1):
                    a = b = 0.0
                    for c in range(d):
                        v = float(q[l][wi, h * group + g, c]) * float(dev[l][t, c])
                        a += v
                        if (t * d + c) not in keep:
                            b += v
                    tot[0] += (a / np.sqrt(d)) ** 2
                    tot[1] += (b / np.sqrt(d)) ** 2
    n = 4 * group * len(pos)
    return tot[0] / n, tot[1] / n


def test_probe_error_brute_force_and_invariants():
    T, d, G, Hq, W = 12, 4, 2, 4, 3
    g = np.random.default_rng(5)
    x = [(g.standard_normal((T, d))).astype(np.float32) for _ in range(4)]
    q = [g.standard_normal((W, Hq, d)).astype(np.float32) for _ in range(4)]
    pos = np.array([4, 8, 11], dtype=np.int32)
    z0, dev, energy = R4.depth_split4(x, False)
    kept = R.select_entries(energy, 9)
    for h in range(2):
        got = R4.probe_error4(dev, kept, q, G, h, pos)
        want = _probe_brute(dev, kept, q, G, h, pos)
        np.testing.assert_allclose(got, want, rtol=1e-12)
        assert got[1] <= got[0]
    assert R4.probe_error4(dev, np.arange(T * d, dtype=np.int32), q, G, 0, pos)[1] == 0.0
    e0 = R4.probe_error4(dev, np.zeros(0, np.int32), q, G, 0, pos)
    assert e0[0] == e0[1]


def test_block_with_repeated_pair_reduces_to_the_two_layer_oracle():
    # integer-valued layers keep every step exact: layers 2, 3 repeat layers 0, 1, so the deviation of layer l is
    # +-(x0 - x1) / 2 = +- c * z1 of the two-layer transform and Eq. 2 must agree between the two oracles
    T, d, G, Hq, W = 16, 8, 2, 4, 4
    g = np.random.default_rng(6)
    x0 = g.integers(-8, 9, (T, d)).astype(np.float32) * 2
    x1 = g.integers(-8, 9, (T, d)).astype(np.float32) * 2
    q0 = g.integers(-3, 4, (W, Hq, d)).astype(np.float32)
    q1 = g.integers(-3, 4, (W, Hq, d)).astype(np.float32)
    pos = np.array([3, 7, 12, 15], dtype=np.int32)
    z0_4, dev, energy = R4.depth_split4([x0, x1, x0, x1], False)
    np.testing.assert_array_equal(dev[0], (x0 - x1) / 2)
    np.testing.assert_array_equal(dev[1], (x1 - x0) / 2)
    np.testing.assert_array_equal(energy, (x0 - x1) ** 2)
    _, z1_2 = R.depth_split(x0, x1, False)
    k = 20
    kept4 = R.select_entries(energy, k)
    kept2 = R.select_entries(z1_2, k)
    assert np.array_equal(kept4, kept2)  # |z1| and the energy order positions the same way (ties included)
    for h in range(2):
        e4 = R4.probe_error4(dev, kept4, [q0, q1, q0, q1], G, h, pos)
        e2 = R.probe_error(z1_2, kept2, q0, q1, G, h, pos)
        np.testing.assert_allclose(e4, e2, rtol=1e-6)


def test_equal_layers_make_the_shared_candidate_exact():
    g = np.random.default_rng(7)
    T, d = 40, 8
    k = synth.round_bf16(g.standard_normal((T, d)).astype(np.float32))
    v = synth.round_bf16(g.standard_normal((T, d)).astype(np.float32))
    u = R4.Unit4([k] * 4, [v] * 4, True, 1, 8)
    assert all(np.all(dv == 0) for dv in u.dev["k"] + u.dev["v"])
    q = g.standard_normal((2, d)).astype(np.float32)
    for l in range(4):
        a = u.attend(R4.SHARED, l, q)
        b = u.attend(R4.EXACT, l, q)
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-12)
    # exact mode is plain attention over the layer's own rows, tails included
    u.append(2, k[0] * 2, v[0] * 3)
    rows_k = np.concatenate([k, (k[0] * 2)[None]], 0).astype(np.float64)
    rows_v = np.concatenate([v, (v[0] * 3)[None]], 0).astype(np.float64)
    s = rows_k @ q[0].astype(np.float64) / np.sqrt(d)
    p = np.exp(s - s.max())
    want = (p / p.sum()) @ rows_v
    np.testing.assert_allclose(u.attend(R4.EXACT, 2, q)[0], want, rtol=1e-10, atol=1e-12)


def test_omega_closed_form():
    om = R4.omega4(1000, 128, 2, 8000)
    assert om[2] == 1.0
    assert om[0] == 0.25
    np.testing.assert_allclose(om[1], 0.25 + 8000 * 12 / (4 * 1000 * 128 * 2))
    assert np.array_equal(R4.omega4(10, 4, 4, 0)[:2], [0.25, 0.25])


def test_unit4_on_the_synthetic_recipe():
    w = synth.WORKLOADS["tiny_b4"]
    ks = synth.block_tensor(w, 0, 0, 1, False)
    vs = synth.block_tensor(w, 0, 0, 1, True)
    u = R4.Unit4(ks, vs, False, w.keep_num, w.keep_den)
    assert u.kept["k"].size == w.k_keep and np.all(np.diff(u.kept["k"]) > 0)
    # needle tokens deviate most: their positions are over-represented among the kept entries
    needles = set(synth.needle_positions(w, 0, 0, 1).tolist())
    frac = np.mean([(i // w.head_dim) in needles for i in u.kept["k"]])
    assert frac > 5 * len(needles) / w.T
    q = synth.decode_q(w, 0, 1)[0].reshape(w.n_q_heads, w.head_dim)[w.group:2 * w.group]
    ex = u.attend(R4.EXACT, 1, q)
    rs = u.attend(R4.RESIDUAL, 1, q)
    sh = u.attend(R4.SHARED, 1, q)
    assert np.abs(rs - ex).max() <= np.abs(sh - ex).max() * 1.5 + 1e-9


def test_fold_of_a_block_of_four():
    g = np.random.default_rng(8)
    T, d, n_tail = 32, 8, 24
    mk = lambda *s: g.standard_normal(s).astype(np.float32)
    u = R4.Unit4([mk(T, d) for _ in range(4)], [mk(T, d) for _ in range(4)], False, 1, 4)
    rows = [[(mk(d), mk(d)) for _ in range(4)] for _ in range(n_tail)]
    for r in rows:
        for l in range(4):
            u.append(l, r[l][0], r[l][1])
    q = mk(2, d)
    before = [u.attend(R4.EXACT, l, q) for l in range(4)]
    u.fold(16, 1, 4)
    assert u.T == T + 16 and all(len(u.tail[("k", l)]) == 8 for l in range(4))
    for l in range(4):
        np.testing.assert_allclose(u.attend(R4.EXACT, l, q), before[l], rtol=1e-12, atol=1e-12)
    # the chunk keeps its own top-k by energy, inside the chunk, ascending overall
    xc = [np.stack([rows[t][l][0] for t in range(16)]) for l in range(4)]
    _, devc, ec = R4.depth_split4(xc, False)
    e = ec.reshape(-1).astype(np.float64)
    order = np.lexsort((np.arange(e.size), -e))
    want = np.sort(order[:(16 * d) // 4]) + T * d
    assert np.array_equal(u.kept["k"][(T * d) // 4:], want)
    np.testing.assert_array_equal(u.dev["k"][2][T:], devc[2])
    # shared mode: the folded tokens become the block mean
    got = u.rows("k", R4.SHARED, 1)[T:T + 16]
    np.testing.assert_allclose(got, np.mean(np.stack(xc).astype(np.float64), axis=0), rtol=1e-6, atol=1e-7)


# ---------------------------------------------------------------- the paper's token rule on blocks of four
def test_token_scores_of_a_block_literally_and_by_reduction():
    """s_t = max |Q (K_t - Khat_t^shared)^T| with K = F4^T Z and Khat^shared = F4^T [Z0; 0; 0; 0], both rebuilt through
    scipy's orthonormal DCT-II, against the oracle's shortcut K - Khat^shared = dev_l; and a block whose layers 2, 3 repeat
    layers 0, 1 must score like the pair oracle (dev = +-(x0 - x1) / 2 = +-c z1)."""
    T, d, G, Hq, W = 20, 8, 2, 4, 5
    g = np.random.default_rng(21)
    x = [g.standard_normal((T, d)).astype(np.float32) for _ in range(4)]
    q = [g.standard_normal((W, Hq, d)).astype(np.float32) for _ in range(4)]
    pos = np.array([3, 7, 12, 15, 19], dtype=np.int32)
    _, dev, _ = R4.depth_split4(x, False)
    x64 = np.stack([a.astype(np.float64) for a in x])
    Z = scipy.fft.dct(x64, type=2, norm="ortho", axis=0)
    Zs = Z.copy()
    Zs[1:] = 0.0
    K = scipy.fft.idct(Z, type=2, norm="ortho", axis=0)
    Ks = scipy.fft.idct(Zs, type=2, norm="ortho", axis=0)
    for h in range(2):
        want = np.zeros(T)
        for l in range(4):
            for gg in range(G):
                s = np.abs(q[l][:, h * G + gg, :].astype(np.float64) @ (K[l] - Ks[l]).T)
                want = np.maximum(want, np.where(np.arange(T)[None, :] <= pos[:, None], s, 0.0).max(axis=0))
        got = R4.token_scores4(dev, q, G, h, pos)
        np.testing.assert_allclose(got, want, rtol=2e-6, atol=2e-6 * np.abs(x64).max() * d)  # (float32 storage of dev)
        assert np.all(got[pos[-1] + 1:] == 0)
    # reduction to the pair oracle with integer-valued layers (every step exact)
    x0 = g.integers(-8, 9, (T, d)).astype(np.float32) * 2
    x1 = g.integers(-8, 9, (T, d)).astype(np.float32) * 2
    q0 = g.integers(-3, 4, (W, Hq, d)).astype(np.float32)
    q1 = g.integers(-3, 4, (W, Hq, d)).astype(np.float32)
    _, dev2, _ = R4.depth_split4([x0, x1, x0, x1], False)
    _, z1 = R.depth_split(x0, x1, False)
    for h in range(2):
        np.testing.assert_allclose(R4.token_scores4(dev2, [q0, q1, q0, q1], G, h, pos), R.token_scores(z1, q0, q1, G, h, pos), rtol=1e-6)


def test_unit4_under_the_token_rule():
    g = np.random.default_rng(22)
    T, d = 48, 8
    mk = lambda: g.standard_normal((T, d)).astype(np.float32)
    u = R4.Unit4([mk() for _ in range(4)], [mk() for _ in range(4)], False, 1, 4, select=False)
    tok = np.array([1, 5, 6, 20, 47], dtype=np.int32)
    u.use_tokens(tok)
    assert np.array_equal(u.kept["k"], u.kept["v"]) and u.kept["k"].size == tok.size * d
    for l in range(4):
        rows = u.rows("k", R4.RESIDUAL, l)
        np.testing.assert_allclose(rows[tok], u.x["k"][l][tok], rtol=0, atol=4e-7 * np.abs(np.stack(u.x["k"])).max())  # kept tokens restored
        other = np.setdiff1d(np.arange(T), tok)
        np.testing.assert_array_equal(rows[other], 0.5 * u.z0["k"][other].astype(np.float64))              # the rest is the block mean
    om = R4.omega4_tokens(1000, 128, 2, 62)
    np.testing.assert_allclose(om, [0.25, 0.25 + (2 * 4 * 62 * 128 * 2 + 4 * 62) / (8 * 1000 * 128 * 2), 1.0])
    # keeping every token restores every layer, keeping none is the shared cache
    u.use_tokens(np.arange(T))
    for l in range(4):
        np.testing.assert_allclose(u.rows("v", R4.RESIDUAL, l), u.x["v"][l], rtol=0, atol=4e-7 * np.abs(np.stack(u.x["v"])).max())
    u.use_tokens(np.zeros(0, np.int32))
    assert np.array_equal(u.rows("k", R4.RESIDUAL, 2), u.rows("k", R4.SHARED, 2))
