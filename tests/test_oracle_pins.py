"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Eq. 1: orthonormal transform -> round trip, Parseval, scipy's orthonormal DCT-II.
Eq. 3: S = everything is lossless, S = empty is the shared cache; selection against library sorts.
Eq. 2: E(exact) = 0, E(residual) = 0 at keep 1 and = E(shared) at keep 0; dense float64 brute force.
Decode: all-exact equals library attention; brute force; softmax invariants.
"""
import numpy as np
import pytest
import scipy.fft
import torch
from hypothesis import given, settings, strategies as st

import brute_force as bf
from oracle import fdkv_ref as R
from paper_2607_06519_b200 import synth

C = np.sqrt(0.5)


def _rand(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


# ---------------------------------------------------------------- Eq. 1
def test_f2_matches_scipy_orthonormal_dct2():
    x = np.random.default_rng(1).standard_normal((2, 37, 16))
    z0, z1 = R.depth_split_f64(x[0], x[1])
    ref = scipy.fft.dct(x, type=2, norm="ortho", axis=0)
    np.testing.assert_allclose(z0, ref[0], rtol=0, atol=1e-14)
    np.testing.assert_allclose(z1, ref[1], rtol=0, atol=1e-14)
    F = bf.dct_matrix(2)
    np.testing.assert_allclose(F, [[C, C], [C, -C]], atol=1e-15)
    np.testing.assert_allclose(F.T @ F, np.eye(2), atol=1e-15)


def test_round_trip_and_parseval():
    x = np.random.default_rng(2).standard_normal((2, 1000))
    z0, z1 = R.depth_split_f64(x[0], x[1])
    y0, y1 = R.depth_merge_f64(z0, z1)
    np.testing.assert_allclose(y0, x[0], atol=1e-14)
    np.testing.assert_allclose(y1, x[1], atol=1e-14)
    assert abs((x ** 2).sum() - (z0 ** 2).sum() - (z1 ** 2).sum()) < 1e-10


def test_stored_coefficients_arithmetic():
    x0, x1 = _rand((64, 16), 3), _rand((64, 16), 4)
    z0, z1 = R.depth_split(x0, x1, bf16=False)
    # fp32: add then multiply by the float32 nearest 1/sqrt(2); compare bit patterns with numpy float32 ops
    c32 = np.float32(C)
    assert c32.view(np.uint32) == 0x3F3504F3
    assert np.array_equal(z0.view(np.uint32), ((x0 + x1) * c32).view(np.uint32))
    assert np.array_equal(z1.view(np.uint32), ((x0 - x1) * c32).view(np.uint32))
    # close to the ideal transform
    i0, i1 = R.depth_split_f64(x0, x1)
    assert np.max(np.abs(z0 - i0)) <= 2e-7 * np.max(np.abs(i0))
    # bf16: rounding agrees with torch's round-to-nearest-even conversion
    b0, b1 = R.depth_split(synth.round_bf16(x0), synth.round_bf16(x1), bf16=True)
    s0, s1 = bf.stored_coefficients(synth.round_bf16(x0), synth.round_bf16(x1), bf16=True)
    assert np.array_equal(b0.view(np.uint32), s0.view(np.uint32))
    assert np.array_equal(b1.view(np.uint32), s1.view(np.uint32))
    assert np.all((b0.view(np.uint32) & 0xFFFF) == 0)


def test_exact_sum_cases():
    # x0 == x1 -> z1 == 0 exactly; x1 == -x0 -> z0 == 0
    x = _rand((33,), 5)
    z0, z1 = R.depth_split(x, x, bf16=False)
    assert np.all(z1 == 0)
    z0, z1 = R.depth_split(x, -x, bf16=False)
    assert np.all(z0 == 0)


# ---------------------------------------------------------------- selection
def _lexsort_select(z1, k):
    key = (z1.ravel().view(np.uint32) & 0x7FFFFFFF).astype(np.int64)
    order = np.lexsort((np.arange(key.size), -key))
    return np.sort(order[:k]).astype(np.int32)


@pytest.mark.parametrize("n,k", [(1000, 0), (1000, 1), (1000, 125), (1000, 999), (1000, 1000), (7, 3)])
def test_selection_vs_lexsort(n, k):
    z = _rand((n,), 10 + k)
    got = R.select_entries(z, k)
    assert np.array_equal(got, _lexsort_select(z, k))
    assert np.all(np.diff(got) > 0)
    if 0 < k < n:
        kept = np.zeros(n, bool)
        kept[got] = True
        assert np.abs(z[kept]).min() >= np.abs(z[~kept]).max()


def test_selection_ties_lowest_index_and_signed_zero():
    z = np.array([1.0, -1.0, 1.0, -1.0, 0.5, 1.0], dtype=np.float32)
    assert R.select_entries(z, 3).tolist() == [0, 1, 2]
    z = np.full(64, -2.0, dtype=np.float32)
    assert R.select_entries(z, 10).tolist() == list(range(10))
    z = np.array([0.0, -0.0, 0.0, -0.0], dtype=np.float32)
    assert R.select_entries(z, 2).tolist() == [0, 1]
    # heavily quantised values (bf16-like): many ties at the threshold
    q = synth.round_bf16(_rand((4096,), 11))
    got = R.select_entries(q, 512)
    assert np.array_equal(got, _lexsort_select(q, 512))
    assert np.array_equal(got, np.sort(np.flatnonzero(bf.kept_mask(q, 512).ravel())))


@settings(max_examples=40, deadline=None)
@given(st.integers(1, 300), st.integers(0, 300), st.integers(0, 2 ** 31 - 1), st.integers(1, 6))
def test_selection_property(n, k, seed, levels):
    k = min(k, n)
    rng = np.random.default_rng(seed)
    z = (rng.integers(-levels, levels + 1, n) * 0.25).astype(np.float32)
    got = R.select_entries(z, k)
    assert got.size == k
    assert np.array_equal(got, _lexsort_select(z, k))


# ---------------------------------------------------------------- Eq. 3 candidates
def test_keep_everything_is_lossless_and_keep_nothing_is_shared():
    x0, x1 = _rand((40, 8), 20), _rand((40, 8), 21)
    z0, z1 = R.depth_split(x0, x1, bf16=False)
    allidx = np.arange(z1.size, dtype=np.int32)
    for layer, x in ((0, x0), (1, x1)):
        rec = R.reconstruct(z0, z1, allidx, R.RESIDUAL, layer, x)
        assert np.max(np.abs(rec - x)) <= 2e-7 * np.max(np.abs(x))
        sh = R.reconstruct(z0, z1, allidx, R.SHARED, layer, x)
        none = R.reconstruct(z0, z1, np.zeros(0, np.int32), R.RESIDUAL, layer, x)
        assert np.array_equal(sh, none)
        np.testing.assert_allclose(sh, C * z0.astype(np.float64), rtol=1e-15)
        ex = R.reconstruct(z0, z1, allidx, R.EXACT, layer, x)
        assert np.array_equal(ex, x.astype(np.float64))
    # shared rows are identical for both layers of the pair
    assert np.array_equal(R.reconstruct(z0, z1, allidx, 0, 0, x0), R.reconstruct(z0, z1, allidx, 0, 1, x1))


def test_reconstruct_matches_dense_formula():
    x0, x1 = _rand((24, 8), 22), _rand((24, 8), 23)
    z0, z1 = R.depth_split(x0, x1, bf16=False)
    kept = R.select_entries(z1, 50)
    mask = bf.kept_mask(z1, 50)
    X_sh, X_rs, X_ex = bf.candidates(z0, z1, mask, (x0, x1))
    for layer, x in ((0, x0), (1, x1)):
        np.testing.assert_allclose(R.reconstruct(z0, z1, kept, 0, layer, x), X_sh[layer], atol=1e-14)
        np.testing.assert_allclose(R.reconstruct(z0, z1, kept, 1, layer, x), X_rs[layer], atol=1e-14)
        np.testing.assert_allclose(R.reconstruct(z0, z1, kept, 2, layer, x), X_ex[layer], atol=0)


# ---------------------------------------------------------------- Eq. 2
def _probe_case(T, d, G, Hkv, W, seed, k):
    x0, x1 = _rand((T, d), seed), _rand((T, d), seed + 1)
    z0, z1 = R.depth_split(x0, x1, bf16=False)
    q = (_rand((W, G * Hkv, d), seed + 2), _rand((W, G * Hkv, d), seed + 3))
    pos = np.sort(np.random.default_rng(seed + 4).choice(T, W, replace=False)).astype(np.int32)
    return z0, z1, q, pos, R.select_entries(z1, k), bf.kept_mask(z1, k)


@pytest.mark.parametrize("T,d,G,Hkv,W,k", [(40, 8, 2, 2, 5, 60), (17, 16, 1, 3, 4, 0), (33, 8, 4, 1, 7, 264)])
def test_probe_error_vs_bruteforce(T, d, G, Hkv, W, k):
    z0, z1, q, pos, kept, mask = _probe_case(T, d, G, Hkv, W, 30, k)
    for h in range(Hkv):
        e_sh, e_rs = R.probe_error(z1, kept, q[0], q[1], G, h, pos)
        b_sh, b_rs = bf.probe_errors(z0, z1, mask, q, G, h, pos)
        assert e_sh == pytest.approx(b_sh, rel=1e-10)
        assert e_rs == pytest.approx(b_rs, rel=1e-10, abs=1e-12)
        if k == 0:
            assert e_rs == e_sh
        if k == T * d:
            assert e_rs == 0.0
        assert e_rs <= e_sh


def test_probe_error_single_query_closed_form():
    # one layer-pair, G = 1, one probe query at the last position, z1 = one nonzero entry:
    # E = 1/(2*1*1) * (q0[c]^2 + q1[c]^2) * (C * v)^2 / d
    T, d = 6, 4
    z1 = np.zeros((T, d), np.float32)
    z1[2, 1] = 3.0
    q0 = _rand((1, 1, d), 40)
    q1 = _rand((1, 1, d), 41)
    e_sh, e_rs = R.probe_error(z1, np.zeros(0, np.int32), q0, q1, 1, 0, np.array([T - 1], np.int32))
    want = 0.5 * (float(q0[0, 0, 1]) ** 2 + float(q1[0, 0, 1]) ** 2) * (C * 3.0) ** 2 / d
    assert e_sh == pytest.approx(want, rel=1e-12)
    assert e_rs == pytest.approx(want, rel=1e-12)
    # the causal mask hides it from a query placed before token 2
    e_sh, _ = R.probe_error(z1, np.zeros(0, np.int32), q0, q1, 1, 0, np.array([1], np.int32))
    assert e_sh == 0.0
    # keeping that entry zeroes the residual-mode error
    _, e_rs = R.probe_error(z1, np.array([2 * d + 1], np.int32), q0, q1, 1, 0, np.array([T - 1], np.int32))
    assert e_rs == 0.0


def test_mode_rule():
    om = R.omega(512, 64, 4, 4096)
    np.testing.assert_allclose(om, [0.5, 0.625, 1.0])
    np.testing.assert_allclose(R.omega(32768, 128, 2, 262144), [0.5, 0.59375, 1.0])
    assert R.mode_rule(5.0, 1.0, om, 0.0)[0] == R.EXACT          # zero penalty: exact has zero error
    assert R.mode_rule(5.0, 1.0, om, 1e9)[0] == R.SHARED         # huge penalty: cheapest mode
    assert R.mode_rule(0.0, 0.0, om, 0.0)[0] == R.SHARED         # all tie -> lowest id
    assert R.mode_rule(1.0, 1.0, om, 0.0)[0] == R.EXACT
    m, loss, margin = R.mode_rule(100.0, 10.0, om, 100.0)
    np.testing.assert_allclose(loss, [150.0, 72.5, 100.0])
    assert m == R.RESIDUAL and margin == pytest.approx((100 - 72.5) / 100)
    # modes only move toward cheaper ids as lambda grows
    last = 2
    for lam in np.geomspace(1e-3, 1e6, 60):
        m = R.mode_rule(100.0, 10.0, om, lam)[0]
        assert m <= last
        last = m


# ---------------------------------------------------------------- decode attention
def test_all_exact_equals_library_attention():
    T, d, G = 77, 16, 3
    k0, k1, v0, v1 = (_rand((T, d), s) for s in (50, 51, 52, 53))
    u = R.Unit(k0, k1, v0, v1, bf16=False, keep_num=1, keep_den=4)
    q = _rand((G, d), 54)
    for layer, (k, v) in enumerate(((k0, v0), (k1, v1))):
        got = u.attend(R.EXACT, layer, q)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q).double()[None, :, None, :],
            torch.from_numpy(k).double()[None, None].expand(1, G, T, d),
            torch.from_numpy(v).double()[None, None].expand(1, G, T, d))[0, :, 0].numpy()
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_exact_tail_equals_attention_over_longer_context():
    T, d, n = 30, 8, 5
    full = [_rand((T + n, d), s) for s in (60, 61, 62, 63)]
    u = R.Unit(*(a[:T] for a in full), bf16=False, keep_num=1, keep_den=4)
    for j in range(n):
        u.append(0, full[0][T + j], full[2][T + j])
        u.append(1, full[1][T + j], full[3][T + j])
    q = _rand((2, d), 64)
    for mode in (R.SHARED, R.RESIDUAL, R.EXACT):
        for layer in (0, 1):
            got = u.attend(mode, layer, q)
            kh = u.rows("k", mode, layer)
            vh = u.rows("v", mode, layer)
            assert kh.shape == (T + n, d)
            assert np.array_equal(kh[T:], full[layer][T:].astype(np.float64))
            assert np.array_equal(vh[T:], full[2 + layer][T:].astype(np.float64))
            for g in range(2):
                np.testing.assert_allclose(got[g], bf.attention(kh, vh, q[g]), rtol=1e-12, atol=1e-14)
    ex = u.attend(R.EXACT, 1, q)
    np.testing.assert_allclose(ex[0], bf.attention(full[1].astype(np.float64), full[3].astype(np.float64), q[0]),
                               rtol=1e-12)


def test_attention_invariants():
    T, d = 50, 8
    kh = np.random.default_rng(70).standard_normal((T, d))
    vh = np.random.default_rng(71).standard_normal((T, d))
    q = _rand((d,), 72)
    out = R.attention(kh, vh, q)
    assert np.all(out <= vh.max(axis=0) + 1e-12) and np.all(out >= vh.min(axis=0) - 1e-12)
    # a constant added to every logit changes nothing: shift k along q's direction is not constant, so use
    # the one-token and uniform special cases instead
    np.testing.assert_allclose(R.attention(kh[:1], vh[:1], q), vh[0], rtol=1e-15)
    np.testing.assert_allclose(R.attention(np.zeros((T, d)), vh, q), vh.mean(axis=0), rtol=1e-13)
    # permuting the rows changes nothing
    perm = np.random.default_rng(73).permutation(T)
    np.testing.assert_allclose(R.attention(kh[perm], vh[perm], q), out, rtol=1e-12)


@settings(max_examples=25, deadline=None)
@given(st.integers(1, 40), st.sampled_from([8, 16]), st.sampled_from([1, 2, 4]), st.integers(0, 10 ** 6),
       st.sampled_from([(0, 1), (1, 8), (1, 2), (1, 1)]))
def test_oracle_vs_bruteforce_small_shapes(T, d, G, seed, keep):
    k0, k1, v0, v1 = (_rand((T, d), seed + i) for i in range(4))
    u = R.Unit(k0, k1, v0, v1, bf16=False, keep_num=keep[0], keep_den=keep[1])
    q = _rand((G, d), seed + 5)
    z0k, z1k = bf.stored_coefficients(k0, k1, False)
    z0v, z1v = bf.stored_coefficients(v0, v1, False)
    mk, mv = bf.kept_mask(z1k, u.k_keep), bf.kept_mask(z1v, u.k_keep)
    assert np.array_equal(np.flatnonzero(mk.ravel()), u.kept["k"])
    assert np.array_equal(np.flatnonzero(mv.ravel()), u.kept["v"])
    Kc = bf.candidates(z0k, z1k, mk, (k0, k1))
    Vc = bf.candidates(z0v, z1v, mv, (v0, v1))
    for mode in range(3):
        for layer in range(2):
            got = u.attend(mode, layer, q)
            for g in range(G):
                np.testing.assert_allclose(got[g], bf.attention(Kc[mode][layer], Vc[mode][layer], q[g]),
                                           rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- closed forms on the synthetic recipe
def test_recipe_variance_ratio_and_probe_scale():
    w = synth.WORKLOADS["tiny"].scaled(T=4096, n_needles=0, fixed_rho=0.8, W=16, name="cf")
    x0, x1 = synth.unit_tensor(w, 0, 0, 0, False)
    z0, z1 = R.depth_split(x0, x1, bf16=False)
    ratio = (z1.astype(np.float64).var(axis=0) / z0.astype(np.float64).var(axis=0)).mean()
    assert ratio == pytest.approx((1 - 0.8) / (1 + 0.8), rel=0.05)
    # E(shared) ~ (T - (W-1)/2) * (1-rho)/2 * mean_c sigma_c^2 for unit-variance queries
    sigma = synth.unit_sigma(w, 0, 0, 0, False).astype(np.float64)
    q0, q1 = synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1)
    pos = synth.probe_positions(w)
    e_sh, _ = R.probe_error(z1, np.zeros(0, np.int32), q0, q1, w.group, 0, pos)
    want = (w.T - (w.W - 1) / 2) * (1 - 0.8) / 2 * np.mean(sigma ** 2)
    assert e_sh == pytest.approx(want, rel=0.25)
    # the exact expectation given the drawn queries and the realised coefficients' second moments
    m2 = (z1.astype(np.float64) ** 2).mean(axis=0)
    qs = np.concatenate([q0[:, 0:w.group, :], q1[:, 0:w.group, :]], axis=1).astype(np.float64)
    want2 = (w.T - (w.W - 1) / 2) * 0.5 / w.head_dim * np.mean(np.sum(qs ** 2 * m2, axis=-1))
    assert e_sh == pytest.approx(want2, rel=0.1)


# ---------------------------------------------------------------- the paper's qualitative claim
def test_residual_restores_a_needle_that_sharing_loses():
    w = synth.WORKLOADS["tiny"]
    k0, k1 = synth.unit_tensor(w, 0, 0, 0, False)
    v0, v1 = synth.unit_tensor(w, 0, 0, 0, True)
    u = R.Unit(k0, k1, v0, v1, bf16=False, keep_num=1, keep_den=8)
    t = int(synth.needle_positions(w, 0, 0, 0)[3])
    q = (k1[t] / np.linalg.norm(k1[t]) * 8.0).astype(np.float32)[None]
    ex = u.attend(R.EXACT, 1, q)[0]
    sh = u.attend(R.SHARED, 1, q)[0]
    rs = u.attend(R.RESIDUAL, 1, q)[0]
    err = lambda a: np.max(np.abs(a - ex)) / np.max(np.abs(ex))
    assert err(sh) > 0.3
    assert err(rs) < 0.25 * err(sh)


# ---------------------------------------------------------------- the paper's token rule
def test_token_rule_vs_bruteforce_and_needles():
    w = synth.WORKLOADS["tiny"]
    pos = synth.probe_positions(w)
    q = (synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1))
    for h in range(w.n_kv_heads):
        k0, k1 = synth.unit_tensor(w, 0, 0, h, False)
        z0, z1 = R.depth_split(k0, k1, bf16=False)
        s = R.token_scores(z1, q[0], q[1], w.group, h, pos)
        # literal form: |Q (K_t - Khat_t^shared)^T| with both key matrices rebuilt through the DCT matrix; the
        # difference of two O(|z0|) reconstructions costs a few ulps of |Q| |z0|, hence the absolute term
        lit = bf.token_scores(z0, z1, q, w.group, h, pos)
        np.testing.assert_allclose(s, lit, rtol=1e-12, atol=1e-12 * float(np.abs(z0).max()) * w.head_dim)
        tok = R.select_tokens(s, w.T // 8)
        order = np.lexsort((np.arange(w.T), -s))
        assert np.array_equal(tok, np.sort(order[: w.T // 8]))
        assert set(synth.needle_positions(w, 0, 0, h).tolist()) <= set(tok.tolist())


def test_token_score_closed_form_single_entry():
    # one non-zero high-frequency coefficient a at (t0, c0): K_t - Khat_t^shared = +-a/sqrt(2) e_c0 in the two layers,
    # so s_t0 = max_q |Q[q][c0]| * |a| / sqrt(2) over the queries at positions >= t0, and every other token scores 0
    T, d, G, Hq, W = 10, 4, 2, 2, 3
    z1 = np.zeros((T, d), dtype=np.float32)
    t0, c0, a = 6, 2, -3.0
    z1[t0, c0] = a
    g = np.random.default_rng(11)
    q0 = g.standard_normal((W, Hq, d)).astype(np.float32)
    q1 = g.standard_normal((W, Hq, d)).astype(np.float32)
    pos = np.array([2, 6, 9], dtype=np.int32)   # the query at position 2 cannot see token 6
    s = R.token_scores(z1, q0, q1, G, 0, pos)
    want = max(abs(float(q[w_, g_, c0])) for q in (q0, q1) for g_ in range(G) for w_ in (1, 2)) * abs(a) * np.sqrt(0.5)
    assert s[t0] == pytest.approx(want, rel=1e-12)
    assert np.count_nonzero(s) == 1


# ---------------------------------------------------------------- token-granular residual (the paper's own rule)
def test_token_rule_candidates_probe_and_attention_vs_bruteforce():
    w = synth.WORKLOADS["tiny"]
    pos = synth.probe_positions(w)
    pq = (synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1))
    h = 1
    k0, k1 = synth.unit_tensor(w, 0, 0, h, False)
    v0, v1 = synth.unit_tensor(w, 0, 0, h, True)
    u = R.Unit(k0, k1, v0, v1, False, 1, 8, select=False)
    s = R.token_scores(u.z1["k"], pq[0], pq[1], w.group, h, pos)
    tok = R.select_tokens(s, u.k_tok)
    assert tok.size == w.T // 8 and np.all(np.diff(tok) > 0)
    u.use_tokens(tok)
    mask = np.zeros((w.T, w.head_dim))
    mask[tok] = 1.0  # Eq. 3's indicator 1[t in S]: whole rows
    assert np.array_equal(np.flatnonzero(mask.ravel()), u.kept["k"])
    e_sh, e_rs = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, pos)
    b_sh, b_rs = bf.probe_errors(u.z0["k"], u.z1["k"], mask, pq, w.group, h, pos)
    assert e_sh == pytest.approx(b_sh, rel=1e-10) and e_rs == pytest.approx(b_rs, rel=1e-10)
    assert e_rs < e_sh
    Kc = bf.candidates(u.z0["k"], u.z1["k"], mask, (k0, k1))
    Vc = bf.candidates(u.z0["v"], u.z1["v"], mask, (v0, v1))
    q = synth.decode_q(w, 0, 1)[0][h * w.group:(h + 1) * w.group]
    got = u.attend(R.RESIDUAL, 1, q)
    for g in range(w.group):
        np.testing.assert_allclose(got[g], bf.attention(Kc[1][1], Vc[1][1], q[g]), rtol=1e-10, atol=1e-12)
    # memory cost of the token form: rows of K and V plus one index per token
    om = R.omega_tokens(w.T, w.head_dim, 4, u.k_tok)
    Td = w.T * w.head_dim
    np.testing.assert_allclose(om, [0.5, (2 * Td * 4 + 2 * u.k_tok * w.head_dim * 4 + 4 * u.k_tok) / (4 * Td * 4), 1.0])
    # keeping every token is lossless, keeping none is the shared cache
    u.use_tokens(np.arange(w.T))
    assert np.max(np.abs(u.rows("k", R.RESIDUAL, 1) - k1)) <= 2e-7 * np.max(np.abs(k1))
    u.use_tokens(np.zeros(0, np.int32))
    assert np.array_equal(u.rows("k", R.RESIDUAL, 0), u.rows("k", R.SHARED, 0))


# ---------------------------------------------------------------- budgeted routing
def test_route_budget_scan_brackets_the_smallest_lambda_that_fits():
    rng = np.random.default_rng(90)
    n = 40
    e_sh = rng.lognormal(3.0, 1.0, n)
    e_rs = e_sh * rng.uniform(0.05, 0.4, n)
    om = R.omega(32768, 128, 2, 262144)
    unit = 4.0 * 32768 * 128 * 2

    def footprint(lam):
        return sum(om[R.mode_rule(a, b, om, lam)[0]] * unit for a, b in zip(e_sh, e_rs))

    # footprint is monotone non-increasing in lambda (the premise of "increase lambda until it fits")
    grid = np.concatenate([[0.0], np.geomspace(1e-3, 1e6, 400)])
    fp = np.array([footprint(l) for l in grid])
    assert np.all(np.diff(fp) <= 1e-6)
    # the analytic threshold: the footprint only changes where two loss lines of a unit cross
    cross = np.concatenate([(e_sh - e_rs) / (om[1] - om[0]), e_rs / (om[2] - om[1]), e_sh / (om[2] - om[0])])
    for frac in (1.0, 0.9, 0.7, 0.6, 0.55, 0.5):
        budget = frac * n * unit
        fits, lam, modes, prev = R.route_budget(e_sh, e_rs, om, unit, budget)
        assert fits
        assert footprint(lam) <= budget
        assert [R.mode_rule(a, b, om, lam)[0] for a, b in zip(e_sh, e_rs)] == modes.tolist()
        if lam > 0:
            assert footprint(prev) > budget and prev < lam <= max(prev * (1 + 2.0 ** -11), 1e-9)
            assert not np.any((grid <= prev) & (fp <= budget))
            assert np.any((cross > prev) & (cross <= lam))         # a crossing inside the bracket explains the step
        else:
            assert np.all(modes == R.EXACT) and prev == -1.0
    # below the all-shared footprint nothing fits
    fits, lam, modes, _ = R.route_budget(e_sh, e_rs, om, unit, 0.49 * n * unit)
    assert not fits and np.isinf(lam) and np.all(modes == 0)
    # one unit, by hand: shared<->residual crossing at (100-10)/(0.59375-0.5) = 960, residual<->exact at 10/0.40625
    fits, lam, modes, prev = R.route_budget([100.0], [10.0], om, unit, 0.6 * unit)
    assert fits and modes.tolist() == [1] and prev < 10.0 / (1 - 0.59375) <= lam
    fits, lam, modes, prev = R.route_budget([100.0], [10.0], om, unit, 0.5 * unit)
    assert fits and modes.tolist() == [0] and prev < 90.0 / 0.09375 <= lam and lam / prev < 1.001


# ---------------------------------------------------------------------------------------------------------
# folding generated tokens into the compressed form (the optional refresh of the Method's last paragraph)
# ---------------------------------------------------------------------------------------------------------
def _unit_with_tail(seed, T=48, d=8, n_tail=40, bf16=False, keep=(1, 4)):
    g = np.random.default_rng(seed)
    mk = lambda *s: (synth.round_bf16(g.standard_normal(s).astype(np.float32)) if bf16 else g.standard_normal(s).astype(np.float32))
    u = R.Unit(mk(T, d), mk(T, d), mk(T, d), mk(T, d), bf16, *keep)
    rows = [(mk(d), mk(d), mk(d), mk(d)) for _ in range(n_tail)]
    for k0, k1, v0, v1 in rows:
        u.append(0, k0, v0)
        u.append(1, k1, v1)
    return u, rows


def test_fold_leaves_exact_mode_unchanged_and_moves_rows():
    u, rows = _unit_with_tail(21)
    q = np.random.default_rng(1).standard_normal((2, 8)).astype(np.float32)
    before = [u.attend(R.EXACT, l, q) for l in range(2)]
    T0 = u.T
    u.fold(32, 1, 4)
    assert u.T == T0 + 32 and len(u.tail[("k", 0)]) == 8 and len(u.tail[("v", 1)]) == 8
    for l in range(2):
        np.testing.assert_allclose(u.attend(R.EXACT, l, q), before[l], rtol=1e-12, atol=1e-12)
    # the chunk keeps its own top-k: floor(32 * 8 / 4) entries, all inside the chunk, ascending overall
    for name in ("k", "v"):
        kept = u.kept[name]
        assert kept.size == (T0 * 8) // 4 + (32 * 8) // 4
        assert np.all(np.diff(kept) > 0)
        assert np.all(kept[(T0 * 8) // 4:] >= T0 * 8)


def test_fold_chunk_selection_is_the_chunks_own_top_k():
    u, rows = _unit_with_tail(22, T=32, d=8, n_tail=16)
    u.fold(16, 1, 4)
    k0 = np.stack([r[0] for r in rows])
    k1 = np.stack([r[1] for r in rows])
    _, z1c = R.depth_split(k0, k1, False)
    mag = np.abs(z1c.reshape(-1)).astype(np.float64)
    order = np.lexsort((np.arange(mag.size), -mag))
    want = np.sort(order[:(16 * 8) // 4]) + 32 * 8
    assert np.array_equal(u.kept["k"][(32 * 8) // 4:], want)
    # stored coefficients of the chunk are Eq. 1 of the chunk's rows
    np.testing.assert_array_equal(u.z1["k"][32:], z1c)


def test_fold_with_everything_kept_is_lossless_in_residual_mode():
    u, rows = _unit_with_tail(23, keep=(1, 1))
    q = np.random.default_rng(2).standard_normal((1, 8)).astype(np.float32)
    ex = u.attend(R.EXACT, 1, q)
    u.fold(40, 1, 1)
    np.testing.assert_allclose(u.attend(R.RESIDUAL, 1, q), ex, rtol=1e-5, atol=1e-6)


def test_fold_in_shared_mode_replaces_tail_rows_by_the_pair_mean():
    u, rows = _unit_with_tail(24, n_tail=16)
    u.fold(16, 1, 4)
    got = u.rows("k", R.SHARED, 0)[48:]
    want = np.stack([(r[0].astype(np.float64) + r[1].astype(np.float64)) / 2 for r in rows])
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-7)
