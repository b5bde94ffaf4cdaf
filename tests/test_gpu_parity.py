"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs.
Integers (indices, modes) and stored coefficients bit-exact; attention within max|d|/max|ref| <= 1e-3 (fp32
storage) or 2e-2 (bf16 storage) per output vector; probe errors within 1e-4 relative."""
import numpy as np
import pytest
import torch

from gpu_util import TOL, check_compression, f32, oracle_layer_out, oracle_unit, vector_errors
from oracle import fdkv_ref as R
from paper_2607_06519_b200 import synth

pytestmark = pytest.mark.gpu

LAMBDAS = [0.0, 50.0, 300.0, 3000.0, 1e4]


def _runner():
    from paper_2607_06519_b200 import runner
    return runner


def _decode_all_layers(pf, w, modes, units, step=0, append=False, out_dtype=None):
    worst = 0.0
    for layer in range(w.n_layers):
        q = pf.decode_q(layer, step)
        kn = vn = None
        if append:
            kn, vn = pf.new_rows(layer, step)
            for (b, p, h), u in units.items():
                if p == layer // 2:
                    u.append(layer & 1, f32(kn)[b, h], f32(vn)[b, h])
        out = pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=out_dtype)
        torch.cuda.synchronize()
        got = f32(out)
        for b in range(w.batch):
            us = {h: units[(b, layer // 2, h)] for h in range(w.n_kv_heads) if (b, layer // 2, h) in units}
            ref = oracle_layer_out(us, modes[b][layer // 2], w, layer, f32(q)[b])
            heads = [i for h in us for i in range(h * w.group, (h + 1) * w.group)]
            err = vector_errors(got[b][heads], ref[heads])
            worst = max(worst, float(err.max()))
    return worst


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_tiny_compress_probe_decode(dtype):
    runner = _runner()
    w = synth.WORKLOADS["tiny"].scaled(dtype=dtype)
    units = {(0, 0, h): oracle_unit(w, 0, 0, h) for h in range(w.n_kv_heads)}
    om = R.omega(w.T, w.head_dim, 2 if dtype == "bf16" else 4, w.k_keep)
    pq = (synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1))
    pos = synth.probe_positions(w)
    e_ref = np.array([R.probe_error(units[(0, 0, h)].z1["k"], units[(0, 0, h)].kept["k"], pq[0], pq[1], w.group, h, pos)
                      for h in range(w.n_kv_heads)])
    for forced in ("probe", [[0, 0]], [[1, 1]], [[2, 2]], [[1, 2]], [[0, 1]]):
        pf = runner.Prefilled(w)
        pf.compress(0)
        for h in range(w.n_kv_heads):
            check_compression(pf.ctx, w, 0, 0, h, units[(0, 0, h)])
        if forced == "probe":
            for lam in LAMBDAS:
                modes, scores = pf.probe(0, lam)
                np.testing.assert_allclose(scores[0], e_ref, rtol=1e-4)
                want = [R.mode_rule(e_ref[h, 0], e_ref[h, 1], om, lam)[0] for h in range(w.n_kv_heads)]
                assert modes[0].tolist() == want
                assert min(R.mode_rule(e_ref[h, 0], e_ref[h, 1], om, lam)[2] for h in range(2)) > 1e-3
            pf.probe(0, 300.0)
            modes = np.array([[1, 1]])
        else:
            modes = np.array(forced)
            pf.ctx.set_modes(0, modes)
        pf.commit(0)
        assert np.array_equal(pf.ctx.get_modes(0).numpy(), modes)
        worst = _decode_all_layers(pf, w, [modes], units, out_dtype=0)
        assert worst <= TOL[dtype], (forced, worst)
        assert pf.ctx.device_status() == 0
        pf.ctx.close()


@pytest.mark.parametrize("dtype,T,d,Hq,Hkv,keep,tail", [
    ("f32", 517, 64, 4, 2, (1, 8), 3),      # ragged T
    ("bf16", 517, 128, 8, 2, (1, 16), 5),   # ragged T, G = 4, d = 128
    ("bf16", 19, 64, 2, 2, (1, 4), 2),      # shorter than one tile, G = 1
    ("f32", 96, 128, 8, 1, (0, 1), 1),      # keep nothing: residual == shared
    ("bf16", 100, 64, 8, 1, (1, 1), 0),     # keep everything, G = 8
    ("bf16", 2100, 128, 4, 1, (1, 32), 40), # several splits, tail longer than a tile
    ("bf16", 5003, 128, 8, 2, (1, 16), 2),  # CTA ranges cut on 16-token slices: partial last tiles, T not a multiple of 16
    ("bf16", 9000, 128, 12, 3, (1, 8), 3),  # three units, ranges of a few slices over one tile, dense lists
])
def test_shapes_and_edges(dtype, T, d, Hq, Hkv, keep, tail):
    runner = _runner()
    w = synth.Workload(name="edge", n_layers=2, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, batch=1, T=T, dtype=dtype,
                       keep_num=keep[0], keep_den=keep[1], n_needles=min(4, T), W=min(8, T), seed=7,
                       n_steps=max(tail, 1))
    pf = runner.Prefilled(w, max_tail=max(tail, 1))
    pf.compress(0)
    units = {(0, 0, h): check_compression(pf.ctx, w, 0, 0, h) for h in range(Hkv)}
    modes = np.array([[(h + 1) % 3 for h in range(Hkv)]])
    pmodes, scores = pf.probe(0, 1.0)
    pq = (synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1))
    for h in range(Hkv):
        u = units[(0, 0, h)]
        e = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, synth.probe_positions(w))
        np.testing.assert_allclose(scores[0, h], e, rtol=1e-4, atol=1e-12)
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    for step in range(max(tail, 1)):
        worst = _decode_all_layers(pf, w, [modes], units, step=step, append=tail > 0)
        assert worst <= TOL[dtype], (step, worst)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_selection_with_massive_ties():
    """Heavily quantised inputs: the threshold bucket holds most entries; ties go to the lowest flat index."""
    runner = _runner()
    from paper_2607_06519_b200 import binding as B
    T, d, H = 300, 64, 2
    rng = np.random.default_rng(5)
    for dtype, tdt in (("f32", torch.float32), ("bf16", torch.bfloat16)):
        cfg = B.Config(2, 2, H, d, 1, T, 1, B.BF16 if dtype == "bf16" else B.F32, 3, 7)
        ctx = B.Context(cfg)
        xs = [(rng.integers(-2, 3, (T, H, d)) * 0.5).astype(np.float32) for _ in range(4)]
        dev = [torch.from_numpy(x).cuda().to(tdt) for x in xs]
        ctx.compress_prefill(0, 0, 1, T, [dev[0], dev[1]], [dev[2], dev[3]])
        for h in range(H):
            for is_v in (0, 1):
                z0, z1 = R.depth_split(xs[2 * is_v][:, h], xs[2 * is_v + 1][:, h], dtype == "bf16")
                kept = R.select_entries(z1, (T * d * 3) // 7)
                idx, val = ctx.get_residual(0, 0, h, is_v)
                assert np.array_equal(idx.cpu().numpy(), kept)
                assert np.array_equal(f32(val).view(np.uint32), z1.ravel()[kept].view(np.uint32))
        assert ctx.device_status() == 0
        ctx.close()


def test_llama_shaped_reduced():
    """Llama-3-8B head geometry (32 query / 8 KV heads, d = 128, bf16), 2 pairs, a few thousand tokens with a
    ragged end, mixed modes, decode with appends: every output vector of every layer."""
    runner = _runner()
    w = synth.WORKLOADS["decode32k"].scaled(n_layers=4, T=4096 + 37, n_needles=16, n_steps=3, name="reduced")
    pf = runner.Prefilled(w, max_tail=8)
    pf.compress(0)
    units = {}
    for p in range(w.n_pairs):
        for h in range(w.n_kv_heads):
            units[(0, p, h)] = check_compression(pf.ctx, w, 0, p, h)
    pmodes, scores = pf.probe(0, 100.0)
    pos = synth.probe_positions(w)
    for p in range(w.n_pairs):
        pq = (synth.probe_q(w, 0, 2 * p), synth.probe_q(w, 0, 2 * p + 1))
        for h in (0, 5):
            u = units[(0, p, h)]
            e = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, pos)
            np.testing.assert_allclose(scores[p, h], e, rtol=1e-4)
    modes = synth.quota_modes(scores[..., 0])
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    by_mode, exact_equiv = pf.ctx.footprint(0)
    assert exact_equiv == 4 * w.T * w.head_dim * 2 * w.n_pairs * w.n_kv_heads
    assert sum(by_mode) < exact_equiv
    for step in range(3):
        worst = _decode_all_layers(pf, w, [modes], units, step=step, append=True)
        assert worst <= TOL["bf16"], (step, worst)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_budgeted_routing_matches_oracle():
    """Smallest lambda that fits a byte budget: the library's search on its own probe errors against the oracle's
    search on the oracle's errors (same modes; lambda equal up to the probe errors' float32 accumulation)."""
    runner = _runner()
    w = synth.WORKLOADS["decode32k"].scaled(n_layers=8, T=1024 + 5, n_needles=8, name="budget")
    pf = runner.Prefilled(w, max_tail=1)
    pf.compress(0)
    pf.probe(0, 0.0)
    pos = synth.probe_positions(w)
    e = np.zeros((w.n_pairs, w.n_kv_heads, 2))
    for p in range(w.n_pairs):
        pq = (synth.probe_q(w, 0, 2 * p), synth.probe_q(w, 0, 2 * p + 1))
        for h in range(w.n_kv_heads):
            u = oracle_unit(w, 0, p, h)
            e[p, h] = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, pos)
    om = R.omega(w.T, w.head_dim, 2, w.k_keep)
    unit_bytes = 4.0 * w.T * w.head_dim * 2
    n = w.n_pairs * w.n_kv_heads
    for frac in (1.0, 0.8, 0.62, 0.55, 0.5):
        budget = int(frac * n * unit_bytes)
        fits, lam, modes = pf.ctx.route_budget(0, budget)
        rf, rl, rm, rprev = R.route_budget(e[..., 0], e[..., 1], om, unit_bytes, budget)
        assert fits and rf
        # the library's lambda routes, under the oracle's rule and errors, as the library says and fits.  The library
        # stops a hair past one unit's crossing computed from ITS errors (float32 accumulation, 1e-6 off the oracle's),
        # so that unit's decision is compared a relative 1e-4 to either side of lambda.
        got = modes.numpy().ravel().tolist()
        lo = [R.mode_rule(a, b, om, lam * (1 - 1e-4))[0] for a, b in e.reshape(-1, 2)]
        hi = [R.mode_rule(a, b, om, lam * (1 + 1e-4))[0] for a, b in e.reshape(-1, 2)]
        assert all(g in (l, h) for g, l, h in zip(got, lo, hi)), frac
        assert sum(l != h for l, h in zip(lo, hi)) <= 2
        assert sum(om[m] for m in got) * unit_bytes <= budget
        # ... and is the smallest such: it lies in the bracket of the oracle's upward scan (previous grid value does not
        # fit, the next does), up to the float32 accumulation of the library's probe errors
        assert (rprev if rprev > 0 else 0.0) * (1 - 1e-4) <= lam <= rl * (1 + 1e-4) + 1e-12, (frac, rprev, lam, rl)
    fits, lam, modes = pf.ctx.route_budget(0, int(0.4 * n * unit_bytes))
    assert not fits and np.isinf(lam) and int(modes.sum()) == 0
    fits, lam, modes = pf.ctx.route_budget(0, int(0.62 * n * unit_bytes))
    pf.commit(0)  # commit packs the budgeted modes
    assert np.array_equal(pf.ctx.get_modes(0).numpy(), modes.numpy())
    by_mode, exact_equiv = pf.ctx.footprint(0)
    assert exact_equiv == int(n * unit_bytes)
    pf.ctx.close()
