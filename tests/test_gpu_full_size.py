"""Parity at the benchmark's sizes, through the same calls and launch configuration bench.py times.

Full-size inputs cannot be checked element by element on the CPU in minutes, so each test checks SAMPLED units /
output vectors against the oracle (which regenerates just those units from their seeds):
 * decode32k  : the benchmark workload itself (32 layers, 32k, bf16, quota mode mix), one decode step.
 * decode128k : 32 layers, 131072 tokens, keep 1/32, 256 needles per head, one decode step.
 * batch8     : 32 layers, 8 sequences x 32k, 128 decode steps appending to the tails, checked at steps 0, 1, 63, 127.
"""
import numpy as np
import pytest
import torch

from gpu_util import TOL, check_compression, f32, oracle_unit, vector_errors
from oracle import fdkv_ref as R
from paper_2607_06519_b200 import synth

pytestmark = pytest.mark.gpu


def _pick_units(modes, b, per_mode):
    """Units (b, pair, head) of one sequence covering every mode: per_mode[m] units of mode m, spread over the pairs."""
    picked = []
    for m, n in enumerate(per_mode):
        cand = [(int(p), int(h)) for p, h in zip(*np.nonzero(modes == m))]
        assert len(cand) >= n, f"mode {m}: {len(cand)} units, wanted {n}"
        step = max(1, len(cand) // max(n, 1))
        picked += [(b, p, h) for (p, h) in cand[::step][:n]]
    return picked


def _prefill(w, seqs, per_mode, n_probe):
    """Compresses, probes and commits the sequences with the benchmark's quota mode mix.  The sampled units are chosen
    AFTER the modes are known, per_mode[b] = (shared, residual, exact) counts for sequence b, so that every test checks
    each reconstruction path; the first n_probe sampled units of a sequence also have their probe errors compared."""
    from paper_2607_06519_b200 import binding as B, runner

    pf = runner.Prefilled(w, max_tail=max(w.n_steps, 1))
    units, modes_all = {}, []
    pos = synth.probe_positions(w)
    tc_before, portable_before = B.kernel_launch_count(B.KERNEL_PROBE_TC), B.kernel_launch_count(B.KERNEL_PROBE_PORTABLE)
    for b in seqs:
        pf.compress(b)
        pmodes, scores = pf.probe(b, 0.0)
        modes = synth.quota_modes(scores[..., 0])
        sample = _pick_units(modes, b, per_mode.get(b, (0, 0, 0)))
        for i, (sb, p, h) in enumerate(sample):
            u = units[(b, p, h)] = check_compression(pf.ctx, w, b, p, h)
            if i < n_probe:
                e = R.probe_error(u.z1["k"], u.kept["k"], synth.probe_q(w, b, 2 * p), synth.probe_q(w, b, 2 * p + 1), w.group,
                                  h, pos)
                np.testing.assert_allclose(scores[p, h], e, rtol=1e-4)
        pf.ctx.set_modes(b, modes)
        pf.commit(b)
        modes_all.append(modes)
    # bf16 storage with head_dim 128: the tcgen05 probe served every call, the portable kernel none
    assert B.kernel_launch_count(B.KERNEL_PROBE_TC) - tc_before == len(seqs)
    assert B.kernel_launch_count(B.KERNEL_PROBE_PORTABLE) == portable_before
    for b, want in per_mode.items():
        got = np.bincount([int(modes_all[seqs.index(b)][p][h]) for (sb, p, h) in units if sb == b], minlength=3)
        assert tuple(got) == tuple(want), (b, got)
    torch.cuda.empty_cache()
    return pf, units, modes_all


def _check_layer(pf, w, layer, step, units, modes_all, q, out):
    worst = 0.0
    got, qh = f32(out), f32(q)
    for (b, p, h), u in units.items():
        if p != layer // 2:
            continue
        G = w.group
        ref = u.attend(int(modes_all[b][p][h]), layer & 1, qh[b][h * G:(h + 1) * G])
        err = vector_errors(got[b][h * G:(h + 1) * G], ref)
        worst = max(worst, float(err.max()))
    return worst


def test_decode32k_benchmark_workload():
    from paper_2607_06519_b200 import binding as B

    w = synth.WORKLOADS["decode32k"]
    pf, units, modes_all = _prefill(w, [0], {0: (3, 3, 2)}, 2)
    assert sorted(np.bincount(modes_all[0].ravel(), minlength=3).tolist()) == sorted([64, 45, 19])
    assert len(units) == 8
    fast_before, portable_before = B.kernel_launch_count(B.KERNEL_DECODE_FAST), B.kernel_launch_count(B.KERNEL_DECODE_PORTABLE)
    stream = torch.cuda.Stream()
    worst = 0.0
    with torch.cuda.stream(stream):
        for layer in range(w.n_layers):
            q = pf.decode_q(layer, 0)
            out = pf.ctx.decode_attn(layer, q, stream=stream)
            stream.synchronize()
            assert torch.isfinite(out.float()).all()
            worst = max(worst, _check_layer(pf, w, layer, 0, units, modes_all, q, out))
    assert worst <= TOL["bf16"], worst
    assert B.kernel_launch_count(B.KERNEL_DECODE_FAST) - fast_before == w.n_layers
    assert B.kernel_launch_count(B.KERNEL_DECODE_PORTABLE) == portable_before
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_prefill32k_probe_errors_and_modes_of_every_unit():
    """The prefill workload at full size: the probe errors of all 128 units against the oracle's (computed once by
    tests/golden/make_probe_errors_32k.py, oracle only), and the modes the rule of Eq. 3 assigns at the calibrated
    lambda*, at lambda* / 64 (mostly exact) and at lambda* x 64 (all shared) -- bit-exact, at lambdas whose smallest
    loss margin is at least 1e-3 so that the float32 accumulation of the GPU errors cannot flip a decision."""
    import json
    import os

    from paper_2607_06519_b200 import runner

    g = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "probe_errors_decode32k.json")))
    w = synth.WORKLOADS["prefill32k"]
    pf = runner.Prefilled(w, max_tail=1)
    pf.compress(0)
    e_ref = np.stack([np.asarray(g["e_shared"]), np.asarray(g["e_residual"])], axis=-1)
    seen = set()
    for case in g["cases"]:
        assert case["min_margin"] >= 1e-3
        pmodes, scores = pf.probe(0, case["lambda"])
        np.testing.assert_allclose(scores, e_ref, rtol=1e-4)
        assert pmodes.ravel().tolist() == case["modes"], case["name"]
        seen |= set(case["modes"])
    assert seen == {0, 1, 2}
    # the probe's modes are what commit packs
    pf.commit(0)
    assert pf.ctx.get_modes(0).numpy().ravel().tolist() == g["cases"][-1]["modes"]
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_decode128k_long_context():
    w = synth.WORKLOADS["decode128k"]
    pf, units, modes_all = _prefill(w, [0], {0: (1, 2, 1)}, 1)
    assert len(units) == 4
    worst = 0.0
    for layer in range(w.n_layers):
        q = pf.decode_q(layer, 0)
        out = pf.ctx.decode_attn(layer, q)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        worst = max(worst, _check_layer(pf, w, layer, 0, units, modes_all, q, out))
    assert worst <= TOL["bf16"], worst
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_batch8_decode_with_tail_appends():
    w = synth.WORKLOADS["batch8"]
    # one unit of each mode, from three different sequences
    pf, units, modes_all = _prefill(w, list(range(w.batch)), {0: (1, 0, 0), 3: (0, 1, 0), 7: (0, 0, 1)}, 0)
    assert sorted(int(modes_all[b][p][h]) for (b, p, h) in units) == [0, 1, 2]
    # generated-token rows of every (sequence, pair, head): [steps, d] for both layers, K and V
    rows = {}
    for b in range(w.batch):
        for p in range(w.n_pairs):
            for h in range(w.n_kv_heads):
                rows[(b, p, h)] = (synth.tail_rows(w, b, p, h, False), synth.tail_rows(w, b, p, h, True))
    dq = {(b, l): synth.decode_q(w, b, l) for b in range(w.batch) for l in range(w.n_layers)}
    from paper_2607_06519_b200 import runner

    worst = 0.0
    for step in range(w.n_steps):
        for layer in range(w.n_layers):
            p, lp = layer // 2, layer & 1
            kn = np.stack([[rows[(b, p, h)][0][lp][step] for h in range(w.n_kv_heads)] for b in range(w.batch)])
            vn = np.stack([[rows[(b, p, h)][1][lp][step] for h in range(w.n_kv_heads)] for b in range(w.batch)])
            q = runner.to_device(np.stack([dq[(b, layer)][step] for b in range(w.batch)]), w.dtype, pf.device)
            out = pf.ctx.decode_attn(layer, q, runner.to_device(kn, w.dtype, pf.device), runner.to_device(vn, w.dtype, pf.device))
            for (b, up, h), u in units.items():
                if up == p:
                    u.append(lp, kn[b, h], vn[b, h])
            if step in (0, 1, 63, 127):
                torch.cuda.synchronize()
                assert torch.isfinite(out.float()).all()
                worst = max(worst, _check_layer(pf, w, layer, step, units, modes_all, q, out))
    assert worst <= TOL["bf16"], worst
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_decode32k_token_rule():
    """The 32k benchmark shape with the paper's token-granular residual: token sets by score band, probe errors and
    attention on the GPU's own sets, sampled units."""
    from paper_2607_06519_b200 import runner

    w = synth.WORKLOADS["decode32k_tok"]
    sample = [(0, 2, 1), (0, 11, 6)]
    pf = runner.Prefilled(w, max_tail=1)
    pf.compress(0)
    pmodes, scores = pf.probe(0, 0.0)
    pos = synth.probe_positions(w)
    units = {}
    for (b, p, h) in sample:
        k0, k1 = synth.unit_tensor(w, 0, p, h, False)
        v0, v1 = synth.unit_tensor(w, 0, p, h, True)
        u = R.Unit(k0, k1, v0, v1, True, w.keep_num, w.keep_den, select=False)
        pq = (synth.probe_q(w, 0, 2 * p), synth.probe_q(w, 0, 2 * p + 1))
        tok, sc = pf.ctx.get_token_set(0, p, h, w.T)
        tok, sc = tok.cpu().numpy(), f32(sc).astype(np.float64)
        s_ref = R.token_scores(u.z1["k"], pq[0], pq[1], w.group, h, pos)
        np.testing.assert_allclose(sc, s_ref, rtol=1e-5, atol=1e-6 * s_ref.max())
        kth = np.sort(s_ref)[::-1][w.k_tok - 1]
        assert tok.size == w.k_tok and np.all(np.diff(tok) > 0)
        assert set(np.flatnonzero(s_ref > kth * (1 + 2e-5)).tolist()) <= set(tok.tolist()) <= set(np.flatnonzero(s_ref >= kth * (1 - 2e-5)).tolist())
        assert set(synth.needle_positions(w, 0, p, h).tolist()) <= set(tok.tolist())  # the planted needles are all kept
        u.use_tokens(tok)
        e = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, pos)
        np.testing.assert_allclose(scores[p, h], e, rtol=1e-4)
        units[(b, p, h)] = u
    modes = synth.quota_modes(scores[..., 0])
    for (b, p, h) in sample:
        modes[p, h] = 1  # make sure the sampled units exercise the residual path
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    worst = 0.0
    for layer in range(w.n_layers):
        q = pf.decode_q(layer, 0)
        out = pf.ctx.decode_attn(layer, q)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        worst = max(worst, _check_layer(pf, w, layer, 0, units, [modes], q, out))
    assert worst <= TOL["bf16"], worst
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_decode32k_blocks_of_four_token_rule():
    """The paper's default pairing at the 32k benchmark shape (blocks of four layers, probe-scored tokens): token sets by
    score band, probe errors and one decode step of all layers on the GPU's own sets, sampled units of each mode."""
    from oracle import fdkv_ref_b4 as R4
    from paper_2607_06519_b200 import runner

    w = synth.WORKLOADS["decode32k_b4_tok"]
    pf = runner.Prefilled(w, max_tail=1)
    pf.compress(0)
    pmodes, scores = pf.probe(0, 0.0)
    pos = synth.probe_positions(w)
    modes = synth.quota_modes(scores[..., 0])
    sample = _pick_units(modes, 0, (1, 2, 1))
    units = {}
    for (b, blk, h) in sample:
        u = R4.Unit4(synth.block_tensor(w, 0, blk, h, False), synth.block_tensor(w, 0, blk, h, True), True, w.keep_num, w.keep_den,
                     select=False)
        pq = [synth.probe_q(w, 0, 4 * blk + l) for l in range(4)]
        tok, sc = pf.ctx.get_token_set(0, blk, h, w.T)
        tok, sc = tok.cpu().numpy(), f32(sc).astype(np.float64)
        s_ref = R4.token_scores4(u.dev["k"], pq, w.group, h, pos)
        np.testing.assert_allclose(sc, s_ref, rtol=1e-5, atol=1e-6 * s_ref.max())
        kth = np.sort(s_ref)[::-1][w.k_tok - 1]
        assert tok.size == w.k_tok and np.all(np.diff(tok) > 0)
        assert set(np.flatnonzero(s_ref > kth * (1 + 2e-5)).tolist()) <= set(tok.tolist()) <= set(np.flatnonzero(s_ref >= kth * (1 - 2e-5)).tolist())
        u.use_tokens(tok)
        e = R4.probe_error4(u.dev["k"], u.kept["k"], pq, w.group, h, pos)
        np.testing.assert_allclose(scores[blk, h], e, rtol=1e-4)
        units[(blk, h)] = u
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    torch.cuda.empty_cache()
    G, worst = w.group, 0.0
    for layer in range(w.n_layers):
        blk, lb = divmod(layer, 4)
        q = pf.decode_q(layer, 0)
        out = pf.ctx.decode_attn(layer, q)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        for (ub, h), u in units.items():
            if ub != blk:
                continue
            ref = u.attend(int(modes[blk][h]), lb, f32(q)[0][h * G:(h + 1) * G])
            worst = max(worst, float(vector_errors(f32(out)[0][h * G:(h + 1) * G], ref).max()))
    assert worst <= TOL["bf16"], worst
    assert pf.ctx.device_status() == 0
    pf.ctx.close()
