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


def _prefill(w, seqs, sample_units, probe_units):
    from paper_2607_06519_b200 import runner

    pf = runner.Prefilled(w, max_tail=max(w.n_steps, 1))
    units, modes_all = {}, []
    pos = synth.probe_positions(w)
    for b in seqs:
        pf.compress(b)
        for (sb, p, h) in sample_units:
            if sb == b:
                units[(b, p, h)] = check_compression(pf.ctx, w, b, p, h)
        pmodes, scores = pf.probe(b, 0.0)
        for (sb, p, h) in probe_units:
            if sb == b:
                u = units[(b, p, h)]
                e = R.probe_error(u.z1["k"], u.kept["k"], synth.probe_q(w, b, 2 * p), synth.probe_q(w, b, 2 * p + 1), w.group,
                                  h, pos)
                np.testing.assert_allclose(scores[p, h], e, rtol=1e-4)
        modes = synth.quota_modes(scores[..., 0])
        pf.ctx.set_modes(b, modes)
        pf.commit(b)
        modes_all.append(modes)
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
    w = synth.WORKLOADS["decode32k"]
    sample = [(0, 0, 0), (0, 7, 3), (0, 15, 7)]
    pf, units, modes_all = _prefill(w, [0], sample, sample[:2])
    assert sorted(np.bincount(modes_all[0].ravel(), minlength=3).tolist()) == sorted([64, 45, 19])
    # make sure the three sampled units cover more than one mode where possible (the mix is fixed by the probe)
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
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_decode128k_long_context():
    w = synth.WORKLOADS["decode128k"]
    sample = [(0, 1, 2), (0, 13, 6)]
    pf, units, modes_all = _prefill(w, [0], sample, sample[:1])
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
    sample = [(0, 0, 1), (3, 9, 5), (7, 15, 0)]
    pf, units, modes_all = _prefill(w, list(range(w.batch)), sample, [])
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
