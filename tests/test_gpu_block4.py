"""GPU parity for depth blocks of four layers (Eq. 1 with B = 4) against oracle/fdkv_ref_b4.py.

Bit-exact: the stored shared coefficient, the kept positions (ties to the lowest index) and the four layers' values
at them, the modes.  Within tolerance: the probe errors (1e-4 relative) and the attention outputs (1e-3 float32,
2e-2 bf16, max|delta| / max|ref| per output vector), in all three modes, with appended tail rows.
"""
import numpy as np
import pytest
import torch

from oracle import fdkv_ref as R
from oracle import fdkv_ref_b4 as R4
from paper_2607_06519_b200 import synth
from gpu_util import TOL, bits, f32, vector_errors

pytestmark = pytest.mark.gpu


def _runner():
    from paper_2607_06519_b200 import runner
    return runner


def oracle_unit4(w, seq, blk, h) -> R4.Unit4:
    return R4.Unit4(synth.block_tensor(w, seq, blk, h, False), synth.block_tensor(w, seq, blk, h, True),
                    w.dtype == "bf16", w.keep_num, w.keep_den)


def check_compression4(ctx, w, seq, blk, h):
    u = oracle_unit4(w, seq, blk, h)
    for is_v, name in ((0, "k"), (1, "v")):
        z0 = ctx.get_shared(seq, blk, h, is_v, w.T)
        assert np.array_equal(bits(z0), u.z0[name].view(np.uint32)), f"z0 {name} block {blk} head {h}"
        idx, val = ctx.get_residual(seq, blk, h, is_v)
        assert idx.numel() == u.k_keep and tuple(val.shape) == (4, u.k_keep)
        assert np.array_equal(idx.cpu().numpy(), u.kept[name]), f"kept positions {name} block {blk} head {h}"
        for l in range(4):
            want = u.dev[name][l].ravel()[u.kept[name]]
            assert np.array_equal(bits(val[l]), want.view(np.uint32)), f"values {name} layer {l} block {blk} head {h}"
    return u


def _decode_check(pf, w, modes, units, step, append, out_dtype=0):
    worst = 0.0
    for layer in range(w.n_layers):
        blk, lb = divmod(layer, 4)
        q = pf.decode_q(layer, step)
        kn = vn = None
        if append:
            kn, vn = pf.new_rows(layer, step)
            for h in range(w.n_kv_heads):
                units[(blk, h)].append(lb, f32(kn)[0, h], f32(vn)[0, h])
        out = pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=out_dtype)
        torch.cuda.synchronize()
        ql = f32(q)[0]
        ref = np.zeros((w.n_q_heads, w.head_dim))
        G = w.group
        for h in range(w.n_kv_heads):
            ref[h * G:(h + 1) * G] = units[(blk, h)].attend(int(modes[blk][h]), lb, ql[h * G:(h + 1) * G])
        worst = max(worst, float(vector_errors(f32(out)[0], ref).max()))
    return worst


@pytest.mark.parametrize("dtype,T,d,Hq,Hkv,keep,tail,n_layers", [
    ("f32", 512, 64, 4, 2, (1, 8), 2, 4),        # the tiny case with one block of four
    ("bf16", 777, 128, 8, 2, (1, 16), 3, 8),     # ragged T, two blocks, the tensor-core decode kernel
    ("bf16", 2100, 128, 4, 1, (1, 32), 5, 4),    # several CTAs per unit, G = 4
    ("f32", 130, 128, 8, 1, (0, 1), 1, 4),       # keep nothing: residual == shared
    ("bf16", 96, 64, 4, 4, (1, 1), 0, 4),        # keep everything, head_dim 64 (portable decode kernel)
])
def test_block4_parity(dtype, T, d, Hq, Hkv, keep, tail, n_layers):
    runner = _runner()
    w = synth.Workload(name="b4", n_layers=n_layers, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, batch=1, T=T, dtype=dtype,
                       keep_num=keep[0], keep_den=keep[1], n_needles=min(4, T), W=min(8, T), seed=11,
                       n_steps=max(tail, 1), block_size=4)
    pf = runner.Prefilled(w, max_tail=max(tail, 1))
    pf.compress(0)
    units = {(b, h): check_compression4(pf.ctx, w, 0, b, h) for b in range(w.n_blocks) for h in range(Hkv)}
    # probe errors and the mode rule
    lam = 1.0
    pmodes, scores = pf.probe(0, lam)
    q_probe = [synth.probe_q(w, 0, l) for l in range(w.n_layers)]
    e_bytes = 2 if dtype == "bf16" else 4
    om = R4.omega4(T, d, e_bytes, w.k_keep)
    for (b, h), u in units.items():
        e = R4.probe_error4(u.dev["k"], u.kept["k"], q_probe[4 * b:4 * b + 4], w.group, h, synth.probe_positions(w))
        np.testing.assert_allclose(scores[b, h], e, rtol=1e-4, atol=1e-12)
        m, _, margin = R.mode_rule(e[0], e[1], om, lam)
        if margin > 1e-3:
            assert int(pmodes[b, h]) == m
    # forced modes covering all three, then decode with tails
    modes = np.array([[(b + h) % 3 for h in range(Hkv)] for b in range(w.n_blocks)], dtype=np.int32)
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    assert np.array_equal(pf.ctx.get_modes(0).numpy(), modes)
    for step in range(max(tail, 1)):
        worst = _decode_check(pf, w, modes, units, step, append=tail > 0)
        assert worst <= TOL[dtype], (step, worst)
    by_mode, exact_equiv = pf.ctx.footprint(0)
    assert exact_equiv == w.n_blocks * Hkv * 2 * 4 * T * d * e_bytes
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_block4_all_modes_each(request):
    """Every unit in one mode at a time (the paper's 'shared-depth only' and 'without exact' ablation settings)."""
    runner = _runner()
    w = synth.Workload(name="b4m", n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=1, T=1500, dtype="bf16",
                       keep_num=1, keep_den=16, n_needles=4, W=8, seed=12, n_steps=1, block_size=4)
    for mode in (0, 1, 2):
        pf = runner.Prefilled(w, max_tail=1)
        pf.compress(0)
        units = {(0, h): oracle_unit4(w, 0, 0, h) for h in range(2)}
        modes = np.full((1, 2), mode, dtype=np.int32)
        pf.ctx.set_modes(0, modes)
        pf.commit(0)
        worst = _decode_check(pf, w, modes, units, 0, append=False)
        assert worst <= TOL["bf16"], (mode, worst)
        assert pf.ctx.device_status() == 0
        pf.ctx.close()


def test_block4_benchmark_workload_sampled():
    """decode32k_b4 (32 layers = 8 blocks, 32k, bf16, quota mode mix) through the calls bench.py times; sampled
    units are checked against the oracle: stored values bit-exact, probe errors, one decode step of all layers."""
    runner = _runner()
    w = synth.WORKLOADS["decode32k_b4"]
    sample = [(0, 2), (3, 5), (7, 7)]
    pf = runner.Prefilled(w, max_tail=1)
    pf.compress(0)
    units = {(b, h): check_compression4(pf.ctx, w, 0, b, h) for (b, h) in sample}
    pmodes, scores = pf.probe(0, 0.0)
    pos = synth.probe_positions(w)
    for (b, h) in sample[:2]:
        u = units[(b, h)]
        e = R4.probe_error4(u.dev["k"], u.kept["k"], [synth.probe_q(w, 0, 4 * b + l) for l in range(4)], w.group, h, pos)
        np.testing.assert_allclose(scores[b, h], e, rtol=1e-4)
    modes = synth.quota_modes(scores[..., 0])
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    assert np.bincount(modes.ravel(), minlength=3).tolist() == [32, 22, 10]
    torch.cuda.empty_cache()
    worst = 0.0
    G = w.group
    for layer in range(w.n_layers):
        blk, lb = divmod(layer, 4)
        q = pf.decode_q(layer, 0)
        out = pf.ctx.decode_attn(layer, q)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        for (b, h), u in units.items():
            if b != blk:
                continue
            ref = u.attend(int(modes[b][h]), lb, f32(q)[0][h * G:(h + 1) * G])
            worst = max(worst, float(vector_errors(f32(out)[0][h * G:(h + 1) * G], ref).max()))
    assert worst <= TOL["bf16"], worst
    by_mode, exact_equiv = pf.ctx.footprint(0)
    assert sum(by_mode) < 0.5 * exact_equiv  # a shared unit stores one of four layers
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_mixed_schedule_two_contexts():
    """The paper's mixed schedule (B = 4 in the middle, B = 2 for the first and last layers) as two contexts: a
    12-layer stack whose layers 0-3 and 8-11 form pairs (one 8-layer context) and whose layers 4-7 form one block
    of four (a second context).  Every layer's output matches the oracle of its own block size."""
    from gpu_util import oracle_unit
    runner = _runner()
    base = dict(n_q_heads=8, n_kv_heads=2, head_dim=128, batch=1, T=900, dtype="bf16", keep_num=1, keep_den=16,
                n_needles=4, W=8, n_steps=1)
    w2 = synth.Workload(name="edge_pairs", n_layers=8, seed=41, **base)                 # model layers 0-3, 8-11
    w4 = synth.Workload(name="middle_block", n_layers=4, seed=42, block_size=4, **base)  # model layers 4-7
    pf2, pf4 = runner.Prefilled(w2, max_tail=1), runner.Prefilled(w4, max_tail=1)
    m2 = np.array([[0, 1], [1, 2], [2, 0], [1, 1]], dtype=np.int32)
    m4 = np.array([[1, 0]], dtype=np.int32)
    pf2.prefill(0, modes=m2)
    pf4.prefill(0, modes=m4)
    u2 = {(p, h): oracle_unit(w2, 0, p, h) for p in range(4) for h in range(2)}
    u4 = {(0, h): oracle_unit4(w4, 0, 0, h) for h in range(2)}
    G = 4
    worst = 0.0
    for model_layer in range(12):
        if 4 <= model_layer < 8:
            pf, w, local = pf4, w4, model_layer - 4
        else:
            pf, w, local = pf2, w2, model_layer if model_layer < 4 else model_layer - 4
        q = pf.decode_q(local, 0)
        out = f32(pf.ctx.decode_attn(local, q, out_dtype=0))[0]
        torch.cuda.synchronize()
        for h in range(2):
            qh = f32(q)[0][h * G:(h + 1) * G]
            if pf is pf4:
                ref = u4[(0, h)].attend(int(m4[0][h]), local, qh)
            else:
                ref = u2[(local // 2, h)].attend(int(m2[local // 2][h]), local & 1, qh)
            worst = max(worst, float(vector_errors(out[h * G:(h + 1) * G], ref).max()))
    assert worst <= TOL["bf16"], worst
    for pf in (pf2, pf4):
        assert pf.ctx.device_status() == 0
        pf.ctx.close()


def test_block4_two_sequences_of_different_length():
    runner = _runner()
    w = synth.Workload(name="b4two", n_layers=4, n_q_heads=4, n_kv_heads=2, head_dim=128, batch=2, T=640, dtype="bf16",
                       keep_num=1, keep_den=8, n_needles=4, W=8, seed=13, n_steps=3, block_size=4, seq_seeds=(13, 14))
    pf = runner.Prefilled(w, max_tail=3)
    modes = np.array([[1, 2]], dtype=np.int32)
    units = {}
    for b in range(2):
        pf.prefill(b, modes=modes)
        for h in range(2):
            units[(b, h)] = R4.Unit4(synth.block_tensor(w, b, 0, h, False), synth.block_tensor(w, b, 0, h, True), True, 1, 8)
    G = 2
    for step in range(3):
        for layer in range(4):
            q = pf.decode_q(layer, step)
            kn, vn = pf.new_rows(layer, step)
            for b in range(2):
                for h in range(2):
                    units[(b, h)].append(layer, f32(kn)[b, h], f32(vn)[b, h])
            out = f32(pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0))
            torch.cuda.synchronize()
            for b in range(2):
                for h in range(2):
                    ref = units[(b, h)].attend(int(modes[0][h]), layer, f32(q)[b][h * G:(h + 1) * G])
                    assert vector_errors(out[b][h * G:(h + 1) * G], ref).max() <= TOL["bf16"]
    assert pf.ctx.device_status() == 0
    pf.ctx.close()
