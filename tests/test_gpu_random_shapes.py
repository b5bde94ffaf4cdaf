"""Randomised small workloads (shapes, keep fractions, mode assignments, tail lengths, both residual rules) through
the whole path against the oracle: a sweep meant to catch index arithmetic that only fails off the beaten path."""
import numpy as np
import pytest
import torch

from gpu_util import TOL, check_compression, f32, oracle_layer_out, oracle_unit, vector_errors
from oracle import fdkv_ref as R
from paper_2607_06519_b200 import synth

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(2024)
    out = []
    for i in range(14):
        dtype = "bf16" if i % 3 else "f32"
        d = 128 if (dtype == "bf16" and i % 2) else int(rng.choice([64, 128]))
        hkv = int(rng.choice([1, 2, 3]))
        g = int(rng.choice([1, 2, 4, 8]))
        T = int(rng.choice([1, 15, 16, 17, 127, 128, 129, 255, 640, 1000, 1537]))
        keep = [(1, 16), (1, 8), (3, 7), (0, 1), (1, 1), (1, 33)][int(rng.integers(0, 6))]
        tail = int(rng.choice([0, 1, 2, 5]))
        W = int(min(T, rng.choice([1, 3, 8, 16])))
        tok = int(dtype == "bf16" and d == 128 and i % 4 == 1)
        out.append((i, dtype, d, hkv, g, T, keep, tail, W, tok))
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: f"{c[0]}-{c[1]}-d{c[2]}-h{c[3]}-g{c[4]}-T{c[5]}-k{c[6][0]}of{c[6][1]}-t{c[7]}-W{c[8]}-r{c[9]}")
def test_random_workload(case):
    from paper_2607_06519_b200 import runner

    i, dtype, d, hkv, g, T, keep, tail, W, tok = case
    w = synth.Workload(name=f"rnd{i}", n_layers=4, n_q_heads=hkv * g, n_kv_heads=hkv, head_dim=d, batch=2, T=T, dtype=dtype,
                       keep_num=keep[0], keep_den=keep[1], n_needles=min(3, T), W=W, seed=100 + i, n_steps=max(tail, 1),
                       residual_rule=tok)
    pf = runner.Prefilled(w, max_tail=max(tail, 1))
    rng = np.random.default_rng(i)
    units, modes_all = {}, []
    pos = synth.probe_positions(w)
    for b in range(w.batch):
        pf.compress(b)
        pmodes, scores = pf.probe(b, 3.0)
        for p in range(w.n_pairs):
            pq = (synth.probe_q(w, b, 2 * p), synth.probe_q(w, b, 2 * p + 1))
            for h in range(hkv):
                if tok:
                    k0, k1 = synth.unit_tensor(w, b, p, h, False)
                    v0, v1 = synth.unit_tensor(w, b, p, h, True)
                    u = R.Unit(k0, k1, v0, v1, True, keep[0], keep[1], select=False)
                    t_gpu, s_gpu = pf.ctx.get_token_set(b, p, h, T)
                    s_ref = R.token_scores(u.z1["k"], pq[0], pq[1], w.group, h, pos)
                    np.testing.assert_allclose(f32(s_gpu), s_ref, rtol=1e-5, atol=1e-6 * max(1.0, s_ref.max()))
                    assert t_gpu.numel() == w.k_tok
                    u.use_tokens(t_gpu.cpu().numpy())
                else:
                    u = check_compression(pf.ctx, w, b, p, h)
                e = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, pos)
                np.testing.assert_allclose(scores[p, h], e, rtol=1e-4, atol=1e-9)
                units[(b, p, h)] = u
        modes = rng.integers(0, 3, (w.n_pairs, hkv)).astype(np.int32)
        pf.ctx.set_modes(b, modes)
        pf.commit(b)
        modes_all.append(modes)
    for step in range(max(tail, 1)):
        for layer in range(w.n_layers):
            q = pf.decode_q(layer, step)
            kn = vn = None
            if tail:
                kn, vn = pf.new_rows(layer, step)
                for (b, p, h), u in units.items():
                    if p == layer // 2:
                        u.append(layer & 1, f32(kn)[b, h], f32(vn)[b, h])
            out = pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0)
            torch.cuda.synchronize()
            for b in range(w.batch):
                us = {h: units[(b, layer // 2, h)] for h in range(hkv)}
                ref = oracle_layer_out(us, modes_all[b][layer // 2], w, layer, f32(q)[b])
                err = vector_errors(f32(out)[b], ref)
                assert err.max() <= TOL[dtype], (step, layer, b, float(err.max()))
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def _cases_new():
    rng = np.random.default_rng(4242)
    out = []
    for i in range(12):
        bs = 4 if i % 2 else 2
        f8 = int(i % 3 != 0)
        if not f8 and bs == 2:
            bs = 4
        hkv = int(rng.choice([1, 2, 3]))
        g = int(rng.choice([1, 2, 4]))
        T = int(rng.choice([1, 15, 16, 17, 127, 128, 129, 255, 640, 1000, 1537]))
        keep = [(1, 16), (1, 8), (3, 7), (0, 1), (1, 1), (1, 33)][int(rng.integers(0, 6))]
        tail = int(rng.choice([0, 1, 3, 130]))
        out.append((i, bs, f8, hkv, g, T, keep, tail))
    return out


@pytest.mark.parametrize("case", _cases_new(), ids=lambda c: f"{c[0]}-B{c[1]}-f8{c[2]}-h{c[3]}-g{c[4]}-T{c[5]}-k{c[6][0]}of{c[6][1]}-t{c[7]}")
def test_random_block4_and_8bit_rows(case):
    """The same sweep over the newer storage forms: blocks of four layers and / or 8-bit row streams (bf16, d = 128)."""
    from oracle import fdkv_ref_b4 as R4
    from oracle import fdkv_ref_fp8 as R8
    from paper_2607_06519_b200 import runner

    i, bs, f8, hkv, g, T, keep, tail = case
    w = synth.Workload(name=f"rn{i}", n_layers=2 * bs, n_q_heads=hkv * g, n_kv_heads=hkv, head_dim=128, batch=1, T=T, dtype="bf16",
                       keep_num=keep[0], keep_den=keep[1], n_needles=min(3, T), W=min(4, T), seed=300 + i, n_steps=max(tail, 1),
                       block_size=bs, row_format=f8)
    pf = runner.Prefilled(w, max_tail=max(tail, 1))
    rng = np.random.default_rng(i)
    modes = rng.integers(0, 3, (w.n_blocks, hkv)).astype(np.int32)
    pf.prefill(0, modes=modes)
    units = {}
    for b in range(w.n_blocks):
        for h in range(hkv):
            if bs == 4:
                ks, vs = synth.block_tensor(w, 0, b, h, False), synth.block_tensor(w, 0, b, h, True)
                units[(b, h)] = R8.Unit4Fp8(ks, vs, True, *keep) if f8 else R4.Unit4(ks, vs, True, *keep)
            else:
                k0, k1 = synth.unit_tensor(w, 0, b, h, False)
                v0, v1 = synth.unit_tensor(w, 0, b, h, True)
                units[(b, h)] = R8.UnitFp8(k0, k1, v0, v1, True, *keep)
    steps = [0] if tail == 0 else list(range(tail))
    check_at = {0, 1, 2, tail - 1}
    for step in steps:
        for layer in range(w.n_layers):
            b, lb = divmod(layer, bs)
            q = pf.decode_q(layer, step)
            kn = vn = None
            if tail:
                kn, vn = pf.new_rows(layer, step)
                for h in range(hkv):
                    units[(b, h)].append(lb, f32(kn)[0, h], f32(vn)[0, h])
            out = pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0)
            if step in check_at:
                torch.cuda.synchronize()
                for h in range(hkv):
                    ref = units[(b, h)].attend(int(modes[b][h]), lb, f32(q)[0][h * g:(h + 1) * g])
                    err = vector_errors(f32(out)[0][h * g:(h + 1) * g], ref).max()
                    assert err <= TOL["bf16"], (step, layer, h, float(err))
    assert pf.ctx.device_status() == 0
    pf.ctx.close()
