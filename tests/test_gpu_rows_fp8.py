"""GPU parity for 8-bit row streams (row_format = e4m3): the committed codes and per-channel scales are bit-exact against
the oracle's quantiser; decode attention over them (f16 tensor-core products on converted fragments, scales folded
into q and applied to the output) matches the oracle's attention over the dequantised rows within the bf16 tolerance, with generated tokens appended to the bf16 tails."""
import numpy as np
import pytest
import torch

from gpu_util import TOL, f32, vector_errors
from oracle import fdkv_ref_fp8 as R8
from paper_2607_06519_b200 import binding as B
from paper_2607_06519_b200 import synth

pytestmark = pytest.mark.gpu


def _unit8(w, p, h):
    k0, k1 = synth.unit_tensor(w, 0, p, h, False)
    v0, v1 = synth.unit_tensor(w, 0, p, h, True)
    return R8.UnitFp8(k0, k1, v0, v1, True, w.keep_num, w.keep_den)


@pytest.mark.parametrize("T,Hq,Hkv,keep,n_steps", [(1300, 8, 2, (1, 16), 3), (2100, 4, 1, (1, 32), 131), (300, 2, 2, (1, 8), 2)])
def test_rows_e4m3_parity(T, Hq, Hkv, keep, n_steps):
    from paper_2607_06519_b200 import runner

    w = synth.Workload(name="f8", n_layers=4, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=128, batch=1, T=T, dtype="bf16",
                       keep_num=keep[0], keep_den=keep[1], n_needles=4, W=8, seed=51, n_steps=n_steps, row_format=1)
    pf = runner.Prefilled(w, max_tail=n_steps)
    modes = np.array([[(p + h) % 3 for h in range(Hkv)] for p in range(2)], dtype=np.int32)
    pf.prefill(0, modes=modes)
    units = {(p, h): _unit8(w, p, h) for p in range(2) for h in range(Hkv)}
    # stored codes and scales
    for (p, h), u in units.items():
        for layer in (2 * p, 2 * p + 1):
            for is_v, name in ((0, "k"), (1, "v")):
                codes, scale = pf.ctx.get_rows_e4m3(0, layer, h, is_v, T)
                want_c, want_s = u.q_x[name][layer & 1] if modes[p][h] == 2 else u.q_z0[name]
                assert np.array_equal(scale.cpu().numpy(), want_s), (p, h, layer, name)
                assert np.array_equal(codes.cpu().numpy(), want_c), (p, h, layer, name)
    # decode, appending generated tokens to the (bf16) tails: the 8-bit tiles and the tails join at the merge
    G = w.group
    for step in range(n_steps):
        worst = 0.0
        for layer in range(4):
            q = pf.decode_q(layer, step)
            kn, vn = pf.new_rows(layer, step)
            for h in range(Hkv):
                units[(layer // 2, h)].append(layer & 1, f32(kn)[0, h], f32(vn)[0, h])
            out = f32(pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0))[0]
            torch.cuda.synchronize()
            for h in range(Hkv):
                ref = units[(layer // 2, h)].attend(int(modes[layer // 2][h]), layer & 1, f32(q)[0][h * G:(h + 1) * G])
                worst = max(worst, float(vector_errors(out[h * G:(h + 1) * G], ref).max()))
        assert worst <= TOL["bf16"], (step, worst)
    for b in range(1):
        pf.ctx.set_tail_len(b, 0)
    by_mode, exact_equiv = pf.ctx.footprint(0)
    assert pf.ctx.decode_bytes(0, 1) < 0.62 * sum(2 * T * 128 * 2 for _ in range(Hkv)) + 64 * 1024 * Hkv
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


@pytest.mark.parametrize("T,keep,tail", [(1300 + 37, (1, 16), 2), (300, (1, 8), 0)])
def test_rows_e4m3_with_token_rule(T, keep, tail):
    """8-bit rows combined with the token rule: the kept tokens' high-frequency rows stay 16-bit (rescaled by the rows'
    channel scales for the 8-bit tiles' products); attention on the GPU's own token set against the oracle."""
    from paper_2607_06519_b200 import runner

    Hq, Hkv = 8, 2
    w = synth.Workload(name="f8tok", n_layers=4, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=128, batch=1, T=T, dtype="bf16",
                       keep_num=keep[0], keep_den=keep[1], n_needles=4, W=8, seed=57, n_steps=max(tail, 1), row_format=1,
                       residual_rule=1)
    pf = runner.Prefilled(w, max_tail=max(tail, 1))
    pf.compress(0)
    pf.probe(0, 1.0)
    units = {}
    for p in range(2):
        for h in range(Hkv):
            u = _unit8(w, p, h)
            tok, _ = pf.ctx.get_token_set(0, p, h, w.T)
            u.use_tokens(tok.cpu().numpy())
            units[(p, h)] = u
    modes = np.array([[1, (p + 1) % 3] for p in range(2)], dtype=np.int32)
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    G = w.group
    worst = 0.0
    for step in range(max(tail, 1)):
        for layer in range(4):
            q = pf.decode_q(layer, step)
            kn = vn = None
            if tail:
                kn, vn = pf.new_rows(layer, step)
                for h in range(Hkv):
                    units[(layer // 2, h)].append(layer & 1, f32(kn)[0, h], f32(vn)[0, h])
            out = f32(pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0))[0]
            torch.cuda.synchronize()
            for h in range(Hkv):
                ref = units[(layer // 2, h)].attend(int(modes[layer // 2][h]), layer & 1, f32(q)[0][h * G:(h + 1) * G])
                worst = max(worst, float(vector_errors(out[h * G:(h + 1) * G], ref).max()))
    assert worst <= TOL["bf16"], worst
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_rows_e4m3_benchmark_workload_sampled():
    """decode32k_fp8 (the 32k workload with 8-bit rows, quota mode mix) through the calls bench.py times: sampled units'
    codes and scales bit-exact, one decode step of all layers within tolerance on those units."""
    from paper_2607_06519_b200 import runner

    w = synth.WORKLOADS["decode32k_fp8"]
    sample = [(0, 1), (9, 4), (15, 7)]
    pf = runner.Prefilled(w, max_tail=1)
    modes = pf.prefill(0)
    units = {(p, h): _unit8(w, p, h) for (p, h) in sample}
    for (p, h), u in units.items():
        codes, scale = pf.ctx.get_rows_e4m3(0, 2 * p + 1, h, 0, w.T)
        want_c, want_s = u.q_x["k"][1] if modes[p][h] == 2 else u.q_z0["k"]
        assert np.array_equal(scale.cpu().numpy(), want_s) and np.array_equal(codes.cpu().numpy(), want_c)
    torch.cuda.empty_cache()
    G = w.group
    worst = 0.0
    for layer in range(w.n_layers):
        q = pf.decode_q(layer, 0)
        out = pf.ctx.decode_attn(layer, q)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        for (p, h), u in units.items():
            if p != layer // 2:
                continue
            ref = u.attend(int(modes[p][h]), layer & 1, f32(q)[0][h * G:(h + 1) * G])
            worst = max(worst, float(vector_errors(f32(out)[0][h * G:(h + 1) * G], ref).max()))
    assert worst <= TOL["bf16"], worst
    by_mode, exact_equiv = pf.ctx.footprint(0)
    assert pf.ctx.decode_bytes(0, 1) < 0.56 * 8 * 2 * w.T * 128 * 2
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_rows_e4m3_with_blocks_of_four():
    """8-bit rows combined with depth blocks of four layers: codes of the shared rows bit-exact, decode with appends."""
    from paper_2607_06519_b200 import runner

    w = synth.Workload(name="f8b4", n_layers=8, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=1, T=900, dtype="bf16",
                       keep_num=1, keep_den=16, n_needles=4, W=8, seed=53, n_steps=2, row_format=1, block_size=4)
    pf = runner.Prefilled(w, max_tail=2)
    modes = np.array([[1, 0], [2, 1]], dtype=np.int32)
    pf.prefill(0, modes=modes)
    units = {(b, h): R8.Unit4Fp8(synth.block_tensor(w, 0, b, h, False), synth.block_tensor(w, 0, b, h, True), True, 1, 16)
             for b in range(2) for h in range(2)}
    for (b, h), u in units.items():
        for lb in range(4):
            codes, scale = pf.ctx.get_rows_e4m3(0, 4 * b + lb, h, 1, w.T)
            want_c, want_s = u.q_x["v"][lb] if modes[b][h] == 2 else u.q_z0["v"]
            assert np.array_equal(scale.cpu().numpy(), want_s) and np.array_equal(codes.cpu().numpy(), want_c)
    G = 4
    for step in range(2):
        for layer in range(8):
            blk, lb = divmod(layer, 4)
            q = pf.decode_q(layer, step)
            kn, vn = pf.new_rows(layer, step)
            for h in range(2):
                units[(blk, h)].append(lb, f32(kn)[0, h], f32(vn)[0, h])
            out = f32(pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0))[0]
            torch.cuda.synchronize()
            for h in range(2):
                ref = units[(blk, h)].attend(int(modes[blk][h]), lb, f32(q)[0][h * G:(h + 1) * G])
                assert vector_errors(out[h * G:(h + 1) * G], ref).max() <= TOL["bf16"], (step, layer, h)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()
