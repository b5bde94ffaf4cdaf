"""GPU parity for the periodic refresh: fdkv_fold_tail moves generated tokens from the exact tails into the compressed
form (chunk-wise Eq. 1 and Eq. 3 under each unit's fixed mode).  Decode outputs before and after folding, with more
tokens appended afterwards and a second fold, must match the oracle's Unit.fold within the attention tolerance."""
import numpy as np
import pytest
import torch

from gpu_util import TOL, f32, oracle_unit, vector_errors
from paper_2607_06519_b200 import binding as B
from paper_2607_06519_b200 import synth

pytestmark = pytest.mark.gpu


def _check_step(pf, w, modes, units, step, check):
    worst = 0.0
    G = w.group
    for layer in range(w.n_layers):
        q = pf.decode_q(layer, step)
        kn, vn = pf.new_rows(layer, step)
        for h in range(w.n_kv_heads):
            units[(layer // 2, h)].append(layer & 1, f32(kn)[0, h], f32(vn)[0, h])
        out = pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0)
        if check:
            torch.cuda.synchronize()
            for h in range(w.n_kv_heads):
                ref = units[(layer // 2, h)].attend(int(modes[layer // 2][h]), layer & 1, f32(q)[0][h * G:(h + 1) * G])
                worst = max(worst, float(vector_errors(f32(out)[0][h * G:(h + 1) * G], ref).max()))
    return worst


@pytest.mark.parametrize("dtype,d,T,keep", [("bf16", 128, 2048, (1, 16)), ("f32", 64, 320, (1, 8))])
def test_fold_tail_matches_the_oracle(dtype, d, T, keep):
    from paper_2607_06519_b200 import runner

    n_steps = 200
    w = synth.Workload(name="fold", n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=d, batch=1, T=T, dtype=dtype,
                       keep_num=keep[0], keep_den=keep[1], n_needles=4, W=8, seed=31, n_steps=n_steps)
    pf = runner.Prefilled(w, max_tail=160, max_fold=160)
    pf.compress(0)
    units = {(p, h): oracle_unit(w, 0, p, h) for p in range(2) for h in range(2)}
    modes = np.array([[0, 1], [2, 1]], dtype=np.int32)
    pf.ctx.set_modes(0, modes)
    pf.commit(0)
    tol = TOL[dtype]
    step = 0
    for _ in range(130):
        worst = _check_step(pf, w, modes, units, step, check=step in (0, 129))
        assert worst <= tol, (step, worst)
        step += 1
    # cannot fold more than the tails hold, nor past the reserved room
    with pytest.raises(B.FdkvError):
        pf.ctx.fold_tail(0, 144)
    by_before, ex_before = pf.ctx.footprint(0)
    pf.ctx.fold_tail(0, 128)
    for u in units.values():
        u.fold(128, *keep)
    by_after, ex_after = pf.ctx.footprint(0)
    e_b = 2 if dtype == "bf16" else 4
    assert ex_after - ex_before == 4 * 4 * 128 * d * e_b            # 4 units x (K, V of 2 layers) x 128 rows
    assert by_after[0] - by_before[0] == 2 * 128 * d * e_b          # the shared unit: one coefficient row per token, K and V
    assert by_after[2] - by_before[2] == 4 * 128 * d * e_b          # the exact unit keeps both layers' rows
    assert by_after[1] - by_before[1] > 2 * 2 * 128 * d * e_b       # two residual units: rows plus their kept entries
    for _ in range(20):  # 2 tokens were left in the tails; 20 more arrive
        worst = _check_step(pf, w, modes, units, step, check=True)
        assert worst <= tol, (step, worst)
        step += 1
    pf.ctx.fold_tail(0, 16)  # a second, small chunk
    for u in units.values():
        u.fold(16, *keep)
    for _ in range(3):
        worst = _check_step(pf, w, modes, units, step, check=True)
        assert worst <= tol, (step, worst)
        step += 1
    with pytest.raises(B.FdkvError) as ei:  # 144 of 160 used
        pf.ctx.fold_tail(0, 32)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_fold_one_sequence_of_a_batch():
    """Folding sequence 1 of two leaves sequence 0 untouched; batched decode afterwards sees T and T + 32."""
    from gpu_util import oracle_unit
    from paper_2607_06519_b200 import runner

    w = synth.Workload(name="fold2", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=2, T=512, dtype="bf16",
                       keep_num=1, keep_den=16, n_needles=4, W=8, seed=33, n_steps=40, seq_seeds=(33, 34))
    pf = runner.Prefilled(w, max_tail=48, max_fold=64)
    modes = np.array([[1, 0]], dtype=np.int32)
    units = {}
    for b in range(2):
        pf.prefill(b, modes=modes)
        for h in range(2):
            units[(b, h)] = oracle_unit(w, b, 0, h)
    G = 4

    def step(j, check):
        for layer in range(2):
            q = pf.decode_q(layer, j)
            kn, vn = pf.new_rows(layer, j)
            for b in range(2):
                for h in range(2):
                    units[(b, h)].append(layer, f32(kn)[b, h], f32(vn)[b, h])
            out = f32(pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0))
            if check:
                torch.cuda.synchronize()
                for b in range(2):
                    for h in range(2):
                        ref = units[(b, h)].attend(int(modes[0][h]), layer, f32(q)[b][h * G:(h + 1) * G])
                        assert vector_errors(out[b][h * G:(h + 1) * G], ref).max() <= TOL["bf16"], (j, layer, b, h)

    for j in range(34):
        step(j, check=j == 33)
    pf.ctx.fold_tail(1, 32)
    for h in range(2):
        units[(1, h)].fold(32, 1, 16)
    for j in range(34, 38):
        step(j, check=True)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_fold_tail_block_of_four():
    """The same refresh for depth blocks of four layers (shared kept set by energy inside the chunk)."""
    from oracle import fdkv_ref_b4 as R4
    from paper_2607_06519_b200 import runner

    w = synth.Workload(name="fold4", n_layers=8, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=1, T=1024, dtype="bf16",
                       keep_num=1, keep_den=16, n_needles=4, W=8, seed=35, n_steps=60, block_size=4)
    pf = runner.Prefilled(w, max_tail=64, max_fold=64)
    modes = np.array([[1, 0], [2, 1]], dtype=np.int32)
    pf.prefill(0, modes=modes)
    units = {(b, h): R4.Unit4(synth.block_tensor(w, 0, b, h, False), synth.block_tensor(w, 0, b, h, True), True, 1, 16)
             for b in range(2) for h in range(2)}
    G = 4

    def step(j, check):
        for layer in range(8):
            blk, lb = divmod(layer, 4)
            q = pf.decode_q(layer, j)
            kn, vn = pf.new_rows(layer, j)
            for h in range(2):
                units[(blk, h)].append(lb, f32(kn)[0, h], f32(vn)[0, h])
            out = f32(pf.ctx.decode_attn(layer, q, kn, vn, out_dtype=0))[0]
            if check:
                torch.cuda.synchronize()
                for h in range(2):
                    ref = units[(blk, h)].attend(int(modes[blk][h]), lb, f32(q)[0][h * G:(h + 1) * G])
                    assert vector_errors(out[h * G:(h + 1) * G], ref).max() <= TOL["bf16"], (j, layer, h)

    for j in range(50):
        step(j, check=j == 49)
    pf.ctx.fold_tail(0, 48)
    for u in units.values():
        u.fold(48, 1, 16)
    for j in range(50, 54):
        step(j, check=True)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()
