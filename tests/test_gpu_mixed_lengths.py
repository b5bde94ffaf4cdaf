"""A batch whose sequences differ widely in length: one long prompt among one-token and few-token prompts.  The decode
launch then cuts a flat (unit, slice) list in which runs of very short units fall to single thread blocks (their
segment tables hold 24 units; the plan moves whole units to neighbours), some blocks get no work at all, and most
ranges are shorter than one tile.  Every sequence's output is compared with the oracle."""
import numpy as np
import pytest
import torch

from gpu_util import TOL, f32, oracle_layer_out, oracle_unit, vector_errors
from paper_2607_06519_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("lengths", [(6000, 1, 1, 1, 1, 1, 1, 1), (1, 3, 1, 6000, 17, 1, 1, 130), (1, 1, 1, 1, 1, 1, 1, 1)])
def test_batch_of_one_long_and_many_short_sequences(lengths):
    from paper_2607_06519_b200 import runner

    hkv, g, d = 8, 2, 128
    base = dict(n_layers=2, n_q_heads=hkv * g, n_kv_heads=hkv, head_dim=d, batch=len(lengths), dtype="bf16", keep_num=1,
                keep_den=8, seed=77, n_steps=2)
    ws = [synth.Workload(name=f"mix{b}", T=T, n_needles=min(2, T), W=min(4, T), **base) for b, T in enumerate(lengths)]
    big = max(range(len(lengths)), key=lambda b: lengths[b])
    first = runner.Prefilled(ws[big], max_tail=2)          # the context is sized for the longest prompt
    pfs = [first if b == big else runner.Prefilled(ws[b], ctx=first.ctx) for b in range(len(lengths))]
    rng = np.random.default_rng(5)
    units, modes = {}, []
    for b, pf in enumerate(pfs):
        m = rng.integers(0, 3, (1, hkv)).astype(np.int32)
        pf.prefill(b, modes=m)
        modes.append(m)
        for h in range(hkv):
            units[(b, h)] = oracle_unit(ws[b], b, 0, h)
    ctx = first.ctx
    for step in range(2):
        for layer in range(2):
            q = torch.stack([pfs[b].decode_q(layer, step)[b] for b in range(len(lengths))])
            rows = [pfs[b].new_rows(layer, step) for b in range(len(lengths))]
            kn = torch.stack([rows[b][0][b] for b in range(len(lengths))])
            vn = torch.stack([rows[b][1][b] for b in range(len(lengths))])
            for b in range(len(lengths)):
                for h in range(hkv):
                    units[(b, h)].append(layer & 1, f32(kn)[b, h], f32(vn)[b, h])
            out = ctx.decode_attn(layer, q, kn, vn, out_dtype=0)
            torch.cuda.synchronize()
            for b in range(len(lengths)):
                ref = oracle_layer_out({h: units[(b, h)] for h in range(hkv)}, modes[b][0], ws[b], layer, f32(q)[b])
                err = vector_errors(f32(out)[b], ref).max()
                assert err <= TOL["bf16"], (lengths, step, layer, b, err)
    assert ctx.device_status() == 0
    ctx.close()
