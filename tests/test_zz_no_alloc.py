"""The allocation-free entry point against the regular one.

fdkv_compress_unit_noalloc exists for callers that cannot call cudaMalloc (a serving engine that owns the whole
device pool, a plugin that is only handed tensors) and have no context whose workspace would hold the scratch.
It must produce, bit for bit, what fdkv_compress_prefill stages for the same unit-tensor -- the selection is
integer work and the coefficients are fixed float32 arithmetic, so the tolerance is zero, as in the other
compression tests -- on two calls in a row (the built-in scratch keeps the first call's data).

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import fdkv_ref as R

pytestmark = pytest.mark.gpu


def _case(seed, T, d, dtype):
    rng = np.random.default_rng(seed)
    xs = [(rng.standard_normal((T, 2, d)) * np.exp(rng.standard_normal(d))).astype(np.float32) for _ in range(4)]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    return [torch.from_numpy(x).cuda().to(tdt) for x in xs]


@pytest.mark.parametrize("dtype,T,d,keep", [("bf16", 1000, 128, (1, 16)), ("f32", 517, 64, (1, 8))])
def test_noalloc_matches_context_path_twice(dtype, T, d, keep):
    from paper_2607_06519_b200 import binding as B

    code = B.BF16 if dtype == "bf16" else B.F32
    ctx = B.Context(B.Config(2, 4, 2, d, 1, T, 1, code, keep[0], keep[1]))
    k = (T * d * keep[0]) // keep[1]
    for call, seed in enumerate((11, 12)):  # two calls in a row, different data
        k0, k1, v0, v1 = _case(seed, T, d, dtype)
        ctx.compress_prefill(0, 0, 1, T, [k0, k1], [v0, v1])
        for h in range(2):
            for is_v, (x0, x1) in enumerate(((k0, k1), (v0, v1))):
                want_z0 = ctx.get_shared(0, 0, h, is_v, T)
                want_idx, want_val = ctx.get_residual(0, 0, h, is_v)
                z0 = torch.empty((T, d), dtype=x0.dtype, device="cuda")
                idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
                val = torch.zeros((k,), dtype=x0.dtype, device="cuda")
                got_k = B.compress_unit_noalloc(x0[:, h], x1[:, h], keep[0], keep[1], z0, idx, val)
                torch.cuda.synchronize()
                assert got_k == k == want_idx.numel()
                assert torch.equal(z0.view(torch.int16 if dtype == "bf16" else torch.int32),
                                   want_z0.view(torch.int16 if dtype == "bf16" else torch.int32)), (call, h, is_v)
                assert torch.equal(idx, want_idx), (call, h, is_v)
                assert torch.equal(val.view(torch.int16 if dtype == "bf16" else torch.int32),
                                   want_val.view(torch.int16 if dtype == "bf16" else torch.int32)), (call, h, is_v)
                if h == 0:
                    # and, on its own feet, against the CPU oracle's Eq. 1 split and entry selection of the same rows
                    a, b = x0[:, h].float().cpu().numpy(), x1[:, h].float().cpu().numpy()
                    ref_z0, ref_z1 = R.depth_split(a, b, dtype == "bf16")
                    ref_idx = R.select_entries(ref_z1, k)
                    assert np.array_equal(z0.float().cpu().numpy().view(np.uint32), ref_z0.view(np.uint32)), (call, is_v)
                    assert np.array_equal(idx.cpu().numpy(), ref_idx), (call, is_v)
                    assert np.array_equal(val.float().cpu().numpy().view(np.uint32), ref_z1.ravel()[ref_idx].view(np.uint32)), (call, is_v)
    assert ctx.device_status() == 0
    ctx.close()


def test_noalloc_rejects_oversize():
    from paper_2607_06519_b200 import binding as B

    T, d = B.NOALLOC_MAX_ELEMS // 128 + 1, 128
    x = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
    z0 = torch.empty_like(x)
    idx = torch.empty(1, dtype=torch.int32, device="cuda")
    val = torch.empty(1, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.FdkvError) as e:
        B.compress_unit_noalloc(x, x, 0, 1, z0, idx, val)
    assert e.value.code == 9
