"""The one-pass ordered select (both storage types) on inputs made of ties: a unit-tensor whose |Z1| takes three values
only, so that the threshold class holds a large share of all entries and the first `need` of them -- in index
order, wherever that count ends: inside a 32-entry word, inside a 32 KiB chunk, dozens of chunks into the tensor --
decide the list.  With float32 storage the same inputs also overflow the candidate list of the threshold refinement
(every key of the threshold's 15-bit class is a candidate), so the full second pass runs.  Compared bit for bit with the
oracle's Eq. 1 split and Eq. 3 entry selection (lowest index wins)."""
import numpy as np
import pytest
import torch

from oracle import fdkv_ref as R

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T,d", [(8192, 128), (8192 - 37, 128), (5000, 64), (130, 128), (16, 64)])
@pytest.mark.parametrize("keep", [(0, 1), (1, 16), (1, 3), (2, 5), (7, 8), (1, 1)])
def test_ties_across_words_and_chunks(T, d, keep, dtype):
    from paper_2607_06519_b200 import binding as B

    rng = np.random.default_rng(1000 * T + 10 * d + keep[0] * 7 + keep[1])
    # x1 = 0 and x0 in {-2 .. 2}: |z1| is one of 0, c, 2c (after rounding); long runs of equal values in places
    x0 = rng.integers(-2, 3, size=(T, d)).astype(np.float32)
    x0[T // 3: T // 3 + max(1, T // 7)] = 1.0       # a run of ties that spans whole chunks
    x0[:, d // 2] = -2.0                             # a channel that is always in the top class
    x1 = np.zeros_like(x0)
    k = (T * d * keep[0]) // keep[1]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    if dtype == "f32":  # float32 keys: a few distinct values inside one 15-bit class, so that the refinement has work to do
        x0 = x0 * (1.0 + rng.integers(0, 3, size=x0.shape).astype(np.float32) * np.float32(2.0 ** -20))
    tx0 = torch.from_numpy(x0).cuda().to(tdt)
    tx1 = torch.from_numpy(x1).cuda().to(tdt)
    z0 = torch.empty((T, d), dtype=tdt, device="cuda")
    idx = torch.full((max(k, 1),), -1, dtype=torch.int32, device="cuda")
    val = torch.zeros((max(k, 1),), dtype=tdt, device="cuda")
    for _ in range(2):  # twice: the look-back records and the ticket of the first call must not leak into the second
        idx.fill_(-1)
        got = B.compress_unit_noalloc(tx0, tx1, keep[0], keep[1], z0, idx, val)
        torch.cuda.synchronize()
        assert got == k
        ref_z0, ref_z1 = R.depth_split(x0, x1, dtype == "bf16")
        ref_idx = R.select_entries(ref_z1, k)
        assert np.array_equal(idx.cpu().numpy()[:k], ref_idx)
        assert np.array_equal(val.float().cpu().numpy()[:k].view(np.uint32), ref_z1.ravel()[ref_idx].view(np.uint32))
        assert np.array_equal(z0.float().cpu().numpy().view(np.uint32), ref_z0.view(np.uint32))
