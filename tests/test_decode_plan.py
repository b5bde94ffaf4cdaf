"""Host logic of the decode launch (no GPU): the cost-weighted cut of a batch's (unit, 16-token slice) list over the
thread blocks.  Properties that must hold for any batch: the ranges tile the list exactly once and in order, every
block has work, the split-K part counts match the ranges, whole blocks per unit when there are enough blocks, and
the blocks' costs are balanced."""
import numpy as np
import pytest


def _slices(T):
    return (T + 15) // 16


def _check_partition(ranges, parts, T, hkv):
    units = len(T) * hkv
    ns = [_slices(T[u // hkv]) for u in range(units)]
    covered = [0] * units
    prev_end = (0, 0)
    touched = [0] * units
    for (b, e) in ranges:
        assert b == prev_end                       # contiguous, in order
        assert e >= b                              # (a block may be left without work when short units were moved)
        (ub, sb), (ue, se) = b, e
        for u in range(ub, min(ue, units - 1) + 1):
            lo = sb if u == ub else 0
            hi = se if u == ue else ns[u]
            if u == ue and ue == units:
                break
            if hi > lo:
                assert 0 <= lo and hi <= ns[u]
                covered[u] += hi - lo
                touched[u] += 1
        prev_end = e
    assert prev_end == (units, 0)
    assert covered == ns                           # every slice exactly once
    assert touched == parts


def _cost(ranges, T, hkv, modes, ratio):
    units = len(T) * hkv
    ns = [_slices(T[u // hkv]) for u in range(units)]
    flat = [m for row in modes for m in row]
    out = []
    for (b, e) in ranges:
        (ub, sb), (ue, se) = b, e
        c = 0.0
        for u in range(ub, min(ue, units - 1) + 1):
            lo = sb if u == ub else 0
            hi = se if u == ue else ns[u]
            if hi > lo:
                c += (hi - lo) * (ratio if flat[u] == 1 else 1.0)
        out.append(c)
    return np.array(out)


def test_llama_32k_whole_blocks_per_unit():
    from paper_2607_06519_b200 import binding as B
    T, hkv = [32768], 8
    modes = [[0, 1, 0, 1, 2, 1, 0, 0]]
    ranges, parts = B.plan_decode(T, modes, hkv, 1, 16, 148)
    assert len(ranges) == 148
    _check_partition(ranges, parts, T, hkv)
    # whole blocks per unit: no range crosses a unit boundary
    for (b, e) in ranges:
        assert e[0] == b[0] or (e[0] == b[0] + 1 and e[1] == 0)
    # blocks of one unit differ by at most one slice, except the block that ends the unit, which is charged extra and
    # gets fewer; residual units get more blocks
    for u in range(8):
        lens = [(e[1] if e[0] == u else _slices(T[0])) - b[1] for (b, e) in ranges if b[0] == u]
        assert max(lens[:-1]) - min(lens[:-1]) <= 1 and 0 < lens[-1] <= min(lens[:-1]) and len(lens) == parts[u]
    res, plain = [parts[u] for u in (1, 3, 5)], [parts[u] for u in (0, 2, 4, 6, 7)]
    assert min(res) > max(plain) and max(res) - min(res) <= 1 and max(plain) - min(plain) <= 1
    # the fitted residual cost (2.12 plain tiles at keep 1/16) balances the blocks within a few per cent
    c = _cost(ranges, T, hkv, modes, 2.12)
    ends_unit = np.array([e[1] == 0 for (b, e) in ranges])
    assert c[~ends_unit].max() / c[~ends_unit].mean() < 1.06 and c[ends_unit].max() <= c[~ends_unit].max()


@pytest.mark.parametrize("seed", range(12))
def test_random_batches_partition(seed):
    from paper_2607_06519_b200 import binding as B
    rng = np.random.default_rng(seed)
    batch = int(rng.integers(1, 9))
    hkv = int(rng.choice([1, 2, 4, 8]))
    T = [int(rng.choice([1, 15, 16, 17, 127, 129, 1000, 4097, 32768, 50001])) for _ in range(batch)]
    modes = rng.integers(0, 3, (batch, hkv)).tolist()
    keep = [(1, 16), (1, 32), (0, 1), (1, 1), (3, 7)][int(rng.integers(0, 5))]
    n_ctas = int(rng.choice([3, 7, 132, 148, 160]))
    for rule, fmt in ((0, 0), (1, 0), (0, 1)):
        ranges, parts = B.plan_decode(T, modes, hkv, keep[0], keep[1], n_ctas, residual_rule=rule, row_format=fmt)
        assert 1 <= len(ranges) <= n_ctas
        _check_partition(ranges, parts, T, hkv)


def test_batch_flat_cut_is_balanced():
    from paper_2607_06519_b200 import binding as B
    T, hkv = [32768] * 8, 8
    rng = np.random.default_rng(3)
    modes = rng.integers(0, 3, (8, hkv)).tolist()
    ranges, parts = B.plan_decode(T, modes, hkv, 1, 16, 148)
    assert len(ranges) == 148
    _check_partition(ranges, parts, T, hkv)
    c = _cost(ranges, T, hkv, modes, 1.59)   # the flat cut weighs a residual tile 1.5 x its bytes
    assert c.max() / c.mean() < 1.08         # (blocks that end a unit are charged extra and get less)


def test_many_one_token_units_fit_the_segment_tables():
    """One long sequence and seven one-token sequences: the cost cut would hand 56 one-slice units to a single block,
    whose table holds 24; the plan spreads them."""
    from paper_2607_06519_b200 import binding as B
    hkv = 8
    for T in ([32768] + [1] * 7, [1] * 7 + [32768], [1, 1, 1, 32768, 1, 1, 1, 1], [1] * 8):
        modes = [[1] * hkv for _ in T]
        for n in (3, 148):
            ranges, parts = B.plan_decode(T, modes, hkv, 1, 16, n)
            _check_partition(ranges, parts, T, hkv)
            for (b, e) in ranges:
                nseg = sum(1 for u in range(b[0], min(e[0], len(T) * hkv - 1) + 1)
                           if (e[1] if u == e[0] else _slices(T[u // hkv])) > (b[1] if u == b[0] else 0) and u < len(T) * hkv)
                assert nseg <= 24


def test_argument_checks():
    from paper_2607_06519_b200 import binding as B
    with pytest.raises(B.FdkvError):
        B.plan_decode([0], [[0]], 1, 1, 16, 148)          # empty sequence
    with pytest.raises(B.FdkvError):
        B.plan_decode([128], [[3]], 1, 1, 16, 148)        # mode out of range
    with pytest.raises(B.FdkvError):
        B.plan_decode([128] * 129, [[0] * 8] * 129, 8, 1, 16, 148)  # more units than the kernel takes (1024)
    with pytest.raises(B.FdkvError):
        B.plan_decode([128], [[0]], 1, 1, 16, 0)          # no blocks
