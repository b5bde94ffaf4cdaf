"""Argument and call-order errors are reported by the host side of the C ABI before anything is launched
(no test here makes the GPU fault, trap or hang): status codes, and the context stays usable afterwards."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _ctx(**kw):
    from paper_2607_06519_b200 import binding as B

    cfg = dict(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, max_batch=2, max_prefill=256, max_tail=2, dtype=B.F32,
               keep_num=1, keep_den=8)
    cfg.update(kw)
    return B, B.Context(B.Config(**cfg))


def _kv(T=256, H=2, d=64, dtype=torch.float32):
    g = torch.Generator(device="cuda").manual_seed(0)
    return [torch.randn((T, H, d), device="cuda", generator=g).to(dtype) for _ in range(4)]


def _code(B, fn):
    with pytest.raises(B.FdkvError) as e:
        fn()
    return e.value.code


def test_call_order_and_argument_checks():
    B, ctx = _ctx()
    k0, k1, v0, v1 = _kv()
    q = torch.randn((1, 4, 64), device="cuda")
    # decode before anything is committed
    assert _code(B, lambda: ctx.decode_attn(0, q)) == 5
    # probe before compress
    pq = [torch.randn((8, 4, 64), device="cuda") for _ in range(2)]
    assert _code(B, lambda: ctx.probe(0, 0, 1, pq, list(range(248, 256)), 1.0)) == 5
    # bad ranges and sizes
    assert _code(B, lambda: ctx.compress_prefill(0, 0, 2, 256, [k0, k1], [v0, v1])) == 1      # pair range beyond n_layers/2
    assert _code(B, lambda: ctx.compress_prefill(5, 0, 1, 256, [k0, k1], [v0, v1])) == 1      # sequence slot
    assert _code(B, lambda: ctx.compress_prefill(0, 0, 1, 257, [k0, k1], [v0, v1])) == 1      # T > max_prefill
    # misaligned pointer (offset by one element) is rejected, not dereferenced
    flat = torch.randn(256 * 2 * 64 + 8, device="cuda")
    bad = flat[1:1 + 256 * 2 * 64].view(256, 2, 64)
    assert _code(B, lambda: ctx.compress_prefill(0, 0, 1, 256, [bad, k1], [v0, v1])) == 1
    # a good compress, then probe argument checks
    ctx.compress_prefill(0, 0, 1, 256, [k0, k1], [v0, v1])
    assert _code(B, lambda: ctx.probe(0, 0, 1, pq, [5, 5, 6, 7, 8, 9, 10, 11], 1.0)) == 1       # not strictly ascending
    assert _code(B, lambda: ctx.probe(0, 0, 1, pq, list(range(249, 257)), 1.0)) == 1            # position >= T
    assert _code(B, lambda: ctx.probe(0, 0, 1, pq, list(range(248, 256)), -1.0)) == 1           # negative lambda
    # commit without modes
    assert _code(B, lambda: ctx.commit(0)) == 5
    assert _code(B, lambda: ctx.set_modes(0, [0, 3])) == 1                                       # mode out of range
    ctx.set_modes(0, [1, 2])
    ctx.commit(0)
    assert _code(B, lambda: ctx.commit(0)) == 5                                                  # already committed
    assert _code(B, lambda: ctx.decode_attn(0, torch.randn((2, 4, 64), device="cuda"))) == 5     # slot 1 not committed
    assert _code(B, lambda: ctx.decode_attn(2, q)) == 1                                          # layer out of range
    # the tail holds max_tail rows per layer; the next append is refused on the host
    kn = torch.randn((1, 2, 64), device="cuda")
    ctx.decode_attn(0, q, kn, kn)
    ctx.decode_attn(0, q, kn, kn)
    assert _code(B, lambda: ctx.decode_attn(0, q, kn, kn)) == 5
    # still usable
    out = ctx.decode_attn(1, q)
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
    assert ctx.device_status() == 0
    ctx.close()


def test_arena_too_small_is_reported_at_commit():
    B, _ = _ctx()
    _.close()
    cfg = B.Config(2, 4, 2, 64, 1, 4096, 1, B.F32, 1, 8)
    worst, _w = B.sizes(cfg)
    ctx = B.Context(cfg, arena_bytes=worst * 3 // 4)  # room for a shared-mode sequence, not for an exact-mode one
    k0, k1, v0, v1 = _kv(T=4096)
    ctx.compress_prefill(0, 0, 1, 4096, [k0, k1], [v0, v1])
    ctx.set_modes(0, [2, 2])
    with pytest.raises(B.FdkvError) as e:
        ctx.commit(0)
    assert e.value.code == 3
    ctx.set_modes(0, [0, 0])
    ctx.commit(0)  # the cheaper modes fit
    by_mode, exact_equiv = ctx.footprint(0)
    assert by_mode[0] == exact_equiv // 2 and by_mode[1] == by_mode[2] == 0
    ctx.close()


def test_reset_frees_the_arena():
    B, ctx = _ctx()
    k0, k1, v0, v1 = _kv()
    for _ in range(3):
        ctx.compress_prefill(0, 0, 1, 256, [k0, k1], [v0, v1])
        ctx.set_modes(0, [2, 2])
        ctx.commit(0)
        assert ctx.get_modes(0).tolist() == [[2, 2]]
        ctx.reset()
    ctx.close()


def test_step_host_call_equals_per_layer_calls():
    """fdkv_decode_step_host (all layers of a step, host buffers) returns what the per-layer device calls return."""
    import torch
    from paper_2607_06519_b200 import binding as B, runner, synth

    w = synth.Workload(name="step", n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=2, T=700, dtype="bf16",
                       keep_num=1, keep_den=16, n_needles=4, W=8, seed=5, n_steps=2, seq_seeds=(5, 6))
    pf = runner.Prefilled(w, max_tail=4)
    for b in range(2):
        pf.prefill(b, modes=np.array([[0, 1], [2, 1]], dtype=np.int32))
    qs = [pf.decode_q(l, 0) for l in range(4)]
    rows = [pf.new_rows(l, 0) for l in range(4)]
    want = [pf.ctx.decode_attn(l, qs[l], rows[l][0], rows[l][1]) for l in range(4)]
    torch.cuda.synchronize()
    for b in range(2):
        pf.ctx.set_tail_len(b, 0)
    hq = torch.stack(qs).cpu().pin_memory()
    hk = torch.stack([r[0] for r in rows]).cpu().pin_memory()
    hv = torch.stack([r[1] for r in rows]).cpu().pin_memory()
    hout = torch.empty(hq.shape, dtype=torch.bfloat16).pin_memory()
    pf.ctx.decode_step_host(hq, hk, hv, hout, B.BF16)
    for l in range(4):
        assert torch.equal(hout[l], want[l].cpu())
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_unsupported_combinations_and_reset_reuse():
    """Configurations the build has no kernels for are refused at creation; a context is reusable after reset."""
    from paper_2607_06519_b200 import binding as B, runner, synth

    base = dict(n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=128, max_batch=1, max_prefill=512, max_tail=4, dtype=B.BF16,
                keep_num=1, keep_den=16)
    for bad in (dict(block_size=3), dict(residual_rule=2), dict(row_format=1, head_dim=64),
                dict(row_format=1, dtype=B.F32), dict(row_format=1, max_fold=16), dict(row_format=1, n_q_heads=16),
                dict(row_format=2), dict(max_fold=-1), dict(n_layers=6, block_size=4)):
        cfg = dict(base)
        cfg.update(bad)
        with pytest.raises(B.FdkvError) as e:
            B.sizes(B.Config(**cfg))
        assert e.value.code == 2, bad
    # fold_tail is refused for the token rule and for 8-bit rows, get_rows_e4m3 without them
    w = synth.Workload(name="reuse", n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=1, T=512, dtype="bf16",
                       keep_num=1, keep_den=16, n_needles=4, W=8, seed=61, n_steps=1, block_size=4)
    pf = runner.Prefilled(w, max_tail=2)
    modes = np.array([[1, 2]], dtype=np.int32)
    pf.prefill(0, modes=modes)
    with pytest.raises(B.FdkvError) as e:
        pf.ctx.get_rows_e4m3(0, 0, 0, 0, 512)
    assert e.value.code == 2
    with pytest.raises(B.FdkvError) as e:
        pf.ctx.fold_tail(0, 16)  # max_fold is 0
    assert e.value.code in (1, 3)
    q = pf.decode_q(1, 0)
    first = pf.ctx.decode_attn(1, q).clone()
    # reset and run the same prompt again through the same context: identical output
    pf.ctx.reset()
    pf.prefill(0, modes=modes)
    again = pf.ctx.decode_attn(1, q)
    torch.cuda.synchronize()
    assert torch.equal(first, again)
    assert pf.ctx.device_status() == 0
    pf.ctx.close()


def test_bounded_device_wait_runs_out_and_reports():
    """Every device-side wait of the library (TMA copies, tensor-core commits) is bounded.  Here one is made to run out
    -- a barrier nobody arrives at, a limit of a thousand polls -- and must come back as FDKV_ERR_TIMEOUT from
    fdkv_device_status, with the kernel ending normally and the context still computing correct results afterwards."""
    B, ctx = _ctx(head_dim=128, dtype=B_BF16(), max_prefill=512)
    k0, k1, v0, v1 = _kv(T=512, d=128, dtype=torch.bfloat16)
    ctx.compress_prefill(0, 0, 1, 512, [k0, k1], [v0, v1])
    ctx.set_modes(0, [1, 0])
    ctx.commit(0)
    q = torch.randn((1, 4, 128), device="cuda").to(torch.bfloat16)
    before = ctx.decode_attn(0, q, out_dtype=B.F32).clone()
    assert ctx.device_status() == 0
    ctx.test_wait_expiry(1024)
    assert ctx.device_status() == 7          # FDKV_ERR_TIMEOUT: the wait gave up and said so
    torch.cuda.synchronize()                 # the device is healthy
    ctx.test_clear_device_status()
    assert ctx.device_status() == 0
    after = ctx.decode_attn(0, q, out_dtype=B.F32)
    torch.cuda.synchronize()
    assert torch.equal(before, after)
    assert ctx.device_status() == 0
    with pytest.raises(B.FdkvError):
        ctx.test_wait_expiry(0)              # limits outside 1 .. 65536 are refused on the host
    ctx.close()


def B_BF16():
    from paper_2607_06519_b200 import binding as B

    return B.BF16
