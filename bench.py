#!/usr/bin/env python
"""Benchmark of the FreqDepthKV hot path on B200.

One JSON line on stdout.  Headline: compressed-KV decode attention tokens/s on the Llama-3-8B-shaped 32k
workload (32 per-layer calls per generated token over the packed cache), with the achieved HBM bandwidth of
the decode kernel on the bytes it actually reads.  The prefill side of the path (depth split + residual
selection, probe) runs once per prompt as set-up and is timed and reported under "prefill".

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload decode32k|decode128k|tiny]

N > 1 (under torchrun) runs N independent replicas of the same workload, one per GPU: the path has no
exchange step, so there is no collective on the data path.
--impl reference times the CPU oracle (test infrastructure) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from one ncu capture (a constant, not
# measured per run; None for workloads without a capture): 142.8 MB read + 3.8 MB written per launch on the 4-layer
# cut of the 32k workload, which has the same 8 units and bytes per launch as the 32-layer workload
NCU_TRAFFIC_BYTES = {
    "decode32k": 146.6e6,
    "decode32k_4l": 146.6e6,
    # 554.0 MB read + 4.5 MB written per launch on the 4-layer cut of the 128k workload
    "decode128k": 558.5e6,
    "decode128k_4l": 558.5e6,
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
    return FALLBACK_HBM_GBS, 1590.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(w, n_units: int):
    """Builds the oracle state of a few units of the workload (untimed set-up of the CPU legs)."""
    from oracle import fdkv_ref as R
    from paper_2607_06519_b200 import synth

    rng = np.random.default_rng(12345)
    picks = [(int(p), int(h)) for p, h in zip(rng.integers(0, w.n_blocks, n_units), rng.integers(0, w.n_kv_heads, n_units))]
    units = []
    for i, (p, h) in enumerate(picks):
        if w.block_size == 4:
            from oracle import fdkv_ref_b4 as R4
            u = R4.Unit4(synth.block_tensor(w, 0, p, h, False), synth.block_tensor(w, 0, p, h, True), w.dtype == "bf16",
                         w.keep_num, w.keep_den)
        else:
            k0, k1 = synth.unit_tensor(w, 0, p, h, False)
            v0, v1 = synth.unit_tensor(w, 0, p, h, True)
            if w.row_format == 1:
                from oracle import fdkv_ref_fp8 as R8
                u = R8.UnitFp8(k0, k1, v0, v1, w.dtype == "bf16", w.keep_num, w.keep_den)
            else:
                u = R.Unit(k0, k1, v0, v1, w.dtype == "bf16", w.keep_num, w.keep_den)
        mode = (0, 1, 0, 2, 1, 0, 1, 0)[i % 8]  # close to the 50/35/15 benchmark mix
        units.append((p, h, mode, u))
    return units


def oracle_step(w, units):
    """One pass of the oracle's decode attention over the sampled units (both layers of each)."""
    from paper_2607_06519_b200 import synth

    t0 = time.perf_counter()
    for p, h, mode, u in units:
        for lp in range(w.block_size):
            q = synth.decode_q(w, 0, w.block_size * p + lp)[0][h * w.group:(h + 1) * w.group]
            u.attend(mode, lp, q)
    return time.perf_counter() - t0


def oracle_prefill_sample(w, units_total: int):
    """The oracle's prefill side (Eq. 1 split, entry selection, Eq. 2 probe errors) on ONE unit, timed and scaled."""
    from oracle import fdkv_ref as R
    from paper_2607_06519_b200 import synth

    p, h = 0, 0
    k0, k1 = synth.unit_tensor(w, 0, p, h, False)
    v0, v1 = synth.unit_tensor(w, 0, p, h, True)
    pq = (synth.probe_q(w, 0, 2 * p), synth.probe_q(w, 0, 2 * p + 1))
    pos = synth.probe_positions(w)
    t0 = time.perf_counter()
    _, z1k = R.depth_split(k0, k1, w.dtype == "bf16")
    _, z1v = R.depth_split(v0, v1, w.dtype == "bf16")
    kept = R.select_entries(z1k, w.k_keep)
    R.select_entries(z1v, w.k_keep)
    t1 = time.perf_counter()
    R.probe_error(z1k, kept, pq[0], pq[1], w.group, h, pos)
    t2 = time.perf_counter()
    return {"compress_ms": (t1 - t0) * 1e3 * units_total, "probe_ms": (t2 - t1) * 1e3 * units_total, "cores": R.threads(),
            "kind": "oracle", "sample": f"1 of {units_total} units (split + selection of K and V, probe errors of K), scaled to all units"}


def run_reference(args, w):
    from oracle import fdkv_ref as R

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_units = {"decode32k": 4, "decode128k": 2}.get(w.name, 2)
    units = oracle_sample(w, n_units)
    total_calls = w.n_layers * w.n_kv_heads * w.batch
    times = [oracle_step(w, units) for _ in range(args.warmup + args.steps)][args.warmup:]
    t_step_sample = float(np.mean(times))
    t_full = t_step_sample * total_calls / (w.block_size * len(units))
    val = w.batch / t_full
    sample = (f"{w.block_size * len(units)} of {total_calls} (layer, KV head) attention units of one decode step, "
              f"scaled to the full step")
    line = {"impl": "reference", "metric": "compressed-KV decode attention tokens/s", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_full * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "context": w.T, "batch": w.batch},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": R.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_ours(args, w):
    import torch

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    line = bench_workload(args, w, dev, dist, rank, local, world, args.steps, args.warmup, not args.no_cpu_baseline)
    if rank == 0 and world == 1 and w.name == "decode32k" and not args.no_also:
        # the other single-GPU configuration the target names (context 131072), a shorter timed region, same JSON line
        from paper_2607_06519_b200 import synth

        torch.cuda.empty_cache()
        w2 = synth.WORKLOADS["decode128k"]
        l2 = bench_workload(args, w2, dev, None, 0, local, 1, min(args.steps, 10), 3, False)
        line["also"] = [{k: l2[k] for k in ("metric", "value", "unit", "steps", "warmup", "ms_per_step", "dtype", "config", "roofline",
                                            "e2e", "gpu_launches", "prefill", "step_bytes")}]
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def bench_workload(args, w, dev, dist, rank, local, world, steps, warmup, with_cpu_baseline):
    """One workload through prefill (timed per call) and the timed decode region; returns rank 0's JSON fields."""
    import torch

    from paper_2607_06519_b200 import binding as B, replicas, runner, synth

    hbm_peak, tf_peak, peak_kind = measured_peaks()
    no_graph = args.no_graph

    # ---------------- set-up: the prefill side of the path, timed per call ----------------
    pf = runner.Prefilled(w, max_tail=max(w.n_steps, 1), device=dev)
    ctx = pf.ctx
    ev = lambda: torch.cuda.Event(enable_timing=True)
    compress_ms, probe_ms, commit_ms = 0.0, 0.0, 0.0
    launches_prefill = B.launch_count()
    esize = 2 if w.dtype == "bf16" else 4
    for b in range(w.batch):
        k_layers, v_layers = [None] * w.n_layers, [None] * w.n_layers
        nb = w.block_size
        for p in range(w.n_blocks):
            t = pf.upload_pair(b, p)
            for lb in range(nb):
                k_layers[nb * p + lb], v_layers[nb * p + lb] = t[f"k{lb}"], t[f"v{lb}"]
        if b == 0:  # untimed pass: first launches pay the lazy loading of every kernel
            ctx.compress_prefill(b, 0, w.n_blocks, w.T, k_layers, v_layers)
            ctx.probe(b, 0, w.n_blocks, pf.upload_probe_q(b), synth.probe_positions(w), 0.0)
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        ctx.compress_prefill(b, 0, w.n_blocks, w.T, k_layers, v_layers)
        e1.record()
        torch.cuda.synchronize()
        compress_ms += e0.elapsed_time(e1)
        q_layers = pf.upload_probe_q(b)
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        modes, scores = ctx.probe(b, 0, w.n_blocks, q_layers, synth.probe_positions(w), 0.0)
        e1.record()
        torch.cuda.synchronize()
        probe_ms += e0.elapsed_time(e1)
        ctx.set_modes(b, synth.quota_modes(scores.cpu().numpy()[..., 0]))
        torch.cuda.synchronize()
        t_c = time.perf_counter()
        ctx.commit(b)  # synchronous: packs the kept streams into the arena
        commit_ms += (time.perf_counter() - t_c) * 1e3
        del k_layers, v_layers, q_layers, t
    launches_prefill = B.launch_count() - launches_prefill
    units = w.batch * w.n_blocks * w.n_kv_heads
    n_ut = 2 * units
    N = w.T * w.head_dim
    if w.residual_rule == 1:
        # token rule: compression is the depth split alone (the probe selects); the probe runs three products
        # (token scores, then the two candidates' errors)
        nbl, nhf = w.block_size, (1 if w.block_size == 2 else 4)  # layers per block; stored high-frequency rows per kept token and tensor
        compress_min_bytes = n_ut * (nbl * N * esize + N * esize) + units * (2 * nhf * w.k_tok * w.head_dim * esize + 4 * w.k_tok)
        probe_flops = 2.0 * units * 3 * (nbl * w.group * w.W) * w.T * w.head_dim
    else:
        # read the block's layers, write the shared coefficient, the index and the kept values
        nbl = w.block_size
        compress_min_bytes = n_ut * (nbl * N * esize + N * esize + w.k_keep * (4 + (1 if nbl == 2 else 4) * esize))
        probe_flops = 2.0 * units * 2 * (nbl * w.group * w.W) * w.T * w.head_dim
    # bytes the compression kernels really move (pairs, entry rule, bf16 / head_dim 128): split reads both layers and
    # writes Z0 and the staged Z1; the one-pass select reads Z1 once more and emits the canonical (index, value) list,
    # the packed decode entries and, for K, the copy of Z1 without the kept entries for the probe
    compress_moved_bytes = None
    if w.residual_rule == 0 and w.block_size == 2 and w.dtype == "bf16" and w.head_dim == 128:
        compress_moved_bytes = n_ut * (5 * N * esize + w.k_keep * (8 + esize)) + units * N * esize
    modes_all = np.stack([ctx.get_modes(b).numpy() for b in range(w.batch)])
    mix = [int((modes_all == m).sum()) for m in range(3)]
    torch.cuda.empty_cache()

    # ---------------- the decode step: one call per layer ----------------
    qs = [pf.decode_q(l, 0) for l in range(w.n_layers)]
    outs = [torch.empty_like(q) for q in qs]
    step_bytes = sum(ctx.decode_bytes(l, w.batch) for l in range(w.n_layers))
    stream = torch.cuda.Stream()
    append = w.n_steps > 1  # batched workload: every step appends one generated token to every layer's tail
    new_k = new_v = None
    step_no = [0]
    if append:
        no_graph = True  # the tail length advances on the device and in the host mirror: launch directly
        steps = min(steps, w.n_steps - warmup - 1)
        tail_fn = synth.block_tail_rows if w.block_size == 4 else synth.tail_rows
        rows = {(b, p, h, v): tail_fn(w, b, p, h, bool(v)) for b in range(w.batch) for p in range(w.n_blocks)
                for h in range(w.n_kv_heads) for v in (0, 1)}
        new_k, new_v = [], []
        for l in range(w.n_layers):
            for v, dst in ((0, new_k), (1, new_v)):
                a = np.stack([[rows[(b, l // w.block_size, h, v)][l % w.block_size] for h in range(w.n_kv_heads)] for b in range(w.batch)])
                dst.append(runner.to_device(np.ascontiguousarray(a.transpose(2, 0, 1, 3)), w.dtype, dev))  # [step][b][h][d]

    def step():
        j = step_no[0]
        for l in range(w.n_layers):
            if append:
                ctx.decode_attn(l, qs[l], new_k[l][j], new_v[l][j], out=outs[l], stream=stream)
            else:
                ctx.decode_attn(l, qs[l], None, None, out=outs[l], stream=stream)
        step_no[0] = j + 1

    launches_per_step = B.launch_count()
    with torch.cuda.stream(stream):
        step()
    stream.synchronize()
    launches_per_step = B.launch_count() - launches_per_step
    graph = None
    if not no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step()
        except Exception as e:  # capture is an optimisation of the launch path only
            sys.stderr.write(f"graph capture failed ({e}); launching directly\n")
            graph = None

    def run_step():
        if graph is not None:
            graph.replay()
        else:
            step()

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            run_step()
    stream.synchronize()
    replicas.barrier(dist)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    e0, e1 = ev(), ev()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(steps):
            run_step()
        e1.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    total_ms = e0.elapsed_time(e1)
    if rank == 0:
        # keep sampling long enough to have seen the GPU under load at least a few times
        if total_ms < 500 and not append:
            with torch.cuda.stream(stream):
                for _ in range(int(600 / max(total_ms / steps, 1e-3)) + 1):
                    run_step()
            stream.synchronize()
        clocks = sampler.stop()
    value, total_s = replicas.whole_job_rate(w.batch * steps, total_ms * 1e-3, dist, dev)
    total_ms = total_s * 1e3
    ms_per_step = total_ms / steps

    # ---------------- end to end: host buffers through the C ABI, copies inside the timed region ----------------
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    hq = [q.cpu().pin_memory() for q in qs]
    hout = [torch.empty(q.shape, dtype=tdt).pin_memory() for q in qs]
    od = B.BF16 if w.dtype == "bf16" else B.F32

    if append:
        torch.cuda.synchronize()
        for b in range(w.batch):
            ctx.set_tail_len(b, 0)
        step_no[0] = 0
        hk = [t.cpu().pin_memory() for t in new_k]
        hv = [t.cpu().pin_memory() for t in new_v]

    # one call per step: every layer's query (and new rows) in one pinned buffer each, all outputs back in one
    hq_all = torch.stack(hq).pin_memory()                      # [L, batch, Hq, d]
    hout_all = torch.empty(hq_all.shape, dtype=tdt).pin_memory()
    if append:
        hk_all = torch.stack(hk).transpose(0, 1).contiguous().pin_memory()  # [step, L, batch, Hkv, d]
        hv_all = torch.stack(hv).transpose(0, 1).contiguous().pin_memory()

    def host_step():
        j = step_no[0]
        if append:
            ctx.decode_step_host(hq_all, hk_all[j], hv_all[j], hout_all, od, stream=stream)
        else:
            ctx.decode_step_host(hq_all, None, None, hout_all, od, stream=stream)
        step_no[0] = j + 1

    for _ in range(min(warmup, 3)):
        host_step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        host_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_val, e2e_s = replicas.whole_job_rate(w.batch * steps, e2e_s, dist, dev)
    h2d = sum(q.numel() * q.element_size() for q in hq)
    if append:
        h2d += sum(2 * t[0].numel() * t[0].element_size() for t in hk)
    d2h = sum(o.numel() * o.element_size() for o in hout)
    assert ctx.device_status() == 0

    if rank != 0:
        return None
    # ---------------- CPU baseline: the oracle on a bounded sample, same box ----------------
    cpu = None
    if with_cpu_baseline:
        from oracle import fdkv_ref as R

        n_units = {"decode32k": 4, "decode128k": 2}.get(w.name, 2)
        ou = oracle_sample(w, n_units)
        reps = 3
        t_s = min(oracle_step(w, ou) for _ in range(reps))
        total_calls = w.n_layers * w.n_kv_heads * w.batch
        t_full = t_s * total_calls / (w.block_size * len(ou))
        cpu = {"value": w.batch / t_full, "unit": "tokens/s", "cores": R.threads(), "kind": "oracle",
               "sample": f"{w.block_size * len(ou)} of {total_calls} (layer, KV head) attention units of one decode step (float64), "
                         f"best of {reps}, scaled to the full step"}
        if w.block_size == 2 and w.residual_rule == 0:
            cpu["prefill"] = oracle_prefill_sample(w, units)

    layer_calls = w.n_layers
    avg_call_s = ms_per_step * 1e-3 / layer_calls
    achieved = step_bytes / layer_calls / avg_call_s / 1e9
    line = {
        "metric": "compressed-KV decode attention tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "context": w.T, "batch": w.batch, "layers": w.n_layers, "q_heads": w.n_q_heads,
                   "kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "keep": f"{w.keep_num}/{w.keep_den}",
                   "residual_rule": "tokens" if w.residual_rule == 1 else "entries", "rows": "e4m3" if w.row_format == 1 else w.dtype,
                   "block_size": w.block_size, "mode_mix_shared_residual_exact": mix, "launch": "cuda_graph" if graph is not None else "stream",
                   "l2": "inputs larger than L2 (each step streams the whole packed cache)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(w.name), "traffic_source": "ncu capture of one launch on the 4-layer cut, a constant (not measured per run)" if NCU_TRAFFIC_BYTES.get(w.name) else None,
                     "of": peak_kind, "frac_of_8TBps_spec": achieved / 8000.0,
                     "bytes_per_launch": step_bytes / layer_calls,
                     "kernel": "decode attention (one layer call: split-K partial + combine), averaged over the timed region"},
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_val, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * steps,
        "clocks": clocks,
        "prefill": {"compress_ms": compress_ms, "commit_ms": commit_ms, "compress_GBps_min_bytes": compress_min_bytes / compress_ms / 1e6,
                    "probe_ms": probe_ms, "probe_TFLOPs": probe_flops / probe_ms / 1e9, "launches": launches_prefill,
                    "probe_frac_of_bf16_peak": probe_flops / probe_ms / 1e9 / tf_peak,
                    "roofline": {
                        "split_select": {"bound": "hbm", "unit": "GB/s", "peak": hbm_peak, "of": peak_kind,
                                         "min_bytes": compress_min_bytes, "achieved_min_bytes": compress_min_bytes / compress_ms / 1e6,
                                         "frac_min_bytes": compress_min_bytes / compress_ms / 1e6 / hbm_peak,
                                         "moved_bytes": compress_moved_bytes,
                                         "achieved_moved_bytes": compress_moved_bytes / compress_ms / 1e6 if compress_moved_bytes else None,
                                         "frac_moved_bytes": compress_moved_bytes / compress_ms / 1e6 / hbm_peak if compress_moved_bytes else None,
                                         "kernels": "depth split + histogram, threshold, one-pass ordered select (one fdkv_compress_prefill call, CUDA events)"},
                        "probe": {"bound": "tensor", "unit": "TFLOP/s", "achieved": probe_flops / probe_ms / 1e9, "peak": tf_peak,
                                  "of": peak_kind + " bf16 burst (a millisecond kernel timed alone)", "frac": probe_flops / probe_ms / 1e9 / tf_peak,
                                  "flops": probe_flops, "kernels": "one fdkv_probe call (error products of both candidates + mode rule, CUDA events)"}}},
        "step_bytes": step_bytes,
    }
    pf.ctx.close()
    del pf, ctx, qs, outs
    torch.cuda.empty_cache()
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="decode32k")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="skip the second workload (decode128k) of the default run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2607_06519_b200 import synth

    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
