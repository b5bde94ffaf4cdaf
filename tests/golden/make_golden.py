"""Writes tests/golden/tiny_*.json from the CPU oracle alone (never from the CUDA path).

Workload: the tiny correctness case (1 layer pair, 4 query heads, 2 KV heads, d = 64, T = 512, keep 1/8,
probe window = last 32 positions, seed 0), once with float32 storage and once with the same draws rounded to
bf16.  Stored: selection summaries, probe errors (Eq. 2 error term), Omega, modes over a lambda sweep, and
decode outputs (first channels) under each forced mode.  Run: python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import fdkv_ref as R  # noqa: E402
from paper_2607_06519_b200 import synth  # noqa: E402

LAMBDAS = [0.0, 50.0, 300.0, 3000.0, 1e4]


def make(dtype: str) -> dict:
    w = synth.WORKLOADS["tiny"].scaled(dtype=dtype)
    bf16 = dtype == "bf16"
    pos = synth.probe_positions(w)
    pq = (synth.probe_q(w, 0, 0), synth.probe_q(w, 0, 1))
    dq = [synth.decode_q(w, 0, layer)[0] for layer in range(2)]
    out = {"workload": "tiny", "dtype": dtype, "k_keep": w.k_keep, "lambdas": LAMBDAS, "heads": []}
    om = R.omega(w.T, w.head_dim, 2 if bf16 else 4, w.k_keep)
    out["omega"] = om.tolist()
    for h in range(w.n_kv_heads):
        k0, k1 = synth.unit_tensor(w, 0, 0, h, False)
        v0, v1 = synth.unit_tensor(w, 0, 0, h, True)
        u = R.Unit(k0, k1, v0, v1, bf16, w.keep_num, w.keep_den)
        rec = {"needles": synth.needle_positions(w, 0, 0, h).tolist()}
        for name in ("k", "v"):
            z1 = u.z1[name].ravel()
            kept = u.kept[name]
            keys = z1.view(np.uint32) & 0x7FFFFFFF
            tau = int(keys[kept].min())
            rec[name] = {
                "tau_key": tau, "n_gt": int((keys > tau).sum()), "n_eq": int((keys == tau).sum()),
                "idx_head": kept[:6].tolist(), "idx_sum": int(kept.astype(np.int64).sum()),
                "val_sum": float(z1[kept].astype(np.float64).sum()),
                "z0_sum": float(u.z0[name].astype(np.float64).sum()),
            }
        e_sh, e_rs = R.probe_error(u.z1["k"], u.kept["k"], pq[0], pq[1], w.group, h, pos)
        rec["e_shared"], rec["e_residual"] = e_sh, e_rs
        rec["modes"] = [R.mode_rule(e_sh, e_rs, om, lam)[0] for lam in LAMBDAS]
        s = R.token_scores(u.z1["k"], pq[0], pq[1], w.group, h, pos)
        tok = R.select_tokens(s, w.T // 8)
        rec["token_rule"] = {"tok_head": tok[:8].tolist(), "tok_sum": int(tok.sum())}
        rec["decode"] = {}
        for layer in range(2):
            q = dq[layer][h * w.group:(h + 1) * w.group]
            for mode, mname in enumerate(("shared", "residual", "exact")):
                o = u.attend(mode, layer, q)
                rec["decode"][f"l{layer}_{mname}"] = {"first3": o[:, :3].tolist(), "max_abs": float(np.abs(o).max())}
        out["heads"].append(rec)
    return out


if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    for dtype in ("f32", "bf16"):
        with open(os.path.join(here, f"tiny_{dtype}.json"), "w") as f:
            json.dump(make(dtype), f, indent=1)
        print("wrote", f.name)
