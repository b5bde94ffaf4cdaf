"""Writes tests/golden/probe_errors_decode32k.json from the CPU oracle alone (never from the CUDA path).

Workload: the 32k prefill case (32 layers = 16 pairs, 8 KV heads, group 4, d = 128, T = 32768, bf16, keep 1/16, probe
window = last 64 positions, seed 2).  For each of the 128 units the oracle regenerates the unit's K tensors from the
seed, applies Eq. 1 and the entry-form selection, and evaluates the error term of Eq. 2 for the shared and the residual
candidate in float64.  Stored: the 128 x 2 errors, Omega, and the lambdas of the full-size mode test (the calibrated lambda*, lambda* / 64,
lambda* x 64, and one that splits the units between residual and exact) with the
modes the rule of Eq. 3 gives there and its smallest margin.  Takes a few minutes per core-hour of oracle work
(about 15-25 minutes on 8 cores).  Run: python tests/golden/make_probe_errors_32k.py
"""
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import fdkv_ref as R  # noqa: E402
from paper_2607_06519_b200 import synth  # noqa: E402


def lambda_star(e_sh, e_rs, om):
    """Geometric mean of the two middle per-unit shared<->residual break-evens (E_sh - E_rs) / (Omega_r - Omega_s):
    the lambda at which the rule splits the units 50 / 50 between shared and residual with the largest margin."""
    be = np.sort(((e_sh - e_rs) / (om[1] - om[0])).ravel())
    n = be.size
    return float(np.sqrt(be[n // 2 - 1] * be[n // 2]))


def modes_and_margin(e_sh, e_rs, om, lam):
    modes, margin = [], np.inf
    for a, b in zip(e_sh.ravel(), e_rs.ravel()):
        m, _, mg = R.mode_rule(a, b, om, lam)
        modes.append(m)
        margin = min(margin, mg)
    return modes, float(margin)


def main():
    w = synth.WORKLOADS["decode32k"]
    pos = synth.probe_positions(w)
    e = np.zeros((w.n_pairs, w.n_kv_heads, 2))
    t0 = time.time()
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "probe_errors_decode32k.json")
    reuse = "--reuse-errors" in sys.argv and os.path.exists(path)  # only rebuild the lambda cases from the stored errors
    if reuse:
        old = json.load(open(path))
        e[..., 0], e[..., 1] = np.asarray(old["e_shared"]), np.asarray(old["e_residual"])
    for p in range(0 if reuse else w.n_pairs):
        pq = (synth.probe_q(w, 0, 2 * p), synth.probe_q(w, 0, 2 * p + 1))
        for h in range(w.n_kv_heads):
            k0, k1 = synth.unit_tensor(w, 0, p, h, False)
            _, z1 = R.depth_split(k0, k1, True)
            kept = R.select_entries(z1, w.k_keep)
            e[p, h] = R.probe_error(z1, kept, pq[0], pq[1], w.group, h, pos)
            print(f"pair {p} head {h}: {e[p, h].tolist()}  ({time.time() - t0:.0f} s)", flush=True)
    om = R.omega(w.T, w.head_dim, 2, w.k_keep)
    lam = lambda_star(e[..., 0], e[..., 1], om)
    out = {"workload": "decode32k", "omega": om.tolist(), "e_shared": e[..., 0].tolist(), "e_residual": e[..., 1].tolist(),
           "cases": []}
    # a fourth lambda between the units' residual<->exact break-evens E_rs / (1 - Omega_r): half residual, half exact
    be_re = np.sort((e[..., 1] / (om[2] - om[1])).ravel())
    lam_re = float(np.sqrt(be_re[be_re.size // 2 - 1] * be_re[be_re.size // 2]))
    for name, l in (("lambda_star", lam), ("lambda_star/64", lam / 64), ("lambda_star*64", lam * 64), ("residual_exact_split", lam_re)):
        # the rule is only comparable where its decision is not a coin toss of the last bits: move lambda in 1 % steps
        # until the smallest relative margin between the best and the second-best loss is at least 1e-3
        modes, margin = modes_and_margin(e[..., 0], e[..., 1], om, l)
        while margin < 1e-3:
            l *= 1.01
            modes, margin = modes_and_margin(e[..., 0], e[..., 1], om, l)
        out["cases"].append({"name": name, "lambda": l, "modes": modes, "min_margin": margin})
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)


if __name__ == "__main__":
    main()
