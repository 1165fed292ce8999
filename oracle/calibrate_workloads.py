"""Measure the block sparsity each synthetic workload reaches under the oracle's Stage 1.

Run from the repository root:  python -m oracle.calibrate_workloads [name ...]

For every named workload (default: all) it generates the seeded inputs on the CPU, routes an
evenly spaced sample of rows with ``dash_oracle.route_row`` and writes
``tests/golden/calibration.json``: achieved sparsity 1 - sum(|S_i|+1)/sum(c_i+1), mean support
size and the generator parameters (rho, shift) it was measured at.  The rho/shift values frozen
in the workload table were chosen by re-running this script until the 75 % / 90 % targets were met.
It calls only the oracle and the input generator.
"""
from __future__ import annotations

import json
import os
import sys

import numpy as np
import torch

from oracle import dash_oracle as orc
from paper_2605_18753_b200 import synth

OUT = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "tests", "golden", "calibration.json")


def measure(w: synth.Workload, n_rows: int = 384, kv_heads=(0, 5)) -> dict:
    B = w.block
    if w.kind == "prefill":
        inp = synth.make_prefill_inputs(w.with_(batch=1), "cpu")
        n = w.seq
        rows = np.unique(np.linspace(0, n - 1, n_rows).astype(np.int64))
        sup, vis = [], []
        for r in [h for h in kv_heads if h < w.h_kv]:
            K = inp["K"][0, :, r:r + 1].double().numpy()
            Kbar = orc.block_summaries(K, B)[:, 0]
            g_q = w.h_q // w.h_kv
            Qr = inp["Q"][0, :, r * g_q:(r + 1) * g_q].double().numpy()
            for i in rows:
                c_i = int(i) // B
                rt = orc.route_row(Qr[i], Kbar, c_i, w.alpha, w.gamma, w.sigma)
                sup.append(rt.support.size)
                vis.append(c_i)
    else:
        wb = w.with_(batch=2)
        inp = synth.make_decode_inputs(wb, "cpu")
        sup, vis = [], []
        g_q = w.h_q // w.h_kv
        for bb in range(wb.batch):
            for r in range(w.h_kv):
                K = inp["K"][bb, :, r:r + 1].double().numpy()
                Kbar = orc.block_summaries(K, B)[:, 0]
                c_i = (w.seq - 1) // B
                q = inp["Q"][bb, r * g_q:(r + 1) * g_q].double().numpy()
                rt = orc.route_row(q, Kbar, c_i, w.alpha, w.gamma, w.sigma)
                sup.append(rt.support.size)
                vis.append(c_i)
    return {"workload": w.name, "alpha": w.alpha, "block": w.block, "gamma": w.gamma, "rho": w.rho,
            "shift": w.shift, "rows_sampled": len(sup),
            "block_sparsity": round(orc.block_sparsity(sup, vis), 4),
            "mean_support": round(float(np.mean(sup)), 2)}


def main(argv):
    names = argv or [k for k in synth.WORKLOADS]
    results = {}
    if os.path.exists(OUT):
        with open(OUT) as f:
            results = json.load(f)
    for name in names:
        if name == "sweep_32k":
            for B in (64, 128):
                for alpha in (1.25, 1.5, 2.0):
                    w = synth.workload(name, block=B, alpha=alpha)
                    res = measure(w)
                    results[f"{name}_B{B}_a{alpha}"] = res
                    print(res, flush=True)
            continue
        res = measure(synth.workload(name))
        results[name] = res
        print(res, flush=True)
    with open(OUT, "w") as f:
        json.dump(results, f, indent=1, sort_keys=True)


if __name__ == "__main__":
    torch.set_num_threads(8)
    main(sys.argv[1:])
