"""Fit the compact model to a workload's synthetic trace with the oracle alone, and store the weights.

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  Section 4.1: "we trained our model and inference network using Adam
with gradient clipping on the data collected from the small cluster".  The recorded traces were never released,
so the data here is the first `--train-steps` steps of the named workload's seeded generator; what the
evaluation scores later are steps after those.

    python -m oracle.fit_elbo --workload n128 --out tests/golden/fitted_n128_compact.npz

Writes an .npz with one array per weight tensor (float32) plus "_meta" (a JSON string: workload, steps,
learning rate, seeds, ELBO per window at the logged steps).  Uses nothing but oracle/ and the seeded input
generators.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np

from oracle import elbo as L
from paper_1803_04209_b200 import inputs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="n128")
    ap.add_argument("--train-steps", type=int, default=1200, help="steps of the workload's trace to fit on")
    ap.add_argument("--iterations", type=int, default=6000)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--lr", type=float, default=2e-3)
    ap.add_argument("--clip", type=float, default=10.0)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--out", required=True)
    args = ap.parse_args()

    wl = inputs.WORKLOADS[args.workload]
    trace = inputs.workload_trace(wl, args.train_steps)
    start = inputs.workload_weights(wl, offsets=True)          # the same seeded initialisation the benchmark uses
    t0 = time.time()
    fitted, history = L.fit(start, trace, wl.lag, steps=args.iterations, batch=args.batch, lr=args.lr,
                            clip=args.clip, seed=args.seed, log_every=max(1, args.iterations // 20))
    meta = {"workload": wl.name, "N": wl.N, "D": wl.D, "H": wl.H, "lag": wl.lag, "train_steps": args.train_steps,
            "iterations": args.iterations, "batch": args.batch, "lr": args.lr, "clip": args.clip, "seed": args.seed,
            "elbo_per_window": history, "seconds": round(time.time() - t0, 1)}
    np.savez_compressed(args.out, _meta=np.array(json.dumps(meta)), **fitted)
    print(json.dumps(meta))


if __name__ == "__main__":
    main()
