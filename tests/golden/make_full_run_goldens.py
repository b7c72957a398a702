#!/usr/bin/env python
"""Writes tests/golden/full_runs.json: full-length runs of the CPU oracle on the seeded workloads.

    python tests/golden/make_full_run_goldens.py [--only NAME ...] [--threads T]

Imports `oracle` and `workloads` only; nothing here comes from the CUDA library.  For every run
the file holds, at a few checkpoints, the consensus distance of Section 6 relative to its
starting value, sum_i ||x_i - xbar||^2 / (the same at step 0), and bit check sums
(workloads.fingerprint) of X, Xhat and S.  A GPU test repeats the run through the C interface
on the same inputs and compares.  Check sums of the inputs are stored too, so that a reader on
another machine can tell "the inputs differ" from "the results differ".

Runs (Algorithm 1 in the three-vector form, oracle.step):
  c1_ring4_topk      4-ring, d = 1024, top-10, gossip only, 200 steps
  c2_ring16_randk    16-ring, logistic regression d = 2000 (4096 samples per worker), random-1 %,
                     gamma = 0.1 (diverges: the consensus distance grows without bound, values stay finite)
  c2_ring16_randk_g006   the same at gamma = 0.00625, the value Table 4 lists for random-1 %
  c2_ring16_qsgd     the same with gsgd_b, s = 16, one norm per row; 2000 steps each
  c3_ring8_sign      8-ring, d = 272 474, scaled sign, gradient pool of 8, 1000 steps
  c4_torus64_topk    8x8 torus, d = 1e6, top-1 %, gradient pool of 8, 500 steps, gamma = 0.2
  c4_torus64_topk_g004   the same at gamma = 0.04 (stable range; Table 4 lists 0.0375 for top-1 %)
  c4_torus64_topk_mom    the same with Algorithm 2 (momentum 0.9, weight decay 1e-4); M is check-summed too
  c6_social32_sign / c6_social32_topk   irregular 32-node graph (up to 15 messages per row), d = 272 474,
                     scaled sign / top-1 %, 1000 steps each
The d = 1e6 runs take about a quarter of an hour each on eight host threads.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)

import oracle      # noqa: E402
import workloads   # noqa: E402

OUT = os.path.join(HERE, "full_runs.json")
CHECKPOINTS = (1, 2, 5, 10, 50, 100, 200, 500, 1000, 2000)
POOL = 8                      # gradient tensors cycled through (step t uses tensor t mod POOL)
SEED_X, SEED_G, SEED_Q, SEED_PROBLEM = 40, 4100, 9, 3
RUNS = ("c1_ring4_topk", "c2_ring16_randk", "c2_ring16_randk_g006", "c2_ring16_qsgd", "c3_ring8_sign",
        "c4_torus64_topk", "c4_torus64_topk_g004", "c4_torus64_topk_mom", "c6_social32_sign", "c6_social32_topk")


def _fp(a):
    return [f"{v:016x}" for v in workloads.fingerprint(a)]


def run(name: str, executor) -> dict:
    wl = workloads.WORKLOADS[name]
    w = wl.mixing()
    p = oracle.Params(wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=SEED_Q)
    X = (workloads.normal_rows(wl.n, wl.d, wl.x_var, SEED_X) if wl.x_var > 0
         else np.zeros((wl.n, wl.d), dtype=np.float32))
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    M = np.zeros_like(X) if wl.momentum > 0 else None
    rec = {"workload": name, "n": wl.n, "d": wl.d, "graph": wl.graph, "Q": wl.q, "k": wl.k, "s": wl.s,
           "bucket": wl.bucket, "eta": wl.eta, "gamma": wl.gamma, "steps": wl.steps,
           "momentum": wl.momentum, "weight_decay": wl.weight_decay,
           "seeds": {"x": SEED_X, "g": SEED_G, "q": SEED_Q, "problem": SEED_PROBLEM},
           "inputs": {"X0": _fp(X)}, "checkpoints": []}
    problem, pool = None, None
    if name.startswith("c2_"):
        problem = workloads.LogisticProblem(wl.n, wl.d, 4096, seed=SEED_PROBLEM)
        rec["inputs"]["samples_per_worker"] = 4096
        rec["loss_at_zero"] = problem.loss(np.zeros(wl.d, dtype=np.float32))
    elif wl.sgd:
        pool = workloads.gradient_pool(wl, POOL, SEED_G)
        rec["inputs"]["G"] = [_fp(g) for g in pool]
    e0 = oracle.consensus_error(X)
    rec["e0"] = e0
    grad_sum = 0
    t_start = time.time()
    for t in range(wl.steps):
        if problem is not None:
            G = problem.gradient(X, t)
            grad_sum = (grad_sum + workloads.fingerprint(G)[0]) % (1 << 64)
        else:
            G = pool[t % POOL] if pool is not None else None
        oracle.step(w, p, X, Xh, S, G, wl.eta if G is not None else 0.0, wl.gamma, t, executor=executor,
                    M=M, lam=wl.weight_decay, beta=wl.momentum)
        if t + 1 in CHECKPOINTS or t + 1 == wl.steps:
            e = oracle.consensus_error(X)
            cp = {"step": t + 1, "consensus": e, "relative": (e / e0 if e0 > 0 else None),
                  "max_abs_x": float(np.max(np.abs(X))), "X": _fp(X), "Xhat": _fp(Xh), "S": _fp(S)}
            if M is not None:
                cp["M"] = _fp(M)
            if problem is not None:
                # the gradients follow X, so this running sum shows whether they were the same
                cp["gradients_so_far"] = f"{grad_sum:016x}"
                cp["loss_of_mean"] = problem.loss(X.mean(axis=0))
            rec["checkpoints"].append(cp)
            print(f"{name}: step {t + 1}  consensus {e:.6e}  ({time.time() - t_start:.0f} s)", flush=True)
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", nargs="*", default=list(RUNS))
    ap.add_argument("--threads", type=int, default=os.cpu_count() or 1)
    args = ap.parse_args()
    doc = {"about": ("Full-length runs of the CPU oracle (oracle.step: Algorithm 1, three vectors per worker) "
                     "written by tests/golden/make_full_run_goldens.py; consensus = sum_i ||x_i - xbar||^2 "
                     "(Section 6, times n) in float64; X / Xhat / S = workloads.fingerprint of the float32 state"),
           "runs": {}}
    if os.path.exists(OUT):
        with open(OUT) as f:
            doc["runs"] = json.load(f).get("runs", {})
    with concurrent.futures.ThreadPoolExecutor(max_workers=args.threads) as ex:
        for name in args.only:
            doc["runs"][name] = run(name, ex if args.threads > 1 else None)
            with open(OUT, "w") as f:
                json.dump(doc, f, indent=1)
                f.write("\n")


if __name__ == "__main__":
    main()
