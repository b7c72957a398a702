"""Full-length runs through the C interface against the stored runs of the CPU oracle.

tests/golden/full_runs.json (written by tests/golden/make_full_run_goldens.py, which calls the
oracle only) holds, for every run and at a few checkpoints up to its last step, the consensus
distance of Section 6 and bit check sums of X, Xhat and S.  Here the library repeats each run on
the same seeded inputs.  Acceptance: the consensus distance agrees within 1e-4 (relative) at every
checkpoint, last step included; and, because the library follows a fixed operation order, the
check sums of the whole float32 state are equal, i.e. the state is the oracle's bit for bit after
every one of the 200 to 2000 steps.  (Check sums are compared when the host-generated inputs have
the stored check sums, which they do wherever numpy draws the same normals.)

The d = 2000 logistic-regression runs evaluate their gradient on the host from the library's X at
every step; those also run the oracle beside the library, step by step.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "full_runs.json")
POOL = 8
MASK64 = (1 << 64) - 1


def _runs():
    with open(GOLDEN) as f:
        return json.load(f)["runs"]


def device_fingerprint(t: torch.Tensor) -> list:
    """workloads.fingerprint of a contiguous float32 device tensor, computed on the device
    (64-bit integer arithmetic wraps, which is the modulus the definition asks for)."""
    words = t.contiguous().view(torch.int32).reshape(-1).to(torch.int64) & 0xFFFFFFFF
    weight = torch.arange(words.numel(), device=t.device, dtype=torch.int64) % workloads.FINGERPRINT_MODULUS + 1
    return [f"{int(words.sum().item()) & MASK64:016x}", f"{int((words * weight).sum().item()) & MASK64:016x}"]


def test_device_fingerprint_is_the_host_one():
    a = workloads.normal_rows(3, 70001, 1.0, 5)
    a[1, 7] = -0.0
    want = [f"{v:016x}" for v in workloads.fingerprint(a)]
    assert device_fingerprint(torch.from_numpy(a).to(DEV)) == want


@pytest.mark.parametrize("name", ["c1_ring4_topk", "c3_ring8_sign", "c4_torus64_topk", "c4_torus64_topk_g004",
                                  "c4_torus64_topk_mom", "c6_social32_sign", "c6_social32_topk"])
def test_full_run_against_stored_oracle_run(name):
    gold = _runs()[name]
    wl = workloads.WORKLOADS[name]
    assert (wl.n, wl.d, wl.k, wl.gamma, wl.eta, wl.steps) == (gold["n"], gold["d"], gold["k"], gold["gamma"],
                                                               gold["eta"], gold["steps"])
    assert (wl.momentum, wl.weight_decay) == (gold.get("momentum", 0.0), gold.get("weight_decay", 0.0))
    seeds = gold["seeds"]
    w = wl.mixing()
    X0 = workloads.normal_rows(wl.n, wl.d, wl.x_var, seeds["x"])
    same_inputs = [f"{v:016x}" for v in workloads.fingerprint(X0)] == gold["inputs"]["X0"]
    dX = torch.from_numpy(X0).to(DEV)
    e0 = oracle.consensus_error(X0) if wl.d <= 4096 else None
    del X0
    dXh, dS = torch.zeros_like(dX), torch.zeros_like(dX)
    dM = torch.zeros_like(dX) if wl.momentum > 0 else None     # Algorithm 2
    pool = None
    if wl.sgd:
        pool = []
        for g, want in zip(workloads.gradient_pool(wl, POOL, seeds["g"]), gold["inputs"]["G"]):
            same_inputs = same_inputs and [f"{v:016x}" for v in workloads.fingerprint(g)] == want
            pool.append(torch.from_numpy(g).to(DEV))
    ch = choco.Choco(w, wl.d, wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=seeds["q"])
    try:
        got_e0 = choco.choco_consensus_error(ch.ctx, dX)
        assert abs(got_e0 - gold["e0"]) <= 1e-9 * gold["e0"]
        if e0 is not None:
            assert e0 == gold["e0"]
        cps = {c["step"]: c for c in gold["checkpoints"]}
        assert max(cps) == wl.steps
        for t in range(wl.steps):
            if dM is not None:
                ch.sgd_momentum_step(dX, dXh, dS, pool[t % POOL], dM, wl.eta, wl.gamma, wl.weight_decay, wl.momentum)
            elif pool is not None:
                ch.sgd_step(dX, dXh, dS, pool[t % POOL], wl.eta, wl.gamma)
            else:
                ch.gossip_step(dX, dXh, dS, wl.gamma)
            c = cps.get(t + 1)
            if c is None:
                continue
            rel = choco.choco_consensus_error(ch.ctx, dX) / gold["e0"]
            assert abs(rel - c["relative"]) <= 1e-4 * c["relative"], f"consensus distance after step {t + 1}"
            if same_inputs:
                for arr, key in ((dX, "X"), (dXh, "Xhat"), (dS, "S")) + (((dM, "M"),) if dM is not None else ()):
                    assert device_fingerprint(arr) == c[key], f"{key} after step {t + 1} differs from the oracle's"
        st = choco.choco_get_stats(ch.ctx)
        assert st["device_timeouts"] == 0
        if wl.q == "topk" and wl.d >= 100000:
            # the steady-state path: every step after the first selects among carried candidates
            assert st["prepared_rows"] >= 0.95 * wl.n * (wl.steps - 1), st
        assert same_inputs, "host-generated inputs differ from the stored ones: check sums were not compared"
    finally:
        ch.close()


@pytest.mark.parametrize("name", ["c2_ring16_randk", "c2_ring16_randk_g006", "c2_ring16_qsgd"])
def test_logistic_regression_full_run(name):
    """4096 samples per worker, 2000 steps; the gradient is the caller's (Algorithm 1), evaluated
    on the host from the library's X and handed to the library and to the oracle running beside it."""
    gold = _runs()[name]
    wl = workloads.WORKLOADS[name]
    seeds = gold["seeds"]
    w = wl.mixing()
    prob = workloads.LogisticProblem(wl.n, wl.d, gold["inputs"]["samples_per_worker"], seed=seeds["problem"])
    X = np.zeros((wl.n, wl.d), dtype=np.float32)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    dX, dXh, dS = (torch.from_numpy(a).to(DEV) for a in (X, Xh, S))
    p = oracle.Params(wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=seeds["q"])
    ch = choco.Choco(w, wl.d, wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=seeds["q"])
    cps = {c["step"]: c for c in gold["checkpoints"]}
    grad_sum = 0
    try:
        for t in range(wl.steps):
            G = prob.gradient(dX.cpu().numpy(), t)
            grad_sum = (grad_sum + workloads.fingerprint(G)[0]) & MASK64
            dG = torch.from_numpy(G).to(DEV)
            oracle.step(w, p, X, Xh, S, G, wl.eta, wl.gamma, t)
            ch.sgd_step(dX, dXh, dS, dG, wl.eta, wl.gamma)
            c = cps.get(t + 1)
            if c is None and (t + 1) % 100:
                continue
            # beside the oracle: identical state
            for got, want, what in ((dX, X, "X"), (dXh, Xh, "Xhat"), (dS, S, "S")):
                assert np.array_equal(got.cpu().numpy(), want), f"{what} after step {t + 1}"
            if c is None:
                continue
            e = choco.choco_consensus_error(ch.ctx, dX)
            assert abs(e - c["consensus"]) <= 1e-4 * c["consensus"], f"consensus distance after step {t + 1}"
            if f"{grad_sum:016x}" == c["gradients_so_far"]:    # the host formed the stored gradients
                for arr, key in ((dX, "X"), (dXh, "Xhat"), (dS, "S")):
                    assert device_fingerprint(arr) == c[key], f"{key} after step {t + 1}"
        assert np.isfinite(X).all()
        if wl.gamma < 0.05 or wl.q == "qsgd":
            assert prob.loss(X.mean(axis=0)) < gold["loss_at_zero"] - 0.01
        assert choco.choco_get_stats(ch.ctx)["device_timeouts"] == 0
    finally:
        ch.close()
