"""Top-k rows whose guessed candidate bound misses are re-collected by the grid-wide rescue
kernels (on by default only for very long rows; switched on here for short ones).  The result
must be the oracle's either way."""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads
from test_gpu_parity import DEV, _dev, _host, assert_state, check_messages

pytestmark = pytest.mark.gpu


def _run(d, ld, k, rescue, burst_steps, steps=9, n=8, select_blocks=None):
    """`burst_steps`: steps whose gradient is -50 x / eta, so that x grows 51-fold and nearly
    every coordinate of the next x - x^ exceeds the bound guessed before the burst."""
    w = workloads.torus(2, 4)
    eta, gamma = 0.05, 0.2
    X = workloads.normal_rows(n, d, 1.0, 9)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    p = oracle.Params("topk", k=k)
    ch = choco.Choco(w, d, "topk", k=k, ld=ld)
    choco.choco_set_rescue(ch.ctx, rescue)
    if select_blocks:
        choco.choco_set_select_blocks(ch.ctx, select_blocks)
    dX, dXh, dS = _dev(X, ld), _dev(Xh, ld), _dev(S, ld)
    try:
        for t in range(steps):
            if t in burst_steps:
                G = (X * np.float32(-50.0 / eta)).astype(np.float32)
            else:
                G = workloads.normal_rows(n, d, 0.01, 700 + t)
            dG = _dev(G, ld)
            msgs = oracle.step(w, p, X, Xh, S, G, eta, gamma, t)
            ch.sgd_step(dX, dXh, dS, dG, eta, gamma)
            torch.cuda.synchronize()
            check_messages(ch.ctx, "topk", msgs, d)
            assert_state(_host(dX, d), X, f"X after step {t}")
            assert_state(_host(dXh, d), Xh, f"Xhat after step {t}")
            assert_state(_host(dS, d), S, f"S after step {t}")
        st = choco.choco_get_stats(ch.ctx)
        assert st["device_timeouts"] == 0
        return st
    finally:
        ch.close()


@pytest.mark.parametrize("d,ld,k", [(50_000, 50_000, 500), (40_003, 40_003, 401), (300_000, 300_004, 300)])
def test_bursts_are_rescued(d, ld, k):
    st = _run(d, ld, k, True, burst_steps=(3, 6))
    assert st["rescued_rows"] >= 8, st              # every row of the step after a burst
    off = _run(d, ld, k, False, burst_steps=(3, 6))
    assert off["rescued_rows"] == 0 and off["exact_rows"] >= 8, off


@pytest.mark.parametrize("blocks", [2, 4])
def test_bursts_with_a_cluster_of_blocks_per_row(blocks):
    """The same with the selection kernel's cluster form: a row whose candidates are unusable is
    handed to the rescue kernels (or selected exactly) by the cluster's first block alone."""
    st = _run(50_000, 50_000, 500, True, burst_steps=(3, 6), select_blocks=blocks)
    assert st["rescued_rows"] >= 8, st
    off = _run(40_003, 40_003, 401, False, burst_steps=(3, 6), select_blocks=blocks)
    assert off["rescued_rows"] == 0 and off["exact_rows"] >= 8, off


def test_rescue_kernels_do_nothing_in_quiet_steps():
    st = _run(50_000, 50_000, 500, True, burst_steps=())
    assert st["rescued_rows"] == 0 and st["exact_rows"] == 0


def test_magnitudes_in_one_first_digit_bin_are_resolved_by_the_second_digit():
    # all magnitudes inside one eighth of an octave (the shape x - x^ takes under the last
    # threshold once the largest entries have been sent): the second 11 bits separate them
    n, d, k = 4, 60_000, 300
    w = workloads.ring(n)
    rng = np.random.default_rng(5)
    X = (rng.uniform(1.0, 1.04, size=(n, d)) * rng.choice([-1.0, 1.0], size=(n, d))).astype(np.float32)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    p = oracle.Params("topk", k=k)
    for rescue in (False, True):
        ch = choco.Choco(w, d, "topk", k=k)
        choco.choco_set_rescue(ch.ctx, rescue)
        hX, hXh, hS = X.copy(), Xh.copy(), S.copy()
        dX, dXh, dS = _dev(hX), _dev(hXh), _dev(hS)
        try:
            for t in range(3):
                msgs = oracle.step(w, p, hX, hXh, hS, None, 0.0, 0.1, t)
                ch.gossip_step(dX, dXh, dS, 0.1)
                torch.cuda.synchronize()
                check_messages(ch.ctx, "topk", msgs, d)
                assert_state(_host(dX, d), hX, f"X after step {t}")
            assert choco.choco_get_stats(ch.ctx)["exact_rows"] == 0
        finally:
            ch.close()


def test_keys_that_agree_in_22_bits_still_fall_back_to_the_exact_selection():
    # a handful of distinct magnitudes, each shared by thousands of coordinates: no bound on
    # the leading 22 bits can cut a row down to the candidate capacity; ties go to the lower index
    n, d, k = 4, 60_000, 300
    w = workloads.ring(n)
    rng = np.random.default_rng(6)
    mags = np.float32(1.0) + rng.integers(0, 4, size=(n, d)).astype(np.float32) * np.float32(2.0 ** -23)
    X = (mags * rng.choice([-1.0, 1.0], size=(n, d))).astype(np.float32)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    p = oracle.Params("topk", k=k)
    ch = choco.Choco(w, d, "topk", k=k)
    choco.choco_set_rescue(ch.ctx, True)
    dX, dXh, dS = _dev(X), _dev(Xh), _dev(S)
    try:
        for t in range(3):
            msgs = oracle.step(w, p, X, Xh, S, None, 0.0, 0.1, t)
            ch.gossip_step(dX, dXh, dS, 0.1)
            torch.cuda.synchronize()
            check_messages(ch.ctx, "topk", msgs, d)
            assert_state(_host(dX, d), X, f"X after step {t}")
        assert choco.choco_get_stats(ch.ctx)["exact_rows"] >= n
    finally:
        ch.close()


def test_only_top_k_has_rescue_kernels():
    ch = choco.Choco(workloads.ring(4), 1000, "sign")
    with pytest.raises(choco.ChocoError):
        choco.choco_set_rescue(ch.ctx, True)
    choco.choco_set_rescue(ch.ctx, False)
    ch.close()
