"""Parity at the full workload sizes, in the launch configuration bench.py times.

The 8x8-torus d = 1e6 top-1 % step is compared whole; the ResNet-50-sized rows (d = 25.6 M,
32 workers) are compared on sampled workers that the oracle computes one by one, plus
properties that hold at any size (the S = W Xhat invariant on a coordinate sample, message
structure).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _exact(got, want, what):
    tol = 1e-5 * max(float(np.max(np.abs(want))), 1e-30)
    assert np.max(np.abs(got - want)) <= tol, what
    assert np.array_equal(got, want), what


def test_config4_full_step():
    wl = workloads.WORKLOADS["c4_torus64_topk"]
    w = wl.mixing()
    X = workloads.normal_rows(wl.n, wl.d, wl.x_var, 40)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    ch = choco.Choco(w, wl.d, "topk", k=wl.k)
    dX, dXh, dS = (torch.from_numpy(a).to(DEV) for a in (X, Xh, S))
    p = oracle.Params("topk", k=wl.k)
    for t in range(2):
        G = workloads.normal_rows(wl.n, wl.d, wl.g_var, 41 + t)
        dG = torch.from_numpy(G).to(DEV)
        msgs = oracle.step(w, p, X, Xh, S, G, wl.eta, wl.gamma, t)
        ch.sgd_step(dX, dXh, dS, dG, wl.eta, wl.gamma)
        torch.cuda.synchronize()
        for i in (0, 9, 63):
            idx = choco.choco_read_message(ch.ctx, i, 0).view(np.uint32)
            val = choco.choco_read_message(ch.ctx, i, 1).view(np.uint32)
            assert np.array_equal(idx, msgs[i].idx) and np.array_equal(val, msgs[i].val.view(np.uint32))
        _exact(dXh.cpu().numpy(), Xh, f"Xhat step {t}")
        _exact(dS.cpu().numpy(), S, f"S step {t}")
        _exact(dX.cpu().numpy(), X, f"X step {t}")
    st = choco.choco_get_stats(ch.ctx)
    assert st["exact_rows"] == 0
    ch.close()


@pytest.mark.parametrize("name", ["c5_ring32_qsgd", "c5_ring32_topk"])
def test_config5_sampled_rows(name):
    wl = workloads.WORKLOADS[name]
    w = wl.mixing()
    n, d = wl.n, wl.d
    free_b = torch.cuda.mem_get_info()[0]
    if free_b < 16 * n * d + (4 << 30):
        pytest.skip("not enough free device memory for the 32 x 25.6M state")
    sample = [0, 17]
    need = sorted({int(c) for i in sample for c in w.col[w.row_ptr[i]:w.row_ptr[i + 1]]})
    # device state generated on the device; the needed rows are copied to the host for the oracle
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    dX = torch.randn(n, d, device=DEV, generator=gen) * float(np.sqrt(wl.x_var))
    dXh = torch.randn(n, d, device=DEV, generator=gen) * 0.05
    dG = torch.randn(n, d, device=DEV, generator=gen) * float(np.sqrt(wl.g_var))
    # S must equal W Xhat: ring weights are 1/3
    dS = (dXh + torch.roll(dXh, 1, 0) + torch.roll(dXh, -1, 0)) * (1.0 / 3.0)
    hX = {j: dX[j].cpu().numpy() for j in need}
    hXh = {j: dXh[j].cpu().numpy() for j in need}
    hS = {j: dS[j].cpu().numpy() for j in sample}
    hG = {j: dG[j].cpu().numpy() for j in sample}
    ch = choco.Choco(w, d, wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=21)
    ch.sgd_step(dX, dXh, dS, dG, wl.eta, wl.gamma)
    torch.cuda.synchronize()
    p = oracle.Params(wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=21)
    msgs = {j: oracle.compress(p, oracle.difference(hX[j], hXh[j]), 0, j) for j in need}
    for j in need:
        if wl.q == "topk":
            assert np.array_equal(choco.choco_read_message(ch.ctx, j, 0).view(np.uint32), msgs[j].idx)
            assert np.array_equal(choco.choco_read_message(ch.ctx, j, 1).view(np.uint32),
                                  msgs[j].val.view(np.uint32))
        else:
            assert np.array_equal(choco.choco_read_message(ch.ctx, j, 0).view(np.uint32), msgs[j].bits)
            assert np.array_equal(choco.choco_read_message(ch.ctx, j, 1).view(np.float32), msgs[j].norms)
            assert np.array_equal(choco.choco_read_message(ch.ctx, j, 2), msgs[j].levels)
    pos = {j: a for a, j in enumerate(need)}
    for i in sample:
        # the oracle's row update on a sub-problem that holds only the needed workers
        sub_X = np.stack([hX[j] for j in need])
        sub_H = np.stack([hXh[j] for j in need])
        sub_S = np.zeros_like(sub_X)
        sub_S[pos[i]] = hS[i]
        sub_G = np.zeros_like(sub_X)
        sub_G[pos[i]] = hG[i]
        rp = np.zeros(len(need) + 1, np.int32)
        col, val = [], []
        for a, j in enumerate(need):
            if j == i:
                for e in range(w.row_ptr[i], w.row_ptr[i + 1]):
                    col.append(pos[int(w.col[e])]); val.append(float(w.val[e]))
            else:
                col.append(a); val.append(1.0)
            rp[a + 1] = len(col)
        sub_w = workloads.MixingCSR(len(need), rp, np.asarray(col, np.int32), np.asarray(val, np.float32))
        sub_msgs = {pos[j]: msgs[j] for j in need}
        oracle._apply_row(pos[i], sub_w, sub_X, sub_H, sub_S, sub_G, sub_msgs, wl.eta, wl.gamma)
        _exact(dXh[i].cpu().numpy(), sub_H[pos[i]], f"Xhat row {i}")
        _exact(dS[i].cpu().numpy(), sub_S[pos[i]], f"S row {i}")
        _exact(dX[i].cpu().numpy(), sub_X[pos[i]], f"X row {i}")
    # property at any size: S = W Xhat still holds on a coordinate sample (float32 rounding)
    cols = torch.randint(0, d, (4096,), device=DEV)
    H = dXh[:, cols].double()
    want = (H + torch.roll(H, 1, 0) + torch.roll(H, -1, 0)) / 3.0
    assert float((dS[:, cols].double() - want).abs().max()) < 1e-5
    assert choco.choco_get_stats(ch.ctx)["exact_rows"] == 0
    ch.close()
