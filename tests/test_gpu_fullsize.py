"""Parity at the full workload sizes, in the launch configuration bench.py times.

The 8x8-torus d = 1e6 top-1 % step is compared whole (its full 500-step run is compared in
test_gpu_full_runs.py); the ResNet-50-sized rows (d = 25.6 M, 32 workers) are compared on a
sampled worker that the oracle follows for several steps together with the workers its result
depends on, plus properties that hold at any size (the S = W Xhat invariant on a coordinate
sample, carried against uncarried compression).
"""
import concurrent.futures
import os

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


CONE_STEPS = 4      # steps the sampled worker is followed for
CONE_ROW = 17       # the sampled worker (its cone 13..21 does not wrap around the ring)


def _segment_csr(m):
    """Rows 0..m-1 of a ring segment: interior rows mix with both neighbours at 1/3 each, in
    ascending column order (as the ring rows they stand for); the two end rows are never updated."""
    rp, col, val = [0], [], []
    for a in range(m):
        if 0 < a < m - 1:
            col += [a - 1, a, a + 1]; val += [1.0 / 3.0] * 3
        else:
            col.append(a); val.append(1.0)
        rp.append(len(col))
    return workloads.MixingCSR(m, np.asarray(rp, np.int32), np.asarray(col, np.int32), np.asarray(val, np.float32))


@pytest.mark.parametrize("name", ["c5_ring32_qsgd", "c5_ring32_topk"])
def test_config5_sampled_row_over_several_steps(name):
    """Worker 17 of the 32-ring after CONE_STEPS steps depends on workers 13..21 at the start.  The
    oracle follows that shrinking cone (it updates 7, 5, 3, 1 rows and forms 9, 7, 5, 3 messages);
    the library runs all 32 rows.  Every message the oracle forms and every row it updates is
    compared bit for bit at every step, so steps 2.. check what the update kernel prepared for
    them: carried top-k candidates selected by the emit kernel with its working arrays in global
    memory, and the gsgd_b messages the update kernel wrote."""
    wl = workloads.WORKLOADS[name]
    w = wl.mixing()
    n, d, T, i0 = wl.n, wl.d, CONE_STEPS, CONE_ROW
    if torch.cuda.mem_get_info()[0] < 24 * n * d + (4 << 30):
        pytest.skip("not enough free device memory for the 32 x 25.6M state")
    cone = list(range(i0 - T, i0 + T + 1))
    m = len(cone)
    for i in cone[1:-1]:    # the segment's column order is the ring's
        assert [int(c) for c in w.col[w.row_ptr[i]:w.row_ptr[i + 1]]] == [i - 1, i, i + 1]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    dX = torch.randn(n, d, device=DEV, generator=gen) * float(np.sqrt(wl.x_var))
    dXh = torch.randn(n, d, device=DEV, generator=gen) * 0.05
    dGs = [torch.randn(n, d, device=DEV, generator=gen) * float(np.sqrt(wl.g_var)) for _ in range(2)]
    dS = (dXh + torch.roll(dXh, 1, 0) + torch.roll(dXh, -1, 0)) * (1.0 / 3.0)   # S = W Xhat on the ring
    X = np.stack([dX[j].cpu().numpy() for j in cone])
    Xh = np.stack([dXh[j].cpu().numpy() for j in cone])
    S = np.stack([dS[j].cpu().numpy() for j in cone])
    Gs = [np.stack([g[j].cpu().numpy() for j in cone]) for g in dGs]
    seg = _segment_csr(m)
    p = oracle.Params(wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=21)
    ch = choco.Choco(w, d, wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=21)
    try:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
            for t in range(T):
                ch.sgd_step(dX, dXh, dS, dGs[t % 2], wl.eta, wl.gamma)
                # the oracle: messages of the rows within distance T - t (keyed by the true worker
                # number), then the rows within distance T - 1 - t
                send = [a for a in range(m) if abs(cone[a] - i0) <= T - t]
                upd = [a for a in range(m) if abs(cone[a] - i0) <= T - 1 - t]
                msgs = dict(zip(send, ex.map(
                    lambda a: oracle.compress(p, oracle.difference(X[a], Xh[a]), t, cone[a]), send)))
                list(ex.map(lambda a: oracle._apply_row(a, seg, X, Xh, S, Gs[t % 2], msgs, wl.eta, wl.gamma), upd))
                torch.cuda.synchronize()
                for a in send:
                    j, mm = cone[a], msgs[a]
                    if wl.q == "topk":
                        assert np.array_equal(choco.choco_read_message(ch.ctx, j, 0).view(np.uint32), mm.idx), (t, j)
                        assert np.array_equal(choco.choco_read_message(ch.ctx, j, 1).view(np.uint32),
                                              mm.val.view(np.uint32)), (t, j)
                    else:
                        assert np.array_equal(choco.choco_read_message(ch.ctx, j, 0).view(np.uint32), mm.bits), (t, j)
                        assert np.array_equal(choco.choco_read_message(ch.ctx, j, 1).view(np.float32), mm.norms), (t, j)
                        assert np.array_equal(choco.choco_read_message(ch.ctx, j, 2), mm.levels), (t, j)
                for a in upd:
                    j = cone[a]
                    _exact(dXh[j].cpu().numpy(), Xh[a], f"Xhat row {j} after step {t}")
                    _exact(dS[j].cpu().numpy(), S[a], f"S row {j} after step {t}")
                    _exact(dX[j].cpu().numpy(), X[a], f"X row {j} after step {t}")
        # property at any size: S = W Xhat still holds on a coordinate sample (float32 rounding)
        cols = torch.randint(0, d, (4096,), device=DEV)
        H = dXh[:, cols].double()
        want = (H + torch.roll(H, 1, 0) + torch.roll(H, -1, 0)) / 3.0
        assert float((dS[:, cols].double() - want).abs().max()) < 1e-5
        st = choco.choco_get_stats(ch.ctx)
        assert st["device_timeouts"] == 0 and st["exact_rows"] == 0, st
        if wl.q == "topk":
            # steps 2.. ran on the candidates the update kernel had collected
            assert st["prepared_rows"] + st["rescued_rows"] == n * (T - 1), st
            assert st["prepared_rows"] >= n * (T - 1) - 8, st
    finally:
        ch.close()


@pytest.mark.parametrize("name", ["c5_ring32_qsgd", "c5_ring32_topk"])
def test_config5_carried_compression_changes_nothing(name):
    """Five steps at full size with the compression carried from step to step (candidates and
    messages prepared by the update kernel) and five with every step compressing afresh from X
    and Xhat: the whole state must be identical."""
    wl = workloads.WORKLOADS[name]
    w = wl.mixing()
    n, d, steps = wl.n, wl.d, 5
    if torch.cuda.mem_get_info()[0] < 36 * n * d + (4 << 30):
        pytest.skip("not enough free device memory for two copies of the 32 x 25.6M state")
    gen = torch.Generator(device=DEV)
    gen.manual_seed(6)
    X0 = torch.randn(n, d, device=DEV, generator=gen) * float(np.sqrt(wl.x_var))
    Gs = [torch.randn(n, d, device=DEV, generator=gen) * float(np.sqrt(wl.g_var)) for _ in range(2)]
    out = []
    for carry in (True, False):
        ch = choco.Choco(w, d, wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=22)
        choco.choco_set_carry(ch.ctx, carry)
        st = [X0.clone(), torch.zeros_like(X0), torch.zeros_like(X0)]
        for t in range(steps):
            ch.sgd_step(st[0], st[1], st[2], Gs[t % 2], wl.eta, wl.gamma)
        torch.cuda.synchronize()
        stats = choco.choco_get_stats(ch.ctx)
        assert stats["device_timeouts"] == 0
        if wl.q == "topk":
            assert (stats["prepared_rows"] > 0) == carry
        out.append(st)
        ch.close()
    for a, b, what in zip(out[0], out[1], ("X", "Xhat", "S")):
        assert torch.equal(a, b), what
