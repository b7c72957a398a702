"""Small problems replay their steady-state step from a captured CUDA graph (on a stream that
can be captured).  The replayed steps must give the oracle's bits like any other step, through
invalidation, a change of the step number, momentum and changing gradient buffers."""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads
from test_gpu_parity import DEV, _dev, _host, assert_state, check_messages

pytestmark = pytest.mark.gpu

KINDS = [
    ("topk", dict(k=37)),
    ("randk", dict(k=37)),
    ("sign", dict()),
    ("qsgd", dict(s=16, bucket=512)),
    ("qsgd", dict(s=16, bucket=0)),
    ("identity", dict()),
]
IDS = ["topk", "randk", "sign", "qsgd512", "qsgd-row", "identity"]


def _run(kind, kw, steps, g_pool, momentum=False, gossip=False, invalidate_at=-1, jump=None,
         graphs=True, d=3001, ld=3004):
    w = workloads.torus(2, 4)
    n = w.n
    X = workloads.normal_rows(n, d, 1.0, 77)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    M = np.zeros_like(X) if momentum else None
    p = oracle.Params(kind, k=kw.get("k", 0), s=kw.get("s", 16), bucket=kw.get("bucket", 0), seed=11)
    ch = choco.Choco(w, d, kind, k=kw.get("k", 0), s=kw.get("s", 16), bucket=kw.get("bucket", 0), seed=11, ld=ld)
    if not graphs:
        choco.choco_set_graphs(ch.ctx, False)
    dX, dXh, dS = _dev(X, ld), _dev(Xh, ld), _dev(S, ld)
    dM = _dev(M, ld) if momentum else None
    pool = [_dev(np.zeros_like(X), ld) for _ in range(g_pool)]
    torch.cuda.synchronize()
    shift = 0
    try:
        with torch.cuda.stream(torch.cuda.Stream()):
            for t in range(steps):
                G = None if gossip else workloads.normal_rows(n, d, 0.01, 300 + t)
                dG = None
                if G is not None:
                    dG = pool[t % g_pool]
                    dG[:, :d].copy_(torch.from_numpy(G).to(DEV))
                if t == invalidate_at:
                    choco.choco_invalidate(ch.ctx)
                if jump and t == jump[0]:
                    shift = jump[1] - t
                    choco.choco_set_step(ch.ctx, jump[1])
                if momentum:
                    msgs = oracle.step(w, p, X, Xh, S, G, 0.05, 0.2, t + shift, M=M, lam=1e-3, beta=0.9)
                    ch.sgd_momentum_step(dX, dXh, dS, dG, dM, 0.05, 0.2, 1e-3, 0.9)
                elif gossip:
                    msgs = oracle.step(w, p, X, Xh, S, None, 0.0, 0.2, t + shift)
                    ch.gossip_step(dX, dXh, dS, 0.2)
                else:
                    msgs = oracle.step(w, p, X, Xh, S, G, 0.05, 0.2, t + shift)
                    ch.sgd_step(dX, dXh, dS, dG, 0.05, 0.2)
                torch.cuda.synchronize()
                check_messages(ch.ctx, kind, msgs, d)
                assert_state(_host(dX, d), X, f"X after step {t}")
                assert_state(_host(dXh, d), Xh, f"Xhat after step {t}")
                assert_state(_host(dS, d), S, f"S after step {t}")
                if momentum:
                    assert_state(_host(dM, d), M, f"M after step {t}")
            st = choco.choco_get_stats(ch.ctx)
            assert st["device_timeouts"] == 0 and st["steps"] == steps
            assert choco.choco_get_step(ch.ctx) == steps + shift
            return st["graph_replays"]
    finally:
        ch.close()


@pytest.mark.parametrize("kind,kw", KINDS, ids=IDS)
def test_replayed_steps_match_the_oracle(kind, kw):
    assert _run(kind, kw, steps=16, g_pool=2, invalidate_at=9, jump=(6, 500)) >= 4


@pytest.mark.parametrize("kind,kw", [KINDS[0], KINDS[2], KINDS[3]], ids=["topk", "sign", "qsgd512"])
def test_replay_with_momentum_and_gossip_only(kind, kw):
    assert _run(kind, kw, steps=10, g_pool=1, momentum=True) >= 3
    assert _run(kind, kw, steps=10, g_pool=1, gossip=True) >= 3


def test_graphs_can_be_turned_off_and_fresh_buffers_are_never_captured():
    assert _run("sign", {}, steps=8, g_pool=1, graphs=False) == 0
    assert _run("topk", dict(k=37), steps=8, g_pool=8) == 0       # every gradient buffer seen once


def test_large_problems_do_not_replay():
    w = workloads.ring(4)
    d = 1_100_000                                                  # n d above the limit
    ch = choco.Choco(w, d, "sign", seed=1)
    X = torch.randn(4, d, device=DEV)
    Xh, S, G = torch.zeros_like(X), torch.zeros_like(X), torch.zeros_like(X)
    torch.cuda.synchronize()
    with torch.cuda.stream(torch.cuda.Stream()):
        for _ in range(6):
            ch.sgd_step(X, Xh, S, G, 0.1, 0.1)
        assert choco.choco_get_stats(ch.ctx)["graph_replays"] == 0
    ch.close()
