"""The timeout status: a kernel's bounded wait that runs out must surface as CHOCO_ERR_TIMEOUT.

No GPU is stalled for this.  The context's test hook sets the number of polls of the kernels'
first wait to zero, so every block "gives up" at once, then sits out its (perfectly healthy)
copies in the second bounded wait and returns without writing its results.  The calls that
synchronise must then report the status, the next step call must refuse, and a fresh context
must carry on from a checkpoint bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("kind,kw", [("topk", dict(k=200)), ("sign", {}), ("qsgd", dict(s=16, bucket=512))])
def test_timeout_is_reported_and_a_fresh_context_recovers(kind, kw):
    w = workloads.ring(4)
    n, d = 4, 20000
    p = oracle.Params(kind, seed=3, **kw)
    X = workloads.normal_rows(n, d, 1.0, 1)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    G = [workloads.normal_rows(n, d, 0.01, 10 + t) for t in range(4)]
    dG = [torch.from_numpy(g).to(DEV) for g in G]
    dX, dXh, dS = (torch.from_numpy(a).to(DEV) for a in (X, Xh, S))
    ch = choco.Choco(w, d, kind, seed=3, **kw)
    for t in range(2):
        oracle.step(w, p, X, Xh, S, G[t], 0.1, 0.2, t)
        ch.sgd_step(dX, dXh, dS, dG[t], 0.1, 0.2)
    assert choco.choco_get_stats(ch.ctx)["device_timeouts"] == 0
    saved = [t.clone() for t in (dX, dXh, dS)]            # a checkpoint after step 2

    choco.choco_debug_set_wait_polls(ch.ctx, 0)
    ch.sgd_step(dX, dXh, dS, dG[2], 0.1, 0.2)              # enqueued; a step call cannot know yet
    with pytest.raises(choco.ChocoError) as err:
        choco.choco_get_stats(ch.ctx)
    assert err.value.code == choco.ERR_TIMEOUT
    torch.cuda.synchronize()                               # the device is alive and well
    for call in (lambda: ch.sgd_step(dX, dXh, dS, dG[3], 0.1, 0.2),
                 lambda: choco.choco_consensus_error(ch.ctx, dX),
                 lambda: choco.choco_read_message(ch.ctx, 0, 0)):
        with pytest.raises(choco.ChocoError) as err:
            call()
        assert err.value.code == choco.ERR_TIMEOUT
    assert choco.choco_get_step(ch.ctx) == 3               # the refused call did not count
    ch.close()

    # recovery: a fresh context on the checkpoint carries on as if nothing had happened
    ch2 = choco.Choco(w, d, kind, seed=3, **kw)
    choco.choco_set_step(ch2.ctx, 2)
    for t in (2, 3):
        oracle.step(w, p, X, Xh, S, G[t], 0.1, 0.2, t)
        ch2.sgd_step(saved[0], saved[1], saved[2], dG[t], 0.1, 0.2)
    torch.cuda.synchronize()
    assert choco.choco_get_stats(ch2.ctx)["device_timeouts"] == 0
    for got, want in zip(saved, (X, Xh, S)):
        assert np.array_equal(got.cpu().numpy(), want)
    ch2.close()
