"""Per-layer compression (choco_layers_*) vs the oracle's step_layers, through the C interface.

Same acceptance as the plain step: indices, packed bits and level fields bit-exact, float32
state within 1e-5 * max|x| and, because the operation order is fixed, identical.
"""
import contextlib

import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads
from test_gpu_parity import DEV, _dev, _host, assert_state, check_messages

pytestmark = pytest.mark.gpu

RAGGED = [5, 1, 2048, 4097, 33, 12, 700]            # layers that start at every alignment

KINDS = [
    ("topk", dict(a=(1, 50))),
    ("randk", dict(a=(1, 50))),
    ("sign", dict()),
    ("qsgd", dict(s=16, bucket=512)),
    ("qsgd", dict(s=4, bucket=0)),
    ("identity", dict()),
    ("qsgd", dict(s=32768, bucket=256)),             # 16-bit level fields
]


def _run(w, sizes, kind, kw, steps, ld=None, momentum=False, gossip_only=False, seed=5,
         check_layers=(), stream=None, g_pool=0, invalidate_at=-1, jump=None, nesterov=False):
    """`stream`: run the steps on that (non-default) stream, where steady-state steps may be
    replayed from a captured graph; returns the number of steps replayed.  `g_pool` > 0: the
    gradients live in that many fixed device tensors that are refilled, so pointers repeat.
    `jump` = (i, t): before the i-th call the step number is set to t on both sides."""
    off = workloads.layer_offsets(sizes)
    n, d = w.n, int(off[-1])
    a_num, a_den = kw.get("a", (1, 1))
    X = workloads.normal_rows(n, d, 1.0, 31)
    for l in range(len(sizes)):                                  # a different scale per layer
        X[:, off[l]:off[l + 1]] *= np.float32(10.0 ** ((l % 5) - 2))
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    M = np.zeros_like(X) if momentum else None
    dX, dXh, dS = _dev(X, ld), _dev(Xh, ld), _dev(S, ld)
    dM = _dev(M, ld) if momentum else None
    p = oracle.Params(kind, s=kw.get("s", 16), bucket=kw.get("bucket", 0), seed=seed)
    h = choco.choco_layers_init(n, off, ld or d, w.row_ptr, w.col, w.val, kind, a_num, a_den,
                                s=kw.get("s", 16), bucket=kw.get("bucket", 0), seed=seed)
    if nesterov:
        choco.choco_layers_set_nesterov(h, True)
    pool = [_dev(np.zeros_like(X), ld) for _ in range(g_pool)]
    t_shift = 0
    torch.cuda.synchronize()
    ctx_mgr = torch.cuda.stream(stream) if stream is not None else contextlib.nullcontext()
    try:
        with ctx_mgr:
            for t in range(steps):
                G = None if gossip_only else workloads.normal_rows(n, d, 0.01, 100 + t)
                if gossip_only:
                    dG = None
                elif pool:
                    dG = pool[t % g_pool]
                    dG[:, :d].copy_(torch.from_numpy(G).to(DEV))
                else:
                    dG = _dev(G, ld)
                if t == invalidate_at:
                    choco.choco_layers_invalidate(h)
                if jump and t == jump[0]:
                    t_shift = jump[1] - t
                    choco.choco_layers_set_step(h, jump[1])
                msgs = oracle.step_layers(w, p, off, a_num, a_den, X, Xh, S, G, 0.05, 0.2, t + t_shift,
                                          M=M, lam=1e-4, beta=0.9, nesterov=nesterov)
                if gossip_only:
                    choco.choco_layers_gossip_step(h, dX, dXh, dS, 0.2)
                elif momentum:
                    choco.choco_layers_sgd_momentum_step(h, dX, dXh, dS, dG, dM, 0.05, 0.2, 1e-4, 0.9)
                else:
                    choco.choco_layers_sgd_step(h, dX, dXh, dS, dG, 0.05, 0.2)
                torch.cuda.synchronize()
                for l in check_layers:
                    ctx, o, length = choco.choco_layers_get_layer(h, l)
                    assert (o, length) == (int(off[l]), int(off[l + 1] - off[l]))
                    check_messages(ctx, kind, msgs[l], length)
                assert_state(_host(dX, d), X, f"X after step {t}")
                assert_state(_host(dXh, d), Xh, f"Xhat after step {t}")
                assert_state(_host(dS, d), S, f"S after step {t}")
                if momentum:
                    assert_state(_host(dM, d), M, f"M after step {t}")
            per_worker, total = choco.choco_layers_message_bytes(h)
            assert total == per_worker * n
            want = sum(next(iter(m.values())).paper_bytes(kind, int(off[l + 1] - off[l]), kw.get("s", 16))
                       for l, m in enumerate(msgs))
            assert per_worker == want
            for l in range(len(sizes)):
                ctx, _, _ = choco.choco_layers_get_layer(h, l)
                assert choco.choco_get_stats(ctx)["device_timeouts"] == 0
            # steps served without a launch per layer: replayed from a graph, or enqueued as
            # launches over all layers at once
            return choco.choco_layers_set_graphs(h) + choco.choco_layers_combined_steps(h)
    finally:
        choco.choco_layers_destroy(h)


@pytest.mark.parametrize("kind,kw", KINDS, ids=[k + "-" + "-".join(f"{a}{b}" for a, b in kw.items()) for k, kw in KINDS])
def test_ragged_layers(kind, kw):
    _run(workloads.torus(2, 4), RAGGED, kind, kw, steps=4, check_layers=range(len(RAGGED)))


@pytest.mark.parametrize("kind,kw", [KINDS[0], KINDS[2], KINDS[3]], ids=["topk", "sign", "qsgd"])
def test_resnet20_layers_on_a_ring(kind, kw):
    sizes = workloads.resnet20_layer_sizes()
    _run(workloads.ring(8), sizes, kind, dict(kw, a=(1, 100)), steps=3, check_layers=(0, 1, 3, 40, 64))


def test_nesterov_momentum_over_layers():
    # per-layer launches first, then the launches over all layers: both take the look-ahead step
    sizes = workloads.resnet20_layer_sizes()[:12]
    for kind, kw in (("topk", dict(a=(1, 20))), ("sign", {}), ("qsgd", dict(s=16, bucket=512))):
        served = _run(workloads.ring(4), sizes, kind, kw, steps=5, momentum=True, nesterov=True)
        assert served >= 2


def test_padded_rows_and_momentum():
    _run(workloads.ring(4), RAGGED, "topk", dict(a=(1, 20)), steps=3, ld=sum(RAGGED) + 11, momentum=True)
    _run(workloads.ring(4), RAGGED, "sign", {}, steps=3, ld=sum(RAGGED) + 8, momentum=True)


@pytest.mark.parametrize("kind,kw", [KINDS[0], KINDS[2], KINDS[5]], ids=["topk", "sign", "identity"])
def test_steady_steps_replayed_from_a_graph_give_the_same_bits(kind, kw):
    # on a stream that can be captured, with gradient buffers that repeat: the first steps run
    # kernel by kernel, each new (buffers, parity) combination is captured once, the rest replay
    replays = _run(workloads.torus(2, 4), RAGGED, kind, kw, steps=12, stream=torch.cuda.Stream(), g_pool=2,
                   check_layers=(0, 2, 3), invalidate_at=7)
    assert replays >= 4
    replays = _run(workloads.ring(4), RAGGED, kind, kw, steps=10, stream=torch.cuda.Stream(), g_pool=1,
                   momentum=True, ld=sum(RAGGED) + 4)
    assert replays >= 3


@pytest.mark.parametrize("kind,kw", [KINDS[1], KINDS[3], KINDS[4]], ids=["randk", "qsgd512", "qsgd-row"])
def test_replayed_steps_of_operators_keyed_by_the_step_number(kind, kw):
    # their generator takes the step number; a replayed launch must see the current one
    replays = _run(workloads.torus(2, 4), RAGGED, kind, kw, steps=14, stream=torch.cuda.Stream(), g_pool=2,
                   check_layers=(0, 2, 3), invalidate_at=6, jump=(4, 1000))
    assert replays >= 3


@pytest.mark.parametrize("kind,kw", [KINDS[0], KINDS[2], KINDS[3]], ids=["topk", "sign", "qsgd512"])
def test_steady_steps_are_launches_over_all_layers(kind, kw):
    """After the first step every step of these operators is enqueued as two or three launches
    whose blocks find their layer in a table, on any stream (here the default one), layers at
    every alignment included; an invalidation sends one step back to the layer-by-layer path."""
    combined = _run(workloads.torus(2, 4), RAGGED, kind, kw, steps=9, check_layers=range(len(RAGGED)),
                    invalidate_at=5)
    assert combined == 9 - 2
    combined = _run(workloads.ring(4), RAGGED, kind, kw, steps=6, momentum=True, ld=sum(RAGGED) + 4)
    assert combined == 6 - 1
    combined = _run(workloads.ring(4), [4096, 8192, 2048 * 3], kind, kw, steps=5, gossip_only=True)   # all aligned
    assert combined == 5 - 1


@pytest.mark.parametrize("kind,kw", [KINDS[0], KINDS[2], KINDS[3]], ids=["topk", "sign", "qsgd512"])
def test_resnet20_layers_for_thirty_steps(kind, kw):
    """The 65 ResNet-20 tensors on an 8-ring beside the oracle for 30 steps: all but the first
    step run as the launches over all layers."""
    sizes = workloads.resnet20_layer_sizes()
    combined = _run(workloads.ring(8), sizes, kind, dict(kw, a=(1, 100)), steps=30, check_layers=(0, 3, 64))
    assert combined == 29


def test_gossip_only_layers():
    _run(workloads.ring(4), RAGGED, "topk", dict(a=(1, 10)), steps=5, gossip_only=True)


def test_rejects_bad_layer_tables():
    w = workloads.ring(4)
    for off in ([1, 5], [0, 5, 5], [0, 7, 3]):
        with pytest.raises(choco.ChocoError):
            choco.choco_layers_init(4, np.asarray(off, np.int64), 16, w.row_ptr, w.col, w.val, "sign")
    with pytest.raises(choco.ChocoError):                        # ld shorter than the layers
        choco.choco_layers_init(4, np.asarray([0, 8, 32], np.int64), 16, w.row_ptr, w.col, w.val, "sign")
    with pytest.raises(choco.ChocoError):                        # a > 1
        choco.choco_layers_init(4, np.asarray([0, 8], np.int64), 8, w.row_ptr, w.col, w.val, "topk", 3, 2)
