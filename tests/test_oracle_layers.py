"""Pins for the oracle's per-layer compression (Section 5, "Setup": every compression scheme
is applied to every layer separately), against definitions written out in numpy."""
import numpy as np

import oracle
import workloads

OFF = workloads.layer_offsets([40, 3, 700, 1, 256, 130])     # ragged, with tiny layers
D = int(OFF[-1])


def _state(n, seed, scales=None):
    X = workloads.normal_rows(n, D, 1.0, seed)
    if scales is not None:                                     # a different magnitude per layer
        for l, sc in enumerate(scales):
            X[:, OFF[l]:OFF[l + 1]] *= np.float32(sc)
    return X, np.zeros_like(X), np.zeros_like(X)


def test_layer_k_is_floor_with_a_floor_of_one():
    assert oracle.layer_k(1, 100, 432) == 4
    assert oracle.layer_k(1, 100, 36864) == 368
    assert oracle.layer_k(1, 100, 16) == 1          # floor(0.16) = 0 would silence the layer
    assert oracle.layer_k(1, 1, 7) == 7


def test_resnet20_shape():
    sizes = workloads.resnet20_layer_sizes()
    assert len(sizes) == 65 and sum(sizes) == 272474
    assert sizes[0] == 3 * 16 * 9 and sizes[-2:] == [640, 10] and max(sizes) == 64 * 64 * 9


def test_identity_does_not_see_layers():
    w = workloads.ring(5)
    X, Xh, S = _state(5, 1)
    G = workloads.normal_rows(5, D, 0.01, 2)
    A = [a.copy() for a in (X, Xh, S)]
    p = oracle.Params("identity")
    for t in range(3):
        oracle.step(w, p, X, Xh, S, G, 0.05, 0.3, t)
        oracle.step_layers(w, p, OFF, 1, 1, A[0], A[1], A[2], G, 0.05, 0.3, t)
    for a, b in zip((X, Xh, S), A):
        assert np.array_equal(a, b)


def test_topk_is_brute_force_inside_every_layer():
    n = 4
    w = workloads.ring(n)
    scales = [1.0, 50.0, 0.01, 3.0, 1000.0, 0.5]               # whole-row top-k would pick layer 4 only
    X, Xh, S = _state(n, 3, scales)
    X0 = X.copy()
    msgs = oracle.step_layers(w, oracle.Params("topk"), OFF, 1, 20, X, Xh, S, None, 0.0, 0.2, 0)
    total = 0
    for l in range(len(OFF) - 1):
        lo, hi = int(OFF[l]), int(OFF[l + 1])
        k = max(1, (hi - lo) // 20)
        total += k
        for i in range(n):
            v = X0[i, lo:hi]
            key = np.abs(v).view(np.uint32).astype(np.int64)
            order = np.lexsort((np.arange(hi - lo), -key))      # |v| descending, then index ascending
            want = np.sort(order[:k]).astype(np.uint32)
            assert np.array_equal(msgs[l][i].idx, want), (l, i)
            assert np.array_equal(msgs[l][i].val, v[want])
            q = np.zeros(hi - lo, np.float32)
            q[want] = v[want]
            assert np.array_equal(Xh[i, lo:hi], q)              # x^ = 0 + q
    assert total == sum(m[0].idx.shape[0] for m in msgs)


def test_sign_scale_is_the_layers_own_mean_magnitude():
    n = 3
    w = workloads.ring(n)
    scales = [1.0, 50.0, 0.01, 3.0, 1000.0, 0.5]
    X, Xh, S = _state(n, 4, scales)
    X0 = X.copy()
    msgs = oracle.step_layers(w, oracle.Params("sign"), OFF, 1, 1, X, Xh, S, None, 0.0, 0.1, 0)
    for l in range(len(OFF) - 1):
        lo, hi = int(OFF[l]), int(OFF[l + 1])
        for i in range(n):
            v = X0[i, lo:hi].astype(np.float64)
            want = np.abs(v).sum() / (hi - lo)
            got = float(msgs[l][i].scale)
            assert abs(got - want) <= 1e-6 * want, (l, i)
            assert np.array_equal(Xh[i, lo:hi], np.where(v < 0, -np.float32(got), np.float32(got)))
    # a single scale for the whole row would be dominated by layer 4
    whole = np.abs(X0[0].astype(np.float64)).mean()
    assert float(msgs[0][0].scale) < 0.05 * whole


def test_qsgd_blocks_restart_at_the_layer():
    n = 3
    w = workloads.ring(n)
    X, Xh, S = _state(n, 5, [1.0, 2.0, 0.1, 7.0, 30.0, 0.3])
    X0 = X.copy()
    bucket = 128
    msgs = oracle.step_layers(w, oracle.Params("qsgd", s=16, bucket=bucket, seed=9), OFF, 1, 1,
                              X, Xh, S, None, 0.0, 0.1, 0)
    for l in range(len(OFF) - 1):
        lo, hi = int(OFF[l]), int(OFF[l + 1])
        nb = (hi - lo + bucket - 1) // bucket
        for i in range(n):
            assert msgs[l][i].norms.shape[0] == nb
            for b in range(nb):
                seg = X0[i, lo + b * bucket: min(hi, lo + (b + 1) * bucket)].astype(np.float64)
                want = np.sqrt((seg * seg).sum())
                assert abs(float(msgs[l][i].norms[b]) - want) <= 2e-6 * want


def test_randk_layers_draw_their_own_subsets():
    n = 3
    w = workloads.ring(n)
    off = workloads.layer_offsets([300, 300, 300, 7])
    X = workloads.normal_rows(n, int(off[-1]), 1.0, 6)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    msgs = oracle.step_layers(w, oracle.Params("randk", seed=21), off, 1, 10, X, Xh, S, None, 0.0, 0.1, 4)
    for l in range(4):
        dl = int(off[l + 1] - off[l])
        k = max(1, dl // 10)
        for i in range(n):
            idx = msgs[l][i].idx
            assert idx.shape[0] == k and len(set(idx.tolist())) == k and idx.max() < dl
            words = oracle.random_words(21 + l, 4, i, oracle.STREAM_RANDK, dl).astype(np.int64)
            want = np.sort(np.lexsort((np.arange(dl), words))[:k])   # k smallest words, ties by index
            assert np.array_equal(idx, want.astype(np.uint32))
    assert not np.array_equal(msgs[0][0].idx, msgs[1][0].idx)        # same length, different layer


def test_layered_gossip_preserves_the_average():
    n = 6
    w = workloads.torus(2, 3)
    X, Xh, S = _state(n, 7)
    mean0 = X.astype(np.float64).mean(axis=0)
    for t in range(20):
        oracle.step_layers(w, oracle.Params("topk"), OFF, 1, 10, X, Xh, S, None, 0.0, 0.2, t)
    assert np.max(np.abs(X.astype(np.float64).mean(axis=0) - mean0)) < 1e-5
