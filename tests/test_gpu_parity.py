"""CUDA library vs CPU oracle, through the C interface, on the same seeded inputs.

Acceptance: selected indices, packed sign bits, level fields and random-k indices are
bit-exact; float32 state within 1e-5 * max|x| of the oracle after a step.  The library
follows a fixed operation order, so the tests additionally require the float32 state to be
identical (values compared with ==, which treats +0 and -0 alike).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_09356_b200 as choco
import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _dev(a, ld=None):
    """Host [n, d] -> device tensor with row pitch ld (a view of a larger buffer when ld > d)."""
    n, d = a.shape
    ld = ld or d
    if ld == d:
        return torch.from_numpy(a).to(DEV).contiguous()
    buf = torch.full((n, ld), float("nan"), dtype=torch.float32, device=DEV)
    buf[:, :d] = torch.from_numpy(a).to(DEV)
    return buf


def _host(t, d):
    return t[:, :d].cpu().numpy()


def assert_state(got, want, what):
    """spec tolerance, then the stricter equality the fixed operation order gives."""
    tol = 1e-5 * max(float(np.max(np.abs(want))), 1e-30)
    assert np.max(np.abs(got.astype(np.float64) - want.astype(np.float64))) <= tol, what
    assert np.array_equal(got, want), f"{what}: within tolerance but not identical"


def check_messages(ctx, kind, msgs, d):
    for i, m in msgs.items():
        p0 = choco.choco_read_message(ctx, i, 0)
        p1 = choco.choco_read_message(ctx, i, 1)
        p2 = choco.choco_read_message(ctx, i, 2)
        if kind in ("topk", "randk"):
            assert np.array_equal(p0.view(np.uint32), m.idx), f"indices of worker {i}"
            assert np.array_equal(p1.view(np.uint32), m.val.view(np.uint32)), f"values of worker {i}"
        elif kind == "sign":
            assert np.array_equal(p0.view(np.uint32), m.bits), f"sign bits of worker {i}"
            assert p1.view(np.float32)[0] == m.scale, f"scale of worker {i}"
        elif kind == "qsgd":
            assert np.array_equal(p0.view(np.uint32), m.bits), f"sign bits of worker {i}"
            assert np.array_equal(p1.view(np.float32), m.norms), f"norms of worker {i}"
            assert np.array_equal(p2, m.levels), f"levels of worker {i}"
        else:
            assert np.array_equal(p1.view(np.float32), m.q)


def run_lockstep(w, kind, n, d, steps, *, k=0, s=16, bucket=0, biased=True, seed=0, ld=None,
                 eta=0.1, gamma=0.2, x_var=1.0, g_var=0.01, sgd=True, momentum=False,
                 x_init=None, check_msgs=True, grad_fn=None, select_blocks=None, nesterov=False,
                 candidate_slot=None):
    ld = ld or d
    X = workloads.normal_rows(n, d, x_var, 1000 + seed) if x_init is None else x_init.copy()
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    M = np.zeros_like(X) if momentum else None
    p = oracle.Params(kind, k=k, s=s, bucket=bucket, biased=biased, seed=seed)
    ch = choco.Choco(w, d, kind, k=k, s=s, bucket=bucket, qsgd_biased=biased, seed=seed, ld=ld)
    if select_blocks:
        choco.choco_set_select_blocks(ch.ctx, select_blocks)
    if candidate_slot:
        choco.choco_debug_set_candidate_slot(ch.ctx, candidate_slot)
    if nesterov:
        choco.choco_set_nesterov(ch.ctx, True)
    dX, dXh, dS = _dev(X, ld), _dev(Xh, ld), _dev(S, ld)
    dM = _dev(M, ld) if momentum else None
    try:
        for t in range(steps):
            if grad_fn is not None:
                G = grad_fn(t, X)
            elif sgd:
                G = workloads.normal_rows(n, d, g_var, 5000 + 97 * seed + t)
            else:
                G = None
            dG = _dev(G, ld) if G is not None else None
            if momentum:
                msgs = oracle.step(w, p, X, Xh, S, G, eta, gamma, t, M=M, lam=1e-3, beta=0.9, nesterov=nesterov)
                ch.sgd_momentum_step(dX, dXh, dS, dG, dM, eta, gamma, 1e-3, 0.9)
            elif G is not None:
                msgs = oracle.step(w, p, X, Xh, S, G, eta, gamma, t)
                ch.sgd_step(dX, dXh, dS, dG, eta, gamma)
            else:
                msgs = oracle.step(w, p, X, Xh, S, None, 0.0, gamma, t)
                ch.gossip_step(dX, dXh, dS, gamma)
            torch.cuda.synchronize()
            if check_msgs:
                check_messages(ch.ctx, kind, msgs, d)
            assert_state(_host(dXh, d), Xh, f"Xhat after step {t}")
            assert_state(_host(dS, d), S, f"S after step {t}")
            assert_state(_host(dX, d), X, f"X after step {t}")
            if momentum:
                assert_state(_host(dM, d), M, f"M after step {t}")
        assert choco.choco_get_step(ch.ctx) == steps
        assert choco.choco_get_stats(ch.ctx)["device_timeouts"] == 0
        if ld != d:   # the pad between rows is never written
            assert bool(torch.isnan(dX[:, d:]).all()) and bool(torch.isnan(dS[:, d:]).all())
        return ch, (dX, dXh, dS), (X, Xh, S)
    except Exception:
        ch.close()
        raise


SHAPES = [(1, None), (31, None), (33, 36), (513, None), (2000, 2000), (4097, 4100), (10007, None)]


@pytest.mark.parametrize("d,ld", SHAPES)
def test_sign_shapes(d, ld):
    ch, _, _ = run_lockstep(workloads.ring(5), "sign", 5, d, 3, ld=ld, seed=d)
    assert choco.choco_message_bytes(ch.ctx)[0] == 4 * ((d + 31) // 32) + 4
    ch.close()


@pytest.mark.parametrize("d,ld", SHAPES)
@pytest.mark.parametrize("bucket", [0, 128, 512, 1024])
def test_qsgd_shapes(d, ld, bucket):
    run_lockstep(workloads.ring(4), "qsgd", 4, d, 3, s=16, bucket=bucket, ld=ld, seed=d + bucket)[0].close()


@pytest.mark.parametrize("s", [2, 4, 8, 32, 128, 256, 512, 32768])
@pytest.mark.parametrize("biased", [True, False])
def test_qsgd_level_counts(s, biased):
    run_lockstep(workloads.ring(4), "qsgd", 4, 3000, 2, s=s, bucket=256, biased=biased, seed=s)[0].close()


@pytest.mark.parametrize("d,ld,bucket", [(4096, None, 512), (5002, None, 128), (5001, None, 512), (3000, None, 0)],
                         ids=["aligned", "8-byte rows", "odd rows", "whole-row norm"])
def test_qsgd_sixteen_bit_levels(d, ld, bucket):
    """s = 2^15 (Table 1's 16-bit row): 16-bit level fields through every kernel that packs or
    reads them, several steps so that carried messages are decoded too, with momentum once."""
    w = workloads.ring(5)
    run_lockstep(w, "qsgd", 5, d, 4, s=32768, bucket=bucket, seed=d, ld=ld)[0].close()
    run_lockstep(w, "qsgd", 5, d, 3, s=32768, bucket=bucket, seed=d + 1, ld=ld, momentum=True)[0].close()


@pytest.mark.parametrize("d,ld", SHAPES)
def test_identity_shapes(d, ld):
    run_lockstep(workloads.torus(3, 3), "identity", 9, d, 2, ld=ld, seed=d, gamma=1.0)[0].close()


@pytest.mark.parametrize("d,k,ld", [(1, 1, None), (31, 5, None), (33, 33, 36), (513, 1, None),
                                    (2000, 20, None), (4097, 300, 4100), (10007, 100, None),
                                    (10007, 10007, None), (50000, 500, None),
                                    (100000, 10000, None), (100000, 50000, None)])   # Table 1's top-10 %, top-50 %
def test_topk_shapes(d, k, ld):
    ch, _, _ = run_lockstep(workloads.ring(5), "topk", 5, d, 3, k=k, ld=ld, seed=d + k)
    assert choco.choco_message_bytes(ch.ctx) == (8 * k, 8 * k * 5)
    ch.close()


@pytest.mark.parametrize("d,k,ld", [(1, 1, None), (33, 7, 36), (2000, 20, None), (4097, 300, None),
                                    (10007, 100, None), (10007, 10007, None), (50000, 5000, None),
                                    (100000, 50000, None)])                          # Table 1's random-50 %
def test_randk_shapes(d, k, ld):
    ch, _, _ = run_lockstep(workloads.ring(5), "randk", 5, d, 3, k=k, ld=ld, seed=d + k)
    assert choco.choco_message_bytes(ch.ctx) == (4 * k, 4 * k * 5)
    ch.close()


@pytest.mark.parametrize("blocks", [2, 4])
@pytest.mark.parametrize("kind,d,k,ld", [("topk", 1, 1, None), ("topk", 33, 33, 36), ("topk", 2000, 20, None),
                                         ("topk", 4097, 300, 4100), ("topk", 10007, 10007, None),
                                         ("topk", 50000, 500, None), ("topk", 300000, 3000, None),
                                         ("randk", 2000, 20, None), ("randk", 50000, 5000, None)])
def test_selection_by_a_cluster_of_blocks_per_row(kind, d, k, ld, blocks):
    """The selection kernel with 2 or 4 blocks per row (normally chosen for large rows only):
    one tile, ragged tiles, k = d, more tiles than threads in a block's pass, several steps so
    that carried candidates are selected from too."""
    ch, _, _ = run_lockstep(workloads.ring(5), kind, 5, d, 4, k=k, ld=ld, seed=d + k + blocks, select_blocks=blocks)
    ch.close()


@pytest.mark.parametrize("slot", [1, 8, 40])
@pytest.mark.parametrize("d,k", [(50000, 500), (300000, 3000), (4097, 300)])
def test_candidates_behind_the_tiles_slots(d, k, slot):
    """With several blocks per row the update kernel places a tile's candidates in the tile's own
    slot.  Slots made too small: most tiles reserve room behind the slots (slot 8, 40), or that
    room runs out and the row is selected from the dense row instead (slot 1).  Same messages and
    state as the oracle either way; with the default slot every step's rows are served from candidates."""
    ch, _, _ = run_lockstep(workloads.ring(5), "topk", 5, d, 6, k=k, seed=d + slot, select_blocks=2, candidate_slot=slot)
    ch.close()
    ch, _, _ = run_lockstep(workloads.ring(5), "topk", 5, d, 6, k=k, seed=d + slot, select_blocks=2)
    st = choco.choco_get_stats(ch.ctx)
    ch.close()
    assert st["prepared_rows"] >= 5 * 5 - 3, st   # (a bound guessed too high may cost a row its candidates)


def test_switching_the_selection_kernel_between_steps():
    """One block per row reads a row's candidates as one contiguous run, a cluster reads them tile
    by tile from the tiles' slots: switching between steps must not hand one kernel the other's
    arrangement (the switch drops the carried candidates)."""
    w = workloads.ring(5)
    n, d, k = 5, 40000, 400
    ch = choco.Choco(w, d, "topk", k=k, seed=3)
    X = workloads.normal_rows(n, d, 1.0, 90)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    p = oracle.Params("topk", k=k, seed=3)
    dX, dXh, dS = _dev(X), _dev(Xh), _dev(S)
    try:
        for t in range(12):
            if t % 3 == 0:
                choco.choco_set_select_blocks(ch.ctx, (2, 1, 4, 1)[t // 3])
            if t == 7:
                choco.choco_debug_set_candidate_slot(ch.ctx, 4)
            G = workloads.normal_rows(n, d, 0.01, 500 + t)
            msgs = oracle.step(w, p, X, Xh, S, G, 0.1, 0.2, t)
            ch.sgd_step(dX, dXh, dS, _dev(G), 0.1, 0.2)
            torch.cuda.synchronize()
            check_messages(ch.ctx, "topk", msgs, d)
            assert_state(_host(dX, d), X, f"X after step {t}")
            assert_state(_host(dS, d), S, f"S after step {t}")
        st = choco.choco_get_stats(ch.ctx)
        assert st["prepared_rows"] >= n * 6, st   # steps that did not follow a switch used carried candidates
    finally:
        ch.close()


@pytest.mark.parametrize("blocks", [2, 4])
def test_ties_with_a_cluster_of_blocks_per_row(blocks):
    """Ties at the k-th key that straddle the blocks' shares: rows of few distinct magnitudes."""
    n, d, k = 4, 60000, 700
    rng = np.random.default_rng(blocks)
    x = np.zeros((n, d), dtype=np.float32)
    x[0] = rng.choice([-2.0, 2.0, 1.0, -1.0], size=d).astype(np.float32)
    x[1] = rng.integers(-3, 4, size=d).astype(np.float32)
    x[2] = rng.standard_normal(d).astype(np.float32)
    x[2, 1000:1400] = x[2, 50]
    x[3] = np.round(rng.standard_normal(d) * 4).astype(np.float32) / 4
    ch, _, _ = run_lockstep(workloads.ring(n), "topk", n, d, 5, k=k, x_init=x, seed=2, select_blocks=blocks)
    ch.close()


@pytest.mark.parametrize("kind,kw", [("topk", dict(k=300)), ("randk", dict(k=300)), ("sign", {}),
                                     ("qsgd", dict(s=16, bucket=256))])
def test_arrays_at_different_offsets_in_a_16_byte_unit(kind, kw):
    """X, Xhat, S, G start 0, 4, 8 and 12 bytes into a 16-byte unit; rows of 4099 floats move
    the offset from row to row; the floats around every array stay untouched."""
    w = workloads.ring(6)
    n, d, steps = 6, 4099, 3
    p = oracle.Params(kind, seed=5, **kw)
    X = workloads.normal_rows(n, d, 1.0, 77)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    guard = 8

    def place(a, off):
        flat = torch.full((guard + off + n * d + guard,), float("nan"), dtype=torch.float32, device=DEV)
        view = flat[guard + off: guard + off + n * d].view(n, d)
        view.copy_(torch.from_numpy(a))
        assert view.data_ptr() % 16 == 4 * off
        return flat, view

    fX, dX = place(X, 0)
    fXh, dXh = place(Xh, 1)
    fS, dS = place(S, 2)
    ch = choco.Choco(w, d, kind, seed=5, **kw)
    try:
        for t in range(steps):
            G = workloads.normal_rows(n, d, 0.01, 900 + t)
            fG, dG = place(G, 3)
            msgs = oracle.step(w, p, X, Xh, S, G, 0.1, 0.2, t)
            ch.sgd_step(dX, dXh, dS, dG, 0.1, 0.2)
            torch.cuda.synchronize()
            check_messages(ch.ctx, kind, msgs, d)
            assert_state(dXh.cpu().numpy(), Xh, f"Xhat after step {t}")
            assert_state(dS.cpu().numpy(), S, f"S after step {t}")
            assert_state(dX.cpu().numpy(), X, f"X after step {t}")
            assert np.array_equal(dG.cpu().numpy(), G)
            for flat, off in ((fX, 0), (fXh, 1), (fS, 2), (fG, 3)):
                assert bool(torch.isnan(flat[:guard + off]).all()) and bool(torch.isnan(flat[guard + off + n * d:]).all())
        assert choco.choco_get_stats(ch.ctx)["device_timeouts"] == 0
    finally:
        ch.close()


def test_topk_ties_zeros_and_signed_zero():
    n, d, k = 4, 9000, 700
    rng = np.random.default_rng(0)
    x = np.zeros((n, d), dtype=np.float32)
    x[0] = rng.choice([-2.0, 2.0, 1.0, -1.0], size=d).astype(np.float32)      # massive ties
    x[1, ::3] = -0.0                                                         # all-zero row, some -0
    x[2] = rng.integers(-3, 4, size=d).astype(np.float32)                   # few distinct values
    x[3] = rng.standard_normal(d).astype(np.float32)
    x[3, 100:140] = x[3, 50]                                                 # a tie at some value
    ch, _, _ = run_lockstep(workloads.ring(n), "topk", n, d, 4, k=k, x_init=x, seed=1)
    st = choco.choco_get_stats(ch.ctx)
    assert st["exact_rows"] > 0          # the tie-heavy rows went through the exact selection
    ch.close()


def test_topk_carry_across_steps():
    """The update kernel prepares the next step's selection; results do not depend on it."""
    w = workloads.torus(4, 4)
    n, d, k, steps = 16, 40000, 400, 12
    ch, (dX, dXh, dS), _ = run_lockstep(w, "topk", n, d, steps, k=k, seed=11, gamma=0.1, check_msgs=False)
    st = choco.choco_get_stats(ch.ctx)
    assert st["prepared_rows"] >= n * (steps - 3)          # all but the first step (and rare misses)
    assert st["prepared_rows"] + st["recompressed_rows"] + st["exact_rows"] >= n * steps
    ch.close()
    # the same run with carrying switched off
    X = workloads.normal_rows(n, d, 1.0, 1000 + 11)
    ch2 = choco.Choco(w, d, "topk", k=k, seed=11)
    choco.choco_set_carry(ch2.ctx, False)
    eX, eXh, eS = _dev(X), torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV)
    for t in range(steps):
        G = _dev(workloads.normal_rows(n, d, 0.01, 5000 + 97 * 11 + t))
        ch2.sgd_step(eX, eXh, eS, G, 0.1, 0.1)
    torch.cuda.synchronize()
    assert choco.choco_get_stats(ch2.ctx)["prepared_rows"] == 0
    assert torch.equal(eX, dX) and torch.equal(eXh, dXh) and torch.equal(eS, dS)
    ch2.close()


def test_topk_values_in_one_histogram_bin_recover_after_exact_selection():
    """All |x - x^| within 5 % of each other: the first histogram cannot separate them, the rows
    are selected exactly, and the bound set there must make the next steps' candidates usable."""
    n, d, k, steps = 4, 200_000, 2000, 6
    rng = np.random.default_rng(12)
    x0 = ((1.0 + 0.05 * rng.random((n, d))) * rng.choice([-1.0, 1.0], size=(n, d))).astype(np.float32)
    ch, _, _ = run_lockstep(workloads.ring(n), "topk", n, d, steps, k=k, seed=3, gamma=0.01, eta=0.01,
                            g_var=1e-8, x_init=x0)
    st = choco.choco_get_stats(ch.ctx)
    ch.close()
    assert st["exact_rows"] <= 2 * n, st
    assert st["prepared_rows"] >= n * (steps - 2), st


@pytest.mark.parametrize("kind,kw", [("sign", {}), ("qsgd", dict(s=16, bucket=512)), ("identity", {})])
def test_dense_carry_across_steps(kind, kw):
    """For dense operators the update kernel writes the next step's messages; switching that
    off (every step compresses from X and Xhat again) must give the same state."""
    w = workloads.ring(6)
    n, d, steps = 6, 30000, 6
    X0 = workloads.normal_rows(n, d, 1.0, 31)
    G = [_dev(workloads.normal_rows(n, d, 0.01, 700 + t)) for t in range(steps)]
    out = []
    for carry in (True, False):
        ch = choco.Choco(w, d, kind, seed=4, **kw)
        choco.choco_set_carry(ch.ctx, carry)
        st = [_dev(X0), torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV)]
        for t in range(steps):
            ch.sgd_step(st[0], st[1], st[2], G[t], 0.05, 0.2)
            if t == 2:      # an external change of X in the middle, announced to the library
                st[0].mul_(1.5)
                choco.choco_invalidate(ch.ctx)
        torch.cuda.synchronize()
        launches = choco.choco_get_stats(ch.ctx)["kernel_launches"]
        out.append((st, launches))
        ch.close()
    for a, b in zip(out[0][0], out[1][0]):
        assert torch.equal(a, b)
    assert out[0][1] < out[1][1]     # carrying saves the separate compression kernels


def test_invalidate_after_external_change():
    w = workloads.ring(4)
    n, d, k = 4, 20000, 200
    X = workloads.normal_rows(n, d, 1.0, 5)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    G = workloads.normal_rows(n, d, 0.01, 6)
    p = oracle.Params("topk", k=k)
    ch = choco.Choco(w, d, "topk", k=k)
    dX, dXh, dS, dG = _dev(X), _dev(Xh), _dev(S), _dev(G)
    oracle.step(w, p, X, Xh, S, G, 0.1, 0.2, 0)
    ch.sgd_step(dX, dXh, dS, dG, 0.1, 0.2)
    # the caller overwrites X in place (say, loads a checkpoint) and tells the library
    X[:] = workloads.normal_rows(n, d, 4.0, 7)
    dX.copy_(torch.from_numpy(X))
    choco.choco_invalidate(ch.ctx)
    oracle.step(w, p, X, Xh, S, G, 0.1, 0.2, 1)
    ch.sgd_step(dX, dXh, dS, dG, 0.1, 0.2)
    torch.cuda.synchronize()
    assert_state(_host(dX, d), X, "X after invalidate")
    assert_state(_host(dXh, d), Xh, "Xhat after invalidate")
    # a change of buffers is noticed without being told
    dX2 = dX.clone()
    oracle.step(w, p, X, Xh, S, G, 0.1, 0.2, 2)
    ch.sgd_step(dX2, dXh, dS, dG, 0.1, 0.2)
    torch.cuda.synchronize()
    assert_state(_host(dX2, d), X, "X after pointer change")
    ch.close()


def test_irregular_graph_sparse_and_dense():
    w = workloads.random_graph(32, 14, 1)
    run_lockstep(w, "topk", 32, 6000, 3, k=60, seed=2)[0].close()
    run_lockstep(w, "sign", 32, 6000, 2, seed=3)[0].close()


@pytest.mark.parametrize("graph", ["torus", "irregular"])
def test_many_neighbours_send_the_same_coordinate(graph):
    """Workers that start from nearly the same x select the same coordinates, so a coordinate of
    s_i receives a term from every neighbour: the sum must still go in CSR order from +0 (the
    update kernel adds one or two terms as they come and redoes coordinates with more in order)."""
    w = workloads.torus(4, 4) if graph == "torus" else workloads.random_graph(32, 14, 1)
    n, d, k = w.n, 8192, 160 if graph == "torus" else 64
    base = workloads.normal_rows(1, d, 1.0, 77)
    x = np.repeat(base, n, axis=0) + workloads.normal_rows(n, d, 1e-6, 78)
    ch, _, _ = run_lockstep(w, "topk", n, d, 5, k=k, x_init=x.astype(np.float32), seed=9, gamma=0.3)
    ch.close()
    # the same through the general path (more entries per tile than the threads hold at once)
    ch, _, _ = run_lockstep(w, "topk", n, d, 3, k=2000, x_init=x.astype(np.float32), seed=10, gamma=0.3)
    ch.close()


def test_momentum_variant():
    run_lockstep(workloads.ring(4), "topk", 4, 5000, 4, k=50, momentum=True, seed=4)[0].close()
    run_lockstep(workloads.ring(4), "sign", 4, 5000, 3, momentum=True, seed=5)[0].close()


@pytest.mark.parametrize("d,ld", [(5000, None), (5002, None), (5001, None)], ids=["aligned", "8-byte rows", "odd rows"])
def test_nesterov_variant(d, ld):
    # the look-ahead step of every update kernel (rows 16-byte aligned, 8-byte aligned, at odd elements)
    w = workloads.ring(4)
    run_lockstep(w, "topk", 4, d, 4, k=50, momentum=True, nesterov=True, seed=4, ld=ld)[0].close()
    run_lockstep(w, "sign", 4, d, 3, momentum=True, nesterov=True, seed=5, ld=ld)[0].close()
    run_lockstep(w, "qsgd", 4, d, 3, bucket=512, momentum=True, nesterov=True, seed=6, ld=ld)[0].close()
    run_lockstep(w, "qsgd", 4, d, 2, momentum=True, nesterov=True, seed=7, ld=ld)[0].close()
    run_lockstep(w, "identity", 4, d, 2, momentum=True, nesterov=True, seed=8, ld=ld)[0].close()


def test_nesterov_switch_changes_the_step_and_back():
    # the setter takes effect on the next call, also where steps are replayed from a graph
    w = workloads.ring(4)
    n, d = 4, 1024
    ch = choco.Choco(w, d, "topk", k=10, seed=2)
    X = workloads.normal_rows(n, d, 1.0, 70)
    Xh, S, M = np.zeros_like(X), np.zeros_like(X), np.zeros_like(X)
    G = workloads.normal_rows(n, d, 0.01, 71)
    p = oracle.Params("topk", k=10, seed=2)
    dX, dXh, dS, dM, dG = _dev(X), _dev(Xh), _dev(S), _dev(M), _dev(G)
    st = torch.cuda.Stream()
    try:
        with torch.cuda.stream(st):
            for t in range(12):
                nes = 4 <= t < 8
                choco.choco_set_nesterov(ch.ctx, nes)
                oracle.step(w, p, X, Xh, S, G, 0.1, 0.2, t, M=M, lam=1e-3, beta=0.9, nesterov=nes)
                ch.sgd_momentum_step(dX, dXh, dS, dG, dM, 0.1, 0.2, 1e-3, 0.9)
                torch.cuda.synchronize()
                assert_state(_host(dX, d), X, f"X after step {t}")
                assert_state(_host(dM, d), M, f"M after step {t}")
    finally:
        ch.close()


def test_config1_full_run_and_consensus():
    wl = workloads.WORKLOADS["c1_ring4_topk"]
    X0 = workloads.normal_rows(wl.n, wl.d, 1.0, 0)
    e0 = oracle.consensus_error(X0)
    ch, (dX, _, _), (X, _, _) = run_lockstep(wl.mixing(), "topk", wl.n, wl.d, wl.steps, k=wl.k,
                                             gamma=wl.gamma, sgd=False, x_init=X0, check_msgs=False)
    got = choco.choco_consensus_error(ch.ctx, dX) / e0
    want = oracle.consensus_error(X) / e0
    assert abs(got - want) <= 1e-4 * want
    assert want < 0.1
    ch.close()


@pytest.mark.parametrize("name", ["c2_ring16_randk", "c2_ring16_qsgd"])
def test_config2_logistic_regression(name):
    wl = workloads.WORKLOADS[name]
    prob = workloads.LogisticProblem(wl.n, wl.d, 256, seed=3)
    x0 = np.zeros((wl.n, wl.d), dtype=np.float32)
    ch, _, (X, _, _) = run_lockstep(wl.mixing(), wl.q, wl.n, wl.d, 120, k=wl.k, s=wl.s,
                                    bucket=wl.bucket, eta=wl.eta, gamma=wl.gamma, x_init=x0, seed=9,
                                    grad_fn=lambda t, x: prob.gradient(x, t), check_msgs=False)
    assert prob.loss(X.mean(axis=0)) < prob.loss(np.zeros(wl.d, np.float32))
    ch.close()


def test_config3_shape_sign():
    wl = workloads.WORKLOADS["c3_ring8_sign"]
    ch, _, _ = run_lockstep(wl.mixing(), "sign", wl.n, wl.d, 4, eta=wl.eta, gamma=wl.gamma,
                            x_var=wl.x_var, g_var=wl.g_var, seed=3)
    assert choco.choco_message_bytes(ch.ctx)[0] == 34064
    ch.close()


def test_resume_from_checkpoint_is_bit_exact():
    w = workloads.ring(6)
    n, d = 6, 7000
    X0 = workloads.normal_rows(n, d, 1.0, 77)
    G = [_dev(workloads.normal_rows(n, d, 0.01, 900 + t)) for t in range(6)]

    def run(ch, state, t0, t1):
        for t in range(t0, t1):
            ch.sgd_step(state[0], state[1], state[2], G[t], 0.05, 0.1)

    a = choco.Choco(w, d, "qsgd", s=16, bucket=512, seed=5)
    sa = [_dev(X0), torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV)]
    run(a, sa, 0, 6)
    b = choco.Choco(w, d, "qsgd", s=16, bucket=512, seed=5)
    sb = [_dev(X0), torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV)]
    run(b, sb, 0, 3)
    saved = [t.clone() for t in sb]
    b.close()
    c = choco.Choco(w, d, "qsgd", s=16, bucket=512, seed=5)
    choco.choco_set_step(c.ctx, 3)
    run(c, saved, 3, 6)
    torch.cuda.synchronize()
    for x, y in zip(sa, saved):
        assert torch.equal(x, y)
    a.close(); c.close()


def test_host_buffer_entry_point():
    w = workloads.ring(4)
    n, d = 4, 5000
    X = workloads.normal_rows(n, d, 1.0, 1)
    G = workloads.normal_rows(n, d, 0.01, 2)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    oX, oXh, oS = X.copy(), Xh.copy(), S.copy()
    ch = choco.Choco(w, d, "topk", k=50)
    p = oracle.Params("topk", k=50)
    for t in range(2):
        oracle.step(w, p, oX, oXh, oS, G, 0.1, 0.2, t)
        choco.choco_sgd_step_host(ch.ctx, X, Xh, S, G, 0.1, 0.2)
        assert_state(X, oX, "X (host call)")
        assert_state(Xh, oXh, "Xhat (host call)")
        assert_state(S, oS, "S (host call)")
    ch.close()


@pytest.mark.parametrize("kind,kw,n", [("topk", dict(k=300), 19), ("sign", {}, 19), ("qsgd", dict(s=16, bucket=512), 8),
                                       ("qsgd", dict(s=16, bucket=0), 3), ("randk", dict(k=300), 19),
                                       ("identity", {}, 5)])
def test_host_buffer_entry_point_in_chunks_of_rows(kind, kw, n):
    """The host entry point uploads, updates and downloads the rows in eight chunks on three
    streams: more rows than chunks (ragged last chunk), as many, fewer; pinned host arrays; every
    operator's update kernel takes a row range."""
    w = workloads.ring(n)
    d = 30000
    host = [torch.from_numpy(a).pin_memory() for a in
            (workloads.normal_rows(n, d, 1.0, 1), np.zeros((n, d), np.float32), np.zeros((n, d), np.float32))]
    X, Xh, S = (t.numpy() for t in host)
    oX, oXh, oS = X.copy(), Xh.copy(), S.copy()
    ch = choco.Choco(w, d, kind, seed=4, **kw)
    p = oracle.Params(kind, seed=4, **kw)
    st = torch.cuda.Stream()
    try:
        with torch.cuda.stream(st):
            for t in range(3):
                G = workloads.normal_rows(n, d, 0.01, 20 + t)
                oracle.step(w, p, oX, oXh, oS, G, 0.1, 0.2, t)
                choco.choco_sgd_step_host(ch.ctx, X, Xh, S, G, 0.1, 0.2)
                assert_state(X, oX, f"X (host call {t})")
                assert_state(Xh, oXh, f"Xhat (host call {t})")
                assert_state(S, oS, f"S (host call {t})")
    finally:
        ch.close()
