"""Pins for the oracle's gossip / SGD step and for the graph constructors.

What the paper fixes and these tests use: Table 2's spectral gaps; average
preservation (Assumption 4); exact averaging as the Q = identity special case
(Appendix A.1); the equivalence of Algorithm 1, its three-vector form and the
error-feedback rewrite (Algorithm 4); linear decay of the Lyapunov function at the
stepsize of Theorem 4.1.
"""
import os

import numpy as np
import pytest

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _fresh(n, d, seed, var=1.0):
    X = workloads.normal_rows(n, d, var, seed)
    return X, np.zeros_like(X), np.zeros_like(X)


# ---------------------------------------------------------------- graphs


def test_table2_spectral_gaps():
    with open(os.path.join(GOLDEN, "table2_spectral_gaps.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 8
    for topo, n, printed, tol in rows:
        n = int(n)
        side = int(round(np.sqrt(n)))
        w = workloads.ring(n) if topo == "ring" else workloads.torus(side, side)
        assert abs(workloads.spectral_gap(w) - float(printed)) <= float(tol), (topo, n)


@pytest.mark.parametrize("w", [workloads.ring(4), workloads.ring(16), workloads.torus(8, 8),
                               workloads.torus(2, 2), workloads.random_graph(32, 14, 1)])
def test_mixing_matrix_assumption(w):
    W = w.dense()
    assert np.allclose(W, W.T, atol=1e-7)
    assert np.allclose(W.sum(axis=0), 1.0, atol=1e-6) and np.allclose(W.sum(axis=1), 1.0, atol=1e-6)
    assert (W >= 0).all() and (np.diag(W) > 0).all()
    assert workloads.spectral_gap(w) > 0
    for i in range(w.n):
        cols = w.col[w.row_ptr[i]:w.row_ptr[i + 1]]
        assert np.all(np.diff(cols) > 0) and i in cols


def test_ring_and_torus_weights():
    assert np.allclose(workloads.ring(8).val, 1 / 3)
    assert np.allclose(workloads.torus(8, 8).val, 1 / 5)
    # the 2x2 torus is a 4-cycle (nodes relabelled): same spectrum as the 4-ring
    assert np.allclose(np.linalg.eigvalsh(workloads.torus(2, 2).dense()),
                       np.linalg.eigvalsh(workloads.ring(4).dense()))
    g = workloads.random_graph(32, 14, 1)
    deg = np.diff(g.row_ptr) - 1
    assert deg.max() <= 14 and deg.max() >= 7 and deg.min() >= 2


# ---------------------------------------------------------------- the step


def test_identity_q_is_exact_gossip():
    w = workloads.torus(3, 3)
    W = w.dense()
    X, Xh, S = _fresh(9, 50, 1)
    X0 = X.astype(np.float64)
    p = oracle.Params("identity")
    oracle.step(w, p, X, Xh, S, None, 0.0, 0.37, 0)
    # x <- x + gamma (W - I) x   (Appendix A.1, CHOCO-Gossip with Q = identity)
    assert np.allclose(X, X0 + 0.37 * (W - np.eye(9)) @ X0, rtol=0, atol=2e-6)
    assert np.array_equal(Xh, X0.astype(np.float32))
    # gamma = 1: X^+ = W X, the exact-averaging example
    X, Xh, S = _fresh(9, 50, 2)
    X0 = X.astype(np.float64)
    oracle.step(w, p, X, Xh, S, None, 0.0, 1.0, 0)
    assert np.allclose(X, W @ X0, rtol=0, atol=2e-6)


@pytest.mark.parametrize("kind", ["topk", "randk", "qsgd", "sign", "identity"])
def test_mean_preserved_and_s_invariant(kind):
    w = workloads.ring(6)
    W = w.dense()
    n, d = 6, 300
    X, Xh, S = _fresh(n, d, 3)
    p = oracle.Params(kind, k=17, s=16, bucket=128, seed=21)
    mean0 = X.astype(np.float64).mean(axis=0)
    for t in range(25):
        oracle.step(w, p, X, Xh, S, None, 0.0, 0.2, t)
        # gossip keeps the average of the iterates (Assumption 4, first property)
        assert np.max(np.abs(X.astype(np.float64).mean(axis=0) - mean0)) < 5e-6
        # s_i = sum_j w_ij x^_j, the quantity the three-vector form carries
        assert np.allclose(S, W @ Xh.astype(np.float64), rtol=0, atol=2e-5)


def test_sgd_term_and_order():
    w = workloads.ring(4)
    X, Xh, S = _fresh(4, 40, 4)
    G = workloads.normal_rows(4, 40, 1.0, 5)
    X0 = X.copy()
    msgs = oracle.step(w, oracle.Params("topk", k=5), X, Xh, S, G, 0.25, 0.1, 0)
    f = np.float32
    for i in range(4):
        q = msgs[i].q
        assert np.array_equal(Xh[i], q)                      # x^ was 0
        acc = np.zeros(40, f)
        for e in range(w.row_ptr[i], w.row_ptr[i + 1]):
            acc = acc + w.val[e] * msgs[int(w.col[e])].q
        assert np.array_equal(S[i], acc)
        want = (X0[i] - f(0.25) * G[i]) + f(0.1) * (S[i] - Xh[i])
        assert np.array_equal(X[i], want)


def test_rows_subset_matches_full_step():
    w = workloads.ring(8)
    X, Xh, S = _fresh(8, 64, 6)
    G = workloads.normal_rows(8, 64, 0.1, 7)
    p = oracle.Params("sign")
    A = [a.copy() for a in (X, Xh, S)]
    oracle.step(w, p, X, Xh, S, G, 0.1, 0.3, 0)
    oracle.step(w, p, A[0], A[1], A[2], G, 0.1, 0.3, 0, rows=[2, 7])
    for full, part in zip((X, Xh, S), A):
        assert np.array_equal(full[[2, 7]], part[[2, 7]])


@pytest.mark.parametrize("kind", ["topk", "sign", "qsgd", "randk"])
def test_three_forms_agree(kind):
    """Algorithm 1 as printed == three-vector form == Algorithm 4, up to rounding."""
    w = workloads.ring(5)
    n, d, T = 5, 48, 12
    x0 = workloads.normal_rows(n, d, 1.0, 8)
    gpool = [workloads.normal_rows(n, d, 0.05, 100 + t) for t in range(T)]
    p = oracle.Params(kind, k=6, s=16, bucket=0, seed=3)
    eta, gamma = 0.05, 0.15
    lit = oracle.alg1_literal(w, p, x0, lambda t, x: gpool[t], eta, gamma, T, final_gossip=True)
    ef = oracle.alg4_error_feedback(w, p, x0, lambda t, x: gpool[t], eta, gamma, T,
                                    final_gossip=True)
    X, Xh, S = x0.copy(), np.zeros_like(x0), np.zeros_like(x0)
    for t in range(T):
        oracle.step(w, p, X, Xh, S, gpool[t], eta, gamma, t)
    assert np.allclose(lit, X, rtol=0, atol=2e-5)
    assert np.allclose(ef, X, rtol=0, atol=2e-5)


def test_consensus_error_definition():
    X = workloads.normal_rows(7, 33, 2.0, 9)
    X64 = X.astype(np.float64)
    want = np.sum((X64 - X64.mean(axis=0, keepdims=True)) ** 2)
    assert oracle.consensus_error(X) == pytest.approx(want, rel=1e-12)


def test_config1_consensus_decays():
    """4-ring, d = 1024, top-k k = 10, gamma = 0.05, 200 gossip steps."""
    wl = workloads.WORKLOADS["c1_ring4_topk"]
    w = wl.mixing()
    X, Xh, S = _fresh(wl.n, wl.d, 0)
    mean0 = X.astype(np.float64).mean(axis=0)
    e0 = oracle.consensus_error(X)
    p = oracle.Params("topk", k=wl.k)
    errs = []
    for t in range(wl.steps):
        oracle.step(w, p, X, Xh, S, None, 0.0, wl.gamma, t)
        errs.append(oracle.consensus_error(X) / e0)
    assert errs[49] < 0.5 and errs[99] < 0.25 and errs[199] < 0.1
    assert errs[199] < errs[99] < errs[49] < errs[9] < 1.0
    assert np.max(np.abs(X.astype(np.float64).mean(axis=0) - mean0)) < 2e-5


def test_lyapunov_contracts_at_theoretical_gamma():
    """Psi = ||X - Xbar||^2 + ||X - X^||^2 shrinks by (1 - rho^2 delta / 82) per step in
    expectation at the stepsize of Theorem 4.1 (top_a is deterministic: every step)."""
    w = workloads.ring(4)
    n, d, k = 4, 256, 16
    rho, beta, delta = workloads.spectral_gap(w), workloads.beta_norm(w), k / d
    gamma = oracle.theoretical_gamma(rho, delta, beta)
    assert 0 < gamma < 0.01
    c = rho * rho * delta / 82

    def psi(X, Xh):
        X64, H64 = X.astype(np.float64), Xh.astype(np.float64)
        return np.sum((X64 - X64.mean(axis=0)) ** 2) + np.sum((X64 - H64) ** 2)

    X, Xh, S = _fresh(n, d, 10)
    p = oracle.Params("topk", k=k)
    # The paper's h gossips with Y, then compresses: (X+, Y+) = (X + gamma Y (W - I),
    # Y + Q(X+ - Y)).  One call here compresses first and gossips last, so the paper's pair
    # (X+, Y+) is (X on entry to a call, X^ on exit from it).
    psi0 = psi(X, Xh)
    prev = psi0
    T = 400
    for t in range(T):
        X_in = X.copy()
        oracle.step(w, p, X, Xh, S, None, 0.0, gamma, t)
        cur = psi(X_in, Xh)
        assert cur <= prev * (1 - c) * (1 + 1e-6)
        prev = cur
    assert prev <= psi0 * (1 - c) ** T


def test_momentum_variant_matches_algorithm2():
    w = workloads.ring(4)
    n, d = 4, 32
    X, Xh, S = _fresh(n, d, 11)
    M = workloads.normal_rows(n, d, 0.5, 12)
    G = workloads.normal_rows(n, d, 1.0, 13)
    X0, M0 = X.copy(), M.copy()
    eta, gamma, lam, beta = 0.1, 0.2, 1e-2, 0.9
    oracle.step(w, oracle.Params("identity"), X, Xh, S, G, eta, gamma, 0, M=M, lam=lam, beta=beta)
    f = np.float32
    v1 = (G + f(lam) * X0) + f(beta) * M0                     # Algorithm 2, momentum update
    assert np.array_equal(M, v1)
    W = w.dense()
    want = (X0.astype(np.float64) - eta * v1) + gamma * ((W - np.eye(n)) @ X0.astype(np.float64))
    assert np.allclose(X, want, rtol=0, atol=3e-6)


def test_nesterov_variant_by_hand_and_special_cases():
    # one worker (W = [1]): the gossip term vanishes and the recursion is a scalar one
    w = workloads.MixingCSR(1, np.array([0, 1], np.int32), np.array([0], np.int32), np.array([1.0], np.float32))
    X = np.zeros((1, 1), np.float32)
    Xh, S, M = X.copy(), X.copy(), X.copy()
    G = np.ones((1, 1), np.float32)
    p = oracle.Params("identity")
    got = []
    for t in range(3):
        oracle.step(w, p, X, Xh, S, G, 0.125, 0.5, t, M=M, lam=0.0, beta=0.5, nesterov=True)
        got.append((float(M[0, 0]), float(X[0, 0])))
    # v: 1, 1.5, 1.75; x: -(1 + .5)/8, that -(1 + .75)/8, that -(1 + .875)/8   (all exact in binary)
    assert got == [(1.0, -0.1875), (1.5, -0.40625), (1.75, -0.640625)]

    w = workloads.ring(4)
    n, d = 4, 32
    Xa, Xh, S = _fresh(n, d, 21)
    M0 = workloads.normal_rows(n, d, 0.5, 22)
    G = workloads.normal_rows(n, d, 1.0, 23)
    X0 = Xa.copy()
    eta, gamma, lam = 0.1, 0.2, 1e-2
    # beta = 0: both variants are plain SGD with weight decay
    runs = []
    for nes in (False, True):
        X, H, Sx, M = X0.copy(), Xh.copy(), S.copy(), M0.copy()
        oracle.step(w, p, X, H, Sx, G, eta, gamma, 0, M=M, lam=lam, beta=0.0, nesterov=nes)
        runs.append((X, M))
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])
    # beta > 0: same memory as Algorithm 2, iterate moved by a further -eta beta v'
    beta = 0.9
    X, H, Sx, M = X0.copy(), Xh.copy(), S.copy(), M0.copy()
    oracle.step(w, p, X, H, Sx, G, eta, gamma, 0, M=M, lam=lam, beta=beta)
    Xn, Hn, Sn, Mn = X0.copy(), Xh.copy(), S.copy(), M0.copy()
    oracle.step(w, p, Xn, Hn, Sn, G, eta, gamma, 0, M=Mn, lam=lam, beta=beta, nesterov=True)
    assert np.array_equal(M, Mn)
    gl = G.astype(np.float64) + lam * X0
    want = X.astype(np.float64) + eta * M - eta * (gl + beta * M)
    assert np.allclose(Xn, want, rtol=0, atol=3e-6)
    assert not np.allclose(Xn, X, rtol=0, atol=1e-3)
