"""Seeded synthetic inputs for CHOCO-Gossip / CHOCO-SGD runs.

This module only *builds inputs*: communication graphs with their mixing
matrices in CSR form, initial iterates, gradient pools and the convex
logistic-regression problem.  It holds none of the method's arithmetic (no
compression operator, no gossip update), so that the CPU oracle and the CUDA
library can both be fed from it without sharing any of the code under test.

Mixing weights follow the rule the paper's experiments use (Section 3, below
Assumption 1): w_ij = 1 / max(deg(i), deg(j)) on edges, with the self-loop
counted in the degree, and the diagonal filled so that rows sum to one.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np

# --------------------------------------------------------------------------
# graphs -> mixing matrix W in CSR (diagonal stored, columns ascending)
# --------------------------------------------------------------------------


@dataclasses.dataclass(frozen=True)
class MixingCSR:
    """W as CSR over n rows: int32 row_ptr[n+1], int32 col[nnz], float32 val[nnz]."""

    n: int
    row_ptr: np.ndarray
    col: np.ndarray
    val: np.ndarray

    def dense(self, dtype=np.float64) -> np.ndarray:
        w = np.zeros((self.n, self.n), dtype=dtype)
        for i in range(self.n):
            for e in range(self.row_ptr[i], self.row_ptr[i + 1]):
                w[i, self.col[e]] = self.val[e]
        return w


def _csr_from_neighbours(neigh: list[set[int]]) -> MixingCSR:
    """Edge sets (without self) -> max-degree weights, self-loop counted in deg."""
    n = len(neigh)
    deg = [len(s) + 1 for s in neigh]          # +1: the self-loop {i} is an edge
    row_ptr = np.zeros(n + 1, dtype=np.int32)
    cols: list[int] = []
    vals: list[float] = []
    for i in range(n):
        off = {j: 1.0 / max(deg[i], deg[j]) for j in neigh[i]}
        diag = 1.0 - sum(off.values())
        row = dict(off)
        row[i] = diag
        for j in sorted(row):
            cols.append(j)
            vals.append(row[j])
        row_ptr[i + 1] = len(cols)
    return MixingCSR(n, row_ptr, np.asarray(cols, dtype=np.int32),
                     np.asarray(vals, dtype=np.float32))


def ring(n: int) -> MixingCSR:
    """Ring of n nodes; for n >= 3 every weight is 1/3 (self and both neighbours)."""
    neigh = [set() for _ in range(n)]
    for i in range(n):
        for j in ((i - 1) % n, (i + 1) % n):
            if j != i:
                neigh[i].add(j)
    return _csr_from_neighbours(neigh)


def torus(rows: int, cols: int) -> MixingCSR:
    """2-D torus; duplicate neighbours (side length 2) are merged, so the 2x2
    torus is the 4-ring.  For sides >= 3 every weight is 1/5."""
    n = rows * cols
    neigh = [set() for _ in range(n)]
    for r in range(rows):
        for c in range(cols):
            i = r * cols + c
            for rr, cc in ((r - 1, c), (r + 1, c), (r, c - 1), (r, c + 1)):
                j = (rr % rows) * cols + (cc % cols)
                if j != i:
                    neigh[i].add(j)
    return _csr_from_neighbours(neigh)


def random_graph(n: int, max_degree: int, seed: int) -> MixingCSR:
    """Connected irregular graph: a ring plus seeded random chords, node degrees
    (without self) capped at max_degree.  A stand-in with the degree profile of
    the paper's 32-node social-network topology (max degree 14); not that graph."""
    rng = np.random.default_rng(seed)
    neigh = [set() for _ in range(n)]
    for i in range(n):
        neigh[i].add((i + 1) % n)
        neigh[(i + 1) % n].add(i)
    hubs = rng.permutation(n)[: max(1, n // 6)]
    for h in hubs:
        want = int(rng.integers(max_degree // 2, max_degree + 1))
        for j in rng.permutation(n):
            if len(neigh[h]) >= want:
                break
            if j != h and j not in neigh[h] and len(neigh[j]) < max_degree:
                neigh[h].add(int(j))
                neigh[int(j)].add(int(h))
    return _csr_from_neighbours(neigh)


def spectral_gap(w: MixingCSR) -> float:
    """1 - |lambda_2(W)| by a dense symmetric eigen-solve (Assumption 1)."""
    ev = np.sort(np.abs(np.linalg.eigvalsh(w.dense())))[::-1]
    return float(1.0 - ev[1])


def beta_norm(w: MixingCSR) -> float:
    """beta = ||I - W||_2 (Theorem 4.1)."""
    return float(np.max(np.abs(np.linalg.eigvalsh(np.eye(w.n) - w.dense()))))


# --------------------------------------------------------------------------
# dense inputs
# --------------------------------------------------------------------------


def normal_rows(n: int, d: int, variance: float, seed: int,
                mean: Optional[np.ndarray] = None) -> np.ndarray:
    """float32 [n, d] ~ N(mean_i, variance); one PCG64 stream per (seed, row)."""
    out = np.empty((n, d), dtype=np.float32)
    sd = math.sqrt(variance)
    for i in range(n):
        rng = np.random.default_rng([seed, i])
        out[i] = rng.standard_normal(d, dtype=np.float32) * np.float32(sd)
        if mean is not None:
            out[i] += np.float32(mean[i])
    return out


def k_of(a_num: int, a_den: int, d: int) -> int:
    """floor(a * d) with a = a_num / a_den, in integer arithmetic."""
    return (d * a_num) // a_den


FINGERPRINT_MODULUS = 65521


def fingerprint(a: np.ndarray) -> tuple[int, int]:
    """Two 64-bit check sums of a float32 array's bit patterns, taken in row-major order:
    the sum of the 32-bit words, and the sum of word_i * (i mod 65521 + 1), both modulo 2^64.
    Equal arrays give equal pairs; a changed, moved or swapped word changes them.  (A way to
    compare a large state with a stored run without storing the state.)"""
    words = np.ascontiguousarray(a, dtype=np.float32).reshape(-1).view(np.uint32).astype(np.uint64)
    weight = (np.arange(words.size, dtype=np.uint64) % np.uint64(FINGERPRINT_MODULUS)) + np.uint64(1)
    with np.errstate(over="ignore"):
        return int(words.sum(dtype=np.uint64)), int((words * weight).sum(dtype=np.uint64))


def gradient_pool(wl: "Workload", count: int, seed: int) -> list[np.ndarray]:
    """`count` pre-generated gradient tensors [n, d] that a run cycles through (step t uses
    tensor t mod count): g ~ N(mu_i, g_var) per coordinate, where mu_i is a per-worker offset
    vector ~ N(0, g_mean_var) shared by all tensors of the pool (workers with different
    objectives), or zero if the workload has no g_mean_var."""
    mu = normal_rows(wl.n, wl.d, wl.g_mean_var, seed + 1_000_003) if wl.g_mean_var > 0 else None
    pool = []
    for p in range(count):
        g = normal_rows(wl.n, wl.d, wl.g_var, seed + p)
        if mu is not None:
            g += mu
        pool.append(g)
    return pool


def resnet20_layer_sizes() -> list[int]:
    """Lengths of the 65 parameter tensors of a CIFAR ResNet-20 in forward order (3x3
    convolutions without bias, each followed by a batch-norm scale and shift; 1x1 projection
    shortcuts where the width changes; a 64 -> 10 classifier).  They add up to 272 474, the
    size the flat-vector workloads use.  Only the shape is taken from the architecture."""
    sizes: list[int] = []

    def conv_bn(cin: int, cout: int, ksz: int):
        sizes.extend([cin * cout * ksz * ksz, cout, cout])

    conv_bn(3, 16, 3)
    width = 16
    for stage_width in (16, 32, 64):
        for block in range(3):
            conv_bn(width, stage_width, 3)
            conv_bn(stage_width, stage_width, 3)
            if block == 0 and width != stage_width:
                conv_bn(width, stage_width, 1)
            width = stage_width
    sizes.extend([64 * 10, 10])
    return sizes


def resnet50_layer_sizes() -> list[int]:
    """Lengths of the 161 parameter tensors of an ImageNet ResNet-50 in forward order (7x7 stem,
    bottleneck blocks [3, 4, 6, 3] of widths 64..512 with fourfold expansion, a batch-norm
    scale and shift after every convolution, 1x1 projection shortcuts at the head of each
    stage, a 2048 -> 1000 classifier).  They add up to 25 557 032."""
    sizes: list[int] = []

    def conv_bn(cin: int, cout: int, ksz: int):
        sizes.extend([cin * cout * ksz * ksz, cout, cout])

    conv_bn(3, 64, 7)
    cin = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for block in range(blocks):
            conv_bn(cin, width, 1)
            conv_bn(width, width, 3)
            conv_bn(width, 4 * width, 1)
            if block == 0:
                conv_bn(cin, 4 * width, 1)
            cin = 4 * width
    sizes.extend([2048 * 1000, 1000])
    return sizes


def layer_offsets(sizes) -> np.ndarray:
    """int64 [len + 1]: first coordinate of every layer of a flat vector, then its length."""
    return np.concatenate([[0], np.cumsum(np.asarray(sizes, dtype=np.int64))]).astype(np.int64)


# --------------------------------------------------------------------------
# the five workload shapes (shapes, scales and stepsizes only)
# --------------------------------------------------------------------------


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n: int
    d: int
    graph: str            # "ring" | "torus8x8" ...
    q: str                # "topk" | "randk" | "qsgd" | "sign"
    k: int = 0
    s: int = 0
    bucket: int = 0
    eta: float = 0.0
    gamma: float = 0.0
    steps: int = 0
    x_var: float = 1.0
    g_var: float = 0.0
    g_mean_var: float = 0.0
    sgd: bool = True
    layers: str = ""      # "" = Q on the whole row; "resnet20" / "resnet50" = Q per layer
    a_num: int = 1        # per-layer top-k / random-k keep max(1, floor(a d_l)), a = a_num / a_den
    a_den: int = 1
    momentum: float = 0.0      # > 0: Algorithm 2 with this momentum factor ...
    weight_decay: float = 0.0  # ... and this weight decay

    def layer_sizes(self) -> list[int]:
        return {"resnet20": resnet20_layer_sizes, "resnet50": resnet50_layer_sizes}[self.layers]()

    def mixing(self) -> MixingCSR:
        if self.graph == "ring":
            return ring(self.n)
        if self.graph.startswith("torus"):
            r, c = self.graph[5:].split("x")
            return torus(int(r), int(c))
        if self.graph == "social32":
            return random_graph(32, 14, 1)
        raise ValueError(self.graph)


WORKLOADS = {
    # average consensus only, 4-ring, top-k k=10
    "c1_ring4_topk": Workload("c1_ring4_topk", 4, 1024, "ring", "topk", k=10,
                              gamma=0.05, steps=200, x_var=1.0, sgd=False),
    # logistic regression d=2000 on a 16-ring: random-k 1 % and QSGD s=16 (whole-row norm)
    "c2_ring16_randk": Workload("c2_ring16_randk", 16, 2000, "ring", "randk",
                                k=k_of(1, 100, 2000), eta=0.1, gamma=0.1, steps=2000, x_var=0.0),
    # random-1 % at the consensus stepsize Table 4 lists for it (at 0.1 the run diverges)
    "c2_ring16_randk_g006": Workload("c2_ring16_randk_g006", 16, 2000, "ring", "randk",
                                     k=k_of(1, 100, 2000), eta=0.1, gamma=0.00625, steps=2000, x_var=0.0),
    "c2_ring16_qsgd": Workload("c2_ring16_qsgd", 16, 2000, "ring", "qsgd", s=16, bucket=0,
                               eta=0.1, gamma=0.1, steps=2000, x_var=0.0),
    # ResNet-20-sized flat vector, 8-ring, scaled sign
    "c3_ring8_sign": Workload("c3_ring8_sign", 8, 272474, "ring", "sign", eta=0.1, gamma=0.4,
                              steps=1000, x_var=0.01, g_var=1e-2, g_mean_var=1e-3),
    # the headline shape: 8x8 torus, d = 1e6, top-1 %
    "c4_torus64_topk": Workload("c4_torus64_topk", 64, 1_000_000, "torus8x8", "topk",
                                k=k_of(1, 100, 1_000_000), eta=0.05, gamma=0.2, steps=500,
                                x_var=1.0, g_var=1e-2),
    # the same at a consensus stepsize in the stable range for top-1 % (Table 4 lists 0.0375 as
    # the tuned value; with 0.2 the differences x - x^ grow over a run, with 0.04 they decay)
    "c4_torus64_topk_g004": Workload("c4_torus64_topk_g004", 64, 1_000_000, "torus8x8", "topk",
                                     k=k_of(1, 100, 1_000_000), eta=0.05, gamma=0.04, steps=500,
                                     x_var=1.0, g_var=1e-2),
    # Algorithm 2 (momentum 0.9, weight decay 1e-4) on the headline shape and on the 32-ring
    "c4_torus64_topk_mom": Workload("c4_torus64_topk_mom", 64, 1_000_000, "torus8x8", "topk",
                                    k=k_of(1, 100, 1_000_000), eta=0.05, gamma=0.04, steps=500,
                                    x_var=1.0, g_var=1e-2, momentum=0.9, weight_decay=1e-4),
    "c5_ring32_qsgd_mom": Workload("c5_ring32_qsgd_mom", 32, 25_557_032, "ring", "qsgd", s=16,
                                   bucket=512, eta=0.1, gamma=0.1, steps=200, x_var=0.01,
                                   g_var=1e-3, momentum=0.9, weight_decay=1e-4),
    # ResNet-50-sized flat vector, 32-ring: QSGD s=16 in 512-buckets, or top-0.1 %
    "c5_ring32_qsgd": Workload("c5_ring32_qsgd", 32, 25_557_032, "ring", "qsgd", s=16,
                               bucket=512, eta=0.1, gamma=0.1, steps=200, x_var=0.01,
                               g_var=1e-3),
    "c5_ring32_topk": Workload("c5_ring32_topk", 32, 25_557_032, "ring", "topk",
                               k=k_of(1, 1000, 25_557_032), eta=0.1, gamma=0.1, steps=200,
                               x_var=0.01, g_var=1e-3),
    # irregular 32-node graph (max degree 14), scaled sign as in the paper's on-device
    # runs: a ResNet-20-sized and an LSTM-sized (28.95 M) flat vector; and top-1 %
    "c6_social32_sign": Workload("c6_social32_sign", 32, 272474, "social32", "sign", eta=0.1,
                                 gamma=0.5, steps=1000, x_var=0.01, g_var=1e-2),
    "c6_social32_sign_lstm": Workload("c6_social32_sign_lstm", 32, 28_950_000, "social32", "sign",
                                      eta=0.1, gamma=0.6, steps=100, x_var=0.01, g_var=1e-3),
    "c6_social32_topk": Workload("c6_social32_topk", 32, 272474, "social32", "topk",
                                 k=k_of(1, 100, 272474), eta=0.1, gamma=0.04, steps=1000,
                                 x_var=0.01, g_var=1e-2),
    # per-layer compression, as in the paper's experiments (Section 5): the same flat vectors
    # cut into the parameter tensors of the network whose size they have
    "l3_ring8_sign_layers": Workload("l3_ring8_sign_layers", 8, 272474, "ring", "sign", eta=0.1, gamma=0.4,
                                     steps=1000, x_var=0.01, g_var=1e-2, layers="resnet20"),
    "l3_ring8_topk_layers": Workload("l3_ring8_topk_layers", 8, 272474, "ring", "topk", eta=0.1, gamma=0.04,
                                     steps=1000, x_var=0.01, g_var=1e-2, layers="resnet20",
                                     a_num=1, a_den=100),
    "l3_ring8_qsgd_layers": Workload("l3_ring8_qsgd_layers", 8, 272474, "ring", "qsgd", s=16, bucket=512,
                                     eta=0.1, gamma=0.1, steps=1000, x_var=0.01, g_var=1e-2,
                                     layers="resnet20"),
    "l5_ring32_qsgd_layers": Workload("l5_ring32_qsgd_layers", 32, 25_557_032, "ring", "qsgd", s=16,
                                      bucket=512, eta=0.1, gamma=0.1, steps=200, x_var=0.01,
                                      g_var=1e-3, layers="resnet50"),
    "l5_ring32_topk_layers": Workload("l5_ring32_topk_layers", 32, 25_557_032, "ring", "topk", eta=0.1,
                                      gamma=0.1, steps=200, x_var=0.01, g_var=1e-3,
                                      layers="resnet50", a_num=1, a_den=1000),
    # mid-sized dense cases (1 GB of state): small enough for a full counter capture,
    # larger than L2
    "p_ring8_qsgd": Workload("p_ring8_qsgd", 8, 8 * 1024 * 1024, "ring", "qsgd", s=16, bucket=512,
                             eta=0.1, gamma=0.1, steps=100, x_var=0.01, g_var=1e-3),
    "p_ring8_sign": Workload("p_ring8_sign", 8, 8 * 1024 * 1024, "ring", "sign", eta=0.1,
                             gamma=0.4, steps=100, x_var=0.01, g_var=1e-3),
}

# The operator settings of Table 1 on its shape (8-ring, ResNet-20-sized vector), each with the
# consensus stepsize Table 4 lists for it.  QSGD with b bits has s = 2^(b-1) levels.  Scaled sign
# is c3_ring8_sign.
for _name, _q, _kw, _gamma in [
    ("t1_ring8_qsgd16", "qsgd", dict(s=32768, bucket=512), 0.2),
    ("t1_ring8_qsgd8", "qsgd", dict(s=128, bucket=512), 0.2),
    ("t1_ring8_qsgd4", "qsgd", dict(s=8, bucket=512), 0.075),
    ("t1_ring8_qsgd2", "qsgd", dict(s=2, bucket=512), 0.025),
    ("t1_ring8_rand50", "randk", dict(k=k_of(1, 2, 272474)), 0.45),
    ("t1_ring8_rand10", "randk", dict(k=k_of(1, 10, 272474)), 0.075),
    ("t1_ring8_rand1", "randk", dict(k=k_of(1, 100, 272474)), 0.00625),
    ("t1_ring8_top50", "topk", dict(k=k_of(1, 2, 272474)), 0.45),
    ("t1_ring8_top10", "topk", dict(k=k_of(1, 10, 272474)), 0.15),
    ("t1_ring8_top1", "topk", dict(k=k_of(1, 100, 272474)), 0.0375),
]:
    WORKLOADS[_name] = Workload(_name, 8, 272474, "ring", _q, eta=0.1, gamma=_gamma, steps=1000,
                                x_var=0.01, g_var=1e-2, g_mean_var=1e-3, **_kw)


# --------------------------------------------------------------------------
# the convex problem of the d = 2000 workload (caller-side gradient of Algorithm 1)
# --------------------------------------------------------------------------


class LogisticProblem:
    """L2-regularised logistic regression split non-IID over n workers.

    Features ~ N(0, 1/d), labels sign(a . w*) for a seeded planted w*; all samples
    are sorted by label and dealt contiguously to the workers.  The gradient is the
    caller's job in Algorithm 1; it is evaluated here in float64 and handed,
    as float32, to whichever implementation is being driven.
    """

    def __init__(self, n: int, d: int, per_worker: int, seed: int, lam: float = 1e-4):
        rng = np.random.default_rng(seed)
        m = n * per_worker
        a = rng.standard_normal((m, d)) / math.sqrt(d)
        w_star = rng.standard_normal(d)
        y = np.where(a @ w_star >= 0.0, 1.0, -1.0)
        order = np.argsort(y, kind="stable")
        self.a = a[order].reshape(n, per_worker, d)
        self.y = y[order].reshape(n, per_worker)
        self.n, self.d, self.per_worker, self.lam, self.seed = n, d, per_worker, lam, seed

    def minibatch(self, step: int, worker: int, batch: int) -> np.ndarray:
        rng = np.random.default_rng([self.seed, 7, step, worker])
        return rng.integers(0, self.per_worker, size=batch)

    def gradient(self, x: np.ndarray, step: int, batch: int = 32) -> np.ndarray:
        """Mini-batch gradient of every worker at its x_i.  Written without a matrix product
        and without numpy's vectorised exp (both pick a code path by CPU model, so their last
        bits can differ between machines): products summed by numpy's fixed pairwise scheme,
        the exponential one sample at a time through the C library."""
        g = np.empty((self.n, self.d), dtype=np.float32)
        for i in range(self.n):
            rows = self.minibatch(step, i, batch)
            a, y = self.a[i, rows], self.y[i, rows]
            xi = x[i].astype(np.float64)
            margin = y * np.sum(a * xi, axis=1)
            # (a margin beyond the range of exp has a vanishing coefficient)
            coef = np.array([-yy / (1.0 + math.exp(mm)) if mm < 700.0 else 0.0 for yy, mm in zip(y, margin)])
            g[i] = ((coef[:, None] * a).sum(axis=0) / batch + self.lam * xi).astype(np.float32)
        return g

    def loss(self, xbar: np.ndarray) -> float:
        a = self.a.reshape(-1, self.d)
        y = self.y.reshape(-1)
        margin = y * (a @ xbar.astype(np.float64))
        return float(np.mean(np.logaddexp(0.0, -margin)) + 0.5 * self.lam * float(xbar @ xbar))
