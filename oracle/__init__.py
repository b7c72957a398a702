"""CPU oracle for the CHOCO-Gossip / CHOCO-SGD step -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes layer over ``choco_oracle.c`` (the arithmetic lives there) plus
three drivers written straight from the paper:

* :func:`step`            -- one call of the three-vector form (Section 3, last
  paragraph): q = Q(x - x^); x^ += q; s += W q; x = (x - eta g) + gamma (s - x^).
* :func:`alg1_literal`    -- Algorithm 1 as printed, every worker holding its own
  copy of x^_j for each neighbour (tiny sizes; cross-check of :func:`step`).
* :func:`alg4_error_feedback` -- the error-feedback rewrite (Algorithm 4).

Nothing here may be imported by the product package; only tests, the smoke check
and the benchmark's CPU-baseline leg use it.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "choco_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

_c_f = ctypes.POINTER(ctypes.c_float)
_c_u32 = ctypes.POINTER(ctypes.c_uint32)
_c_u8 = ctypes.POINTER(ctypes.c_uint8)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no FMA contraction) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-Wall", "-shared", "-fPIC",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_tree_sum.restype = ctypes.c_float
        _lib.oracle_qsgd_tau.restype = ctypes.c_float
        _lib.oracle_qsgd_level_bits.restype = ctypes.c_int32
        _lib.oracle_consensus_error.restype = ctypes.c_double
    return _lib


def _f(a: np.ndarray):
    assert a.dtype == np.float32 and a.flags.c_contiguous
    return a.ctypes.data_as(_c_f)


def _u32(a: np.ndarray):
    assert a.dtype == np.uint32 and a.flags.c_contiguous
    return a.ctypes.data_as(_c_u32)


def _u8(a: np.ndarray):
    assert a.dtype == np.uint8 and a.flags.c_contiguous
    return a.ctypes.data_as(_c_u8)


# ---------------------------------------------------------------------------
# generator
# ---------------------------------------------------------------------------

STREAM_RANDK = 0
STREAM_DITHER = 1


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_u32(c), _u32(k), _u32(out))
    return out


def random_words(seed: int, step: int, worker: int, stream: int, d: int) -> np.ndarray:
    words = np.zeros(d, dtype=np.uint32)
    lib().oracle_random_words(ctypes.c_uint64(seed), ctypes.c_uint64(step),
                              ctypes.c_uint32(worker), ctypes.c_uint32(stream),
                              ctypes.c_int64(d), _u32(words))
    return words


def words_to_unit(words: np.ndarray) -> np.ndarray:
    u = np.zeros(words.shape[0], dtype=np.float32)
    lib().oracle_words_to_unit(_u32(words), ctypes.c_int64(words.shape[0]), _f(u))
    return u


def tree_sum(a: np.ndarray) -> np.float32:
    tmp = np.ascontiguousarray(a, dtype=np.float32).copy()
    return np.float32(lib().oracle_tree_sum(_f(tmp), ctypes.c_int64(tmp.shape[0])))


def qsgd_tau(length: int, s: int) -> np.float32:
    return np.float32(lib().oracle_qsgd_tau(ctypes.c_int64(length), ctypes.c_int32(s)))


def qsgd_level_bits(s: int) -> int:
    return int(lib().oracle_qsgd_level_bits(ctypes.c_int32(s)))


# ---------------------------------------------------------------------------
# compression operators (Appendix C)
# ---------------------------------------------------------------------------


@dataclasses.dataclass
class Params:
    """Q and its parameter.  kind in {"identity", "topk", "randk", "qsgd", "sign"}."""

    kind: str
    k: int = 0            # topk / randk: floor(a d)
    s: int = 16           # qsgd: 2^(b-1) levels
    bucket: int = 0       # qsgd: block length, 0 = whole row
    biased: bool = True   # qsgd: divide by tau
    seed: int = 0


@dataclasses.dataclass
class Message:
    """What one worker sends, plus the dense q it stands for."""

    q: np.ndarray                         # float32 [d]
    mask: Optional[np.ndarray] = None     # uint8 [d] for sparse Q, else None
    idx: Optional[np.ndarray] = None      # uint32 [k] ascending (topk, randk)
    val: Optional[np.ndarray] = None      # float32 [k]
    bits: Optional[np.ndarray] = None     # uint32 [ceil(d/32)] sign plane (sign, qsgd)
    scale: Optional[np.float32] = None    # sign: ||v||_1 / d
    norms: Optional[np.ndarray] = None    # qsgd: float32 per block
    levels: Optional[np.ndarray] = None   # qsgd: packed level fields (uint8)

    def paper_bytes(self, kind: str, d: int, s: int = 16) -> int:
        """Message size by the paper's accounting (Appendix C)."""
        if kind == "topk":
            return 8 * int(self.idx.shape[0])
        if kind == "randk":
            return 4 * int(self.idx.shape[0])
        if kind == "sign":
            return 4 * ((d + 31) // 32) + 4
        if kind == "qsgd":
            return int(self.norms.nbytes + self.bits.nbytes + self.levels.nbytes)
        return 4 * d


def select_largest(key: np.ndarray, k: int) -> np.ndarray:
    key = np.ascontiguousarray(key, dtype=np.uint32)
    idx = np.zeros(k, dtype=np.uint32)
    rc = lib().oracle_select_largest(_u32(key), ctypes.c_int64(key.shape[0]), ctypes.c_int64(k),
                                     _u32(idx))
    if rc:
        raise ValueError(f"oracle_select_largest rc={rc}")
    return idx


def compress_topk(v: np.ndarray, k: int) -> Message:
    d = v.shape[0]
    idx = np.zeros(k, dtype=np.uint32)
    val = np.zeros(k, dtype=np.float32)
    q = np.zeros(d, dtype=np.float32)
    mask = np.zeros(d, dtype=np.uint8)
    rc = lib().oracle_compress_topk(_f(v), ctypes.c_int64(d), ctypes.c_int64(k), _u32(idx),
                                    _f(val), _f(q), _u8(mask))
    if rc:
        raise ValueError(f"oracle_compress_topk rc={rc}")
    return Message(q=q, mask=mask, idx=idx, val=val)


def compress_randk(v: np.ndarray, words: np.ndarray, k: int) -> Message:
    d = v.shape[0]
    idx = np.zeros(k, dtype=np.uint32)
    val = np.zeros(k, dtype=np.float32)
    q = np.zeros(d, dtype=np.float32)
    mask = np.zeros(d, dtype=np.uint8)
    rc = lib().oracle_compress_randk(_f(v), _u32(words), ctypes.c_int64(d), ctypes.c_int64(k),
                                     _u32(idx), _f(val), _f(q), _u8(mask))
    if rc:
        raise ValueError(f"oracle_compress_randk rc={rc}")
    return Message(q=q, mask=mask, idx=idx, val=val)


def compress_sign(v: np.ndarray) -> Message:
    d = v.shape[0]
    bits = np.zeros((d + 31) // 32, dtype=np.uint32)
    scale = ctypes.c_float(0.0)
    q = np.zeros(d, dtype=np.float32)
    rc = lib().oracle_compress_sign(_f(v), ctypes.c_int64(d), _u32(bits), ctypes.byref(scale),
                                    _f(q))
    if rc:
        raise ValueError(f"oracle_compress_sign rc={rc}")
    return Message(q=q, bits=bits, scale=np.float32(scale.value))


def compress_qsgd(v: np.ndarray, u: np.ndarray, s: int, bucket: int, biased: bool) -> Message:
    d = v.shape[0]
    blen = bucket if bucket > 0 else d
    nb = (d + blen - 1) // blen
    wbits = qsgd_level_bits(s)
    norms = np.zeros(nb, dtype=np.float32)
    bits = np.zeros((d + 31) // 32, dtype=np.uint32)
    levels = np.zeros((d * wbits + 7) // 8, dtype=np.uint8)
    q = np.zeros(d, dtype=np.float32)
    rc = lib().oracle_compress_qsgd(_f(v), _f(u), ctypes.c_int64(d), ctypes.c_int32(s),
                                    ctypes.c_int64(bucket), ctypes.c_int32(1 if biased else 0),
                                    _f(norms), _u32(bits), _u8(levels), _f(q))
    if rc:
        raise ValueError(f"oracle_compress_qsgd rc={rc}")
    return Message(q=q, bits=bits, norms=norms, levels=levels)


def difference(x: np.ndarray, xhat: np.ndarray) -> np.ndarray:
    v = np.zeros_like(x)
    lib().oracle_difference(_f(x), _f(xhat), ctypes.c_int64(x.shape[0]), _f(v))
    return v


def compress(p: Params, v: np.ndarray, step: int, worker: int) -> Message:
    """q = Q(v) for worker `worker` at step `step` (Algorithm 1, the compression step)."""
    d = v.shape[0]
    if p.kind == "identity":
        return Message(q=v.copy())
    if p.kind == "topk":
        return compress_topk(v, p.k)
    if p.kind == "randk":
        return compress_randk(v, random_words(p.seed, step, worker, STREAM_RANDK, d), p.k)
    if p.kind == "sign":
        return compress_sign(v)
    if p.kind == "qsgd":
        u = words_to_unit(random_words(p.seed, step, worker, STREAM_DITHER, d))
        return compress_qsgd(v, u, p.s, p.bucket, p.biased)
    raise ValueError(p.kind)


# ---------------------------------------------------------------------------
# the step, three-vector form
# ---------------------------------------------------------------------------


def _apply_row(i, w, X, Xhat, S, G, msgs, eta, gamma, M=None, lam=0.0, beta=0.0, nesterov=False):
    d = X.shape[1]
    lo, hi = int(w.row_ptr[i]), int(w.row_ptr[i + 1])
    cols = [int(c) for c in w.col[lo:hi]]
    nnb = len(cols)
    self_pos = cols.index(i)
    qarr = (_c_f * nnb)(*[_f(msgs[j].q) for j in cols])
    sparse = msgs[cols[0]].mask is not None
    marr = (_c_u8 * nnb)(*[_u8(msgs[j].mask) for j in cols]) if sparse else None
    wv = np.ascontiguousarray(w.val[lo:hi], dtype=np.float32)
    g = _f(G[i]) if G is not None else None
    if M is None:
        lib().oracle_apply_row(ctypes.c_int64(d), _f(X[i]), _f(Xhat[i]), _f(S[i]), g,
                               ctypes.c_int32(nnb), qarr, marr, _f(wv),
                               ctypes.c_int32(self_pos), ctypes.c_float(eta),
                               ctypes.c_float(gamma))
    else:
        lib().oracle_apply_row_momentum(ctypes.c_int64(d), _f(X[i]), _f(Xhat[i]), _f(S[i]), g,
                                        _f(M[i]), ctypes.c_int32(nnb), qarr, marr, _f(wv),
                                        ctypes.c_int32(self_pos), ctypes.c_float(eta),
                                        ctypes.c_float(gamma), ctypes.c_float(lam),
                                        ctypes.c_float(beta), ctypes.c_int32(1 if nesterov else 0))


def step(w, p: Params, X: np.ndarray, Xhat: np.ndarray, S: np.ndarray,
         G: Optional[np.ndarray], eta: float, gamma: float, t: int,
         rows: Optional[Sequence[int]] = None, M: Optional[np.ndarray] = None,
         lam: float = 0.0, beta: float = 0.0, executor=None, nesterov: bool = False) -> dict:
    """One call on float32 [n, d] arrays, in place.  Returns {worker: Message}.

    With `rows`, only those workers are updated (their neighbours' messages are still
    formed): a way to check single rows of a large problem.  With `M` the momentum
    variant of Algorithm 2 is applied instead of the plain SGD step; `nesterov` takes that
    step along (g + lam x) + beta v' instead of the new memory v' (Appendix D names the
    variant without a formula: the usual look-ahead form is the reading).  `executor` (a
    concurrent.futures executor of threads; the C routines run without the interpreter
    lock) only spreads the per-worker calls over host cores: all messages are formed
    before any row is updated, and rows are independent of each other, so the result
    is the same.
    """
    n = X.shape[0]
    todo = list(range(n)) if rows is None else list(rows)
    need = set()
    for i in todo:
        need.update(int(c) for c in w.col[w.row_ptr[i]:w.row_ptr[i + 1]])
    need = sorted(need)
    run = map if executor is None else executor.map
    msgs = dict(zip(need, run(lambda j: compress(p, difference(X[j], Xhat[j]), t, j), need)))
    list(run(lambda i: _apply_row(i, w, X, Xhat, S, G, msgs, eta, gamma, M, lam, beta, nesterov), todo))
    return msgs


def layer_k(a_num: int, a_den: int, length: int) -> int:
    """Entries a sparse Q keeps of a layer: floor(a d_l), but at least one (with floor(a d_l)
    = 0 a small layer would never be transmitted)."""
    return max(1, (length * a_num) // a_den)


def step_layers(w, p: Params, layer_off: Sequence[int], a_num: int, a_den: int,
                X: np.ndarray, Xhat: np.ndarray, S: np.ndarray, G: Optional[np.ndarray],
                eta: float, gamma: float, t: int, M: Optional[np.ndarray] = None,
                lam: float = 0.0, beta: float = 0.0, nesterov: bool = False,
                rows: Optional[Sequence[int]] = None) -> list:
    """Per-layer compression (Section 5, "Setup": every compression scheme is applied to
    every layer separately): the columns [layer_off[l], layer_off[l+1]) of the arrays are
    layer l, and one call of :func:`step` is made on each layer as a problem of its own
    -- its own k = layer_k(a, d_l) for top-k / random-k, its own scale (sign) or blocks
    (qsgd), the generator keyed with seed + l and the coordinate's index inside the layer.
    Returns the per-layer message dictionaries."""
    out = []
    for l in range(len(layer_off) - 1):
        lo, hi = int(layer_off[l]), int(layer_off[l + 1])
        pl = dataclasses.replace(p, seed=p.seed + l)
        if p.kind in ("topk", "randk"):
            pl = dataclasses.replace(pl, k=layer_k(a_num, a_den, hi - lo))
        parts = [np.ascontiguousarray(A[:, lo:hi]) if A is not None else None
                 for A in (X, Xhat, S, G, M)]
        out.append(step(w, pl, parts[0], parts[1], parts[2], parts[3], eta, gamma, t,
                        rows=rows, M=parts[4], lam=lam, beta=beta, nesterov=nesterov))
        for A, part in ((X, parts[0]), (Xhat, parts[1]), (S, parts[2]), (M, parts[4])):
            if A is not None:
                A[:, lo:hi] = part
    return out


def consensus_error(X: np.ndarray) -> float:
    """sum_i ||x_i - xbar||^2 in float64 (Section 6's distance times n)."""
    X = np.ascontiguousarray(X, dtype=np.float32)
    return float(lib().oracle_consensus_error(_f(X), ctypes.c_int64(X.shape[0]),
                                              ctypes.c_int64(X.shape[1]),
                                              ctypes.c_int64(X.shape[1])))


def theoretical_gamma(rho: float, delta: float, beta: float) -> float:
    """Consensus stepsize of Theorem 4.1."""
    return rho * rho * delta / (16 * rho + rho * rho + 4 * beta * beta + 2 * rho * beta * beta
                                - 8 * rho * delta)


# ---------------------------------------------------------------------------
# Algorithm 1 as printed, and its error-feedback rewrite (tiny sizes)
# ---------------------------------------------------------------------------


def _line2(x, hat, nbrs, wts, gamma):
    n, d = x.shape
    for i in range(n):
        corr = np.zeros(d, dtype=np.float32)
        for e, j in enumerate(nbrs[i]):
            corr = corr + wts[i][e] * (hat[i][j] - hat[i][i])
        x[i] = x[i] + np.float32(gamma) * corr


def alg1_literal(w, p: Params, x0: np.ndarray, grads, eta: float, gamma: float,
                 steps: int, final_gossip: bool = False) -> np.ndarray:
    """Algorithm 1 with per-neighbour copies.  `x0` is x^(-1/2) [n, d]; `grads(t, X)`
    returns the [n, d] float32 gradients at x^(t) (or None for pure gossip).  Returns
    x^(T-1/2), the iterate after the last SGD step, or x^(T) (one more gossip step) with
    `final_gossip`.  float32 throughout."""
    n, d = x0.shape
    x = x0.astype(np.float32).copy()
    nbrs = [[int(c) for c in w.col[w.row_ptr[i]:w.row_ptr[i + 1]]] for i in range(n)]
    wts = [w.val[w.row_ptr[i]:w.row_ptr[i + 1]].astype(np.float32) for i in range(n)]
    # hat[i][j]: worker i's copy of x^_j
    hat = [{j: np.zeros(d, dtype=np.float32) for j in nbrs[i]} for i in range(n)]
    for t in range(steps):
        _line2(x, hat, nbrs, wts, gamma)                       # gossip step
        q = [compress(p, difference(x[i], hat[i][i]), t, i).q for i in range(n)]   # compression
        for i in range(n):                                     # exchange q, update the copies
            for j in nbrs[i]:
                hat[i][j] = hat[i][j] + q[j]
        g = grads(t, x) if grads is not None else None         # gradient evaluation
        if g is not None:
            x = x - np.float32(eta) * g                        # gradient step
    if final_gossip:
        _line2(x, hat, nbrs, wts, gamma)
    return x


def alg4_error_feedback(w, p: Params, x0: np.ndarray, grads, eta: float, gamma: float,
                        steps: int, final_gossip: bool = False) -> np.ndarray:
    """Algorithm 4: the same iterates with v = x^(t) - x^(t-1) + m, q = Q(v),
    m <- v - q in place of the compression step, x^(-1) = 0."""
    n, d = x0.shape
    x = x0.astype(np.float32).copy()
    nbrs = [[int(c) for c in w.col[w.row_ptr[i]:w.row_ptr[i + 1]]] for i in range(n)]
    wts = [w.val[w.row_ptr[i]:w.row_ptr[i + 1]].astype(np.float32) for i in range(n)]
    hat = [{j: np.zeros(d, dtype=np.float32) for j in nbrs[i]} for i in range(n)]
    x_prev = np.zeros((n, d), dtype=np.float32)
    mem = np.zeros((n, d), dtype=np.float32)
    for t in range(steps):
        _line2(x, hat, nbrs, wts, gamma)
        q = []
        for i in range(n):
            v = (x[i] - x_prev[i]) + mem[i]
            qi = compress(p, np.ascontiguousarray(v), t, i).q
            mem[i] = v - qi
            q.append(qi)
        x_prev = x.copy()
        for i in range(n):
            for j in nbrs[i]:
                hat[i][j] = hat[i][j] + q[j]
        g = grads(t, x) if grads is not None else None
        if g is not None:
            x = x - np.float32(eta) * g
    if final_gossip:
        _line2(x, hat, nbrs, wts, gamma)
    return x
