"""Pins for the oracle's compression operators (Appendix C) and its generator.

Every check compares the oracle with something other than itself: published
known-answer vectors, brute force written with numpy's sort, closed forms, the
contraction bound of Definition 3.1, sizes the paper prints.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- generator


def test_philox_known_answers():
    for r in _rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_random_words_keying():
    d = 37
    w = oracle.random_words(seed=0x0123456789ABCDEF, step=(5 << 32) | 9, worker=3, stream=1, d=d)
    for c in (0, 1, 5, 36):
        ref = oracle.philox4x32_10([c // 4, 3, 9, (5 << 8) | 1], [0x89ABCDEF, 0x01234567])
        assert int(w[c]) == int(ref[c % 4])
    # a different step, worker or stream gives different words; same inputs repeat
    assert np.array_equal(w, oracle.random_words(0x0123456789ABCDEF, (5 << 32) | 9, 3, 1, d))
    for other in (oracle.random_words(0x0123456789ABCDEF, (5 << 32) | 10, 3, 1, d),
                  oracle.random_words(0x0123456789ABCDEF, (5 << 32) | 9, 4, 1, d),
                  oracle.random_words(0x0123456789ABCDEF, (5 << 32) | 9, 3, 0, d)):
        assert not np.array_equal(w, other)


def test_unit_interval_statistics():
    u = oracle.words_to_unit(oracle.random_words(7, 0, 0, 1, 1 << 18))
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(float(u.mean()) - 0.5) < 4e-3
    assert abs(float(u.var()) - 1.0 / 12.0) < 2e-3
    hist, _ = np.histogram(u, bins=16, range=(0.0, 1.0))
    expect = u.size / 16
    assert float(((hist - expect) ** 2 / expect).sum()) < 50.0          # chi^2, 15 dof
    # neighbouring coordinates uncorrelated
    assert abs(float(np.corrcoef(u[:-1], u[1:])[0, 1])) < 0.01


def test_words_to_unit_exact_values():
    """u = (word >> 8) * 2^-24: the TOP 24 bits, so the low byte never matters and the
    largest word stays below one.  (The low 24 bits, or a 23-bit shift, fail these.)"""
    words = np.array([0, 0xFF, 0x100, 0x80000000, 0xFFFFFFFF, 0x00FFFFFF, 0x12345678], dtype=np.uint32)
    want = [0.0, 0.0, 2.0 ** -24, 0.5, 1.0 - 2.0 ** -24, 0xFFFF * 2.0 ** -24, 0x123456 * 2.0 ** -24]
    got = oracle.words_to_unit(words)
    assert got.dtype == np.float32
    assert [float(x) for x in got] == want


def test_tree_sum_matches_hand_tree():
    a = np.array([1e8, 1.0, -1e8, 1.0, 3.0], dtype=np.float32)
    # ((a0+a1)+(a2+a3)) + a4 with float32 rounding at every node
    f = np.float32
    want = f(f(f(a[0] + a[1]) + f(a[2] + a[3])) + a[4])
    assert oracle.tree_sum(a) == want
    rng = np.random.default_rng(0)
    for m in (1, 2, 3, 7, 8, 9, 1000, 1025):
        x = rng.standard_normal(m).astype(np.float32)
        # exact sum in float64 is within a few ulps * log2(m) of the float32 tree
        assert abs(float(oracle.tree_sum(x)) - float(x.astype(np.float64).sum())) <= \
            1e-6 * float(np.abs(x).sum()) + 1e-12
    # padding with zeros to a power of two does not change the result
    x = rng.standard_normal(37).astype(np.float32)
    assert oracle.tree_sum(x) == oracle.tree_sum(np.concatenate([x, np.zeros(27, np.float32)]))


# ---------------------------------------------------------------- top_a


def _brute_topk(v, k):
    key = np.abs(v).view(np.uint32).astype(np.int64)
    order = np.lexsort((np.arange(v.size), -key))      # key descending, then index ascending
    return np.sort(order[:k]).astype(np.uint32)


@pytest.mark.parametrize("d,k", [(1, 1), (7, 3), (32, 5), (33, 33), (100, 1), (257, 40),
                                 (1024, 10)])
def test_topk_brute_force(d, k):
    rng = np.random.default_rng(d * 1000 + k)
    v = rng.standard_normal(d).astype(np.float32)
    m = oracle.compress_topk(v, k)
    want = _brute_topk(v, k)
    assert np.array_equal(m.idx, want)
    assert np.array_equal(m.val, v[want])
    dense = np.zeros(d, np.float32)
    dense[want] = v[want]
    assert np.array_equal(m.q, dense)
    assert m.mask.sum() == k and np.all(m.mask[want] == 1)


def test_topk_ties_take_lowest_indices():
    v = np.array([1, -2, 2, 0.5, 2, -2, 1, 2], dtype=np.float32)
    assert list(oracle.compress_topk(v, 3).idx) == [1, 2, 4]
    assert list(oracle.compress_topk(v, 5).idx) == [1, 2, 4, 5, 7]
    z = np.zeros(9, dtype=np.float32)
    z[4] = -0.0
    assert list(oracle.compress_topk(z, 4).idx) == [0, 1, 2, 3]
    many = np.full(300, 3.0, dtype=np.float32)
    many[::2] *= -1
    assert np.array_equal(oracle.compress_topk(many, 120).idx, np.arange(120, dtype=np.uint32))


def test_topk_full_is_identity_and_contraction():
    rng = np.random.default_rng(3)
    v = rng.standard_normal(500).astype(np.float32)
    assert np.array_equal(oracle.compress_topk(v, 500).q, v)
    v64 = v.astype(np.float64)
    for k in (1, 5, 50, 250, 499):
        q = oracle.compress_topk(v, k).q.astype(np.float64)
        # delta = k/d contraction of Definition 3.1 (deterministic for top_a)
        assert np.sum((q - v64) ** 2) <= (1 - k / 500) * np.sum(v64 ** 2) * (1 + 1e-12)


# ---------------------------------------------------------------- random_a


def test_randk_structure_and_message():
    d, k = 2000, 20
    rng = np.random.default_rng(1)
    v = rng.standard_normal(d).astype(np.float32)
    p = oracle.Params("randk", k=k, seed=11)
    m = oracle.compress(p, v, step=4, worker=2)
    assert m.idx.shape == (k,) and np.all(np.diff(m.idx.astype(np.int64)) > 0)
    assert m.idx.max() < d
    assert np.array_equal(m.val, v[m.idx])
    dense = np.zeros(d, np.float32)
    dense[m.idx] = v[m.idx]
    assert np.array_equal(m.q, dense)
    # the k smallest words, brute force
    w = oracle.random_words(11, 4, 2, oracle.STREAM_RANDK, d)
    order = np.lexsort((np.arange(d), w.astype(np.int64)))
    assert np.array_equal(m.idx, np.sort(order[:k]).astype(np.uint32))
    # masks differ across steps and workers, repeat for the same (step, worker)
    assert np.array_equal(m.idx, oracle.compress(p, v, 4, 2).idx)
    assert not np.array_equal(m.idx, oracle.compress(p, v, 5, 2).idx)
    assert not np.array_equal(m.idx, oracle.compress(p, v, 4, 3).idx)


def test_randk_forced_words():
    v = np.arange(1, 9, dtype=np.float32)
    words = np.array([5, 1, 9, 1, 7, 0, 3, 1], dtype=np.uint32)
    m = oracle.compress_randk(v, words, 3)
    assert list(m.idx) == [1, 3, 5]                       # 0 first, then the two lowest-index ones
    assert list(m.val) == [2.0, 4.0, 6.0]


def test_randk_uniform_and_delta_in_expectation():
    d, k, trials = 200, 20, 3000
    rng = np.random.default_rng(2)
    v = rng.standard_normal(d).astype(np.float32)
    v64 = v.astype(np.float64)
    p = oracle.Params("randk", k=k, seed=99)
    counts = np.zeros(d)
    err = 0.0
    for t in range(trials):
        m = oracle.compress(p, v, step=t, worker=0)
        counts[m.idx] += 1
        err += np.sum((m.q.astype(np.float64) - v64) ** 2)
    # E||Q(v) - v||^2 = (1 - k/d) ||v||^2 with equality for the biased random_a
    assert abs(err / trials / ((1 - k / d) * np.sum(v64 ** 2)) - 1.0) < 0.01
    expect = trials * k / d
    chi2 = float(((counts - expect) ** 2 / (expect * (1 - k / d))).sum())
    assert chi2 < d + 5 * np.sqrt(2 * d)


# ---------------------------------------------------------------- sign


def test_sign_closed_form_bits_and_size():
    rng = np.random.default_rng(5)
    for d in (1, 31, 32, 33, 100, 2000):
        v = rng.standard_normal(d).astype(np.float32)
        if d > 3:
            v[3] = 0.0
        m = oracle.compress_sign(v)
        v64 = v.astype(np.float64)
        l1 = np.abs(v64).sum()
        assert abs(float(m.scale) - l1 / d) <= 1e-6 * l1 / d
        # ||sign(v) - v||^2 = ||v||^2 - ||v||_1^2 / d, i.e. delta of Appendix C with equality
        q64 = m.q.astype(np.float64)
        assert np.sum((q64 - v64) ** 2) == pytest.approx(np.sum(v64 ** 2) - l1 * l1 / d,
                                                         rel=1e-5, abs=1e-9)
        neg = v < 0
        assert np.array_equal(m.q, np.where(neg, -m.scale, m.scale).astype(np.float32))
        unpacked = (m.bits[:, None] >> np.arange(32, dtype=np.uint32)[None, :]) & 1
        flat = unpacked.reshape(-1)
        assert np.array_equal(flat[:d].astype(bool), neg)
        assert not flat[d:].any()
        assert m.paper_bytes("sign", d) * 8 >= d + 32 > (m.paper_bytes("sign", d) - 4) * 8 - 32


def test_message_sizes_printed_in_paper():
    for op, d, param, nbytes, printed in _rows("message_sizes.txt"):
        d, param, nbytes = int(d), int(param), int(nbytes)
        v = np.ones(d, dtype=np.float32)
        if op == "full":
            got = oracle.Message(q=v).paper_bytes("identity", d)
        elif op == "sign":
            got = oracle.compress_sign(v).paper_bytes("sign", d)
        elif op == "topk":
            got = oracle.compress_topk(v, param).paper_bytes("topk", d)
            assert got * 8 == 2 * 32 * param
        else:
            got = oracle.compress(oracle.Params("randk", k=param), v, 0, 0).paper_bytes("randk", d)
            assert got * 8 == 32 * param
        assert got == nbytes
        if printed != "-":
            assert round(got / 2 ** 20, len(printed.split(".")[1])) == float(printed)


# ---------------------------------------------------------------- gsgd_b


def test_qsgd_zero_dither_is_floor_quantiser():
    # nu = 5 for (3, -4): s|v|/nu = 9.6 and 12.8 with s = 16 -> levels 9 and 12
    v = np.array([3.0, -4.0], dtype=np.float32)
    m = oracle.compress_qsgd(v, np.zeros(2, np.float32), s=16, bucket=0, biased=False)
    assert m.norms[0] == np.float32(5.0)
    assert list(m.levels) == [9 | (12 << 4)]
    assert list(m.bits) == [0b10]
    assert np.allclose(m.q, [5.0 * 9 / 16, -5.0 * 12 / 16], rtol=1e-7)
    # biased form divides by tau = 1 + min(d/s^2, sqrt(d)/s)
    mb = oracle.compress_qsgd(v, np.zeros(2, np.float32), s=16, bucket=0, biased=True)
    tau = 1 + min(2 / 256, np.sqrt(2) / 16)
    assert np.allclose(mb.q, m.q / tau, rtol=1e-6)


# v = (1, -2, 2, 0, 0, 0, 0, 0, 0, 4): the squares sum to 25, so nu = 5 exactly.
_HAND_V = np.array([1, -2, 2, 0, 0, 0, 0, 0, 0, 4], dtype=np.float32)


@pytest.mark.parametrize("s,u,levels,packed", [
    # s = 2, 1-bit fields: s|v|/nu = .4 .8 .8 0 ... 1.6 -> only the last reaches 1 (saturated)
    (2, 0.0, [0, 0, 0, 0, 0, 0, 0, 0, 0, 1], [0b00000000, 0b10]),
    # the same with u = 1/2: .9 1.3 1.3 .5 ... 2.1 -> 0 1 1 0 ... 1 (2 saturates to s - 1 = 1)
    (2, 0.5, [0, 1, 1, 0, 0, 0, 0, 0, 0, 1], [0b00000110, 0b10]),
    # s = 4, 2-bit fields: .8 1.6 1.6 0 ... 3.2 -> 0 1 1 0 ... 3; coordinate c at bits 2c, 2c+1
    (4, 0.0, [0, 1, 1, 0, 0, 0, 0, 0, 0, 3], [0b00010100, 0, 0b1100]),
    # s = 128, 8-bit fields: 25.6 51.2 51.2 0 ... 102.4 -> one byte per coordinate
    (128, 0.0, [25, 51, 51, 0, 0, 0, 0, 0, 0, 102], [25, 51, 51, 0, 0, 0, 0, 0, 0, 102]),
    # s = 2^15 (16 bits per coordinate with the sign: Table 1's first QSGD row), 16-bit fields,
    # low byte first: 6553.6 13107.2 13107.2 0 ... 26214.4 -> 0x1999 0x3333 0x3333 0 ... 0x6666
    (32768, 0.0, [6553, 13107, 13107, 0, 0, 0, 0, 0, 0, 26214],
     [0x99, 0x19, 0x33, 0x33, 0x33, 0x33] + [0] * 12 + [0x66, 0x66]),
    # u = 1/2 moves 6553.6 and 26214.4 up by one, 13107.2 stays, zeros stay
    (32768, 0.5, [6554, 13107, 13107, 0, 0, 0, 0, 0, 0, 26214],
     [0x9A, 0x19, 0x33, 0x33, 0x33, 0x33] + [0] * 12 + [0x66, 0x66]),
])
def test_qsgd_level_fields_by_hand(s, u, levels, packed):
    """Level fields of 1, 2, 8 and 16 bits written out by hand (Appendix C: a level is an integer
    in {0..s-1}; stored in the smallest of 1, 2, 4, 8, 16 bits, coordinate c at bit c * width)."""
    m = oracle.compress_qsgd(_HAND_V, np.full(10, u, np.float32), s=s, bucket=0, biased=False)
    assert m.norms[0] == np.float32(5.0)
    assert list(m.levels) == packed
    assert list(m.bits) == [0b10]                       # only coordinate 1 is negative
    want_q = np.array([5.0 / s * l for l in levels], dtype=np.float32)
    want_q[1] = -want_q[1]
    assert np.array_equal(m.q, want_q)


def test_qsgd_tau_values():
    assert float(oracle.qsgd_tau(512, 16)) == pytest.approx(1 + np.sqrt(512) / 16, rel=1e-7)
    assert float(oracle.qsgd_tau(40, 16)) == pytest.approx(1.15625, rel=1e-7)
    assert float(oracle.qsgd_tau(2000, 16)) == pytest.approx(1 + np.sqrt(2000) / 16, rel=1e-7)
    assert [oracle.qsgd_level_bits(s) for s in (2, 4, 8, 16, 32, 128, 256, 32768)] == [1, 2, 4, 4, 8, 8, 8, 16]


def test_qsgd_one_hot_saturates():
    v = np.zeros(8, dtype=np.float32)
    v[5] = -2.5
    m = oracle.compress_qsgd(v, np.full(8, 0.75, np.float32), s=16, bucket=0, biased=False)
    lev = [(int(m.levels[c // 2]) >> (4 * (c % 2))) & 15 for c in range(8)]
    assert lev == [0, 0, 0, 0, 0, 15, 0, 0]               # floor(16 + .75) = 16 -> 15
    assert m.q[5] == np.float32(-2.5 * 15 / 16)
    z = oracle.compress_qsgd(np.zeros(8, np.float32), np.full(8, 0.99, np.float32), 16, 0, True)
    assert not z.q.any() and not z.levels.any() and z.norms[0] == 0.0


def test_qsgd_buckets_and_layout():
    rng = np.random.default_rng(8)
    d, bucket, s = 1064, 512, 16
    v = rng.standard_normal(d).astype(np.float32)
    u = rng.random(d).astype(np.float32)
    m = oracle.compress_qsgd(v, u, s, bucket, True)
    assert m.norms.shape == (3,)
    for b, (lo, hi) in enumerate([(0, 512), (512, 1024), (1024, 1064)]):
        seg = v[lo:hi].astype(np.float64)
        nu = np.sqrt(np.sum(seg ** 2))
        assert float(m.norms[b]) == pytest.approx(nu, rel=1e-6)
        tau = 1 + min((hi - lo) / s ** 2, np.sqrt(hi - lo) / s)
        lev = np.array([(int(m.levels[c // 2]) >> (4 * (c % 2))) & 15 for c in range(lo, hi)])
        want = np.minimum(np.floor(s * np.abs(seg) / nu + u[lo:hi]), s - 1)
        # float32 vs float64 may differ only where r + u sits on an integer boundary
        assert np.mean(lev != want) < 0.01 and np.max(np.abs(lev - want)) <= 1
        qq = np.sign(seg + 0.0) * float(m.norms[b]) / (tau * s) * lev
        qq[seg == 0] = np.abs(qq[seg == 0])
        assert np.allclose(m.q[lo:hi], qq, rtol=1e-5, atol=0)
    assert m.paper_bytes("qsgd", d) == 3 * 4 + 4 * ((d + 31) // 32) + d // 2


def test_qsgd_unbiased_and_contraction():
    d, s, trials = 256, 16, 2000
    rng = np.random.default_rng(4)
    v = rng.standard_normal(d).astype(np.float32)
    v64 = v.astype(np.float64)
    mean = np.zeros(d)
    err_b = 0.0
    pu = oracle.Params("qsgd", s=s, bucket=0, biased=False, seed=5)
    pb = oracle.Params("qsgd", s=s, bucket=0, biased=True, seed=5)
    for t in range(trials):
        mean += oracle.compress(pu, v, t, 1).q
        err_b += np.sum((oracle.compress(pb, v, t, 1).q.astype(np.float64) - v64) ** 2)
    mean /= trials
    nu = np.sqrt(np.sum(v64 ** 2))
    # unbiased form: E q = v; per-coordinate std of the mean is <= nu / (2 s sqrt(trials))
    assert np.max(np.abs(mean - v64)) < 6 * nu / (2 * s * np.sqrt(trials))
    tau = 1 + min(d / s ** 2, np.sqrt(d) / s)
    assert err_b / trials <= (1 - 1 / tau) * np.sum(v64 ** 2)
