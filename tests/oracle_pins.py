"""Pins that tie the CPU oracle to the paper and to plain mathematics.

Every function takes the loaded oracle library (so that the very same checks can be
run against deliberately broken copies of the oracle, see test_oracle_mutants.py)
and raises AssertionError when the oracle disagrees with

  * hand-worked iterations of Algorithm 1 (tests/golden/*.txt),
  * exact rational arithmetic (fractions.Fraction) for the mean of |x| (Def. 4),
  * brute-force Python loops for bit packing and for sorting by magnitude (Def. 2),
  * the contraction property of Def. 1 and the identities that follow from Def. 4,
  * the error recursion e_{t+1} = v_t - p_t and Lemma 3,
  * plain SGD for the identity operator with one worker,
  * Def. 3 / Assumption 4 averaged exactly over every k-subset of a small vector.
"""
from __future__ import annotations

import math
import os
from fractions import Fraction

import numpy as np

import oracle
from oracle import IDENTITY, SIGN, TOPK, RANDK

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


# ----------------------------------------------------------------------------- helpers

def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":")
            out[key.strip()] = [float(v) for v in vals.split()]
    return out


def decode_sign(words, scales, off):
    off = np.asarray(off, dtype=np.int64)
    d = int(off[-1])
    out = np.zeros(d, np.float32)
    woff = 0
    for t in range(len(off) - 1):
        n = int(off[t + 1] - off[t])
        for j in range(n):
            bit = (int(words[woff + j // 32]) >> (j % 32)) & 1
            out[off[t] + j] = -scales[t] if bit else scales[t]
        woff += (n + 31) // 32
    return out


def decode_topk(idx, val, d):
    out = np.zeros(d, np.float32)
    out[np.asarray(idx, dtype=np.int64)] = val
    return out


def brute_topk(x, k):
    """Indices of the k largest |x| (ties to the lower index), ascending.  Pure Python."""
    order = sorted(range(len(x)), key=lambda j: (-abs(float(x[j])), j))
    return sorted(order[:k])


def exact_mean_abs_f32(x):
    """float32 nearest to the exact rational mean of |x|."""
    total = sum((Fraction(abs(float(v))) for v in x), Fraction(0))
    mean = total / len(x)
    f = np.float32(float(mean))           # Fraction -> double is correctly rounded
    # resolve double rounding: pick the float32 neighbour closest to the exact mean
    cands = [f, np.nextafter(f, np.float32(np.inf)), np.nextafter(f, np.float32(-np.inf))]
    return min(cands, key=lambda c: abs(Fraction(float(c)) - mean))


# ----------------------------------------------------------------------------- golden

def _run_golden(L, name, up, down):
    g = read_golden(name)
    N, d = int(g["N"][0]), int(g["d"][0])
    off = np.asarray(g["off"], dtype=np.int64)
    k = np.asarray(g["k"], dtype=np.int64) if "k" in g else None
    lr = g["lr"][0]
    X = np.tile(np.asarray(g["x0"], np.float32), (N, 1)).copy()
    e = np.zeros(d, np.float32)
    step = 1
    while f"g.{step}.0" in g:
        G = np.asarray([g[f"g.{step}.{i}"] for i in range(N)], np.float32)
        r = oracle.step(X, e, G, lr, off, up, down, k=k, _lib=L)
        for i in range(N):
            if up == SIGN:
                assert r.up_scales[i].tolist() == g[f"up_scales.{step}.{i}"], (name, step, i, "up_scales")
                assert r.up_words[i].tolist() == g[f"up_words.{step}.{i}"], (name, step, i, "up_words")
            if up == TOPK:
                assert r.up_idx[i].tolist() == g[f"up_idx.{step}.{i}"], (name, step, i, "up_idx")
                assert r.up_val[i].tolist() == g[f"up_val.{step}.{i}"], (name, step, i, "up_val")
            assert X[i].tolist() == g[f"x.{step}.{i}"], (name, step, i, "x", X[i])
        assert r.v.tolist() == g[f"v.{step}"], (name, step, "v", r.v)
        if down == SIGN:
            assert r.down_scales.tolist() == g[f"down_scales.{step}"], (name, step, "down_scales")
            assert r.down_words.tolist() == g[f"down_words.{step}"], (name, step, "down_words")
        if down == TOPK:
            assert r.down_idx.tolist() == g[f"down_idx.{step}"], (name, step, "down_idx")
            assert r.down_val.tolist() == g[f"down_val.{step}"], (name, step, "down_val")
        assert e.tolist() == g[f"e.{step}"], (name, step, "e", e)
        step += 1
    assert step > 1


def pin_golden_sign(L):
    _run_golden(L, "sign_two_steps.txt", SIGN, SIGN)


def pin_golden_blockwise(L):
    _run_golden(L, "blockwise_one_step.txt", SIGN, SIGN)


def pin_golden_topk(L):
    _run_golden(L, "topk_one_step.txt", TOPK, TOPK)


# ----------------------------------------------------------------------------- scaled sign

def pin_scale_is_exact_mean(L):
    """Def. 4: the scale is ||x||_1 / d.  Compared with exact rational arithmetic."""
    rng = np.random.default_rng(11)
    for n in (1, 2, 3, 5, 31, 32, 33, 100, 257, 1000, 4097):
        x = rng.standard_normal(n).astype(np.float32)
        assert oracle.scale(x, _lib=L) == exact_mean_abs_f32(x), n
        x = (rng.standard_normal(n) * np.exp(rng.uniform(-20, 20, n))).astype(np.float32)
        assert oracle.scale(x, _lib=L) == exact_mean_abs_f32(x), ("wide", n)
    # closed forms
    assert oracle.scale(np.full(64, -0.75, np.float32), _lib=L) == np.float32(0.75)
    assert oracle.scale(np.asarray([1, -2, 3, -4], np.float32), _lib=L) == np.float32(2.5)
    assert oracle.scale(np.asarray([0.0, -0.0, 0.0], np.float32), _lib=L) == np.float32(0.0)
    assert oracle.scale(np.asarray([3.0, 0.0, 0.0], np.float32), _lib=L) == np.float32(1.0)


def pin_tree_shape(L):
    """The binary64 sum follows the balanced tree over the zero-padded power of two.

    Expected values derived by hand from IEEE round-to-nearest-even:
    2^53 + 1 rounds back to 2^53, while 1 + 1 = 2 is added exactly.
    """
    big = float(2 ** 53)
    t = lambda v: oracle.tree_abs_sum(np.asarray(v, np.float32), _lib=L)
    assert t([big, 1, 1, 1]) == big + 2          # (big+1) + (1+1); a running sum gives big
    assert t([1, 1, 1, big]) == big + 2          # (1+1) + (1+big)
    assert t([big, 1, 1]) == big                 # (big+1) + (1+0) = big + 1 -> ties to even
    assert t([1, big, 1, 1, 1, 1, 1, 1]) == big + 6   # ((1+big)+(1+1)) + ((1+1)+(1+1))
    assert t([big, 1, 1, 1, 1]) == big + 4       # padded to 8: ((big+1)+(1+1)) + ((1+0)+0) = (big+2)+1 -> ties to even
    assert t([-1.5, 2.5]) == 4.0
    x = np.random.default_rng(5).standard_normal(1000).astype(np.float32)
    assert abs(t(x) - math.fsum(abs(float(v)) for v in x)) <= 1e-12 * 1000


def pin_sign_bits_bruteforce(L):
    """Bit b of word w of segment t is set iff element off[t]+32w+b < 0; padding bits 0."""
    rng = np.random.default_rng(3)
    sizes = [1, 7, 32, 33, 64, 95, 1, 130]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    x = rng.standard_normal(int(off[-1])).astype(np.float32)
    x[::11] = 0.0
    x[5::13] = -0.0
    words, scales, dec = oracle.sign_compress(x, off, _lib=L)
    assert len(words) == sum((n + 31) // 32 for n in sizes)
    woff = 0
    negatives = 0
    for t, n in enumerate(sizes):
        seg = x[off[t]:off[t + 1]]
        expect = [0] * ((n + 31) // 32)
        for j in range(n):
            if float(seg[j]) < 0.0:
                expect[j // 32] |= 1 << (j % 32)
                negatives += 1
        assert [int(w) for w in words[woff:woff + len(expect)]] == expect, t
        assert scales[t] == exact_mean_abs_f32(seg), t
        for j in range(n):
            want = -scales[t] if float(seg[j]) < 0.0 else scales[t]
            assert dec[off[t] + j] == want
        woff += len(expect)
    assert sum(bin(int(w)).count("1") for w in words) == negatives
    assert np.array_equal(decode_sign(words, scales, off), dec)


def pin_sign_contraction(L):
    """Def. 1 with Def. 4: ||x - C(x)||^2 = ||x||^2 - d s^2 <= (1 - delta)||x||^2, delta -> 2/pi on Gaussians."""
    rng = np.random.default_rng(7)
    n = 200_000
    x = rng.standard_normal(n).astype(np.float32)
    _, scales, dec = oracle.sign_compress(x, [0, n], _lib=L)
    x64, c64 = x.astype(np.float64), dec.astype(np.float64)
    lhs = np.sum((x64 - c64) ** 2)
    rhs = np.sum(x64 ** 2) - n * float(scales[0]) ** 2
    assert abs(lhs - rhs) <= 1e-6 * rhs
    delta = 1.0 - lhs / np.sum(x64 ** 2)
    assert abs(delta - 2.0 / math.pi) < 0.01
    assert abs(float(scales[0]) - math.sqrt(2.0 / math.pi)) < 0.01


def pin_blockwise_reduces_to_sign(L):
    """Def. 5 with one block is Def. 4; with several blocks it is Def. 4 per block."""
    rng = np.random.default_rng(9)
    x = rng.standard_normal(300).astype(np.float32)
    w1, s1, d1 = oracle.sign_compress(x, [0, 300], _lib=L)
    assert s1[0] == exact_mean_abs_f32(x)
    off = [0, 64, 96, 300]
    w, s, d = oracle.sign_compress(x, off, _lib=L)
    wcat, dcat = [], []
    for t in range(3):
        wt, st, dt = oracle.sign_compress(x[off[t]:off[t + 1]], [0, off[t + 1] - off[t]], _lib=L)
        assert st[0] == s[t]
        wcat.append(wt)
        dcat.append(dt)
    assert np.array_equal(np.concatenate(wcat), w) and np.array_equal(np.concatenate(dcat), d)
    # idempotence when the block length is a power of two (n * s / n is exact)
    x = rng.standard_normal(256).astype(np.float32)
    _, s_a, d_a = oracle.sign_compress(x, [0, 256], _lib=L)
    w_b, s_b, d_b = oracle.sign_compress(d_a, [0, 256], _lib=L)
    assert s_a[0] == s_b[0] and np.array_equal(d_a, d_b)


# ----------------------------------------------------------------------------- top-k

def pin_topk_bruteforce(L):
    """Def. 2 against a full Python sort, with heavy ties, zeros and +-pairs."""
    rng = np.random.default_rng(13)
    cases = []
    cases.append((rng.integers(-3, 4, 200).astype(np.float32), 17))          # many ties
    cases.append((np.zeros(50, np.float32), 5))                               # all equal (zeros)
    cases.append((np.full(40, -2.0, np.float32), 7))                          # all equal, negative
    cases.append((np.asarray([1, -1, 1, -1, 1, -1], np.float32), 3))          # +- pairs
    cases.append((rng.standard_normal(1000).astype(np.float32), 1))           # k = 1
    cases.append((rng.standard_normal(64).astype(np.float32), 64))            # k = n
    cases.append((np.asarray([0.0, -0.0, 1e-40, -1e-40, 0.0], np.float32), 3))  # denormals, signed zeros
    cases.append((rng.standard_normal(3000).astype(np.float32), 30))
    for x, k in cases:
        idx, val, dec = oracle.topk_compress(x, [0, len(x)], [k], _lib=L)
        want = brute_topk(x, k)
        assert idx.tolist() == want, (k, idx[:8], want[:8])
        assert np.array_equal(val.view(np.uint32), x[want].view(np.uint32))
        expect_dec = np.zeros_like(x)
        expect_dec[want] = x[want]
        assert np.array_equal(dec, expect_dec)
        x64 = x.astype(np.float64)
        assert np.sum((x64 - dec) ** 2) <= (1 - k / len(x)) * np.sum(x64 ** 2) + 1e-12
    # segment-wise: flat indices, each segment independent
    x = rng.integers(-5, 6, 150).astype(np.float32)
    off, k = [0, 10, 11, 80, 150], [3, 1, 7, 70]
    idx, val, dec = oracle.topk_compress(x, off, k, _lib=L)
    want = []
    for t in range(4):
        want += [off[t] + j for j in brute_topk(x[off[t]:off[t + 1]], k[t])]
    assert idx.tolist() == want and np.array_equal(val, x[want])


def pin_topk_quantile(L):
    """On Gaussians the 1 % magnitude threshold is the textbook two-sided quantile 2.576 sigma."""
    n = 400_000
    x = np.random.default_rng(17).standard_normal(n).astype(np.float32)
    k = n // 100
    idx, val, _ = oracle.topk_compress(x, [0, n], [k], _lib=L)
    assert len(idx) == k and np.all(np.diff(idx.astype(np.int64)) > 0)
    assert abs(np.min(np.abs(val)) - 2.5758) < 0.03
    mask = np.ones(n, bool)
    mask[idx] = False
    assert np.max(np.abs(x[mask])) <= np.min(np.abs(val))


# ----------------------------------------------------------------------------- random-k

def pin_randk_all_subsets(L):
    """Def. 3 over every k-subset of a small vector, in exact rational arithmetic:
    the mean of C(x) is (k/d) x (Assumption 4) and the mean of ||x - C(x)||^2 is (1 - k/d) ||x||^2
    (Def. 1 holds with equality and delta = k/d)."""
    from itertools import combinations
    x = np.asarray([1.5, -2.25, 0.0, 3.0, -0.125, 7.0, -1.0], np.float32)
    d = len(x)
    xq = [Fraction(float(v)) for v in x]
    for k in (1, 3, 6, 7):
        subsets = list(combinations(range(d), k))
        mean = [Fraction(0)] * d
        err = Fraction(0)
        for S in subsets:
            idx, val, dec = oracle.randk_compress(x, [0, d], [k], np.asarray(S, np.uint32), _lib=L)
            assert idx.tolist() == list(S) and np.array_equal(val, x[list(S)])
            assert all((dec[j] == x[j]) if j in S else (dec[j] == 0.0) for j in range(d))
            for j in range(d):
                mean[j] += Fraction(float(dec[j]))
                err += (xq[j] - Fraction(float(dec[j]))) ** 2
        assert all(mean[j] / len(subsets) == Fraction(k, d) * xq[j] for j in range(d))
        assert err / len(subsets) == (1 - Fraction(k, d)) * sum(v * v for v in xq)


def pin_randk_segments_and_rejects(L):
    """Flat indices, one subset per segment; a subset that leaves its segment, repeats an index or
    is not ascending is refused."""
    x = (np.arange(30, dtype=np.float32) - 11.5)
    off, k = [0, 4, 5, 30], [2, 1, 6]
    S = np.asarray([1, 3, 4, 5, 9, 10, 20, 28, 29], np.uint32)
    idx, val, dec = oracle.randk_compress(x, off, k, S, _lib=L)
    assert idx.tolist() == S.tolist() and np.array_equal(val, x[S.astype(np.int64)])
    want = np.zeros_like(x)
    want[S.astype(np.int64)] = x[S.astype(np.int64)]
    assert np.array_equal(dec, want)
    for bad in ([1, 4, 4, 5, 9, 10, 20, 28, 29],      # first segment reaches into the second
                [1, 3, 4, 5, 9, 9, 20, 28, 29],       # repeated index
                [3, 1, 4, 5, 9, 10, 20, 28, 29],      # descending
                [1, 3, 3, 5, 9, 10, 20, 28, 29]):     # second segment's index outside it
        try:
            oracle.randk_compress(x, off, k, np.asarray(bad, np.uint32), _lib=L)
        except ValueError:
            continue
        raise AssertionError(f"subset {bad} was accepted")


def pin_randk_step_special_cases(L):
    """Whole iterations with random-k: with every index kept it is the identity operator's step, and
    with the subsets that top-k would pick it is the top-k step, bit for bit; in general p + e' = v
    with e' = +0 on the downlink subset, and each worker's update uses its own subset."""
    rng = np.random.default_rng(91)
    off = np.asarray([0, 7, 40, 101], np.int64)
    d, N = 101, 3
    n = np.diff(off)
    G = rng.standard_normal((N, d)).astype(np.float32)
    X0 = rng.standard_normal((N, d)).astype(np.float32)
    e0 = (rng.standard_normal(d) * 0.1).astype(np.float32)
    # (a) k_t = n_t
    full = np.arange(d, dtype=np.uint32)
    Xa, ea, Xb, eb = X0.copy(), e0.copy(), X0.copy(), e0.copy()
    ra = oracle.step(Xa, ea, G, 0.1, off, RANDK, RANDK, k=n, up_sets=np.tile(full, (N, 1)), down_set=full, _lib=L)
    rb = oracle.step(Xb, eb, G, 0.1, off, IDENTITY, IDENTITY, _lib=L)
    assert np.array_equal(Xa, Xb) and np.array_equal(ea, eb) and np.array_equal(ra.v, rb.v)
    # (b) the subsets of top-k
    k = np.asarray([2, 5, 9], np.int64)
    Xa, ea, Xb, eb = X0.copy(), e0.copy(), X0.copy(), e0.copy()
    rb = oracle.step(Xb, eb, G, 0.1, off, TOPK, TOPK, k=k, _lib=L)
    try:
        ra = oracle.step(Xa, ea, G, 0.1, off, RANDK, RANDK, k=k, up_sets=rb.up_idx, down_set=rb.down_idx, _lib=L)
    except RuntimeError as err:  # top-k's own index lists must be valid subsets
        raise AssertionError(str(err))
    assert np.array_equal(Xa, Xb) and np.array_equal(ea, eb)
    assert np.array_equal(ra.up_val, rb.up_val) and np.array_equal(ra.down_val, rb.down_val)
    # (c) arbitrary subsets, the iteration written out with numpy float32
    sets = np.stack([np.concatenate([np.sort(rng.choice(int(n[t]), int(k[t]), replace=False)) + off[t] for t in range(3)])
                     for _ in range(N + 1)]).astype(np.uint32)
    Xa, ea = X0.copy(), e0.copy()
    ra = oracle.step(Xa, ea, G, 0.1, off, RANDK, RANDK, k=k, up_sets=sets[:N], down_set=sets[N], _lib=L)
    P = np.zeros((N, d), np.float32)
    for i in range(N):
        P[i, sets[i].astype(np.int64)] = G[i, sets[i].astype(np.int64)]
    acc = np.zeros(d, np.float32)
    for i in range(N):
        acc = acc + P[i]
    v = e0 + acc / np.float32(N)
    p = np.zeros(d, np.float32)
    p[sets[N].astype(np.int64)] = v[sets[N].astype(np.int64)]
    assert np.array_equal(ra.v, v) and np.array_equal(ea, v - p) and np.all(ea[sets[N].astype(np.int64)] == 0.0)
    assert np.array_equal(ra.down_idx, sets[N]) and np.array_equal(ra.down_val, v[sets[N].astype(np.int64)])
    for i in range(N):
        assert np.array_equal(Xa[i], X0[i] - np.float32(0.1) * ((p - P[i]) + G[i]))


# ----------------------------------------------------------------------------- whole step

def _random_problem(rng, N, off, integer=False):
    d = int(off[-1])
    if integer:
        G = rng.integers(-8, 9, (N, d)).astype(np.float32)
    else:
        G = rng.standard_normal((N, d)).astype(np.float32)
    return G


def pin_error_recursion(L):
    """e_{t+1} = v_t - p_t: decoded message plus new error gives back v
    (exactly for top-k and identity, within one rounding for scaled sign)."""
    rng = np.random.default_rng(21)
    off = np.asarray([0, 5, 37, 100, 164], np.int64)
    d, N = 164, 3
    k = np.asarray([2, 4, 9, 1], np.int64)
    for up, down in ((SIGN, SIGN), (TOPK, TOPK), (IDENTITY, IDENTITY), (SIGN, TOPK), (TOPK, SIGN),
                     (IDENTITY, SIGN), (SIGN, IDENTITY)):
        X = rng.standard_normal((N, d)).astype(np.float32)
        e = rng.standard_normal(d).astype(np.float32) * np.float32(0.1)
        e0 = e.copy()
        G = _random_problem(rng, N, off)
        r = oracle.step(X, e, G, 0.1, off, up, down, k=k, _lib=L)
        # v from its definition, evaluated independently in float32 numpy
        if up == SIGN:
            P = np.stack([decode_sign(r.up_words[i], r.up_scales[i], off) for i in range(N)])
        elif up == TOPK:
            P = np.stack([decode_topk(r.up_idx[i], r.up_val[i], d) for i in range(N)])
        else:
            P = G
        acc = np.zeros(d, np.float32)
        for i in range(N):
            acc = acc + P[i]
        v = e0 + acc / np.float32(N)
        assert np.array_equal(v, r.v), (up, down)
        if down == SIGN:
            p = decode_sign(r.down_words, r.down_scales, off)
            # e' = fl(v - p): off from the exact difference by at most half a unit in its own last place
            assert np.all(np.abs((p.astype(np.float64) + e) - r.v) <= 0.5 * np.spacing(np.abs(e)).astype(np.float64))
        elif down == TOPK:
            p = decode_topk(r.down_idx, r.down_val, d)
            assert np.array_equal(p + e, r.v)
            assert np.all(e[r.down_idx.astype(np.int64)] == 0.0)
        else:
            assert np.all(e == 0.0)


def pin_identity_one_worker_is_sgd(L):
    """Algorithm 1 with C = identity and N = 1 is x <- x - eta g."""
    rng = np.random.default_rng(23)
    d = 257
    X = rng.standard_normal((1, d)).astype(np.float32)
    e = np.zeros(d, np.float32)
    ref = X.copy()
    for step in range(5):
        G = rng.standard_normal((1, d)).astype(np.float32)
        oracle.step(X, e, G, 0.05, [0, 100, d], IDENTITY, IDENTITY, _lib=L)
        ref = ref - np.float32(0.05) * G
        assert np.array_equal(X, ref) and np.all(e == 0.0)


def pin_identical_workers(L):
    """Equal gradients on N = 2^m workers with e = 0: v = p^i, C(v) = v, e' = 0, x <- x - eta g."""
    rng = np.random.default_rng(29)
    d, N = 128, 4
    g = rng.integers(-8, 9, d).astype(np.float32)      # scales are exact binary fractions
    G = np.tile(g, (N, 1))
    X = np.tile(rng.standard_normal(d).astype(np.float32), (N, 1)).copy()
    x0 = X[0].copy()
    e = np.zeros(d, np.float32)
    r = oracle.step(X, e, G, 0.5, [0, 64, 128], SIGN, SIGN, _lib=L)
    assert np.array_equal(r.v, decode_sign(r.up_words[0], r.up_scales[0], [0, 64, 128]))
    assert np.array_equal(r.down_words, r.up_words[0]) and np.array_equal(r.down_scales, r.up_scales[0])
    assert np.all(e == 0.0)
    for i in range(N):
        assert np.array_equal(X[i], x0 - np.float32(0.5) * g)


def pin_lemma3_exact(L):
    """Lemma 3: mean_i x_t^i - (x_0 - eta sum_tau mean_i g_tau^i) = eta e_t.

    Small integers, power-of-two sizes and eta = 1/2 keep every operation exact, so
    the identity has to hold to the last bit over several iterations.
    """
    rng = np.random.default_rng(31)
    for up, down, off, k, N in ((SIGN, SIGN, [0, 4, 8], None, 2),
                                (TOPK, TOPK, [0, 16, 24], [3, 2], 4),
                                (SIGN, TOPK, [0, 4, 8], [1, 2], 2),
                                (IDENTITY, SIGN, [0, 4, 8], None, 2)):
        off = np.asarray(off, np.int64)
        d = int(off[-1])
        x0 = rng.integers(-4, 5, d).astype(np.float32)
        X = np.tile(x0, (N, 1)).copy()
        e = np.zeros(d, np.float32)
        gsum = np.zeros(d, np.float64)
        for step in range(4):
            G = _random_problem(rng, N, off, integer=True)
            oracle.step(X, e, G, 0.5, off, up, down, k=k, _lib=L)
            gsum += G.astype(np.float64).mean(axis=0)
            xbar = X.astype(np.float64).mean(axis=0)
            xhat = x0.astype(np.float64) - 0.5 * gsum
            assert np.array_equal(xbar - xhat, 0.5 * e.astype(np.float64)), (up, down, step)
        assert np.any(e != 0.0)


def pin_lemma3_float(L):
    """Lemma 3 on Gaussian data holds up to binary32 rounding accumulated over the steps."""
    rng = np.random.default_rng(37)
    off = np.asarray([0, 100, 130, 400], np.int64)
    d, N, lr = 400, 5, 0.1
    for up, down, k in ((SIGN, SIGN, None), (TOPK, TOPK, [5, 2, 20])):
        X = np.zeros((N, d), np.float32)
        e = np.zeros(d, np.float32)
        gsum = np.zeros(d, np.float64)
        for step in range(20):
            G = _random_problem(rng, N, off)
            oracle.step(X, e, G, lr, off, up, down, k=k, _lib=L)
            gsum += G.astype(np.float64).mean(axis=0)
        lhs = X.astype(np.float64).mean(axis=0) + lr * gsum
        assert np.max(np.abs(lhs - lr * e.astype(np.float64))) < 2e-5
        assert np.max(np.abs(e)) > 0.1


def pin_golden_averaging(L):
    """Hand-worked model-averaging iteration (tests/golden/averaging_step.txt)."""
    g = read_golden("averaging_step.txt")
    N = int(g["N"][0])
    X = np.asarray([g[f"x0.{i}"] for i in range(N)], np.float32)
    e = np.asarray(g["e0"], np.float32)
    G = np.asarray([g[f"g.{i}"] for i in range(N)], np.float32)
    v, xbar = oracle.average_step(X, e, G, g["lr"][0], _lib=L)
    assert v.tolist() == g["v"] and xbar.tolist() == g["xbar"] and e.tolist() == g["e"]
    for i in range(N):
        assert X[i].tolist() == g[f"x.{i}"], (i, X[i])


def pin_averaging_properties(L):
    """Averaging iteration: the error is cleared, all local models coincide afterwards (exactly on
    dyadic data), the mean model is the plain mean, and Lemma 3 keeps holding across a run that
    mixes compressed iterations with an averaging one every 3rd step."""
    rng = np.random.default_rng(41)
    off = np.asarray([0, 4, 8], np.int64)
    N, d, lr = 2, 8, 0.5
    x0 = rng.integers(-4, 5, d).astype(np.float32)
    X = np.tile(x0, (N, 1)).copy()
    e = np.zeros(d, np.float32)
    gsum = np.zeros(d, np.float64)
    for step in range(6):
        G = rng.integers(-8, 9, (N, d)).astype(np.float32)
        if (step + 1) % 3 == 0:
            xbar_before = X.astype(np.float64).mean(axis=0)
            v, xbar = oracle.average_step(X, e, G, lr, _lib=L)
            assert np.array_equal(xbar.astype(np.float64), xbar_before)
            assert np.all(e == 0.0)
            assert all(np.array_equal(X[i], X[0]) for i in range(N))
        else:
            oracle.step(X, e, G, lr, off, SIGN, SIGN, _lib=L)
            assert not all(np.array_equal(X[i], X[0]) for i in range(N))
        gsum += G.astype(np.float64).mean(axis=0)
        lhs = X.astype(np.float64).mean(axis=0) - (x0.astype(np.float64) - lr * gsum)
        assert np.array_equal(lhs, lr * e.astype(np.float64)), step
    # the plain mean on Gaussian rows, against numpy in higher precision
    Xg = rng.standard_normal((5, 300)).astype(np.float32)
    assert np.max(np.abs(oracle.mean_params(Xg, _lib=L) - Xg.astype(np.float64).mean(axis=0))) < 1e-6


def pin_sumsq_and_delta(L):
    """Squared norms against exact rational arithmetic, and the measured contraction of Def. 1
    computed from them: for the scaled sign delta = d s^2 / ||x||^2 (-> 2/pi on Gaussians), for
    top-k delta = ||C(x)||^2 / ||x||^2 >= k/d."""
    rng = np.random.default_rng(43)
    for n in (1, 3, 64, 1000):
        x = (rng.standard_normal(n) * np.exp(rng.uniform(-5, 5, n))).astype(np.float32)
        exact = sum((Fraction(float(v)) ** 2 for v in x), Fraction(0))
        got = oracle.tree_sumsq(x, _lib=L)
        assert abs(Fraction(got) - exact) <= exact * Fraction(1, 10 ** 14), n
    assert oracle.tree_sumsq(np.asarray([3, -4], np.float32), _lib=L) == 25.0
    x = rng.standard_normal(100_000).astype(np.float32)
    _, s, dec = oracle.sign_compress(x, [0, x.size], _lib=L)
    xx = oracle.tree_sumsq(x, _lib=L)
    delta = x.size * float(s[0]) ** 2 / xx
    resid = oracle.tree_sumsq(x - dec, _lib=L)
    assert abs((1 - resid / xx) - delta) < 1e-6 and abs(delta - 2 / math.pi) < 0.01
    k = 1000
    _, val, dec = oracle.topk_compress(x, [0, x.size], [k], _lib=L)
    delta_k = oracle.tree_sumsq(val, _lib=L) / xx
    assert abs((1 - oracle.tree_sumsq(x - dec, _lib=L) / xx) - delta_k) < 1e-9 and delta_k >= k / x.size


def pin_bf16_widening(L):
    """bfloat16 -> binary32 against values worked out by hand from the format (1 sign bit, 8 exponent
    bits with bias 127, 7 fraction bits): 0x3DCD = 2^-4 (1 + 77/128), 0x4049 = 2 (1 + 73/128),
    0xC2F7 = -64 (1 + 119/128), 0x7F7F = 2^127 (2 - 2^-7), 0x0001 = 2^-126 2^-7 (subnormal)."""
    bits = np.asarray([0x3F80, 0xBF80, 0x0000, 0x8000, 0x3DCD, 0x4049, 0xC2F7, 0x7F7F, 0x0001], np.uint16)
    out = oracle.widen_bf16(bits, _lib=L)
    want = [1.0, -1.0, 0.0, -0.0, 0.10009765625, 3.140625, -123.5, (2.0 - 2.0 ** -7) * 2.0 ** 127, 2.0 ** -133]
    assert [float(v) for v in out] == want
    assert math.copysign(1.0, float(out[3])) == -1.0 and math.copysign(1.0, float(out[2])) == 1.0


def pin_sumsq_tree_shape(L):
    """The squared norm follows the same balanced tree as the L1 norm (the order is part of what the
    CUDA path has to reproduce bit for bit).  Expected values by hand from round-to-nearest-even:
    (2^27)^2 = 2^54 has a unit in the last place of 4, so 2^54 + 1 rounds back, 2^54 + 2 is a tie
    that goes to the even neighbour (2^54; but 2^54 + 6 goes up to 2^54 + 8), sums of small squares are exact."""
    b = float(2 ** 27)
    big = float(2 ** 54)
    t = lambda v: oracle.tree_sumsq(np.asarray(v, np.float32), _lib=L)
    assert t([b, 1, 1, 1, 1, 1, 1, 1]) == big + 4     # ((big+1)+(1+1)) + ((1+1)+(1+1)) = big + 4; a running sum stays at big
    assert t([b, 2, 1, 1]) == big + 8                 # (big+4) + (1+1) = big + 6 -> tie to even; a running sum gives big + 4
    assert t([1, 1, b, 2]) == big + 8                 # (1+1) + (big+4)
    assert t([b, 1, 1]) == big                        # padded to 4: (big+1) + (1+0) = big + 1 -> big
    assert t([1, 1, 1, 1, b, 1, 1, 1, 1]) == big + 4  # padded to 16: (4 + ((big+1)+(1+1))) + (1+0+...) = (big+4) + 1 -> big + 4
    assert t([-3, 4]) == 25.0


# ----------------------------------------------------------------------------- seeded subsets (Def. 3)

def _philox_kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            ctr, key, out = (tuple(int(w, 16) for w in part.split()) for part in line.split("|"))
            rows.append((ctr, key, out))
    assert len(rows) == 3
    return rows


def pin_philox_known_answers(L):
    """The generator against its published known-answer vectors."""
    for ctr, key, out in _philox_kat():
        got = oracle.philox4x32_10(ctr, key, _lib=L)
        assert tuple(int(w) for w in got) == out, (ctr, key, [hex(int(w)) for w in got])


def pin_subset_scores_layout(L):
    """Which counter word, key word and output word go where, from the published vectors alone:
    seed 0, epoch 0, row 0, segment 0 is counter (0,0,0,0) under key (0,0), whose block the first
    vector gives; elements 0..3 take its words in order, shifted right by two."""
    (_, _, out0) = _philox_kat()[0]
    sc = oracle.subset_scores(0, 0, 0, 0, 4, _lib=L)
    assert [int(v) for v in sc] == [w >> 2 for w in out0]
    # the two highest of (6627e8d5, e169c58d, bc57ac4c, 9b00dbd8) are elements 1 and 2; the highest is 1
    assert list(oracle.subset_from_scores(sc, 2, _lib=L)) == [1, 2]
    assert list(oracle.subset_from_scores(sc, 1, _lib=L)) == [1]
    assert list(oracle.subset_from_scores(sc, 3, _lib=L)) == [1, 2, 3]
    # the third vector, read as (block, segment, row, epoch) under seed = k1:k0
    (c, k, out) = _philox_kat()[2]
    seed = (k[1] << 32) | k[0]
    blk = oracle.philox4x32_10(c, k, _lib=L)
    assert tuple(int(w) for w in blk) == out
    # element 4q+m of (segment c1, row c2, epoch c3) has block q = c0: too far out to list a segment
    # of that length, so take q = 1 and check it against the block function itself, word by word,
    # and that every one of the six inputs matters
    base = dict(seed=seed, epoch=c[3], row=c[2], t=c[1])
    sc = oracle.subset_scores(base["seed"], base["epoch"], base["row"], base["t"], 8, _lib=L)
    want = oracle.philox4x32_10((1, c[1], c[2], c[3]), k, _lib=L)
    assert [int(v) for v in sc[4:8]] == [int(w) >> 2 for w in want]
    for name, other in (("seed", seed ^ 1), ("seed", seed ^ (1 << 32)), ("epoch", c[3] ^ 1), ("row", c[2] ^ 1), ("t", c[1] ^ 1)):
        changed = dict(base, **{name: other})
        sc2 = oracle.subset_scores(changed["seed"], changed["epoch"], changed["row"], changed["t"], 8, _lib=L)
        assert not np.array_equal(sc, sc2), name
    # swapping two of the inputs is not the same draw either
    assert not np.array_equal(oracle.subset_scores(5, 1, 2, 3, 8, _lib=L), oracle.subset_scores(5, 2, 1, 3, 8, _lib=L))
    assert not np.array_equal(oracle.subset_scores(5, 1, 2, 3, 8, _lib=L), oracle.subset_scores(5, 1, 3, 2, 8, _lib=L))
    assert not np.array_equal(oracle.subset_scores(5, 1, 2, 3, 8, _lib=L), oracle.subset_scores(5, 3, 2, 1, 8, _lib=L))


def pin_subset_from_scores_is_uniform(L):
    """Ranking by scores: over all orderings of distinct scores every k-subset comes out equally
    often (Def. 3 asks for the uniform distribution over k-subsets), listed ascending; equal
    scores go to the lower index (checked against a plain Python sort over every score vector
    from a three-letter alphabet)."""
    import itertools
    n = 5
    for k in (1, 2, 3, 5):
        counts = {}
        for perm in itertools.permutations(range(10, 10 + n)):
            sub = tuple(int(v) for v in oracle.subset_from_scores(np.asarray(perm, np.uint32) * 1000003, k, _lib=L))
            assert list(sub) == sorted(set(sub)) and len(sub) == k and all(0 <= j < n for j in sub)
            top = tuple(sorted(sorted(range(n), key=lambda j: -perm[j])[:k]))
            assert sub == top
            counts[sub] = counts.get(sub, 0) + 1
        assert len(counts) == math.comb(n, k) and len(set(counts.values())) == 1, (k, counts)
    for scores in itertools.product((0, 7, 9), repeat=4):
        for k in (1, 2, 3, 4):
            want = sorted(sorted(range(4), key=lambda j: (-scores[j], j))[:k])
            got = [int(v) for v in oracle.subset_from_scores(np.asarray(scores, np.uint32), k, _lib=L)]
            assert got == want, (scores, k, got, want)


def pin_subset_draw_layout(L):
    """draw_subsets: row r, segment t holds flat indices of segment t, k_t of them, ascending, equal to
    the ranking of that (row, segment)'s own scores; rows differ; the iteration accepts them."""
    off = np.asarray([0, 5, 6, 40, 173], np.int64)
    k = np.asarray([2, 1, 34, 17], np.int64)
    rows, seed, epoch = 4, 0x1234567890abcdef, 7
    sets = oracle.draw_subsets(seed, epoch, rows, off, k, _lib=L)
    koff = np.concatenate([[0], np.cumsum(k)])
    assert sets.shape == (rows, int(k.sum()))
    for r in range(rows):
        for t in range(4):
            n = int(off[t + 1] - off[t])
            sc = oracle.subset_scores(seed, epoch, r, t, n, _lib=L)
            want = sorted(sorted(range(n), key=lambda j: (-int(sc[j]), j))[:int(k[t])])
            got = [int(v) for v in sets[r, koff[t]:koff[t + 1]]]
            assert got == [int(off[t]) + j for j in want], (r, t)
    assert list(sets[0, koff[2]:koff[3]]) == list(range(6, 40))        # k_t = n_t keeps the whole segment
    assert not np.array_equal(sets[0], sets[1])
    assert not np.array_equal(sets, oracle.draw_subsets(seed, epoch + 1, rows, off, k, _lib=L))
    assert np.array_equal(sets, oracle.draw_subsets(seed, epoch, rows, off, k, _lib=L))
    rng = np.random.default_rng(5)
    N = rows - 1
    G = rng.standard_normal((N, 173)).astype(np.float32)
    X = np.zeros((N, 173), np.float32)
    e = np.zeros(173, np.float32)
    r = oracle.step(X, e, G, 0.1, off, RANDK, RANDK, k=k, up_sets=sets[:N], down_set=sets[N], _lib=L)
    assert np.array_equal(r.up_idx, sets[:N]) and np.array_equal(r.down_idx, sets[N])


def pin_subset_statistics(L):
    """Over many draws: every element is kept with frequency k/n, every pair with k(k-1)/(n(n-1)), and
    E ||C(x) - x||^2 = (1 - k/n) ||x||^2 (Assumption 4 with delta = k/d, the value the paper states for
    random-k), all within five standard deviations of the uniform law."""
    n, k, draws = 24, 6, 6000
    off, karr = np.asarray([0, n], np.int64), np.asarray([k], np.int64)
    single = np.zeros(n)
    pair = np.zeros((n, n))
    rng = np.random.default_rng(11)
    x = rng.standard_normal(n)
    resid = 0.0
    for epoch in range(draws):
        sub = oracle.draw_subsets(99, epoch, 1, off, karr, _lib=L)[0].astype(np.int64)
        single[sub] += 1
        pair[np.ix_(sub, sub)] += 1
        keep = np.zeros(n, bool)
        keep[sub] = True
        resid += float(np.sum(x[~keep] ** 2))
    p1 = k / n
    assert np.all(np.abs(single / draws - p1) < 5 * math.sqrt(p1 * (1 - p1) / draws)), single / draws
    p2 = k * (k - 1) / (n * (n - 1))
    offdiag = pair[~np.eye(n, dtype=bool)] / draws
    assert np.all(np.abs(offdiag - p2) < 5 * math.sqrt(p2 * (1 - p2) / draws)), (offdiag.min(), offdiag.max(), p2)
    want = (1 - k / n) * float(np.sum(x ** 2))
    assert abs(resid / draws - want) < 0.03 * want, (resid / draws, want)
    # different rows and different seeds are different streams with the same law
    a = oracle.draw_subsets(1, 0, 64, np.asarray([0, 4096], np.int64), np.asarray([41], np.int64), _lib=L)
    assert len({tuple(r) for r in a}) == 64
    flat = np.bincount(a.ravel(), minlength=4096)
    assert flat.max() <= 6      # 64 * 41 draws over 4096 positions: no position favoured


ALL_PINS = [
    pin_golden_sign, pin_golden_blockwise, pin_golden_topk,
    pin_scale_is_exact_mean, pin_tree_shape, pin_sign_bits_bruteforce, pin_sign_contraction,
    pin_blockwise_reduces_to_sign, pin_topk_bruteforce, pin_topk_quantile,
    pin_error_recursion, pin_identity_one_worker_is_sgd, pin_identical_workers,
    pin_lemma3_exact, pin_lemma3_float, pin_bf16_widening, pin_sumsq_tree_shape, pin_golden_averaging, pin_averaging_properties, pin_sumsq_and_delta,
    pin_randk_all_subsets, pin_randk_segments_and_rejects, pin_randk_step_special_cases,
    pin_philox_known_answers, pin_subset_scores_layout, pin_subset_from_scores_is_uniform, pin_subset_draw_layout,
    pin_subset_statistics,
]
