"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test checks the oracle against something other than itself: values the
paper prints, closed forms, exact enumeration, library routines on special
cases, exact rational arithmetic.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- number system

def test_worked_examples(oracle):
    """Sec. 3.2 prints w = 3 -> (e = 1, p = 0.5); the rest follow from Eq. 5-7 by hand."""
    for line in open(os.path.join(GOLDEN, "worked_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w, s, e, p = line.split()
        cls, s_o, e_o, m_o = oracle.decode(float(w))
        assert cls == 1
        assert (s_o, e_o) == (int(s), int(e))
        assert m_o == int(float(p) * 2 ** 23)


def test_decode_matches_eq_5_7_in_exact_arithmetic(oracle):
    """e = floor(log2 |w|), p = |w| / 2^e - 1, checked with exact rationals."""
    rng = np.random.default_rng(1)
    ws = np.concatenate([rng.normal(0, 1, 200), rng.normal(0, 1e-3, 100), rng.normal(0, 300, 100)])
    for w in ws.astype(np.float32):
        cls, s, e, m = oracle.decode(w)
        a = abs(Fraction(float(w)))
        assert cls == 1 and s == (1 if w < 0 else 0)
        assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
        assert a / Fraction(2) ** e - 1 == Fraction(m, 2 ** 23)


def test_zero_subnormal_nonfinite_classes(oracle):
    assert oracle.decode(0.0)[0] == 0
    assert oracle.decode(-0.0)[0] == 0
    assert oracle.decode(1e-45)[0] == 0
    assert oracle.decode(np.inf)[0] == 2
    assert oracle.decode(np.nan)[0] == 2
    w = np.array([[1.0, np.inf]], dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.sample_level(w, 0, 0, 2)


# ------------------------------------------------------------------------ Philox

def test_philox_known_answers(oracle):
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(t, 16) for t in line.split()]
        assert list(oracle.philox4x32_10(v[:4], v[4:6])) == v[6:]
        n += 1
    assert n >= 2


def test_draw_bit_uses_the_documented_counter_layout(oracle):
    """Draw j of weight i in layer L under seed S is word j%4 of
    Philox(counter=(j/4, L, lo(i), hi(i)), key=(lo(S), hi(S))) compared with p * 2^32."""
    rng = np.random.default_rng(2)
    for _ in range(200):
        seed = int(rng.integers(0, 2 ** 63)) * 2 + int(rng.integers(0, 2))
        layer = int(rng.integers(0, 2 ** 32))
        idx = int(rng.integers(0, 2 ** 40))
        j = int(rng.integers(0, 64))
        m = int(rng.integers(0, 2 ** 23))
        r = oracle.philox4x32_10([j >> 2, layer, idx & 0xFFFFFFFF, idx >> 32],
                                 [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.draw_bit(seed, layer, idx, j, m) == int(int(r[j & 3]) < (m << 9))


def test_draw_bits_are_balanced_and_uncorrelated(oracle):
    """Bit frequency and lag-1 serial test of the Bernoulli stream at p = 1/2 and p = 1/4."""
    for m, p in ((1 << 22, 0.5), (1 << 21, 0.25)):
        bits = np.array([oracle.draw_bit(5, 3, i, j, m) for i in range(600) for j in range(32)])
        n = bits.size
        z = (bits.sum() - n * p) / np.sqrt(n * p * (1 - p))
        assert abs(z) < 4.5
        pairs = bits[:-1] * bits[1:]
        z2 = (pairs.sum() - (n - 1) * p * p) / np.sqrt((n - 1) * p * p * (1 - p * p))
        assert abs(z2) < 4.5


# ------------------------------------------------------ sampled weights (Eq. 4, 8)

def _real_weight(W, e_base, log2k):
    """Sampled real value W_k * 2^e_base / k as exact float64."""
    return W.astype(np.float64) * np.exp2(e_base.astype(np.float64))[:, None] / (1 << log2k)


def test_powers_of_two_are_reproduced_exactly(oracle):
    """p = 0 (filled markers of Fig. 1b): every draw picks the lower shift, so the layer
    equals an ordinary convolution, here torch.conv2d in float64 (exact at these sizes)."""
    import torch

    rng = np.random.default_rng(3)
    w = (np.exp2(rng.integers(-9, 3, size=(6, 4, 3, 3))) * rng.choice([-1.0, 1.0], size=(6, 4, 3, 3))
         ).astype(np.float32)
    x = rng.integers(0, 16, size=(2, 4, 9, 7), dtype=np.uint8)
    for seed, log2k in ((0, 0), (11, 3), (12, 6)):
        W, eb, c = oracle.sample_level(w, seed, 1, log2k)
        assert not c.any()
        g = oracle.geom(x.shape, oracle.NCHW, oracle.U8, w.shape, 1, 1, 1)
        acc = oracle.conv_acc(x, g, {log2k: W}, uniform_log2k=log2k)
        got = acc.astype(np.float64) * np.exp2(float(eb[0])) / (1 << log2k)
        ref = torch.nn.functional.conv2d(torch.from_numpy(x.astype(np.float64)),
                                         torch.from_numpy(w.astype(np.float64)), padding=1).numpy()
        assert np.array_equal(got, ref)


def test_variance_closed_form_and_one_over_k(oracle):
    """Var(w_bar) = -2^(2e+1) + 3 * 2^e |w| - w^2 (Fig. 1c), divided by k for k draws (Eq. 10);
    at |w| = 4/3 * 2^e it meets the bound w^2 / (8k)."""
    n = 40000
    for wval in (3.0, 4.0 / 3.0, -0.8125, 0.3):
        w = np.full((1, n), wval, dtype=np.float32)
        wf = float(np.float32(wval))
        e = int(np.floor(np.log2(abs(wf))))
        var1 = -2.0 ** (2 * e + 1) + 3 * 2.0 ** e * abs(wf) - wf * wf
        prev = None
        for log2k in (0, 1, 2, 3, 4):
            k = 1 << log2k
            W, eb, _ = oracle.sample_level(w, 77, 0, log2k)
            r = _real_weight(W, eb, log2k)[0]
            assert abs(r.mean() - wf) < 5 * np.sqrt(var1 / k / n) + 1e-12      # unbiased (Sec. 3.1)
            emp = r.var()
            # variance of a sample variance of n iid draws ~ 2 var^2 / n  (loose 6-sigma gate)
            assert abs(emp - var1 / k) < 6 * (var1 / k) * np.sqrt(2.0 / n) + 0.02 * var1 / k
            assert emp <= wf * wf / (8 * k) * 1.05                           # Eq. 10
            assert np.sqrt(emp) / abs(r.mean()) <= 1 / np.sqrt(8 * k) * 1.03  # Eq. 11
            if prev is not None:
                assert 0.42 < emp / prev < 0.58
            prev = emp
    assert abs((-2.0 ** 1 + 3 * (4.0 / 3.0) - (4.0 / 3.0) ** 2) - (4.0 / 3.0) ** 2 / 8) < 1e-12


def test_counts_are_binomial(oracle):
    """c_k ~ Binomial(k, p) (Eq. 8 and the supplement's Eq. 12): chi-square over many weights."""
    n = 30000
    for wval, log2k in ((1.25, 2), (1.5, 3), (1.9, 4), (-1.0625, 4)):
        k = 1 << log2k
        p = abs(wval) - 1.0
        w = np.full((1, n), wval, dtype=np.float32)
        _, _, c = oracle.sample_level(w, 123, 9, log2k)
        obs = np.bincount(c[0].astype(np.int64), minlength=k + 1).astype(np.float64)
        exp = stats.binom.pmf(np.arange(k + 1), k, p) * n
        keep = exp > 5
        obs_k = np.append(obs[keep], obs[~keep].sum())
        exp_k = np.append(exp[keep], exp[~keep].sum())
        if exp_k[-1] == 0:
            obs_k, exp_k = obs_k[:-1], exp_k[:-1]
        chi2 = ((obs_k - exp_k) ** 2 / exp_k).sum()
        assert chi2 < stats.chi2.ppf(1 - 1e-5, len(exp_k) - 1)


def test_progressive_levels_share_draws(oracle):
    """Level k uses draws 0..k-1 of one stream: counts are prefix sums of the same bits."""
    rng = np.random.default_rng(5)
    w = rng.normal(0, 0.3, size=(3, 50)).astype(np.float32)
    counts = {}
    for log2k in range(0, 7):
        _, _, c = oracle.sample_level(w, 99, 4, log2k)
        counts[log2k] = c.astype(np.int64)
    for o in range(3):
        for i in range(50):
            cls, s, e, m = oracle.decode(w[o, i])
            bits = [oracle.draw_bit(99, 4, o * 50 + i, j, m) for j in range(64)]
            for log2k in range(0, 7):
                expect = sum(bits[: 1 << log2k])
                # weights flushed by the window carry no draws
                if e < _ebase_layer(oracle, w):
                    expect = 0
                assert counts[log2k][o, i] == expect
    for log2k in range(0, 6):
        assert np.all(counts[log2k + 1] >= counts[log2k])
        assert np.all(counts[log2k + 1] - counts[log2k] <= (1 << log2k))


def _ebase_layer(oracle, w, exp_bits=4):
    es = [oracle.decode(v)[2] for v in w.ravel() if oracle.decode(v)[0] == 1]
    return max(es) - (2 ** exp_bits - 1)


def test_window_flushes_small_weights_and_normalises(oracle):
    w = np.array([[1.0, 2.0 ** -15, 2.0 ** -16, 1.5 * 2.0 ** -20, 0.0],
                  [2.0 ** -3, 2.0 ** -18, 2.0 ** -19, -2.0 ** -4, 0.0]], dtype=np.float32)
    W, eb, _ = oracle.sample_level(w, 0, 0, 0, exp_bits=4, norm=0)
    assert list(eb) == [-15, -15]
    assert list(W[0]) == [2 ** 15, 1, 0, 0, 0]
    assert list(W[1]) == [2 ** 12, 0, 0, -(2 ** 11), 0]
    W, eb, _ = oracle.sample_level(w, 0, 0, 0, exp_bits=4, norm=1)
    assert list(eb) == [-15, -18]
    assert list(W[1]) == [2 ** 15, 1, 0, -(2 ** 14), 0]
    W, eb, _ = oracle.sample_level(w, 0, 0, 1, exp_bits=2, norm=0)
    assert list(eb) == [-3, -3]
    assert list(W[0]) == [2 * 8, 0, 0, 0, 0]
    assert W[1][0] == 2 and W[1][3] == 0      # 2^-3 sits on the floor, 2^-4 is flushed
    Wz, ebz, _ = oracle.sample_level(np.zeros((2, 3), np.float32), 0, 0, 2)
    assert not Wz.any() and list(ebz) == [0, 0]


# ----------------------------------------------- brute force on tiny layers (Eq. 9)

def _shift_form(x, s, e, bits):
    """Eq. 9 before the final shift: s * sum_j x << (e + b_j), for e >= 0, in Python ints."""
    return (-1 if s else 1) * sum(int(x) << (e + b) for b in bits)


def test_shift_form_equals_integer_product(oracle):
    rng = np.random.default_rng(6)
    w = np.array([[3.0, -5.0, 1.0, 6.5, -1.75, 2.25]], dtype=np.float32)   # all e >= 0
    x = rng.integers(0, 16, size=(1, 6, 1, 1), dtype=np.uint8)
    for log2k in (0, 1, 2, 3):
        k = 1 << log2k
        W, eb, c = oracle.sample_level(w.reshape(1, 6, 1, 1), 31, 2, log2k, exp_bits=4)
        g = oracle.geom(x.shape, oracle.NCHW, oracle.U8, (1, 6, 1, 1), 1, 1, 0)
        acc = int(oracle.conv_acc(x, g, {log2k: W}, uniform_log2k=log2k)[0, 0, 0, 0])
        total = 0
        for i in range(6):
            _, s, e, m = oracle.decode(w[0, i])
            bits = [oracle.draw_bit(31, 2, i, j, m) for j in range(k)]
            total += _shift_form(x[0, i, 0, 0], s, e, bits)
        # the oracle keeps the accumulator in units of 2^e_base
        assert Fraction(acc) * Fraction(2) ** int(eb[0]) == total


def test_brute_force_enumeration_of_all_draw_outcomes(oracle):
    """d = 2 weights, k = 2 draws: all 16 bit patterns.  (i) with injected bits the oracle's
    accumulator equals Eq. 9 evaluated directly; (ii) over many seeds the accumulator follows
    the exact distribution those patterns and their probabilities define."""
    w = np.array([[[[1.25]], [[-3.0]]]], dtype=np.float32)          # p = 0.25, 0.5
    x = np.array([[[[7]], [[5]]]], dtype=np.uint8)
    g = oracle.geom(x.shape, oracle.NCHW, oracle.U8, w.shape, 1, 1, 0)
    ps = [0.25, 0.5]
    dec = [oracle.decode(v) for v in w.ravel()]
    exact = {}
    for pattern in itertools.product([0, 1], repeat=4):
        b = [pattern[0:2], pattern[2:4]]
        val = sum(_shift_form(x.ravel()[i], dec[i][1], dec[i][2], b[i]) for i in range(2))
        prob = 1.0
        for i in range(2):
            for bit in b[i]:
                prob *= ps[i] if bit else 1 - ps[i]
        counts = np.array([sum(b[0]), sum(b[1])], dtype=np.uint32).reshape(w.shape)
        W, eb, _ = oracle.sample_level(w, 0, 0, 1, counts_in=counts)
        acc = int(oracle.conv_acc(x, g, {1: W}, uniform_log2k=1)[0, 0, 0, 0])
        assert Fraction(acc) * Fraction(2) ** int(eb[0]) == val
        exact[val] = exact.get(val, 0.0) + prob
    n = 20000
    hist = {}
    for seed in range(n):
        W, eb, _ = oracle.sample_level(w, seed, 0, 1)
        acc = int(oracle.conv_acc(x, g, {1: W}, uniform_log2k=1)[0, 0, 0, 0])
        val = int(Fraction(acc) * Fraction(2) ** int(eb[0]))
        hist[val] = hist.get(val, 0) + 1
    assert set(hist) <= set(exact)
    keys = sorted(exact)
    obs = np.array([hist.get(v, 0) for v in keys], dtype=np.float64)
    exp = np.array([exact[v] for v in keys]) * n
    chi2 = ((obs - exp) ** 2 / exp).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-5, len(keys) - 1)


# -------------------------------------------------- the layer as a whole (Eq. 1)

def test_unbiased_and_convergent_layer(oracle):
    """Mean over seeds approaches sum x_i w_i within 5 sigma of the bound Var <= w^2 / (8k)
    plus the mass flushed by the exponent window; psb64 alone is already within that bound."""
    rng = np.random.default_rng(8)
    d, O, S = 48, 5, 300
    w = rng.normal(0, 0.2, size=(O, d, 1, 1)).astype(np.float32)
    x = rng.integers(0, 16, size=(1, d, 1, 1), dtype=np.uint8)
    g = oracle.geom(x.shape, oracle.NCHW, oracle.U8, w.shape, 1, 1, 0)
    ref = (w.reshape(O, d).astype(np.float64) @ x.reshape(d).astype(np.float64))
    xs = x.reshape(d).astype(np.float64)
    for log2k in (0, 3, 6):
        k = 1 << log2k
        ys = np.zeros((S, O))
        for s in range(S):
            W, eb, _ = oracle.sample_level(w, 1000 + s, 0, log2k)
            acc = oracle.conv_acc(x, g, {log2k: W}, uniform_log2k=log2k).reshape(O)
            ys[s] = acc.astype(np.float64) * np.exp2(eb.astype(np.float64)) / k
        flushed = np.zeros(O)
        sig = np.zeros(O)
        for o in range(O):
            wo = w[o].reshape(d).astype(np.float64)
            small = np.abs(wo) < 2.0 ** float(eb[o])
            flushed[o] = np.abs(wo[small] * xs[small]).sum()
            sig[o] = np.sqrt((xs ** 2 * wo ** 2).sum() / (8 * k))
        assert np.all(np.abs(ys.mean(0) - ref) <= 5 * sig / np.sqrt(S) + flushed + 1e-9)
        assert np.all(np.abs(ys[0] - ref) <= 5 * sig + flushed + 1e-9)


def test_conv_indexing_against_library_convolution(oracle):
    """Strides, padding, groups, both layouts, both input types: exact integer filters pushed
    through the oracle's contraction equal torch.conv2d in float64."""
    import torch

    rng = np.random.default_rng(9)
    cases = [  # N, C, H, W, O, KH, KW, groups, stride, pad
        (2, 6, 9, 8, 4, 3, 3, 1, 1, 1), (1, 6, 11, 7, 6, 3, 3, 2, 2, 1), (2, 8, 7, 7, 8, 3, 3, 8, 2, 1),
        (1, 3, 12, 12, 5, 7, 7, 1, 2, 3), (2, 5, 6, 6, 7, 1, 1, 1, 2, 0), (3, 16, 1, 1, 10, 1, 1, 1, 1, 0),
        (1, 4, 6, 9, 4, 3, 1, 1, 1, 0), (1, 4, 8, 8, 4, 3, 3, 4, 1, 1),
    ]
    for (N, Cc, H, W, O, KH, KW, groups, stride, pad) in cases:
        for dtype, lo, hi in ((np.uint8, 0, 256), (np.int8, -128, 128)):
            x = rng.integers(lo, hi, size=(N, Cc, H, W)).astype(dtype)
            Wi = rng.integers(-2 ** 20, 2 ** 20, size=(O, Cc // groups, KH, KW)).astype(np.int64)
            ref = torch.nn.functional.conv2d(torch.from_numpy(x.astype(np.float64)),
                                             torch.from_numpy(Wi.astype(np.float64)), None, stride, pad,
                                             1, groups).numpy().astype(np.int64)
            dt = oracle.U8 if dtype == np.uint8 else oracle.S8
            g = oracle.geom(x.shape, oracle.NCHW, dt, Wi.shape, groups, stride, pad)
            assert np.array_equal(oracle.conv_acc(x, g, {2: Wi}, uniform_log2k=2), ref)
            xh = np.ascontiguousarray(x.transpose(0, 2, 3, 1))
            gh = oracle.geom(xh.shape, oracle.NHWC, dt, Wi.shape, groups, stride, pad)
            acc_h = oracle.conv_acc(xh, gh, {2: Wi}, uniform_log2k=2)
            assert np.array_equal(acc_h, ref.transpose(0, 2, 3, 1))
            pts = np.stack([rng.integers(0, N, 20), rng.integers(0, O, 20),
                            rng.integers(0, ref.shape[2], 20), rng.integers(0, ref.shape[3], 20)], 1)
            got = oracle.conv_acc_points(xh, gh, {2: Wi}, pts, uniform_log2k=2)
            assert np.array_equal(got, ref[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]])


def test_per_location_draw_counts_select_the_level(oracle):
    """A location with map value l uses the level-l filter; levels differ only through the map."""
    rng = np.random.default_rng(10)
    x = rng.integers(0, 16, size=(2, 5, 6, 4), dtype=np.uint8)           # NHWC
    Ws = {l: rng.integers(-999, 999, size=(3, 4, 3, 3)).astype(np.int64) for l in (0, 2, 4)}
    g = oracle.geom(x.shape, oracle.NHWC, oracle.U8, (3, 4, 3, 3), 1, 1, 1)
    kmap = rng.choice([0, 2, 4], size=(2, 5, 6)).astype(np.uint8)
    acc = oracle.conv_acc(x, g, Ws, kmap=kmap)
    for l in (0, 2, 4):
        full = oracle.conv_acc(x, g, {l: Ws[l]}, uniform_log2k=l)
        assert np.array_equal(acc[kmap == l], full[kmap == l])
    with pytest.raises(ValueError):
        oracle.conv_acc(x, g, {0: Ws[0]}, kmap=kmap)


# ---------------------------------------------------------------------- epilogue

def _round_to_f32(fr):
    """Nearest binary32 to an exact rational, ties to even (normal range only)."""
    if fr == 0:
        return np.float32(0.0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = 0
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    scaled = a * 2 ** 23
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return np.float32(sign * float(Fraction(n, 2 ** 23) * Fraction(2) ** e))


def test_dequant_is_one_correctly_rounded_fma(oracle):
    """y = round(round_f32(acc) * scale * 2^(e_base - log2k) + bias) with a single rounding of
    the sum, checked in exact rational arithmetic; includes accumulators beyond 2^24 and 2^53."""
    rng = np.random.default_rng(11)
    accs = [0, 1, -1, 2 ** 24 + 1, -(2 ** 24 + 3), 2 ** 40 + 12345, 3 * 2 ** 52 + 1, 2 ** 53 + 1,
            -(2 ** 61 + 2 ** 37 + 1)] + [int(v) for v in rng.integers(-2 ** 45, 2 ** 45, 300)]
    for acc in accs:
        scale = np.float32(rng.uniform(0.5, 1.5) * 2.0 ** int(rng.integers(-8, 3)))
        bias = np.float32(rng.normal(0, 1.0))
        e_base = int(rng.integers(-24, -4))
        log2k = int(rng.integers(0, 7))
        a32 = _round_to_f32(Fraction(acc))
        exact = Fraction(float(a32)) * Fraction(float(scale)) * Fraction(2) ** (e_base - log2k) \
            + Fraction(float(bias))
        want = _round_to_f32(exact)
        got = np.float32(oracle.dequant_one(acc, scale, e_base, log2k, bias))
        assert got == want, (acc, scale, bias, e_base, log2k)
        assert np.float32(oracle.dequant_one(acc, scale, e_base, log2k, bias, relu=True)) == max(want, np.float32(0))
        rq, rs = int(rng.integers(-128, 128)), np.float32(rng.uniform(0.01, 0.2))
        want_r = _round_to_f32(Fraction(float(want)) + Fraction(rq) * Fraction(float(rs)))
        assert np.float32(oracle.dequant_one(acc, scale, e_base, log2k, bias, res_q=rq, res_scale=rs)) == want_r


def test_requant_rounds_half_to_even_and_saturates(oracle):
    one = np.float32(1.0)
    assert [oracle.requant_one(v, one, 0, 255) for v in (0.5, 1.5, 2.5, 3.5, 254.5, 255.5, 1e9, -0.5, -3.0)] \
        == [0, 2, 2, 4, 254, 255, 255, 0, 0]
    assert [oracle.requant_one(v, one, -128, 127) for v in (-0.5, -1.5, -2.5, -128.5, -1e12, 127.5)] \
        == [0, -2, -2, -128, -128, 127]
    assert oracle.requant_one(np.float32(3.0), np.float32(0.25), 0, 15) == 1        # 0.75 -> 1
    assert oracle.requant_one(np.float32(10.0), np.float32(0.25), 0, 15) == 2       # 2.5 -> 2
    rng = np.random.default_rng(12)
    for _ in range(300):
        y, inv = np.float32(rng.normal(0, 20)), np.float32(rng.uniform(0.1, 3))
        t = _round_to_f32(Fraction(float(y)) * Fraction(float(inv)))
        fr = Fraction(float(t))
        n = fr.numerator // fr.denominator
        rem = fr - n
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
            n += 1
        assert oracle.requant_one(y, inv, -128, 127) == min(max(n, -128), 127)


def test_epilogue_over_a_tensor_matches_the_scalar_rule(oracle):
    rng = np.random.default_rng(13)
    for layout in (oracle.NCHW, oracle.NHWC):
        xs = (2, 3, 4, 5) if layout == oracle.NCHW else (2, 4, 5, 3)
        g = oracle.geom(xs, layout, oracle.U8, (6, 3, 1, 1), 1, 1, 0)
        shp = oracle.out_shape(g)
        acc = rng.integers(-2 ** 30, 2 ** 30, size=shp).astype(np.int64)
        scale = rng.uniform(0.5, 1.5, 6).astype(np.float32)
        bias = rng.normal(0, 1, 6).astype(np.float32)
        eb = rng.integers(-30, -20, 6).astype(np.int32)
        res = rng.integers(-128, 128, size=shp).astype(np.int8)
        kmap = rng.integers(0, 5, size=(2, 4, 5)).astype(np.uint8)
        y, q = oracle.epilogue(acc, g, scale, bias, eb, True, np.float32(0.7), 0, 15, residual=res,
                               residual_scale=np.float32(0.05), kmap=kmap)
        for _ in range(60):
            n, o, oy, ox = (int(rng.integers(0, m)) for m in (2, 6, 4, 5))
            idx = (n, o, oy, ox) if layout == oracle.NCHW else (n, oy, ox, o)
            want = oracle.dequant_one(acc[idx], scale[o], eb[o], kmap[n, oy, ox], bias[o],
                                      res_q=res[idx], res_scale=np.float32(0.05), relu=True)
            assert y[idx] == np.float32(want)
            assert q[idx] == oracle.requant_one(want, np.float32(0.7), 0, 15)


# ----------------------------------------------------------------------- pooling

def test_pooling_against_library_routines(oracle):
    import torch

    rng = np.random.default_rng(14)
    x = rng.integers(0, 256, size=(2, 5, 9, 11), dtype=np.uint8)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(x.astype(np.float32)), 3, 2, 1).numpy()
    assert np.array_equal(oracle.maxpool_u8(x, oracle.NCHW, 3, 2, 1), ref.astype(np.uint8))
    xh = np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    assert np.array_equal(oracle.maxpool_u8(xh, oracle.NHWC, 3, 2, 1), ref.astype(np.uint8).transpose(0, 2, 3, 1))
    mul = np.float32(0.013)
    got = oracle.global_avgpool_u8(xh, oracle.NHWC, mul, 0, 255)
    sums = x.astype(np.int64).sum(axis=(2, 3))
    for n in range(2):
        for c in range(5):
            assert got[n, c] == oracle.requant_one(np.float32(sums[n, c]), mul, 0, 255)
    assert np.array_equal(got, oracle.global_avgpool_u8(x, oracle.NCHW, mul, 0, 255))
