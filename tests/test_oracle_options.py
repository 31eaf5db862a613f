"""Pins of the oracle's optional readings: the Bernoulli gate at the floor of the exponent window
(Sec. 3.1, "Stochastic multiplication", Eq. 2-3) and probabilities on a grid of 2^b points with a
b-bit comparator and packed draws (Sec. 4.4; supplement, "Stochastic multiplier").

Checked against exact rationals, closed-form moments, chi-square tests, brute-force enumeration and
the Philox output recomputed word by word.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats


# ------------------------------------------------------------------ the gate below the window

def test_gate_probability_is_the_weight_over_the_window_floor(oracle):
    """Below the window a weight w becomes s 2^e_base B_q with q = |w| / 2^e_base (Eq. 2: Pr[B_w = 1] = w):
    thr / 2^32 equals q exactly while q 2^32 is an integer, and is its floor otherwise."""
    rng = np.random.default_rng(2)
    e_base = -6
    for dist in list(range(1, 12)) + [20, 31, 33, 41, 45]:
        for w in (rng.uniform(1.0, 2.0, 6) * 2.0 ** (e_base - dist)).astype(np.float32):
            live, base, sh, thr = oracle.classify(w, e_base, 0, 1)
            q = Fraction(float(w)) / Fraction(2) ** e_base
            assert 0 < q < 1
            exact = q * 2 ** 32
            assert thr == int(exact)                       # floor
            if dist <= 9:
                assert Fraction(thr) == exact              # exact
            assert (live, base, sh) == ((1, 0, 0) if thr else (0, 0, 0))
            assert oracle.classify(-w, e_base, 0, 1) == (live, base, sh, thr)
            assert oracle.classify(w, e_base, 0, 0) == (0, 0, 0, 0)     # default: flushed


def test_gate_is_unbiased_with_the_bernoulli_variance(oracle):
    """E[W_k 2^e_base / k] = w and Var = 2^(2 e_base) q (1 - q) / k <= 2^e_base |w| / k (Eq. 3 scaled)."""
    rng = np.random.default_rng(3)
    big = np.float32(1.0)                                    # fixes the window: e_max = 0
    small = (rng.uniform(0.05, 0.95, 40) * rng.choice([-1, 1], 40) * 2.0 ** -7).astype(np.float32)
    w = np.concatenate([[big], small])[None, :]
    for log2k in (0, 2, 4):
        k = 1 << log2k
        S = 3000
        vals = np.zeros((S, w.size))
        for seed in range(S):
            W, eb, c, cls = oracle.sample_level_ex(w, seed, 1, log2k, exp_bits=3, underflow=1)
            assert eb[0] == -7 and cls[0, 0] == 1 and (cls[0, 1:] == 2).all()
            assert (np.abs(W[0, 1:]) == c[0, 1:]).all() and (c[0, 1:] <= k).all()
            vals[seed] = W[0] * 2.0 ** float(eb[0]) / k
        q = np.abs(small.astype(np.float64)) / 2.0 ** -7
        var = (2.0 ** -7) ** 2 * q * (1 - q) / k
        assert np.all(np.abs(vals[:, 1:].mean(0) - small) <= 5 * np.sqrt(var / S))
        emp = vals[:, 1:].var(0)
        assert np.all(np.abs(emp - var) <= 0.2 * var + 1e-12)
        assert np.all(var <= 2.0 ** -7 * np.abs(small) / k)


def test_gate_counts_are_binomial(oracle):
    q = 0.3125
    w = np.full((1, 4001), np.float32(q * 2.0 ** -7), dtype=np.float32)
    w[0, 0] = 1.0
    for log2k in (2, 4):
        k = 1 << log2k
        _, _, c, _ = oracle.sample_level_ex(w, 77, 3, log2k, exp_bits=3, underflow=1)
        obs = np.bincount(c[0, 1:], minlength=k + 1)
        exp = stats.binom.pmf(np.arange(k + 1), k, q) * 4000
        keep = exp > 5
        chi = ((obs[keep] - exp[keep]) ** 2 / exp[keep]).sum() + (obs[~keep].sum() - exp[~keep].sum()) ** 2 / max(exp[~keep].sum(), 1e-9)
        assert chi < stats.chi2.ppf(0.999, keep.sum())


def test_enumeration_of_a_layer_with_one_weight_in_the_window_and_one_below(oracle):
    """Two weights, two draws: all 16 bit patterns.  W = s (base k + c) 2^sh with base 1 inside the window and 0
    below; the accumulator of x = (3, 5) follows; the sampled distribution matches the product of binomials."""
    w = np.array([[0.75, -0.4 * 2.0 ** -4]], dtype=np.float32)      # e_max = -1, exp_bits 2: e_base = -4
    x = np.array([3, 5])
    p0, q1 = 0.5, 0.4 * 2.0 ** -4 / 2.0 ** -4
    dist = {}
    for bits in itertools.product([0, 1], repeat=4):
        c = np.array([[bits[0] + bits[1], bits[2] + bits[3]]], dtype=np.uint32)
        W, eb, _, cls = oracle.sample_level_ex(w, 0, 0, 1, exp_bits=2, underflow=1, counts_in=c)
        assert eb[0] == -4 and tuple(cls[0]) == (1, 2)
        assert W[0, 0] == (2 + c[0, 0]) * 2 ** 3 and W[0, 1] == -int(c[0, 1])
        acc = int((x * W[0]).sum())
        pr = np.prod([p0 if b else 1 - p0 for b in bits[:2]]) * np.prod([q1 if b else 1 - q1 for b in bits[2:]])
        dist[acc] = dist.get(acc, 0.0) + pr
    mean = sum(a * pr for a, pr in dist.items()) * 2.0 ** -4 / 2
    assert abs(mean - float((x * w[0].astype(np.float64)).sum())) < 1e-6          # unbiased, both kinds of weight
    S = 20000
    hist = {}
    for seed in range(S):
        W = oracle.sample_level_ex(w, seed, 0, 1, exp_bits=2, underflow=1)[0]
        a = int((x * W[0]).sum())
        hist[a] = hist.get(a, 0) + 1
    assert set(hist) <= set(dist)
    keys = sorted(dist)
    obs = np.array([hist.get(a, 0) for a in keys], float)
    exp = np.array([dist[a] for a in keys]) * S
    assert ((obs - exp) ** 2 / exp).sum() < stats.chi2.ppf(0.999, len(keys) - 1)


def test_layer_with_a_narrow_window_is_unbiased_without_any_flush_term(oracle):
    """With the gate, the mean over seeds of a whole layer's output converges to the float product although
    most weights lie below a window of only four octaves (no slack term for flushed weights)."""
    rng = np.random.default_rng(5)
    O, D, S, log2k = 6, 300, 1500, 2
    w = rng.normal(0, 0.05, size=(O, D)).astype(np.float32)
    x = rng.integers(0, 16, size=D).astype(np.float64)
    k = 1 << log2k
    outs = np.zeros((S, O))
    for seed in range(S):
        W, eb, _, cls = oracle.sample_level_ex(w, seed, 2, log2k, exp_bits=2, underflow=1)
        outs[seed] = (W * x).sum(1) * 2.0 ** eb.astype(np.float64) / k
    assert (cls == 2).mean() > 0.2
    ref = (w.astype(np.float64) * x).sum(1)
    # per-weight variance: inside the window Fig. 1c's closed form, below it the Bernoulli one
    W, eb, _, cls = oracle.sample_level_ex(w, 0, 2, log2k, exp_bits=2, underflow=1)
    a = np.abs(w.astype(np.float64))
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    var_in = (-2.0 ** (2 * e + 1) + 3 * 2.0 ** e * a - a * a) / k
    fl = 2.0 ** eb.astype(np.float64)[:, None]
    var_gate = fl * fl * (a / fl) * (1 - a / fl) / k
    var = np.where(cls == 1, var_in, np.where(cls == 2, var_gate, 0.0))
    sigma = np.sqrt((var * x * x).sum(1) / S)
    assert np.all(np.abs(outs.mean(0) - ref) <= 5 * sigma + 2.0 ** -32 * (a * x).sum(1))
    # the flushing default is biased on the same layer: the gate is what removes it
    flushed = np.zeros((200, O))
    for seed in range(200):
        Wf, ebf, _ = oracle.sample_level(w, seed, 2, log2k, exp_bits=2)
        flushed[seed] = (Wf * x).sum(1) * 2.0 ** ebf.astype(np.float64) / k
    assert np.abs(flushed.mean(0) - ref).max() > 20 * sigma.max()


def test_options_off_reproduce_the_plain_sampler(oracle):
    rng = np.random.default_rng(6)
    w = rng.normal(0, 0.1, size=(5, 7, 3, 3)).astype(np.float32)
    w.reshape(-1)[::9] = 0
    for norm in (0, 1):
        for l in (0, 3, 6):
            a = oracle.sample_level(w, 9, 4, l, exp_bits=3, norm=norm)
            b = oracle.sample_level_ex(w, 9, 4, l, exp_bits=3, norm=norm)
            assert all(np.array_equal(u, v) for u, v in zip(a, b[:3]))


# ------------------------------------------------------------- probabilities on a grid

def test_probabilities_round_to_the_nearest_grid_point_and_carry_into_the_exponent(oracle):
    """Sec. 4.4: regular grid with p = 0, without p = 1; a p that rounds to 1 is the next power of two."""
    rng = np.random.default_rng(7)
    for b in (1, 2, 4, 6, 8):
        for w in np.concatenate([rng.normal(0, 1, 300), [1.0, 1.9999999, -3.9999998, 0.999999, 2.0 ** -20 * 1.97]]).astype(np.float32):
            if w == 0:
                continue
            cls, e, pq = oracle.quantise(w, b)
            assert cls == 1 and 0 <= pq < 2 ** b
            a = abs(Fraction(float(w)))
            value = Fraction(2) ** e * (1 + Fraction(pq, 2 ** b))
            e0 = oracle.decode(w)[2]
            assert abs(value - a) <= Fraction(2) ** e0 * Fraction(1, 2 ** (b + 1))     # nearest grid point
            if e != e0:
                assert e == e0 + 1 and pq == 0 and a >= Fraction(2) ** e0 * (2 - Fraction(1, 2 ** (b + 1)))
    assert oracle.quantise(np.float32(1.5), 4) == (1, 0, 8)
    assert oracle.quantise(np.float32(1.96875), 4) == (1, 1, 0)          # 1 + 15.5/16 rounds up: carries
    assert oracle.quantise(np.float32(1.96874), 4) == (1, 0, 15)


def test_packed_draws_use_the_documented_fields(oracle):
    """Draw j = bit field (j mod n) of word ((j / n) mod 4) of Philox call j / (4 n), n = floor(32 / b)."""
    seed, layer, index = 2 ** 35 + 11, 6, 2 ** 33 + 5
    for b in (4, 6, 8, 3):
        n = 32 // b
        for j in list(range(0, 4 * n + 3)) + [63]:
            r = oracle.philox4x32_10([j // (4 * n), layer, index & 0xFFFFFFFF, index >> 32], [seed & 0xFFFFFFFF, seed >> 32])
            field = (int(r[(j // n) % 4]) >> ((j % n) * b)) & (2 ** b - 1)
            for thr in (0, 1, field, field + 1, 2 ** b - 1):
                assert oracle.draw_bit_packed(seed, layer, index, j, thr, b) == (1 if field < thr else 0)


@pytest.mark.parametrize("b", [4, 6, 8])
def test_counts_with_quantised_probabilities_are_binomial_at_the_grid_point(oracle, b):
    pq = 5 if b == 4 else (37 if b == 6 else 201)
    on_grid = np.float32(0.25 * (1 + pq / 2 ** b))                   # exactly representable: no rounding
    off_grid = np.float32(float(on_grid) * (1 + 0.3 / 2 ** (b + 1)))  # rounds to the same grid point
    for wv in (on_grid, off_grid):
        assert oracle.quantise(wv, b)[1:] == (-2, pq)
        w = np.full((1, 4000), wv, dtype=np.float32)
        for log2k in (3, 5):
            k = 1 << log2k
            W, eb, c, _ = oracle.sample_level_ex(w, 31, 2, log2k, prob_bits=b)
            assert np.array_equal(W[0], (k + c[0].astype(np.int64)) << 15)
            obs = np.bincount(c[0], minlength=k + 1)
            exp = stats.binom.pmf(np.arange(k + 1), k, pq / 2 ** b) * 4000
            keep = exp > 5
            chi = ((obs[keep] - exp[keep]) ** 2 / exp[keep]).sum()
            assert chi < stats.chi2.ppf(0.999, keep.sum())
    # levels share draws, also with packed draws
    w = np.random.default_rng(8).normal(0, 0.1, size=(3, 50)).astype(np.float32)
    c = [oracle.sample_level_ex(w, 5, 1, l, prob_bits=b)[2].astype(np.int64) for l in range(7)]
    for l in range(6):
        assert np.all(c[l + 1] >= c[l]) and np.all(c[l + 1] - c[l] <= (1 << l))


def test_deterministic_variant_takes_the_upper_shift_in_p_k_of_k_cases(oracle):
    """Sec. 4.4: with b-bit probabilities nothing is gained beyond 2^b draws; p = 3/16 can be served by the
    upper shift in 3 of 16 cases."""
    w = np.array([[0.25 * (1 + 3 / 16), -0.5 * (1 + 11 / 16), 0.125]], dtype=np.float32)
    for log2k in (4, 5, 6):
        k = 1 << log2k
        W, eb, c, _ = oracle.sample_level_ex(w, 123, 0, log2k, prob_bits=4, deterministic=1)
        assert list(c[0]) == [3 * k // 16, 11 * k // 16, 0]
        real = W[0] * 2.0 ** float(eb[0]) / k
        assert np.array_equal(real, w[0].astype(np.float64))          # exact: no randomness left
        assert np.array_equal(W, oracle.sample_level_ex(w, 999, 7, log2k, prob_bits=4, deterministic=1)[0])
    W, eb, c, _ = oracle.sample_level_ex(w, 1, 0, 2, prob_bits=4, deterministic=1)       # k = 4 < 16: rounded
    assert list(c[0]) == [1, 3, 0]
    with pytest.raises(ValueError):
        oracle.sample_level_ex(w, 1, 0, 2, prob_bits=0, deterministic=1)


def test_gate_with_quantised_probabilities(oracle):
    """Below the window with b-bit probabilities: q is rounded to the grid; a q that rounds to 1 is the window's
    floor itself (a weight inside the window with p = 0); a q that rounds to 0 contributes nothing."""
    e_base = -3
    assert oracle.classify(np.float32(0.75 * 2.0 ** -3), e_base, 4, 1) == (1, 0, 0, 12)
    assert oracle.classify(np.float32(0.99 * 2.0 ** -3), e_base, 4, 1) == (1, 1, 0, 0)
    assert oracle.classify(np.float32(0.02 * 2.0 ** -3), e_base, 4, 1) == (0, 0, 0, 0)
    assert oracle.classify(np.float32(0.04 * 2.0 ** -3), e_base, 4, 1) == (1, 0, 0, 1)
