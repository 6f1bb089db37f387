"""Pins for the checker's integer generator and delay draws (CPU only)."""
import math

import numpy as np
from scipy import stats

from oracle import rng


def test_mix_matches_published_splitmix64_sequence():
    # SplitMix64 (Steele, Lea, Flood 2014) seeded with 0: its n-th output is the
    # mixing function applied to n * golden-gamma, which is draw(key=0, n-1).
    published = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert [rng.draw(0, n) for n in range(3)] == published


def test_stream_keys_separate_inputs():
    keys = {rng.stream_key(s, st, c) for s in (0, 1) for st in (0, 1, 2) for c in range(50)}
    assert len(keys) == 2 * 3 * 50


def test_integer_log2_against_libm():
    g = np.random.default_rng(5)
    for r in [1, 2, 3, (1 << 63), (1 << 64) - 1, 0x8000000000000001] + \
            [int(v) for v in g.integers(1, 1 << 63, size=200)]:
        want = 64.0 - math.log2(r)
        got = rng.neg_log2_q32(r) / 2.0 ** 32
        assert abs(got - want) < 2.0 ** -29, (r, got, want)
    assert rng.neg_log2_q32(0) == rng.neg_log2_q32(1) == 64 << 32
    assert rng.neg_log2_q32((1 << 64) - 1) >= 1


def test_exp_draws_have_the_right_distribution():
    key = rng.stream_key(7, rng.STREAM_COMPUTE, 3)
    mean_ticks = rng.to_ticks(1.0)
    n = 60000
    t = np.array([rng.exp_ticks(rng.draw(key, k), mean_ticks) for k in range(n)], dtype=np.float64)
    x = t / mean_ticks
    assert abs(x.mean() - 1.0) < 4.0 / math.sqrt(n)          # 4 sigma
    assert stats.kstest(x, "expon").pvalue > 1e-3
    assert t.min() >= 1


def test_exp_scales_with_mean_and_floors_at_one_tick():
    r = 0x123456789ABCDEF0
    base = rng.exp_ticks(r, 1 << 20)
    assert abs(rng.exp_ticks(r, 10 << 20) - 10 * base) <= 10
    assert rng.exp_ticks((1 << 64) - 1, 1 << 20) == 1
    # closed form at u = 1/2: -ln(1/2) = ln 2
    assert abs(rng.exp_ticks(1 << 63, 1 << 20) - math.log(2) * 2 ** 20) <= 1


def test_uniform_ticks_cover_the_closed_range():
    key = rng.stream_key(1, rng.STREAM_NETWORK, 0)
    lo, hi = 10, 17
    seen = {rng.uniform_ticks(rng.draw(key, k), lo, hi) for k in range(2000)}
    assert seen == set(range(lo, hi + 1))
    assert rng.uniform_ticks(12345, 9, 9) == 9


def test_sample_index_uniform_and_in_range():
    key = rng.stream_key(0, rng.STREAM_SAMPLE, 2)
    n = 37
    idx = np.array([rng.sample_index(rng.draw(key, k), n) for k in range(37000)])
    assert idx.min() >= 0 and idx.max() == n - 1
    counts = np.bincount(idx, minlength=n)
    assert stats.chisquare(counts).pvalue > 1e-3
    assert rng.sample_index((1 << 64) - 1, n) == n - 1 and rng.sample_index(0, n) == 0


def test_tick_conversion_rounds_half_up():
    assert rng.to_ticks(1.0) == 1 << 20 and rng.to_ticks(0.5) == 1 << 19
    assert rng.to_ticks(0.1) == 104858
    assert rng.to_q16(10.0) == 10 << 16
