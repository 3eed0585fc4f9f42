"""Pins of the oracle's probabilistic quantizer Q_p (Sec. IV-A, Eq. (7)) and of its counter-based generator."""
import math
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2501_09849_b200 import inputs

f32 = np.float32
GOLDEN = Path(__file__).resolve().parent / "golden" / "philox4x32_10_kat.txt"


def test_philox_known_answer_vectors():
    rows = [l.split() for l in GOLDEN.read_text().splitlines() if l and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        assert list(oracle.philox4x32_10(v[0:4], v[4:6])) == v[6:10]


def test_uniform_numbers_layout_and_range():
    # element e uses word e mod 4 of the block with counter (e div 4) and key = seed, top 24 bits
    seed = 0x299f31d0a4093822
    for e in (0, 1, 2, 3, 4, 7, 1 << 33, (1 << 34) + 5):
        blk = oracle.philox4x32_10([(e >> 2) & 0xffffffff, (e >> 2) >> 32, 0, 0], [seed & 0xffffffff, seed >> 32])
        u = oracle.uniform(seed, e)
        assert u == float(int(blk[e & 3]) >> 8) / 2.0 ** 24
        assert 0.0 <= u < 1.0
    us = np.array([oracle.uniform(3, e) for e in range(4000)])
    assert abs(us.mean() - 0.5) < 0.02 and abs(us.var() - 1 / 12) < 0.01
    assert len(set(us)) > 3990


def test_two_level_sampling_is_the_logistic_threshold():
    # levels {0, q}: P(q | theta) = sigma(alpha q (2 theta - q)); inversion visits level 0 first, so the index is 1
    # exactly when u >= 1 - sigma
    q, alpha = f32(0.5), f32(6.0)
    x = inputs.normal((5000,), 0.6, seed=1) + f32(0.25)
    idx, u, lo_, hi_ = oracle.sample(x, q, 0, 1, alpha, 0, seed=9)
    s = 1.0 / (1.0 + np.exp(-float(alpha) * float(q) * (2.0 * x.astype(np.float64) - float(q))))
    clear = np.abs(u - (1.0 - s)) > 1e-12
    assert np.array_equal(idx[clear], (u >= 1.0 - s).astype(np.int32)[clear])
    assert 0.3 < idx.mean() < 0.7


def test_sampled_index_brackets_its_uniform_number():
    x = inputs.normal((20000,), 0.2, seed=2)
    for window in (0, 5):
        idx, u, a, b = oracle.sample(x, f32(0.1), -4, 3, f32(60.0), window, seed=5, first_index=12345)
        assert np.all(a <= u) and np.all((u < b) | (b > 1.0 - 1e-12))
        assert idx.min() >= -4 and idx.max() <= 3
        # the same elements under another seed or offset draw other numbers
        idx2, u2, _, _ = oracle.sample(x, f32(0.1), -4, 3, f32(60.0), window, seed=6, first_index=12345)
        idx3, u3, _, _ = oracle.sample(x, f32(0.1), -4, 3, f32(60.0), window, seed=5, first_index=12346)
        assert not np.array_equal(u, u2) and np.array_equal(u[1:], u3[:-1])


@pytest.mark.parametrize("theta,alpha,window", [(0.13, 100.0, 0), (-0.31, 30.0, 0), (0.6, 3.0, 5), (1.9, 2.0, 5)])
def test_sample_frequencies_follow_the_cpmf(theta, alpha, window):
    n = 200000
    lo, hi, q = (0, 15, f32(0.25)) if window else (-4, 3, f32(0.1))
    x = np.full(n, theta, dtype=f32)
    idx, _, _, _ = oracle.sample(x, q, lo, hi, f32(alpha), window, seed=77)
    P = oracle.cpmf(float(f32(theta)), float(q), lo, hi, float(f32(alpha)), window)
    freq = np.bincount(idx - lo, minlength=hi - lo + 1) / n
    sigma = np.sqrt(P * (1 - P) / n)
    assert np.all(np.abs(freq - P) <= 4.5 * sigma + 1e-9)
    assert np.all(freq[P == 0] == 0)


def test_large_alpha_sampling_is_the_uniform_quantizer():
    # Remark of Sec. IV-A: Q_p picks the nearest level with probability -> 1 as alpha grows
    x = inputs.normal((20000,), 0.25, seed=5)
    q = f32(0.1)
    uu = x.astype(np.float64) / float(q)
    away = np.abs(uu - np.floor(uu) - 0.5) > 0.05
    hard, _ = oracle.hard(x, q, -4, 3)
    idx, _, _, _ = oracle.sample(x, q, -4, 3, f32(1e6), 0, seed=1)
    assert np.array_equal(idx[away], hard[away])


def test_expected_sampled_value_is_the_soft_value():
    # Q_d = E{Q_p} (Sec. IV-B, Eq. (8)): Monte-Carlo mean over many seeds
    x = np.array([0.03, 0.12, -0.26, 0.31], dtype=f32)
    q, lo, hi, alpha = f32(0.1), -4, 3, f32(80.0)
    reps = 20000
    xs = np.tile(x, reps)
    idx, _, _, _ = oracle.sample(xs, q, lo, hi, alpha, 0, seed=123)
    mean = (idx.reshape(reps, 4) * float(q)).mean(axis=0)
    soft = oracle.soft(x, q, lo, hi, alpha)
    _, _, _, var = oracle.partials(x, q, lo, hi, alpha)
    assert np.all(np.abs(mean - soft) <= 4.5 * np.sqrt(var / reps) + 1e-9)
