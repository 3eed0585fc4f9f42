"""GPU parity of the probabilistic quantizer Q_p (cdl_quantize_sample) against the CPU oracle.

Both sides draw the same uniform number per element (Philox4x32-10, bit-exact) and invert the CPMF in increasing
level order; the oracle sums in double precision, the kernel in binary32.  A sampled index is therefore required
to bracket its uniform number within 4e-6 of the oracle's cumulative probabilities (several answers are valid
only that close to a boundary), and to equal the oracle's index outright for all but a 1e-4 fraction."""
import numpy as np
import pytest

import oracle
import paper_2501_09849_b200 as cdl
from paper_2501_09849_b200 import inputs

pytestmark = pytest.mark.gpu
f32 = np.float32
DELTA = 4e-6


@pytest.fixture(scope="module")
def torch():
    import torch
    cdl.load_library()
    return torch


def run_sample(torch, x, P, seed, first_index=0, offset=0, want_y=True):
    n = x.size
    xb = torch.empty(n + offset + 8, dtype=torch.float32, device="cuda")
    xd = xb[offset:offset + n]
    xd.copy_(torch.from_numpy(x.reshape(-1)))
    idx = torch.full((n + offset + 8,), 99, dtype=torch.int8 if P.lo < 0 else torch.uint8, device="cuda")
    y = torch.full((n + offset + 8,), 7.0, dtype=torch.float32, device="cuda") if want_y else None
    hist = torch.full((P.nlev,), 5, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_sample(xd, n, P, seed, first_index, idx[offset:offset + n], None if y is None else y[offset:offset + n], hist)
    torch.cuda.synchronize()
    assert int(idx[offset + n]) == 99
    yy = None if y is None else y[offset:offset + n].cpu().numpy()
    return idx[offset:offset + n].cpu().numpy().astype(np.int32), yy, hist.cpu().numpy().view(np.uint64)


def check_against_oracle(idx, y, hist, x, P, seed, first_index=0):
    ref, u, a, b = oracle.sample(x, f32(P.q), P.lo, P.hi, f32(P.alpha), P.window, seed, first_index)
    ref, u = ref.reshape(-1), u.reshape(-1)
    lev = np.arange(P.lo, P.hi + 1)
    same = idx == ref
    assert same.mean() >= 1.0 - 1e-4, same.mean()
    # where they differ, the kernel's level must still bracket u within DELTA of the oracle's cumulative sums
    bad = np.flatnonzero(~same)
    for e in bad[:200]:
        Pm = oracle.cpmf(float(x.reshape(-1)[e]), float(f32(P.q)), P.lo, P.hi, float(f32(P.alpha)), P.window)
        F = np.cumsum(Pm)
        k = idx[e] - P.lo
        assert 0 <= k < lev.size and Pm[k] > 0
        below = F[k - 1] if k > 0 else 0.0
        assert below - DELTA <= u[e] <= F[k] + DELTA, (e, idx[e], ref[e], u[e], below, F[k])
    if y is not None:
        assert np.array_equal(y, idx.astype(f32) * f32(P.q))
    assert np.array_equal(hist, np.bincount(idx - P.lo, minlength=lev.size).astype(np.uint64))


@pytest.mark.parametrize("q,lo,hi,alpha,window", [
    (0.1, -4, 3, 100.0, 0),        # alpha q^2 = 1: loop over the whole alphabet
    (0.1, -4, 3, 5000.0, 0),       # alpha q^2 = 50: nearest-three path
    (0.25, 0, 15, 50.0, 5),        # window of five, alpha q^2 = 3.1
    (0.56, 0, 15, 100.0, 5),       # window of five requested, alpha q^2 = 31: nearest-three path
    (0.02, -7, 7, 50.0, 0),        # wide: alpha q^2 = 0.02, all 15 levels matter
    (0.25, 0, 15, 20.0, 3),        # other odd window
    (0.05, -128, 127, 40.0, 0),    # 256 levels
    (0.3, 2, 2, 10.0, 0),          # single level
])
def test_sampled_indices_match_the_oracle(torch, q, lo, hi, alpha, window):
    n = 200003
    centre = 0.5 * (lo + hi) * q
    x = (inputs.normal((n,), max(hi - lo, 2) * q / 4.0, seed=lo + hi + 7) + f32(centre)).astype(f32)
    if lo == 0:
        x = np.abs(x)
    P = cdl.QuantParams(q, lo, hi, alpha, window=window)
    idx, y, hist = run_sample(torch, x, P, seed=2024)
    check_against_oracle(idx, y, hist, x, P, 2024)


@pytest.mark.parametrize("n", [0, 1, 3, 5, 1023, 4097])
@pytest.mark.parametrize("offset,first_index", [(0, 0), (1, 0), (0, 6), (3, (1 << 35) + 1)])
def test_sizes_offsets_and_counter_origin(torch, n, offset, first_index):
    x = inputs.normal((n,), 0.3, seed=n + 1)
    P = cdl.QuantParams(0.1, -4, 3, 60.0)
    idx, y, hist = run_sample(torch, x, P, seed=(1 << 40) + 17, first_index=first_index, offset=offset, want_y=(n % 2 == 0))
    assert hist.sum() == n
    if n:
        check_against_oracle(idx, y, hist, x, P, (1 << 40) + 17, first_index)


def test_partitioned_calls_reproduce_the_single_call(torch):
    # the draw depends on (seed, element number) only: two calls on the halves, the second with its first_index,
    # give the same bytes as one call - for aligned and unaligned split points
    n = 100000
    x = inputs.half_normal((n,), seed=3)
    P = cdl.QuantParams(0.25, 0, 15, 50.0, window=5)
    whole, _, hist = run_sample(torch, x, P, seed=5)
    for cut in (40000, 33333):
        a, _, ha = run_sample(torch, x[:cut], P, seed=5)
        b, _, hb = run_sample(torch, x[cut:], P, seed=5, first_index=cut)
        assert np.array_equal(np.concatenate([a, b]), whole)
        assert np.array_equal(ha + hb, hist)
    other, _, _ = run_sample(torch, x, P, seed=6)
    assert not np.array_equal(other, whole)


def test_large_alpha_sampling_equals_the_hard_index(torch):
    x = inputs.normal((100000,), 0.25, seed=5)
    q = float(f32(0.1))
    P = cdl.QuantParams(q, -4, 3, 1e7)
    idx, _, _ = run_sample(torch, x, P, seed=1)
    hard, _ = oracle.hard(x, f32(q), -4, 3)
    u = x.astype(np.float64) / q
    away = np.abs(u - np.floor(u) - 0.5) > 0.01
    assert np.array_equal(idx[away], hard[away])
