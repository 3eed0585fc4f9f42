"""GPU parity of the quantizer kernels against the CPU oracle, element by element, through the C ABI.

Bars: hard indices and histograms bit-exact; soft values and gradients within 1e-5 relative with the
absolute floors the arithmetic implies (q for Q_d, max(1, alpha q^2 / 2) |g| for the theta-gradient, term
magnitudes of Lemma 1 for the reduced sums); entropy within 1e-6 bits.
"""
import math

import numpy as np
import pytest

import oracle
import paper_2501_09849_b200 as cdl
from paper_2501_09849_b200 import inputs

pytestmark = pytest.mark.gpu
f32 = np.float32
RTOL = 1e-5
# Floor of the reduced sums grad_q / grad_alpha, in units of the oracle's term-magnitude scale (sum of |g| times
# the magnitudes of the terms of Eq. (9b) resp. of dQ_d/dalpha): a third of a binary32 ulp of those terms.  It only
# matters where the terms cancel inside every element (alpha q^2 << 1: Q_d ~ theta, both partials ~ 0).
MAG_FLOOR = 2e-8
PURE_REL = {"grad_q": 0.0, "grad_alpha": 0.0}     # largest pure relative error seen where it is meaningful


@pytest.fixture(scope="module")
def torch():
    import torch
    cdl.load_library()
    return torch


def dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def idx_dtype(torch, lo):
    return torch.int8 if lo < 0 else torch.uint8


def run_hard(torch, x, P, offset=0):
    """Returns (idx int32 numpy, hist uint64 numpy).  offset shifts every buffer by that many elements."""
    n = x.size
    xb = torch.empty(n + offset + 8, dtype=torch.float32, device="cuda")
    xd = xb[offset:offset + n]
    xd.copy_(torch.from_numpy(x.reshape(-1)))
    ib = torch.full((n + offset + 8,), 99, dtype=idx_dtype(torch, P.lo), device="cuda")
    idx = ib[offset:offset + n]
    hist = torch.full((P.nlev,), 12345, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_hard(xd, n, P, idx, hist)
    torch.cuda.synchronize()
    assert int(ib[offset + n]) == 99 and (offset == 0 or int(ib[offset - 1]) == 99)
    return idx.cpu().numpy().astype(np.int32), hist.cpu().numpy().view(np.uint64)


def run_soft(torch, x, P, with_idx=True, offset=0):
    n = x.size
    xb = torch.empty(n + offset + 8, dtype=torch.float32, device="cuda")
    xd = xb[offset:offset + n]
    xd.copy_(torch.from_numpy(x.reshape(-1)))
    yb = torch.full((n + offset + 8,), 7.0, dtype=torch.float32, device="cuda")
    y = yb[offset:offset + n]
    idx = torch.empty(n, dtype=idx_dtype(torch, P.lo), device="cuda") if with_idx else None
    hist = torch.empty(P.nlev, dtype=torch.int64, device="cuda") if with_idx else None
    cdl.cdl_quantize_soft(xd, n, P, y, idx, hist)
    torch.cuda.synchronize()
    assert float(yb[offset + n]) == 7.0
    if with_idx:
        return y.cpu().numpy(), idx.cpu().numpy().astype(np.int32), hist.cpu().numpy().view(np.uint64)
    return y.cpu().numpy(), None, None


def run_backward(torch, x, g, P, offset=0):
    n = x.size
    xb = torch.empty(n + offset + 8, dtype=torch.float32, device="cuda")
    gb = torch.empty(n + offset + 8, dtype=torch.float32, device="cuda")
    xd, gd = xb[offset:offset + n], gb[offset:offset + n]
    xd.copy_(torch.from_numpy(x.reshape(-1)))
    gd.copy_(torch.from_numpy(g.reshape(-1)))
    ob = torch.full((n + offset + 8,), 7.0, dtype=torch.float32, device="cuda")
    gx = ob[offset:offset + n]
    s = torch.full((2,), 1e300, dtype=torch.float64, device="cuda")
    cdl.cdl_quantize_backward(xd, gd, n, P, gx, s[0:1], s[1:2])
    torch.cuda.synchronize()
    assert float(ob[offset + n]) == 7.0
    s = s.cpu().numpy()
    return gx.cpu().numpy(), float(s[0]), float(s[1])


def assert_soft_close(y, ref, q):
    err = np.abs(y.astype(np.float64) - ref)
    tol = RTOL * np.abs(ref) + RTOL * float(f32(q))
    worst = int(np.argmax(err - tol))
    assert np.all(err <= tol), f"soft: err {err[worst]:.3e} > tol {tol[worst]:.3e} at {worst} (ref {ref[worst]!r})"


def assert_sum_close(name, got, ref_sum, ref_abs, ref_mag):
    """A reduced sum against the oracle's: |err| <= 1e-5 sum|g d_i| + MAG_FLOOR * term magnitudes; and where the
    sum is cancellation-dominated neither across elements (|sum| >= 1e-2 sum|g d_i|) nor inside them
    (sum|g d_i| >= 1e-1 of the term magnitudes), 1e-5 purely relative to the sum itself."""
    err = abs(got - ref_sum)
    assert err <= RTOL * ref_abs + MAG_FLOOR * ref_mag + 1e-300, (name, got, ref_sum, ref_abs, ref_mag)
    if abs(ref_sum) >= 1e-2 * ref_abs and ref_abs >= 1e-1 * ref_mag and ref_sum != 0.0:
        rel = err / abs(ref_sum)
        PURE_REL[name] = max(PURE_REL[name], rel)
        assert rel <= RTOL, (name, "pure relative error", rel, got, ref_sum)


@pytest.fixture(scope="module", autouse=True)
def report_pure_relative_error():
    yield
    print("\nlargest pure relative error of the reduced sums where they are not cancellation-dominated: "
          "grad_q %.3g, grad_alpha %.3g" % (PURE_REL["grad_q"], PURE_REL["grad_alpha"]))


def assert_backward_close(gx, gq, ga, ref, g, q, alpha, rate_weight=0.0, level_prob=None):
    a = float(f32(alpha)) * float(f32(q)) ** 2
    floor = np.abs(g.reshape(-1).astype(np.float64)) * max(1.0, a / 2.0)
    if level_prob is not None and rate_weight:
        # rate term = -2 alpha q^2 Cov(log2 pbar, J): scale by the spread of log2 pbar and of J (std ~ 1/sqrt(2a))
        L = np.log2(np.maximum(level_prob, 2.0 ** -30))
        floor = floor + rate_weight * 2.0 * a * max(float(L.max() - L.min()), 1.0) * (2.0 + 1.0 / math.sqrt(2.0 * a))
    r = ref["grad_x"].reshape(-1)
    err = np.abs(gx.astype(np.float64) - r)
    tol = RTOL * np.abs(r) + RTOL * floor + 1e-30
    worst = int(np.argmax(err - tol))
    assert np.all(err <= tol), f"grad_x: err {err[worst]:.3e} > tol {tol[worst]:.3e} at {worst} (ref {r[worst]!r})"
    assert_sum_close("grad_q", gq, ref["grad_q"], ref["abs_q"], ref["mag_q"])
    assert_sum_close("grad_alpha", ga, ref["grad_alpha"], ref["abs_alpha"], ref["mag_alpha"])


# ----------------------------------------------------------------------------------------------- tiny layer
def test_tiny_layer_quantizers_match_the_oracle(torch):
    case, w, a = inputs.tiny_layer(seed=0)
    for t, Q in ((w, case.wq), (a, case.aq)):
        P = cdl.QuantParams(Q.q, Q.lo, Q.hi, Q.alpha, Q.rate_weight)
        ref_idx, ref_hist = oracle.hard(t, f32(Q.q), Q.lo, Q.hi)
        idx, hist = run_hard(torch, t, P)
        assert np.array_equal(idx, ref_idx.reshape(-1)) and np.array_equal(hist, ref_hist)
        for window in (0, 5):
            P.window = window
            y, idx2, hist2 = run_soft(torch, t, P)
            assert np.array_equal(idx2, ref_idx.reshape(-1)) and np.array_equal(hist2, ref_hist)
            assert_soft_close(y, oracle.soft(t, f32(Q.q), Q.lo, Q.hi, f32(Q.alpha), window).reshape(-1), Q.q)
            g = inputs.normal(t.shape, 1.0, seed=0, stream=5)
            # uniform level probabilities (initial state) and the histogram's own probabilities
            H, lp, n = oracle.entropy(ref_hist)
            for probs in (None, np.full(Q.nlev, 1.0 / Q.nlev), lp):
                P.level_prob = None if probs is None else dev(torch, probs.astype(f32))
                probs32 = None if probs is None else probs.astype(f32).astype(np.float64)
                ref = oracle.backward(t, g, f32(Q.q), Q.lo, Q.hi, f32(Q.alpha), window, f32(Q.rate_weight), probs32)
                gx, gq, ga = run_backward(torch, t, g, P)
                assert_backward_close(gx, gq, ga, ref, g, Q.q, Q.alpha, Q.rate_weight, probs32)
            P.level_prob = None


def test_zero_rate_weight_is_plain_uniform_quantization_gradient(torch):
    case, w, _ = inputs.tiny_layer(seed=0)
    Q = case.wq
    g = inputs.normal(w.shape, 1.0, seed=1)
    lp = dev(torch, np.random.default_rng(0).dirichlet(np.ones(Q.nlev)).astype(f32))
    base = run_backward(torch, w, g, cdl.QuantParams(Q.q, Q.lo, Q.hi, Q.alpha))
    zero = run_backward(torch, w, g, cdl.QuantParams(Q.q, Q.lo, Q.hi, Q.alpha, 0.0, lp))
    assert np.array_equal(base[0], zero[0])


# ----------------------------------------------------------------------------------------------- entropy
def test_entropy_matches_the_oracle(torch):
    rng = np.random.default_rng(3)
    cases = [np.full(16, 7), np.array([0, 0, 9, 0]), np.array([5]), np.zeros(6, dtype=np.int64),
             rng.integers(0, 1 << 40, size=256), rng.integers(0, 50, size=15), np.array([1, (1 << 62)])]
    for h in cases:
        h = h.astype(np.uint64)
        hd = dev(torch, h.view(np.int64))
        H = torch.zeros(1, dtype=torch.float64, device="cuda")
        lp = torch.zeros(h.size, dtype=torch.float32, device="cuda")
        n = torch.zeros(1, dtype=torch.int64, device="cuda")
        cdl.cdl_index_entropy(hd, h.size, H, lp, n)
        refH, refp, refn = oracle.entropy(h)
        assert abs(float(H.cpu()[0]) - refH) <= 1e-6
        assert int(n.cpu()[0]) == refn
        np.testing.assert_allclose(lp.cpu().numpy(), refp, rtol=1e-6, atol=1e-38)
        cdl.cdl_index_entropy(hd, h.size, H)      # optional outputs omitted
        assert abs(float(H.cpu()[0]) - refH) <= 1e-6


# ----------------------------------------------------------------------------------------------- edge cases
@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 1023, 4097, 100003])
@pytest.mark.parametrize("offset", [0, 1])
def test_sizes_tails_and_unaligned_buffers(torch, n, offset):
    x = inputs.normal((n,), 0.3, seed=n + 1)
    g = inputs.normal((n,), 1.0, seed=n + 2)
    P = cdl.QuantParams(0.07, -7, 7, 60.0, window=5)
    ref_idx, ref_hist = oracle.hard(x, f32(P.q), P.lo, P.hi)
    idx, hist = run_hard(torch, x, P, offset)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist) and hist.sum() == n
    if n == 0:
        return
    for window in (0, 5):
        P.window = window
        y, idx2, hist2 = run_soft(torch, x, P, True, offset)
        assert np.array_equal(idx2, ref_idx) and np.array_equal(hist2, ref_hist)
        assert_soft_close(y, oracle.soft(x, f32(P.q), P.lo, P.hi, f32(P.alpha), window), P.q)
        gx, gq, ga = run_backward(torch, x, g, P, offset)
        assert_backward_close(gx, gq, ga, oracle.backward(x, g, f32(P.q), P.lo, P.hi, f32(P.alpha), window), g, P.q, P.alpha)


@pytest.mark.parametrize("lo,hi", [(3, 3), (0, 1), (-1, 1), (-128, 127), (0, 255), (-5, -2), (200, 255)])
def test_degenerate_and_maximal_alphabets(torch, lo, hi):
    nlev = hi - lo + 1
    q = 0.05
    centre = 0.5 * (lo + hi) * q
    x = (inputs.normal((20011,), max(nlev, 2) * q / 3.0, seed=nlev) + f32(centre)).astype(f32)
    g = inputs.normal(x.shape, 1.0, seed=nlev + 1)
    for alpha in (3.0, 400.0):
        for window in (0, 3, 5, 9):
            P = cdl.QuantParams(q, lo, hi, alpha, window=window)
            ref_idx, ref_hist = oracle.hard(x, f32(q), lo, hi)
            y, idx, hist = run_soft(torch, x, P)
            assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist)
            assert_soft_close(y, oracle.soft(x, f32(q), lo, hi, f32(alpha), window), q)
            gx, gq, ga = run_backward(torch, x, g, P)
            assert_backward_close(gx, gq, ga, oracle.backward(x, g, f32(q), lo, hi, f32(alpha), window), g, q, alpha)


def test_exact_midpoints_clamping_nan_and_signed_zero(torch):
    q = f32(0.5)
    x = np.array([0.25, 0.75, 1.25, -0.25, -0.75, 100.0, -100.0, np.inf, -np.inf, np.nan, 0.0, -0.0,
                  1e-45, -1e-45, 3.4e38, -3.4e38], dtype=f32)
    P = cdl.QuantParams(q, -2, 3, 10.0)
    ref_idx, ref_hist = oracle.hard(x, q, -2, 3)
    idx, hist = run_hard(torch, x, P)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist)
    assert list(idx[:12]) == [0, 2, 2, 0, -2, 3, -2, 3, -2, -2, 0, 0]
    # exact midpoints with the 5-level window: the lower of two equally near levels centres the window
    xm = ((np.arange(0, 15) + 0.5) * 0.25).astype(f32)
    Pw = cdl.QuantParams(0.25, 0, 15, 2.0, window=5)
    y, _, _ = run_soft(torch, xm, Pw)
    assert_soft_close(y, oracle.soft(xm, f32(0.25), 0, 15, f32(2.0), 5), 0.25)


def test_histogram_accumulate_flag_and_run_to_run_determinism(torch):
    x = inputs.relu_normal((300001,), seed=4)
    P = cdl.QuantParams(0.25, 0, 15)
    n = x.size
    xd = dev(torch, x)
    idx = torch.empty(n, dtype=torch.uint8, device="cuda")
    hist = torch.zeros(16, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_hard(xd, n, P, idx, hist)
    first_idx, first_hist = idx.clone(), hist.clone()
    P.flags = cdl.CDL_HIST_ACCUMULATE
    cdl.cdl_quantize_hard(xd, n, P, idx, hist)
    assert torch.equal(hist, 2 * first_hist) and torch.equal(idx, first_idx)
    P.flags = 0
    cdl.cdl_quantize_hard(xd, n, P, idx, hist)
    assert torch.equal(hist, first_hist) and int(hist.sum()) == n
    ref_idx, ref_hist = oracle.hard(x, f32(0.25), 0, 15)
    assert np.array_equal(first_hist.cpu().numpy().view(np.uint64), ref_hist)
    assert ref_hist[0] > n // 2 - 2000          # the post-ReLU zero spike really is there


# ----------------------------------------------------------------------------------------------- sweep grid
@pytest.mark.parametrize("L", [1, 3, 7, 15, 127])
@pytest.mark.parametrize("alpha", [1.0, 100.0, 1e4])
def test_bandwidth_sweep_grid_parity(torch, L, alpha):
    # the sweep's parameter grid on a size the oracle finishes in seconds; step q = 4 / L covers +-4 sigma
    n = (1 << 18) + 77 if L == 127 else (1 << 20) + 77
    x = inputs.normal_laplace_mixture((n,), seed=L)
    g = inputs.normal((n,), 1.0, seed=L + 100)
    q = float(f32(4.0 / L))
    P = cdl.QuantParams(q, -L, L, alpha)
    ref_idx, ref_hist = oracle.hard(x, f32(q), -L, L)
    y, idx, hist = run_soft(torch, x, P)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist)
    assert_soft_close(y, oracle.soft(x, f32(q), -L, L, f32(alpha)), q)
    gx, gq, ga = run_backward(torch, x, g, P)
    assert_backward_close(gx, gq, ga, oracle.backward(x, g, f32(q), -L, L, f32(alpha)), g, q, alpha)


def test_sweep_point_at_two_to_the_24_elements(torch):
    # 2^24 + 77 elements: every thread of the persistent grid runs several grid-stride iterations, every block
    # flushes its private histogram once, and a scalar tail remains.  Hard (with histogram), soft with index and
    # histogram, and backward against the oracle, element by element.
    n, L, alpha = (1 << 24) + 77, 7, 100.0
    x = inputs.normal_laplace_mixture((n,), seed=24)
    g = inputs.normal((n,), 1.0, seed=124)
    q = float(f32(4.0 / L))
    P = cdl.QuantParams(q, -L, L, alpha)
    ref_idx, ref_hist = oracle.hard(x, f32(q), -L, L)
    idx, hist = run_hard(torch, x, P)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist) and int(hist.sum()) == n
    y, idx, hist = run_soft(torch, x, P)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist)
    assert_soft_close(y, oracle.soft(x, f32(q), -L, L, f32(alpha)), q)
    gx, gq, ga = run_backward(torch, x, g, P)
    assert_backward_close(gx, gq, ga, oracle.backward(x, g, f32(q), -L, L, f32(alpha)), g, q, alpha)


def test_bench_size_activations_window_five_and_rate_term(torch):
    # The activation tensor of the benchmark's layer at its full size (256 x 14 x 14 x 256 = 12,845,056 half-normal
    # values, 16 levels, window of five, alpha = 100, step from the mean magnitude), in the launch configuration
    # the benchmark times: soft value + index + histogram, entropy, and the backward pass with the rate term fed
    # by the histogram's own level probabilities; all against the oracle, element by element.
    case, _, a = inputs.resnet18_layer3_conv(seed=3)
    Q = case.aq
    x = a.reshape(-1)
    assert x.size == 12845056 and Q.window == 5
    g = inputs.normal((x.size,), 1.0, seed=3, stream=5)
    P = cdl.QuantParams(Q.q, Q.lo, Q.hi, Q.alpha, Q.rate_weight, window=Q.window)
    ref_idx, ref_hist = oracle.hard(x, f32(Q.q), Q.lo, Q.hi)
    y, idx, hist = run_soft(torch, x, P)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist)
    assert_soft_close(y, oracle.soft(x, f32(Q.q), Q.lo, Q.hi, f32(Q.alpha), Q.window), Q.q)
    hd = dev(torch, ref_hist.view(np.int64))
    H = torch.zeros(1, dtype=torch.float64, device="cuda")
    lp = torch.zeros(Q.nlev, dtype=torch.float32, device="cuda")
    cdl.cdl_index_entropy(hd, Q.nlev, H, lp)
    refH, refp, _ = oracle.entropy(ref_hist)
    assert abs(float(H.cpu()[0]) - refH) <= 1e-6
    P.level_prob = lp
    probs = lp.cpu().numpy().astype(np.float64)          # the binary32 probabilities the kernel reads
    np.testing.assert_allclose(probs, refp, rtol=1e-6, atol=1e-38)
    gx, gq, ga = run_backward(torch, x, g, P)
    ref = oracle.backward(x, g, f32(Q.q), Q.lo, Q.hi, f32(Q.alpha), Q.window, f32(Q.rate_weight), probs)
    assert_backward_close(gx, gq, ga, ref, g, Q.q, Q.alpha, Q.rate_weight, probs)


def test_paper_native_six_bit_point(torch):
    # b = 6 for weights (-32..31) and activations (0..63), alpha = beta = 500, step from the mean magnitude
    w = inputs.he_normal(2304, (2304, 64), seed=6)
    a = inputs.half_normal((200000,), seed=7)
    for t, lo, hi, window in ((w, -32, 31, 0), (a, 0, 63, 5)):
        q = inputs.step_from_mean_abs(t, 6)
        P = cdl.QuantParams(q, lo, hi, 500.0, window=window)
        g = inputs.normal(t.shape, 1.0, seed=8)
        ref_idx, ref_hist = oracle.hard(t, f32(q), lo, hi)
        y, idx, hist = run_soft(torch, t, P)
        assert np.array_equal(idx, ref_idx.reshape(-1)) and np.array_equal(hist, ref_hist)
        assert_soft_close(y, oracle.soft(t, f32(q), lo, hi, f32(500.0), window).reshape(-1), q)
        gx, gq, ga = run_backward(torch, t, g, P)
        assert_backward_close(gx, gq, ga, oracle.backward(t, g, f32(q), lo, hi, f32(500.0), window), g, q, 500.0)


def test_large_alpha_soft_equals_hard_levels(torch):
    # Remark of Sec. IV-A on the GPU path itself: for huge alpha Q_d is the nearest level
    x = inputs.normal((100000,), 0.25, seed=5)
    q = float(f32(0.1))
    P = cdl.QuantParams(q, -4, 3, 1e7)
    y, idx, _ = run_soft(torch, x, P)
    u = x.astype(np.float64) / q
    away = np.abs(u - np.floor(u) - 0.5) > 0.01
    np.testing.assert_allclose(y[away], (idx[away] * np.float64(q)).astype(f32), rtol=1e-6, atol=0)


def test_mismatched_alignments_take_the_scalar_path(torch):
    # x 16-byte aligned but outputs shifted by one element: no common 128-bit phase exists
    n = 5003
    x = inputs.normal((n,), 0.3, seed=21)
    g = inputs.normal((n,), 1.0, seed=22)
    P = cdl.QuantParams(0.07, -7, 7, 60.0, window=5)
    xd, gd = dev(torch, x), dev(torch, g)
    yb = torch.empty(n + 1, dtype=torch.float32, device="cuda")
    ib = torch.empty(n + 1, dtype=torch.int8, device="cuda")
    hist = torch.empty(15, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_soft(xd, n, P, yb[1:], ib[1:], hist)
    ref_idx, ref_hist = oracle.hard(x, f32(P.q), P.lo, P.hi)
    assert np.array_equal(ib[1:].cpu().numpy().astype(np.int32), ref_idx)
    assert np.array_equal(hist.cpu().numpy().view(np.uint64), ref_hist)
    assert_soft_close(yb[1:].cpu().numpy(), oracle.soft(x, f32(P.q), P.lo, P.hi, f32(P.alpha), 5), P.q)
    s = torch.zeros(2, dtype=torch.float64, device="cuda")
    cdl.cdl_quantize_backward(xd, gd, n, P, yb[1:], s[0:1], s[1:2])
    ref = oracle.backward(x, g, f32(P.q), P.lo, P.hi, f32(P.alpha), 5)
    sc = s.cpu().numpy()
    assert_backward_close(yb[1:].cpu().numpy(), float(sc[0]), float(sc[1]), ref, g, P.q, P.alpha)
    cdl.cdl_quantize_backward(xd, gd, n, P, None, s[0:1], None)       # optional outputs
    assert_sum_close("grad_q", float(s.cpu()[0]), ref["grad_q"], ref["abs_q"], ref["mag_q"])


@pytest.mark.parametrize("q,lo,hi,alpha,window", [
    (0.1, -4, 3, 100.0, 0), (0.1, -4, 3, 5000.0, 0), (0.25, 0, 15, 50.0, 5), (0.56, 0, 15, 100.0, 5),
    (0.02, -7, 7, 50.0, 0), (0.05, -128, 127, 40.0, 0), (0.3, 2, 2, 10.0, 0)])
def test_soft_histogram_and_its_entropy(torch, q, lo, hi, alpha, window):
    # Sec. V-C, Eq. (25): sum of CPMFs per level in 2^-32 fixed point, entropy of the marginal PMF via cdl_index_entropy
    n = 300007
    centre = 0.5 * (lo + hi) * q
    x = (inputs.normal((n,), max(hi - lo, 2) * q / 4.0, seed=lo + hi + 3) + f32(centre)).astype(f32)
    if lo == 0:
        x = np.abs(x)
    P = cdl.QuantParams(q, lo, hi, alpha, window=window)
    xd = dev(torch, x)
    y = torch.empty(n, dtype=torch.float32, device="cuda")
    sh = torch.full((P.nlev,), 77, dtype=torch.int64, device="cuda")
    hist = torch.empty(P.nlev, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_soft(xd, n, P, y, None, hist, soft_hist=sh)
    ref = oracle.mpmf(x, f32(q), lo, hi, f32(alpha), window)
    got = sh.cpu().numpy().view(np.uint64).astype(np.float64) / 2.0 ** 32
    assert np.all(np.abs(got - ref) <= 5e-6 * ref + 1e-9 * n + 1e-6), np.max(np.abs(got - ref))
    assert abs(got.sum() - n) <= 2e-6 * n
    # the soft value and the count histogram of the same call are unchanged by the extra output
    assert_soft_close(y.cpu().numpy(), oracle.soft(x, f32(q), lo, hi, f32(alpha), window), q)
    assert np.array_equal(hist.cpu().numpy().view(np.uint64), oracle.hard(x, f32(q), lo, hi)[1])
    H = torch.zeros(1, dtype=torch.float64, device="cuda")
    lp = torch.zeros(P.nlev, dtype=torch.float32, device="cuda")
    cdl.cdl_index_entropy(sh, P.nlev, H, lp)
    p = ref / ref.sum()
    refH = float(-np.sum(p[p > 0] * np.log2(p[p > 0])))
    assert abs(float(H.cpu()[0]) - refH) <= 2e-5
    np.testing.assert_allclose(lp.cpu().numpy(), p, rtol=1e-5, atol=1e-9)
    # determinism: integer accumulation gives the same bits on a second run
    sh2 = torch.zeros(P.nlev, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_soft(xd, n, P, y, None, None, soft_hist=sh2)
    assert torch.equal(sh, sh2)


@pytest.mark.parametrize("aq2", [12.5, 40.0, 63.9, 64.1, 300.0])
@pytest.mark.parametrize("lo,hi", [(-7, 7), (0, 15)])
def test_three_level_path_on_both_sides_of_the_residual_switch(torch, aq2, lo, hi):
    # alpha q^2 <= 64 takes theta - k q from one fused multiply-add, above it as a two-float sum: both must hold the
    # tolerance where the logits are most sensitive -- right at and next to the midpoints between levels, at the
    # largest |k| -- and for large theta far outside the alphabet
    q = 0.37
    alpha = aq2 / (q * q)
    rng = np.random.default_rng(int(aq2 * 10) + hi)
    mids = (np.arange(lo, hi) + 0.5) * q
    x = np.concatenate([mids, mids * (1 + 1e-6), mids * (1 - 1e-6), mids + 1e-4 * q, mids - 1e-4 * q,
                        rng.uniform((lo - 1) * q, (hi + 1) * q, 4000), [1e3, -1e3, 0.0, hi * q, lo * q]]).astype(f32)
    x = np.resize(x, 8192)
    g = rng.normal(0, 1, x.size).astype(f32)
    P = cdl.QuantParams(q, lo, hi, alpha)
    y, idx, hist = run_soft(torch, x, P, True)
    ref_idx, _ = oracle.hard(x, f32(q), lo, hi)
    assert np.array_equal(idx, ref_idx)
    assert_soft_close(y, oracle.soft(x, f32(q), lo, hi, f32(alpha), 0), q)
    gx, gq, ga = run_backward(torch, x, g, P)
    assert_backward_close(gx, gq, ga, oracle.backward(x, g, f32(q), lo, hi, f32(alpha), 0), g, q, alpha)


@pytest.mark.parametrize("window", [1, 3])
@pytest.mark.parametrize("aq2", [12.5, 300.0])
def test_small_windows_in_the_three_level_regime(torch, window, aq2):
    # alpha q^2 > 12 with a window below five: a window of one keeps the nearest level alone (Q_d is that level, all
    # gradients vanish, also right next to a midpoint where three levels would blend), a window of three keeps the
    # nearest level and its two neighbours.  Elements at and next to the midpoints, at the edges and outside.
    q, lo, hi = 0.37, -7, 7
    alpha = aq2 / (q * q)
    rng = np.random.default_rng(int(aq2) + window)
    mids = (np.arange(lo, hi) + 0.5) * q
    x = np.concatenate([mids, mids * (1 + 1e-6), mids * (1 - 1e-6), mids + 1e-3 * q, mids - 1e-3 * q,
                        rng.uniform((lo - 1) * q, (hi + 1) * q, 4000), [1e3, -1e3, 0.0, hi * q, lo * q]]).astype(f32)
    x = np.resize(x, 8192 + 3)
    g = rng.normal(0, 1, x.size).astype(f32)
    P = cdl.QuantParams(q, lo, hi, alpha, window=window)
    y, idx, _ = run_soft(torch, x, P)
    assert np.array_equal(idx, oracle.hard(x, f32(q), lo, hi)[0])
    ref_y = oracle.soft(x, f32(q), lo, hi, f32(alpha), window)
    assert_soft_close(y, ref_y, q)
    gx, gq, ga = run_backward(torch, x, g, P)
    ref = oracle.backward(x, g, f32(q), lo, hi, f32(alpha), window)
    assert_backward_close(gx, gq, ga, ref, g, q, alpha)
    if window == 1:
        assert np.all(gx == 0.0) and np.all(ref["grad_x"] == 0.0)
        lev = np.arange(lo, hi + 1) * float(f32(q))
        assert np.all(np.min(np.abs(ref_y[:, None] - lev[None, :]), axis=1) == 0.0)     # the oracle's Q_d is a level


# ------------------------------------------------------- whole index set, window narrower than the index set
@pytest.mark.parametrize("lo,hi,q,alpha", [
    (-32, 31, 0.05, 20.0),      # alpha q^2 log2 e = 0.072: powers of b carried as 1 + beta_j
    (-32, 31, 0.05, 60.0),      # 0.216: powers of b by repeated multiplication
    (0, 63, 0.06, 25.0),        # unsigned index set with half of the data at its lower edge
    (-128, 127, 0.03, 30.0),    # the widest index set, 0.039
])
def test_table_form_of_the_level_sums(torch, lo, hi, q, alpha):
    # The soft and backward passes over the whole index set when levels further than jmax steps from the nearest
    # one carry no weight and 2 jmax + 1 < nlev: level weights G_j b^j from a table and a recurrence instead of
    # one exponential per level, for the warps whose elements all lie jmax levels inside the index set.  Data:
    # half of the tensor near the middle of the index set, half a normal/Laplace mixture wide enough that some
    # elements sit at the edges (levels on one side only) and far outside; rate term with non-uniform level
    # probabilities; an element count that leaves a scalar tail.
    n = (1 << 17) + 3
    x = (inputs.normal_laplace_mixture((n,), seed=lo + 300) * f32(0.45 * hi * q)).astype(f32)
    if lo == 0:
        x = np.maximum(x, f32(0.0)) + (x < 0) * f32(-0.02) * (np.arange(n) % 7 == 0)
        x = x.astype(f32)
    # first half: within three levels of the middle of the index set, so that whole warps are far from its edges
    # (the table form is taken warp by warp); second half: the wide data, edges and outliers included
    mid = 0.5 * (lo + hi) * q
    x[: n // 2] = (mid + np.clip(inputs.normal((n // 2,), 1.5 * q, seed=hi + 500), -3.0 * q, 3.0 * q)).astype(f32)
    g = inputs.normal((n,), 1.0, seed=hi + 400)
    nlev = hi - lo + 1
    ref_idx, ref_hist = oracle.hard(x, f32(q), lo, hi)
    P = cdl.QuantParams(q, lo, hi, alpha)
    y, idx, hist = run_soft(torch, x, P)
    assert np.array_equal(idx, ref_idx) and np.array_equal(hist, ref_hist)
    assert int(ref_hist[0]) > 0 and int(ref_hist[-1]) > 0          # both edges of the index set are reached
    assert_soft_close(y, oracle.soft(x, f32(q), lo, hi, f32(alpha)), q)
    gx, gq, ga = run_backward(torch, x, g, P)
    assert_backward_close(gx, gq, ga, oracle.backward(x, g, f32(q), lo, hi, f32(alpha)), g, q, alpha)
    # rate term: probabilities from the tensor's own histogram, floored so that empty levels stay finite
    probs = (ref_hist.astype(np.float64) + 1.0) / float(ref_hist.sum() + nlev)
    probs32 = probs.astype(f32).astype(np.float64)
    Pr = cdl.QuantParams(q, lo, hi, alpha, 0.02, dev(torch, probs.astype(f32)))
    gx, gq, ga = run_backward(torch, x, g, Pr)
    ref = oracle.backward(x, g, f32(q), lo, hi, f32(alpha), 0, f32(0.02), probs32)
    assert_backward_close(gx, gq, ga, ref, g, q, alpha, 0.02, probs32)


def test_table_form_non_finite_inputs_give_nan_and_leave_their_neighbours_alone(torch):
    # the soft value of a NaN or infinite element is NaN (the header's contract); the finite elements of its
    # warp, which takes the level loop because of it while the other warps take the table form, are unaffected
    lo, hi, q, alpha = -32, 31, 0.05, 20.0
    x = np.clip(inputs.normal((4096,), 0.1, seed=77), -0.2, 0.2).astype(f32)     # |index| <= 4: far from the edges
    bad = {5: np.nan, 130: np.inf, 2051: -np.inf}
    for i, v in bad.items():
        x[i] = v
    y, idx, _ = run_soft(torch, x, cdl.QuantParams(q, lo, hi, alpha))
    assert all(np.isnan(y[i]) for i in bad)
    assert [int(idx[i]) for i in bad] == [lo, hi, lo]
    ok = np.ones(x.size, dtype=bool)
    ok[list(bad)] = False
    assert_soft_close(y[ok], oracle.soft(x[ok], f32(q), lo, hi, f32(alpha)), q)
