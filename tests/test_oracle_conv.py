"""Pins of the oracle's convolution products (strided cross-correlation with zero padding on index tensors):
each is checked against something that is not its own loop nest -- an explicit patch gather followed by the
(separately pinned) matrix product, scipy's correlate2d, the adjoint identities that define the two backward
products, and hand-made kernels whose result is known."""
import numpy as np
import pytest
from scipy import signal

import oracle


def rand_case(rng, N, H, W, C, CO, R, S, unsigned=True):
    X = rng.integers(0, 16, (N, H, W, C)).astype(np.uint8) if unsigned else rng.integers(-8, 8, (N, H, W, C)).astype(np.int8)
    Wt = rng.integers(-7, 8, (R * S * C, CO)).astype(np.int8)
    return X, Wt


def patches(X, R, S, ph, pw):
    """Explicit im2col: row (n,p,q), column (r*S+s)*C+c, zero outside the tensor."""
    N, H, W, C = X.shape
    P, Q = H + 2 * ph - R + 1, W + 2 * pw - S + 1
    Xp = np.zeros((N, H + 2 * ph, W + 2 * pw, C), dtype=X.dtype)
    Xp[:, ph:ph + H, pw:pw + W, :] = X
    cols = np.empty((N, P, Q, R, S, C), dtype=X.dtype)
    for r in range(R):
        for s in range(S):
            cols[:, :, :, r, s, :] = Xp[:, r:r + P, s:s + Q, :]
    return cols.reshape(N * P * Q, R * S * C)


@pytest.mark.parametrize("N,H,W,C,CO,R,S,ph,pw", [(2, 5, 6, 3, 4, 3, 3, 1, 1), (1, 7, 4, 2, 5, 1, 1, 0, 0),
                                                  (2, 6, 6, 2, 3, 5, 3, 2, 1), (1, 5, 5, 2, 2, 3, 3, 0, 0),
                                                  (1, 4, 4, 1, 1, 3, 3, 2, 2)])
def test_forward_equals_patch_gather_times_matrix(N, H, W, C, CO, R, S, ph, pw):
    rng = np.random.default_rng(11)
    for unsigned in (True, False):
        X, Wt = rand_case(rng, N, H, W, C, CO, R, S, unsigned)
        got = oracle.conv_fwd(X, Wt, R, S, ph, pw)
        want = oracle.gemm_fwd(patches(X, R, S, ph, pw), Wt)
        assert np.array_equal(got.reshape(want.shape), want)
        # and against numpy's own integer matmul of the same gather
        assert np.array_equal(want, patches(X, R, S, ph, pw).astype(np.int64) @ Wt.astype(np.int64))


def test_forward_single_channel_equals_scipy_correlate2d():
    rng = np.random.default_rng(12)
    X = rng.integers(0, 16, (1, 9, 8, 1)).astype(np.uint8)
    k = rng.integers(-7, 8, (3, 5)).astype(np.int8)
    got = oracle.conv_fwd(X, k.reshape(15, 1), 3, 5, 1, 2)[0, :, :, 0]
    want = signal.correlate2d(X[0, :, :, 0].astype(np.int64), k.astype(np.int64), mode="same", boundary="fill")
    assert np.array_equal(got, want)
    got_valid = oracle.conv_fwd(X, k.reshape(15, 1), 3, 5, 0, 0)[0, :, :, 0]
    assert np.array_equal(got_valid, signal.correlate2d(X[0, :, :, 0].astype(np.int64), k.astype(np.int64), mode="valid"))


@pytest.mark.parametrize("R,S,ph,pw", [(3, 3, 1, 1), (1, 1, 0, 0), (3, 5, 1, 2), (3, 3, 0, 0), (3, 3, 2, 2)])
def test_backward_products_are_the_adjoints_of_the_forward(R, S, ph, pw):
    # <conv(X, Wt), G> = <X, dX(G, Wt)> = <Wt, dW(X, G)>, exactly, in integers: fixes every index, sign and flip
    rng = np.random.default_rng(13)
    N, H, W, C, CO = 2, 6, 5, 3, 4
    X = rng.integers(-8, 8, (N, H, W, C)).astype(np.int8)
    Wt = rng.integers(-7, 8, (R * S * C, CO)).astype(np.int8)
    Y = oracle.conv_fwd(X, Wt, R, S, ph, pw)
    G = rng.integers(-127, 128, Y.shape).astype(np.int8)
    lhs = int((Y * G.astype(np.int64)).sum())
    dX = oracle.conv_dx(G, Wt, X.shape, R, S, ph, pw)
    dW = oracle.conv_dw(X, G, R, S, ph, pw)
    assert int((dX * X.astype(np.int64)).sum()) == lhs
    assert int((dW * Wt.astype(np.int64)).sum()) == lhs
    # adjointness holds for every X and Wt only if dX, dW are the right linear maps: probe with unit tensors
    for _ in range(6):
        E = np.zeros_like(X)
        E[tuple(rng.integers(0, d) for d in X.shape)] = 1
        assert int((oracle.conv_fwd(E, Wt, R, S, ph, pw) * G.astype(np.int64)).sum()) == int(dX[E == 1][0])
        F = np.zeros_like(Wt)
        F[tuple(rng.integers(0, d) for d in Wt.shape)] = 1
        assert int((oracle.conv_fwd(X, F, R, S, ph, pw) * G.astype(np.int64)).sum()) == int(dW[F == 1][0])


def test_delta_kernels_shift_and_one_by_one_is_a_matrix_product():
    rng = np.random.default_rng(14)
    N, H, W, C = 2, 5, 6, 3
    X = rng.integers(0, 16, (N, H, W, C)).astype(np.uint8)
    # 3x3 kernel with a single one at tap (r, s), identity over channels: output(p, q) = X(p-1+r, q-1+s)
    for r in range(3):
        for s in range(3):
            Wt = np.zeros((9 * C, C), dtype=np.int8)
            for c in range(C):
                Wt[(r * 3 + s) * C + c, c] = 1
            Y = oracle.conv_fwd(X, Wt, 3, 3, 1, 1)
            want = np.zeros((N, H, W, C), dtype=np.int64)
            for p in range(H):
                for q in range(W):
                    h, w = p - 1 + r, q - 1 + s
                    if 0 <= h < H and 0 <= w < W:
                        want[:, p, q, :] = X[:, h, w, :]
            assert np.array_equal(Y, want)
    Wt = rng.integers(-7, 8, (C, 4)).astype(np.int8)
    G = rng.integers(-127, 128, (N, H, W, 4)).astype(np.int8)
    assert np.array_equal(oracle.conv_fwd(X, Wt, 1, 1, 0, 0).reshape(-1, 4), oracle.gemm_fwd(X.reshape(-1, C), Wt))
    assert np.array_equal(oracle.conv_dx(G, Wt, X.shape, 1, 1, 0, 0).reshape(-1, C), oracle.gemm_dx(G.reshape(-1, 4), Wt))
    assert np.array_equal(oracle.conv_dw(X, G, 1, 1, 0, 0), oracle.gemm_dw(X.reshape(-1, C), G.reshape(-1, 4)))


def strided_patches(X, R, S, ph, pw, stride):
    """Explicit im2col of a strided convolution: row (n,p,q), column (r*S+s)*C+c, zero outside the tensor."""
    N, H, W, C = X.shape
    P, Q = (H + 2 * ph - R) // stride + 1, (W + 2 * pw - S) // stride + 1
    Xp = np.zeros((N, H + 2 * ph + stride, W + 2 * pw + stride, C), dtype=X.dtype)
    Xp[:, ph:ph + H, pw:pw + W, :] = X
    cols = np.empty((N, P, Q, R, S, C), dtype=X.dtype)
    for r in range(R):
        for s in range(S):
            cols[:, :, :, r, s, :] = Xp[:, r:r + stride * P:stride, s:s + stride * Q:stride, :][:, :P, :Q, :]
    return cols.reshape(N * P * Q, R * S * C)


@pytest.mark.parametrize("N,H,W,C,CO,R,S,ph,pw,stride", [(2, 8, 6, 3, 4, 3, 3, 1, 1, 2), (1, 7, 9, 2, 5, 1, 1, 0, 0, 2),
                                                         (2, 9, 8, 2, 3, 7, 7, 3, 3, 2), (1, 10, 10, 2, 2, 3, 3, 1, 1, 3),
                                                         (1, 6, 6, 1, 2, 2, 2, 0, 0, 2)])
def test_strided_products(N, H, W, C, CO, R, S, ph, pw, stride):
    # forward: an explicit strided patch gather times the (separately pinned) matrix product, and the stride-1
    # result sampled at every stride-th position; backward: the adjoint identities, exactly, in integers
    rng = np.random.default_rng(21)
    X = rng.integers(-8, 8, (N, H, W, C)).astype(np.int8)
    Wt = rng.integers(-7, 8, (R * S * C, CO)).astype(np.int8)
    Y = oracle.conv_fwd(X, Wt, R, S, ph, pw, stride)
    P, Q = oracle.conv_out_dims(H, W, R, S, ph, pw, stride)
    assert Y.shape == (N, P, Q, CO)
    want = strided_patches(X, R, S, ph, pw, stride).astype(np.int64) @ Wt.astype(np.int64)
    assert np.array_equal(Y.reshape(want.shape), want)
    dense = oracle.conv_fwd(X, Wt, R, S, ph, pw, 1)
    assert np.array_equal(Y, dense[:, ::stride, ::stride, :][:, :P, :Q, :])
    G = rng.integers(-127, 128, Y.shape).astype(np.int8)
    lhs = int((Y * G.astype(np.int64)).sum())
    dX = oracle.conv_dx(G, Wt, X.shape, R, S, ph, pw, stride)
    dW = oracle.conv_dw(X, G, R, S, ph, pw, stride)
    assert int((dX * X.astype(np.int64)).sum()) == lhs
    assert int((dW * Wt.astype(np.int64)).sum()) == lhs
    for _ in range(8):
        E = np.zeros_like(X)
        E[tuple(rng.integers(0, d) for d in X.shape)] = 1
        assert int((oracle.conv_fwd(E, Wt, R, S, ph, pw, stride) * G.astype(np.int64)).sum()) == int(dX[E == 1][0])
        F = np.zeros_like(Wt)
        F[tuple(rng.integers(0, d) for d in Wt.shape)] = 1
        assert int((oracle.conv_fwd(X, F, R, S, ph, pw, stride) * G.astype(np.int64)).sum()) == int(dW[F == 1][0])
    # the data gradient of a strided layer is the stride-1 data gradient of the gradient with zeros put between its
    # pixels (a textbook identity): build that dilated gradient and compare
    Pd, Qd = oracle.conv_out_dims(H, W, R, S, ph, pw, 1)
    Gd = np.zeros((N, Pd, Qd, CO), dtype=np.int8)
    Gd[:, ::stride, ::stride, :][:, :P, :Q, :] = G
    assert np.array_equal(dX, oracle.conv_dx(Gd, Wt, X.shape, R, S, ph, pw, 1))
