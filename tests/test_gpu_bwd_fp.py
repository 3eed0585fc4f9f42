"""Backward products with a real-valued gradient (two int8 digits per entry, exact integer products per digit):
bit-exact against the oracle's digit chain, and within the stated bound of the products with the real gradient."""
import numpy as np
import pytest

import oracle
import paper_2501_09849_b200 as cdl

pytestmark = pytest.mark.gpu
f32 = np.float32


@pytest.fixture(scope="module")
def torch():
    import torch
    cdl.load_library()
    return torch


def dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def padded(a, ld):
    out = np.zeros((a.shape[0], ld), dtype=a.dtype)
    out[:, :a.shape[1]] = a
    return out


@pytest.mark.parametrize("M,K,N", [(64, 256, 128), (300, 520, 130), (1000, 144, 16), (2048, 1152, 256)])
def test_two_digit_backward_products(torch, M, K, N):
    rng = np.random.default_rng(M + K)
    A = (rng.integers(0, 16, (M, K)) * (rng.random((M, K)) < 0.6)).astype(np.uint8)
    W = rng.integers(-7, 8, (K, N)).astype(np.int8)
    G = (rng.normal(0, 1e-2, (M, N)) * rng.lognormal(0, 1, (M, N))).astype(f32)      # heavy-tailed, like gradients
    absmax = float(np.abs(G).max())
    a, w = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7)
    lda, ldw = (K + 15) // 16 * 16, (N + 15) // 16 * 16
    nb = cdl.cdl_qlinear_bwd_fp_workspace_bytes(M, N, K)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    dX = torch.full((M, K), 7.0, dtype=torch.float32, device="cuda")
    dW = torch.full((K, N), 7.0, dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_bwd_fp(dev(torch, G), absmax, dev(torch, padded(A, lda)), lda, a, dev(torch, padded(W, ldw)), ldw, w,
                           M, N, K, dX, dW, ws, nb)
    torch.cuda.synchronize()
    assert cdl.cdl_workspace_status(ws, check=False) == 0
    # the oracle's chain: digits, exact integer products per digit, binary32 rescale per digit, one binary32 addition
    i1, i2, q1, q2 = oracle.gradient_digits(G, absmax)
    I1, I2 = i1.astype(np.int8), i2.astype(np.int8)

    def combine(acc1, acc2, qb):
        t1 = acc1.astype(f32) * f32(q1 * f32(qb))
        t2 = acc2.astype(f32) * f32(q2 * f32(qb))
        return (t1 + t2).astype(f32)
    ref_dx = combine(oracle.gemm_dx(I1, W), oracle.gemm_dx(I2, W), w.q)
    ref_dw = combine(oracle.gemm_dw(A, I1), oracle.gemm_dw(A, I2), a.q)
    assert np.array_equal(dX.cpu().numpy(), ref_dx)
    assert np.array_equal(dW.cpu().numpy(), ref_dw)
    # and against the products with the real gradient (binary64): error <= (absmax / 64516) * sum |operand| + rounding
    Wv = W.astype(np.float64) * np.float64(f32(w.q))
    Av = A.astype(np.float64) * np.float64(f32(a.q))
    Gd = G.astype(np.float64)
    true_dx, true_dw = Gd @ Wv.T, Av.T @ Gd
    eps = absmax / 64516.0
    bound_dx = eps * np.abs(Wv).sum(axis=1)[None, :] * 1.001 + 4e-7 * (np.abs(Gd) @ np.abs(Wv).T)
    bound_dw = eps * np.abs(Av).sum(axis=0)[:, None] * 1.001 + 4e-7 * (np.abs(Av).T @ np.abs(Gd))
    assert (np.abs(ref_dx - true_dx) <= bound_dx).all()
    assert (np.abs(ref_dw - true_dw) <= bound_dw).all()
    # the two-digit result is far closer to the real-gradient product than the one-digit (int8 gradient) reading
    one_digit = oracle.gemm_dx(I1, W).astype(np.float64) * float(q1) * float(f32(w.q))
    assert np.abs(ref_dx - true_dx).max() < 0.02 * np.abs(one_digit - true_dx).max()


def test_single_outputs_and_saturation(torch):
    rng = np.random.default_rng(5)
    M, K, N = 130, 144, 48
    A = rng.integers(0, 16, (M, K)).astype(np.uint8)
    W = rng.integers(-7, 8, (K, N)).astype(np.int8)
    G = rng.normal(0, 1.0, (M, N)).astype(f32)
    absmax = 1.5                                       # smaller than the data: the tails saturate
    a, w = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7)
    nb = cdl.cdl_qlinear_bwd_fp_workspace_bytes(M, N, K)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    i1, i2, q1, q2 = oracle.gradient_digits(G, absmax)
    dX = torch.empty((M, K), dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_bwd_fp(dev(torch, G), absmax, None, 0, None, dev(torch, W), N, w, M, N, K, dX, None, ws, nb)
    t = (oracle.gemm_dx(i1.astype(np.int8), W).astype(f32) * f32(q1 * f32(w.q)) +
         oracle.gemm_dx(i2.astype(np.int8), W).astype(f32) * f32(q2 * f32(w.q))).astype(f32)
    assert np.array_equal(dX.cpu().numpy(), t)
    dW = torch.empty((K, N), dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_bwd_fp(dev(torch, G), absmax, dev(torch, A), K, a, None, 0, None, M, N, K, None, dW, ws, nb)
    t = (oracle.gemm_dw(A, i1.astype(np.int8)).astype(f32) * f32(q1 * f32(a.q)) +
         oracle.gemm_dw(A, i2.astype(np.int8)).astype(f32) * f32(q2 * f32(a.q))).astype(f32)
    assert np.array_equal(dW.cpu().numpy(), t)


def test_convolution_form(torch):
    rng = np.random.default_rng(17)
    N, H, W, C, CO, R, S = 3, 10, 9, 128, 192, 3, 3
    X = (rng.integers(0, 16, (N, H, W, C)) * (rng.random((N, H, W, C)) < 0.6)).astype(np.uint8)
    Wt = rng.integers(-7, 8, (R * S * C, CO)).astype(np.int8)
    G = (rng.normal(0, 1e-2, (N, H, W, CO)) * rng.lognormal(0, 1, (N, H, W, CO))).astype(f32)
    absmax = float(np.abs(G).max())
    x, w = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7)
    shape = cdl.ConvShape(N, H, W, C, R, S)
    nb = cdl.cdl_qconv_bwd_fp_workspace_bytes(shape, CO)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    dX = torch.full((N, H, W, C), 7.0, dtype=torch.float32, device="cuda")
    dW = torch.full((R * S * C, CO), 7.0, dtype=torch.float32, device="cuda")
    cdl.cdl_qconv_bwd_fp(dev(torch, G), absmax, dev(torch, X), x, dev(torch, Wt), CO, w, shape, CO, dX, dW, ws, nb)
    torch.cuda.synchronize()
    assert cdl.cdl_workspace_status(ws, check=False) == 0
    i1, i2, q1, q2 = oracle.gradient_digits(G, absmax)
    I1, I2 = i1.astype(np.int8), i2.astype(np.int8)

    def combine(acc1, acc2, qb):
        return (acc1.astype(f32) * f32(q1 * f32(qb)) + acc2.astype(f32) * f32(q2 * f32(qb))).astype(f32)
    assert np.array_equal(dX.cpu().numpy(), combine(oracle.conv_dx(I1, Wt, X.shape, R, S, 1, 1), oracle.conv_dx(I2, Wt, X.shape, R, S, 1, 1), w.q))
    assert np.array_equal(dW.cpu().numpy(), combine(oracle.conv_dw(X, I1, R, S, 1, 1), oracle.conv_dw(X, I2, R, S, 1, 1), x.q))
