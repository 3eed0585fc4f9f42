"""Layer products with few output channels (N in {4, 8, 16, 32}) take streaming integer-dot-product kernels instead
of tensor-core tiles.  Same contract as every other shape: the integer accumulators equal the oracle's exact
products (Sec. III: products of indices, rescaled by q_w q_a), the float outputs are their binary32 rescale."""
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


def pad_cols(a, mult=16):
    ld = (a.shape[1] + mult - 1) // mult * mult
    out = np.zeros((a.shape[0], ld), dtype=a.dtype)
    out[:, :a.shape[1]] = a
    return out, ld


# ragged M (not a multiple of 32 / 128), several row chunks, K with and without the staged path (K N + 256 K > 96 KB)
SHAPES = [(1, 16, 4), (33, 144, 16), (1000, 144, 16), (4099, 64, 8), (517, 256, 32), (2051, 576, 16), (700, 1024, 32),
          (260, 48, 4), (131, 2048, 16), (300, 20, 8), (50000, 272, 32)]


@pytest.mark.parametrize("M,K,N", SHAPES)
@pytest.mark.parametrize("signed_a", [False, True])
def test_skinny_products_match_oracle(torch, M, K, N, signed_a):
    rng = np.random.default_rng(1000 * N + K + M + int(signed_a))
    if signed_a:
        A = rng.integers(-127, 128, (M, K)).astype(np.int8)
        a = cdl.IndexDesc(0.125, -127, 127)
    else:
        A = rng.integers(0, 256, (M, K)).astype(np.uint8)
        a = cdl.IndexDesc(0.125, 0, 255)
    W = rng.integers(-127, 128, (K, N)).astype(np.int8)
    G = rng.integers(-127, 128, (M, N)).astype(np.int8)
    w, g = cdl.IndexDesc(0.03125, -127, 127), cdl.IndexDesc(0.0078125, -127, 127)
    bias = rng.normal(0, 1.0, N).astype(f32)
    Ap, lda = pad_cols(A)
    Wp, ldw = pad_cols(W)
    Gp, ldg = pad_cols(G)
    nb = max(cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K), cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K))
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    dA, dW_, dG = dev(torch, Ap), dev(torch, Wp), dev(torch, Gp)

    acc = torch.full((M, N), -1, dtype=torch.int32, device="cuda")
    y = torch.full((M, N), -1.0, dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_fwd(dA, lda, a, dW_, ldw, w, M, N, K, acc, y, dev(torch, bias), ws, nb)
    cdl.cdl_workspace_status(ws)
    ref = oracle.gemm_fwd(A, W)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), ref)
    y_ref = (ref.astype(f32) * f32(f32(a.q) * f32(w.q)) + bias).astype(f32)
    assert np.array_equal(y.cpu().numpy(), y_ref)
    # float output alone, no bias
    y2 = torch.full((M, N), -1.0, dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_fwd(dA, lda, a, dW_, ldw, w, M, N, K, None, y2, None, ws, nb)
    assert np.array_equal(y2.cpu().numpy(), ref.astype(f32) * f32(f32(a.q) * f32(w.q)))

    dxa = torch.full((M, K), -1, dtype=torch.int32, device="cuda")
    dx = torch.full((M, K), -1.0, dtype=torch.float32, device="cuda")
    dwa = torch.full((K, N), -1, dtype=torch.int32, device="cuda")
    dw = torch.full((K, N), -1.0, dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_bwd(dG, ldg, g, dA, lda, a, dW_, ldw, w, M, N, K, dxa, dx, dwa, dw, ws, nb)
    cdl.cdl_workspace_status(ws)
    rdx, rdw = oracle.gemm_dx(G, W), oracle.gemm_dw(A, G)
    assert np.array_equal(dxa.cpu().numpy().astype(np.int64), rdx)
    assert np.array_equal(dwa.cpu().numpy().astype(np.int64), rdw)
    assert np.array_equal(dx.cpu().numpy(), rdx.astype(f32) * f32(f32(g.q) * f32(w.q)))
    assert np.array_equal(dw.cpu().numpy(), rdw.astype(f32) * f32(f32(g.q) * f32(a.q)))
    # float outputs alone (dW then accumulates in the workspace)
    dx2 = torch.full((M, K), -1.0, dtype=torch.float32, device="cuda")
    dw2 = torch.full((K, N), -1.0, dtype=torch.float32, device="cuda")
    cdl.cdl_qlinear_bwd(dG, ldg, g, dA, lda, a, dW_, ldw, w, M, N, K, None, dx2, None, dw2, ws, nb)
    cdl.cdl_workspace_status(ws)
    assert np.array_equal(dx2.cpu().numpy(), dx.cpu().numpy())
    assert np.array_equal(dw2.cpu().numpy(), dw.cpu().numpy())


def test_skinny_rows_with_a_leading_dimension_wider_than_the_matrix(torch):
    """Columns beyond K (of A), N (of W, G) inside the leading dimension hold junk that no product may read."""
    M, K, N = 777, 144, 16
    rng = np.random.default_rng(5)
    lda, ldw, ldg = 176, 48, 32
    Ap = rng.integers(0, 16, (M, lda)).astype(np.uint8)
    Wp = rng.integers(-7, 8, (K, ldw)).astype(np.int8)
    Gp = rng.integers(-127, 128, (M, ldg)).astype(np.int8)
    A, W, G = Ap[:, :K], Wp[:, :N], Gp[:, :N]
    a, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(0.001, -127, 127)
    nb = max(cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K), cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K))
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    dxa = torch.empty((M, K), dtype=torch.int32, device="cuda")
    dwa = torch.empty((K, N), dtype=torch.int32, device="cuda")
    cdl.cdl_qlinear_fwd(dev(torch, Ap), lda, a, dev(torch, Wp), ldw, w, M, N, K, acc, None, None, ws, nb)
    cdl.cdl_qlinear_bwd(dev(torch, Gp), ldg, g, dev(torch, Ap), lda, a, dev(torch, Wp), ldw, w, M, N, K, dxa, None, dwa,
                        None, ws, nb)
    cdl.cdl_workspace_status(ws)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), oracle.gemm_fwd(A, W))
    assert np.array_equal(dxa.cpu().numpy().astype(np.int64), oracle.gemm_dx(G, W))
    assert np.array_equal(dwa.cpu().numpy().astype(np.int64), oracle.gemm_dw(A, G))
