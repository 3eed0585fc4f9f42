"""The forward products' fused output: the hard index of the next layer's quantizer must be, byte for byte, what
quantizing the float output gives (oracle: exact product -> binary32 rescale (+ bias) -> hard index)."""
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


def ref_index(acc, qa, qw, bias, nq, lo, hi):
    y = acc.astype(f32) * f32(f32(qa) * f32(qw))
    if bias is not None:
        y = (y + bias.astype(f32)).astype(f32)
    idx, _ = oracle.hard(y.reshape(-1), f32(nq), lo, hi)
    return y, idx.reshape(acc.shape)


@pytest.mark.parametrize("M,K,N,lo,hi", [(300, 520, 256, 0, 15), (130, 144, 48, -7, 7), (64, 256, 128, 0, 255),
                                         (257, 160, 20, 0, 15),
                                         (900, 320, 64, 0, 15), (1300, 144, 112, -7, 7)])    # 256-row tiles of one CTA
def test_linear_forward_emits_the_next_layers_index(torch, M, K, N, lo, hi):
    rng = np.random.default_rng(M + N)
    A = rng.integers(0, 16, (M, K)).astype(np.uint8)
    W = rng.integers(-7, 8, (K, N)).astype(np.int8)
    bias = rng.normal(0, 2.0, N).astype(f32)
    a, w = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7)
    # a step that makes many outputs land on or next to rounding ties: products are multiples of 0.005
    nq = 0.25 if hi != 255 else 0.05
    nxt = cdl.IndexDesc(nq, lo, hi)
    ldw = (N + 15) // 16 * 16
    Wp = np.zeros((K, ldw), dtype=np.int8)
    Wp[:, :N] = W
    lda = (K + 15) // 16 * 16
    Ap = np.zeros((M, lda), dtype=np.uint8)
    Ap[:, :K] = A
    nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    acc_ref = oracle.gemm_fwd(A, W)
    for use_bias, want_y in ((False, False), (True, True)):
        b = bias if use_bias else None
        y = torch.empty((M, N), dtype=torch.float32, device="cuda") if want_y else None
        idx = torch.full((M, N), 99, dtype=torch.int8 if lo < 0 else torch.uint8, device="cuda")
        cdl.cdl_qlinear_fwd_next(dev(torch, Ap), lda, a, dev(torch, Wp), ldw, w, M, N, K, nxt, idx,
                                 y_out=y, bias=dev(torch, b) if use_bias else None, ws=ws, ws_bytes=nb)
        torch.cuda.synchronize()
        y_ref, idx_ref = ref_index(acc_ref, a.q, w.q, b, nq, lo, hi)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), idx_ref)
        if want_y:
            assert np.array_equal(y.cpu().numpy(), y_ref)
    assert cdl.cdl_workspace_status(ws, check=False) == 0


def test_convolution_forward_emits_the_next_layers_index(torch):
    rng = np.random.default_rng(9)
    N, H, W, C, CO, R, S = 3, 10, 9, 128, 256, 3, 3
    X = (rng.integers(0, 16, (N, H, W, C)) * (rng.random((N, H, W, C)) < 0.6)).astype(np.uint8)
    Wt = rng.integers(-7, 8, (R * S * C, CO)).astype(np.int8)
    x, w, nxt = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(0.5, 0, 15)
    shape = cdl.ConvShape(N, H, W, C, R, S)
    nb = cdl.cdl_qconv_workspace_bytes(shape, CO)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    idx = torch.full((N, H, W, CO), 99, dtype=torch.uint8, device="cuda")
    cdl.cdl_qconv_fwd_next(dev(torch, X), x, dev(torch, Wt), CO, w, shape, CO, nxt, idx, ws=ws, ws_bytes=nb)
    torch.cuda.synchronize()
    assert cdl.cdl_workspace_status(ws, check=False) == 0
    _, idx_ref = ref_index(oracle.conv_fwd(X, Wt, R, S, 1, 1), x.q, w.q, None, nxt.q, 0, 15)
    got = idx.cpu().numpy().astype(np.int64)
    assert np.array_equal(got, idx_ref)
    assert (got == 0).mean() > 0.3 and (got == 15).any()          # the clamp at 0 acts as the ReLU; the range is used
