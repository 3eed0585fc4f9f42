"""GPU parity of the convolution products computed from the NHWC index tensors (patch matrix never stored)
against the CPU oracle's direct convolution: int32 accumulators bit-exact, float outputs equal to the accumulator
times the binary32 product of the steps."""
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


def scaled(acc, qa, qb, bias=None):
    y = acc.astype(f32) * f32(f32(qa) * f32(qb))
    if bias is not None:
        y = (y + bias.astype(f32)).astype(f32)
    return y


def make(seed, N, H, W, C, CO, R, S, unsigned=True, stride=1, ph=None, pw=None):
    rng = np.random.default_rng(seed)
    ph = (R - 1) // 2 if ph is None else ph
    pw = (S - 1) // 2 if pw is None else pw
    P, Q = oracle.conv_out_dims(H, W, R, S, ph, pw, stride)
    # activations: 4-bit indices with many zeros (post-ReLU); weights 15 levels; gradients 8-bit
    X = (rng.integers(0, 16, (N, H, W, C)) * (rng.random((N, H, W, C)) < 0.6)).astype(np.uint8) if unsigned \
        else rng.integers(-8, 8, (N, H, W, C)).astype(np.int8)
    Wt = rng.integers(-7, 8, (R * S * C, CO)).astype(np.int8)
    G = rng.integers(-127, 128, (N, P, Q, CO)).astype(np.int8)
    return X, Wt, G


def run_all(torch, X, Wt, G, R, S, unsigned=True, bias=None, stride=1, ph=None, pw=None):
    N, H, W, C = X.shape
    CO = Wt.shape[1]
    shape = cdl.ConvShape(N, H, W, C, R, S, stride, ph, pw)
    ph, pw = shape.pad_h, shape.pad_w
    P, Q = shape.P, shape.Q
    assert G.shape == (N, P, Q, CO)
    x = cdl.IndexDesc(0.25, 0, 15) if unsigned else cdl.IndexDesc(0.25, -8, 7)
    w, g = cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    nb = cdl.cdl_qconv_workspace_bytes(shape, CO)
    assert nb >= 256
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    Xd, Wd, Gd = dev(torch, X), dev(torch, Wt), dev(torch, G)
    acc = torch.full((N, P, Q, CO), -9, dtype=torch.int32, device="cuda")
    y = torch.full((N, P, Q, CO), float("nan"), dtype=torch.float32, device="cuda")
    bd = dev(torch, bias) if bias is not None else None
    cdl.cdl_qconv_fwd(Xd, x, Wd, CO, w, shape, CO, acc, y, bd, ws, nb)
    dxa = torch.full((N, H, W, C), -9, dtype=torch.int32, device="cuda")
    dx = torch.full((N, H, W, C), float("nan"), dtype=torch.float32, device="cuda")
    dwa = torch.full((R * S * C, CO), -9, dtype=torch.int32, device="cuda")
    dw = torch.full((R * S * C, CO), float("nan"), dtype=torch.float32, device="cuda")
    cdl.cdl_qconv_bwd(Gd, g, Xd, x, Wd, CO, w, shape, CO, dxa, dx, dwa, dw, ws, nb)
    torch.cuda.synchronize()
    assert cdl.cdl_workspace_status(ws, check=False) == 0
    ref = oracle.conv_fwd(X, Wt, R, S, ph, pw, stride)
    assert np.array_equal(acc.cpu().numpy(), ref.astype(np.int32))
    assert np.array_equal(y.cpu().numpy(), scaled(ref, x.q, w.q, bias))
    ref_dx = oracle.conv_dx(G, Wt, X.shape, R, S, ph, pw, stride)
    assert np.array_equal(dxa.cpu().numpy(), ref_dx.astype(np.int32))
    assert np.array_equal(dx.cpu().numpy(), scaled(ref_dx, g.q, w.q))
    ref_dw = oracle.conv_dw(X, G, R, S, ph, pw, stride)
    assert np.array_equal(dwa.cpu().numpy(), ref_dw.astype(np.int32))
    assert np.array_equal(dw.cpu().numpy(), scaled(ref_dw, g.q, x.q))


def test_one_tile_3x3(torch):
    # 128 pixels = one tile; every pixel row of the patch matrix crosses an image border somewhere
    X, Wt, G = make(1, 2, 8, 8, 128, 128, 3, 3)
    run_all(torch, X, Wt, G, 3, 3)


def test_cta_pair_tiles_3x3_exact_and_ragged(torch):
    X, Wt, G = make(2, 4, 8, 8, 128, 256, 3, 3)              # 256 pixels: one pair tile
    run_all(torch, X, Wt, G, 3, 3)
    X, Wt, G = make(3, 3, 10, 9, 256, 256, 3, 3)             # 270 pixels: ragged second tile, blocks straddle images
    run_all(torch, X, Wt, G, 3, 3, bias=np.linspace(-1, 1, 256).astype(f32))


def test_signed_activations_one_by_one_and_wide_filters(torch):
    X, Wt, G = make(4, 2, 7, 5, 128, 256, 1, 1, unsigned=False)
    run_all(torch, X, Wt, G, 1, 1, unsigned=False)
    X, Wt, G = make(5, 1, 9, 11, 128, 128, 5, 3)
    run_all(torch, X, Wt, G, 5, 3)
    X, Wt, G = make(6, 2, 6, 20, 128, 128, 3, 7)             # padding 3 along w: whole rows of zeros at the border
    run_all(torch, X, Wt, G, 3, 7)


def test_resnet_layer_geometry_14x14(torch):
    # the 14 x 14 images of the ResNet-18 layer this library is benchmarked on (fewer images): 128-pixel blocks
    # never line up with image rows, every block mixes several rows and images
    X, Wt, G = make(7, 6, 14, 14, 256, 256, 3, 3)
    run_all(torch, X, Wt, G, 3, 3)


@pytest.mark.parametrize("C,CO", [(64, 64), (64, 128), (192, 64), (128, 192), (320, 256),
                                  (64, 256), (256, 64)])     # 64-byte rows of X under a CTA pair: forward, and dX
def test_channel_counts_that_are_not_multiples_of_128(torch, C, CO):
    # a tap then fills its last 128-channel block only partly: the missing channels read as zero
    X, Wt, G = make(20 + C + CO, 3, 9, 10, C, CO, 3, 3)
    run_all(torch, X, Wt, G, 3, 3)


def test_resnet_layer1_geometry_sampled(torch):
    # 64 -> 64 channels on 56 x 56 images (ResNet-18 layer1), fewer images; whole images checked
    X, Wt, G = make(31, 8, 56, 56, 64, 64, 3, 3)
    run_all(torch, X, Wt, G, 3, 3)


@pytest.mark.parametrize("N,H,W,C,CO,R,S,stride,ph,pw", [
    (3, 12, 12, 64, 128, 3, 3, 2, 1, 1),      # the opener of a ResNet stage: 3 x 3, stride 2, padding 1
    (2, 14, 10, 128, 256, 3, 3, 2, 1, 1),
    (3, 7, 7, 256, 256, 3, 3, 2, 1, 1),       # odd image: the four pixel classes of the data gradient differ in size
    (3, 12, 12, 64, 128, 1, 1, 2, 0, 0),      # the 1 x 1 stride-2 shortcut: three of four input pixels get no gradient
    (2, 9, 11, 128, 64, 1, 1, 2, 0, 0),
    (2, 16, 16, 64, 64, 7, 7, 2, 3, 3),       # 7 x 7 stride 2 (49 taps)
    (2, 8, 8, 128, 128, 2, 2, 2, 0, 0),       # even filters: non-overlapping 2 x 2 patches
    (2, 10, 10, 64, 128, 4, 4, 2, 1, 1),
    (2, 13, 13, 128, 128, 3, 3, 3, 1, 1),     # stride 3: nine pixel classes
    (1, 17, 9, 64, 64, 5, 3, 4, 2, 0),        # stride 4, unequal padding
    (8, 24, 24, 64, 128, 3, 3, 2, 1, 1),      # large enough for 256-row tiles: scattered rows of the four classes, dW
    (9, 23, 25, 128, 64, 1, 1, 2, 0, 0),      # the same for the shortcut, ragged in every dimension
])
def test_strided_convolutions(torch, N, H, W, C, CO, R, S, stride, ph, pw):
    X, Wt, G = make(40 + H + R + stride, N, H, W, C, CO, R, S, stride=stride, ph=ph, pw=pw)
    run_all(torch, X, Wt, G, R, S, stride=stride, ph=ph, pw=pw)


@pytest.mark.parametrize("R,S,ph,pw", [(3, 3, 0, 0), (3, 3, 2, 2), (5, 5, 1, 3), (2, 2, 1, 0), (4, 4, 1, 1)])
def test_stride_one_with_other_paddings(torch, R, S, ph, pw):
    # no padding (the output shrinks), more than "same" padding (it grows), even filters
    X, Wt, G = make(50 + R + ph, 2, 9, 10, 128, 128, R, S, ph=ph, pw=pw)
    run_all(torch, X, Wt, G, R, S, ph=ph, pw=pw)


def test_resnet_stage_opener_and_shortcut_at_their_geometry(torch):
    # ResNet-18 layer2.0 (3 x 3, stride 2, 64 -> 128 channels on 56 x 56 images) and its 1 x 1 stride-2 shortcut, on
    # four images; float outputs only, compared over whole tensors
    for R, pad in ((3, 1), (1, 0)):
        N, H, W, C, CO = 4, 56, 56, 64, 128
        X, Wt, G = make(60 + R, N, H, W, C, CO, R, R, stride=2, ph=pad, pw=pad)
        shape = cdl.ConvShape(N, H, W, C, R, R, 2, pad, pad)
        x, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
        nb = cdl.cdl_qconv_workspace_bytes(shape, CO)
        ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
        Xd, Wd, Gd = dev(torch, X), dev(torch, Wt), dev(torch, G)
        y = torch.full((N, shape.P, shape.Q, CO), float("nan"), dtype=torch.float32, device="cuda")
        dx = torch.full((N, H, W, C), float("nan"), dtype=torch.float32, device="cuda")
        dw = torch.full((R * R * C, CO), float("nan"), dtype=torch.float32, device="cuda")
        cdl.cdl_qconv_fwd(Xd, x, Wd, CO, w, shape, CO, None, y, None, ws, nb)
        cdl.cdl_qconv_bwd(Gd, g, Xd, x, Wd, CO, w, shape, CO, None, dx, None, dw, ws, nb)
        torch.cuda.synchronize()
        assert cdl.cdl_workspace_status(ws, check=False) == 0
        assert np.array_equal(y.cpu().numpy(), scaled(oracle.conv_fwd(X, Wt, R, R, pad, pad, 2), x.q, w.q))
        assert np.array_equal(dx.cpu().numpy(), scaled(oracle.conv_dx(G, Wt, X.shape, R, R, pad, pad, 2), g.q, w.q))
        assert np.array_equal(dw.cpu().numpy(), scaled(oracle.conv_dw(X, G, R, R, pad, pad, 2), g.q, x.q))


def test_unsupported_shapes_are_refused(torch):
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    t = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    y = torch.zeros(1 << 16, dtype=torch.float32, device="cuda")
    x, w = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7)
    for shape, co in ((cdl.ConvShape(1, 4, 4, 32, 3, 3), 128), (cdl.ConvShape(1, 8, 8, 128, 8, 3), 128),
                      (cdl.ConvShape(1, 4, 4, 128, 3, 3), 96), (cdl.ConvShape(1, 9, 9, 128, 3, 3, stride=5), 128),
                      (cdl.ConvShape(1, 4, 4, 128, 3, 3, pad_h=3), 128), (cdl.ConvShape(1, 2, 2, 128, 5, 5, pad_h=1, pad_w=1), 128)):
        assert cdl.cdl_qconv_workspace_bytes(shape, co) == 0
        assert cdl.cdl_qconv_fwd(t, x, t, co, w, shape, co, None, y, None, ws, 1 << 20, check=False) == -1


def test_resnet18_layer3_full_size_sampled(torch):
    # the benchmarked geometry, 256 images of 14 x 14 x 256 -> 256 channels, in the launch configuration bench.py
    # times; the oracle computes whole images (forward, dX) and whole rows of dW chosen across taps and channels
    N, H, W, C, CO, R, S = 256, 14, 14, 256, 256, 3, 3
    X, Wt, G = make(8, N, H, W, C, CO, R, S)
    shape = cdl.ConvShape(N, H, W, C, R, S)
    x, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    nb = cdl.cdl_qconv_workspace_bytes(shape, CO)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    Xd, Wd, Gd = dev(torch, X), dev(torch, Wt), dev(torch, G)
    y = torch.empty((N, H, W, CO), dtype=torch.float32, device="cuda")
    dx = torch.empty((N, H, W, C), dtype=torch.float32, device="cuda")
    dw = torch.empty((R * S * C, CO), dtype=torch.float32, device="cuda")
    cdl.cdl_qconv_fwd(Xd, x, Wd, CO, w, shape, CO, None, y, None, ws, nb)
    cdl.cdl_qconv_bwd(Gd, g, Xd, x, Wd, CO, w, shape, CO, None, dx, None, dw, ws, nb)
    torch.cuda.synchronize()
    assert cdl.cdl_workspace_status(ws, check=False) == 0
    yh, dxh, dwh = y.cpu().numpy(), dx.cpu().numpy(), dw.cpu().numpy()
    for n in (0, 131, 255):
        assert np.array_equal(yh[n:n + 1], scaled(oracle.conv_fwd(X[n:n + 1], Wt, R, S, 1, 1), x.q, w.q))
        assert np.array_equal(dxh[n:n + 1], scaled(oracle.conv_dx(G[n:n + 1], Wt, (1, H, W, C), R, S, 1, 1), g.q, w.q))
    # rows k = (r*S + s)*C + c of dW: column k of the patch matrix is X shifted by the tap, zero outside
    ks = [0, 255, 256 + 17, 4 * 256 + 100, 5 * 256 + 255, 8 * 256, 8 * 256 + 255, 2 * 256 + 128]
    Xp = np.zeros((N, H + 2, W + 2, C), dtype=X.dtype)
    Xp[:, 1:H + 1, 1:W + 1, :] = X
    cols = np.stack([Xp[:, (k // C) // S:(k // C) // S + H, (k // C) % S:(k // C) % S + W, k % C].reshape(-1) for k in ks], axis=1)
    ref = oracle.gemm_dw(np.ascontiguousarray(cols), G.reshape(-1, CO))
    assert np.array_equal(dwh[ks], scaled(ref, g.q, x.q))
    # every entry of the three outputs was written (nothing left of the poison below would survive a re-run)
    assert np.isfinite(yh).all() and np.isfinite(dxh).all() and np.isfinite(dwh).all()
