"""GPU parity of the index GEMMs (forward, dX, dW) against the CPU oracle: int32 accumulators bit-exact,
float outputs equal to the accumulator times the binary32 product of the steps."""
import numpy as np
import pytest

import oracle
import paper_2501_09849_b200 as cdl
from paper_2501_09849_b200 import inputs

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


def ld16(n):
    return (n + 15) // 16 * 16


def run_fwd(torch, A, W, a, w, bias=None, want_acc=True, want_y=True):
    M, K = A.shape
    N = W.shape[1]
    lda, ldw = ld16(K), ld16(N)
    Ad, Wd = dev(torch, padded(A, lda)), dev(torch, padded(W, ldw))
    acc = torch.full((M, N), -7, dtype=torch.int32, device="cuda") if want_acc else None
    y = torch.full((M, N), -7.0, dtype=torch.float32, device="cuda") if want_y else None
    nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K)
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    bd = None if bias is None else dev(torch, bias)
    cdl.cdl_qlinear_fwd(Ad, lda, a, Wd, ldw, w, M, N, K, acc, y, bd, ws, nb)
    cdl.cdl_workspace_status(ws)
    return (None if acc is None else acc.cpu().numpy()), (None if y is None else y.cpu().numpy())


def run_bwd(torch, G, A, W, g, a, w, want=("dXacc", "dX", "dWacc", "dW")):
    M, N = G.shape
    K = A.shape[1] if A is not None else W.shape[0]
    ldg, lda, ldw = ld16(N), ld16(K), ld16(N)
    Gd = dev(torch, padded(G, ldg))
    Ad = None if A is None else dev(torch, padded(A, lda))
    Wd = None if W is None else dev(torch, padded(W, ldw))
    out = {}
    if "dXacc" in want:
        out["dXacc"] = torch.full((M, K), -7, dtype=torch.int32, device="cuda")
    if "dX" in want:
        out["dX"] = torch.full((M, K), -7.0, dtype=torch.float32, device="cuda")
    if "dWacc" in want:
        out["dWacc"] = torch.full((K, N), -7, dtype=torch.int32, device="cuda")
    if "dW" in want:
        out["dW"] = torch.full((K, N), -7.0, dtype=torch.float32, device="cuda")
    nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K)
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    cdl.cdl_qlinear_bwd(Gd, ldg, g, Ad, lda, a, Wd, ldw, w, M, N, K, out.get("dXacc"), out.get("dX"),
                        out.get("dWacc"), out.get("dW"), ws, nb)
    cdl.cdl_workspace_status(ws)
    return {k: v.cpu().numpy() for k, v in out.items()}


def scaled(acc, qa, qb, bias=None):
    s = f32(qa) * f32(qb)                       # product of the steps formed once in binary32
    y = acc.astype(f32) * s                     # int32 -> binary32 (round to nearest), one binary32 multiply
    if bias is not None:
        y = y + bias.astype(f32)[None, :]
    return y


def check_all_products(torch, A, W, G, a, w, g):
    ref_f = oracle.gemm_fwd(A, W)
    ref_x = oracle.gemm_dx(G, W)
    ref_w = oracle.gemm_dw(A, G)
    for r in (ref_f, ref_x, ref_w):
        assert np.abs(r).max() < 2 ** 31
    acc, y = run_fwd(torch, A, W, a, w)
    assert np.array_equal(acc.astype(np.int64), ref_f)
    assert np.array_equal(y, scaled(ref_f, a.q, w.q))
    out = run_bwd(torch, G, A, W, g, a, w)
    assert np.array_equal(out["dXacc"].astype(np.int64), ref_x)
    assert np.array_equal(out["dWacc"].astype(np.int64), ref_w)
    assert np.array_equal(out["dX"], scaled(ref_x, g.q, w.q))
    assert np.array_equal(out["dW"], scaled(ref_w, g.q, a.q))


def test_tiny_layer_products_from_quantized_tensors(torch):
    # the whole tiny layer: quantize on the GPU, multiply the GPU's own indices, compare with the oracle chain
    case, wt, at = inputs.tiny_layer(seed=0)
    M, K, N = case.M, case.K, case.N
    ref_wi, _ = oracle.hard(wt, f32(case.wq.q), case.wq.lo, case.wq.hi)
    ref_ai, _ = oracle.hard(at, f32(case.aq.q), case.aq.lo, case.aq.hi)
    gt = inputs.normal((M, N), 1e-2, seed=0, stream=9)
    qg = float(f32(np.abs(gt).max() / 127.0))
    ref_gi, _ = oracle.hard(gt, f32(qg), -127, 127)
    wi = torch.empty((K, N), dtype=torch.int8, device="cuda")
    ai = torch.empty((M, K), dtype=torch.uint8, device="cuda")
    gi = torch.empty((M, N), dtype=torch.int8, device="cuda")
    cdl.cdl_quantize_hard(dev(torch, wt), wt.size, cdl.QuantParams(case.wq.q, case.wq.lo, case.wq.hi), wi)
    cdl.cdl_quantize_hard(dev(torch, at), at.size, cdl.QuantParams(case.aq.q, case.aq.lo, case.aq.hi), ai)
    cdl.cdl_quantize_hard(dev(torch, gt), gt.size, cdl.QuantParams(qg, -127, 127), gi)
    A, W, G = ai.cpu().numpy(), wi.cpu().numpy(), gi.cpu().numpy()
    assert np.array_equal(A, ref_ai.astype(np.uint8)) and np.array_equal(W, ref_wi.astype(np.int8))
    assert np.array_equal(G, ref_gi.astype(np.int8))
    a, w, g = cdl.IndexDesc(case.aq.q, 0, 15), cdl.IndexDesc(case.wq.q, -7, 7), cdl.IndexDesc(qg, -127, 127)
    check_all_products(torch, A, W, G, a, w, g)
    bias = inputs.normal((N,), 1.0, seed=3)
    _, y = run_fwd(torch, A, W, a, w, bias=bias, want_acc=False)
    assert np.array_equal(y, scaled(oracle.gemm_fwd(A, W), a.q, w.q, bias))


@pytest.mark.parametrize("M,K,N", [(1, 16, 16), (5, 20, 7), (130, 147, 64), (257, 144, 16), (300, 520, 130),
                                   (64, 2304, 256), (1000, 64, 1000),
                                   # 256-row tiles of one CTA (at most 128 output columns, at least 512 rows), ragged
                                   # in every dimension: forward and dW of the first, forward of the other two, and
                                   # dX / dW of the last (640 and 1152 rows of the transposed operand)
                                   (1000, 640, 64), (2048 + 77, 200, 128), (700, 1152, 96)])
def test_ragged_shapes_and_signedness(torch, M, K, N):
    for a_lo, a_hi in ((0, 255), (-128, 127), (0, 15)):
        A = inputs.uniform_indices((M, K), a_lo, a_hi, seed=M + K)
        W = inputs.uniform_indices((K, N), -128, 127, seed=N + 1)
        G = inputs.uniform_indices((M, N), -127, 127, seed=M + 2)
        a, w, g = cdl.IndexDesc(0.25, a_lo, a_hi), cdl.IndexDesc(0.02, -128, 127), cdl.IndexDesc(1e-3, -127, 127)
        check_all_products(torch, A, W, G, a, w, g)


def test_optional_outputs_and_operands(torch):
    M, K, N = 70, 96, 40
    A = inputs.uniform_indices((M, K), 0, 15, seed=1)
    W = inputs.uniform_indices((K, N), -7, 7, seed=2)
    G = inputs.uniform_indices((M, N), -127, 127, seed=3)
    a, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    acc, y = run_fwd(torch, A, W, a, w, want_y=False)
    assert y is None and np.array_equal(acc.astype(np.int64), oracle.gemm_fwd(A, W))
    out = run_bwd(torch, G, None, W, g, None, w, want=("dX",))
    assert np.array_equal(out["dX"], scaled(oracle.gemm_dx(G, W), g.q, w.q))
    out = run_bwd(torch, G, A, None, g, a, None, want=("dWacc",))
    assert np.array_equal(out["dWacc"].astype(np.int64), oracle.gemm_dw(A, G))


def test_cifar_resnet20_conv_shape_full_compare(torch):
    # (M, K, N) = (131072, 144, 16): operands drawn from the quantized tensors' own level histograms
    case, wt, at = inputs.cifar_resnet20_conv()
    M, K, N = case.M, case.K, case.N
    wi, _ = oracle.hard(wt, f32(case.wq.q), case.wq.lo, case.wq.hi)
    _, ah = oracle.hard(at, f32(case.aq.q), case.aq.lo, case.aq.hi)
    A = inputs.indices_from_histogram((M, K), ah, 0, seed=case.seed, stream=3)
    W = wi.astype(np.int8)
    G = inputs.uniform_indices((M, N), -127, 127, seed=case.seed, stream=4)
    a, w, g = cdl.IndexDesc(case.aq.q, 0, 15), cdl.IndexDesc(case.wq.q, -1, 1), cdl.IndexDesc(1e-3, -127, 127)
    check_all_products(torch, A, W, G, a, w, g)


def test_resnet18_layer3_shape_sampled_compare(torch):
    # (M, K, N) = (50176, 2304, 256) in the launch configuration the benchmark times.  The oracle checks
    # whole rows of the forward / dX outputs (both M edges and rows spread over every tile row) and, for dW
    # (which reduces over all of M), whole K x N sub-blocks spread over every tile of the output.
    case, wt, at = inputs.resnet18_layer3_conv()
    M, K, N = case.M, case.K, case.N
    wi, _ = oracle.hard(wt, f32(case.wq.q), case.wq.lo, case.wq.hi)
    _, ah = oracle.hard(at[:8], f32(case.aq.q), case.aq.lo, case.aq.hi)
    A = inputs.indices_from_histogram((M, K), ah, 0, seed=case.seed, stream=3)
    W = wi.astype(np.int8)
    G = inputs.uniform_indices((M, N), -127, 127, seed=case.seed, stream=4)
    a, w, g = cdl.IndexDesc(case.aq.q, 0, 15), cdl.IndexDesc(case.wq.q, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    acc, y = run_fwd(torch, A, W, a, w)
    out = run_bwd(torch, G, A, W, g, a, w)
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([np.arange(0, 3), np.arange(M - 3, M), np.arange(125, 131),
                                     rng.integers(0, M, size=180)]))
    ref_f = oracle.gemm_fwd(A[rows], W)
    assert np.array_equal(acc[rows].astype(np.int64), ref_f)
    assert np.array_equal(y[rows], scaled(ref_f, a.q, w.q))
    ref_x = oracle.gemm_dx(G[rows], W)
    assert np.array_equal(out["dXacc"][rows].astype(np.int64), ref_x)
    assert np.array_equal(out["dX"][rows], scaled(ref_x, g.q, w.q))
    ks = np.unique(np.concatenate([np.arange(0, 2), np.arange(K - 2, K), np.arange(127, 129), rng.integers(0, K, size=40)]))
    ns = np.unique(np.concatenate([np.arange(0, 2), np.arange(N - 2, N), rng.integers(0, N, size=20)]))
    ref_w = oracle.gemm_dw(np.ascontiguousarray(A[:, ks]), np.ascontiguousarray(G[:, ns]))
    assert np.array_equal(out["dWacc"][np.ix_(ks, ns)].astype(np.int64), ref_w)
    assert np.array_equal(out["dW"][np.ix_(ks, ns)], scaled(ref_w, g.q, a.q))
    # properties that hold at any size: column sums of the forward accumulators
    colsum = A.astype(np.int64).sum(axis=0) @ W.astype(np.int64)
    assert np.array_equal(acc.astype(np.int64).sum(axis=0), colsum)


def test_long_reduction_beyond_int32_is_summed_exactly(torch):
    # dW over M rows whose worst-case (and, for the constant operands, actual) total exceeds 2^31: the float output
    # must equal float(int64 sum) * scale; asking for the int32 accumulators is refused.
    M, K, N = 70001, 160, 48
    a, g = cdl.IndexDesc(0.25, 0, 255), cdl.IndexDesc(1e-3, -127, 127)
    for kind in ("constant", "random"):
        if kind == "constant":
            A = np.full((M, K), 255, dtype=np.uint8)
            G = np.full((M, N), 127, dtype=np.int8)
            G[:, 1::2] = -127
        else:
            A = inputs.uniform_indices((M, K), 0, 255, seed=11)
            G = inputs.uniform_indices((M, N), -127, 127, seed=12)
        ref = oracle.gemm_dw(A, G)
        if kind == "constant":
            assert np.abs(ref).max() >= 2 ** 31
        out = run_bwd(torch, G, A, None, g, a, None, want=("dW",))
        assert np.array_equal(out["dW"], scaled(ref, g.q, a.q))
    ldg, lda = ld16(N), ld16(K)
    nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K)
    buf = torch.zeros(max(nb, M * lda), dtype=torch.uint8, device="cuda")
    rc = cdl.cdl_qlinear_bwd(buf, ldg, g, buf, lda, a, None, ldg, None, M, N, K, None, None, buf, None, buf, nb, check=False)
    assert rc == -5


def test_resnet18_conv1_and_fc_shapes(torch):
    # ResNet-18's first conv as an im2col GEMM at batch 16 (M = 16*112*112, K = 147 padded to a pitch of 160,
    # N = 64) with 8-bit activation indices (first layer kept at 8 bits, Sec. VI-B.2): dW reduces over 200704 rows,
    # beyond what int32 guarantees, so only its float output exists.  And the FC layer (256, 512, 1000 -> pitch 1008).
    M, K, N = 16 * 112 * 112, 147, 64
    A = inputs.uniform_indices((M, K), 0, 255, seed=21)
    W = inputs.uniform_indices((K, N), -3, 3, seed=22)
    G = inputs.uniform_indices((M, N), -127, 127, seed=23)
    a, w, g = cdl.IndexDesc(0.02, 0, 255), cdl.IndexDesc(0.05, -3, 3), cdl.IndexDesc(1e-3, -127, 127)
    acc, y = run_fwd(torch, A, W, a, w)
    out = run_bwd(torch, G, A, W, g, a, w, want=("dX", "dW"))
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([np.arange(0, 2), np.arange(M - 2, M), np.arange(127, 130), rng.integers(0, M, size=300)]))
    ref_f = oracle.gemm_fwd(A[rows], W)
    assert np.array_equal(acc[rows].astype(np.int64), ref_f) and np.array_equal(y[rows], scaled(ref_f, a.q, w.q))
    assert np.array_equal(out["dX"][rows], scaled(oracle.gemm_dx(G[rows], W), g.q, w.q))
    ks = np.unique(np.concatenate([[0, 1, 127, 128, 145, 146], rng.integers(0, K, size=10)]))
    ref_w = oracle.gemm_dw(np.ascontiguousarray(A[:, ks]), G)
    assert np.array_equal(out["dW"][ks], scaled(ref_w, g.q, a.q))
    # FC layer
    M, K, N = 256, 512, 1000
    A = inputs.uniform_indices((M, K), 0, 15, seed=24)
    W = inputs.uniform_indices((K, N), -3, 3, seed=25)
    G = inputs.uniform_indices((M, N), -127, 127, seed=26)
    check_all_products(torch, A, W, G, cdl.IndexDesc(0.25, 0, 15), w, g)


def test_float_only_outputs_with_a_ragged_last_round_of_tiles(torch):
    # 89 x 2 tiles of 256 x 256 on 74 CTA-pair slots: two whole rounds and 30 tiles left over, ragged in all three
    # dimensions, float output only.  Every element of the float output must equal the int32 accumulators of a
    # second run times the step product, bit for bit; the accumulators themselves are compared with the oracle on
    # rows of the last round's tiles (the last 15 tile rows), of the earlier rounds and of both edges.  A bias goes
    # through the same path; repeated calls on the same buffers give the same bits.
    M, K, N = 89 * 256 - 100, 1584, 384
    A = inputs.uniform_indices((M, K), 0, 15, seed=61)
    W = inputs.uniform_indices((K, N), -7, 7, seed=62)
    G = inputs.uniform_indices((M, N), -127, 127, seed=63)
    a, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    bias = inputs.normal((N,), 1.0, seed=64)
    acc, _ = run_fwd(torch, A, W, a, w, want_y=False)
    for rep in range(2):
        _, y = run_fwd(torch, A, W, a, w, want_acc=False)
        assert np.array_equal(y, scaled(acc.astype(np.int64), a.q, w.q)), rep
    _, yb = run_fwd(torch, A, W, a, w, bias=bias, want_acc=False)
    assert np.array_equal(yb, scaled(acc.astype(np.int64), a.q, w.q, bias))
    rng = np.random.default_rng(2)
    rows = np.unique(np.concatenate([np.arange(0, 3), np.arange(M - 3, M), np.arange(74 * 256 - 2, 74 * 256 + 2),
                                     rng.integers(74 * 256, M, size=200), rng.integers(0, 74 * 256, size=100)]))
    assert np.array_equal(acc[rows].astype(np.int64), oracle.gemm_fwd(A[rows], W))
    # dX of the same shape family: (M, N) x (K, N)^T with K = 512 -> 89 x 2 tiles again, reduced dimension N = 1584
    M2, N2, K2 = M, 1584, 512
    G2 = inputs.uniform_indices((M2, N2), -127, 127, seed=65)
    W2 = inputs.uniform_indices((K2, N2), -7, 7, seed=66)
    full = run_bwd(torch, G2, None, W2, g, None, w, want=("dXacc",))["dXacc"]
    only = run_bwd(torch, G2, None, W2, g, None, w, want=("dX",))["dX"]
    assert np.array_equal(only, scaled(full.astype(np.int64), g.q, w.q))
    assert np.array_equal(full[rows].astype(np.int64), oracle.gemm_dx(G2[rows], W2))


@pytest.mark.parametrize("M,K,N", [(4096 + 5, 640, 512), (300, 2304, 256), (50176, 256, 272), (1031, 1152, 1000)])
def test_float_only_outputs_with_fewer_tiles_than_slots(torch, M, K, N):
    # Products with fewer 256 x 256 tiles than CTA-pair slots and float outputs only: the reduced dimension is split
    # over the slots (the weight gradient reduces over M with a handful of tiles); all three products against the oracle.
    A = inputs.uniform_indices((M, K), 0, 15, seed=M % 97)
    W = inputs.uniform_indices((K, N), -7, 7, seed=K % 97)
    G = inputs.uniform_indices((M, N), -127, 127, seed=N % 97)
    a, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    _, y = run_fwd(torch, A, W, a, w, want_acc=False)
    out = run_bwd(torch, G, A, W, g, a, w, want=("dX", "dW"))
    if M * K * N <= 3e9:
        assert np.array_equal(y, scaled(oracle.gemm_fwd(A, W), a.q, w.q))
        assert np.array_equal(out["dX"], scaled(oracle.gemm_dx(G, W), g.q, w.q))
        assert np.array_equal(out["dW"], scaled(oracle.gemm_dw(A, G), g.q, a.q))
    else:
        rng = np.random.default_rng(3)
        rows = np.unique(np.concatenate([np.arange(0, 2), np.arange(M - 2, M), rng.integers(0, M, size=200)]))
        assert np.array_equal(y[rows], scaled(oracle.gemm_fwd(A[rows], W), a.q, w.q))
        assert np.array_equal(out["dX"][rows], scaled(oracle.gemm_dx(G[rows], W), g.q, w.q))
        ks = np.unique(np.concatenate([[0, 1, K - 1], rng.integers(0, K, size=12)]))
        assert np.array_equal(out["dW"][ks], scaled(oracle.gemm_dw(np.ascontiguousarray(A[:, ks]), G), g.q, a.q))


def test_step_replayed_from_a_cuda_graph_equals_the_step_launched_call_by_call(torch):
    # the recorded step must write exactly what the eager step writes (same kernels, same launch shapes); the
    # products themselves are checked against the oracle above
    from paper_2501_09849_b200.layer import CdlLayerStep
    case, wt, at = inputs.tiny_layer(seed=4)
    M, K, N = case.M, case.K, case.N
    step = CdlLayerStep(torch, M, K, N, at.size, case.wq, case.aq, q_g=1e-3)
    step.w.copy_(dev(torch, wt).reshape(-1))
    step.x.copy_(dev(torch, at).reshape(-1))
    ai, _ = oracle.hard(at, f32(case.aq.q), case.aq.lo, case.aq.hi)
    step.A_idx[:, :K].copy_(dev(torch, ai.astype(np.uint8).reshape(M, K)))
    step.dY.copy_(dev(torch, inputs.normal((M, N), 3e-2, seed=4, stream=7)))
    step.gx_in.copy_(dev(torch, inputs.normal((at.size,), 1e-2, seed=4, stream=8)))
    outs = ("w_soft", "W_idx", "x_soft", "X_idx", "hist_w", "hist_x", "prob_w", "prob_x", "Y", "G_idx", "dA", "dW",
            "dx", "dw")

    def snapshot():
        torch.cuda.synchronize()
        return {k: getattr(step, k).clone() for k in outs}

    def clear():
        step.hist_w.zero_()
        step.hist_x.zero_()
        step.scalars.zero_()

    clear()
    step.run()
    eager = snapshot()
    eager_scalars = step.scalars.clone()
    graph = step.capture()
    for _ in range(2):
        for k in outs:
            getattr(step, k).zero_()
        clear()
        graph.replay()
        got = snapshot()
        for k in outs:
            assert torch.equal(got[k], eager[k]), k
        # entropies are pure functions of the histograms; the four gradient scalars are sums of float64 atomics
        assert torch.equal(step.scalars[:2], eager_scalars[:2])
        assert torch.allclose(step.scalars[2:], eager_scalars[2:], rtol=1e-9, atol=1e-12)
    assert cdl.cdl_workspace_status(step.ws, check=False) == 0


class _LoopbackCollective:
    """Stands in for torch.distributed on one GPU: two ranks run one after the other.  In the recording pass every
    tensor a rank hands to all_reduce is stored; in the second pass all_reduce returns the sum over both ranks."""

    class ReduceOp:
        SUM = "sum"

    def __init__(self):
        self.recorded, self.total, self.slot = {}, None, 0

    def all_reduce(self, t, op=None):
        key = self.slot
        self.slot += 1
        if self.total is None:
            self.recorded.setdefault(key, []).append(t.clone())
        else:
            t.copy_(self.total[key])


def test_two_row_blocks_with_the_exchange_equal_the_whole_batch(torch):
    # the data-parallel step on one GPU: the batch rows are split in two blocks, each block runs the real kernels
    # through CdlLayerStep.run(exchange=...), and what the exchange hands over is the sum of both blocks.  Histogram,
    # entropy, level probabilities, dW, dL/dw and every row of dL/dx must be the bits of the whole-batch step.
    from paper_2501_09849_b200 import sharding
    from paper_2501_09849_b200.layer import CdlLayerStep
    case, wt, at = inputs.tiny_layer(seed=6)
    M, K, N = case.M, case.K, case.N
    case.aq.window = 5
    ai = oracle.hard(at, f32(case.aq.q), case.aq.lo, case.aq.hi)[0].astype(np.uint8).reshape(M, K)
    dY = inputs.normal((M, N), 3e-2, seed=6, stream=7)
    gx = inputs.normal((M, K), 1e-2, seed=6, stream=8)

    def make(r0, r1):
        st = CdlLayerStep(torch, r1 - r0, K, N, (r1 - r0) * K, case.wq, case.aq, q_g=1e-3)
        st.w.copy_(dev(torch, wt).reshape(-1))
        st.x.copy_(dev(torch, at[r0:r1]).reshape(-1))
        st.A_idx[:, :K].copy_(dev(torch, ai[r0:r1]))
        st.dY.copy_(dev(torch, dY[r0:r1]))
        st.gx_in.copy_(dev(torch, gx[r0:r1]).reshape(-1))
        return st

    whole = make(0, M)
    whole.run()
    blocks = [sharding.row_range(M, r, 2) for r in range(2)]
    parts = [make(r0, r1) for r0, r1 in blocks]
    link = _LoopbackCollective()
    for st in parts:                      # recording pass: what each rank would send
        link.slot = 0
        st.run(exchange=sharding.StepExchange(link, 2), rows_global=M)
    torch.cuda.synchronize()
    # the last recorded tensor (the two batch scalars) depends on the exchanged probabilities: take it from pass two
    link.total = {k: v[0] + v[1] for k, v in link.recorded.items()}
    scal = []
    for st in parts:
        link.slot = 0
        ex = sharding.StepExchange(link, 2)
        st.scalars.zero_()
        orig = ex.batch_scalars
        ex.batch_scalars = lambda t, orig=orig: scal.append(t.clone())      # summed by hand below
        st.run(exchange=ex, rows_global=M)
        assert [c[0] for c in ex.calls] == ["histogram", "accumulators"] and [c[1] for c in ex.calls] == ["int64", "int32"]
    torch.cuda.synchronize()
    for st in parts:
        for k in ("hist_x", "prob_x", "dW", "dw", "hist_w", "prob_w", "W_idx"):
            assert torch.equal(getattr(st, k), getattr(whole, k)), k
        assert torch.equal(st.scalars[:4], whole.scalars[:4]) or torch.allclose(st.scalars[2:4], whole.scalars[2:4], rtol=1e-12)
        assert torch.equal(st.scalars[:2], whole.scalars[:2])            # H(w) and H(x) of the whole batch, never a sum
    assert torch.equal(torch.cat([st.dx for st in parts]), whole.dx)
    assert torch.equal(torch.cat([st.Y for st in parts]), whole.Y)
    assert torch.allclose(scal[0] + scal[1], whole.scalars[4:6], rtol=1e-11, atol=1e-14)


def test_convolution_form_step_graph_equals_call_by_call(torch):
    # the three-stream recording of the step in convolution form has its own dependencies (the forward product waits
    # for X_idx, the activation backward pass for the data gradient): it must write what the serial step writes
    from paper_2501_09849_b200.layer import CdlLayerStep
    n_img, H, W, C, CO = 4, 8, 8, 128, 128
    M, K = n_img * H * W, 9 * C
    wq = inputs.Quantizer(0.02, -7, 7, 80.0, 0.01, 0)
    xq = inputs.Quantizer(0.25, 0, 15, 300.0, 0.01, 5)
    step = CdlLayerStep(torch, M, K, CO, M * C, wq, xq, q_g=1e-3, conv=cdl.ConvShape(n_img, H, W, C, 3, 3))
    step.w.copy_(dev(torch, inputs.normal((K * CO,), 0.05, seed=6, stream=1)))
    step.x.copy_(dev(torch, np.maximum(inputs.normal((M * C,), 1.0, seed=6, stream=2), 0).astype(f32)))
    step.dY.copy_(dev(torch, inputs.normal((M, CO), 3e-2, seed=6, stream=3)))
    outs = ("w_soft", "W_idx", "x_soft", "X_idx", "hist_w", "hist_x", "prob_w", "prob_x", "Y", "G_idx", "gx_in", "dW",
            "dx", "dw")
    step.run()
    torch.cuda.synchronize()
    eager = {k: getattr(step, k).clone() for k in outs}
    eager_scalars = step.scalars.clone()
    # the forward output and the data gradient of the serial step against the oracle's convolution
    Xi, Wi, Gi = (eager[k].cpu().numpy() for k in ("X_idx", "W_idx", "G_idx"))
    acc = oracle.conv_fwd(Xi.reshape(n_img, H, W, C), Wi, 3, 3, 1, 1).reshape(M, CO)
    assert np.array_equal(eager["Y"].cpu().numpy(), scaled(acc, xq.q, wq.q))
    accx = oracle.conv_dx(Gi.reshape(n_img, H, W, CO), Wi, (n_img, H, W, C), 3, 3, 1, 1).reshape(-1)
    assert np.array_equal(eager["gx_in"].cpu().numpy(), scaled(accx, 1e-3, wq.q))
    graph = step.capture()
    for _ in range(2):
        for k in outs:
            getattr(step, k).zero_()
        graph.replay()
        torch.cuda.synchronize()
        for k in outs:
            assert torch.equal(getattr(step, k), eager[k]), k
        assert torch.equal(step.scalars[:2], eager_scalars[:2])
        assert torch.allclose(step.scalars[2:], eager_scalars[2:], rtol=1e-9, atol=1e-12)
    assert cdl.cdl_workspace_status(step.ws, check=False) == 0
