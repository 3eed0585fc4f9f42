"""The no-allocation weight-gradient entry point against the regular one.

cdl_qlinear_bwd_dw_noalloc exists for callers that cannot call cudaMalloc (a framework allocator owns the
device memory, or the step loop must not take cudaMalloc's implicit synchronisation): its scratch is a static
array inside the library.  The test calls it twice in a row through the C ABI, with different inputs, and
requires the same dW as cdl_qlinear_bwd each time (integer accumulation, so the comparison is exact - the
tolerance the other GEMM tests use); the second call would expose accumulators or a status word left
uncleared by the first.  This file sorts last so that a run stopping at the first failure has already run
every other test.
"""
import numpy as np
import pytest

import paper_2501_09849_b200 as cdl
from paper_2501_09849_b200 import inputs

pytestmark = pytest.mark.gpu


def test_noalloc_dw_matches_regular_entry_point_twice_in_a_row():
    import torch
    cdl.load_library()
    a, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(1e-3, -127, 127)
    # (M, K, N): a split reduction (few output tiles, long M), a ragged one, a single-split one, and one whose
    # output is tiled in 256-row blocks of one CTA (at most 128 columns, 640 rows)
    for call, (M, K, N) in enumerate([(4096, 256, 128), (3000, 144, 16), (300, 640, 256), (2000, 640, 64)]):
        A = torch.from_numpy(inputs.uniform_indices((M, K), 0, 15, seed=40 + call)).cuda()
        G = torch.from_numpy(inputs.uniform_indices((M, N), -127, 127, seed=50 + call)).cuda()
        nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K)
        ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
        ref = torch.full((K, N), -1.0, dtype=torch.float32, device="cuda")
        cdl.cdl_qlinear_bwd(G, N, g, A, K, a, None, N, None, M, N, K, None, None, None, ref, ws, nb)
        cdl.cdl_workspace_status(ws)
        for repeat in range(2):
            out = torch.full((K, N), -2.0, dtype=torch.float32, device="cuda")
            cdl.cdl_qlinear_bwd_dw_noalloc(G, N, g, A, K, a, M, N, K, out)
            assert cdl.cdl_noalloc_status() == 0          # synchronises; no device-side wait gave up
            assert torch.equal(out, ref), (M, K, N, repeat)
        # and against plain integer arithmetic on the host, so that both being wrong together cannot pass
        acc = A.cpu().numpy().astype(np.int64).T @ G.cpu().numpy().astype(np.int64)
        expect = acc.astype(np.float32) * (np.float32(g.q) * np.float32(a.q))
        assert np.array_equal(ref.cpu().numpy(), expect)


def test_noalloc_dw_rejects_sizes_beyond_its_static_scratch():
    import torch
    cdl.load_library()
    a, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(1e-3, -127, 127)
    K, N, M = 2048, 1024, 16          # K * N = 2^21 > CDL_NOALLOC_MAX_DW_ELEMS
    assert K * N > cdl.CDL_NOALLOC_MAX_DW_ELEMS
    buf = torch.zeros(16, dtype=torch.uint8, device="cuda")
    rc = cdl.cdl_qlinear_bwd_dw_noalloc(buf, N, g, buf, K, a, M, N, K, buf, check=False)
    assert rc == -9 and "built-in scratch" in cdl.cdl_strerror(rc)


def test_noalloc_dw_rejects_reductions_too_long_for_int32():
    # cdl_qlinear_bwd cuts such a reduction into exact parts and sums them in int64 slabs; the built-in scratch has
    # no room for slabs, so the entry point refuses (documented limit M * max|a| * max|g| < 2^31)
    import torch
    cdl.load_library()
    a, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(1e-3, -127, 127)
    buf = torch.zeros(16, dtype=torch.uint8, device="cuda")
    M_ok, M_bad = (1 << 31) // (15 * 127) - 16, ((1 << 31) // (15 * 127) // 16 + 1) * 16
    assert M_bad * 15 * 127 >= 1 << 31 > M_ok * 15 * 127
    rc = cdl.cdl_qlinear_bwd_dw_noalloc(buf, 16, g, buf, 16, a, M_bad, 16, 16, buf, check=False)
    assert rc == -5 and "overflow" in cdl.cdl_strerror(rc)
