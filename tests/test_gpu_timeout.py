"""The device-side timeout path, exercised without touching the product kernels and without hanging anything.

Every mbarrier wait of the tensor-core kernels goes through one bounded helper (csrc/cdl_wait.cuh); when it runs out
the kernel writes a record into the status block at the start of its workspace, which cdl_workspace_status reports as
CDL_ERR_TIMEOUT and clears.  Here a small kernel built only by this test calls that same helper with a 1 ms limit on a
barrier that is one arrival short: the wait gives up, the record is written, the kernel exits normally.
"""
import ctypes
import subprocess
from pathlib import Path

import pytest

import paper_2501_09849_b200 as cdl

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parents[1]
TIMEOUT = -7


@pytest.fixture(scope="module")
def probe(tmp_path_factory):
    out = tmp_path_factory.mktemp("wait_probe") / "libwait_probe.so"
    subprocess.run(["/usr/local/cuda/bin/nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-std=c++17",
                    "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared", "-I", str(ROOT / "include"),
                    "-I", str(ROOT / "paper_2501_09849_b200" / "csrc"), "-o", str(out),
                    str(ROOT / "tests" / "cuda" / "wait_probe.cu")], check=True)
    lib = ctypes.CDLL(str(out))
    lib.wait_probe.argtypes = [ctypes.c_void_p, ctypes.c_ulonglong, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    lib.wait_probe.restype = ctypes.c_int
    return lib


def test_expired_wait_is_reported_once_and_then_cleared(probe):
    import torch
    cdl.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    # a recycled allocation may hold anything, e.g. the bare code without its tags: that is not a record
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    ws.view(torch.int32)[0] = TIMEOUT
    assert cdl.cdl_workspace_status(ws, check=False) == 0
    outcome = torch.zeros(1, dtype=torch.int32, device="cuda")
    # all arrivals made: the wait completes, nothing is recorded
    assert probe.wait_probe(ws.data_ptr(), 1_000_000, 3, 3, outcome.data_ptr(), stream) == 0
    assert cdl.cdl_workspace_status(ws, check=False) == 0 and int(outcome.cpu()[0]) == 1
    # one arrival short: the wait runs out after 1 ms, the kernel records it and returns
    assert probe.wait_probe(ws.data_ptr(), 1_000_000, 2, 3, outcome.data_ptr(), stream) == 0
    assert cdl.cdl_workspace_status(ws, check=False) == TIMEOUT and int(outcome.cpu()[0]) == 2
    assert cdl.cdl_workspace_status(ws, check=False) == 0            # reading cleared the record
    assert probe.wait_probe(ws.data_ptr(), 1_000_000, 0, 1, outcome.data_ptr(), stream) == 0
    with pytest.raises(cdl.CdlError, match="wait expired"):
        cdl.cdl_workspace_status(ws)
    # the context is still usable: a product call on the same workspace runs and reports no timeout
    M, K, N = 256, 128, 64
    nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K)
    ws2 = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    A = torch.ones((M, K), dtype=torch.uint8, device="cuda")
    W = torch.ones((K, N), dtype=torch.int8, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    cdl.cdl_qlinear_fwd(A, K, cdl.IndexDesc(1.0, 0, 15), W, N, cdl.IndexDesc(1.0, -7, 7), M, N, K, acc, None, None, ws2, nb)
    assert cdl.cdl_workspace_status(ws2, check=False) == 0
    assert bool((acc == K).all())
