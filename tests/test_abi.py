"""Host-side checks of the C ABI that need no GPU: the library builds, loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2501_09849_b200 as cdl
from paper_2501_09849_b200 import build as cdl_build

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def lib():
    cdl_build.build()
    return cdl.load_library()


def declared_functions():
    text = (ROOT / "include" / "cdl.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cdl_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"cdl_quantize_soft", "cdl_quantize_hard", "cdl_quantize_backward", "cdl_index_entropy",
            "cdl_qlinear_fwd", "cdl_qlinear_bwd"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(n for n in cdl.__all__ if n.startswith("cdl_")) == set(names)


def test_version_and_strerror(lib):
    assert cdl.cdl_version() == 100
    assert cdl.cdl_strerror(0) == "ok"
    for code in range(-8, 0):
        assert cdl.cdl_strerror(code) not in ("ok", "unknown status")
    assert cdl.cdl_strerror(-99) == "unknown status"


def test_struct_layout_matches_the_header(lib):
    from paper_2501_09849_b200.api import _IndexDescC, _QuantParamsC
    assert ctypes.sizeof(_QuantParamsC) == 40 and _QuantParamsC.level_prob.offset == 24
    assert ctypes.sizeof(_IndexDescC) == 12


ARG, ALIGN, RANGE, WS, OVF = -1, -2, -3, -4, -5


def test_quantizer_argument_errors_need_no_device(lib):
    P = cdl.QuantParams
    x = 0x1000  # fake, never dereferenced: validation fails first
    assert cdl.cdl_quantize_hard(None, 4, P(0.1, -1, 1), check=False) == ARG
    assert cdl.cdl_quantize_hard(x, -1, P(0.1, -1, 1), check=False) == ARG
    assert cdl.cdl_quantize_hard(x + 2, 4, P(0.1, -1, 1), check=False) == ALIGN
    assert cdl.cdl_quantize_hard(x, 4, P(0.0, -1, 1), check=False) == RANGE
    assert cdl.cdl_quantize_hard(x, 4, P(float("nan"), -1, 1), check=False) == RANGE
    assert cdl.cdl_quantize_hard(x, 4, P(float("inf"), -1, 1), check=False) == RANGE
    assert cdl.cdl_quantize_hard(x, 4, P(0.1, 3, 1), check=False) == RANGE
    assert cdl.cdl_quantize_hard(x, 4, P(0.1, -128, 128), check=False) == RANGE      # 257 levels
    assert cdl.cdl_quantize_hard(x, 4, P(0.1, -129, 0), check=False) == RANGE
    assert cdl.cdl_quantize_hard(x, 4, P(0.1, -1, 128), check=False) == RANGE        # not an int8
    assert cdl.cdl_quantize_hard(x, 4, P(0.1, 1, 256), check=False) == RANGE         # not a uint8
    assert cdl.cdl_quantize_hard(x, 4, P(0.1, -1, 1, flags=0x80), check=False) == ARG
    assert cdl.cdl_quantize_soft(x, 4, P(0.1, -1, 1, alpha=5.0), None, check=False) == ARG
    assert cdl.cdl_quantize_soft(x, 4, P(0.1, -1, 1, alpha=0.0), x, check=False) == RANGE
    assert cdl.cdl_quantize_soft(x, 4, P(0.1, -1, 1, alpha=-2.0), x, check=False) == RANGE
    assert cdl.cdl_quantize_soft(x, 4, P(0.1, -7, 7, alpha=5.0, window=4), x, check=False) == ARG
    assert cdl.cdl_quantize_soft(x, 4, P(0.1, -7, 7, alpha=5.0, window=-1), x, check=False) == ARG
    assert cdl.cdl_quantize_soft(x, 4, P(1e30, -7, 7, alpha=1e30), x, check=False) == RANGE
    assert cdl.cdl_quantize_backward(x, None, 4, P(0.1, -1, 1, alpha=5.0), check=False) == ARG
    assert cdl.cdl_quantize_backward(x, x, 4, P(0.1, -1, 1, alpha=5.0, rate_weight=-1.0), check=False) == RANGE
    assert cdl.cdl_quantize_backward(x, x, 4, P(0.1, -1, 1, alpha=5.0), grad_q=x + 4, check=False) == ALIGN
    assert cdl.cdl_index_entropy(None, 4, x, check=False) == ARG
    assert cdl.cdl_index_entropy(x, 0, x, check=False) == RANGE
    assert cdl.cdl_index_entropy(x, 257, x, check=False) == RANGE
    assert cdl.cdl_index_entropy(x + 4, 4, x, check=False) == ALIGN
    with pytest.raises(cdl.CdlError, match="out of range"):
        cdl.cdl_quantize_hard(x, 4, P(0.0, -1, 1))


def test_qlinear_argument_errors_need_no_device(lib):
    D = cdl.IndexDesc
    p, ws = 0x10000, 0x20000
    a, w, g = D(0.25, 0, 15), D(0.02, -7, 7), D(1e-3, -127, 127)
    ok = dict(M=64, N=128, K=256)
    nb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, 64, 128, 256)
    assert nb >= 256 and cdl.cdl_workspace_bytes(99, 64, 128, 256) == 0 and cdl.cdl_workspace_bytes(1, 0, 1, 1) == 0
    f = cdl.cdl_qlinear_fwd
    assert f(None, 256, a, p, 128, w, **ok, y_out=p, ws=ws, ws_bytes=nb, check=False) == ARG
    assert f(p, 256, a, p, 128, w, **ok, ws=ws, ws_bytes=nb, check=False) == ARG                 # no output
    assert f(p, 255, a, p, 128, w, **ok, y_out=p, ws=ws, ws_bytes=nb, check=False) == ARG        # lda < K
    assert f(p, 264, a, p, 128, w, **ok, y_out=p, ws=ws, ws_bytes=nb, check=False) == ALIGN      # lda % 16
    assert f(p + 8, 256, a, p, 128, w, **ok, y_out=p, ws=ws, ws_bytes=nb, check=False) == ALIGN
    assert f(p, 256, a, p, 128, D(0.02, 0, 200), **ok, y_out=p, ws=ws, ws_bytes=nb, check=False) == RANGE
    assert f(p, 256, a, p, 128, w, **ok, y_out=p, ws=None, ws_bytes=nb, check=False) == WS
    assert f(p, 256, a, p, 128, w, **ok, y_out=p, ws=ws + 16, ws_bytes=nb, check=False) == WS
    assert f(p, 256, a, p, 128, w, **ok, y_out=p, ws=ws, ws_bytes=nb - 1, check=False) == WS
    big = 1 << 18
    assert f(p, big, D(1.0, 0, 255), p, 128, D(1.0, -128, 127), M=64, N=128, K=big, acc_out=p, ws=ws,
             ws_bytes=cdl.cdl_workspace_bytes(1, 64, 128, big), check=False) == OVF
    b = cdl.cdl_qlinear_bwd
    nbb = cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, 64, 128, 256)
    assert b(p, 128, g, p, 256, a, p, 128, w, **ok, ws=ws, ws_bytes=nbb, check=False) == ARG     # no output
    assert b(p, 128, g, None, 256, a, p, 128, w, **ok, dW=p, ws=ws, ws_bytes=nbb, check=False) == ARG
    assert b(p, 128, g, p, 256, a, None, 128, w, **ok, dX=p, ws=ws, ws_bytes=nbb, check=False) == ARG
    assert b(p, 120, g, p, 256, a, p, 128, w, **ok, dX=p, ws=ws, ws_bytes=nbb, check=False) == ARG
    assert b(p, 128, g, p, 256, a, p, 128, w, **ok, dX=p, ws=ws, ws_bytes=0, check=False) == WS
    M = 1 << 20
    assert b(p, 128, g, p, 256, D(1.0, 0, 255), p, 128, w, M=M, N=128, K=256, dWacc=p, ws=ws,
             ws_bytes=cdl.cdl_workspace_bytes(2, M, 128, 256), check=False) == OVF


def test_real_gradient_products_check_every_argument_before_enqueueing(lib):
    # Without a device any enqueue attempt would come back as a launch error: a range / alignment / argument status
    # therefore shows that the check ran before the first memset or kernel launch.
    D = cdl.IndexDesc
    p, ws = 0x10000, 0x20000
    a, w = D(0.25, 0, 15), D(0.02, -7, 7)
    M, N, K = 64, 120, 256                     # N not a multiple of 16: the digit planes would be cleared first
    nb = cdl.cdl_qlinear_bwd_fp_workspace_bytes(M, N, K)
    f = cdl.cdl_qlinear_bwd_fp
    assert f(p, 1.0, p, 256, D(0.25, 0, 300), p, 128, w, M, N, K, dW=p, ws=ws, ws_bytes=nb, check=False) == RANGE
    assert f(p, 1.0, p, 256, D(0.25, 5, 1), p, 128, w, M, N, K, dW=p, ws=ws, ws_bytes=nb, check=False) == RANGE
    assert f(p, 1.0, p, 264, a, p, 128, w, M, N, K, dW=p, ws=ws, ws_bytes=nb, check=False) == ALIGN      # lda % 16
    assert f(p, 1.0, p, 240, a, p, 128, w, M, N, K, dW=p, ws=ws, ws_bytes=nb, check=False) == ARG        # lda < K
    assert f(p, 1.0, p, 256, a, p, 128, D(0.02, 0, 200), M, N, K, dX=p, ws=ws, ws_bytes=nb, check=False) == RANGE
    assert f(p, 1.0, p, 256, a, p + 8, 128, w, M, N, K, dX=p, ws=ws, ws_bytes=nb, check=False) == ALIGN
    assert f(p, 1.0, p, 256, a, p, 112, w, M, N, K, dX=p, ws=ws, ws_bytes=nb, check=False) == ARG        # ldw < N
    assert f(p, 1.0, p, 256, a, p, 128, w, M, N, K, dX=p + 2, ws=ws, ws_bytes=nb, check=False) == ALIGN
    shape = cdl.ConvShape(2, 8, 8, 64, 3, 3)
    nc = cdl.cdl_qconv_bwd_fp_workspace_bytes(shape, 64)
    c = cdl.cdl_qconv_bwd_fp
    assert c(p, 1.0, p, D(0.25, 0, 300), p, 64, w, shape, 64, dW=p, ws=ws, ws_bytes=nc, check=False) == RANGE
    assert c(p, 1.0, p + 4, a, p, 64, w, shape, 64, dW=p, ws=ws, ws_bytes=nc, check=False) == ALIGN
    assert c(p, 1.0, p, a, p, 72, w, shape, 64, dX=p, ws=ws, ws_bytes=nc, check=False) == ALIGN          # ldw % 16
    assert c(p, 1.0, p, a, p, 48, w, shape, 64, dX=p, ws=ws, ws_bytes=nc, check=False) == ARG            # ldw < C_out
    assert c(p, 1.0, p, a, p, 64, D(0.02, 0, 200), shape, 64, dX=p, ws=ws, ws_bytes=nc, check=False) == RANGE


def test_missing_library_raises_instead_of_falling_back(monkeypatch, tmp_path):
    from paper_2501_09849_b200 import api
    monkeypatch.setattr(api, "_LIB", None)
    monkeypatch.setattr(api, "_PKG", tmp_path)
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        api.cdl_version()
