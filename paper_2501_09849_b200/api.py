"""ctypes binding of libcdl.so: same names as the C ABI (include/cdl.h), argument marshalling only.

Tensors are torch CUDA tensors used as plain device buffers (``data_ptr()``); the stream defaults to
torch's current CUDA stream.  Nothing here computes anything and there is no fallback: if the library
has not been built, the first call raises.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

__all__ = [
    "CdlError", "QuantParams", "IndexDesc", "library_path", "load_library",
    "cdl_version", "cdl_strerror", "cdl_quantize_hard", "cdl_quantize_soft", "cdl_quantize_backward", "cdl_quantize_sample",
    "cdl_index_entropy", "cdl_qlinear_fwd", "cdl_qlinear_bwd", "cdl_qlinear_bwd_dw_noalloc", "cdl_noalloc_status",
    "cdl_workspace_bytes", "cdl_workspace_status", "cdl_rescale_acc", "CDL_NOALLOC_MAX_DW_ELEMS",
    "cdl_huffman_lengths", "cdl_qconv_bwd_fp", "cdl_qconv_bwd_fp_workspace_bytes", "cdl_qlinear_bwd_fp", "cdl_qlinear_bwd_fp_workspace_bytes", "cdl_qlinear_fwd_next", "cdl_qconv_fwd_next", "ConvShape", "cdl_qconv_fwd", "cdl_qconv_bwd", "cdl_qconv_workspace_bytes",
    "CDL_HIST_ACCUMULATE", "CDL_OP_QLINEAR_FWD", "CDL_OP_QLINEAR_BWD", "CDL_MAX_LEVELS",
]

CDL_HIST_ACCUMULATE = 0x1
CDL_OP_QLINEAR_FWD = 1
CDL_OP_QLINEAR_BWD = 2
CDL_MAX_LEVELS = 256
CDL_NOALLOC_MAX_DW_ELEMS = 1 << 20

_PKG = Path(__file__).resolve().parent
_LIB = None


class CdlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {cdl_strerror(status)} (status {status})")


class _QuantParamsC(C.Structure):
    _fields_ = [("q", C.c_float), ("lo", C.c_int32), ("hi", C.c_int32), ("alpha", C.c_float),
                ("rate_weight", C.c_float), ("level_prob", C.c_void_p), ("window", C.c_int32),
                ("flags", C.c_uint32)]


class _IndexDescC(C.Structure):
    _fields_ = [("q", C.c_float), ("lo", C.c_int32), ("hi", C.c_int32)]


class QuantParams:
    """cdl_quant_params: (q, lo, hi, alpha, rate_weight, level_prob, window, flags)."""

    def __init__(self, q, lo, hi, alpha=1.0, rate_weight=0.0, level_prob=None, window=0, flags=0):
        self.q, self.lo, self.hi, self.alpha = float(q), int(lo), int(hi), float(alpha)
        self.rate_weight, self.level_prob, self.window, self.flags = float(rate_weight), level_prob, int(window), int(flags)

    @property
    def nlev(self):
        return self.hi - self.lo + 1

    def _c(self):
        return _QuantParamsC(self.q, self.lo, self.hi, self.alpha, self.rate_weight, _ptr(self.level_prob),
                             self.window, self.flags)


class IndexDesc:
    """cdl_index_desc: step size and index range of a GEMM operand."""

    def __init__(self, q, lo, hi):
        self.q, self.lo, self.hi = float(q), int(lo), int(hi)

    def _c(self):
        return _IndexDescC(self.q, self.lo, self.hi)


def library_path() -> Path:
    return _PKG / "libcdl.so"


def load_library():
    """Load libcdl.so (built in-tree by ``python -m paper_2501_09849_b200.build``); raises if it is missing."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not path.exists():
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2501_09849_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(str(path))
    P, I32, I64 = C.c_void_p, C.c_int32, C.c_int64
    lib.cdl_version.restype = C.c_int
    lib.cdl_strerror.restype = C.c_char_p
    lib.cdl_strerror.argtypes = [C.c_int]
    lib.cdl_quantize_hard.argtypes = [P, I64, P, P, P, P]
    lib.cdl_quantize_soft.argtypes = [P, I64, P, P, P, P, P, P]
    lib.cdl_quantize_backward.argtypes = [P, P, I64, P, P, P, P, P]
    lib.cdl_quantize_sample.argtypes = [P, I64, P, C.c_uint64, C.c_uint64, P, P, P, P]
    lib.cdl_index_entropy.argtypes = [P, I32, P, P, P, P]
    lib.cdl_qlinear_fwd.argtypes = [P, I64, P, P, I64, P, I32, I32, I32, P, P, P, P, C.c_size_t, P]
    lib.cdl_qlinear_bwd.argtypes = [P, I64, P, P, I64, P, P, I64, P, I32, I32, I32, P, P, P, P, P, C.c_size_t, P]
    lib.cdl_qlinear_bwd_dw_noalloc.argtypes = [P, I64, P, P, I64, P, I32, I32, I32, P, P]
    lib.cdl_qlinear_fwd_next.argtypes = [P, I64, P, P, I64, P, I32, I32, I32, P, P, P, P, P, P, C.c_size_t, P]
    lib.cdl_qconv_fwd_next.argtypes = [P, P, P, I64, P, P, I32, P, P, P, P, P, P, C.c_size_t, P]
    lib.cdl_qlinear_fwd_next.restype = C.c_int
    lib.cdl_qconv_fwd_next.restype = C.c_int
    lib.cdl_qlinear_bwd_fp.argtypes = [P, C.c_float, P, I64, P, P, I64, P, I32, I32, I32, P, P, P, C.c_size_t, P]
    lib.cdl_qlinear_bwd_fp.restype = C.c_int
    lib.cdl_qlinear_bwd_fp_workspace_bytes.argtypes = [I32, I32, I32]
    lib.cdl_qlinear_bwd_fp_workspace_bytes.restype = C.c_size_t
    lib.cdl_qconv_bwd_fp.argtypes = [P, C.c_float, P, P, P, I64, P, P, I32, P, P, P, C.c_size_t, P]
    lib.cdl_qconv_bwd_fp.restype = C.c_int
    lib.cdl_qconv_bwd_fp_workspace_bytes.argtypes = [P, I32]
    lib.cdl_qconv_bwd_fp_workspace_bytes.restype = C.c_size_t
    lib.cdl_huffman_lengths.argtypes = [P, I32, P, P, P, P]
    lib.cdl_huffman_lengths.restype = C.c_int
    lib.cdl_qconv_fwd.argtypes = [P, P, P, I64, P, P, I32, P, P, P, P, C.c_size_t, P]
    lib.cdl_qconv_bwd.argtypes = [P, P, P, P, P, I64, P, P, I32, P, P, P, P, P, C.c_size_t, P]
    lib.cdl_qconv_workspace_bytes.argtypes = [P, I32]
    lib.cdl_qconv_workspace_bytes.restype = C.c_size_t
    lib.cdl_workspace_bytes.argtypes = [I32, I32, I32, I32]
    lib.cdl_workspace_bytes.restype = C.c_size_t
    lib.cdl_workspace_status.argtypes = [P, P]
    lib.cdl_noalloc_status.argtypes = [P]
    lib.cdl_rescale_acc.argtypes = [P, I32, I64, C.c_float, C.c_float, P, P]
    lib.cdl_rescale_acc.restype = C.c_int
    lib.cdl_noalloc_status.restype = C.c_int
    for name in ("cdl_quantize_hard", "cdl_quantize_soft", "cdl_quantize_backward", "cdl_quantize_sample", "cdl_index_entropy",
                 "cdl_qlinear_fwd", "cdl_qlinear_bwd", "cdl_qlinear_bwd_dw_noalloc", "cdl_workspace_status",
                 "cdl_qconv_fwd", "cdl_qconv_bwd"):
        getattr(lib, name).restype = C.c_int
    _LIB = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return C.c_void_p(t)
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        if not torch.cuda.is_available():   # no device: the call fails in the library, not here
            return None
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return C.c_void_p(stream)
    return C.c_void_p(stream.cuda_stream)


def _check(rc, where, check):
    if check and rc != 0:
        raise CdlError(rc, where)
    return rc


def cdl_version() -> int:
    return int(load_library().cdl_version())


def cdl_strerror(status: int) -> str:
    return load_library().cdl_strerror(int(status)).decode()


def cdl_quantize_hard(x, n, p: QuantParams, idx_out=None, hist=None, stream=None, check=True):
    pc = p._c()
    rc = load_library().cdl_quantize_hard(_ptr(x), n, C.byref(pc), _ptr(idx_out), _ptr(hist), _stream(stream))
    return _check(rc, "cdl_quantize_hard", check)


def cdl_quantize_soft(x, n, p: QuantParams, y_soft, idx_out=None, hist=None, stream=None, check=True, soft_hist=None):
    pc = p._c()
    rc = load_library().cdl_quantize_soft(_ptr(x), n, C.byref(pc), _ptr(y_soft), _ptr(idx_out), _ptr(hist), _ptr(soft_hist),
                                          _stream(stream))
    return _check(rc, "cdl_quantize_soft", check)


def cdl_quantize_sample(x, n, p: QuantParams, seed, first_index=0, idx_out=None, y_out=None, hist=None, stream=None,
                        check=True):
    pc = p._c()
    rc = load_library().cdl_quantize_sample(_ptr(x), n, C.byref(pc), int(seed), int(first_index), _ptr(idx_out),
                                            _ptr(y_out), _ptr(hist), _stream(stream))
    return _check(rc, "cdl_quantize_sample", check)


def cdl_quantize_backward(x, grad_out, n, p: QuantParams, grad_x=None, grad_q=None, grad_alpha=None, stream=None,
                          check=True):
    pc = p._c()
    rc = load_library().cdl_quantize_backward(_ptr(x), _ptr(grad_out), n, C.byref(pc), _ptr(grad_x), _ptr(grad_q),
                                              _ptr(grad_alpha), _stream(stream))
    return _check(rc, "cdl_quantize_backward", check)


def cdl_index_entropy(hist, nlev, H_bits, level_prob=None, n_out=None, stream=None, check=True):
    rc = load_library().cdl_index_entropy(_ptr(hist), nlev, _ptr(H_bits), _ptr(level_prob), _ptr(n_out),
                                          _stream(stream))
    return _check(rc, "cdl_index_entropy", check)


def cdl_workspace_bytes(op, M, N, K) -> int:
    return int(load_library().cdl_workspace_bytes(op, M, N, K))


def cdl_workspace_status(ws, stream=None, check=True):
    rc = load_library().cdl_workspace_status(_ptr(ws), _stream(stream))
    return _check(rc, "cdl_workspace_status", check)


def cdl_qlinear_fwd_next(A_idx, lda, a: IndexDesc, W_idx, ldw, w: IndexDesc, M, N, K, next: IndexDesc, idx_next,
                         acc_out=None, y_out=None, bias=None, ws=None, ws_bytes=0, stream=None, check=True):
    ac, wc, nc = a._c(), w._c(), next._c()
    rc = load_library().cdl_qlinear_fwd_next(_ptr(A_idx), lda, C.byref(ac), _ptr(W_idx), ldw, C.byref(wc), M, N, K,
                                             _ptr(acc_out), _ptr(y_out), _ptr(bias), C.byref(nc), _ptr(idx_next),
                                             _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qlinear_fwd_next", check)


def cdl_qconv_fwd_next(X_idx, x: IndexDesc, W_idx, ldw, w: IndexDesc, shape, C_out, next: IndexDesc, idx_next,
                       acc_out=None, y_out=None, bias=None, ws=None, ws_bytes=0, stream=None, check=True):
    xc, wc, sc, nc = x._c(), w._c(), shape._c(), next._c()
    rc = load_library().cdl_qconv_fwd_next(_ptr(X_idx), C.byref(xc), _ptr(W_idx), ldw, C.byref(wc), C.byref(sc), C_out,
                                           _ptr(acc_out), _ptr(y_out), _ptr(bias), C.byref(nc), _ptr(idx_next),
                                           _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qconv_fwd_next", check)


def cdl_qlinear_bwd_fp_workspace_bytes(M, N, K):
    return int(load_library().cdl_qlinear_bwd_fp_workspace_bytes(M, N, K))


def cdl_qlinear_bwd_fp(G, g_absmax, A_idx, lda, a, W_idx, ldw, w, M, N, K, dX=None, dW=None, ws=None, ws_bytes=0,
                       stream=None, check=True):
    ac = a._c() if a is not None else None
    wc = w._c() if w is not None else None
    rc = load_library().cdl_qlinear_bwd_fp(_ptr(G), float(g_absmax), _ptr(A_idx), lda,
                                           C.byref(ac) if ac is not None else None, _ptr(W_idx), ldw,
                                           C.byref(wc) if wc is not None else None, M, N, K, _ptr(dX), _ptr(dW),
                                           _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qlinear_bwd_fp", check)


def cdl_qconv_bwd_fp_workspace_bytes(shape, C_out):
    sc = shape._c()
    return int(load_library().cdl_qconv_bwd_fp_workspace_bytes(C.byref(sc), C_out))


def cdl_qconv_bwd_fp(G, g_absmax, X_idx, x, W_idx, ldw, w, shape, C_out, dX=None, dW=None, ws=None, ws_bytes=0,
                     stream=None, check=True):
    sc = shape._c()
    xc = x._c() if x is not None else None
    wc = w._c() if w is not None else None
    rc = load_library().cdl_qconv_bwd_fp(_ptr(G), float(g_absmax), _ptr(X_idx), C.byref(xc) if xc is not None else None,
                                         _ptr(W_idx), ldw, C.byref(wc) if wc is not None else None, C.byref(sc), C_out,
                                         _ptr(dX), _ptr(dW), _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qconv_bwd_fp", check)


def cdl_huffman_lengths(hist, nlev, lengths=None, total_bits=None, avg_bits=None, stream=None, check=True):
    rc = load_library().cdl_huffman_lengths(_ptr(hist), nlev, _ptr(lengths), _ptr(total_bits), _ptr(avg_bits),
                                            _stream(stream))
    return _check(rc, "cdl_huffman_lengths", check)


def cdl_qlinear_fwd(A_idx, lda, a: IndexDesc, W_idx, ldw, w: IndexDesc, M, N, K, acc_out=None, y_out=None, bias=None,
                    ws=None, ws_bytes=0, stream=None, check=True):
    ac, wc = a._c(), w._c()
    rc = load_library().cdl_qlinear_fwd(_ptr(A_idx), lda, C.byref(ac), _ptr(W_idx), ldw, C.byref(wc), M, N, K,
                                        _ptr(acc_out), _ptr(y_out), _ptr(bias), _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qlinear_fwd", check)


def cdl_qlinear_bwd(G_idx, ldg, g: IndexDesc, A_idx, lda, a, W_idx, ldw, w, M, N, K, dXacc=None, dX=None,
                    dWacc=None, dW=None, ws=None, ws_bytes=0, stream=None, check=True):
    gc = g._c()
    ac = a._c() if a is not None else None
    wc = w._c() if w is not None else None
    rc = load_library().cdl_qlinear_bwd(_ptr(G_idx), ldg, C.byref(gc), _ptr(A_idx), lda,
                                        C.byref(ac) if ac is not None else None, _ptr(W_idx), ldw,
                                        C.byref(wc) if wc is not None else None, M, N, K, _ptr(dXacc), _ptr(dX),
                                        _ptr(dWacc), _ptr(dW), _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qlinear_bwd", check)


class _ConvShapeC(C.Structure):
    _fields_ = [("N", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("C", C.c_int32), ("R", C.c_int32), ("S", C.c_int32),
                ("stride", C.c_int32), ("pad_h", C.c_int32), ("pad_w", C.c_int32)]


class ConvShape:
    """cdl_conv_shape: input tensor N x H x W x C, filter R x S, stride, zero padding (default (R-1)/2, (S-1)/2)."""

    def __init__(self, N, H, W, C, R, S, stride=1, pad_h=None, pad_w=None):
        self.N, self.H, self.W, self.C, self.R, self.S = int(N), int(H), int(W), int(C), int(R), int(S)
        self.stride = int(stride)
        self.pad_h = (self.R - 1) // 2 if pad_h is None else int(pad_h)
        self.pad_w = (self.S - 1) // 2 if pad_w is None else int(pad_w)

    @property
    def P(self):
        """output rows per image"""
        return (self.H + 2 * self.pad_h - self.R) // self.stride + 1

    @property
    def Q(self):
        """output columns per image"""
        return (self.W + 2 * self.pad_w - self.S) // self.stride + 1

    def _c(self):
        return _ConvShapeC(self.N, self.H, self.W, self.C, self.R, self.S, self.stride, self.pad_h, self.pad_w)


def cdl_qconv_workspace_bytes(shape: ConvShape, C_out):
    sc = shape._c()
    return int(load_library().cdl_qconv_workspace_bytes(C.byref(sc), C_out))


def cdl_qconv_fwd(X_idx, x: IndexDesc, W_idx, ldw, w: IndexDesc, shape: ConvShape, C_out, acc_out=None, y_out=None,
                  bias=None, ws=None, ws_bytes=0, stream=None, check=True):
    xc, wc, sc = x._c(), w._c(), shape._c()
    rc = load_library().cdl_qconv_fwd(_ptr(X_idx), C.byref(xc), _ptr(W_idx), ldw, C.byref(wc), C.byref(sc), C_out,
                                      _ptr(acc_out), _ptr(y_out), _ptr(bias), _ptr(ws), ws_bytes, _stream(stream))
    return _check(rc, "cdl_qconv_fwd", check)


def cdl_qconv_bwd(G_idx, g: IndexDesc, X_idx, x, W_idx, ldw, w, shape: ConvShape, C_out, dXacc=None, dX=None,
                  dWacc=None, dW=None, ws=None, ws_bytes=0, stream=None, check=True):
    gc, sc = g._c(), shape._c()
    xc = x._c() if x is not None else None
    wc = w._c() if w is not None else None
    rc = load_library().cdl_qconv_bwd(_ptr(G_idx), C.byref(gc), _ptr(X_idx), C.byref(xc) if xc is not None else None,
                                      _ptr(W_idx), ldw, C.byref(wc) if wc is not None else None, C.byref(sc), C_out,
                                      _ptr(dXacc), _ptr(dX), _ptr(dWacc), _ptr(dW), _ptr(ws), ws_bytes,
                                      _stream(stream))
    return _check(rc, "cdl_qconv_bwd", check)


def cdl_qlinear_bwd_dw_noalloc(G_idx, ldg, g: IndexDesc, A_idx, lda, a: IndexDesc, M, N, K, dW, stream=None, check=True):
    """dW = (g.q a.q) A_idx^T G_idx for callers that cannot allocate device memory: the scratch is a static array
    inside the library (K * N <= CDL_NOALLOC_MAX_DW_ELEMS).  Calls that overlap on the GPU race on that array."""
    gc, ac = g._c(), a._c()
    rc = load_library().cdl_qlinear_bwd_dw_noalloc(_ptr(G_idx), ldg, C.byref(gc), _ptr(A_idx), lda, C.byref(ac), M, N, K,
                                                   _ptr(dW), _stream(stream))
    return _check(rc, "cdl_qlinear_bwd_dw_noalloc", check)


def cdl_noalloc_status(stream=None, check=True):
    """Synchronises the stream and reports a device-side timeout of the last cdl_qlinear_bwd_dw_noalloc call on the
    current device (the record lives in the library's built-in scratch); allocates nothing."""
    rc = load_library().cdl_noalloc_status(_stream(stream))
    return _check(rc, "cdl_noalloc_status", check)


def cdl_rescale_acc(acc, acc_bits, n, q_x, q_y, out, stream=None, check=True):
    rc = load_library().cdl_rescale_acc(_ptr(acc), acc_bits, n, float(q_x), float(q_y), _ptr(out), _stream(stream))
    return _check(rc, "cdl_rescale_acc", check)
