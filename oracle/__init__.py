"""CPU oracle for the CDL quantized layer: thin numpy/ctypes face of cdl_oracle.c.

TEST INFRASTRUCTURE ONLY.  The arithmetic lives in ``cdl_oracle.c`` (plain C,
double precision, one function per definition of the paper); this module only
compiles it with gcc, loads it and marshals numpy arrays.  It imports nothing
from the CUDA package, and the CUDA package imports nothing from here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "cdl_oracle.c"
_SO = _HERE / "libcdl_oracle.so"

MAX_LEVELS = 256


def build(force: bool = False) -> Path:
    """Compile cdl_oracle.c into libcdl_oracle.so (no-op when up to date)."""
    if force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _SO.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_SO))
        c = ctypes
        P = c.c_void_p
        lib.cdl_oracle_threads.restype = c.c_int
        lib.cdl_oracle_set_threads.restype = c.c_int
        lib.cdl_oracle_set_threads.argtypes = [c.c_int]
        lib.cdl_oracle_cpmf.argtypes = [c.c_double, c.c_double, c.c_int, c.c_int, c.c_double, c.c_int, P]
        lib.cdl_oracle_soft.argtypes = [P, c.c_int64, c.c_float, c.c_int, c.c_int, c.c_float, c.c_int, P]
        lib.cdl_oracle_partials.argtypes = [P, c.c_int64, c.c_float, c.c_int, c.c_int, c.c_float, c.c_int,
                                            P, P, P, P]
        lib.cdl_oracle_hard.argtypes = [P, c.c_int64, c.c_float, c.c_int, c.c_int, P, P]
        lib.cdl_oracle_entropy.argtypes = [P, c.c_int, P, P, P]
        lib.cdl_oracle_backward.argtypes = [P, P, c.c_int64, c.c_float, c.c_int, c.c_int, c.c_float, c.c_int,
                                            c.c_float, P, P, P, P, P, P, P, P]
        lib.cdl_oracle_gemm_fwd.argtypes = [P, c.c_int64, c.c_int, P, c.c_int64, c.c_int, c.c_int, c.c_int, P]
        lib.cdl_oracle_gemm_dx.argtypes = [P, c.c_int64, P, c.c_int64, c.c_int, c.c_int, c.c_int, P]
        lib.cdl_oracle_gemm_dw.argtypes = [P, c.c_int64, c.c_int, P, c.c_int64, c.c_int, c.c_int, c.c_int, P]
        lib.cdl_oracle_conv_fwd.argtypes = [P, c.c_int, P, c.c_int64] + [c.c_int] * 10 + [P]
        lib.cdl_oracle_conv_dx.argtypes = [P, P, c.c_int64] + [c.c_int] * 10 + [P]
        lib.cdl_oracle_conv_dw.argtypes = [P, c.c_int, P] + [c.c_int] * 10 + [P]
        for f in (lib.cdl_oracle_conv_fwd, lib.cdl_oracle_conv_dx, lib.cdl_oracle_conv_dw):
            f.restype = None
        lib.cdl_oracle_mpmf.argtypes = [P, c.c_int64, c.c_float, c.c_int, c.c_int, c.c_float, c.c_int, P]
        lib.cdl_oracle_mpmf.restype = None
        lib.cdl_oracle_philox4x32_10.argtypes = [P, P, P]
        lib.cdl_oracle_philox4x32_10.restype = None
        lib.cdl_oracle_uniform.argtypes = [c.c_uint64, c.c_uint64]
        lib.cdl_oracle_uniform.restype = c.c_double
        lib.cdl_oracle_sample.argtypes = [P, c.c_int64, c.c_float, c.c_int, c.c_int, c.c_float, c.c_int, c.c_uint64,
                                          c.c_uint64, P, P, P, P]
        lib.cdl_oracle_sample.restype = None
        for f in ("cpmf", "soft", "partials", "hard", "entropy", "backward", "gemm_fwd", "gemm_dx", "gemm_dw"):
            getattr(lib, "cdl_oracle_" + f).restype = None
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _check_levels(lo, hi):
    if not (1 <= hi - lo + 1 <= MAX_LEVELS):
        raise ValueError("index set must have 1..256 levels")


def threads() -> int:
    """Host threads the oracle's parallel loops use."""
    return int(_load().cdl_oracle_threads())


def set_threads(n: int) -> int:
    """Sets the number of host threads of the oracle's parallel loops; returns the count in effect."""
    return int(_load().cdl_oracle_set_threads(int(n)))


def cpmf(theta, q, lo, hi, alpha, window=0):
    """P_alpha(. | theta) over the levels lo..hi (Sec. IV-A, Eq. (4)); float64[nlev]."""
    _check_levels(lo, hi)
    P = np.empty(hi - lo + 1, dtype=np.float64)
    _load().cdl_oracle_cpmf(float(theta), float(q), lo, hi, float(alpha), window, _ptr(P))
    return P


def soft(x, q, lo, hi, alpha, window=0):
    """Q_d(x) element-wise (Sec. IV-B, Eq. (8)); float64, same shape as x."""
    _check_levels(lo, hi)
    x = _f32(x)
    y = np.empty(x.shape, dtype=np.float64)
    _load().cdl_oracle_soft(_ptr(x), x.size, q, lo, hi, alpha, window, _ptr(y))
    return y


def partials(x, q, lo, hi, alpha, window=0):
    """(dQ_d/dtheta, dQ_d/dq, dQ_d/dalpha, Var{Q_p|theta}) element-wise (Lemma 1)."""
    _check_levels(lo, hi)
    x = _f32(x)
    outs = [np.empty(x.shape, dtype=np.float64) for _ in range(4)]
    _load().cdl_oracle_partials(_ptr(x), x.size, q, lo, hi, alpha, window, *[_ptr(o) for o in outs])
    return tuple(outs)


def hard(x, q, lo, hi):
    """Hard indices (int32, shape of x) and their histogram (uint64[nlev])."""
    _check_levels(lo, hi)
    x = _f32(x)
    idx = np.empty(x.shape, dtype=np.int32)
    hist = np.zeros(hi - lo + 1, dtype=np.uint64)
    _load().cdl_oracle_hard(_ptr(x), x.size, q, lo, hi, _ptr(idx), _ptr(hist))
    return idx, hist


def entropy(hist):
    """(H in bits, level probabilities float64[nlev], n) of a level histogram (Sec. V-C)."""
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    H = np.zeros(1, dtype=np.float64)
    p = np.empty(hist.size, dtype=np.float64)
    n = np.zeros(1, dtype=np.uint64)
    _load().cdl_oracle_entropy(_ptr(hist), hist.size, _ptr(H), _ptr(p), _ptr(n))
    return float(H[0]), p, int(n[0])


def backward(x, g, q, lo, hi, alpha, window=0, rate_weight=0.0, level_prob=None):
    """Quantizer backward (Sec. V-B).  Returns a dict with grad_x (float64 array),
    grad_q, grad_alpha and the comparison scales abs_q, abs_alpha, mag_q, mag_alpha."""
    _check_levels(lo, hi)
    x = _f32(x)
    g = _f32(g)
    assert x.shape == g.shape
    lp = None if level_prob is None else np.ascontiguousarray(level_prob, dtype=np.float64)
    if lp is not None:
        assert lp.size == hi - lo + 1
    gx = np.empty(x.shape, dtype=np.float64)
    s = np.zeros(6, dtype=np.float64)
    sp = [ctypes.c_void_p(s.ctypes.data + 8 * i) for i in range(6)]
    _load().cdl_oracle_backward(_ptr(x), _ptr(g), x.size, q, lo, hi, alpha, window, rate_weight,
                                _ptr(lp), _ptr(gx), *sp)
    return {"grad_x": gx, "grad_q": float(s[0]), "grad_alpha": float(s[1]),
            "abs_q": float(s[2]), "abs_alpha": float(s[3]), "mag_q": float(s[4]), "mag_alpha": float(s[5])}


def _idx_bytes(a):
    a = np.asarray(a)
    if a.dtype not in (np.int8, np.uint8):
        raise TypeError("index operands are int8 or uint8")
    assert a.ndim == 2 and a.strides[1] == 1
    return a, a.strides[0], int(a.dtype == np.uint8)


def gemm_fwd(A, W):
    """ACC[m,n] = sum_k A[m,k] W[k,n] as int64; A int8|uint8 [M,K], W int8 [K,N]."""
    A, lda, au = _idx_bytes(A)
    W, ldw, wu = _idx_bytes(W)
    assert not wu and A.shape[1] == W.shape[0]
    M, K = A.shape
    N = W.shape[1]
    acc = np.empty((M, N), dtype=np.int64)
    _load().cdl_oracle_gemm_fwd(_ptr(A), lda, au, _ptr(W), ldw, M, N, K, _ptr(acc))
    return acc


def gemm_dx(G, W):
    """ACC[m,k] = sum_n G[m,n] W[k,n] as int64; G int8 [M,N], W int8 [K,N]."""
    G, ldg, gu = _idx_bytes(G)
    W, ldw, wu = _idx_bytes(W)
    assert not gu and not wu and G.shape[1] == W.shape[1]
    M, N = G.shape
    K = W.shape[0]
    acc = np.empty((M, K), dtype=np.int64)
    _load().cdl_oracle_gemm_dx(_ptr(G), ldg, _ptr(W), ldw, M, N, K, _ptr(acc))
    return acc


def gemm_dw(A, G):
    """ACC[k,n] = sum_m A[m,k] G[m,n] as int64; A int8|uint8 [M,K], G int8 [M,N]."""
    A, lda, au = _idx_bytes(A)
    G, ldg, gu = _idx_bytes(G)
    assert not gu and A.shape[0] == G.shape[0]
    M, K = A.shape
    N = G.shape[1]
    acc = np.empty((K, N), dtype=np.int64)
    _load().cdl_oracle_gemm_dw(_ptr(A), lda, au, _ptr(G), ldg, M, N, K, _ptr(acc))
    return acc


def _conv_dims(X, Wt, R, S):
    X = np.ascontiguousarray(X)
    if X.dtype not in (np.int8, np.uint8) or X.ndim != 4:
        raise TypeError("X is an int8 or uint8 [N,H,W,C] index tensor")
    Wt, ldw, wu = _idx_bytes(Wt)
    N, H, W, C = X.shape
    assert not wu and Wt.shape[0] == R * S * C
    return X, Wt, ldw, (N, H, W, C), Wt.shape[1]


def conv_out_dims(H, W, R, S, pad_h, pad_w, stride=1):
    return (H + 2 * pad_h - R) // stride + 1, (W + 2 * pad_w - S) // stride + 1


def conv_fwd(X, Wt, R, S, pad_h, pad_w, stride=1):
    """Strided cross-correlation with zero padding on indices, int64: X [N,H,W,C] int8|uint8, Wt [(r*S+s)*C+c, CO]
    int8 -> [N,P,Q,CO]."""
    X, Wt, ldw, (N, H, W, C), CO = _conv_dims(X, Wt, R, S)
    P, Q = conv_out_dims(H, W, R, S, pad_h, pad_w, stride)
    acc = np.empty((N, P, Q, CO), dtype=np.int64)
    _load().cdl_oracle_conv_fwd(_ptr(X), int(X.dtype == np.uint8), _ptr(Wt), ldw, N, H, W, C, R, S, pad_h, pad_w, CO,
                                stride, _ptr(acc))
    return acc


def conv_dx(G, Wt, x_shape, R, S, pad_h, pad_w, stride=1):
    """Adjoint of conv_fwd in X: G [N,P,Q,CO] int8, Wt as in conv_fwd -> [N,H,W,C] int64."""
    N, H, W, C = x_shape
    G = np.ascontiguousarray(G)
    Wt, ldw, wu = _idx_bytes(Wt)
    CO = Wt.shape[1]
    assert G.dtype == np.int8 and not wu and Wt.shape[0] == R * S * C
    assert G.shape == (N,) + conv_out_dims(H, W, R, S, pad_h, pad_w, stride) + (CO,)
    acc = np.empty((N, H, W, C), dtype=np.int64)
    _load().cdl_oracle_conv_dx(_ptr(G), _ptr(Wt), ldw, N, H, W, C, R, S, pad_h, pad_w, CO, stride, _ptr(acc))
    return acc


def conv_dw(X, G, R, S, pad_h, pad_w, stride=1):
    """Adjoint of conv_fwd in Wt: X [N,H,W,C] int8|uint8, G [N,P,Q,CO] int8 -> [(r*S+s)*C+c, CO] int64."""
    X = np.ascontiguousarray(X)
    G = np.ascontiguousarray(G)
    N, H, W, C = X.shape
    CO = G.shape[3]
    assert X.dtype in (np.int8, np.uint8) and G.dtype == np.int8
    assert G.shape == (N,) + conv_out_dims(H, W, R, S, pad_h, pad_w, stride) + (CO,)
    acc = np.empty((R * S * C, CO), dtype=np.int64)
    _load().cdl_oracle_conv_dw(_ptr(X), int(X.dtype == np.uint8), _ptr(G), N, H, W, C, R, S, pad_h, pad_w, CO, stride,
                               _ptr(acc))
    return acc


def gradient_digits(G, g_absmax):
    """Two-digit integer expansion of a real gradient tensor (backward products with an unquantized dL/dY):
    q1 = g_absmax / 127, q2 = q1 / 254 (binary32), i1 = hard index of g on step q1 in [-127, 127], r = the binary32
    value nearest g - i1 q1, i2 = hard index of r on step q2.  Returns (i1, i2, q1, q2)."""
    f32 = np.float32
    G = _f32(G)
    q1 = f32(f32(g_absmax) / f32(127.0))
    q2 = f32(q1 / f32(254.0))
    i1, _ = hard(G.reshape(-1), q1, -127, 127)
    # g - i1 q1 with one rounding: the product has at most 31 significant bits and the difference of two nearby
    # numbers is exact in binary64, so rounding the binary64 result to binary32 is the fused operation
    r = (G.reshape(-1).astype(np.float64) - i1.astype(np.float64) * np.float64(q1)).astype(f32)
    i2, _ = hard(r, q2, -127, 127)
    return i1.reshape(G.shape), i2.reshape(G.shape), q1, q2


def huffman_lengths(hist):
    """Code lengths of a Huffman code for the symbols with a non-zero count (Sec. VI-B: the average number of bits per
    weight / activation is measured with Huffman coding), by the textbook construction: repeatedly merge the two
    lightest subtrees.  Unused symbols get length 0; a single used symbol gets one bit.  Returns (lengths, total bits
    sum_k hist[k] * length[k]); the lengths depend on how ties are broken, the total does not."""
    import heapq
    h = [int(v) for v in np.asarray(hist).reshape(-1)]
    lengths = [0] * len(h)
    used = [k for k, c in enumerate(h) if c > 0]
    if len(used) == 1:
        lengths[used[0]] = 1
    elif len(used) > 1:
        heap = [(h[k], k, (k,)) for k in used]          # (weight, tie-break, symbols below this subtree)
        heapq.heapify(heap)
        nxt = len(h)
        while len(heap) > 1:
            w0, _, s0 = heapq.heappop(heap)
            w1, _, s1 = heapq.heappop(heap)
            for k in s0 + s1:
                lengths[k] += 1
            heapq.heappush(heap, (w0 + w1, nxt, s0 + s1))
            nxt += 1
    return np.array(lengths, dtype=np.int64), sum(c * l for c, l in zip(h, lengths))


def philox4x32_10(ctr, key):
    """One block of Philox4x32-10: ctr 4 x uint32, key 2 x uint32 -> 4 x uint32."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    _load().cdl_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def uniform(seed, e):
    """The uniform number in [0,1) element number e draws under `seed`."""
    return float(_load().cdl_oracle_uniform(int(seed), int(e)))


def sample(x, q, lo, hi, alpha, window=0, seed=0, first_index=0):
    """Q_p(x) by inversion (Sec. IV-A, Eq. (7)).  Returns (idx int32, u, cdf_lo, cdf_hi): the sampled indices, each
    element's uniform number and the cumulative probabilities just below / through the chosen level."""
    _check_levels(lo, hi)
    x = _f32(x)
    idx = np.empty(x.shape, dtype=np.int32)
    u, a, b = (np.empty(x.shape, dtype=np.float64) for _ in range(3))
    _load().cdl_oracle_sample(_ptr(x), x.size, q, lo, hi, alpha, window, int(seed), int(first_index),
                              _ptr(idx), _ptr(u), _ptr(a), _ptr(b))
    return idx, u, a, b


def mpmf(x, q, lo, hi, alpha, window=0):
    """Soft histogram sum_i P(. | x[i]) (Sec. V-C, Eq. (25) times n); float64[nlev]."""
    _check_levels(lo, hi)
    x = _f32(x)
    sums = np.zeros(hi - lo + 1, dtype=np.float64)
    _load().cdl_oracle_mpmf(_ptr(x), x.size, q, lo, hi, alpha, window, _ptr(sums))
    return sums
