"""ctypes binding of ``niti_oracle.c`` (host pointers, numpy arrays).

Test infrastructure: see the header of ``niti_oracle.c``.  ``build()`` compiles the C file
with gcc into ``libniti_oracle.so`` next to it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "niti_oracle.c")
_LIB = os.path.join(_HERE, "libniti_oracle.so")

OK, ERR_ARG, ERR_RANGE, ERR_OVERFLOW = 0, 1, 4, 7
ROUND_PSR, ROUND_NEAREST = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _declare(_lib)
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops of the oracle use (OMP_NUM_THREADS or the core count)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


_i8p = C.POINTER(C.c_int8)
_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_i64 = C.c_int64
_i32 = C.c_int32
_int = C.c_int


def _declare(L):
    L.niti_ref_bitwidth.restype = _i32
    L.niti_ref_bitwidth.argtypes = [_i64p, _i64]
    for f in (L.niti_ref_psr, L.niti_ref_round_nearest):
        f.restype = _i32
        f.argtypes = [_i64, _i32, _i32]
    L.niti_ref_round_stochastic.restype = _i32
    L.niti_ref_round_stochastic.argtypes = [_i64, _i32, _i32, _i64]
    L.niti_ref_shift_round.restype = _int
    L.niti_ref_shift_round.argtypes = [_i64p, _i64, _i32, _i32, _i8p, _i32p, _i32p]
    L.niti_ref_overflows_int32.restype = _int
    L.niti_ref_overflows_int32.argtypes = [_i64p, _i64]
    for f in (L.niti_ref_fc_fwd_acc, L.niti_ref_fc_dgrad_acc, L.niti_ref_fc_wgrad_acc):
        f.restype = None
        f.argtypes = [_i8p, _i8p, _i64p, _i64, _i64, _i64]
    for f in (L.niti_ref_conv_fwd_acc_s, L.niti_ref_conv_dgrad_acc_s, L.niti_ref_conv_wgrad_acc_s):
        f.restype = None
        f.argtypes = [_i8p, _i8p, _i64p] + [_i64] * 9
    L.niti_ref_xent_acc.restype = _int
    L.niti_ref_xent_acc.argtypes = [_i8p, _i32, _i32p, _i64p, _i64, _i64]
    L.niti_ref_count_correct.restype = _i32
    L.niti_ref_count_correct.argtypes = [_i8p, _i32p, _i64, _i64]
    L.niti_ref_sgd_update.restype = None
    L.niti_ref_sgd_update.argtypes = [_i8p, _i8p, _i64]
    L.niti_ref_relu_fwd.restype = None
    L.niti_ref_relu_fwd.argtypes = [_i8p, _i8p, _i64]
    L.niti_ref_relu_bwd.restype = None
    L.niti_ref_relu_bwd.argtypes = [_i8p, _i8p, _i8p, _i64]
    L.niti_ref_maxpool2_fwd.restype = None
    L.niti_ref_maxpool2_fwd.argtypes = [_i8p, _i8p, _i64, _i64, _i64, _i64]
    L.niti_ref_maxpool2_bwd.restype = None
    L.niti_ref_maxpool2_bwd.argtypes = [_i8p, _i8p, _i8p, _i64, _i64, _i64, _i64]
    L.niti_ref_linear_fwd.restype = _int
    L.niti_ref_linear_fwd.argtypes = [_i8p, _i32, _i8p, _i32, _i8p, _i32p, _i32p, _i64, _i64, _i64,
                                      _int, _int]
    L.niti_ref_linear_bwd.restype = _int
    L.niti_ref_linear_bwd.argtypes = [_i8p, _i8p, _i8p, _i8p, _i8p, _i8p, _i32p, _i32p, _i64, _i64,
                                      _i64, _int, _int]
    L.niti_ref_conv_fwd_s.restype = _int
    L.niti_ref_conv_fwd_s.argtypes = [_i8p, _i32, _i8p, _i32, _i8p, _i32p, _i32p] + [_i64] * 9 + \
        [_int, _int]
    L.niti_ref_conv_dgrad_s.restype = _int
    L.niti_ref_conv_dgrad_s.argtypes = [_i8p, _i8p, _i8p, _i8p, _i32p] + [_i64] * 9 + [_int]
    L.niti_ref_conv_wgrad_s.restype = _int
    L.niti_ref_conv_wgrad_s.argtypes = [_i8p, _i8p, _i8p, _i32p] + [_i64] * 9 + [_int, _int]
    L.niti_ref_int_xent.restype = _int
    L.niti_ref_int_xent.argtypes = [_i8p, _i32, _i32p, _i8p, _i32p, _i32p, _i64, _i64, _int]


def _p8(a):
    return None if a is None else a.ctypes.data_as(_i8p)


def _p32(a):
    return a.ctypes.data_as(_i32p)


def _p64(a):
    return a.ctypes.data_as(_i64p)


def _c8(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.int8
    return a


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle returned error code %d" % code)
        self.code = code


def _check(rc, allow_overflow=False):
    if rc == OK or (allow_overflow and rc == ERR_OVERFLOW):
        return rc
    raise OracleError(rc)


# ---- scalar / tensor rounding primitives -------------------------------------------------

def bitwidth(v) -> int:
    v = np.ascontiguousarray(v, dtype=np.int64)
    return int(lib().niti_ref_bitwidth(_p64(v), v.size))


def psr(x: int, bp: int, mbits: int = 7) -> int:
    return int(lib().niti_ref_psr(int(x), bp, mbits))


def round_nearest(x: int, bp: int, mbits: int = 7) -> int:
    return int(lib().niti_ref_round_nearest(int(x), bp, mbits))


def round_stochastic(x: int, bp: int, mbits: int, r: int) -> int:
    return int(lib().niti_ref_round_stochastic(int(x), bp, mbits, int(r)))


def shift_round(acc, mbits=7, round_mode=ROUND_PSR):
    """Returns (q int8 with acc's shape, b, bp)."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    q = np.empty(acc.shape, dtype=np.int8)
    b = np.zeros(1, np.int32)
    bp = np.zeros(1, np.int32)
    _check(lib().niti_ref_shift_round(_p64(acc), acc.size, mbits, round_mode, _p8(q), _p32(b),
                                      _p32(bp)))
    return q, int(b[0]), int(bp[0])


# ---- accumulators (int64) ----------------------------------------------------------------

def fc_fwd_acc(a, w):
    a, w = _c8(a), _c8(w)
    M, K = a.shape
    N = w.shape[0]
    acc = np.empty((M, N), np.int64)
    lib().niti_ref_fc_fwd_acc(_p8(a), _p8(w), _p64(acc), M, N, K)
    return acc


def fc_dgrad_acc(e, w):
    e, w = _c8(e), _c8(w)
    M, N = e.shape
    K = w.shape[1]
    acc = np.empty((M, K), np.int64)
    lib().niti_ref_fc_dgrad_acc(_p8(e), _p8(w), _p64(acc), M, N, K)
    return acc


def fc_wgrad_acc(a, e):
    a, e = _c8(a), _c8(e)
    M, K = a.shape
    N = e.shape[1]
    acc = np.empty((N, K), np.int64)
    lib().niti_ref_fc_wgrad_acc(_p8(a), _p8(e), _p64(acc), M, N, K)
    return acc


def conv_out_hw(H, W, R, S, pad, stride=1):
    """Output size of a convolution: (H + 2 pad - R) // stride + 1."""
    return (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1


def conv_fwd_acc(x, w, pad=1, stride=1):
    x, w = _c8(x), _c8(w)
    B, H, W, Ci = x.shape
    Co, R, S, _ = w.shape
    Ho, Wo = conv_out_hw(H, W, R, S, pad, stride)
    acc = np.empty((B, Ho, Wo, Co), np.int64)
    lib().niti_ref_conv_fwd_acc_s(_p8(x), _p8(w), _p64(acc), B, H, W, Ci, Co, R, S, pad, stride)
    return acc


def conv_dgrad_acc(e, w, in_hw, pad=1, stride=1):
    e, w = _c8(e), _c8(w)
    B = e.shape[0]
    H, W = in_hw
    Co, R, S, Ci = w.shape
    assert e.shape[1:3] == conv_out_hw(H, W, R, S, pad, stride)
    acc = np.empty((B, H, W, Ci), np.int64)
    lib().niti_ref_conv_dgrad_acc_s(_p8(e), _p8(w), _p64(acc), B, H, W, Ci, Co, R, S, pad, stride)
    return acc


def conv_wgrad_acc(x, e, rs=(3, 3), pad=1, stride=1):
    x, e = _c8(x), _c8(e)
    B, H, W, Ci = x.shape
    Co = e.shape[3]
    R, S = rs
    assert e.shape[1:3] == conv_out_hw(H, W, R, S, pad, stride)
    acc = np.empty((Co, R, S, Ci), np.int64)
    lib().niti_ref_conv_wgrad_acc_s(_p8(x), _p8(e), _p64(acc), B, H, W, Ci, Co, R, S, pad, stride)
    return acc


def xent_acc(a, s_a, labels):
    a = _c8(a)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    B, N = a.shape
    e32 = np.empty((B, N), np.int64)
    _check(lib().niti_ref_xent_acc(_p8(a), s_a, _p32(labels), _p64(e32), B, N))
    return e32


# ---- elementwise ops ---------------------------------------------------------------------

def sgd_update(w, g):
    """Returns the updated copy of w."""
    w = _c8(w).copy()
    g = _c8(g)
    lib().niti_ref_sgd_update(_p8(w), _p8(g), w.size)
    return w


def relu_fwd(x):
    x = _c8(x)
    y = np.empty_like(x)
    lib().niti_ref_relu_fwd(_p8(x), _p8(y), x.size)
    return y


def relu_bwd(y, e_out):
    y, e_out = _c8(y), _c8(e_out)
    e_in = np.empty_like(e_out)
    lib().niti_ref_relu_bwd(_p8(y), _p8(e_out), _p8(e_in), y.size)
    return e_in


def maxpool2_fwd(x):
    x = _c8(x)
    B, H, W, Cc = x.shape
    y = np.empty((B, H // 2, W // 2, Cc), np.int8)
    lib().niti_ref_maxpool2_fwd(_p8(x), _p8(y), B, H, W, Cc)
    return y


def maxpool2_bwd(x, e_out):
    x, e_out = _c8(x), _c8(e_out)
    B, H, W, Cc = x.shape
    e_in = np.empty_like(x)
    lib().niti_ref_maxpool2_bwd(_p8(x), _p8(e_out), _p8(e_in), B, H, W, Cc)
    return e_in


# ---- composed layer ops (argument lists mirror the GPU library) --------------------------

def linear_fwd(a, s_a, w, s_w, relu=False, round_mode=ROUND_PSR, allow_overflow=False):
    """Returns (out int8 [M,N], s_out, b)."""
    a, w = _c8(a), _c8(w)
    M, K = a.shape
    N = w.shape[0]
    out = np.empty((M, N), np.int8)
    s = np.zeros(1, np.int32)
    b = np.zeros(1, np.int32)
    _check(lib().niti_ref_linear_fwd(_p8(a), s_a, _p8(w), s_w, _p8(out), _p32(s), _p32(b), M, N, K,
                                     int(relu), round_mode), allow_overflow)
    return out, int(s[0]), int(b[0])


def linear_bwd(a, e, w, need_e_prev=True, mask=None, m_u=5, round_mode=ROUND_PSR,
               allow_overflow=False):
    """Returns (e_prev int8 [M,K] or None, g int8 [N,K], b_e, b_g)."""
    a, e, w = _c8(a), _c8(e), _c8(w)
    M, K = a.shape
    N = e.shape[1]
    g = np.empty((N, K), np.int8)
    e_prev = np.empty((M, K), np.int8) if need_e_prev else None
    if mask is not None:
        mask = _c8(mask)
    be = np.zeros(1, np.int32)
    bg = np.zeros(1, np.int32)
    _check(lib().niti_ref_linear_bwd(_p8(a), _p8(e), _p8(w), _p8(e_prev), _p8(mask), _p8(g),
                                     _p32(be), _p32(bg), M, N, K, m_u, round_mode), allow_overflow)
    return e_prev, g, int(be[0]), int(bg[0])


def conv_fwd(x, s_x, w, s_w, pad=1, relu=False, round_mode=ROUND_PSR, allow_overflow=False, stride=1):
    """Returns (y int8 NHWC, s_y, b)."""
    x, w = _c8(x), _c8(w)
    B, H, W, Ci = x.shape
    Co, R, S, _ = w.shape
    Ho, Wo = conv_out_hw(H, W, R, S, pad, stride)
    y = np.empty((B, Ho, Wo, Co), np.int8)
    s = np.zeros(1, np.int32)
    b = np.zeros(1, np.int32)
    _check(lib().niti_ref_conv_fwd_s(_p8(x), s_x, _p8(w), s_w, _p8(y), _p32(s), _p32(b), B, H, W, Ci,
                                     Co, R, S, pad, stride, int(relu), round_mode), allow_overflow)
    return y, int(s[0]), int(b[0])


def conv_dgrad(e, w, in_hw, pad=1, mask=None, round_mode=ROUND_PSR, allow_overflow=False, stride=1):
    """Returns (e_prev int8 [B,H,W,Ci], b)."""
    e, w = _c8(e), _c8(w)
    B = e.shape[0]
    H, W = in_hw
    Co, R, S, Ci = w.shape
    assert e.shape[1:3] == conv_out_hw(H, W, R, S, pad, stride)
    e_prev = np.empty((B, H, W, Ci), np.int8)
    if mask is not None:
        mask = _c8(mask)
    b = np.zeros(1, np.int32)
    _check(lib().niti_ref_conv_dgrad_s(_p8(e), _p8(w), _p8(e_prev), _p8(mask), _p32(b), B, H, W, Ci,
                                       Co, R, S, pad, stride, round_mode), allow_overflow)
    return e_prev, int(b[0])


def conv_wgrad(x, e, rs=(3, 3), pad=1, m_u=5, round_mode=ROUND_PSR, allow_overflow=False, stride=1):
    """Returns (g int8 [Co,R,S,Ci], b)."""
    x, e = _c8(x), _c8(e)
    B, H, W, Ci = x.shape
    Co = e.shape[3]
    R, S = rs
    assert e.shape[1:3] == conv_out_hw(H, W, R, S, pad, stride)
    g = np.empty((Co, R, S, Ci), np.int8)
    b = np.zeros(1, np.int32)
    _check(lib().niti_ref_conv_wgrad_s(_p8(x), _p8(e), _p8(g), _p32(b), B, H, W, Ci, Co, R, S, pad,
                                       stride, m_u, round_mode), allow_overflow)
    return g, int(b[0])


def int_xent(a, s_a, labels, round_mode=ROUND_PSR):
    """Returns (e int8 [B,N], b, n_correct)."""
    a = _c8(a)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    B, N = a.shape
    e = np.empty((B, N), np.int8)
    b = np.zeros(1, np.int32)
    nc = np.zeros(1, np.int32)
    _check(lib().niti_ref_int_xent(_p8(a), s_a, _p32(labels), _p8(e), _p32(b), _p32(nc), B, N,
                                   round_mode))
    return e, int(b[0]), int(nc[0])
