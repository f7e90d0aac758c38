"""ctypes binding of libniti_b200.so: same names and argument order as include/niti.h.

Tensors are torch CUDA tensors (int8 payloads, int32 device scalars); torch is used for device
memory and streams only.  The workspace is a torch buffer owned by this object and handed to
the library on every call."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libniti_b200.so")

OK, ERR_ARG, ERR_SHAPE, ERR_WORKSPACE, ERR_RANGE, ERR_CUDA, ERR_DEVICE = range(7)
ROUND_PSR, ROUND_NEAREST = 0, 1
OP_LINEAR_FWD, OP_LINEAR_BWD, OP_CONV_FWD, OP_CONV_DGRAD, OP_CONV_WGRAD, OP_INT_XENT = range(6)
OP_LINEAR_BWD_UPDATE, OP_CONV_WGRAD_UPDATE = 6, 7
REDUCE_MAX_U32, REDUCE_MAX_U64, REDUCE_SUM_I32, REDUCE_SCATTER_SUM_I32, ALLGATHER_I8 = 0, 1, 2, 3, 4
_REDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int)

EXPORTS = [
    "niti_create", "niti_destroy", "niti_last_error", "niti_check", "niti_workspace_bytes",
    "niti_set_engine", "niti_set_reduce_hook", "niti_set_dp_shard", "niti_set_tap_cache", "niti_begin_step", "niti_launch_count", "niti_tc_launch_count", "niti_tc_pair_launch_count",
    "niti_redo_count", "niti_selftest_timeout", "niti_profile_enable", "niti_profile_read_launches",
    "niti_profile_read", "niti_linear_fwd", "niti_linear_bwd", "niti_conv_fwd",
    "niti_conv_dgrad", "niti_conv_wgrad", "niti_conv_fwd_pool", "niti_conv_fwd_strided", "niti_conv_dgrad_strided", "niti_conv_wgrad_strided",
    "niti_conv_wgrad_update", "niti_linear_bwd_update", "niti_int_xent", "niti_int_xent_noalloc", "niti_int_sgd_update",
    "niti_relu_fwd",
    "niti_relu_bwd", "niti_maxpool2_fwd", "niti_maxpool2_bwd", "niti_maxpool2_fwd_idx", "niti_maxpool2_bwd_idx",
]


class NitiError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("niti error %d: %s" % (code, msg))
        self.code = code


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads the built shared library; raises if it has not been built (no fallback exists)."""
    if not os.path.exists(_LIB_PATH):
        raise NitiError(ERR_CUDA, "%s is missing: run paper_2009_13108_b200/build.py" % _LIB_PATH)
    if os.path.dirname(_LIB_PATH) == _HERE:
        from .build import built_from_current_sources
        if built_from_current_sources() is False:
            import warnings
            warnings.warn("libniti_b200.so was built from other sources than the ones in csrc/: "
                          "run `python __graft_entry__.py` (or paper_2009_13108_b200/build.py) to rebuild it",
                          RuntimeWarning, stacklevel=2)
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
    lib.niti_create.argtypes = [C.POINTER(vp), i32]
    lib.niti_destroy.argtypes = [vp]
    lib.niti_last_error.argtypes = [vp]
    lib.niti_last_error.restype = C.c_char_p
    lib.niti_check.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    lib.niti_workspace_bytes.argtypes = [i32, C.POINTER(i64), i32]
    lib.niti_workspace_bytes.restype = sz
    lib.niti_set_engine.argtypes = [vp, i32]
    lib.niti_set_reduce_hook.argtypes = [vp, _REDUCE_FN, vp]
    lib.niti_set_dp_shard.argtypes = [vp, i32, i32]
    lib.niti_set_tap_cache.argtypes = [vp, vp, sz]
    lib.niti_begin_step.argtypes = [vp, vp, vp, sz]
    lib.niti_launch_count.argtypes = [vp]
    lib.niti_launch_count.restype = C.c_uint64
    lib.niti_tc_launch_count.argtypes = [vp]
    lib.niti_tc_launch_count.restype = C.c_uint64
    lib.niti_tc_pair_launch_count.argtypes = [vp]
    lib.niti_tc_pair_launch_count.restype = C.c_uint64
    lib.niti_profile_read_launches.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), i32]
    lib.niti_redo_count.argtypes = [vp, vp]
    lib.niti_selftest_timeout.argtypes = [vp, vp]
    lib.niti_redo_count.restype = C.c_int64
    lib.niti_profile_enable.argtypes = [vp, i32]
    lib.niti_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint64),
                                      C.POINTER(C.c_double)]
    lib.niti_linear_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, sz]
    lib.niti_linear_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32,
                                    vp, sz]
    lib.niti_conv_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp] + [i32] * 10 + [vp, sz]
    lib.niti_conv_dgrad.argtypes = [vp, vp, vp, vp, vp, vp, vp] + [i32] * 9 + [vp, sz]
    lib.niti_conv_wgrad.argtypes = [vp, vp, vp, vp, vp, vp] + [i32] * 10 + [vp, sz]
    lib.niti_conv_fwd_pool.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp] + [i32] * 10 + [vp, sz]
    lib.niti_conv_fwd_strided.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp] + [i32] * 11 + [vp, sz]
    lib.niti_conv_dgrad_strided.argtypes = [vp, vp, vp, vp, vp, vp, vp] + [i32] * 10 + [vp, sz]
    lib.niti_conv_wgrad_strided.argtypes = [vp, vp, vp, vp, vp, vp] + [i32] * 11 + [vp, sz]
    lib.niti_conv_wgrad_update.argtypes = [vp, vp, vp, vp, vp, vp] + [i32] * 10 + [vp, sz]
    lib.niti_linear_bwd_update.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, sz]
    lib.niti_int_xent.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, sz]
    lib.niti_int_xent_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32]
    lib.niti_int_sgd_update.argtypes = [vp, vp, vp, vp, i64]
    lib.niti_relu_fwd.argtypes = [vp, vp, vp, vp, i64]
    lib.niti_relu_bwd.argtypes = [vp, vp, vp, vp, vp, i64]
    lib.niti_maxpool2_fwd.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32]
    lib.niti_maxpool2_bwd.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32]
    lib.niti_maxpool2_fwd_idx.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32]
    lib.niti_maxpool2_bwd_idx.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32]
    return lib


def _ptr(t):
    return None if t is None else t.data_ptr()


class Niti:
    """One library context on one CUDA device plus a growable workspace."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise NitiError(ERR_CUDA, "no CUDA device: this library has no CPU path")
        self.lib = load_library()
        self.device = torch.device("cuda", device)
        h = C.c_void_p()
        rc = self.lib.niti_create(C.byref(h), device)
        if rc != OK:
            raise NitiError(rc, "niti_create failed (needs an sm_100 device)")
        self.h = h
        self._ws = torch.empty(1 << 20, dtype=torch.uint8, device=self.device)

    def close(self):
        if getattr(self, "h", None):
            self.lib.niti_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- helpers ----
    def _stream(self):
        return torch.cuda.current_stream(self.device).cuda_stream

    def _ck(self, rc):
        if rc != OK:
            raise NitiError(rc, self.lib.niti_last_error(self.h).decode())

    def workspace_bytes(self, op, dims) -> int:
        arr = (C.c_int64 * len(dims))(*dims)
        return int(self.lib.niti_workspace_bytes(op, arr, len(dims)))

    def set_reduce_hook(self, fn):
        """Exact data parallelism: ``fn(view, kind)`` combines the device tensor ``view`` (a slice of
        the workspace: int32 for REDUCE_MAX_U32 / REDUCE_SUM_I32, int64 for REDUCE_MAX_U64; the values
        to maximise are non-negative) in place over the ranks, ordered on the current stream.
        ``None`` removes the hook.  See ``dist_reducer`` for torch.distributed."""
        if fn is None:
            self._ck(self.lib.niti_set_reduce_hook(self.h, None, None))
            self._reduce_cb = None
            return

        def cb(user, stream, ptr, count, kind):
            try:
                dtype, size = {REDUCE_MAX_U32: (torch.int32, 4), REDUCE_MAX_U64: (torch.int64, 8),
                               REDUCE_SUM_I32: (torch.int32, 4), REDUCE_SCATTER_SUM_I32: (torch.int32, 4),
                               ALLGATHER_I8: (torch.int8, 1)}[kind]
                if kind == ALLGATHER_I8 and not (0 <= ptr - self._ws.data_ptr() < self._ws.numel()):
                    # the gathered tensor is the caller's gradient or weight tensor, not the workspace
                    fn(_device_view(ptr, count, self.device), kind)
                    return 0
                off = ptr - self._ws.data_ptr()
                if off < 0 or off + count * size > self._ws.numel():
                    return 2
                fn(self._ws[off:off + count * size].view(dtype), kind)
                return 0
            except Exception as exc:          # an exception must not cross the C boundary
                self._reduce_error = exc
                return 1

        self._reduce_cb = _REDUCE_FN(cb)      # keep the callback object alive
        self._ck(self.lib.niti_set_reduce_hook(self.h, self._reduce_cb, None))

    def set_dp_shard(self, rank: int, world: int):
        """niti_set_dp_shard: with world > 1 weight gradients are reduce-scattered, rounded per shard and
        all-gathered as int8; the reduction hook must handle REDUCE_SCATTER_SUM_I32 and ALLGATHER_I8."""
        self._ck(self.lib.niti_set_dp_shard(self.h, rank, world))

    def set_tap_cache(self, nbytes: int):
        """niti_set_tap_cache with a buffer of ``nbytes`` owned by this object (0 removes it): the gathered
        taps of a few-channel first layer are kept between its forward and its weight-gradient call."""
        self._tap = torch.empty(nbytes, dtype=torch.uint8, device=self.device) if nbytes else None
        self._ck(self.lib.niti_set_tap_cache(self.h, _ptr(self._tap), nbytes))

    def reserve_workspace(self, nbytes: int):
        if self._ws.numel() < nbytes:
            self._ck(self.lib.niti_begin_step(self.h, None, None, 0))      # the old buffer's headers are gone
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)

    def begin_step(self):
        """niti_begin_step on this object's workspace: one memset clears the headers that the next 64
        calls would otherwise clear one by one."""
        self._ck(self.lib.niti_begin_step(self.h, self._stream(), self._ws.data_ptr(), self._ws.numel()))

    def _ws_for(self, op, dims):
        need = self.workspace_bytes(op, dims)
        if need == 0:
            raise NitiError(ERR_ARG, "bad dims for workspace query")
        self.reserve_workspace(need)
        return self._ws.data_ptr(), self._ws.numel()

    def scalar(self, value: int = 0):
        return torch.full((1,), value, dtype=torch.int32, device=self.device)

    def set_engine(self, engine: int) -> int:
        return self.lib.niti_set_engine(self.h, engine)

    def launch_count(self) -> int:
        return int(self.lib.niti_launch_count(self.h))

    def tc_launch_count(self) -> int:
        return int(self.lib.niti_tc_launch_count(self.h))

    def tc_pair_launch_count(self) -> int:
        return int(self.lib.niti_tc_pair_launch_count(self.h))

    def redo_count(self) -> int:
        return int(self.lib.niti_redo_count(self.h, self._stream()))

    def selftest_timeout(self):
        self._ck(self.lib.niti_selftest_timeout(self.h, self._stream()))

    def profile_enable(self, on: bool):
        self._ck(self.lib.niti_profile_enable(self.h, int(on)))

    def profile_read_launches(self, max_n: int = 8192):
        """[(ms, int8 ops)] of every recorded tensor-core launch, in launch order."""
        ms = (C.c_double * max_n)()
        ops = (C.c_double * max_n)()
        n = self.lib.niti_profile_read_launches(self.h, ms, ops, max_n)
        if n < 0:
            raise NitiError(ERR_CUDA, "niti_profile_read_launches failed")
        return [(ms[i], ops[i]) for i in range(n)]

    def profile_read(self):
        """(summed ms, launches, summed int8 ops) of the tensor-core kernel since the last read."""
        ms, nl, ops = C.c_double(0), C.c_uint64(0), C.c_double(0)
        self._ck(self.lib.niti_profile_read(self.h, C.byref(ms), C.byref(nl), C.byref(ops)))
        return ms.value, int(nl.value), ops.value

    def check(self) -> int:
        st = C.c_uint32(0)
        rc = self.lib.niti_check(self.h, self._stream(), C.byref(st))
        if rc != OK:
            raise NitiError(rc, "device status 0x%x" % st.value)
        return st.value

    # ---- layer ops (names follow include/niti.h) ----
    def linear_fwd(self, a, s_a, w, s_w, out=None, s_out=None, b_out=None, relu=False,
                   round_mode=ROUND_PSR):
        M, K = a.shape
        N = w.shape[0]
        out = out if out is not None else torch.empty((M, N), dtype=torch.int8, device=self.device)
        s_out = s_out if s_out is not None else self.scalar()
        b_out = b_out if b_out is not None else self.scalar()
        ws, wsb = self._ws_for(OP_LINEAR_FWD, [M, N, K])
        self._ck(self.lib.niti_linear_fwd(self.h, self._stream(), _ptr(a), _ptr(s_a), _ptr(w),
                                          _ptr(s_w), _ptr(out), _ptr(s_out), _ptr(b_out), M, N, K,
                                          int(relu), round_mode, ws, wsb))
        return out, s_out, b_out

    def linear_bwd(self, a, e, w, need_e_prev=True, relu_mask_src=None, e_prev=None, g=None,
                   b_e=None, b_g=None, m_u=5, round_mode=ROUND_PSR):
        M, K = a.shape
        N = e.shape[1]
        g = g if g is not None else torch.empty((N, K), dtype=torch.int8, device=self.device)
        if need_e_prev and e_prev is None:
            e_prev = torch.empty((M, K), dtype=torch.int8, device=self.device)
        b_e = b_e if b_e is not None else self.scalar()
        b_g = b_g if b_g is not None else self.scalar()
        ws, wsb = self._ws_for(OP_LINEAR_BWD, [M, N, K])
        self._ck(self.lib.niti_linear_bwd(self.h, self._stream(), _ptr(a), _ptr(e), _ptr(w),
                                          _ptr(e_prev) if need_e_prev else None,
                                          _ptr(relu_mask_src), _ptr(g), _ptr(b_e), _ptr(b_g), M, N,
                                          K, m_u, round_mode, ws, wsb))
        return (e_prev if need_e_prev else None), g, b_e, b_g

    def conv_fwd(self, x, s_x, w, s_w, y=None, s_y=None, b_y=None, pad=1, relu=False,
                 round_mode=ROUND_PSR, stride=1):
        """niti_conv_fwd (stride 1) / niti_conv_fwd_strided."""
        B, H, W, Ci = x.shape
        Co, R, S, _ = w.shape
        Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
        y = y if y is not None else torch.empty((B, Ho, Wo, Co), dtype=torch.int8, device=self.device)
        s_y = s_y if s_y is not None else self.scalar()
        b_y = b_y if b_y is not None else self.scalar()
        ws, wsb = self._ws_for(OP_CONV_FWD, [B, H, W, Ci, Co, R, S, pad, stride])
        if stride == 1:
            self._ck(self.lib.niti_conv_fwd(self.h, self._stream(), _ptr(x), _ptr(s_x), _ptr(w),
                                            _ptr(s_w), _ptr(y), _ptr(s_y), _ptr(b_y), B, H, W, Ci, Co,
                                            R, S, pad, int(relu), round_mode, ws, wsb))
        else:
            self._ck(self.lib.niti_conv_fwd_strided(self.h, self._stream(), _ptr(x), _ptr(s_x), _ptr(w),
                                                    _ptr(s_w), _ptr(y), _ptr(s_y), _ptr(b_y), B, H, W, Ci, Co,
                                                    R, S, pad, stride, int(relu), round_mode, ws, wsb))
        return y, s_y, b_y

    def conv_fwd_pool(self, x, s_x, w, s_w, y=None, y_pool=None, s_y=None, b_y=None, pad=1, relu=True,
                      round_mode=ROUND_PSR):
        """niti_conv_fwd_pool: the convolution's output and its 2 x 2 max-pool in one call."""
        B, H, W, Ci = x.shape
        Co, R, S, _ = w.shape
        Ho, Wo = H + 2 * pad - R + 1, W + 2 * pad - S + 1
        y = y if y is not None else torch.empty((B, Ho, Wo, Co), dtype=torch.int8, device=self.device)
        y_pool = y_pool if y_pool is not None else torch.empty((B, Ho // 2, Wo // 2, Co), dtype=torch.int8,
                                                               device=self.device)
        s_y = s_y if s_y is not None else self.scalar()
        b_y = b_y if b_y is not None else self.scalar()
        ws, wsb = self._ws_for(OP_CONV_FWD, [B, H, W, Ci, Co, R, S, pad])
        self._ck(self.lib.niti_conv_fwd_pool(self.h, self._stream(), _ptr(x), _ptr(s_x), _ptr(w), _ptr(s_w),
                                             _ptr(y), _ptr(y_pool), _ptr(s_y), _ptr(b_y), B, H, W, Ci, Co, R, S,
                                             pad, int(relu), round_mode, ws, wsb))
        return y, y_pool, s_y, b_y

    def conv_dgrad(self, e, w, in_hw, e_prev=None, relu_mask_src=None, b_e=None, pad=1,
                   round_mode=ROUND_PSR, stride=1):
        B = e.shape[0]
        H, W = in_hw
        Co, R, S, Ci = w.shape
        e_prev = e_prev if e_prev is not None else torch.empty((B, H, W, Ci), dtype=torch.int8,
                                                                device=self.device)
        b_e = b_e if b_e is not None else self.scalar()
        ws, wsb = self._ws_for(OP_CONV_DGRAD, [B, H, W, Ci, Co, R, S, pad, stride])
        if stride == 1:
            self._ck(self.lib.niti_conv_dgrad(self.h, self._stream(), _ptr(e), _ptr(w), _ptr(e_prev),
                                              _ptr(relu_mask_src), _ptr(b_e), B, H, W, Ci, Co, R, S,
                                              pad, round_mode, ws, wsb))
        else:
            self._ck(self.lib.niti_conv_dgrad_strided(self.h, self._stream(), _ptr(e), _ptr(w), _ptr(e_prev),
                                                      _ptr(relu_mask_src), _ptr(b_e), B, H, W, Ci, Co, R, S,
                                                      pad, stride, round_mode, ws, wsb))
        return e_prev, b_e

    def conv_wgrad(self, x, e, rs=(3, 3), g=None, b_g=None, pad=1, m_u=5, round_mode=ROUND_PSR, stride=1):
        B, H, W, Ci = x.shape
        Co = e.shape[3]
        R, S = rs
        g = g if g is not None else torch.empty((Co, R, S, Ci), dtype=torch.int8, device=self.device)
        b_g = b_g if b_g is not None else self.scalar()
        ws, wsb = self._ws_for(OP_CONV_WGRAD, [B, H, W, Ci, Co, R, S, pad, stride])
        if stride == 1:
            self._ck(self.lib.niti_conv_wgrad(self.h, self._stream(), _ptr(x), _ptr(e), _ptr(g),
                                              _ptr(b_g), B, H, W, Ci, Co, R, S, pad, m_u, round_mode,
                                              ws, wsb))
        else:
            self._ck(self.lib.niti_conv_wgrad_strided(self.h, self._stream(), _ptr(x), _ptr(e), _ptr(g),
                                                      _ptr(b_g), B, H, W, Ci, Co, R, S, pad, stride, m_u,
                                                      round_mode, ws, wsb))
        return g, b_g

    def conv_wgrad_update(self, x, e, w, b_g=None, pad=1, m_u=5, round_mode=ROUND_PSR):
        """Weight gradient of the convolution subtracted from w in place (the gradient is not returned)."""
        B, H, W, Ci = x.shape
        Co, R, S, _ = w.shape
        b_g = b_g if b_g is not None else self.scalar()
        ws, wsb = self._ws_for(OP_CONV_WGRAD_UPDATE, [B, H, W, Ci, Co, R, S, pad])
        self._ck(self.lib.niti_conv_wgrad_update(self.h, self._stream(), _ptr(x), _ptr(e), _ptr(w),
                                                 _ptr(b_g), B, H, W, Ci, Co, R, S, pad, m_u,
                                                 round_mode, ws, wsb))
        return w, b_g

    def linear_bwd_update(self, a, e, w, need_e_prev=True, relu_mask_src=None, e_prev=None,
                          b_e=None, b_g=None, m_u=5, round_mode=ROUND_PSR):
        """linear_bwd with the weight update fused in: e_prev from the old weights, then w updated in place."""
        M, K = a.shape
        N = e.shape[1]
        if need_e_prev and e_prev is None:
            e_prev = torch.empty((M, K), dtype=torch.int8, device=self.device)
        b_e = b_e if b_e is not None else self.scalar()
        b_g = b_g if b_g is not None else self.scalar()
        ws, wsb = self._ws_for(OP_LINEAR_BWD_UPDATE, [M, N, K])
        self._ck(self.lib.niti_linear_bwd_update(self.h, self._stream(), _ptr(a), _ptr(e), _ptr(w),
                                                 _ptr(e_prev) if need_e_prev else None,
                                                 _ptr(relu_mask_src), _ptr(b_e), _ptr(b_g), M, N, K,
                                                 m_u, round_mode, ws, wsb))
        return (e_prev if need_e_prev else None), b_e, b_g

    def int_xent(self, a, s_a, labels, e=None, b_e=None, n_correct=None, round_mode=ROUND_PSR):
        B, N = a.shape
        e = e if e is not None else torch.empty((B, N), dtype=torch.int8, device=self.device)
        b_e = b_e if b_e is not None else self.scalar()
        n_correct = n_correct if n_correct is not None else self.scalar()
        ws, wsb = self._ws_for(OP_INT_XENT, [B, N])
        self._ck(self.lib.niti_int_xent(self.h, self._stream(), _ptr(a), _ptr(s_a), _ptr(labels),
                                        _ptr(e), _ptr(b_e), _ptr(n_correct), B, N, round_mode, ws,
                                        wsb))
        return e, b_e, n_correct

    def int_xent_noalloc(self, a, s_a, labels, e, b_e=None, n_correct=None, round_mode=ROUND_PSR):
        """niti_int_xent_noalloc: the caller passes every buffer (this wrapper allocates nothing
        either); no context, no workspace.  Returns the library's return code."""
        B, N = a.shape
        return int(self.lib.niti_int_xent_noalloc(self._stream(), _ptr(a), _ptr(s_a), _ptr(labels),
                                                  _ptr(e), _ptr(b_e), _ptr(n_correct), B, N,
                                                  round_mode))

    def int_sgd_update(self, w, g):
        self._ck(self.lib.niti_int_sgd_update(self.h, self._stream(), _ptr(w), _ptr(g), w.numel()))
        return w

    def relu_fwd(self, x, y=None):
        y = y if y is not None else torch.empty_like(x)
        self._ck(self.lib.niti_relu_fwd(self.h, self._stream(), _ptr(x), _ptr(y), x.numel()))
        return y

    def relu_bwd(self, y, e_out, e_in=None):
        e_in = e_in if e_in is not None else torch.empty_like(e_out)
        self._ck(self.lib.niti_relu_bwd(self.h, self._stream(), _ptr(y), _ptr(e_out), _ptr(e_in),
                                        y.numel()))
        return e_in

    def maxpool2_fwd(self, x, y=None):
        B, H, W, Cc = x.shape
        y = y if y is not None else torch.empty((B, H // 2, W // 2, Cc), dtype=torch.int8,
                                                device=self.device)
        self._ck(self.lib.niti_maxpool2_fwd(self.h, self._stream(), _ptr(x), _ptr(y), B, H, W, Cc))
        return y

    def maxpool2_fwd_idx(self, x, y=None, idx=None):
        """Max-pool that also records the routing codes (half a byte per output element)."""
        B, H, W, Cc = x.shape
        y = y if y is not None else torch.empty((B, H // 2, W // 2, Cc), dtype=torch.int8,
                                                device=self.device)
        idx = idx if idx is not None else torch.empty((B, H // 2, W // 2, Cc // 2), dtype=torch.uint8,
                                                      device=self.device)
        self._ck(self.lib.niti_maxpool2_fwd_idx(self.h, self._stream(), _ptr(x), _ptr(y), _ptr(idx),
                                                B, H, W, Cc))
        return y, idx

    def maxpool2_bwd_idx(self, e_out, idx, in_shape, e_in=None, relu=False):
        B, H, W, Cc = in_shape
        e_in = e_in if e_in is not None else torch.empty(tuple(in_shape), dtype=torch.int8,
                                                         device=self.device)
        self._ck(self.lib.niti_maxpool2_bwd_idx(self.h, self._stream(), _ptr(e_out), _ptr(idx),
                                                _ptr(e_in), B, H, W, Cc, int(relu)))
        return e_in

    def maxpool2_bwd(self, x, e_out, e_in=None, relu=False):
        B, H, W, Cc = x.shape
        e_in = e_in if e_in is not None else torch.empty_like(x)
        self._ck(self.lib.niti_maxpool2_bwd(self.h, self._stream(), _ptr(x), _ptr(e_out),
                                            _ptr(e_in), B, H, W, Cc, int(relu)))
        return e_in


def _device_view(ptr: int, nbytes: int, device):
    """An int8 tensor over ``nbytes`` of device memory at ``ptr`` (memory owned by someone else)."""
    class _Mem:
        __cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|i1", "data": (ptr, False), "version": 3}
    return torch.as_tensor(_Mem(), device=device)


def dist_reducer(group=None):
    """A reduction hook for ``Niti.set_reduce_hook`` over a torch.distributed process group (NCCL: the
    collectives are ordered on the current stream; gloo: through the host).  Reduce-scatter and
    all-gather run in place on the tensor the library hands over; backends without a reduce-scatter
    (gloo) all-reduce instead, which leaves the same sums in the rank's slice."""
    import torch.distributed as dist

    def reduce(view, kind):
        if kind == REDUCE_SCATTER_SUM_I32:
            world, rank = dist.get_world_size(group), dist.get_rank(group)
            n = view.numel() // world
            if dist.get_backend(group) == "nccl":
                dist.reduce_scatter_tensor(view[rank * n:(rank + 1) * n], view, op=dist.ReduceOp.SUM, group=group)
            else:
                dist.all_reduce(view, op=dist.ReduceOp.SUM, group=group)
        elif kind == ALLGATHER_I8:
            world, rank = dist.get_world_size(group), dist.get_rank(group)
            n = view.numel() // world
            if dist.get_backend(group) == "nccl":
                dist.all_gather_into_tensor(view, view[rank * n:(rank + 1) * n], group=group)
            else:
                parts = [torch.empty(n, dtype=view.dtype, device=view.device) for _ in range(world)]
                dist.all_gather(parts, view[rank * n:(rank + 1) * n].clone(), group=group)
                for r, part in enumerate(parts):
                    view[r * n:(r + 1) * n].copy_(part)
        else:
            op = dist.ReduceOp.SUM if kind == REDUCE_SUM_I32 else dist.ReduceOp.MAX
            dist.all_reduce(view, op=op, group=group)

    return reduce
