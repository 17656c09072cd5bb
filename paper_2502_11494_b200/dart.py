"""Thin ctypes binding of ``libdart.so`` (declared in ``include/dart.h``).

Argument marshalling only: every step of the reduction runs in the library's CUDA kernels.
There is no CPU fallback; if the library is missing the first use raises.  The module-level
functions carry the C names; :class:`Dart` wraps a context for torch tensors (torch supplies
device memory and streams, nothing else).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdart.so")

DART_OK = 0
DART_ERR_NULL, DART_ERR_BAD_SHAPE, DART_ERR_ALIGN, DART_ERR_ALIAS = -1, -2, -3, -4
DART_ERR_CUDA, DART_ERR_NOMEM, DART_ERR_TIMEOUT, DART_ERR_CHECK, DART_ERR_UNSUPPORTED = -5, -6, -7, -8, -9
DART_FLAG_HOST_STAGING = 1
DART_PATH_AUTO, DART_PATH_STAGED, DART_PATH_FUSED, DART_PATH_TWO_PASS, DART_PATH_RESIDENT, DART_PATH_SPLIT, DART_PATH_PAIRED = 0, 1, 2, 3, 4, 5, 6
DART_RETAIN_AUTO, DART_RETAIN_SERIAL, DART_RETAIN_LISTS, DART_RETAIN_BANDS, DART_RETAIN_FUSED = 0, 1, 2, 3, 4
DART_RULE_QUOTAS, DART_RULE_GLOBAL, DART_RULE_UNION = 0, 1, 2
DART_PIVOTS_BY_SCORE, DART_PIVOTS_MIXED, DART_PIVOTS_RANDOM = 0, 1, 2

EXPORTS = (
    "dart_create", "dart_destroy", "dart_set_shape", "dart_reduce", "dart_reduce_ex", "dart_reduce_host",
    "dart_status", "dart_status_detail", "dart_last_cuda_error", "dart_workspace_bytes", "dart_launch_count",
    "dart_profile_enable", "dart_profile_read", "dart_strerror", "dart_version", "dart_pivots_static",
    "dart_gather_rows",
)
DART_STATIC_MAX_ROWS = 262144


class dart_desc(ctypes.Structure):
    _fields_ = [("B_max", ctypes.c_int32), ("S_max", ctypes.c_int32), ("d", ctypes.c_int32),
                ("P_max", ctypes.c_int32), ("Kp_max", ctypes.c_int32), ("device", ctypes.c_int32),
                ("flags", ctypes.c_uint32)]


class dart_opts(ctypes.Structure):
    _fields_ = [("norm_kind", ctypes.c_int32), ("pivot_smallest", ctypes.c_int32), ("path", ctypes.c_int32),
                ("wait_limit", ctypes.c_int32), ("sweep_lag", ctypes.c_int32),
                ("test_withhold_pivots", ctypes.c_int32), ("retention", ctypes.c_int32), ("rule", ctypes.c_int32),
                ("cosine_on_hidden", ctypes.c_int32), ("text_pivots", ctypes.c_int32), ("pivots_in", ctypes.c_void_p),
                ("cu_seqlens", ctypes.c_void_p), ("resident_split", ctypes.c_int32), ("pivot_source", ctypes.c_int32),
                ("n_text_pivots", ctypes.c_int32), ("seed", ctypes.c_uint64), ("sample_base", ctypes.c_int32),
                ("tune", ctypes.c_int32)]


class dart_debug(ctypes.Structure):
    _fields_ = [("l1", ctypes.c_void_p), ("ssq", ctypes.c_void_p), ("pivot_idx", ctypes.c_void_p),
                ("sim", ctypes.c_void_p), ("eps", ctypes.c_void_p), ("keep", ctypes.c_void_p),
                ("owner", ctypes.c_void_p)]


class DartError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (what, dart_strerror(code), code))


_lib = None


def lib() -> ctypes.CDLL:
    """Load libdart.so (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("%s is missing: build it with `python -m paper_2502_11494_b200.build`; "
                               "the reduction has no fallback path" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64p, i32p = ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p
        L.dart_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(dart_desc)]
        L.dart_destroy.argtypes = [vp]
        L.dart_set_shape.argtypes = [vp, i32, i32]
        L.dart_reduce.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, i32p, i64p, vp]
        L.dart_reduce_ex.argtypes = [vp, vp, vp, i64p, i32, i32, i32, i32, vp, i32p, i64p,
                                     ctypes.POINTER(dart_opts), ctypes.POINTER(dart_debug), vp]
        L.dart_reduce_host.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, i32p, i64p]
        L.dart_status.argtypes = [vp]
        L.dart_status_detail.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
        L.dart_last_cuda_error.argtypes = [vp]
        L.dart_workspace_bytes.argtypes = [vp]
        L.dart_workspace_bytes.restype = ctypes.c_size_t
        L.dart_launch_count.argtypes = [vp]
        L.dart_launch_count.restype = ctypes.c_int64
        L.dart_profile_enable.argtypes = [vp, i32]
        L.dart_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32),
                                        ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_int)]
        L.dart_pivots_static.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32p, i32, vp]
        L.dart_gather_rows.argtypes = [vp, i32p, i32, i32, i32, i32, vp, i32, vp]
        L.dart_strerror.argtypes = [i32]
        L.dart_strerror.restype = ctypes.c_char_p
        L.dart_version.argtypes = []
        _lib = L
    return _lib


# ---- the C entry points under their own names (raw pointers as ints) ---------------------------

def dart_strerror(code: int) -> str:
    return lib().dart_strerror(code).decode()


def dart_version() -> int:
    return lib().dart_version()


def dart_create(B_max, S_max, d, P_max, Kp_max, device=0, flags=0):
    """-> (return code, context handle)."""
    h = ctypes.c_void_p()
    desc = dart_desc(B_max, S_max, d, P_max, Kp_max, device, flags)
    rc = lib().dart_create(ctypes.byref(h), ctypes.byref(desc))
    return rc, h


def dart_destroy(ctx) -> int:
    return lib().dart_destroy(ctx)


def dart_set_shape(ctx, B, S) -> int:
    return lib().dart_set_shape(ctx, B, S)


def dart_reduce(ctx, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos, stream) -> int:
    return lib().dart_reduce(ctx, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos, stream)


def dart_reduce_ex(ctx, hidden, keys, pos_in, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos,
                   opts: Optional[dart_opts], dbg: Optional[dart_debug], stream) -> int:
    return lib().dart_reduce_ex(ctx, hidden, keys, pos_in, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx,
                                out_pos, ctypes.byref(opts) if opts is not None else None,
                                ctypes.byref(dbg) if dbg is not None else None, stream)


def dart_reduce_host(ctx, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos) -> int:
    return lib().dart_reduce_host(ctx, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos)


def dart_pivots_static(keys, B, S, d, vis_offset, n_vis, n_pivot, pivot_idx, device, stream) -> int:
    """Context-free, allocation-free pivot selection (raw device pointers); see include/dart.h."""
    return lib().dart_pivots_static(keys, B, S, d, vis_offset, n_vis, n_pivot, pivot_idx, device, stream)


def dart_gather_rows(src, idx, B, S, S_out, row_bytes, out, device, stream) -> int:
    """Context-free row gather by a packed index list (raw device pointers); see include/dart.h."""
    return lib().dart_gather_rows(src, idx, B, S, S_out, row_bytes, out, device, stream)


def dart_status(ctx) -> int:
    return lib().dart_status(ctx)


def dart_status_detail(ctx):
    """-> (return code, [which wait, task index, CTA]) of the last error that dart_status reported."""
    d = (ctypes.c_int32 * 11)()
    rc = lib().dart_status_detail(ctx, d)
    return rc, list(d)


def dart_last_cuda_error(ctx) -> int:
    return lib().dart_last_cuda_error(ctx)


def dart_workspace_bytes(ctx) -> int:
    return lib().dart_workspace_bytes(ctx)


def dart_launch_count(ctx) -> int:
    return lib().dart_launch_count(ctx)


def dart_profile_enable(ctx, on: bool) -> int:
    return lib().dart_profile_enable(ctx, int(on))


def dart_profile_read(ctx):
    """-> (return code, {kernel name: (milliseconds, launches)}) accumulated since the last read."""
    cap = 16
    ms = (ctypes.c_float * cap)()
    n_l = (ctypes.c_int32 * cap)()
    names = (ctypes.c_char_p * cap)()
    n = ctypes.c_int(cap)
    rc = lib().dart_profile_read(ctx, ms, n_l, names, ctypes.byref(n))
    return rc, {names[k].decode(): (float(ms[k]), int(n_l[k])) for k in range(n.value)} if rc == 0 else {}


# ---- torch convenience wrapper --------------------------------------------------------------------

def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


class Dart:
    """A reduction context bound to one CUDA device.  ``reduce`` enqueues on torch's current stream."""

    def __init__(self, B_max, S_max, d, P_max, Kp_max, device=0, flags=0):
        rc, self._h = dart_create(B_max, S_max, d, P_max, Kp_max, device, flags)
        if rc != DART_OK:
            self._h = None
            raise DartError(rc, "dart_create")
        self.B_max, self.S_max, self.d, self.P_max, self.Kp_max, self.device = B_max, S_max, d, P_max, Kp_max, device

    def close(self):
        if getattr(self, "_h", None) is not None:
            dart_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h

    def reduce(self, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, pos_in=None, out=None, opts=None,
               debug=False, stream=None):
        """hidden/keys: [B, S, d] bf16 CUDA tensors.  Returns (out_hidden, out_idx, out_pos[, dbg dict])."""
        import torch

        B, S, d = hidden.shape
        if not (hidden.is_cuda and hidden.is_contiguous() and hidden.dtype == torch.bfloat16):
            raise ValueError("hidden must be a contiguous bf16 CUDA tensor")
        if keys is not None and not (keys.is_cuda and keys.is_contiguous() and keys.dtype == torch.bfloat16
                                     and keys.shape == hidden.shape):
            raise ValueError("keys must be a contiguous bf16 CUDA tensor shaped like hidden")
        if d != self.d:
            raise ValueError("row width %d differs from the context's %d" % (d, self.d))
        rc = dart_set_shape(self._h, B, S)
        if rc != DART_OK:
            raise DartError(rc, "dart_set_shape")
        S_out = S - n_vis + n_keep
        dev = hidden.device
        if out is None:
            if not (0 < n_keep <= n_vis <= S):
                raise DartError(DART_ERR_BAD_SHAPE, "dart_reduce")
            out = (torch.empty((B, S_out, d), dtype=torch.bfloat16, device=dev),
                   torch.empty((B, S_out), dtype=torch.int32, device=dev),
                   torch.empty((B, S_out), dtype=torch.int64, device=dev))
        oh, oi, op = out
        dbg_t, dbg_s = None, None
        if debug:
            dbg_t = {
                "l1": torch.empty((B, n_vis), dtype=torch.float32, device=dev),
                "ssq": torch.empty((B, n_vis), dtype=torch.float32, device=dev),
                "pivot_idx": torch.empty((B, n_pivot), dtype=torch.int32, device=dev),
                "sim": torch.empty((B, n_pivot, n_vis), dtype=torch.float32, device=dev),
                "eps": torch.empty((B, n_pivot), dtype=torch.float32, device=dev),
                "keep": torch.empty((B, n_vis), dtype=torch.uint8, device=dev),
                "owner": torch.empty((B, n_vis), dtype=torch.int32, device=dev),
            }
            dbg_s = dart_debug(**{k: v.data_ptr() for k, v in dbg_t.items()})
        st = stream if stream is not None else torch.cuda.current_stream(dev)
        rc = dart_reduce_ex(self._h, _ptr(hidden), _ptr(keys), _ptr(pos_in), vis_offset, n_vis, n_pivot, n_keep,
                            _ptr(oh), _ptr(oi), _ptr(op), opts, dbg_s, ctypes.c_void_p(st.cuda_stream))
        if rc != DART_OK:
            raise DartError(rc, "dart_reduce_ex")
        return (oh, oi, op, dbg_t) if debug else (oh, oi, op)

    def status(self) -> int:
        return dart_status(self._h)
