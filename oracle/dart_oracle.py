"""ctypes front end of the DART oracle (TEST INFRASTRUCTURE, not the product).

The arithmetic lives in ``dart_oracle.c`` (plain C, fp64, single-threaded), written from the
paper's definitions (Def. 1-2, Eq. 7, Eq. 9-10, the K-norm footnote of Sec. 3.3).  This module
only compiles it with gcc and marshals numpy arrays.  Nothing here imports or is imported by the
CUDA path.  bf16 tensors are passed as their uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dart_oracle.c")
_LIB = os.path.join(_HERE, "libdart_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile dart_oracle.c into libdart_oracle.so next to it (gcc, -O2, no fast-math)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math", "-ffp-contract=off",
             "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("dart_oracle_scores", "dart_oracle_pivots", "dart_oracle_similarity",
                     "dart_oracle_retention", "dart_oracle_retention_global", "dart_oracle_retention_any",
                     "dart_oracle_retention_union", "dart_oracle_similarity_any", "dart_oracle_compact",
                     "dart_oracle_gather_rows", "dart_oracle_reduce", "dart_oracle_reduce_ex", "dart_oracle_retention_union_any",
                     "dart_oracle_retention_global_any", "dart_oracle_pivots_mixed", "dart_oracle_pivots_random"):
            getattr(_lib, name).restype = ctypes.c_int
        _lib.dart_oracle_splitmix64.restype = ctypes.c_uint64
        _lib.dart_oracle_splitmix64.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
    return _lib


def _p(a, ctype):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ctype))
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _u16(a) -> np.ndarray:
    """bf16 bits as a C-contiguous uint16 array; accepts numpy uint16/int16 or a torch bf16 CPU tensor."""
    if hasattr(a, "detach"):  # torch tensor
        import torch

        t = a.detach().cpu().contiguous()
        if t.dtype == torch.bfloat16:
            t = t.view(torch.int16)
        a = t.numpy()
    a = np.ascontiguousarray(a)
    if a.dtype == np.int16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected bf16 bit patterns (uint16), got %s" % a.dtype)
    return a


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError("%s failed with oracle error %d" % (what, rc))


def scores(keys, vis_offset: int, n_vis: int):
    """keys [S, d] bf16 bits -> (l1 [n_vis], l2 [n_vis]) fp64 (K-norm footnote; Eq. 7's norms)."""
    k = _u16(keys)
    S, d = k.shape
    l1 = np.empty(n_vis, np.float64)
    l2 = np.empty(n_vis, np.float64)
    _check(_load().dart_oracle_scores(_p(k, ctypes.c_uint16), S, d, vis_offset, n_vis,
                                      _p(l1, ctypes.c_double), _p(l2, ctypes.c_double)), "scores")
    return l1, l2


def pivots(score, P: int, largest: bool = True):
    """score [n_vis] fp64 -> (pivot_idx [P] int32 in rank order, relative gap) (Def. 1)."""
    s = np.ascontiguousarray(score, np.float64)
    piv = np.empty(P, np.int32)
    gap = ctypes.c_double(0.0)
    _check(_load().dart_oracle_pivots(_p(s, ctypes.c_double), s.shape[0], P, int(bool(largest)),
                                      _p(piv, ctypes.c_int32), ctypes.byref(gap)), "pivots")
    return piv, gap.value


def similarity(keys, vis_offset: int, n_vis: int, pivot_idx, l2):
    """dup [P, n_vis] fp64, Eq. 7."""
    k = _u16(keys)
    S, d = k.shape
    piv = np.ascontiguousarray(pivot_idx, np.int32)
    n2 = np.ascontiguousarray(l2, np.float64)
    dup = np.empty((piv.shape[0], n_vis), np.float64)
    _check(_load().dart_oracle_similarity(_p(k, ctypes.c_uint16), S, d, vis_offset, n_vis,
                                          _p(piv, ctypes.c_int32), piv.shape[0],
                                          _p(n2, ctypes.c_double), _p(dup, ctypes.c_double)), "similarity")
    return dup


def retention(dup, pivot_idx, n_keep: int):
    """dup [P, n_vis] -> (keep uint8 [n_vis], owner int32 [n_vis], eps [P], gap) (Eq. 9-10)."""
    dd = np.ascontiguousarray(dup, np.float64)
    P, n_vis = dd.shape
    piv = np.ascontiguousarray(pivot_idx, np.int32)
    keep = np.empty(n_vis, np.uint8)
    owner = np.empty(n_vis, np.int32)
    eps = np.empty(P, np.float64)
    gap = ctypes.c_double(0.0)
    _check(_load().dart_oracle_retention(_p(dd, ctypes.c_double), _p(piv, ctypes.c_int32), n_vis, P, n_keep,
                                         _p(keep, ctypes.c_uint8), _p(owner, ctypes.c_int32),
                                         _p(eps, ctypes.c_double), ctypes.byref(gap)), "retention")
    return keep, owner, eps, gap.value


def similarity_any(keys, vis_offset: int, n_vis: int, pivot_idx):
    """Eq. 7 for pivots that may be text tokens (indices relative to the vision block) -> dup [P, n_vis]."""
    k = _u16(keys)
    S, d = k.shape
    piv = np.ascontiguousarray(pivot_idx, np.int32)
    dup = np.empty((len(piv), n_vis), np.float64)
    _check(_load().dart_oracle_similarity_any(_p(k, ctypes.c_uint16), S, d, vis_offset, n_vis, _p(piv, ctypes.c_int32),
                                              len(piv), _p(dup, ctypes.c_double)), "similarity_any")
    return dup


def retention_any(dup, pivot_idx, n_keep: int):
    """Quota retention where pivots outside [0, n_vis) are text tokens: (keep, owner, eps, gap)."""
    dd = np.ascontiguousarray(dup, np.float64)
    P, n_vis = dd.shape
    piv = np.ascontiguousarray(pivot_idx, np.int32)
    keep = np.empty(n_vis, np.uint8)
    owner = np.empty(n_vis, np.int32)
    eps = np.empty(P, np.float64)
    gap = ctypes.c_double(0.0)
    _check(_load().dart_oracle_retention_any(_p(dd, ctypes.c_double), _p(piv, ctypes.c_int32), n_vis, P, n_keep,
                                             _p(keep, ctypes.c_uint8), _p(owner, ctypes.c_int32),
                                             _p(eps, ctypes.c_double), ctypes.byref(gap)), "retention_any")
    return keep, owner, eps, gap.value


def splitmix64(seed: int, k: int) -> int:
    """Output number k (0-based) of a SplitMix64 generator seeded with ``seed``."""
    return int(_load().dart_oracle_splitmix64(ctypes.c_uint64(seed & (2**64 - 1)), ctypes.c_uint64(k & (2**64 - 1))))


def pivots_mixed(score_all, vis_offset: int, n_vis: int, Pv: int, Pt: int, largest: bool = True):
    """score_all [S] -> [Pv + Pt] pivots relative to the vision block: Pv vision tokens, then Pt text tokens, each by rank."""
    s = np.ascontiguousarray(score_all, np.float64)
    piv = np.empty(Pv + Pt, np.int32)
    _check(_load().dart_oracle_pivots_mixed(_p(s, ctypes.c_double), s.shape[0], vis_offset, n_vis, Pv, Pt, int(bool(largest)),
                                            _p(piv, ctypes.c_int32)), "pivots_mixed")
    return piv


def pivots_random(seed: int, b: int, n_vis: int, P: int):
    """P distinct random vision tokens of sample b: the smallest 32-bit SplitMix64 tickets, smallest first."""
    piv = np.empty(P, np.int32)
    _check(_load().dart_oracle_pivots_random(ctypes.c_uint64(seed & (2**64 - 1)), b, n_vis, P, _p(piv, ctypes.c_int32)), "pivots_random")
    return piv


def retention_union(dup, pivot_idx, n_keep: int, text_pivots: bool = False):
    """Independent pivots: (keep, owner, eps [P], gap, n_kept); a token two pivots take counts once."""
    dd = np.ascontiguousarray(dup, np.float64)
    P, n_vis = dd.shape
    piv = np.ascontiguousarray(pivot_idx, np.int32)
    keep = np.empty(n_vis, np.uint8)
    owner = np.empty(n_vis, np.int32)
    eps = np.empty(P, np.float64)
    gap = ctypes.c_double(0.0)
    cnt = ctypes.c_int32(0)
    fn = _load().dart_oracle_retention_union_any if text_pivots else _load().dart_oracle_retention_union
    _check(fn(_p(dd, ctypes.c_double), _p(piv, ctypes.c_int32), n_vis, P, n_keep,
                                               _p(keep, ctypes.c_uint8), _p(owner, ctypes.c_int32),
                                               _p(eps, ctypes.c_double), ctypes.byref(gap), ctypes.byref(cnt)), "retention_union")
    return keep, owner, eps, gap.value, cnt.value


def retention_global(dup, pivot_idx, n_keep: int, text_pivots: bool = False):
    """dup [P, n_vis] -> (keep, owner, eps [P], gap) with one threshold on max_i dup for all pivots."""
    dd = np.ascontiguousarray(dup, np.float64)
    P, n_vis = dd.shape
    piv = np.ascontiguousarray(pivot_idx, np.int32)
    keep = np.empty(n_vis, np.uint8)
    owner = np.empty(n_vis, np.int32)
    eps = np.empty(P, np.float64)
    gap = ctypes.c_double(0.0)
    fn = _load().dart_oracle_retention_global_any if text_pivots else _load().dart_oracle_retention_global
    _check(fn(_p(dd, ctypes.c_double), _p(piv, ctypes.c_int32), n_vis, P, n_keep,
                                                _p(keep, ctypes.c_uint8), _p(owner, ctypes.c_int32),
                                                _p(eps, ctypes.c_double), ctypes.byref(gap)), "retention_global")
    return keep, owner, eps, gap.value


def gather_rows(src, idx):
    """src [B, S, w] 16-bit words (bf16 bits), idx [B, S_out] int32 -> out [B, S_out, w] (bit copies)."""
    a = _u16(src)
    B, S, w = a.shape
    ii = np.ascontiguousarray(idx, np.int32)
    S_out = ii.shape[1]
    out = np.empty((B, S_out, w), np.uint16)
    _check(_load().dart_oracle_gather_rows(_p(a, ctypes.c_uint16), _p(ii, ctypes.c_int32), B, S, S_out, w,
                                           _p(out, ctypes.c_uint16)), "gather_rows")
    return out


def compact(keep, hidden, vis_offset: int, n_vis: int, pos_in=None):
    """keep [n_vis], hidden [S, d] bf16 bits -> (out_hidden [S_out, d] uint16, out_idx int32, out_pos int64)."""
    h = _u16(hidden)
    S, d = h.shape
    kp = np.ascontiguousarray(keep, np.uint8)
    S_out = S - n_vis + int(kp.astype(np.int64).sum())
    pos = None if pos_in is None else np.ascontiguousarray(pos_in, np.int64)
    oh = np.empty((S_out, d), np.uint16)
    oi = np.empty(S_out, np.int32)
    op = np.empty(S_out, np.int64)
    so = ctypes.c_int(0)
    _check(_load().dart_oracle_compact(_p(kp, ctypes.c_uint8), _p(h, ctypes.c_uint16), _p(pos, ctypes.c_int64),
                                       S, d, vis_offset, n_vis, _p(oh, ctypes.c_uint16), _p(oi, ctypes.c_int32),
                                       _p(op, ctypes.c_int64), ctypes.byref(so)), "compact")
    assert so.value == S_out
    return oh, oi, op


@dataclass
class OracleResult:
    out_hidden: np.ndarray  # [B, S_out, d] uint16 (bf16 bits)
    out_idx: np.ndarray     # [B, S_out] int32
    out_pos: np.ndarray     # [B, S_out] int64
    l1: np.ndarray          # [B, n_vis] fp64
    l2: np.ndarray          # [B, n_vis] fp64
    pivot_idx: np.ndarray   # [B, P] int32, rank order
    dup: np.ndarray | None  # [B, P, n_vis] fp64
    keep: np.ndarray        # [B, n_vis] uint8
    owner: np.ndarray       # [B, n_vis] int32
    eps: np.ndarray         # [B, P] fp64
    pivot_gap: np.ndarray   # [B] relative score gap along the pivot ranking
    retain_gap: np.ndarray  # [B] absolute dup gap at the retention boundaries
    cu_seqlens: np.ndarray | None = None  # [B + 1] int32, rule 2 only: sample b's rows are cu[b] .. cu[b + 1] of the flat outputs

    @property
    def margin(self) -> np.ndarray:
        """Per-sample selection margin: the smaller of the two gaps."""
        return np.minimum(self.pivot_gap, self.retain_gap)


def reduce(hidden, keys, vis_offset: int, n_vis: int, n_pivot: int, n_keep: int,
           pos_in=None, norm_kind: int = 1, largest: bool = True, want_dup: bool = True,
           want_hidden: bool = True, pivots_in=None, rule: int = 0, cosine_on_hidden: bool = False,
           text_pivots: bool = False, pivot_source: int = 0, n_text_pivots: int = 0, seed: int = 0) -> OracleResult:
    """The whole step over a batch.  hidden/keys: [B, S, d] bf16 bits (keys None -> hidden is scored).
    pivots_in: None, or [B, n_pivot] distinct vision-relative indices that replace the pivot step.
    rule: 0 quotas with masking, 1 one threshold for all pivots, 2 independent pivots (flat outputs + .cu_seqlens).
    rule: 0 = per-pivot thresholds from equal quotas, 1 = one threshold for all pivots.
    cosine_on_hidden: pivots by the key rows' scores, Eq. 7 on the hidden rows (then .l2 holds the hidden rows' norms).
    text_pivots: entries of pivots_in outside [0, n_vis) name text tokens (indices relative to the vision block).
    pivot_source (without pivots_in): 0 = vision tokens by score, 1 = n_pivot - n_text_pivots vision and n_text_pivots text
    tokens by score, 2 = random vision tokens from ``seed``."""
    h = _u16(hidden)
    B, S, d = h.shape
    k = None if keys is None else _u16(keys)
    if k is not None and k.shape != h.shape:
        raise ValueError("keys and hidden must have the same shape")
    pos = None if pos_in is None else np.ascontiguousarray(pos_in, np.int64)
    S_out = S - n_vis + n_keep
    oh = np.empty((B, S_out, d), np.uint16) if want_hidden else None
    oi = np.empty((B, S_out), np.int32)
    op = np.empty((B, S_out), np.int64)
    l1 = np.empty((B, n_vis), np.float64)
    l2 = np.empty((B, n_vis), np.float64)
    piv = np.empty((B, n_pivot), np.int32)
    dup = np.empty((B, n_pivot, n_vis), np.float64) if want_dup else None
    keep = np.empty((B, n_vis), np.uint8)
    owner = np.empty((B, n_vis), np.int32)
    eps = np.empty((B, n_pivot), np.float64)
    pg = np.empty(B, np.float64)
    rg = np.empty(B, np.float64)
    cu = None
    if rule == 2:  # the packed length depends on the data: what is not written stays -1 / 0
        cu = np.zeros(B + 1, np.int32)
        oi.fill(-1)
        op.fill(-1)
        if oh is not None:
            oh.fill(0)
    piv_in = None if pivots_in is None else np.ascontiguousarray(pivots_in, np.int32)
    if piv_in is not None and piv_in.shape != (B, n_pivot):
        raise ValueError("pivots_in must be [B, n_pivot]")
    _check(_load().dart_oracle_reduce_ex(
        _p(h, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(pos, ctypes.c_int64), _p(piv_in, ctypes.c_int32),
        B, S, d, vis_offset, n_vis, n_pivot, n_keep, norm_kind, int(bool(largest)), int(rule), int(bool(cosine_on_hidden)), int(bool(text_pivots)),
        int(pivot_source), int(n_text_pivots), ctypes.c_uint64(seed & (2**64 - 1)),
        _p(oh, ctypes.c_uint16), _p(oi, ctypes.c_int32), _p(op, ctypes.c_int64),
        _p(l1, ctypes.c_double), _p(l2, ctypes.c_double), _p(piv, ctypes.c_int32), _p(dup, ctypes.c_double),
        _p(keep, ctypes.c_uint8), _p(owner, ctypes.c_int32), _p(eps, ctypes.c_double),
        _p(pg, ctypes.c_double), _p(rg, ctypes.c_double), _p(cu, ctypes.c_int32)), "reduce")
    if rule == 2:  # flat outputs [B * S_out(, d)], rows beyond cu[B] are -1 / 0
        oh = None if oh is None else oh.reshape(B * S_out, d)
        oi, op = oi.reshape(-1), op.reshape(-1)
    return OracleResult(oh, oi, op, l1, l2, piv, dup, keep, owner, eps, pg, rg, cu)
