"""CPU oracle for the VarDrop hot path.  TEST INFRASTRUCTURE ONLY.

ctypes front end of ``vardrop_oracle.c`` (plain C, fp64, written from the paper).  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA library and its
Python binding never do, and share no code with it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "vardrop_oracle.c"
_LIB = _HERE / "libvardrop_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP).  Rebuilds when the source is newer than the library."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(str(_LIB))
        _lib.vdo_num_threads.restype = C.c_int
        _lib.vdo_quota.restype = C.c_int64
        _lib.vdo_quota.argtypes = [C.c_int64, C.c_int32, C.c_double]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(_load().vdo_num_threads())


def default_band(L: int) -> tuple[int, int]:
    """Default candidate band: DC excluded, cut-off = half of the non-negative-frequency bins (25 at L = 96,
    Appendix E)."""
    nb = L // 2 + 1
    return 1, (nb + 1) // 2


def dft_amplitudes(x: np.ndarray, f_lo: int, f_hi: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    B, N, L = x.shape
    amp = np.empty((B, N, f_hi - f_lo), dtype=np.float64)
    _load().vdo_dft_amplitudes(_p(x), C.c_int(B), C.c_int(N), C.c_int(L), C.c_int(f_lo), C.c_int(f_hi), _p(amp))
    return amp


def hash(x: np.ndarray, k: int, f_lo: int = 0, f_hi: int = 0, scope: int = 0):
    """Algorithm 1.  Returns (keys[S,N] uint64, freqs[S,N,k] int32, abar[S,N,nf] float64)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    B, N, L = x.shape
    if f_lo == 0 and f_hi == 0:
        f_lo, f_hi = default_band(L)
    S = 1 if scope == 0 else B
    keys = np.empty((S, N), dtype=np.uint64)
    freqs = np.empty((S, N, k), dtype=np.int32)
    abar = np.empty((S, N, f_hi - f_lo), dtype=np.float64)
    _load().vdo_hash(_p(x), C.c_int(B), C.c_int(N), C.c_int(L), C.c_int(k), C.c_int(f_lo), C.c_int(f_hi),
                     C.c_int(scope), _p(keys), _p(freqs), _p(abar))
    return keys, freqs, abar


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.empty(4, dtype=np.uint32)
    _load().vdo_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def quota(size: int, gs: int, rate: float) -> int:
    return int(_load().vdo_quota(C.c_int64(size), C.c_int32(gs), C.c_double(rate)))


def select(keys: np.ndarray, gs: int, rate: float, seed: int, step: int) -> dict:
    """Grouping + Eq. 1 / Eq. 2.  ``keys`` is [S, N] (or [N]) uint64."""
    keys = np.ascontiguousarray(np.atleast_2d(keys), dtype=np.uint64)
    S, N = keys.shape
    out = dict(
        group_id=np.empty((S, N), np.int32), group_offsets=np.empty((S, N + 1), np.int32),
        members=np.empty((S, N), np.int32), n_groups=np.empty(S, np.int32),
        sel_idx=np.empty((S, N), np.int32), n_sel=np.empty(S, np.int32), inv_idx=np.empty((S, N), np.int32))
    _load().vdo_select(_p(keys), C.c_int(S), C.c_int(N), C.c_int32(gs), C.c_double(rate), C.c_uint64(seed),
                       C.c_uint32(step), _p(out["group_id"]), _p(out["group_offsets"]), _p(out["members"]),
                       _p(out["n_groups"]), _p(out["sel_idx"]), _p(out["n_sel"]), _p(out["inv_idx"]))
    return out


def attn_fwd(q, k, v, sel=None, scale: float | None = None):
    """Eq. 3 over the kept tokens.  q, k, v: [B,N,H,D] (any float dtype, used as fp64).  Returns (o[B,Ns,H,D], lse[B,H,Ns])."""
    q, k, v = (np.ascontiguousarray(a, dtype=np.float64) for a in (q, k, v))
    B, N, H, D = q.shape
    scale = D ** -0.5 if scale is None else scale
    if sel is None:
        Ns, sp = N, None
    else:
        sel = np.ascontiguousarray(sel, dtype=np.int32)
        Ns, sp = int(sel.shape[0]), _p(sel)
    o = np.empty((B, Ns, H, D), np.float64)
    lse = np.empty((B, H, Ns), np.float64)
    _load().vdo_attn_fwd(_p(q), _p(k), _p(v), C.c_int(B), C.c_int(N), C.c_int(H), C.c_int(D), sp, C.c_int(Ns),
                         C.c_double(scale), _p(o), _p(lse))
    return o, lse


def attn_bwd(q, k, v, d_o, sel=None, scale: float | None = None):
    """Derivative of Eq. 3, scattered to the full layout.  Returns (dq, dk, dv), each [B,N,H,D] float64."""
    q, k, v, d_o = (np.ascontiguousarray(a, dtype=np.float64) for a in (q, k, v, d_o))
    B, N, H, D = q.shape
    scale = D ** -0.5 if scale is None else scale
    if sel is None:
        Ns, sp = N, None
    else:
        sel = np.ascontiguousarray(sel, dtype=np.int32)
        Ns, sp = int(sel.shape[0]), _p(sel)
    assert d_o.shape == (B, Ns, H, D)
    dq, dk, dv = (np.empty((B, N, H, D), np.float64) for _ in range(3))
    _load().vdo_attn_bwd(_p(q), _p(k), _p(v), _p(d_o), C.c_int(B), C.c_int(N), C.c_int(H), C.c_int(D), sp,
                         C.c_int(Ns), C.c_double(scale), _p(dq), _p(dk), _p(dv))
    return dq, dk, dv


def rank_gaps(abar: np.ndarray, k: int) -> np.ndarray:
    """Smallest relative gap (A_(i) - A_(i+1)) / A_(i), i = 1..k, between neighbours of the sorted top (k+1) mean
    amplitudes of every variate: the margin by which a variate's hash is decided."""
    top = -np.sort(-abar, axis=-1)[..., : k + 1]
    return ((top[..., :-1] - top[..., 1:]) / np.maximum(top[..., :-1], 1e-300)).min(axis=-1)


def pearson_max(x: np.ndarray) -> np.ndarray:
    """Appendix A, Eq. 4: for every instance and variate, the largest Pearson correlation coefficient with any other
    variate of the same window (a constant variate correlates 0 with everything).  x [B, N, L] -> [B, N] float64."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    B, N, L = x.shape
    out = np.empty((B, N), dtype=np.float64)
    _load().vdo_pearson_max(_p(x), B, N, L, _p(out))
    return out



def gather_rows(x: np.ndarray, sel: np.ndarray, n_sel: np.ndarray, fill: float = 0.0) -> np.ndarray:
    """Sec. 3.3 on the raw window: rows 0..n_sel-1 of instance b are x[b, sel[s(b), j], :]; the other rows keep ``fill``.
    sel is [S, N] (S = 1 or B), n_sel [S]."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    sel = np.ascontiguousarray(np.atleast_2d(sel), dtype=np.int32)
    n_sel = np.ascontiguousarray(np.atleast_1d(n_sel), dtype=np.int32)
    B, N, L = x.shape
    out = np.full((B, N, L), fill, dtype=np.float32)
    _load().vdo_gather_rows(_p(x), C.c_int(B), C.c_int(N), C.c_int(L), _p(sel), _p(n_sel), C.c_int(sel.shape[0]), _p(out))
    return out
