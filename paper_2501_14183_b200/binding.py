"""ctypes binding of libvardrop.so: argument marshalling only.

Every function has the name and the argument order of its C entry point in ``include/vardrop.h``; tensors are
``torch.Tensor`` objects on the CUDA device (PyTorch is used for device memory and streams only), the stream is
PyTorch's current stream.  There is no CPU path: if the CUDA library cannot be loaded the import of a symbol fails
with the loader's error.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libvardrop.so"
_lib = None

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE = range(7)
SCOPE_BATCH_MEAN, SCOPE_PER_INSTANCE = 0, 1


class HashCfg(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("L", C.c_int32), ("k", C.c_int32), ("f_lo", C.c_int32),
                ("f_hi", C.c_int32), ("scope", C.c_int32)]


class SelectCfg(C.Structure):
    _fields_ = [("S", C.c_int32), ("N", C.c_int32), ("gs", C.c_int32), ("rate", C.c_double), ("seed", C.c_uint64),
                ("step", C.c_uint32)]


class AttnCfg(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("H", C.c_int32), ("D", C.c_int32), ("sm_scale", C.c_float), ("S", C.c_int32),
                ("sB", C.c_int64), ("sN", C.c_int64), ("sH", C.c_int64)]          # element strides of q, k, v; all 0 = contiguous


class GatherCfg(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("L", C.c_int32), ("S", C.c_int32)]


class PearsonCfg(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("L", C.c_int32), ("threshold", C.c_float)]


class VardropError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = load()
        super().__init__(f"{where}: {lib.vardrop_status_string(status).decode()} ({status}): {lib.vardrop_last_error().decode()}")


EXPORTS = ("vardrop_status_string", "vardrop_last_error", "vardrop_version", "vardrop_ws_status", "vardrop_probe_bounded_wait", "vardrop_hash_workspace_bytes", "vardrop_hash",
           "vardrop_select_workspace_bytes", "vardrop_select", "vardrop_select_static", "vardrop_gather_rows", "vardrop_attn_workspace_bytes", "vardrop_attn_fwd",
           "vardrop_attn_bwd", "vardrop_pearson_workspace_bytes", "vardrop_pearson_max", "vardrop_launch_count", "vardrop_profile_enable", "vardrop_profile_kernels",
           "vardrop_profile_kernel_name", "vardrop_profile_read")


def load() -> C.CDLL:
    """Loads the in-tree shared library (no fallback: a missing library is an error)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2501_14183_b200.build`")
        lib = C.CDLL(str(_LIB_PATH))
        for name in ("vardrop_status_string", "vardrop_last_error", "vardrop_version"):
            getattr(lib, name).restype = C.c_char_p
        lib.vardrop_status_string.argtypes = [C.c_int]
        for name in ("vardrop_hash_workspace_bytes", "vardrop_select_workspace_bytes", "vardrop_attn_workspace_bytes",
                     "vardrop_pearson_workspace_bytes"):
            getattr(lib, name).restype = C.c_size_t
            getattr(lib, name).argtypes = [C.c_void_p]
        lib.vardrop_ws_status.restype = C.c_int
        lib.vardrop_ws_status.argtypes = [C.c_void_p, C.c_void_p]
        lib.vardrop_probe_bounded_wait.restype = C.c_int
        lib.vardrop_probe_bounded_wait.argtypes = [C.c_void_p, C.c_size_t, C.c_uint, C.c_void_p]
        lib.vardrop_hash.restype = C.c_int
        lib.vardrop_hash.argtypes = [C.c_void_p] * 6 + [C.c_size_t, C.c_void_p]
        lib.vardrop_select.restype = C.c_int
        lib.vardrop_select.argtypes = [C.c_void_p] * 10 + [C.c_size_t, C.c_void_p]
        lib.vardrop_select_static.restype = C.c_int
        lib.vardrop_select_static.argtypes = [C.c_void_p] * 10
        lib.vardrop_gather_rows.restype = C.c_int
        lib.vardrop_gather_rows.argtypes = [C.c_void_p] * 6
        lib.vardrop_attn_fwd.restype = C.c_int
        lib.vardrop_attn_fwd.argtypes = [C.c_void_p] * 9 + [C.c_size_t, C.c_void_p]
        lib.vardrop_attn_bwd.restype = C.c_int
        lib.vardrop_attn_bwd.argtypes = [C.c_void_p] * 14 + [C.c_size_t, C.c_void_p]
        lib.vardrop_pearson_max.restype = C.c_int
        lib.vardrop_pearson_max.argtypes = [C.c_void_p] * 5 + [C.c_size_t, C.c_void_p]
        lib.vardrop_launch_count.restype = C.c_longlong
        lib.vardrop_profile_kernel_name.restype = C.c_char_p
        lib.vardrop_profile_kernel_name.argtypes = [C.c_int]
        lib.vardrop_profile_enable.argtypes = [C.c_int]
        lib.vardrop_profile_read.argtypes = [C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
        _lib = lib
    return _lib


def _ptr(t):
    return None if t is None else t.data_ptr()        # a plain int converts to void* without a ctypes object per argument


try:
    _raw_stream = torch._C._cuda_getCurrentRawStream    # the stream handle without building a Stream object
except AttributeError:                                   # pragma: no cover
    _raw_stream = None


def _stream():
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != OK:
        raise VardropError(status, where)


def vardrop_hash_workspace_bytes(cfg: HashCfg) -> int:
    return int(load().vardrop_hash_workspace_bytes(C.byref(cfg)))


def vardrop_select_workspace_bytes(cfg: SelectCfg) -> int:
    return int(load().vardrop_select_workspace_bytes(C.byref(cfg)))


def vardrop_attn_workspace_bytes(cfg: AttnCfg) -> int:
    return int(load().vardrop_attn_workspace_bytes(C.byref(cfg)))


def vardrop_hash(x, cfg: HashCfg, keys, freqs, amp_dbg, ws) -> None:
    _check(load().vardrop_hash(_ptr(x), C.byref(cfg), _ptr(keys), _ptr(freqs), _ptr(amp_dbg), _ptr(ws),
                               ws.numel() * ws.element_size(), _stream()), "vardrop_hash")


def vardrop_select(keys, cfg: SelectCfg, group_id, group_offsets, members, n_groups, sel_idx, n_sel, inv_idx, ws) -> None:
    _check(load().vardrop_select(_ptr(keys), C.byref(cfg), _ptr(group_id), _ptr(group_offsets), _ptr(members), _ptr(n_groups),
                                 _ptr(sel_idx), _ptr(n_sel), _ptr(inv_idx), _ptr(ws), ws.numel() * ws.element_size(),
                                 _stream()), "vardrop_select")


def vardrop_select_static(keys, cfg: SelectCfg, group_id, group_offsets, members, n_groups, sel_idx, n_sel, inv_idx) -> None:
    """vardrop_select for callers that cannot allocate: no workspace argument, the scratch is a fixed array inside the
    library (S * N <= 16384).  Calls whose GPU work overlaps share that array and race."""
    _check(load().vardrop_select_static(_ptr(keys), C.byref(cfg), _ptr(group_id), _ptr(group_offsets), _ptr(members),
                                        _ptr(n_groups), _ptr(sel_idx), _ptr(n_sel), _ptr(inv_idx), _stream()),
           "vardrop_select_static")


def vardrop_gather_rows(x, sel_idx, n_sel, cfg: GatherCfg, x_sel) -> None:
    _check(load().vardrop_gather_rows(_ptr(x), _ptr(sel_idx), _ptr(n_sel), C.byref(cfg), _ptr(x_sel), _stream()), "vardrop_gather_rows")


def vardrop_attn_fwd(q, k, v, sel_idx, n_sel, cfg: AttnCfg, o, lse, ws) -> None:
    _check(load().vardrop_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(sel_idx), _ptr(n_sel), C.byref(cfg), _ptr(o), _ptr(lse),
                                   _ptr(ws), ws.numel() * ws.element_size(), _stream()), "vardrop_attn_fwd")


def vardrop_attn_bwd(q, k, v, o, lse, d_o, sel_idx, n_sel, inv_idx, cfg: AttnCfg, dq, dk, dv, ws) -> None:
    _check(load().vardrop_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o), _ptr(sel_idx), _ptr(n_sel),
                                   _ptr(inv_idx), C.byref(cfg), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws),
                                   ws.numel() * ws.element_size(), _stream()), "vardrop_attn_bwd")


def vardrop_pearson_workspace_bytes(cfg: PearsonCfg) -> int:
    return int(load().vardrop_pearson_workspace_bytes(C.byref(cfg)))


def vardrop_pearson_max(x, cfg: PearsonCfg, max_rho, n_above, ws) -> None:
    _check(load().vardrop_pearson_max(_ptr(x), C.byref(cfg), _ptr(max_rho), _ptr(n_above), _ptr(ws), ws.numel() * ws.element_size(),
                                      _stream()), "vardrop_pearson_max")


def vardrop_launch_count() -> int:
    return int(load().vardrop_launch_count())


def vardrop_profile_enable(on: bool) -> None:
    _check(load().vardrop_profile_enable(1 if on else 0), "vardrop_profile_enable")


def vardrop_profile_read() -> dict:
    """{kernel name: (total milliseconds, launches)} for everything recorded since the timer was armed."""
    lib = load()
    out = {}
    for kid in range(lib.vardrop_profile_kernels()):
        ms, n = C.c_double(0.0), C.c_longlong(0)
        _check(lib.vardrop_profile_read(kid, C.byref(ms), C.byref(n)), "vardrop_profile_read")
        out[lib.vardrop_profile_kernel_name(kid).decode()] = (ms.value, int(n.value))
    return out


def vardrop_ws_status(ws) -> int:
    """Device-side status word of a workspace (synchronises the current stream)."""
    return int(load().vardrop_ws_status(_ptr(ws), _stream()))


ws_status = vardrop_ws_status


def vardrop_probe_bounded_wait(ws, limit_us: int) -> None:
    _check(load().vardrop_probe_bounded_wait(_ptr(ws), ws.numel() * ws.element_size(), int(limit_us), _stream()), "vardrop_probe_bounded_wait")


# ---- buffer helpers (allocation only) -----------------------------------------------------------------------
def alloc_ws(nbytes: int, device="cuda"):
    """A zero-filled workspace: its status word is only ever set by the library, never cleared."""
    return torch.zeros(max(256, (nbytes + 255) // 256 * 256), dtype=torch.uint8, device=device)


def alloc_hash_outputs(cfg: HashCfg, device="cuda", want_freqs=True, want_amp=False):
    S = 1 if cfg.scope == 0 else cfg.B
    f_lo, f_hi = (cfg.f_lo, cfg.f_hi) if (cfg.f_lo or cfg.f_hi) else (1, (cfg.L // 2 + 1 + 1) // 2)
    keys = torch.empty((S, cfg.N), dtype=torch.int64, device=device)     # uint64 payload
    freqs = torch.empty((S, cfg.N, cfg.k), dtype=torch.int32, device=device) if want_freqs else None
    amp = torch.empty((S, cfg.N, f_hi - f_lo), dtype=torch.float32, device=device) if want_amp else None
    return keys, freqs, amp


def alloc_select_outputs(cfg: SelectCfg, device="cuda"):
    i32 = dict(dtype=torch.int32, device=device)
    return dict(group_id=torch.empty((cfg.S, cfg.N), **i32), group_offsets=torch.empty((cfg.S, cfg.N + 1), **i32),
                members=torch.empty((cfg.S, cfg.N), **i32), n_groups=torch.empty((cfg.S,), **i32),
                sel_idx=torch.empty((cfg.S, cfg.N), **i32), n_sel=torch.empty((cfg.S,), **i32),
                inv_idx=torch.empty((cfg.S, cfg.N), **i32))
