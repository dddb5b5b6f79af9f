"""B200 (sm_100a) implementation of VarDrop's per-batch training path behind a C ABI (see include/vardrop.h).

``binding`` holds the ctypes front end (same names as the C entry points), ``inputs`` the seeded synthetic
workloads, ``build`` the nvcc build step.
"""
from . import binding, inputs  # noqa: F401
from .binding import (AttnCfg, HashCfg, SelectCfg, VardropError, vardrop_attn_bwd, vardrop_attn_fwd,  # noqa: F401
                      vardrop_attn_workspace_bytes, vardrop_hash, vardrop_hash_workspace_bytes, vardrop_select,
                      vardrop_select_workspace_bytes)
