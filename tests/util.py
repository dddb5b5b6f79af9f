"""Helpers shared by the GPU parity tests: filtered inputs, dtype conversions, tolerances."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2501_14183_b200 import inputs

# Tolerances for bf16 attention against the fp64 oracle (bf16 inputs, fp32 accumulation, P and dS rounded to bf16).
ATTN_MAX_ABS = 2e-2
ATTN_MEAN_ABS = 2e-3
RANK_GAP = 1e-3


def gap_filtered_windows(x: np.ndarray, k: int, f_lo: int = 0, f_hi: int = 0, scope: int = 0):
    """Returns (x', keys, freqs, abar, n_replaced): variates whose hash is decided by a relative amplitude gap below
    RANK_GAP (in any hash row) are overwritten with a copy of a clearly decided variate, so that every hash of x' is
    decided by a margin no fp32 transform can flip."""
    x = x.copy()
    keys, freqs, abar = oracle.hash(x, k, f_lo, f_hi, scope)
    gaps = oracle.rank_gaps(abar, k).min(axis=0)          # per variate, worst over hash rows
    bad = np.nonzero(gaps <= RANK_GAP)[0]
    good = np.nonzero(gaps > 10 * RANK_GAP)[0]
    assert len(good) > 0
    for i, n in enumerate(bad):
        x[:, n] = x[:, good[i % len(good)]]
    if len(bad):
        keys, freqs, abar = oracle.hash(x, k, f_lo, f_hi, scope)
        assert oracle.rank_gaps(abar, k).min() > RANK_GAP
    return x, keys, freqs, abar, len(bad)


def bf16_tokens(B, N, H, D, std, seed, count=4, device="cuda"):
    """bf16 device tensors and their exact float64 images."""
    arrs = inputs.make_tokens(B, N, H, D, std, seed, count)
    dev = [torch.from_numpy(a).to(device=device, dtype=torch.bfloat16).contiguous() for a in arrs]
    ref = [t.double().cpu().numpy() for t in dev]
    return dev, ref


def assert_attn_close(got: np.ndarray, want: np.ndarray, what: str):
    err = np.abs(got.astype(np.float64) - want)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    assert err.max() <= ATTN_MAX_ABS, f"{what}: max abs error {err.max():.3e} > {ATTN_MAX_ABS}"
    assert err.mean() <= ATTN_MEAN_ABS, f"{what}: mean abs error {err.mean():.3e} > {ATTN_MEAN_ABS}"
