"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *draws data*: periodic multivariate windows x[B, N, L] whose
variates share a limited number of periodic templates (so that many variates
are redundant, as Sec. 1 / Appendix B of the paper report for Electricity and
Traffic), and i.i.d. normal Q/K/V/dO variate tokens.  It holds none of the
method's arithmetic (no DFT, ranking, hashing, grouping, sampling, attention)
and is the only module shared by the CPU oracle's tests and the CUDA path's
tests and benchmark.

Workload recipe (all draws from numpy's PCG64 seeded with ``seed``):

* a *template* is an ordered tuple of ``m`` distinct periods from the
  workload's period pool, an amplitude ladder a_1 = 1, a_{i+1} = a_i / U(1.5, 3)
  and one phase per component, U(0, 2 pi);
* a share ``shared`` of the variates draw their template from the workload's
  ``n_templates`` shared templates, the rest get a private random template;
* variate n, instance b:
  x[b, n, t] = sum_i a_i (1 + U(-jitter, jitter)) sin(2 pi (t + tau_b) / p_i + phi_i + N(0, 0.1))
               + N(0, sigma^2),
  tau_b an integer time shift shared by all variates of instance b (sliding
  windows), then z-normalised per window.
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    N: int
    L: int
    k: int
    rate: float
    H: int
    D: int
    n_templates: int
    m: int                      # sinusoids per template
    sigma: float                # additive noise std
    shared: float               # share of variates on a shared template
    periods: tuple = ()
    fixed_templates: tuple = () # explicit period tuples (Tiny)
    qkv_std: float = 1.0
    jitter: float = 0.2
    seed: int = 20250114

    @property
    def tokens(self) -> int:
        return self.B * self.N


_P96 = (24, 12, 8, 72, 6)                    # 168 mod 96 = 72
_P720 = (24, 12, 168, 48, 8, 6, 336)
_P336 = (336, 168, 112, 84, 56, 48, 42, 28, 24, 16, 14, 12, 8, 7, 6)

WORKLOADS = {
    "tiny": Workload("tiny", B=4, N=21, L=96, k=2, rate=0.5, H=4, D=32, n_templates=4, m=2,
                     sigma=0.1, shared=1.0, jitter=0.0,
                     fixed_templates=((24, 12), (24, 72), (48, 8), (32, 16)),
                     qkv_std=1.0, seed=20250114),
    "elec": Workload("elec", B=32, N=321, L=96, k=3, rate=0.3, H=8, D=64, n_templates=40, m=3,
                     sigma=0.1, shared=0.8, periods=_P96, qkv_std=math.sqrt(1.0 / 8.0), seed=20250115),
    "traffic": Workload("traffic", B=32, N=862, L=96, k=3, rate=0.2, H=8, D=64, n_templates=60, m=3,
                        sigma=0.05, shared=0.95, periods=_P96, qkv_std=math.sqrt(1.0 / 8.0), seed=20250116),
    "long": Workload("long", B=16, N=862, L=720, k=5, rate=0.2, H=8, D=64, n_templates=80, m=5,
                     sigma=0.1, shared=1.0, periods=_P720, qkv_std=math.sqrt(1.0 / 8.0), seed=20250117),
    "scale": Workload("scale", B=8, N=8192, L=336, k=4, rate=0.1, H=8, D=64, n_templates=512, m=4,
                      sigma=0.1, shared=0.95, periods=_P336, qkv_std=math.sqrt(1.0 / 8.0), seed=20250118),
}


def _draw_template_periods(rng: np.random.Generator, w: Workload, count: int) -> list[tuple]:
    """``count`` ordered m-tuples of distinct periods, distinct from each other while the pool allows."""
    if w.fixed_templates:
        return [tuple(w.fixed_templates[i % len(w.fixed_templates)]) for i in range(count)]
    n_ordered = math.perm(len(w.periods), w.m)
    if n_ordered <= 4096:
        every = list(itertools.permutations(w.periods, w.m))
        order = rng.permutation(len(every))
        return [every[order[i % len(every)]] for i in range(count)]
    seen, out = set(), []
    while len(out) < count:
        t = tuple(int(p) for p in rng.choice(w.periods, size=w.m, replace=False))
        if t not in seen:
            seen.add(t)
            out.append(t)
    return out


def make_windows(w: Workload, seed: int | None = None, B: int | None = None, N: int | None = None) -> np.ndarray:
    """x[B, N, L] float32, C-contiguous, per the module's recipe."""
    B = w.B if B is None else B
    N = w.N if N is None else N
    rng = np.random.default_rng(w.seed if seed is None else seed)
    n_t = max(1, min(w.n_templates, N))
    periods = _draw_template_periods(rng, w, n_t)
    ratios = rng.uniform(1.5, 3.0, size=(n_t, w.m))
    amps = np.ones((n_t, w.m))
    for i in range(1, w.m):
        amps[:, i] = amps[:, i - 1] / ratios[:, i]
    phases = rng.uniform(0.0, 2.0 * np.pi, size=(n_t, w.m))

    is_shared = rng.uniform(size=N) < w.shared
    tmpl = rng.integers(0, n_t, size=N)
    # private templates for the non-shared variates
    P = np.empty((N, w.m)); A = np.empty((N, w.m)); PH = np.empty((N, w.m))
    for n in range(N):
        if is_shared[n]:
            P[n] = periods[tmpl[n]]; A[n] = amps[tmpl[n]]; PH[n] = phases[tmpl[n]]
        else:
            P[n] = _draw_template_periods(rng, w, 1)[0]
            a = np.ones(w.m)
            r = rng.uniform(1.5, 3.0, size=w.m)
            for i in range(1, w.m):
                a[i] = a[i - 1] / r[i]
            A[n] = a
            PH[n] = rng.uniform(0.0, 2.0 * np.pi, size=w.m)
    A = A * (1.0 + rng.uniform(-w.jitter, w.jitter, size=A.shape))
    PH = PH + rng.normal(0.0, 0.1, size=PH.shape)
    tau = rng.integers(0, 4 * w.L, size=B).astype(np.float64)

    t = np.arange(w.L, dtype=np.float64)
    x = np.zeros((B, N, w.L), dtype=np.float64)
    for i in range(w.m):
        arg = 2.0 * np.pi * (t[None, None, :] + tau[:, None, None]) / P[None, :, i, None] + PH[None, :, i, None]
        x += A[None, :, i, None] * np.sin(arg)
    x += rng.normal(0.0, w.sigma, size=x.shape)
    x -= x.mean(axis=-1, keepdims=True)
    x /= x.std(axis=-1, keepdims=True) + 1e-12
    return np.ascontiguousarray(x.astype(np.float32))


def make_sinusoid_windows(B: int, N: int, L: int, bins, amps, seed: int, noise: float = 0.0) -> np.ndarray:
    """Windows that are sums of integer-bin sinusoids: x[b,n,t] = sum_i amps[n][i] sin(2 pi bins[n][i] t / L + phase).

    ``bins`` and ``amps`` are [N, m]; phases are uniform random per (b, n, i).  Not z-normalised, so the
    amplitudes the caller asked for are the amplitudes of the signal.
    """
    rng = np.random.default_rng(seed)
    bins = np.asarray(bins, dtype=np.float64).reshape(N, -1)
    amps = np.asarray(amps, dtype=np.float64).reshape(N, -1)
    ph = rng.uniform(0.0, 2.0 * np.pi, size=(B, N, bins.shape[1]))
    t = np.arange(L, dtype=np.float64)
    x = np.zeros((B, N, L))
    for i in range(bins.shape[1]):
        x += amps[None, :, i, None] * np.sin(2.0 * np.pi * bins[None, :, i, None] * t[None, None, :] / L + ph[:, :, i, None])
    if noise > 0.0:
        x += rng.normal(0.0, noise, size=x.shape)
    return np.ascontiguousarray(x.astype(np.float32))


def make_tokens(B: int, N: int, H: int, D: int, std: float, seed: int, count: int = 4):
    """``count`` float32 arrays [B, N, H, D] of N(0, std^2) draws (callers round them to bf16)."""
    rng = np.random.default_rng(seed)
    return [np.ascontiguousarray(rng.normal(0.0, std, size=(B, N, H, D)).astype(np.float32)) for _ in range(count)]


def make_keys(N: int, n_groups: int, k: int, f_hi: int, seed: int, skew: float = 1.0) -> np.ndarray:
    """Random packed hash keys [N] uint64 with about ``n_groups`` distinct values (12 bits per ranked bin, rank-1 bin most
    significant) and a Zipf-like group-size distribution; used to drive grouping and sampling directly."""
    rng = np.random.default_rng(seed)
    distinct = set()
    while len(distinct) < n_groups:
        f = rng.choice(np.arange(1, f_hi), size=k, replace=False)
        key = 0
        for v in f:
            key = (key << 12) | int(v)
        distinct.add(key)
    distinct = np.array(sorted(distinct), dtype=np.uint64)
    wts = 1.0 / np.arange(1, n_groups + 1) ** skew
    wts /= wts.sum()
    pick = rng.choice(n_groups, size=N, p=wts)
    return np.ascontiguousarray(distinct[rng.permutation(n_groups)][pick])
