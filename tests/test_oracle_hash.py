"""Pins for the oracle's k-DFH (Algorithm 1): closed forms, identities, library special cases and the labels the
paper prints.  None of these re-types the oracle's own formula."""
import os

import numpy as np
import pytest

import oracle
from paper_2501_14183_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        return [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]


def unpack(key, k):
    return tuple((int(key) >> (12 * (k - 1 - j))) & 0xFFF for j in range(k))


# --- step 1: amplitudes -------------------------------------------------------------------------------
@pytest.mark.parametrize("L", [96, 97, 336, 720])
def test_pure_sinusoid_closed_form(L):
    # A sin(2 pi f0 t / L + phi), integer 0 < f0 < L/2: |X_f0| = A L / 2 and every other bin is zero.
    f0, A = 7, 1.75
    t = np.arange(L)
    x = (A * np.sin(2 * np.pi * f0 * t / L + 0.3)).astype(np.float32)[None, None, :]
    amp = oracle.dft_amplitudes(x, 0, L // 2 + 1)[0, 0]
    assert abs(amp[f0] - A * L / 2) < 2e-5 * L
    others = np.delete(amp, f0)
    assert np.all(np.abs(others) < 2e-5 * L)


@pytest.mark.parametrize("L", [96, 97, 336])
def test_parseval(L):
    rng = np.random.default_rng(L)
    x = rng.normal(size=(2, 3, L)).astype(np.float32)
    amp = oracle.dft_amplitudes(x, 0, L // 2 + 1)
    w = np.full(L // 2 + 1, 2.0)
    w[0] = 1.0
    if L % 2 == 0:
        w[-1] = 1.0
    lhs = (x.astype(np.float64) ** 2).sum(-1)
    rhs = (w * amp ** 2).sum(-1) / L
    np.testing.assert_allclose(lhs, rhs, rtol=1e-12)


@pytest.mark.parametrize("L,lo,hi", [(96, 1, 25), (336, 0, 169), (720, 3, 181), (50, 1, 13)])
def test_matches_library_rfft(L, lo, hi):
    rng = np.random.default_rng(7 * L)
    x = rng.normal(size=(3, 5, L)).astype(np.float32)
    ref = np.abs(np.fft.rfft(x.astype(np.float64), axis=-1))[..., lo:hi]
    np.testing.assert_allclose(oracle.dft_amplitudes(x, lo, hi), ref, rtol=1e-10, atol=1e-10)


def test_trend_amplitudes_closed_form():
    # x_t = t: |X_f| = L / (2 sin(pi f / L)) for f >= 1 (geometric-series derivative).
    L = 96
    x = np.arange(L, dtype=np.float32)[None, None, :]
    amp = oracle.dft_amplitudes(x, 1, 25)[0, 0]
    f = np.arange(1, 25)
    np.testing.assert_allclose(amp, L / (2 * np.sin(np.pi * f / L)), rtol=1e-12)


# --- steps 2-5: low-pass, batch mean, ranking, packing --------------------------------------------------
def test_default_band_is_paper_cutoff():
    for tag, *rest in _golden_lines("paper_hash_labels.txt"):
        if tag == "cutoff":
            L, eps = int(rest[0]), int(rest[1])
            assert oracle.default_band(L) == (1, eps)


def test_sinusoid_hashes_to_its_own_bin():
    L, B, N = 96, 4, 24
    bins = np.arange(1, 25)[:, None]
    x = inputs.make_sinusoid_windows(B, N, L, bins, np.ones((N, 1)), seed=1)
    keys, freqs, _ = oracle.hash(x, k=1)
    assert keys.shape == (1, N)
    assert [int(v) for v in keys[0]] == list(range(1, 25))
    assert freqs[0, :, 0].tolist() == list(range(1, 25))


@pytest.mark.parametrize("B", [1, 5])
def test_sum_of_sinusoids_ranked_by_amplitude(B):
    # Orthogonality (Appendix C): the top-k bins of a sum of integer-bin sinusoids are its k largest
    # components in amplitude order, whatever the phases and the batch size.
    L, k = 96, 3
    rng = np.random.default_rng(3)
    N = 40
    bins = np.stack([rng.choice(np.arange(1, 25), size=5, replace=False) for _ in range(N)])
    amps = np.stack([np.sort(rng.uniform(0.2, 3.0, size=5))[::-1] * np.array([1, .8, .6, .4, .2]) for _ in range(N)])
    x = inputs.make_sinusoid_windows(B, N, L, bins, amps, seed=4)
    keys, freqs, abar = oracle.hash(x, k=k)
    assert np.array_equal(freqs[0], bins[:, :k])
    for n in range(N):
        assert unpack(keys[0, n], k) == tuple(bins[n, :k])
    # mean amplitude at a component bin is a_i L / 2
    for n in range(N):
        np.testing.assert_allclose(abar[0, n, bins[n] - 1], amps[n] * L / 2, rtol=1e-5)


def test_order_is_part_of_the_hash():
    # Fig. 6(a): 4-12-8 and 12-4-8 are different groups.
    L = 96
    cases = [ln[1:] for ln in _golden_lines("paper_hash_labels.txt") if ln[0] == "distinct"]
    for a, b in cases:
        fa = [int(v) for v in a.split("-")]
        fb = [int(v) for v in b.split("-")]
        k = len(fa)
        amps = np.array([[1.0 / (1.6 ** i) for i in range(k)]] * 2)
        x = inputs.make_sinusoid_windows(2, 2, L, np.array([fa, fb]), amps, seed=5)
        keys, freqs, _ = oracle.hash(x, k=k)
        assert freqs[0, 0].tolist() == fa and freqs[0, 1].tolist() == fb
        assert keys[0, 0] != keys[0, 1]
        assert sorted(fa) == sorted(fb)


def test_flat_trend_hashes_1_2_3():
    # Fig. 9(a): a flat, trend-like variate carries the label 1-2-3.
    (label,) = [ln[1] for ln in _golden_lines("paper_hash_labels.txt") if ln[0] == "trend"]
    want = [int(v) for v in label.split("-")]
    L = 96
    x = (0.01 * np.arange(L, dtype=np.float32) + 3.0)[None, None, :].repeat(4, axis=0)
    _, freqs, _ = oracle.hash(x, k=3)
    assert freqs[0, 0].tolist() == want


def test_reconstruction_error_theorem():
    # Theorem 1 / Appendix C: rebuilding the signal from its k dominant components leaves an MSE of
    # half the sum of the squared amplitudes of the others.
    L, k = 96, 3
    bins = np.array([[4, 12, 8, 20, 16, 2]])
    amps = np.array([[2.0, 1.5, 1.0, 0.5, 0.3, 0.2]])
    rng = np.random.default_rng(0)
    ph = rng.uniform(0, 2 * np.pi, size=6)
    t = np.arange(L)
    comps = [amps[0, i] * np.sin(2 * np.pi * bins[0, i] * t / L + ph[i]) for i in range(6)]
    x = np.sum(comps, axis=0)
    _, freqs, _ = oracle.hash(x.astype(np.float32)[None, None, :], k=k)
    top = freqs[0, 0].tolist()
    assert top == [4, 12, 8]
    recon = np.sum([comps[i] for i in range(6) if bins[0, i] in top], axis=0)
    mse = np.mean((x - recon) ** 2)
    assert abs(mse - 0.5 * np.sum(amps[0, 3:] ** 2)) < 1e-12


def test_batch_mean_is_mean_of_amplitudes():
    # Step 3 averages amplitudes, not spectra: two instances with opposite phase do not cancel.
    L = 96
    t = np.arange(L)
    x = np.stack([np.sin(2 * np.pi * 5 * t / L), -np.sin(2 * np.pi * 5 * t / L)])[:, None, :].astype(np.float32)
    keys, freqs, abar = oracle.hash(x, k=1)
    assert freqs[0, 0, 0] == 5
    assert abs(abar[0, 0, 4] - L / 2) < 1e-4
    # and equals the mean of the per-instance amplitudes the library transform gives
    ref = np.abs(np.fft.rfft(x.astype(np.float64), axis=-1))[:, :, 1:25].mean(axis=0)
    np.testing.assert_allclose(abar[0], ref, rtol=1e-10, atol=1e-10)


def test_batch_mean_changes_the_ranking():
    # instance 0 is dominated by bin 3, instance 1 (larger) by bin 9: the batch hash follows the mean.
    L = 96
    bins = np.array([[3, 9]])
    x0 = inputs.make_sinusoid_windows(1, 1, L, bins, np.array([[1.0, 0.5]]), seed=1)
    x1 = inputs.make_sinusoid_windows(1, 1, L, bins, np.array([[1.0, 3.0]]), seed=2)
    x = np.concatenate([x0, x1], axis=0)
    _, f_batch, _ = oracle.hash(x, k=2, scope=0)
    _, f_inst, _ = oracle.hash(x, k=2, scope=1)
    assert f_batch[0, 0].tolist() == [9, 3]
    assert f_inst[0, 0].tolist() == [3, 9] and f_inst[1, 0].tolist() == [9, 3]


def test_ties_rank_lower_bin_first():
    # all-zero window: every amplitude is exactly 0 -> the k lowest candidate bins in ascending order.
    x = np.zeros((2, 1, 96), dtype=np.float32)
    _, freqs, _ = oracle.hash(x, k=4)
    assert freqs[0, 0].tolist() == [1, 2, 3, 4]
    _, freqs, _ = oracle.hash(x, k=3, f_lo=0, f_hi=10)
    assert freqs[0, 0].tolist() == [0, 1, 2]


def test_low_pass_removes_high_bins():
    L = 96
    x = inputs.make_sinusoid_windows(2, 1, L, np.array([[30, 6]]), np.array([[5.0, 1.0]]), seed=9)
    _, f_lp, _ = oracle.hash(x, k=1)                           # cut-off 25: bin 30 is filtered out
    _, f_all, _ = oracle.hash(x, k=1, f_lo=1, f_hi=L // 2 + 1)
    assert f_lp[0, 0, 0] == 6 and f_all[0, 0, 0] == 30


def test_scale_and_noise_invariance():
    # "Noise Robustness": positive rescaling and small broadband noise leave the hash unchanged when the
    # rank gaps are large.
    L, N = 96, 30
    rng = np.random.default_rng(11)
    bins = np.stack([rng.choice(np.arange(1, 25), size=3, replace=False) for _ in range(N)])
    amps = np.tile(np.array([[3.0, 2.0, 1.0]]), (N, 1))
    x = inputs.make_sinusoid_windows(4, N, L, bins, amps, seed=12)
    k0, _, _ = oracle.hash(x, k=3)
    k1, _, _ = oracle.hash((x * 7.5).astype(np.float32), k=3)
    k2, _, _ = oracle.hash((x + rng.normal(0, 0.05, size=x.shape)).astype(np.float32), k=3)
    assert np.array_equal(k0, k1) and np.array_equal(k0, k2)


def test_key_packing_layout():
    L = 720
    x = inputs.make_sinusoid_windows(1, 1, L, np.array([[100, 7, 150, 33, 2]]), np.array([[5., 4., 3., 2., 1.]]), seed=2)
    keys, freqs, _ = oracle.hash(x, k=5)
    assert freqs[0, 0].tolist() == [100, 7, 150, 33, 2]
    assert int(keys[0, 0]) == (((((100 << 12) | 7) << 12 | 150) << 12 | 33) << 12) | 2


def test_workload_generator_redundancy():
    # the synthetic Electricity-shaped windows group into far fewer hashes than variates
    w = inputs.WORKLOADS["elec"]
    x = inputs.make_windows(w, B=8)
    keys, _, _ = oracle.hash(x, k=w.k)
    G = len(np.unique(keys[0]))
    assert 10 <= G <= w.N // 2
