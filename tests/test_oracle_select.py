"""Pins for the oracle's grouping and stratified sampling (Eq. 1, Eq. 2, delta) and its Philox generator."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2501_14183_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as fh:
        rows = [[int(t, 16) for t in ln.split()] for ln in fh if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for w in rows:
        assert oracle.philox4x32_10(w[:4], w[4:6]).tolist() == w[6:]


def brute_partition(keys):
    """O(N^2) equality partition, groups ordered by key, members by index."""
    N = len(keys)
    seen, groups = set(), []
    for key in sorted(set(int(v) for v in keys)):
        groups.append([n for n in range(N) if int(keys[n]) == key])
    return groups


@pytest.mark.parametrize("N,G,seed", [(1, 1, 0), (21, 4, 1), (64, 64, 2), (97, 1, 3), (321, 40, 4)])
def test_groups_match_brute_force(N, G, seed):
    keys = inputs.make_keys(N, min(G, N), k=3, f_hi=25, seed=seed)
    r = oracle.select(keys, gs=10, rate=1.0, seed=5, step=0)
    groups = brute_partition(keys)
    assert r["n_groups"][0] == len(groups)
    off = r["group_offsets"][0]
    assert off[0] == 0 and np.all(off[len(groups):] == N)
    for g, mem in enumerate(groups):
        assert r["members"][0, off[g]:off[g + 1]].tolist() == mem
        assert np.all(r["group_id"][0, mem] == g)


def test_permuting_variates_permutes_membership():
    N = 200
    keys = inputs.make_keys(N, 17, k=3, f_hi=25, seed=8)
    perm = np.random.default_rng(0).permutation(N)
    a = oracle.select(keys, gs=5, rate=1.0, seed=1, step=0)
    b = oracle.select(keys[perm], gs=5, rate=1.0, seed=1, step=0)
    # variate perm[i] of the first call is variate i of the second: same group id, same group sizes
    assert np.array_equal(a["group_id"][0][perm], b["group_id"][0])
    assert np.array_equal(np.diff(a["group_offsets"][0]), np.diff(b["group_offsets"][0]))
    assert a["n_sel"][0] == b["n_sel"][0]


@pytest.mark.parametrize("gs", [1, 5, 10, 20])
def test_eq1_counts_and_delta(gs):
    # rate = 1: |S_g| = min(|G_g|, gs), n_sel = sum_g min(|G_g|, gs), delta = 1 - n_sel / N.
    N = 321
    keys = inputs.make_keys(N, 33, k=3, f_hi=25, seed=21)
    r = oracle.select(keys, gs=gs, rate=1.0, seed=3, step=7)
    sizes = [len(g) for g in brute_partition(keys)]
    want = sum(min(s, gs) for s in sizes)
    assert r["n_sel"][0] == want
    sel = r["sel_idx"][0, :want]
    assert np.all(r["sel_idx"][0, want:] == -1)
    assert np.all(np.diff(sel) > 0)                              # ascending, no duplicates
    per_group = np.bincount(r["group_id"][0, sel], minlength=len(sizes))
    assert per_group.tolist() == [min(s, gs) for s in sizes]     # every group keeps exactly its quota
    delta = 1.0 - want / N
    assert abs(delta - (1.0 - sum(min(s, gs) for s in sizes) / N)) < 1e-15
    if gs == 1:
        assert want == len(sizes)                                # one representative per group
    inv = r["inv_idx"][0]
    assert np.array_equal(np.nonzero(inv >= 0)[0], sel)
    assert inv[sel].tolist() == list(range(want))


def test_rate_quota_formula():
    for size in [1, 2, 3, 7, 10, 33, 100, 8192]:
        for rate in [0.1, 0.2, 0.3, 0.5, 1.0]:
            for gs in [0, 1, 5, 20]:
                want = max(1, math.ceil(size * round(rate * 1e6) / 1e6 - 1e-12))
                want = min(size, want, gs if gs > 0 else size)
                assert oracle.quota(size, gs, rate) == want, (size, gs, rate)
    N = 862
    keys = inputs.make_keys(N, 60, k=3, f_hi=25, seed=2)
    r = oracle.select(keys, gs=0, rate=0.2, seed=9, step=1)
    sizes = [len(g) for g in brute_partition(keys)]
    assert r["n_sel"][0] == sum(max(1, -(-s * 200000 // 1000000)) for s in sizes)


def test_monotone_in_gs_and_rate():
    # Fig. 4: fewer tokens are dropped as gs grows.
    keys = inputs.make_keys(500, 25, k=4, f_hi=25, seed=3)
    ns = [int(oracle.select(keys, gs=g, rate=1.0, seed=1, step=0)["n_sel"][0]) for g in (1, 2, 5, 10, 20, 50, 0)]
    assert ns == sorted(ns) and ns[-1] == 500
    nr = [int(oracle.select(keys, gs=0, rate=r, seed=1, step=0)["n_sel"][0]) for r in (0.05, 0.1, 0.3, 0.5, 0.9, 1.0)]
    assert nr == sorted(nr) and nr[-1] == 500


def test_selection_is_uniform_without_replacement():
    # one group of 12, quota 4: over many steps every member is kept with frequency 4/12, every pair with
    # frequency (4*3)/(12*11); chi-square / z bounds are loose enough to be deterministic-safe, tight enough
    # to catch a biased or with-replacement draw.
    size, quota, trials = 12, 4, 6000
    keys = np.full(size, 0x004_00C_008, dtype=np.uint64)
    cnt = np.zeros(size)
    pair = np.zeros((size, size))
    for step in range(trials):
        r = oracle.select(keys, gs=quota, rate=1.0, seed=0xABCDEF0123, step=step)
        s = r["sel_idx"][0, :quota]
        assert r["n_sel"][0] == quota and len(set(s.tolist())) == quota
        cnt[s] += 1
        pair[np.ix_(s, s)] += 1
    exp = trials * quota / size
    chi2 = ((cnt - exp) ** 2 / exp).sum()
    assert chi2 < 40.0                                          # 11 dof; P(chi2 > 40) ~ 4e-5
    pexp = trials * quota * (quota - 1) / (size * (size - 1))
    off = pair[~np.eye(size, dtype=bool)]
    assert np.all(np.abs(off - pexp) < 6 * math.sqrt(pexp))


def test_selection_depends_on_seed_step_and_is_reproducible():
    keys = inputs.make_keys(300, 10, k=3, f_hi=25, seed=3)
    a = oracle.select(keys, gs=5, rate=1.0, seed=1, step=0)
    b = oracle.select(keys, gs=5, rate=1.0, seed=1, step=0)
    c = oracle.select(keys, gs=5, rate=1.0, seed=1, step=1)
    d = oracle.select(keys, gs=5, rate=1.0, seed=2, step=0)
    assert np.array_equal(a["sel_idx"], b["sel_idx"])
    assert not np.array_equal(a["sel_idx"], c["sel_idx"])
    assert not np.array_equal(a["sel_idx"], d["sel_idx"])


def test_priorities_follow_the_counter_scheme():
    # group g, member j (rank in ascending n), scope s: priority = word 0 of Philox(counter (j, g, s, step)).
    keys = inputs.make_keys(60, 5, k=3, f_hi=25, seed=4)
    keys2 = np.stack([keys, keys[::-1].copy()])
    seed, step, gs = 0x1234_5678_9ABC_DEF0, 42, 3
    r = oracle.select(keys2, gs=gs, rate=1.0, seed=seed, step=step)
    for s in range(2):
        off = r["group_offsets"][s]
        kept = set(r["sel_idx"][s, :r["n_sel"][s]].tolist())
        for g in range(r["n_groups"][s]):
            mem = r["members"][s, off[g]:off[g + 1]]
            pri = [(int(oracle.philox4x32_10([j, g, s, step], [seed & 0xFFFFFFFF, seed >> 32])[0]), j)
                   for j in range(len(mem))]
            want = {int(mem[j]) for _, j in sorted(pri)[:min(gs, len(mem))]}
            assert want == kept & set(mem.tolist())


def test_scopes_are_independent():
    keys = inputs.make_keys(100, 8, k=3, f_hi=25, seed=5)
    both = oracle.select(np.stack([keys, keys]), gs=4, rate=1.0, seed=7, step=3)
    assert np.array_equal(both["group_id"][0], both["group_id"][1])
    assert not np.array_equal(both["sel_idx"][0], both["sel_idx"][1])   # the scope enters the counter
