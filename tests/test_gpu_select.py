"""Parity of vardrop_select with the oracle: every output bit-exact (integer work)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_14183_b200 import binding as vd
from paper_2501_14183_b200 import inputs

pytestmark = pytest.mark.gpu


def run_select(keys, gs, rate, seed, step):
    keys = np.atleast_2d(keys)
    S, N = keys.shape
    cfg = vd.SelectCfg(S, N, gs, rate, seed, step)
    kd = torch.from_numpy(keys.view(np.int64)).cuda()
    out = vd.alloc_select_outputs(cfg)
    ws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(cfg))
    vd.vardrop_select(kd, cfg, out["group_id"], out["group_offsets"], out["members"], out["n_groups"], out["sel_idx"],
                      out["n_sel"], out["inv_idx"], ws)
    torch.cuda.synchronize()
    assert vd.ws_status(ws) == vd.OK
    return {k: v.cpu().numpy() for k, v in out.items()}


def check(keys, gs, rate, seed, step):
    want = oracle.select(keys, gs, rate, seed, step)
    got = run_select(keys, gs, rate, seed, step)
    for name in ("n_groups", "n_sel", "group_id", "group_offsets", "members", "sel_idx", "inv_idx"):
        assert np.array_equal(got[name], want[name]), name
    return got


@pytest.mark.parametrize("N,G", [(1, 1), (2, 2), (21, 4), (127, 9), (128, 128), (129, 1), (257, 30), (321, 40), (862, 60),
                                 (1000, 1000), (3000, 7), (8192, 512)])
@pytest.mark.parametrize("gs,rate", [(10, 1.0), (0, 0.2), (3, 0.5)])
def test_select_parity(N, G, gs, rate):
    keys = inputs.make_keys(N, G, k=4, f_hi=85, seed=N + G)
    check(keys, gs, rate, seed=0xC0FFEE1234567, step=N % 7)


def test_select_degenerate_groups():
    same = np.full(2000, (5 << 24) | (9 << 12) | 2, dtype=np.uint64)
    got = check(same, 10, 1.0, seed=1, step=0)
    assert got["n_groups"][0] == 1 and got["n_sel"][0] == 10
    distinct = np.arange(1, 1501, dtype=np.uint64)[np.random.default_rng(0).permutation(1500)]
    got = check(distinct, 10, 1.0, seed=1, step=0)
    assert got["n_groups"][0] == 1500 and got["n_sel"][0] == 1500
    check(np.full(300, 0xFFFFFFFFFFFFFFF, dtype=np.uint64), 0, 0.1, seed=3, step=9)     # 60-bit keys (k = 5)


def test_select_group_sizes_around_the_counting_limit():
    """The one-CTA path ranks members by counting inside groups of up to 64 and sorts when some group is longer: both sides of it."""
    rng = np.random.default_rng(11)
    for sizes in ([64, 64, 64], [65, 64, 64], [64, 1, 63, 2], [300, 5, 5, 5], [1] * 40 + [64]):
        keys = np.concatenate([np.full(n, 100 + 7 * i, dtype=np.uint64) for i, n in enumerate(sizes)])
        keys = keys[rng.permutation(len(keys))]
        for gs, rate in ((10, 1.0), (0, 0.3)):
            check(keys, gs, rate, seed=99, step=4)


def test_select_long_rows():
    """Rows beyond the one-CTA path: grouping with its working arrays in shared memory (up to 18432 variates), at that
    limit, and on the global arrays beyond it; several rows at once; one group only and all-distinct keys."""
    for N, G in ((18432, 700), (18433, 50), (24000, 3000)):
        check(inputs.make_keys(N, G, k=4, f_hi=169, seed=N), 10, 1.0, seed=42, step=2)
    rows = np.stack([inputs.make_keys(2500, 30 + 40 * s, k=3, f_hi=49, seed=90 + s) for s in range(3)])
    check(rows, 0, 0.25, seed=7, step=1)
    rows = np.stack([inputs.make_keys(19000, 100 + 900 * s, k=4, f_hi=169, seed=190 + s) for s in range(2)])
    check(rows, 4, 0.5, seed=8, step=6)
    got = check(np.full(5000, 77, dtype=np.uint64), 0, 0.1, seed=3, step=0)
    assert got["n_groups"][0] == 1 and got["n_sel"][0] == 500
    distinct = np.arange(1, 4097, dtype=np.uint64)[np.random.default_rng(1).permutation(4096)]
    got = check(distinct, 10, 1.0, seed=1, step=0)
    assert got["n_groups"][0] == 4096 and got["n_sel"][0] == 4096


def test_select_middle_rows():
    """Rows of 2049 .. 8192 variates: ragged sizes, keys that differ in all 64 bits or in a single one, one group, two groups
    of very different size, many equal groups of 512, 20 and 2 members, several rows at once."""
    rng = np.random.default_rng(5)
    wide = rng.integers(0, 2**63, size=5000, dtype=np.uint64) * np.uint64(2) + rng.integers(0, 2, size=5000, dtype=np.uint64)
    wide[rng.integers(0, 5000, size=700)] = wide[0]                        # one longer group among distinct keys
    wide[1] = np.uint64(0xFFFFFFFFFFFFFFFF)
    wide[2] = np.uint64(0)
    check(wide, 10, 1.0, seed=12, step=3)
    check(wide, 0, 0.3, seed=12, step=4)
    one_bit = (rng.integers(0, 2, size=8191, dtype=np.uint64) << np.uint64(63)) | np.uint64(0x123)
    got = check(one_bit, 0, 0.01, seed=2, step=0)
    assert got["n_groups"][0] == 2
    for N in (2049, 3073, 8191, 8192):
        for sizes in ([N], [N - 1, 1], [512] * (N // 512) + [N % 512], [20] * (N // 20) + [N % 20], [2] * (N // 2) + [N % 2]):
            sizes = [n for n in sizes if n > 0]
            keys = np.concatenate([np.full(n, (i * 0x9E3779B97F4A7C15) % 2**48, dtype=np.uint64) for i, n in enumerate(sizes)])
            keys = keys[rng.permutation(len(keys))]
            check(keys, 7, 0.4, seed=N, step=len(sizes) % 5)
    rows = np.stack([inputs.make_keys(6000, 10 + 700 * s, k=5, f_hi=361, seed=60 + s) for s in range(4)])
    check(rows, 0, 0.1, seed=31, step=2)


def test_select_random_configurations():
    """Seeded random draws of (N, rows, groups, gs, rate, k) on both sides of every size limit of the kernels
    (2048: one-CTA path; 18432: grouping in shared memory; 65536: the largest N)."""
    rng = np.random.default_rng(123)
    for it in range(24):
        N = int(rng.choice([63, 64, 65, 700, 2047, 2048, 2049, 4096, 8192, 18432, 18433, 30000, 65536]))
        S = int(rng.choice([1, 1, 2, 3])) if N <= 20000 else 1
        G = int(rng.integers(1, max(2, N // int(rng.choice([1, 2, 8, 50, 400])))))
        gs = int(rng.choice([0, 1, 3, 10, 100]))
        rate = float(rng.choice([0.05, 0.2, 0.5, 1.0]))
        k = int(rng.choice([3, 4, 5]))
        rows = np.stack([inputs.make_keys(N, G, k=k, f_hi=int(rng.choice([25, 49, 169, 361])), seed=1000 * it + s) for s in range(S)])
        check(rows, gs, rate, seed=int(rng.integers(0, 2**62)), step=int(rng.integers(0, 1000)))


def test_select_multiple_scopes():
    rows = np.stack([inputs.make_keys(500, 20 + s, k=3, f_hi=25, seed=s) for s in range(5)])
    got = check(rows, 5, 1.0, seed=77, step=3)
    assert len(set(got["n_sel"].tolist())) > 1


def test_select_paper_hyperparameters():
    # (k, gs) of Appendix E on keys hashed from the synthetic workloads
    for name, gs in (("elec", 10), ("traffic", 10), ("tiny", 5)):
        w = inputs.WORKLOADS[name]
        keys, _, _ = oracle.hash(inputs.make_windows(w, B=4), w.k)
        got = check(keys, gs, 1.0, seed=20250114, step=1)
        sizes = np.diff(got["group_offsets"][0][: got["n_groups"][0] + 1])
        assert got["n_sel"][0] == np.minimum(sizes, gs).sum()           # Eq. 1 summed over groups


def test_select_reproducible_and_step_dependent():
    keys = inputs.make_keys(862, 60, k=3, f_hi=25, seed=2)
    a = run_select(keys, 0, 0.2, seed=5, step=10)
    b = run_select(keys, 0, 0.2, seed=5, step=10)
    c = run_select(keys, 0, 0.2, seed=5, step=11)
    assert np.array_equal(a["sel_idx"], b["sel_idx"])
    assert not np.array_equal(a["sel_idx"], c["sel_idx"])
    assert a["n_sel"][0] == c["n_sel"][0]


def test_select_argument_errors():
    keys = torch.zeros((1, 8), dtype=torch.int64, device="cuda")
    cfg = vd.SelectCfg(1, 8, 0, 0.5, 1, 0)
    out = vd.alloc_select_outputs(cfg)
    args = (out["group_id"], out["group_offsets"], out["members"], out["n_groups"], out["sel_idx"], out["n_sel"], out["inv_idx"])
    small = vd.alloc_ws(256)
    with pytest.raises(vd.VardropError) as e:
        vd.vardrop_select(keys, cfg, *args, small[:128])
    assert e.value.status == vd.ERR_WORKSPACE
    ws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(cfg))
    for bad in (vd.SelectCfg(1, 8, 0, 0.0, 1, 0), vd.SelectCfg(1, 8, 0, 1.5, 1, 0), vd.SelectCfg(1, 0, 0, 0.5, 1, 0), vd.SelectCfg(0, 8, 0, 0.5, 1, 0)):
        with pytest.raises(vd.VardropError) as e:
            vd.vardrop_select(keys, bad, *args, ws)
        assert e.value.status == vd.ERR_INVALID_ARG
