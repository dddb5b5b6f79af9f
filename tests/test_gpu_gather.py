"""vardrop_gather_rows (Sec. 3.3, the drop applied to the raw lookback window) against the oracle: a copy, so bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_14183_b200 import binding as vd
from paper_2501_14183_b200 import inputs

pytestmark = pytest.mark.gpu


def run(x, sel, n_sel):
    B, N, L = x.shape
    S = sel.shape[0]
    out = torch.full((B, N, L), float("nan"), dtype=torch.float32, device="cuda")
    vd.vardrop_gather_rows(torch.from_numpy(x).cuda(), torch.from_numpy(sel).cuda(), torch.from_numpy(n_sel).cuda(),
                           vd.GatherCfg(B, N, L, S), out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("B,N,L,S", [(4, 21, 96, 1), (3, 130, 97, 1), (5, 300, 336, 5), (2, 2049, 20, 1), (1, 7, 1, 1), (2, 64, 720, 2)])
def test_gather_rows_matches_oracle_bit_for_bit(B, N, L, S):
    rng = np.random.default_rng(B * 1000 + N + L)
    x = rng.normal(size=(B, N, L)).astype(np.float32)
    sel = np.full((S, N), -1, np.int32)
    n_sel = np.zeros(S, np.int32)
    for s in range(S):
        k = int(rng.integers(0 if S > 1 else 1, N + 1))
        sel[s, :k] = np.sort(rng.choice(N, size=k, replace=False))
        n_sel[s] = k
    got = run(x, sel, n_sel)
    want = oracle.gather_rows(x, sel, n_sel, fill=np.nan)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))          # copied rows and untouched rows (still the NaN fill)


def test_gather_rows_after_select_on_a_workload():
    w = inputs.WORKLOADS["traffic"]
    x = inputs.make_windows(w)
    hcfg = vd.HashCfg(w.B, w.N, w.L, w.k, 0, 0, 0)
    keys, freqs, _ = vd.alloc_hash_outputs(hcfg)
    hws = vd.alloc_ws(vd.vardrop_hash_workspace_bytes(hcfg))
    xd = torch.from_numpy(x).cuda()
    vd.vardrop_hash(xd, hcfg, keys, freqs, None, hws)
    scfg = vd.SelectCfg(1, w.N, 0, w.rate, 11, 2)
    so = vd.alloc_select_outputs(scfg)
    sws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(scfg))
    vd.vardrop_select(keys, scfg, so["group_id"], so["group_offsets"], so["members"], so["n_groups"], so["sel_idx"], so["n_sel"], so["inv_idx"], sws)
    out = torch.zeros_like(xd)
    vd.vardrop_gather_rows(xd, so["sel_idx"], so["n_sel"], vd.GatherCfg(w.B, w.N, w.L, 1), out)
    torch.cuda.synchronize()
    want = oracle.gather_rows(x, so["sel_idx"].cpu().numpy(), so["n_sel"].cpu().numpy())
    assert np.array_equal(out.cpu().numpy(), want)


def test_gather_rows_rejects_bad_configurations():
    x = torch.zeros((2, 4, 8), device="cuda")
    sel = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    n = torch.ones((1,), dtype=torch.int32, device="cuda")
    with pytest.raises(vd.VardropError) as e:
        vd.vardrop_gather_rows(x, sel, n, vd.GatherCfg(2, 4, 8, 3), torch.empty_like(x))
    assert e.value.status == vd.ERR_INVALID_ARG
    with pytest.raises(vd.VardropError):
        vd.vardrop_gather_rows(x, None, n, vd.GatherCfg(2, 4, 8, 1), torch.empty_like(x))
