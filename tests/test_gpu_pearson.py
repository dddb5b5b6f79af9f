"""Parity of vardrop_pearson_max (tensor-core products of two-term bf16 unit vectors) with the fp64 oracle of Eq. 4."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_14183_b200 import binding as vd
from paper_2501_14183_b200 import inputs

pytestmark = pytest.mark.gpu

# statistics in fp32 (relative 1e-6 at these lengths), values as hi + lo bf16 terms (2^-16 relative, the lo.lo product
# dropped), fp32 accumulation over at most a few thousand terms: a coefficient is off by a few 1e-6; 1e-4 is the contract
RHO_TOL = 1e-4


def run_pearson(x, threshold=0.9):
    B, N, L = x.shape
    cfg = vd.PearsonCfg(B, N, L, threshold)
    out = torch.full((B, N), float("nan"), dtype=torch.float32, device="cuda")
    above = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ws = vd.alloc_ws(vd.vardrop_pearson_workspace_bytes(cfg))
    ws[256:].view(torch.int16).fill_(0x7FC1)          # scratch contents must not matter (the status word stays zero)
    vd.vardrop_pearson_max(torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda(), cfg, out, above, ws)
    torch.cuda.synchronize()
    assert vd.ws_status(ws) == vd.OK
    return out.cpu().numpy().astype(np.float64), above.cpu().numpy()


def check(x, threshold=0.9):
    want = oracle.pearson_max(x)
    got, above = run_pearson(x, threshold)
    np.testing.assert_allclose(got, want, rtol=0, atol=RHO_TOL)
    # the count is an integer decided by a float: it may differ from the fp64 count only by variates within the tolerance of the threshold
    sure = (want >= threshold + RHO_TOL).sum(axis=1)
    maybe = (np.abs(want - threshold) < RHO_TOL).sum(axis=1)
    assert np.all(above >= sure) and np.all(above <= sure + maybe), (above, sure, maybe)
    return got


@pytest.mark.parametrize("B,N,L", [(1, 1, 96), (2, 2, 96), (3, 21, 96), (2, 127, 96), (2, 128, 64), (1, 129, 100), (2, 321, 96),
                                   (1, 300, 720), (1, 260, 336), (2, 40, 7), (1, 515, 130)])
def test_pearson_parity_random(B, N, L):
    rng = np.random.default_rng(B * 100 + N + L)
    x = rng.normal(size=(B, N, L)).astype(np.float32)
    if N > 4:
        x[:, 3] = 0.9 * x[:, 1] + 0.1 * x[:, 3]                       # some strong pairs
        x[:, N - 1] = -x[:, 0]                                        # and an anti-correlated one
    x += rng.normal(size=(B, N, 1)).astype(np.float32) * 5.0          # non-zero means
    check(x)


@pytest.mark.parametrize("name", ["tiny", "elec", "traffic", "long"])
def test_pearson_parity_workloads(name):
    w = inputs.WORKLOADS[name]
    x = inputs.make_windows(w, B=min(w.B, 2))
    got = check(x)
    print(f"[{name}] share of variates with a partner above 0.9: {(got > 0.9).mean():.3f}")


def test_pearson_constant_variates_and_threshold():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(1, 10, 96)).astype(np.float32)
    x[0, 4] = 3.0                                                     # constant: rho = 0 with everything
    x[0, 7] = x[0, 2]                                                 # duplicate: rho = 1
    got = check(x, threshold=0.5)
    assert abs(got[0, 7] - 1.0) < RHO_TOL and abs(got[0, 2] - 1.0) < RHO_TOL
    assert got[0, 4] == 0.0


def test_pearson_whole_scale_instance_against_the_oracle():
    # the Scale-shaped window (N = 8192, L = 336), one instance, every variate against the oracle (a couple of seconds of fp64 on the host)
    w = inputs.WORKLOADS["scale"]
    x = inputs.make_windows(w, B=1)
    got, _ = run_pearson(x)
    want = oracle.pearson_max(x)
    assert np.abs(got - want).max() < RHO_TOL


def test_pearson_argument_errors():
    x = torch.zeros((1, 4, 96), device="cuda")
    out = torch.zeros((1, 4), device="cuda")
    above = torch.zeros((1,), dtype=torch.int32, device="cuda")
    ws = vd.alloc_ws(vd.vardrop_pearson_workspace_bytes(vd.PearsonCfg(1, 4, 96, 0.9)))
    for cfg, status in [(vd.PearsonCfg(0, 4, 96, 0.9), vd.ERR_INVALID_ARG), (vd.PearsonCfg(1, 4, 1, 0.9), vd.ERR_INVALID_ARG),
                        (vd.PearsonCfg(1, 4, 96, 1.5), vd.ERR_INVALID_ARG)]:
        with pytest.raises(vd.VardropError) as e:
            vd.vardrop_pearson_max(x, cfg, out, above, ws)
        assert e.value.status == status
    with pytest.raises(vd.VardropError) as e:
        vd.vardrop_pearson_max(x, vd.PearsonCfg(1, 4, 96, 0.9), out, above, ws[:256])
    assert e.value.status == vd.ERR_WORKSPACE
