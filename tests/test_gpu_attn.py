"""Parity of vardrop_attn_fwd / vardrop_attn_bwd (bf16 tensor-core kernels) with the fp64 oracle.
Tolerance: max-abs 2e-2 and mean-abs 2e-3 on outputs and gradients."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_14183_b200 import binding as vd
from util import assert_attn_close, bf16_tokens

pytestmark = pytest.mark.gpu


def run_attention(dev, B, N, H, D, sel, poison=True):
    """Runs forward and backward through the C ABI.  `sel` is None (all tokens) or a sorted int array.
    Returns o[B,Ns,H,D], lse[B,H,Ns], dq, dk, dv (numpy, float64) and the device status."""
    q, k, v, d_full = dev
    cfg = vd.AttnCfg(B, N, H, D, 0.0)
    ws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(cfg))
    if poison:
        ws.view(torch.int16).fill_(0x7FC1)        # bf16 NaN pattern everywhere in the scratch
        ws[:4] = 0                                # except the status word, which the caller zeroes (the library only sets it)
    fill = float("nan") if poison else 0.0
    o = torch.full((B, N, H, D), fill, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, H, N), fill, dtype=torch.float32, device="cuda")
    if sel is None:
        Ns, sel_t, nsel_t, inv_t = N, None, None, None
        d_o = d_full
    else:
        Ns = len(sel)
        sel_pad = np.full(N, -1, np.int32); sel_pad[:Ns] = sel
        inv = np.full(N, -1, np.int32); inv[sel] = np.arange(Ns, dtype=np.int32)
        sel_t = torch.from_numpy(sel_pad).cuda(); inv_t = torch.from_numpy(inv).cuda()
        nsel_t = torch.tensor([Ns], dtype=torch.int32, device="cuda")
        d_o = torch.full((B, N, H, D), fill, dtype=torch.bfloat16, device="cuda")      # rows past Ns may hold anything
        d_o[:, :Ns] = d_full[:, :Ns]
    vd.vardrop_attn_fwd(q, k, v, sel_t, nsel_t, cfg, o, lse, ws)
    dq, dk, dv = (torch.full((B, N, H, D), fill, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, sel_t, nsel_t, inv_t, cfg, dq, dk, dv, ws)
    torch.cuda.synchronize()
    status = vd.ws_status(ws)
    f = lambda t: t.double().cpu().numpy()
    return f(o)[:, :Ns], f(lse)[:, :, :Ns], f(dq), f(dk), f(dv), status, (o, lse)


def check_case(B, N, H, D, sel, std, seed):
    dev, ref = bf16_tokens(B, N, H, D, std, seed)
    o, lse, dq, dk, dv, status, raw = run_attention(dev, B, N, H, D, sel)
    assert status == vd.OK
    Ns = N if sel is None else len(sel)
    wo, wl = oracle.attn_fwd(ref[0], ref[1], ref[2], sel)
    assert_attn_close(o, wo, "o")
    assert_attn_close(lse, wl, "lse")
    wq, wk, wv = oracle.attn_bwd(ref[0], ref[1], ref[2], ref[3][:, :Ns], sel)
    assert_attn_close(dq, wq, "dq")
    assert_attn_close(dk, wk, "dk")
    assert_attn_close(dv, wv, "dv")
    if sel is not None:
        dropped = np.setdiff1d(np.arange(N), sel)
        for g in (dq, dk, dv):
            assert np.all(g[:, dropped] == 0.0)                      # exact zeros at dropped variates
        # rows of o / lse past n_sel are left untouched (still the NaN fill)
        assert torch.isnan(raw[0][:, Ns:].float()).all() and torch.isnan(raw[1][:, :, Ns:]).all()


def pick(N, Ns, seed):
    return np.sort(np.random.default_rng(seed).choice(N, size=Ns, replace=False)).astype(np.int32)


@pytest.mark.parametrize("B,N,H,D,Ns", [
    (2, 21, 4, 32, 11), (1, 7, 1, 64, 1), (2, 40, 2, 64, 40), (2, 300, 2, 64, 128), (1, 300, 3, 64, 129),
    (2, 321, 2, 64, 97), (1, 600, 2, 64, 300), (1, 500, 2, 32, 257), (3, 130, 1, 64, 127)])
@pytest.mark.parametrize("std", [1.0, 0.3536])
def test_attention_selected(B, N, H, D, Ns, std):
    check_case(B, N, H, D, pick(N, Ns, seed=N + Ns), std, seed=N * 7 + Ns)


@pytest.mark.parametrize("B,N,H,D", [(2, 21, 4, 32), (1, 128, 2, 64), (2, 200, 2, 64), (1, 385, 2, 64), (1, 256, 1, 32), (1, 1, 1, 64)])
def test_attention_all_tokens(B, N, H, D):
    check_case(B, N, H, D, None, 1.0, seed=N)


@pytest.mark.parametrize("B,N,H,D,Ns", [(1, 512, 2, 64, 200), (1, 513, 2, 64, 200), (1, 512, 2, 64, 256), (1, 512, 1, 64, 384),
                                        (1, 512, 1, 64, 512), (1, 640, 2, 32, 384), (2, 1100, 1, 64, 640)])
def test_attention_selected_at_path_boundaries(B, N, H, D, Ns):
    """Both sides of the largest N whose kept rows are gathered by the tile loads themselves (512), kept counts that fill
    whole tiles exactly (two, three, four tiles on the gathered path; three and five on the staged one), head size 32."""
    check_case(B, N, H, D, pick(N, Ns, seed=N * 3 + Ns), 1.0, seed=N + 11 * Ns)


def test_attention_random_configurations():
    """Seeded random draws of (B, N, H, D, kept count, value scale): gathered, staged and all-token paths, one to six tiles.
    Value scales stay at or below 1: the absolute tolerance is stated for unit-scale tokens (bf16 rounding of P and dS is
    relative, so gradients of larger tokens carry proportionally larger absolute errors)."""
    rng = np.random.default_rng(2025)
    for it in range(14):
        N = int(rng.integers(2, 760))
        D = int(rng.choice([64, 64, 32]))
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        Ns = int(rng.integers(1, N + 1))
        sel = None if it % 4 == 3 else pick(N, Ns, seed=it)
        check_case(B, N, H, D, sel, float(rng.choice([1.0, 0.3536, 0.6])), seed=500 + it)


@pytest.mark.parametrize("B,N,H,D,Ns,std", [(3, 341, 2, 32, 326, 2.0), (2, 604, 1, 64, 210, 2.0), (1, 300, 2, 64, None, 3.0)])
def test_attention_large_tokens_relative_error(B, N, H, D, Ns, std):
    """Tokens a few times the unit scale: peaky softmax rows and gradients of tens.  The errors of the bf16 products are
    relative, so the bound is the unit-scale tolerance times the largest magnitude of the tensor."""
    dev, ref = bf16_tokens(B, N, H, D, std, seed=N + 5)
    sel = None if Ns is None else pick(N, Ns, seed=N)
    o, lse, dq, dk, dv, status, _ = run_attention(dev, B, N, H, D, sel)
    assert status == vd.OK
    n_rows = N if sel is None else len(sel)
    wo, wl = oracle.attn_fwd(ref[0], ref[1], ref[2], sel)
    wq, wk, wv = oracle.attn_bwd(ref[0], ref[1], ref[2], ref[3][:, :n_rows], sel)
    for got, want, name in ((o, wo, "o"), (lse, wl, "lse"), (dq, wq, "dq"), (dk, wk, "dk"), (dv, wv, "dv")):
        bound = 2e-2 * max(1.0, float(np.abs(want).max()))
        err = float(np.abs(got - want).max())
        assert np.all(np.isfinite(got)) and err <= bound, f"{name}: max abs error {err:.3e} > {bound:.3e}"


def test_attention_identity_selection_equals_all_token_path():
    B, N, H, D = 1, 200, 2, 64
    dev, _ = bf16_tokens(B, N, H, D, 1.0, seed=3)
    a = run_attention(dev, B, N, H, D, None, poison=False)
    b = run_attention(dev, B, N, H, D, np.arange(N, dtype=np.int32), poison=False)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])       # forward is bit-reproducible
    for x, y in zip(a[3:5], b[3:5]):
        assert np.array_equal(x, y)                                        # dk, dv too
    np.testing.assert_allclose(a[2], b[2], atol=1e-2)                      # dq: atomics, order may differ


def test_attention_forward_is_deterministic():
    B, N, H, D = 2, 300, 2, 64
    dev, _ = bf16_tokens(B, N, H, D, 1.0, seed=4)
    sel = pick(N, 200, 1)
    a = run_attention(dev, B, N, H, D, sel, poison=False)
    b = run_attention(dev, B, N, H, D, sel, poison=False)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[3], b[3]) and np.array_equal(a[4], b[4])


@pytest.mark.parametrize("B,N,H,D,Ns", [(2, 300, 2, 64, 260), (2, 600, 2, 64, 300), (1, 700, 2, 64, None), (2, 321, 2, 64, 97)])
def test_attention_backward_is_reproducible(B, N, H, D, Ns):
    """Gathered, staged and all-token paths with several tiles: every gradient is bit for bit the same from run to run while
    no (instance, head) pair has more than two key tiles' worth of additions per accumulator row (two fp32 addends commute);
    with more tiles dq may differ in the last bits only.  Guards the shared-memory hand-offs inside the backward kernel."""
    dev, _ = bf16_tokens(B, N, H, D, 1.0, seed=N + (Ns or 0))
    sel = None if Ns is None else pick(N, Ns, 3)
    runs = [run_attention(dev, B, N, H, D, sel, poison=False) for _ in range(3)]
    tiles = -(-(Ns or N) // 128)
    for r in runs[1:]:
        assert np.array_equal(runs[0][3], r[3]) and np.array_equal(runs[0][4], r[4])          # dk, dv
        if tiles <= 2:
            assert np.array_equal(runs[0][2], r[2])                                            # dq
        else:
            np.testing.assert_allclose(runs[0][2], r[2], rtol=0, atol=2e-3)


def test_attention_argument_errors():
    q = torch.zeros((1, 8, 1, 64), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((1, 1, 8), device="cuda")
    ws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(vd.AttnCfg(1, 8, 1, 64, 0.0)))
    with pytest.raises(vd.VardropError) as e:
        vd.vardrop_attn_fwd(q, q, q, None, None, vd.AttnCfg(1, 8, 1, 128, 0.0), q, lse, ws)
    assert e.value.status == vd.ERR_UNSUPPORTED
    with pytest.raises(vd.VardropError) as e:
        vd.vardrop_attn_fwd(q, q, q, None, None, vd.AttnCfg(1, 8, 1, 64, 0.0), q, lse, ws[:256])
    assert e.value.status == vd.ERR_WORKSPACE
    with pytest.raises(vd.VardropError) as e:
        vd.vardrop_attn_fwd(q, None, q, None, None, vd.AttnCfg(1, 8, 1, 64, 0.0), q, lse, ws)
    assert e.value.status == vd.ERR_INVALID_ARG


def test_attention_per_instance_selections():
    """One selection per instance (S = B): every instance keeps its own variates, with different counts, spanning one and two tiles."""
    B, N, H, D = 4, 300, 2, 64
    dev, ref = bf16_tokens(B, N, H, D, 1.0, seed=21)
    q, k, v, d_full = dev
    counts = [17, 128, 129, 260]
    sels = [pick(N, c, seed=100 + i) for i, c in enumerate(counts)]
    sel_pad = np.full((B, N), -1, np.int32); inv = np.full((B, N), -1, np.int32)
    for b, s_ in enumerate(sels):
        sel_pad[b, :len(s_)] = s_
        inv[b, s_] = np.arange(len(s_), dtype=np.int32)
    cfg = vd.AttnCfg(B, N, H, D, 0.0, B)
    ws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(cfg))
    ws.view(torch.int16).fill_(0x7FC1)
    ws[:4] = 0                                    # the status word is the caller's to zero
    nan = float("nan")
    o = torch.full((B, N, H, D), nan, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, H, N), nan, dtype=torch.float32, device="cuda")
    d_o = torch.full((B, N, H, D), nan, dtype=torch.bfloat16, device="cuda")
    for b, c in enumerate(counts):
        d_o[b, :c] = d_full[b, :c]
    sel_t, inv_t = torch.from_numpy(sel_pad).cuda(), torch.from_numpy(inv).cuda()
    nsel_t = torch.tensor(counts, dtype=torch.int32, device="cuda")
    vd.vardrop_attn_fwd(q, k, v, sel_t, nsel_t, cfg, o, lse, ws)
    dq, dk, dv = (torch.full((B, N, H, D), nan, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, sel_t, nsel_t, inv_t, cfg, dq, dk, dv, ws)
    torch.cuda.synchronize()
    assert vd.ws_status(ws) == vd.OK
    for b, (c, s_) in enumerate(zip(counts, sels)):
        cut = [r[b:b + 1] for r in ref]
        wo, wl = oracle.attn_fwd(cut[0], cut[1], cut[2], s_)
        assert_attn_close(o[b:b + 1, :c].double().cpu().numpy(), wo, f"o[{b}]")
        assert_attn_close(lse[b:b + 1, :, :c].double().cpu().numpy(), wl, f"lse[{b}]")
        wq, wk, wv = oracle.attn_bwd(cut[0], cut[1], cut[2], cut[3][:, :c], s_)
        for got, want, name in ((dq, wq, "dq"), (dk, wk, "dk"), (dv, wv, "dv")):
            g = got[b:b + 1].double().cpu().numpy()
            assert_attn_close(g, want, f"{name}[{b}]")
            assert np.all(g[:, np.setdiff1d(np.arange(N), s_)] == 0.0)
        assert torch.isnan(o[b, c:].float()).all()


def run_strided(q, k, v, d_full, B, N, H, D, sel):
    """q, k, v are (possibly non-contiguous) views [B, N, H, D] with a contiguous head dimension; their strides go into the config."""
    assert q.stride() == k.stride() == v.stride() and q.stride(3) == 1
    cfg = vd.AttnCfg(B, N, H, D, 0.0, 1, q.stride(0), q.stride(1), q.stride(2))
    ws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(cfg))
    o = torch.full((B, N, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, H, N), float("nan"), dtype=torch.float32, device="cuda")
    if sel is None:
        Ns, sel_t, nsel_t, inv_t, d_o = N, None, None, None, d_full
    else:
        Ns = len(sel)
        sel_pad = np.full(N, -1, np.int32); sel_pad[:Ns] = sel
        inv = np.full(N, -1, np.int32); inv[sel] = np.arange(Ns, dtype=np.int32)
        sel_t, inv_t = torch.from_numpy(sel_pad).cuda(), torch.from_numpy(inv).cuda()
        nsel_t = torch.tensor([Ns], dtype=torch.int32, device="cuda")
        d_o = torch.full((B, N, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        d_o[:, :Ns] = d_full[:, :Ns]
    vd.vardrop_attn_fwd(q, k, v, sel_t, nsel_t, cfg, o, lse, ws)
    dq, dk, dv = (torch.full((B, N, H, D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(3))
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, sel_t, nsel_t, inv_t, cfg, dq, dk, dv, ws)
    torch.cuda.synchronize()
    assert vd.ws_status(ws) == vd.OK
    f = lambda t: t.double().cpu().numpy()
    return f(o)[:, :Ns], f(lse)[:, :, :Ns], f(dq), f(dk), f(dv)


@pytest.mark.parametrize("layout", ["fused_qkv", "padded_heads", "padded_tokens", "token_slice"])
@pytest.mark.parametrize("B,N,H,D,Ns", [(2, 300, 2, 64, 140), (1, 700, 2, 64, 300), (2, 200, 3, 64, None), (1, 600, 2, 64, None), (2, 90, 2, 32, 50)])
def test_attention_strided_qkv(layout, B, N, H, D, Ns):
    """q, k, v as views of larger buffers (the element strides of the configuration): slices of a fused [B, N, 3, H, D] projection,
    heads padded to D + 8, tokens padded by 8 elements (no row view: the library stages), and a slice along N of a longer
    sequence.  Results must match the oracle run on contiguous copies."""
    dev, ref = bf16_tokens(B, N, H, D, 0.5, seed=N + H)
    gen = torch.Generator(device="cuda").manual_seed(5)
    junk = lambda *shape: (torch.rand(shape, device="cuda", generator=gen) * 8 - 4).to(torch.bfloat16)       # what lies between the rows
    if layout == "fused_qkv":
        buf = junk(B, N, 3, H, D)
        views = [buf[:, :, i] for i in range(3)]
    elif layout == "padded_heads":
        bufs = [junk(B, N, H, D + 8) for _ in range(3)]
        views = [b[..., :D] for b in bufs]
    elif layout == "padded_tokens":
        bufs = [junk(B, N, H * D + 8) for _ in range(3)]
        views = [b[..., : H * D].unflatten(-1, (H, D)) for b in bufs]
    else:
        bufs = [junk(B, N + 37, H, D) for _ in range(3)]
        views = [b[:, 16: 16 + N] for b in bufs]
    for view, t in zip(views, dev[:3]):
        view.copy_(t)
    sel = None if Ns is None else pick(N, Ns, seed=N)
    o, lse, dq, dk, dv = run_strided(views[0], views[1], views[2], dev[3], B, N, H, D, sel)
    n_rows = N if sel is None else len(sel)
    wo, wl = oracle.attn_fwd(ref[0], ref[1], ref[2], sel)
    wq, wk, wv = oracle.attn_bwd(ref[0], ref[1], ref[2], ref[3][:, :n_rows], sel)
    for got, want, name in ((o, wo, "o"), (lse, wl, "lse"), (dq, wq, "dq"), (dk, wk, "dk"), (dv, wv, "dv")):
        assert_attn_close(got, want, f"{layout} {name}")


def test_attention_stride_validation():
    q = torch.zeros((1, 8, 2, 64), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros_like(q)
    lse = torch.zeros((1, 2, 8), device="cuda")
    ws = vd.alloc_ws(1 << 20)
    for strides in [(8 * 128, 128, 60), (8 * 128, 132, 64), (100, 128, 64), (8 * 128, 64, 128)]:
        with pytest.raises(vd.VardropError) as e:
            vd.vardrop_attn_fwd(q, q, q, None, None, vd.AttnCfg(1, 8, 2, 64, 0.0, 1, *strides), o, lse, ws)
        assert e.value.status == vd.ERR_INVALID_ARG


def test_backward_without_a_fresh_forward_is_reported():
    """The forward pass leaves state for exactly one backward pass in the workspace; a second backward on it is flagged in the
    device status word instead of silently adding into a consumed accumulator."""
    B, N, H, D = 1, 300, 2, 64
    dev, _ = bf16_tokens(B, N, H, D, 1.0, seed=3)
    q, k, v, d_o = dev
    cfg = vd.AttnCfg(B, N, H, D, 0.0)
    ws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(cfg))
    o = torch.zeros_like(q); lse = torch.zeros((B, H, N), device="cuda")
    dq, dk, dv = (torch.zeros_like(q) for _ in range(3))
    vd.vardrop_attn_fwd(q, k, v, None, None, cfg, o, lse, ws)
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, None, None, None, cfg, dq, dk, dv, ws)
    assert vd.ws_status(ws) == vd.OK
    first = dq.clone()
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, None, None, None, cfg, dq, dk, dv, ws)          # no forward in between
    assert vd.ws_status(ws) == vd.ERR_INVALID_ARG
    ws[:4] = 0                                                                                 # the caller clears the word ...
    vd.vardrop_attn_fwd(q, k, v, None, None, cfg, o, lse, ws)                                  # ... and the pair works again
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, None, None, None, cfg, dq, dk, dv, ws)
    assert vd.ws_status(ws) == vd.OK
    np.testing.assert_allclose(dq.float().cpu().numpy(), first.float().cpu().numpy(), rtol=0, atol=2e-3)
