"""The whole hot path through the C ABI on the benchmark's configurations and launch shapes, against the oracle:
hash -> select bit-exact on rank-gap filtered inputs, attention forward/backward within tolerance on sampled
(instance, head) problems the oracle can afford."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_14183_b200 import binding as vd
from paper_2501_14183_b200 import inputs
from util import assert_attn_close, gap_filtered_windows

pytestmark = pytest.mark.gpu
SEED, STEP = 20250114, 5


def run_path(w, x, toks, vardrop=True):
    dev = [torch.from_numpy(t).cuda().to(torch.bfloat16) for t in toks]
    q, k, v, d_o = dev
    acfg = vd.AttnCfg(w.B, w.N, w.H, w.D, 0.0)
    aws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(acfg))
    o = torch.zeros_like(q)
    lse = torch.zeros((w.B, w.H, w.N), dtype=torch.float32, device="cuda")
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    sel = None
    if vardrop:
        hcfg = vd.HashCfg(w.B, w.N, w.L, w.k, 0, 0, 0)
        keys, freqs, _ = vd.alloc_hash_outputs(hcfg)
        hws = vd.alloc_ws(vd.vardrop_hash_workspace_bytes(hcfg))
        vd.vardrop_hash(torch.from_numpy(x).cuda(), hcfg, keys, freqs, None, hws)
        scfg = vd.SelectCfg(1, w.N, 0, w.rate, SEED, STEP)
        sel = vd.alloc_select_outputs(scfg)
        sws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(scfg))
        vd.vardrop_select(keys, scfg, sel["group_id"], sel["group_offsets"], sel["members"], sel["n_groups"], sel["sel_idx"],
                          sel["n_sel"], sel["inv_idx"], sws)
        vd.vardrop_attn_fwd(q, k, v, sel["sel_idx"], sel["n_sel"], acfg, o, lse, aws)
        vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, sel["sel_idx"], sel["n_sel"], sel["inv_idx"], acfg, dq, dk, dv, aws)
        torch.cuda.synchronize()
        assert vd.ws_status(hws) == vd.OK and vd.ws_status(sws) == vd.OK
        sel = {k_: v_.cpu().numpy() for k_, v_ in sel.items()}
        sel["keys"] = keys.cpu().numpy().view(np.uint64)
    else:
        vd.vardrop_attn_fwd(q, k, v, None, None, acfg, o, lse, aws)
        vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, None, None, None, acfg, dq, dk, dv, aws)
        torch.cuda.synchronize()
    assert vd.ws_status(aws) == vd.OK
    return dev, sel, o, lse, dq, dk, dv


def check_attention_samples(w, dev, idx, o, lse, dq, dk, dv, pairs):
    """Oracle on single (b, h) problems cut out of the batch."""
    Ns = w.N if idx is None else len(idx)
    for b, h in pairs:
        cut = [t[b:b + 1, :, h:h + 1].double().cpu().numpy() for t in dev]
        wo, wl = oracle.attn_fwd(cut[0], cut[1], cut[2], idx)
        assert_attn_close(o[b:b + 1, :Ns, h:h + 1].double().cpu().numpy(), wo, f"o[{b},{h}]")
        assert_attn_close(lse[b:b + 1, h:h + 1, :Ns].double().cpu().numpy(), wl, f"lse[{b},{h}]")
        wq, wk, wv = oracle.attn_bwd(cut[0], cut[1], cut[2], cut[3][:, :Ns], idx)
        assert_attn_close(dq[b:b + 1, :, h:h + 1].double().cpu().numpy(), wq, f"dq[{b},{h}]")
        assert_attn_close(dk[b:b + 1, :, h:h + 1].double().cpu().numpy(), wk, f"dk[{b},{h}]")
        assert_attn_close(dv[b:b + 1, :, h:h + 1].double().cpu().numpy(), wv, f"dv[{b},{h}]")


@pytest.mark.parametrize("name", ["tiny", "elec", "traffic", "long", "scale"])
def test_whole_path_on_workload(name):
    w = inputs.WORKLOADS[name]
    x, okeys, _, _, _ = gap_filtered_windows(inputs.make_windows(w), w.k)
    toks = inputs.make_tokens(w.B, w.N, w.H, w.D, w.qkv_std, seed=w.seed + 1)
    dev, sel, o, lse, dq, dk, dv = run_path(w, x, toks)
    assert np.array_equal(sel["keys"], okeys)
    want = oracle.select(okeys, 0, w.rate, SEED, STEP)
    for key in ("n_groups", "n_sel", "group_id", "group_offsets", "members", "sel_idx", "inv_idx"):
        assert np.array_equal(sel[key], want[key]), key
    n_sel = int(want["n_sel"][0])
    idx = want["sel_idx"][0, :n_sel]
    print(f"[{name}] groups={int(want['n_groups'][0])} kept={n_sel} of {w.N} (delta={1 - n_sel / w.N:.3f})")
    pairs = [(0, 0), (w.B - 1, w.H - 1), (w.B // 2, w.H // 2)] if name != "tiny" else [(b, h) for b in range(w.B) for h in range(w.H)]
    check_attention_samples(w, dev, idx, o, lse, dq, dk, dv, pairs)
    dropped = np.setdiff1d(np.arange(w.N), idx)
    for g in (dq, dk, dv):
        assert not g[:, torch.from_numpy(dropped).cuda()].any()               # exact zeros at every dropped variate


@pytest.mark.parametrize("name,pairs", [("traffic", [(0, 0), (31, 7)]), ("scale", [(3, 5)])])
def test_vardrop_off_full_attention(name, pairs):
    w = inputs.WORKLOADS[name]
    toks = inputs.make_tokens(w.B, w.N, w.H, w.D, w.qkv_std, seed=w.seed + 1)
    dev, _, o, lse, dq, dk, dv = run_path(w, None, toks, vardrop=False)
    check_attention_samples(w, dev, None, o, lse, dq, dk, dv, pairs)


def test_whole_path_per_instance_scope():
    """Every instance hashed, grouped and sampled on its own (hash scope 1, S = B selections) and attended with its own
    kept set: the algorithm of the paper run with batch size one per instance."""
    w = inputs.WORKLOADS["elec"]
    B = 6
    x, okeys, _, _, _ = gap_filtered_windows(inputs.make_windows(w, B=B), w.k, scope=1)
    toks = inputs.make_tokens(B, w.N, w.H, w.D, w.qkv_std, seed=5)
    dev = [torch.from_numpy(t).cuda().to(torch.bfloat16) for t in toks]
    q, k, v, d_o = dev
    hcfg = vd.HashCfg(B, w.N, w.L, w.k, 0, 0, 1)
    keys, freqs, _ = vd.alloc_hash_outputs(hcfg)
    hws = vd.alloc_ws(vd.vardrop_hash_workspace_bytes(hcfg))
    vd.vardrop_hash(torch.from_numpy(x).cuda(), hcfg, keys, freqs, None, hws)
    scfg = vd.SelectCfg(B, w.N, 0, w.rate, SEED, STEP)
    sel = vd.alloc_select_outputs(scfg)
    sws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(scfg))
    vd.vardrop_select(keys, scfg, sel["group_id"], sel["group_offsets"], sel["members"], sel["n_groups"], sel["sel_idx"], sel["n_sel"],
                      sel["inv_idx"], sws)
    acfg = vd.AttnCfg(B, w.N, w.H, w.D, 0.0, B)
    aws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(acfg))
    o = torch.zeros_like(q)
    lse = torch.zeros((B, w.H, w.N), dtype=torch.float32, device="cuda")
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    vd.vardrop_attn_fwd(q, k, v, sel["sel_idx"], sel["n_sel"], acfg, o, lse, aws)
    vd.vardrop_attn_bwd(q, k, v, o, lse, d_o, sel["sel_idx"], sel["n_sel"], sel["inv_idx"], acfg, dq, dk, dv, aws)
    torch.cuda.synchronize()
    assert vd.ws_status(hws) == vd.OK and vd.ws_status(aws) == vd.OK
    assert np.array_equal(keys.cpu().numpy().view(np.uint64), okeys)
    want = oracle.select(okeys, 0, w.rate, SEED, STEP)
    assert np.array_equal(sel["sel_idx"].cpu().numpy(), want["sel_idx"]) and np.array_equal(sel["n_sel"].cpu().numpy(), want["n_sel"])
    assert len(set(want["n_sel"].tolist())) > 1 or not np.array_equal(want["sel_idx"][0], want["sel_idx"][1])
    for b in (0, B - 1):
        c = int(want["n_sel"][b]); idx = want["sel_idx"][b, :c]
        cut = [t[b:b + 1].double().cpu().numpy() for t in dev]
        wo, _ = oracle.attn_fwd(cut[0], cut[1], cut[2], idx)
        assert_attn_close(o[b:b + 1, :c].double().cpu().numpy(), wo, f"o[{b}]")
        wq, wk, wv = oracle.attn_bwd(cut[0], cut[1], cut[2], cut[3][:, :c], idx)
        assert_attn_close(dq[b:b + 1].double().cpu().numpy(), wq, f"dq[{b}]")
        assert_attn_close(dk[b:b + 1].double().cpu().numpy(), wk, f"dk[{b}]")
        assert_attn_close(dv[b:b + 1].double().cpu().numpy(), wv, f"dv[{b}]")


@pytest.mark.parametrize("name", ["elec", "traffic"])
def test_back_to_back_steps_match_isolated_steps(name):
    """Steps queued without any synchronisation (kernels chained by programmatic dependent launches, shared workspaces and
    selection buffers reused from step to step) give bit for bit what the same steps give when the device is synchronised
    after every call."""
    import bench
    w = inputs.WORKLOADS[name]
    device = torch.device("cuda", 0)
    names = ("o", "lse", "dq", "dk", "dv")

    def run(sync_each_call):
        path = bench.Path(w, device, seed=w.seed, slots=3)
        for d in path.dev:
            for n in ("dq", "dk", "dv"):
                d[n].fill_(float("nan"))
        if sync_each_call:
            real = {}
            for fn in ("vardrop_hash", "vardrop_select", "vardrop_attn_fwd", "vardrop_attn_bwd"):
                real[fn] = getattr(vd, fn)

                def wrapped(*a, _f=real[fn]):
                    _f(*a)
                    torch.cuda.synchronize()
                setattr(vd, fn, wrapped)
        try:
            torch.cuda.synchronize()
            for s in range(3):
                path.step(s)
        finally:
            if sync_each_call:
                for fn, f in real.items():
                    setattr(vd, fn, f)
        torch.cuda.synchronize()
        path.check_status()
        return [{n: path.dev[s][n].clone() for n in names} for s in range(3)], int(path.sel["n_sel"].item())

    chained, kept = run(False)
    isolated, kept_i = run(True)
    assert kept == kept_i
    for s in range(3):
        for n in names:
            a, b = chained[s][n], isolated[s][n]
            if n == "o":
                a, b = a[:, :kept], b[:, :kept]
            elif n == "lse":
                a, b = a[:, :, :kept], b[:, :, :kept]
            if not torch.equal(a.view(torch.uint8), b.view(torch.uint8)):
                diff = (a.float() - b.float()).abs()
                diff = torch.nan_to_num(diff, nan=1e9)
                raise AssertionError(f"step {s} tensor {n}: {int((diff > 0).sum())} differing elements, max {float(diff.max()):.3e}, "
                                     f"first at {torch.nonzero(diff > 0)[0].tolist()}")


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """Failure handling without a fault: a warp waits 500 microseconds on a barrier nothing completes, through the bounded wait every
    kernel uses; the status word then reads TIMEOUT, and a normal call on the same stream with a fresh status word still works."""
    ws = vd.alloc_ws(4096)
    vd.vardrop_probe_bounded_wait(ws, 500)
    assert vd.vardrop_ws_status(ws) == vd.ERR_TIMEOUT
    vd.vardrop_probe_bounded_wait(ws, 200)                      # the word is sticky: still the first problem
    assert vd.vardrop_ws_status(ws) == vd.ERR_TIMEOUT
    w = inputs.WORKLOADS["tiny"]
    x = torch.from_numpy(inputs.make_windows(w)).cuda()
    hcfg = vd.HashCfg(w.B, w.N, w.L, w.k, 0, 0, 0)
    keys, freqs, _ = vd.alloc_hash_outputs(hcfg)
    hws = vd.alloc_ws(vd.vardrop_hash_workspace_bytes(hcfg))
    vd.vardrop_hash(x, hcfg, keys, freqs, None, hws)
    assert vd.vardrop_ws_status(hws) == vd.OK
    want, _, _ = oracle.hash(inputs.make_windows(w), w.k)
    assert np.array_equal(keys.cpu().numpy().view(np.uint64), want)
    with pytest.raises(vd.VardropError):
        vd.vardrop_probe_bounded_wait(ws, 0)


class Guarded:
    """Buffers cut out of larger allocations whose margins hold a known pattern: any write outside a buffer shows up in a margin."""
    MARGIN = 4096          # bytes on each side (a multiple of every alignment the library asks for)

    def __init__(self):
        self.items = []

    def alloc(self, shape, dtype, fill=0):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((n + 2 * self.MARGIN,), 0xA5, dtype=torch.uint8, device="cuda")
        view = raw[self.MARGIN: self.MARGIN + n].view(dtype).view(shape)
        view.fill_(fill)
        self.items.append((raw, n))
        return view

    def check(self):
        for raw, n in self.items:
            assert bool((raw[: self.MARGIN] == 0xA5).all()) and bool((raw[self.MARGIN + n:] == 0xA5).all()), "a margin was written"


@pytest.mark.parametrize("name,N", [("elec", None), ("traffic", None), ("scale", 2304)])
def test_no_write_outside_any_output_or_workspace(name, N):
    """Every output and every workspace of a whole step sits between guard margins: gathered, staged and many-tile launch shapes
    (the Scale shape cut to 2304 variates keeps the three-kernel selection and the four-warpgroup attention kernels in play)."""
    w = inputs.WORKLOADS[name]
    N = w.N if N is None else N
    B = min(w.B, 4)
    x = torch.from_numpy(inputs.make_windows(w, B=B, N=N)).cuda()
    toks = [torch.from_numpy(t).cuda().to(torch.bfloat16) for t in inputs.make_tokens(B, N, w.H, w.D, w.qkv_std, seed=9)]
    g = Guarded()
    hcfg = vd.HashCfg(B, N, w.L, w.k, 0, 0, 0)
    scfg = vd.SelectCfg(1, N, 0, w.rate, SEED, STEP)
    acfg = vd.AttnCfg(B, N, w.H, w.D, 0.0)
    keys = g.alloc((1, N), torch.int64)
    freqs = g.alloc((1, N, w.k), torch.int32)
    hws = g.alloc((vd.vardrop_hash_workspace_bytes(hcfg),), torch.uint8)
    sws = g.alloc((vd.vardrop_select_workspace_bytes(scfg),), torch.uint8)
    aws = g.alloc((vd.vardrop_attn_workspace_bytes(acfg),), torch.uint8)
    so = {n_: g.alloc(s_, torch.int32) for n_, s_ in (("group_id", (1, N)), ("group_offsets", (1, N + 1)), ("members", (1, N)), ("n_groups", (1,)),
                                                       ("sel_idx", (1, N)), ("n_sel", (1,)), ("inv_idx", (1, N)))}
    o, dq, dk, dv = (g.alloc((B, N, w.H, w.D), torch.bfloat16) for _ in range(4))
    lse = g.alloc((B, w.H, N), torch.float32)
    xs = g.alloc((B, N, w.L), torch.float32)
    vd.vardrop_hash(x, hcfg, keys, freqs, None, hws)
    vd.vardrop_select(keys, scfg, so["group_id"], so["group_offsets"], so["members"], so["n_groups"], so["sel_idx"], so["n_sel"], so["inv_idx"], sws)
    vd.vardrop_gather_rows(x, so["sel_idx"], so["n_sel"], vd.GatherCfg(B, N, w.L, 1), xs)
    vd.vardrop_attn_fwd(toks[0], toks[1], toks[2], so["sel_idx"], so["n_sel"], acfg, o, lse, aws)
    vd.vardrop_attn_bwd(toks[0], toks[1], toks[2], o, lse, toks[3], so["sel_idx"], so["n_sel"], so["inv_idx"], acfg, dq, dk, dv, aws)
    vd.vardrop_attn_fwd(toks[0], toks[1], toks[2], None, None, acfg, o, lse, aws)                      # and the all-token kernels
    vd.vardrop_attn_bwd(toks[0], toks[1], toks[2], o, lse, toks[3], None, None, None, acfg, dq, dk, dv, aws)
    torch.cuda.synchronize()
    for ws in (hws, sws, aws):
        assert vd.ws_status(ws) == vd.OK
    g.check()
