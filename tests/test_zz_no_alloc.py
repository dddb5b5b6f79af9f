"""vardrop_select_static: the variant of vardrop_select for callers that cannot allocate device memory (code running
under a locked or exhausted framework allocator, plug-ins that only receive input and output buffers).  Its scratch
is a fixed array inside the library, so the test checks two things a user relies on: it gives exactly the answers of
vardrop_select, and a second call right after the first is not disturbed by what the first left in that array.
Collected last on purpose (file name), so a failure here cannot hide another test's result."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_14183_b200 import binding as vd
from paper_2501_14183_b200 import inputs

pytestmark = pytest.mark.gpu

NAMES = ("group_id", "group_offsets", "members", "n_groups", "sel_idx", "n_sel", "inv_idx")


def with_workspace(keys_t, cfg):
    out = vd.alloc_select_outputs(cfg)
    ws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(cfg))
    vd.vardrop_select(keys_t, cfg, *(out[n] for n in NAMES), ws)
    return out


def without_workspace(keys_t, cfg, out):
    vd.vardrop_select_static(keys_t, cfg, *(out[n] for n in NAMES))


def test_static_variant_matches_on_two_calls_in_a_row():
    # two different problems back to back on one stream: a large one, then a smaller one with other groups, so stale
    # counters or ranks from the first call would show up in the second
    cases = [(inputs.make_keys(8192, 512, k=4, f_hi=85, seed=1), vd.SelectCfg(1, 8192, 0, 0.1, 99, 7)),
             (inputs.make_keys(862, 60, k=3, f_hi=25, seed=2), vd.SelectCfg(1, 862, 10, 1.0, 5, 8))]
    keys_t = [torch.from_numpy(k.reshape(1, -1).view(np.int64)).cuda() for k, _ in cases]
    outs = [vd.alloc_select_outputs(cfg) for _, cfg in cases]          # outputs are the caller's: allocated up front
    torch.cuda.synchronize()
    torch_before = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    for kt, (_, cfg), out in zip(keys_t, cases, outs):
        without_workspace(kt, cfg, out)                                # the two calls in a row, nothing in between
    torch.cuda.synchronize()
    # the point of the variant: no device memory was obtained anywhere, neither through torch's allocator nor behind its back
    assert torch.cuda.memory_allocated() == torch_before
    assert torch.cuda.mem_get_info()[0] == free_before
    for kt, (keys, cfg), out in zip(keys_t, cases, outs):
        want = with_workspace(kt, cfg)
        torch.cuda.synchronize()
        for name in NAMES:
            assert torch.equal(out[name], want[name]), name              # integer work: bit-exact
        ref = oracle.select(keys.reshape(1, -1), cfg.gs, cfg.rate, cfg.seed, cfg.step)       # and pinned to the oracle, not only to its sibling
        for name in NAMES:
            assert np.array_equal(out[name].cpu().numpy(), ref[name]), name


def test_static_variant_repeats_and_handles_several_hash_rows():
    rows = np.stack([inputs.make_keys(500, 20 + s, k=3, f_hi=25, seed=s) for s in range(4)])
    kt = torch.from_numpy(rows.view(np.int64)).cuda()
    cfg = vd.SelectCfg(4, 500, 5, 1.0, 77, 3)
    a, b = vd.alloc_select_outputs(cfg), vd.alloc_select_outputs(cfg)
    without_workspace(kt, cfg, a)
    without_workspace(kt, cfg, b)
    want = with_workspace(kt, cfg)
    torch.cuda.synchronize()
    for name in NAMES:
        assert torch.equal(a[name], want[name]) and torch.equal(b[name], want[name]), name


def test_static_variant_rejects_sizes_beyond_its_scratch():
    cfg = vd.SelectCfg(1, 16385, 0, 0.5, 1, 0)
    out = vd.alloc_select_outputs(cfg)
    kt = torch.zeros((1, 16385), dtype=torch.int64, device="cuda")
    with pytest.raises(vd.VardropError) as e:
        without_workspace(kt, cfg, out)
    assert e.value.status == vd.ERR_UNSUPPORTED and "16384" in str(e.value)
    cfg = vd.SelectCfg(2, 8192, 0, 0.5, 1, 0)                            # exactly at the limit is accepted
    out = vd.alloc_select_outputs(cfg)
    kt = torch.from_numpy(np.stack([inputs.make_keys(8192, 100, k=3, f_hi=25, seed=s) for s in (3, 4)]).view(np.int64)).cuda()
    without_workspace(kt, cfg, out)
    want = with_workspace(kt, cfg)
    torch.cuda.synchronize()
    for name in NAMES:
        assert torch.equal(out[name], want[name]), name
