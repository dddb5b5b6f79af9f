#!/usr/bin/env python
"""Benchmark of the VarDrop hot path on B200.

One *step* = one pass of the whole path over one synthetic batch: vardrop_hash -> vardrop_select ->
vardrop_attn_fwd (gather + attention) -> vardrop_attn_bwd (+ scatter), all through the C ABI.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload elec|traffic|long|scale|tiny]
  python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...     (N > 1: one rank per GPU)
  python bench.py --impl reference ...     (the CPU oracle, as it stands, on the host cores)

Rank 0 prints ONE JSON line.  `value` is variate tokens per second (B * N per step) of the whole job with inputs
resident in HBM; `e2e` is the same with host buffers and the copies inside the timed region; `roofline` describes
the kernel with the largest share of the step; `cpu_baseline` is the oracle timed on this machine's cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "variate_tokens_per_s"
UNIT = "tokens/s"
SEED, STEP0 = 20250114, 1
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        peaks = dict(FALLBACK_PEAKS)
        peaks.update({k: float(d[k]) for k in FALLBACK_PEAKS if k in d})
        return peaks, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------------------
# clocks: nvidia-smi sampled during the timed region
# ------------------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.file:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            # the busiest half of the samples is the load: the region is short next to the sampling period
            busy = sorted(sm)[len(sm) // 2:]
            out.update(sm_mhz=float(np.median(busy)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------------------------
# the GPU arm
# ------------------------------------------------------------------------------------------------------------
class Path:
    """Device buffers and the four C-ABI calls of one step; `slots` rotating input/output sets keep the working set
    larger than L2 so that every step reads its inputs from HBM."""

    def __init__(self, w, device, seed, slots):
        import torch
        from paper_2501_14183_b200 import binding as vd
        from paper_2501_14183_b200 import inputs
        self.torch, self.vd, self.w = torch, vd, w
        self.hcfg = vd.HashCfg(w.B, w.N, w.L, w.k, 0, 0, 0)
        self.scfg = vd.SelectCfg(1, w.N, 0, w.rate, SEED, STEP0)
        self.acfg = vd.AttnCfg(w.B, w.N, w.H, w.D, 0.0)
        bf = dict(dtype=torch.bfloat16, device=device)
        self.host, self.dev = [], []
        x = inputs.make_windows(w, seed=seed)
        toks = inputs.make_tokens(w.B, w.N, w.H, w.D, w.qkv_std, seed=seed + 1)
        for s in range(slots):
            hx = torch.from_numpy(np.roll(x, s, axis=0).copy()).pin_memory()            # same variates, instances rotated
            ht = [torch.from_numpy(np.roll(t, s, axis=0).copy()).to(torch.bfloat16).pin_memory() for t in toks]
            self.host.append((hx, ht))
            d = dict(x=hx.to(device), q=ht[0].to(device), k=ht[1].to(device), v=ht[2].to(device), d_o=ht[3].to(device),
                     o=torch.zeros((w.B, w.N, w.H, w.D), **bf), lse=torch.zeros((w.B, w.H, w.N), dtype=torch.float32, device=device),
                     dq=torch.empty((w.B, w.N, w.H, w.D), **bf), dk=torch.empty((w.B, w.N, w.H, w.D), **bf),
                     dv=torch.empty((w.B, w.N, w.H, w.D), **bf))
            self.dev.append(d)
        self.keys, self.freqs, _ = vd.alloc_hash_outputs(self.hcfg, device=device)
        self.sel = vd.alloc_select_outputs(self.scfg, device=device)
        self.hws = vd.alloc_ws(vd.vardrop_hash_workspace_bytes(self.hcfg), device)
        self.sws = vd.alloc_ws(vd.vardrop_select_workspace_bytes(self.scfg), device)
        self.aws = vd.alloc_ws(vd.vardrop_attn_workspace_bytes(self.acfg), device)
        self.host_out = [torch.empty((w.B, w.N, w.H, w.D), dtype=torch.bfloat16).pin_memory() for _ in range(4)]
        self.host_sel = torch.empty((w.N + 1,), dtype=torch.int32).pin_memory()
        self.step_no = 0

    def input_bytes(self):
        w = self.w
        return w.B * w.N * w.L * 4 + 4 * w.B * w.N * w.H * w.D * 2

    def output_bytes(self):
        w = self.w
        return 4 * w.B * w.N * w.H * w.D * 2 + (w.N + 1) * 4

    def step(self, slot, vardrop=True):
        vd, d, s = self.vd, self.dev[slot], self.sel
        self.scfg.step = STEP0 + self.step_no
        self.step_no += 1
        if vardrop:
            vd.vardrop_hash(d["x"], self.hcfg, self.keys, self.freqs, None, self.hws)
            vd.vardrop_select(self.keys, self.scfg, s["group_id"], s["group_offsets"], s["members"], s["n_groups"], s["sel_idx"],
                              s["n_sel"], s["inv_idx"], self.sws)
            sel, nsel, inv = s["sel_idx"], s["n_sel"], s["inv_idx"]
        else:
            sel = nsel = inv = None
        vd.vardrop_attn_fwd(d["q"], d["k"], d["v"], sel, nsel, self.acfg, d["o"], d["lse"], self.aws)
        vd.vardrop_attn_bwd(d["q"], d["k"], d["v"], d["o"], d["lse"], d["d_o"], sel, nsel, inv, self.acfg, d["dq"], d["dk"], d["dv"],
                            self.aws)

    def step_e2e(self, slot):
        """Same step with host buffers: inputs copied from pinned host memory, outputs copied back."""
        d = self.dev[slot]
        hx, ht = self.host[slot]
        d["x"].copy_(hx, non_blocking=True)
        for name, t in zip(("q", "k", "v", "d_o"), ht):
            d[name].copy_(t, non_blocking=True)
        self.step(slot)
        for h, name in zip(self.host_out, ("o", "dq", "dk", "dv")):
            h.copy_(d[name], non_blocking=True)
        self.host_sel[: self.w.N].copy_(self.sel["sel_idx"][0], non_blocking=True)
        self.host_sel[self.w.N:].copy_(self.sel["n_sel"], non_blocking=True)

    def check_status(self):
        for ws in (self.hws, self.sws, self.aws):
            st = self.vd.ws_status(ws)
            if st != self.vd.OK:
                raise RuntimeError(f"device status {st} after the timed region")


def time_region(torch, fn, steps, dist_barrier):
    """K calls of fn(i) between two CUDA events, a barrier + synchronize on both sides; milliseconds."""
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist_barrier()
    torch.cuda.synchronize()
    start.record()
    t0 = time.perf_counter()
    for i in range(steps):
        fn(i)
    time_region.host_ms = (time.perf_counter() - t0) * 1e3          # host time spent issuing the K steps
    stop.record()
    torch.cuda.synchronize()
    dist_barrier()
    return start.elapsed_time(stop)


def recorded_traffic(kernel, workload):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, or None when there is no capture for this
    workload or the kernel's source file has changed since the capture."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        rec = json.load(fh).get(kernel)
    if not rec or rec.get("workload") != workload:
        return None
    src = os.path.join(ROOT, "paper_2501_14183_b200", "csrc", rec["source_file"])
    with open(src, "rb") as fh:
        if hashlib.sha256(fh.read()).hexdigest() != rec["source_sha256"]:
            return None
    return rec["dram_bytes_per_launch"]


def kernel_work(w, n_sel, selected=True):
    """Algorithmic work of one launch of each kernel (what the method must move or compute): (bytes, flops).
    flops is None for the kernels that only move data."""
    row = w.H * w.D * 2
    kept = w.B * n_sel
    full = w.B * w.N
    grads = 3 * (full if selected else kept) * row                  # dq, dk, dv come back in the full layout
    return {
        "hash_kernel": (w.B * w.N * w.L * 4 + w.N * (8 + 4 * w.k), None),
        "select_small_kernel": (w.N * (8 + 6 * 4), None),
        "select_count_kernel": (w.N * (8 + 4 * 4), None),
        "select_group_kernel": (w.N * 6 * 4, None),
        "select_sample_kernel": (w.N * 4 * 4, None),
        "gather_kernel": (2 * 3 * kept * row, None),
        "attn_fwd_kernel": (3 * kept * row + kept * row + kept * w.H * 4, 4.0 * w.B * w.H * n_sel * n_sel * w.D),
        "bwd_prep_kernel": (2 * kept * row + kept * row + kept * w.H * 64 * 4, None),
        "attn_bwd_kernel": (5 * kept * row + kept * w.H * 4 + grads, 10.0 * w.B * w.H * n_sel * n_sel * w.D),
        "bwd_convert_kernel": (kept * row + kept * w.H * 64 * 4, None),
    }


def kernel_table(per_kernel, work, peaks):
    """Per kernel: launches, average duration, share of the step, and the roofline that binds it.  A kernel with both
    bytes and flops is bound by whichever needs longer at the measured peak (attention over a few hundred kept tokens
    moves more bytes, relative to the HBM peak, than it computes relative to the tensor peak)."""
    kernels = {}
    total_ms = sum(v[0] for v in per_kernel.values()) or 1.0
    for name, (tot, n) in per_kernel.items():
        if n == 0:
            continue
        nbytes, flops = work[name]
        avg_s = tot / n * 1e-3
        t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
        t_tensor = flops / (peaks["bf16_tflops"] * 1e12) if flops else 0.0
        if t_tensor > t_hbm:
            bound, ach, peak, unit = "tensor", flops / avg_s / 1e12, peaks["bf16_tflops"], "TFLOP/s"
        else:
            bound, ach, peak, unit = "hbm", nbytes / avg_s / 1e9, peaks["hbm_gbs"], "GB/s"
        kernels[name] = {"launches": n, "avg_us": tot / n * 1e3, "share": tot / total_ms, "bound": bound,
                         "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                         "algorithmic_bytes": nbytes, "algorithmic_flops": flops}
    return kernels


def pearson_leg(torch, vd, path, w, peaks, barrier, args):
    """Times vardrop_pearson_max (maximum Pearson correlation per variate, Appendix A / Eq. 4) on the workload's windows and, unless
    --no-cpu, the oracle on one instance.  Algorithmic work: 2 B N^2 L flop (every pair once per direction)."""
    import oracle
    device = path.dev[0]["x"].device
    cfg = vd.PearsonCfg(w.B, w.N, w.L, 0.9)
    out = torch.empty((w.B, w.N), dtype=torch.float32, device=device)
    above = torch.empty((w.B,), dtype=torch.int32, device=device)
    ws = vd.alloc_ws(vd.vardrop_pearson_workspace_bytes(cfg), device)
    slots = len(path.dev)
    k = max(3, min(args.steps, 20))
    for i in range(3):
        vd.vardrop_pearson_max(path.dev[i % slots]["x"], cfg, out, above, ws)
    vd.vardrop_profile_enable(True)
    ms = time_region(torch, lambda i: vd.vardrop_pearson_max(path.dev[i % slots]["x"], cfg, out, above, ws), k, barrier)
    per = vd.vardrop_profile_read()
    vd.vardrop_profile_enable(False)
    if vd.ws_status(ws) != vd.OK:
        raise RuntimeError("device status set by vardrop_pearson_max")
    flops = 2.0 * w.B * float(w.N) ** 2 * w.L
    t_max = per["pearson_max_kernel"][0] / k * 1e-3
    res = {"ms_per_call": ms / k, "normalize_us": per["pearson_normalize_kernel"][0] / k * 1e3, "max_kernel_us": t_max * 1e6,
           "algorithmic_flops": flops, "tflops": flops / t_max / 1e12, "frac_of_bf16_peak": flops / t_max / 1e12 / peaks["bf16_tflops"],
           "share_above_0.9": float(above.float().mean().item()) / w.N, "note": "timed with the per-kernel event timer armed"}
    if not args.no_cpu:
        x1 = path.host[0][0][:1].numpy()
        t0 = time.perf_counter()
        oracle.pearson_max(x1)
        res["oracle_ms_per_instance"] = (time.perf_counter() - t0) * 1e3
        res["oracle_cores"] = oracle.num_threads()
    return res


def run_gpu(args):
    import torch
    from paper_2501_14183_b200 import binding as vd
    from paper_2501_14183_b200 import dist_util, inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()

    vd.load()                                  # fails loudly when the CUDA library is missing
    w = inputs.WORKLOADS[args.workload]
    peaks, peak_kind = load_peaks()
    set_bytes = w.B * w.N * w.L * 4 + 9 * w.B * w.N * w.H * w.D * 2
    slots = max(2, min(16, -(-512 * 2 ** 20 // set_bytes)))          # rotate through >= 512 MB (L2 is 126 MB)
    path = Path(w, device, seed=dist_util.rank_seed(w.seed, rank), slots=slots)

    for i in range(args.warmup):
        path.step(i % slots)
    torch.cuda.synchronize()
    path.check_status()
    n_sel = int(path.sel["n_sel"].item())
    n_groups = int(path.sel["n_groups"].item())

    # ---- timed region: K whole steps, device resident ---------------------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = vd.vardrop_launch_count()
    ms = time_region(torch, lambda i: path.step(i % slots), args.steps, barrier)
    host_ms = time_region.host_ms
    launches = vd.vardrop_launch_count() - launches0
    # ---- same K steps with the per-kernel event timer armed (durations for the roofline) ----------------------
    vd.vardrop_profile_enable(True)
    ms_armed = time_region(torch, lambda i: path.step(i % slots), args.steps, barrier)
    per_kernel = vd.vardrop_profile_read()
    vd.vardrop_profile_enable(False)
    # ---- end to end: host buffers, copies inside the timed region ----------------------------------------------
    for i in range(2):
        path.step_e2e(i % slots)
    ms_e2e = time_region(torch, lambda i: path.step_e2e(i % slots), args.steps, barrier)
    # ---- VarDrop off: the same attention kernels on all N tokens ---------------------------------------------
    off = None
    if not args.no_off:
        for i in range(3):
            path.step(i % slots, vardrop=False)
        k_off = max(3, min(args.steps, 20))
        vd.vardrop_profile_enable(True)
        ms_off = time_region(torch, lambda i: path.step(i % slots, vardrop=False), k_off, barrier)
        pk_off = vd.vardrop_profile_read()
        vd.vardrop_profile_enable(False)
        fl = 14.0 * w.B * w.H * float(w.N) ** 2 * w.D
        t_attn = (pk_off["attn_fwd_kernel"][0] + pk_off["attn_bwd_kernel"][0]) / k_off * 1e-3
        off = {"ms_per_step": ms_off / k_off, "tokens_per_s": w.tokens / (ms_off / k_off * 1e-3), "n_tokens": w.N,
               "attn_fwd_ms": pk_off["attn_fwd_kernel"][0] / k_off, "attn_bwd_ms": pk_off["attn_bwd_kernel"][0] / k_off,
               "attn_tflops": fl / t_attn / 1e12, "attn_frac_of_bf16_peak": fl / t_attn / 1e12 / peaks["bf16_tflops"],
               "kernels": kernel_table(pk_off, kernel_work(w, w.N, selected=False), peaks),
               "note": "timed with the per-kernel event timer armed"}
    pearson = pearson_leg(torch, vd, path, w, peaks, barrier, args) if args.pearson else None
    clocks = sampler.stop() if rank == 0 else None
    path.check_status()

    ms, ms_e2e = dist_util.max_over_ranks([ms, ms_e2e], dist, device)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    tokens = w.tokens * world
    kernels = kernel_table(per_kernel, kernel_work(w, n_sel), peaks)
    top = max(kernels, key=lambda k: kernels[k]["share"])
    roofline = {"kernel": top, "bound": kernels[top]["bound"], "achieved": kernels[top]["achieved"], "peak": kernels[top]["peak"],
                "unit": kernels[top]["unit"], "frac": kernels[top]["frac"], "traffic": recorded_traffic(top, w.name),
                "peak_source": f"{peak_kind} (burst figure for tensor work)",
                "timing": "CUDA events around every launch, second pass of the same K steps",
                "ms_per_step_with_timer_armed": ms_armed / args.steps}

    cpu = None if args.no_cpu else cpu_baseline(w, reps=2)
    line = {
        "metric": METRIC, "value": dist_util.aggregate_throughput(w.tokens, world, ms / args.steps * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "host_issue_ms_per_step": host_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 attention (fp32 accumulate), fp32 FFT, integer grouping", "data": "synthetic",
        "config": {"workload": f"{w.name}: B={w.B} N={w.N} L={w.L} k={w.k} rate={w.rate} H={w.H} D={w.D}",
                   "kept_tokens": n_sel, "groups": n_groups, "delta": 1.0 - n_sel / w.N,
                   "l2": f"inputs and outputs rotate through {slots} sets ({slots * set_bytes / 2 ** 20:.0f} MiB > 126 MiB L2)",
                   "parallelism": f"dp{world} (independent batches per rank, no collective)"},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": tokens / (ms_e2e / args.steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": path.input_bytes(),
                "d2h_bytes_per_step": path.output_bytes(), "ms_per_step": ms_e2e / args.steps},
        "roofline": roofline, "kernels": kernels, "vardrop_off": off, "cpu_baseline": cpu,
    }
    if pearson is not None:
        line["pearson"] = pearson
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------------------
# the oracle on the host cores (CPU baseline and the `--impl reference` arm)
# ------------------------------------------------------------------------------------------------------------
def oracle_plan(w, seconds_per_step):
    """How many instances the oracle's DFT and attention legs take per step so that a step costs about
    `seconds_per_step` on this machine (assuming ~0.4 GFLOP/s per core for its plain fp64 loops); both legs are
    scaled back to the whole batch."""
    import oracle
    rate = 0.4e9 * max(1, oracle.num_threads())
    budget = rate * seconds_per_step / 2.0                      # flop per leg
    lo, hi = oracle.default_band(w.L)
    hash_per_b = 4.0 * w.N * (hi - lo) * w.L
    n_kept = max(1.0, w.N * w.rate * 1.5)
    attn_per_b = 20.0 * w.H * n_kept * n_kept * w.D
    bh = int(max(1, min(w.B, budget // hash_per_b)))
    bs = int(max(1, min(w.B, budget // attn_per_b)))
    return bh, bs


def oracle_step(w, x, toks, step, plan):
    """One pass of the path by the oracle on a bounded sample: k-DFH over the first `bh` instances, grouping and
    sampling on all N variates, attention forward and backward on the first `bs` instances.  Returns seconds scaled
    to the whole batch."""
    import oracle
    bh, bs = plan
    t0 = time.perf_counter()
    keys, _, _ = oracle.hash(x[:bh], w.k)
    t1 = time.perf_counter()
    sel = oracle.select(keys, 0, w.rate, SEED, step)
    n_sel = int(sel["n_sel"][0])
    idx = sel["sel_idx"][0, :n_sel]
    t2 = time.perf_counter()
    q, k, v, d_o = (t[:bs] for t in toks)
    oracle.attn_fwd(q, k, v, idx)
    oracle.attn_bwd(q, k, v, d_o[:, :n_sel], idx)
    t3 = time.perf_counter()
    return (t1 - t0) * (w.B / bh) + (t2 - t1) + (t3 - t2) * (w.B / bs)


def oracle_inputs(w):
    from paper_2501_14183_b200 import inputs
    import torch
    x = inputs.make_windows(w)
    toks = [torch.from_numpy(t).to(torch.bfloat16).double().numpy() for t in inputs.make_tokens(w.B, w.N, w.H, w.D, w.qkv_std, seed=w.seed + 1)]
    return x, toks


def sample_text(w, plan):
    return (f"k-DFH on {plan[0]} of {w.B} instances and fp64 attention fwd+bwd on {plan[1]} of {w.B} instances, each scaled to "
            f"the batch; grouping and sampling on all {w.N} variates")


def cpu_baseline(w, reps):
    import oracle
    x, toks = oracle_inputs(w)
    plan = oracle_plan(w, seconds_per_step=5.0)
    oracle_step(w, x, toks, 0, plan)
    secs = [oracle_step(w, x, toks, 1 + r, plan) for r in range(reps)]
    s = float(np.mean(secs))
    return {"value": w.tokens / s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": sample_text(w, plan) + f"; mean of {reps} passes", "seconds_per_step": s}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2501_14183_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    x, toks = oracle_inputs(w)
    plan = oracle_plan(w, seconds_per_step=min(5.0, 100.0 / (args.steps + args.warmup)))
    for i in range(args.warmup):
        oracle_step(w, x, toks, i, plan)
    secs = [oracle_step(w, x, toks, args.warmup + i, plan) for i in range(args.steps)]
    s = float(np.mean(secs))
    value = w.tokens / s
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: B={w.B} N={w.N} L={w.L} k={w.k} rate={w.rate} H={w.H} D={w.D}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample_text(w, plan)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="elec", choices=["tiny", "elec", "traffic", "long", "scale"])
    ap.add_argument("--impl", default="vardrop", choices=["vardrop", "reference"])
    ap.add_argument("--no-off", action="store_true", help="skip the VarDrop-off comparison pass")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU baseline (profiling runs)")
    ap.add_argument("--pearson", action="store_true", help="also time the variate-redundancy check (Appendix A, Eq. 4) on the workload's windows")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
