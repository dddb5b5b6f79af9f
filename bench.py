#!/usr/bin/env python
"""Benchmark of the VarDrop hot path on B200.

One *step* = one pass of the whole path over one synthetic batch: vardrop_hash -> vardrop_select ->
vardrop_attn_fwd (gather + attention) -> vardrop_attn_bwd (+ scatter), all through the C ABI.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload scale|traffic|long|elec|tiny]   (default: scale)
  python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...     (N > 1: one rank per GPU)
  python bench.py --impl reference ...     (the CPU oracle, as it stands, on the host cores)

Rank 0 prints ONE JSON line.  `value` is variate tokens per second (B * N per step) of the whole job with inputs
resident in HBM; `e2e` is the same with host buffers and the copies inside the timed region; `roofline` describes
the kernel with the largest share of the step; `targets` holds the all-token N = 862 attention and the k-DFH / selection /
gather fractions from a short Traffic-shaped pass; `cpu_baseline` is the oracle timed on this machine's cores.
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

    def __init__(self, w, device, seed, slots, host_slots=2):
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
            hx = torch.from_numpy(np.roll(x, s, axis=0).copy())                         # same variates, instances rotated
            ht = [torch.from_numpy(np.roll(t, s, axis=0).copy()).to(torch.bfloat16) for t in toks]
            if s < host_slots:                                                          # pinned copies for the end-to-end leg
                hx, ht = hx.pin_memory(), [t.pin_memory() for t in ht]
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
        self.step_no = 0

    def host_x(self, slot):
        """The windows of device slot `slot` as a numpy array (slot s holds the batch rotated by s instances)."""
        return self.dev[slot]["x"].cpu().numpy()

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

    def e2e_setup(self):
        """Streams, events and host buffers of the pipelined end-to-end step: input copies of step i + 1 and output copies of
        step i - 1 run on their own streams beside the kernels of step i (PCIe is full duplex), two device slots and two
        host output sets in rotation."""
        t, w = self.torch, self.w
        self.s_in, self.s_out = t.cuda.Stream(), t.cuda.Stream()
        mk = lambda: [t.cuda.Event() for _ in range(2)]
        self.ev_in, self.ev_comp, self.ev_out = mk(), mk(), mk()
        cur = t.cuda.current_stream()
        for e in self.ev_in + self.ev_comp + self.ev_out:
            e.record(cur)
        self.host_out = [[t.empty((w.B, w.N, w.H, w.D), dtype=t.bfloat16).pin_memory() for _ in range(4)] for _ in range(2)]
        self.host_sel = [t.empty((w.N + 1,), dtype=t.int32).pin_memory() for _ in range(2)]

    def e2e_begin(self):
        t = self.torch
        ev = t.cuda.Event()
        ev.record()
        self.s_in.wait_event(ev)
        self.s_out.wait_event(ev)

    def e2e_drain(self):
        cur = self.torch.cuda.current_stream()
        for e in self.ev_out:
            cur.wait_event(e)

    def step_e2e(self, i):
        """Same step with host buffers: every step copies its inputs from pinned host memory and its outputs back, the
        copies of neighbouring steps overlapping this step's kernels (one cudaMemcpyAsync per tensor)."""
        t = self.torch
        slot = i % 2
        d = self.dev[slot]
        hx, ht = self.host[slot]
        cur = t.cuda.current_stream()
        with t.cuda.stream(self.s_in):
            self.s_in.wait_event(self.ev_comp[slot])        # the step that last read this slot's inputs is done
            d["x"].copy_(hx, non_blocking=True)
            for name, src in zip(("q", "k", "v", "d_o"), ht):
                d[name].copy_(src, non_blocking=True)
            self.ev_in[slot].record(self.s_in)
        cur.wait_event(self.ev_in[slot])
        cur.wait_event(self.ev_out[slot])                   # this slot's previous outputs have left the device
        self.step(slot)
        hs = self.host_sel[slot]
        hs[: self.w.N].copy_(self.sel["sel_idx"][0], non_blocking=True)     # the selection buffers are shared by the slots:
        hs[self.w.N:].copy_(self.sel["n_sel"], non_blocking=True)           # copied in stream order, before the next step
        self.ev_comp[slot].record(cur)
        with t.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_comp[slot])
            for h, name in zip(self.host_out[slot], ("o", "dq", "dk", "dv")):
                h.copy_(d[name], non_blocking=True)
            self.ev_out[slot].record(self.s_out)

    def check_status(self):
        for ws in (self.hws, self.sws, self.aws):
            st = self.vd.vardrop_ws_status(ws)
            if st != self.vd.OK:
                raise RuntimeError(f"device status {st} after the timed region")


MIN_REGION_S = 0.3          # a timed region is repeated until it has lasted this long
MIN_INTERVALS = 50          # and has produced at least this many event intervals


def time_region(torch, fn, steps, dist_barrier, min_seconds=None, min_intervals=None, begin=None, drain=None):
    """Times calls of fn(i) with CUDA events on the launching stream.

    One pass is exactly `steps` calls between a barrier + synchronize on both sides, with an event after every block of
    steps (a block is one step when steps <= 64).  Passes are repeated until the accumulated device time reaches
    `min_seconds` and at least `min_intervals` block intervals exist.  Returns a dict: `median` and `mean` milliseconds
    per step (median over the block intervals, mean over whole passes), `intervals`, `passes`, `total_ms`, and
    `host_ms_per_step` (host time spent issuing the calls).  `begin()` runs right after the first event of a pass and
    `drain()` right before its last one (used by the pipelined end-to-end step to tie its copy streams to the events)."""
    min_seconds = MIN_REGION_S if min_seconds is None else min(min_seconds, MIN_REGION_S)
    min_intervals = MIN_INTERVALS if min_intervals is None else min(min_intervals, MIN_INTERVALS)
    block = max(1, steps // 64)
    per_step, pass_ms, host_s, passes, i_global = [], [], 0.0, 0, 0
    while True:
        marks = [torch.cuda.Event(enable_timing=True)]
        sizes = []
        dist_barrier()
        torch.cuda.synchronize()
        marks[0].record()
        if begin is not None:
            begin()
        t0 = time.perf_counter()
        done = 0
        while done < steps:
            n = min(block, steps - done)
            for _ in range(n):
                fn(i_global)
                i_global += 1
            done += n
            if drain is not None and done == steps:
                drain()
            ev = torch.cuda.Event(enable_timing=True)
            ev.record()
            marks.append(ev)
            sizes.append(n)
        host_s += time.perf_counter() - t0
        torch.cuda.synchronize()
        dist_barrier()
        for a, b, n in zip(marks[:-1], marks[1:], sizes):
            per_step.append(a.elapsed_time(b) / n)
        pass_ms.append(marks[0].elapsed_time(marks[-1]))
        passes += 1
        if (sum(pass_ms) >= min_seconds * 1e3 and len(per_step) >= min_intervals) or passes >= 2000:
            break
    return {"median": float(np.median(per_step)), "mean": float(sum(pass_ms) / (passes * steps)), "intervals": len(per_step),
            "passes": passes, "total_ms": float(sum(pass_ms)), "host_ms_per_step": host_s * 1e3 / (passes * steps)}


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
    t = time_region(torch, lambda i: vd.vardrop_pearson_max(path.dev[i % slots]["x"], cfg, out, above, ws), k, barrier)
    per = vd.vardrop_profile_read()
    vd.vardrop_profile_enable(False)
    if vd.vardrop_ws_status(ws) != vd.OK:
        raise RuntimeError("device status set by vardrop_pearson_max")
    flops = 2.0 * w.B * float(w.N) ** 2 * w.L
    t_max = per["pearson_max_kernel"][0] / per["pearson_max_kernel"][1] * 1e-3
    res = {"ms_per_call": t["median"], "normalize_us": per["pearson_normalize_kernel"][0] / per["pearson_normalize_kernel"][1] * 1e3,
           "max_kernel_us": t_max * 1e6,
           "algorithmic_flops": flops, "tflops": flops / t_max / 1e12, "frac_of_bf16_peak": flops / t_max / 1e12 / peaks["bf16_tflops"],
           "share_above_0.9": float(above.float().mean().item()) / w.N, "note": "timed with the per-kernel event timer armed"}
    if not args.no_cpu:
        import oracle
        x1 = path.host[0][0][:1].numpy()
        t0 = time.perf_counter()
        oracle.pearson_max(x1)
        res["oracle_ms_per_instance"] = (time.perf_counter() - t0) * 1e3
        res["oracle_cores"] = oracle.num_threads()
    return res


def per_launch(per_kernel):
    """{kernel: (total ms, launches)} -> the same with zero-launch kernels dropped."""
    return {k: v for k, v in per_kernel.items() if v[1] > 0}


def measure_off(torch, vd, path, w, peaks, barrier, steps):
    """VarDrop off: the same attention kernels on all N tokens (the paper's inference / ground configuration), timed with
    the per-kernel event timer armed."""
    slots = len(path.dev)
    for i in range(3):
        path.step(i % slots, vardrop=False)
    vd.vardrop_profile_enable(True)
    t = time_region(torch, lambda i: path.step(i % slots, vardrop=False), steps, barrier, min_seconds=0.15, min_intervals=20)
    pk = per_launch(vd.vardrop_profile_read())
    vd.vardrop_profile_enable(False)
    fwd_ms = pk["attn_fwd_kernel"][0] / pk["attn_fwd_kernel"][1]
    bwd_ms = pk["attn_bwd_kernel"][0] / pk["attn_bwd_kernel"][1]
    fl_f, fl_b = 4.0 * w.B * w.H * float(w.N) ** 2 * w.D, 10.0 * w.B * w.H * float(w.N) ** 2 * w.D
    tf = (fl_f + fl_b) / ((fwd_ms + bwd_ms) * 1e-3) / 1e12
    return {"ms_per_step": t["median"], "tokens_per_s": w.tokens / (t["median"] * 1e-3), "n_tokens": w.N,
            "attn_fwd_ms": fwd_ms, "attn_bwd_ms": bwd_ms,
            "attn_fwd_tflops": fl_f / (fwd_ms * 1e-3) / 1e12, "attn_bwd_tflops": fl_b / (bwd_ms * 1e-3) / 1e12,
            "attn_tflops": tf, "attn_frac_of_bf16_peak": tf / peaks["bf16_tflops"],
            "attn_frac_of_bf16_sustained_peak": tf / peaks["bf16_tflops_sustained"],
            "kernels": kernel_table(pk, kernel_work(w, w.N, selected=False), peaks),
            "note": "attention kernels timed by CUDA events around every launch (timer armed)"}


def traffic_targets(torch, vd, inputs, dist_util, device, rank, peaks, barrier, main_w, main_path, main_kernels, main_off):
    """The figures the throughput targets are stated on, from a short pass over the Traffic-shaped workload (N = 862): all-token
    attention forward + backward against the dense bf16 peak, and the k-DFH, selection and gather kernels against the HBM
    peak.  When the main workload is Traffic itself its own tables are reused."""
    if main_w.name == "traffic":
        kernels, off = main_kernels, main_off
    else:
        w = inputs.WORKLOADS["traffic"]
        path = Path(w, device, seed=dist_util.rank_seed(w.seed, rank), slots=8, host_slots=0)
        slots = len(path.dev)
        for i in range(5):
            path.step(i % slots)
        torch.cuda.synchronize()
        n_sel = int(path.sel["n_sel"].item())
        vd.vardrop_profile_enable(True)
        time_region(torch, lambda i: path.step(i % slots), 50, barrier, min_seconds=0.05, min_intervals=20)
        kernels = kernel_table(per_launch(vd.vardrop_profile_read()), kernel_work(w, n_sel), peaks)
        vd.vardrop_profile_enable(False)
        off = measure_off(torch, vd, path, w, peaks, barrier, 20)
        path.check_status()
        del path
        torch.cuda.empty_cache()
    if off is None:
        return None
    pick = lambda name: ({"avg_us": kernels[name]["avg_us"], "frac_of_hbm_peak": kernels[name]["frac"]} if name in kernels else None)
    return {"workload": "traffic: B=32 N=862 L=96 k=3 rate=0.2 H=8 D=64",
            "n862_attn_fwd_us": off["attn_fwd_ms"] * 1e3, "n862_attn_bwd_us": off["attn_bwd_ms"] * 1e3,
            "n862_attn_tflops": off["attn_tflops"], "n862_attn_frac_of_bf16_peak": off["attn_frac_of_bf16_peak"],
            "n862_attn_target_frac": 0.5,
            "hash": pick("hash_kernel"), "select": pick("select_small_kernel"), "gather": pick("gather_kernel"),
            "hbm_target_frac": 0.6,
            "note": "per-kernel durations by CUDA events around every launch; fractions use algorithmic bytes / flops and the measured peaks"}


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
    gpu_keys = path.keys.cpu().numpy().view(np.uint64).copy()        # hash values of slot (warmup - 1) % slots, for the tie-flip count
    keys_slot = (args.warmup - 1) % slots

    # ---- timed region: passes of K whole steps, device resident -----------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = vd.vardrop_launch_count()
    t_main = time_region(torch, lambda i: path.step(i % slots), args.steps, barrier)
    launches = vd.vardrop_launch_count() - launches0
    # ---- the same steps with the per-kernel event timer armed (durations for the roofline) --------------------
    vd.vardrop_profile_enable(True)
    t_armed = time_region(torch, lambda i: path.step(i % slots), args.steps, barrier, min_seconds=0.15, min_intervals=20)
    per_kernel = per_launch(vd.vardrop_profile_read())
    vd.vardrop_profile_enable(False)
    # ---- end to end: host buffers, copies inside the timed region ----------------------------------------------
    path.e2e_setup()
    for i in range(3):
        path.step_e2e(i)
    torch.cuda.synchronize()
    t_e2e = time_region(torch, path.step_e2e, args.steps, barrier, begin=path.e2e_begin, drain=path.e2e_drain)
    clocks = sampler.stop() if rank == 0 else None
    # ---- VarDrop off, the target figures at N = 862, the redundancy check ---------------------------------------
    off = None if args.no_off else measure_off(torch, vd, path, w, peaks, barrier, max(3, min(args.steps, 20)))
    kernels = kernel_table(per_kernel, kernel_work(w, n_sel), peaks)
    targets = None
    if not args.no_targets and rank == 0 and world == 1:
        targets = traffic_targets(torch, vd, inputs, dist_util, device, rank, peaks, barrier, w, path, kernels, off)
    pearson = pearson_leg(torch, vd, path, w, peaks, barrier, args) if args.pearson else None
    path.check_status()

    ms, ms_mean, ms_e2e = dist_util.max_over_ranks([t_main["median"], t_main["mean"], t_e2e["median"]], dist, device)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    tokens = w.tokens * world
    top = max(kernels, key=lambda k: kernels[k]["share"])
    roofline = {"kernel": top, "bound": kernels[top]["bound"], "achieved": kernels[top]["achieved"], "peak": kernels[top]["peak"],
                "unit": kernels[top]["unit"], "frac": kernels[top]["frac"], "traffic": recorded_traffic(top, w.name),
                "peak_source": f"{peak_kind} (burst figure for tensor work)",
                "timing": "CUDA events around every launch, separate passes of the same K steps",
                "ms_per_step_with_timer_armed": t_armed["median"]}

    cpu, ties = (None, None) if args.no_cpu else cpu_baseline(w, reps=2, gpu_keys=gpu_keys, keys_x=path.host_x(keys_slot))
    line = {
        "metric": METRIC, "value": dist_util.aggregate_throughput(w.tokens, world, ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_mean": ms_mean, "host_issue_ms_per_step": t_main["host_ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 attention (fp32 accumulate), fp32 FFT, integer grouping", "data": "synthetic",
        "config": {"workload": f"{w.name}: B={w.B} N={w.N} L={w.L} k={w.k} rate={w.rate} H={w.H} D={w.D}",
                   "kept_tokens": n_sel, "groups": n_groups, "delta": 1.0 - n_sel / w.N,
                   "tie_flips": ties,
                   "l2": f"inputs and outputs rotate through {slots} sets ({slots * set_bytes / 2 ** 20:.0f} MiB > 126 MiB L2)",
                   "parallelism": f"dp{world} (independent batches per rank, no collective)"},
        "timing": {"statistic": "median of per-block CUDA-event intervals (a block is max(1, K // 64) steps); passes of exactly K steps "
                                f"repeated until {MIN_REGION_S} s and {MIN_INTERVALS} intervals; max over ranks",
                   "intervals": t_main["intervals"], "passes": t_main["passes"], "timed_ms_total": t_main["total_ms"]},
        "clocks": clocks, "gpu_launches": launches, "gpu_launches_per_step": launches / (t_main["passes"] * args.steps),
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": path.input_bytes(),
                "d2h_bytes_per_step": path.output_bytes(), "ms_per_step": ms_e2e,
                "pipeline": "copies on two extra streams beside the kernels, two slots in rotation; every step copies all its inputs in and all its outputs out"},
        "roofline": roofline, "kernels": kernels, "vardrop_off": off, "targets": targets, "cpu_baseline": cpu,
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


def cpu_baseline(w, reps, gpu_keys=None, keys_x=None):
    """The oracle as it stands, timed on a bounded sample (see sample_text).  With `gpu_keys` (the hash values the CUDA path
    produced for the windows `keys_x`) it also hashes that whole batch once and counts the variates whose hash differs: ties
    the fp32 transform decides the other way on unfiltered inputs, and how many of those lie inside the 1e-3 relative gap."""
    import oracle
    x, toks = oracle_inputs(w)
    plan = oracle_plan(w, seconds_per_step=5.0)
    oracle_step(w, x, toks, 0, plan)
    secs = [oracle_step(w, x, toks, 1 + r, plan) for r in range(reps)]
    s = float(np.mean(secs))
    ties = None
    if gpu_keys is not None:
        okeys, _, abar = oracle.hash(keys_x, w.k)
        differ = okeys[0] != gpu_keys[0]
        inside = oracle.rank_gaps(abar, w.k)[0] <= 1e-3
        ties = {"variates": int(w.N), "hash_differs": int(differ.sum()), "of_which_inside_1e-3_gap": int((differ & inside).sum()),
                "variates_inside_1e-3_gap": int(inside.sum())}
    return {"value": w.tokens / s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": sample_text(w, plan) + f"; mean of {reps} passes", "seconds_per_step": s}, ties


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
    ap.add_argument("--workload", default="scale", choices=["tiny", "elec", "traffic", "long", "scale"],
                    help="default: the largest single-GPU configuration")
    ap.add_argument("--impl", default="vardrop", choices=["vardrop", "reference"])
    ap.add_argument("--no-off", action="store_true", help="skip the VarDrop-off comparison pass")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU baseline (profiling runs)")
    ap.add_argument("--single-pass", action="store_true", help="one pass of K steps per timed region, no repetition (for ncu captures)")
    ap.add_argument("--no-targets", action="store_true", help="skip the short Traffic-shaped pass behind the `targets` block")
    ap.add_argument("--pearson", action="store_true", help="also time the variate-redundancy check (Appendix A, Eq. 4) on the workload's windows")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.single_pass:
        global MIN_REGION_S, MIN_INTERVALS
        MIN_REGION_S, MIN_INTERVALS = 0.0, 1
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
