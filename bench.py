"""Benchmark of the tropical-convolution hot path on B200.

One step = forward + backward of one layer of each mode (max_plus, min_plus, compound,
parallel) at N=128, C=K=64, 32x32, 3x3, stride 1, pad 1, fp32 (the configuration the
headline metric is quoted on), on seeded synthetic tensors.  The metric is tropical
Gop/s: operations of the paper's complexity analysis (additions + comparisons +
multiplications, Section 4.1), forward and backward each credited with the forward
count, divided by device time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

`--impl reference` times the CPU checker under oracle/ (as it stands) on the host cores
on a bounded sample of the same workload.  With N > 1 (torchrun) every rank runs the same
independent replica: the path has no inter-GPU exchange.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

MODES = [("max_plus", "default"), ("min_plus", "default"), ("compound", "default"),
         ("parallel", "default")]
WORKLOAD = "cfg2: one layer of each mode fwd+bwd fp32, N=128 C=K=64 32x32 3x3 s1 p1"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch at the bench's full size
# (N=128), from one-pass ncu captures of those two counters, summarised in
# profiles/dram_traffic_cfg2_n128.md.  bwd_params is the grad_w kernel of the call.
DRAM_BYTES_FULL = {("parallel", "fwd_winners"): 645.95e6, ("compound", "fwd_winners"): 646.41e6,
                   ("compound", "bwd_params"): 758.98e6, ("parallel", "bwd_params"): 758.98e6,
                   ("compound", "bwd_grad_x"): 601.37e6, ("parallel", "bwd_grad_x"): 601.37e6,
                   ("max_plus", "bwd_grad_x"): 70.50e6, ("min_plus", "bwd_grad_x"): 70.50e6}
# probe variants whose best gives the add+max/min peak of a mode's instruction mix
PROBES = {"max_plus": ("f32_add_max2", "f32_add_max3", "f32_add2_max3"),
          "min_plus": ("f32_add_max2", "f32_add_max3", "f32_add2_max3"),
          "compound": ("f32_add_minmax2", "f32_add_minmax3", "f32_add2_minmax3"),
          "parallel": ("f32_2add_minmax2", "f32_2add_minmax3", "f32_2add2_minmax3")}
# the same for the bf16 kernels: tap sums by add, by fma(x, 1, w), or the two alternating
PROBES_BF16 = {"max_plus": ("bf16x2_add_max", "bf16x2_fma_max", "bf16x2_mix_max"),
               "min_plus": ("bf16x2_add_max", "bf16x2_fma_max", "bf16x2_mix_max"),
               "compound": ("bf16x2_add_minmax", "bf16x2_fma_minmax", "bf16x2_mix_minmax"),
               "parallel": ("bf16x2_2add_minmax", "bf16x2_2fma_minmax", "bf16x2_2mix_minmax")}
# register-only probes of the winner-emitting Sum-form inner loop (sums, extrema, FMA keys, key fold)
WIN_PROBES = {"compound": "f32_win_compound", "parallel": "f32_win_parallel"}


def layer_ops(d):
    """Operations of Section 4.1 for one forward pass (python restatement for the CPU arm)."""
    from paper_2504_06881_b200 import inputs
    OH, OW = inputs.output_hw(d)
    P = d["N"] * d["K"] * OH * OW
    C, RS = d["C"], d["R"] * d["S"]
    if d["mode"] == "compound":
        return ((RS * C + 2 * C - 1) + 2 * (RS - 1) * C + 2 * C) * P
    if d["mode"] == "parallel":
        return ((2 * RS * C + 2 * C - 1) + 2 * (RS - 1) * C + 2 * C) * P
    chan = d["chan"] if d["chan"] != "default" else "full"
    if chan == "sum":
        return ((C - 1 + RS * C) + (RS - 1) * C) * P
    return (RS * C + (RS * C - 1)) * P


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.samples.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0])); mx = float(s[1])
            except ValueError:
                continue
            for name, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------ CPU arm (the checker)
def time_oracle_sample(n_sample: int):
    """One fwd+bwd of each mode on an n_sample-image slice of the workload, on the host cores."""
    from oracle import tconv_oracle as ora
    from paper_2504_06881_b200 import inputs
    t_total, ops = 0.0, 0.0
    for i, (mode, chan) in enumerate(MODES):
        d, dist = inputs.cfg2(mode, chan, N=n_sample)
        t = inputs.draw(d, 1020 + i, **dist)
        two = mode in ("compound", "parallel")
        w2 = t["w2"] if mode == "parallel" else None
        al, be = (t["alpha"], t["beta"]) if two else (None, None)
        t0 = time.perf_counter()
        ora.forward(d, t["x"], t["w"], w2, al, be, t["bias"])
        ora.backward(d, t["x"], t["w"], t["g"], w2, al, be)
        t_total += time.perf_counter() - t0
        ops += 2 * layer_ops(d)
    return t_total, ops


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import tconv_oracle as ora
    ora.build()
    cores = ora.threads()
    # the checker's backward runs one thread per image: one image per core keeps every
    # core busy and makes a step a few seconds of CPU work
    n_sample = max(1, min(128, cores))
    for _ in range(args.warmup):
        time_oracle_sample(1)
    t_sum, ops_sum = 0.0, 0.0
    for _ in range(args.steps):
        t, ops = time_oracle_sample(n_sample)
        t_sum += t; ops_sum += ops
    value = ops_sum / t_sum / 1e9
    sample = f"{n_sample} of 128 images of each layer per step (fwd+bwd, all four modes)"
    line = {"impl": "reference", "metric": "tropical conv fwd+bwd Gop/s", "value": value, "unit": "Gop/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * t_sum / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "Gop/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "Gop/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ GPU arm
class Layer:
    """Device-resident tensors of one layer plus its outputs, allocated once."""

    def __init__(self, mode, chan, seed, torch, tconv, inputs, dev, n_images=128, dtype="f32", desc=None,
                 e2e=True):
        self.d, dist = desc if desc is not None else inputs.cfg2(mode, chan, N=n_images)
        self.d = dict(self.d, dtype=dtype)
        d = self.d
        mode = d["mode"]
        t = inputs.draw(d, seed, **dist)
        dt = tconv.TORCH_DTYPE[dtype]
        self.host = {k: torch.from_numpy(v).to(dt if k in ("x", "w", "w2", "g") else torch.float32)
                     for k, v in t.items()}
        if e2e:
            self.host = {k: v.pin_memory() for k, v in self.host.items()}
        self.two = mode in ("compound", "parallel")
        self.par = mode == "parallel"
        self.dev = {k: v.to(dev, non_blocking=True) for k, v in self.host.items()}
        N, C, H, W, K = d["N"], d["C"], d["H"], d["W"], d["K"]
        OH, OW = tconv.tconv_output_shape(d)
        f32 = torch.float32
        self.y = torch.empty((N, K, OH, OW), dtype=dt, device=dev)
        self.win = tconv.winner_buffer(d, dev)
        self.ws = torch.empty(tconv.tconv_workspace_bytes(d, True), dtype=torch.uint8, device=dev)
        self.gx = torch.empty((N, C, H, W), dtype=dt, device=dev)
        self.gw = torch.empty((K, C, 3, 3), dtype=f32, device=dev)
        self.gw2 = torch.empty((K, C, 3, 3), dtype=f32, device=dev) if self.par else None
        self.ga = torch.empty((K, C), dtype=f32, device=dev) if self.two else None
        self.gb = torch.empty((K, C), dtype=f32, device=dev) if self.two else None
        self.gbias = torch.empty((K,), dtype=f32, device=dev)
        self.ops = 2 * tconv.tconv_paper_ops(d)
        self.taps = N * K * OH * OW * C * 9
        self.tconv = tconv
        self.ev_done = self.ev_out = None   # last kernels / last device-to-host copies of the e2e leg
        if not e2e:
            return
        # pinned host landing buffers of the end-to-end leg
        self.h_y = torch.empty((N, K, OH, OW), dtype=dt).pin_memory()
        self.h_gx = torch.empty((N, C, H, W), dtype=dt).pin_memory()
        self.h_small = {k: torch.empty_like(getattr(self, k), device="cpu").pin_memory()
                        for k in ("gw", "gw2", "ga", "gb", "gbias") if getattr(self, k) is not None}

    def fwd(self, with_winners=True):
        v = self.dev
        rc = self.tconv.tconv_forward(self.d, v["x"], v["w"], v["w2"] if self.par else None,
                                      v["alpha"] if self.two else None, v["beta"] if self.two else None,
                                      v["bias"], self.y, self.win if with_winners else None, self.ws)
        if rc != 0:
            raise self.tconv.TconvError(rc, "tconv_forward")

    def bwd(self, parts="all"):
        """parts: "all", "x" (grad_x only) or "params" (every parameter gradient)."""
        v = self.dev
        gx = self.gx if parts in ("all", "x") else None
        P = parts in ("all", "params")
        rc = self.tconv.tconv_backward(self.d, v["x"], v["w"], v["w2"] if self.par else None,
                                       v["alpha"] if self.two else None, v["beta"] if self.two else None,
                                       v["g"], self.win, gx, self.gw if P else None,
                                       self.gw2 if P else None, self.ga if P else None,
                                       self.gb if P else None, self.gbias if P else None, self.ws)
        if rc != 0:
            raise self.tconv.TconvError(rc, "tconv_backward")

    def e2e_step(self, torch, s_h2d, s_d2h):
        """Host buffers in, host buffers out, copies inside the timed region.  The copies run on
        their own streams so that one layer's transfers overlap the kernels of the others (each layer
        owns its device buffers): inputs are overwritten only after the previous kernels that read
        them, outputs only after the previous device-to-host copies of them; the kernels wait for
        their inputs, the device-to-host copies for the kernels."""
        names = ["x", "w", "bias", "g"] + (["w2"] if self.par else []) + (["alpha", "beta"] if self.two else [])
        cur = torch.cuda.current_stream()
        if self.ev_done is not None:
            s_h2d.wait_event(self.ev_done)
        with torch.cuda.stream(s_h2d):
            for k in names:
                self.dev[k].copy_(self.host[k], non_blocking=True)
            ev_in = torch.cuda.Event()
            ev_in.record(s_h2d)
        cur.wait_event(ev_in)
        if self.ev_out is not None:
            cur.wait_event(self.ev_out)
        self.fwd()
        self.bwd()
        self.ev_done = torch.cuda.Event()
        self.ev_done.record(cur)
        s_d2h.wait_event(self.ev_done)
        with torch.cuda.stream(s_d2h):
            self.h_y.copy_(self.y, non_blocking=True)
            self.h_gx.copy_(self.gx, non_blocking=True)
            for k, h in self.h_small.items():
                h.copy_(getattr(self, k), non_blocking=True)
            self.ev_out = torch.cuda.Event()
            self.ev_out.record(s_d2h)
        h2d = sum(self.host[k].numel() * self.host[k].element_size() for k in names)
        d2h = sum(h.numel() * h.element_size() for h in [self.h_y, self.h_gx] + list(self.h_small.values()))
        return h2d, d2h


def measure_alu_peak(torch, tconv):
    """Best measured taps/s over the candidate instruction mixes, per mode, for fp32 and for bf16.
    Every mix runs in two forms: with a few extra adds per iteration that advance its operands
    (8 % of a max-plus probe's instructions, left uncorrected) and with the operands advanced by
    feeding tap sums back (no extra instruction); the better of the two counts.  Returns (peaks
    fp32, peaks bf16, rates)."""
    sink = torch.zeros(4, device="cuda")
    names, i = {}, 0
    while tconv.tconv_alu_probe_name(i) is not None:
        names[tconv.tconv_alu_probe_name(i)] = i
        i += 1
    rate = {}
    for name, v in names.items():
        for _ in range(2):
            tconv.tconv_alu_probe(v, 2000, sink)
        best = None
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); taps = tconv.tconv_alu_probe(v, 2000, sink); e1.record()
            torch.cuda.synchronize()
            r = taps / (e0.elapsed_time(e1) * 1e-3)
            best = r if best is None else max(best, r)
        rate[name] = best
    # every mix in both forms: operands advanced by extra adds, or by feeding tap sums back ("_fb")
    both = lambda ps: [rate[p] for p in ps] + [rate[p + "_fb"] for p in ps]
    peaks = {m: max(both(ps)) for m, ps in PROBES.items()}
    peaks16 = {m: max(both(ps)) for m, ps in PROBES_BF16.items()}
    return peaks, peaks16, rate


# headline layers of the benchmark spec's target outside the bench step: (name, inputs.<cfg>, dtype)
HEADLINE = [("cfg3a parallel f32", "cfg3a", "f32"), ("cfg3a parallel bf16", "cfg3a", "bf16"),
            ("cfg3b parallel f32", "cfg3b", "f32"), ("cfg3b parallel bf16", "cfg3b", "bf16"),
            ("cfg4 compound bf16", "cfg4", "bf16")]


def time_headline_layers(torch, tconv, inputs, dev, peaks, peaks16):
    """Winner-free forward (ms, Ttap/s, fraction of the mode's measured add+max/min peak), forward
    with winners and full backward of the other headline layers, 5 repeats each (median)."""
    out = {}
    for name, cfg, dtype in HEADLINE:
        d, dist = getattr(inputs, cfg)(dtype)
        L = Layer(None, None, 1030, torch, tconv, inputs, dev, dtype=dtype, desc=(d, dist), e2e=False)
        rec = {}
        for what, fn in (("fwd", lambda: L.fwd(False)), ("fwd_winners", L.fwd), ("bwd", L.bwd)):
            fn()
            ts = []
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record(); torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            rec[what + "_ms"] = float(np.median(ts))
            rec[what + "_kernel"] = tconv.tconv_last_kernel()
        pk = (peaks if dtype == "f32" else peaks16)[d["mode"]]
        rec["taps"] = L.taps
        rec["fwd_Ttap_s"] = L.taps / (rec["fwd_ms"] * 1e-3) / 1e12
        rec["fwd_frac_of_alu_peak"] = L.taps / (rec["fwd_ms"] * 1e-3) / pk
        rec["alu_peak_Ttap_s"] = pk / 1e12
        out[name] = rec
        del L
        torch.cuda.empty_cache()
    return out


def max_over_ranks(torch, dist, values, device, world):
    """The replicas' times combine as the slowest rank's (the only exchange of a run: the data
    path itself has no collective)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_value(world, ops_per_step, steps, ms):
    """Whole-job throughput in Gop/s: every replica runs the same steps in the slowest rank's time."""
    return world * ops_per_step * steps / (ms * 1e-3) / 1e9


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2504_06881_b200 import inputs, tconv

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    layers = [Layer(m, c, 1020 + i, torch, tconv, inputs, dev) for i, (m, c) in enumerate(MODES)]
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step():
        for L in layers:
            L.fwd()
            L.bwd()

    # ---- device-resident timing: W warm-up steps, then exactly K steps
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = tconv.tconv_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = tconv.tconv_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if tconv.tconv_device_status() != 0:
        raise SystemExit("a device-side wait timed out during the timed region")

    # ---- end to end: host buffers in and out, copies inside the timed region
    s_h2d, s_d2h = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(2):
        for L in layers:
            L.e2e_step(torch, s_h2d, s_d2h)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h2d = d2h = 0
    f0.record()
    for _ in range(args.steps):
        h2d = d2h = 0
        for L in layers:
            a, b = L.e2e_step(torch, s_h2d, s_d2h)
            h2d += a; d2h += b
    for L in layers:                      # the timed region ends when the last result is on the host
        torch.cuda.current_stream().wait_event(L.ev_out)
    f1.record()
    barrier()
    ms_e2e = f0.elapsed_time(f1)

    # ---- per-call times of every mode (for the roofline of the dominant kernel)
    per = {}
    for L in layers:
        rec = {}
        for what, fn in (("fwd", lambda: L.fwd(False)), ("fwd_winners", L.fwd), ("bwd", L.bwd),
                         ("bwd_grad_x", lambda: L.bwd("x")), ("bwd_params", lambda: L.bwd("params"))):
            ts = []
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record(); torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            rec[what] = float(np.median(ts))
            rec[what + "_kernel"] = tconv.tconv_last_kernel()
        per[L.d["mode"]] = rec
    peaks, peaks16, probe_rates = measure_alu_peak(torch, tconv)
    headline = time_headline_layers(torch, tconv, inputs, dev, peaks, peaks16) if (rank == 0 and not args.no_headline) else None

    ms, ms_e2e = max_over_ranks(torch, dist, [ms, ms_e2e], dev, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ops_step = sum(L.ops for L in layers)
    value = aggregate_value(world, ops_step, args.steps, ms)
    e2e_value = aggregate_value(world, ops_step, args.steps, ms_e2e)

    # dominant kernel = the call with the largest time in a step; its roofline is the
    # add+max/min ALU peak of that mode (a tap = one x+w term folded into min and/or max)
    dom_mode, dom_what = max(((m, w) for m in per for w in ("fwd_winners", "bwd_grad_x", "bwd_params")),
                             key=lambda mw: per[mw[0]][mw[1]])
    L = next(x for x in layers if x.d["mode"] == dom_mode)
    achieved = L.taps / (per[dom_mode][dom_what] * 1e-3) / 1e12
    roofline = {"bound": "alu", "kernel": per[dom_mode][dom_what + "_kernel"], "call": f"{dom_mode} {dom_what}",
                "achieved": achieved, "peak": peaks[dom_mode] / 1e12, "unit": "Ttap/s",
                "frac": achieved / (peaks[dom_mode] / 1e12),
                "traffic": DRAM_BYTES_FULL.get((dom_mode, dom_what)),
                "traffic_note": "DRAM bytes per launch, one-pass ncu capture at this size (profiles/dram_traffic_cfg2_n128.md)",
                "peak_source": ("measured in this run: best register-only add+max/min probe of the mode (taps/s "
                                "of the winner-free instruction mix, 1 add + 1-2 compares per tap); winner emission "
                                "and the backward do other work per tap than that mix and are held to the same "
                                "denominator")}
    if dom_what == "fwd_winners" and dom_mode in WIN_PROBES:
        # secondary: against a register-only replay of the kernel's own winner-emitting loop
        roofline["frac_of_own_mix"] = achieved / (probe_rates[WIN_PROBES[dom_mode]] / 1e12)
    fwd_frac = {m: {"ms": per[m]["fwd"], "Ttap_s": L2.taps / (per[m]["fwd"] * 1e-3) / 1e12,
                    "frac_of_alu_peak": L2.taps / (per[m]["fwd"] * 1e-3) / peaks[m],
                    "kernel": per[m]["fwd_kernel"]}
                for m, L2 in ((x.d["mode"], x) for x in layers)}

    # ---- CPU baseline: the checker as it stands, bounded sample, host cores of this machine
    from oracle import tconv_oracle as ora
    ora.build()
    n_sample = max(1, min(128, 2 * ora.threads()))   # two images per core: about 10 s
    tc, opsc = time_oracle_sample(n_sample)
    cpu = {"value": opsc / tc / 1e9, "unit": "Gop/s", "cores": ora.threads(), "kind": "oracle",
           "sample": f"{n_sample} of 128 images of each layer, fwd+bwd, all four modes ({tc:.1f} s)"}

    line = {"metric": "tropical conv fwd+bwd Gop/s", "value": value, "unit": "Gop/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": "per-step working set ~1.6 GB exceeds the 126 MB L2",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "Gop/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu,
            "per_mode_ms": per, "forward_vs_alu_peak": fwd_frac, "headline_layers": headline,
            "alu_peak_Ttap_s": {"f32": {m: v / 1e12 for m, v in peaks.items()},
                                "bf16": {m: v / 1e12 for m, v in peaks16.items()}},
            "alu_probe_Ttap_s": {k: v / 1e12 for k, v in probe_rates.items()},
            "alu_probe_note": ("register-only loops; plain names advance their operands with extra adds (5 per 64 "
                               "taps, uncorrected), _fb names feed tap sums back (no extra instruction); a mode's "
                               "peak is the best of all its mixes in both forms")}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_single(args):
    """One call of one layer, repeated: the small, single-kernel case the ncu captures under
    profiles/ are taken on (`--only MODE --what fwd|fwd_winners|bwd --images N [--dtype bf16]`)."""
    import torch
    from paper_2504_06881_b200 import inputs, tconv
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    L = Layer(args.only, "default", 1020, torch, tconv, inputs, dev, n_images=args.images, dtype=args.dtype)
    fn = {"fwd": lambda: L.fwd(False), "fwd_winners": L.fwd, "bwd": L.bwd}[args.what]
    L.fwd()
    for _ in range(max(args.warmup, 1)):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    print(json.dumps({"only": args.only, "what": args.what, "images": args.images, "dtype": args.dtype,
                      "ms": ms, "Ttap_s": L.taps / (ms * 1e-3) / 1e12, "kernel": tconv.tconv_last_kernel()}))


def run_cfg5(args):
    """Training step of the ResNet-18-shaped hybrid network (N=64, 224x224, stages 2-4 tropical,
    bf16 tropical kernels): step time, summed tropical-layer time and tropical Gop/s."""
    import torch
    from paper_2504_06881_b200 import tconv
    from paper_2504_06881_b200.nn import HybridResNet18, TropicalConvFn
    torch.cuda.set_device(0)
    torch.manual_seed(1050)
    rs = np.random.RandomState(1050)
    N = 64
    net = HybridResNet18(mode=args.only or "compound", dtype="bf16", fused_bn=args.fused_bn).cuda()
    TropicalConvFn.fuse_cast = bool(args.fuse_cast)
    x = torch.from_numpy(rs.standard_normal((N, 3, 224, 224)).astype(np.float32)).cuda()
    labels = torch.from_numpy(rs.randint(0, 1000, N)).cuda()
    opt = torch.optim.SGD(net.parameters(), lr=0.01, momentum=0.9)

    def step():
        loss = torch.nn.functional.cross_entropy(net(x), labels)
        opt.zero_grad()
        loss.backward()
        opt.step()
        return loss

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    TropicalConvFn.events = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        loss = step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    ev = TropicalConvFn.events
    TropicalConvFn.events = None
    t_fwd = sum(a.elapsed_time(b) for k, d, a, b in ev if k == "fwd") / args.steps
    t_bwd = sum(a.elapsed_time(b) for k, d, a, b in ev if k == "bwd") / args.steps
    ops = sum(2 * tconv.tconv_paper_ops(d) for k, d, a, b in ev if k == "fwd") / args.steps
    taps = sum(d["N"] * d["K"] * d["C"] * 9 * tconv.tconv_output_shape(d)[0] * tconv.tconv_output_shape(d)[1]
               for k, d, a, b in ev if k == "fwd") / args.steps
    print(json.dumps({"workload": "cfg5: ResNet-18-shaped hybrid net, N=64, 224x224, stages 2-4 tropical (bf16 kernels)",
                      "mode": args.only or "compound", "fused_bn": bool(args.fused_bn),
                      "float_x_read_by_the_kernels": bool(args.fuse_cast), "step_ms": ms, "tropical_fwd_ms": t_fwd,
                      "tropical_bwd_ms": t_bwd, "tropical_layers": len([1 for e in ev if e[0] == "fwd"]) // args.steps,
                      "tropical_taps_fwd": taps, "tropical_Gop_s_fwd_bwd": ops / ((t_fwd + t_bwd) * 1e-3) / 1e9,
                      "loss": float(loss.detach())}))


def run_dw(args):
    """Depthwise (groups = C) layer of a MobileNetV2-shaped stage: N=128, C=144, 56x56, 3x3, stride 1,
    pad 1 (the expanded 24-channel stage at t=6), mode --only (default compound), --dtype.  The form is
    memory bound (9 taps per output): forward, forward with winner codes and backward are reported as
    algorithmic GB/s against the measured copy bandwidth."""
    import torch
    from paper_2504_06881_b200 import inputs, tconv
    torch.cuda.set_device(0)
    mode = args.only or "compound"
    N, C, H, W = args.images, 144, 56, 56
    d = inputs.layer(N, C, H, W, C, 3, 3, stride=1, pad=1, mode=mode, dtype=args.dtype)
    dt = tconv.TORCH_DTYPE[args.dtype]
    es = 4 if args.dtype == "f32" else 2
    rs = np.random.RandomState(1060)
    f = lambda *sh: torch.from_numpy(rs.standard_normal(sh).astype(np.float32)).cuda()
    x, g = f(N, C, H, W).to(dt), f(N, C, H, W).to(dt)
    w, w2 = (0.1 * f(C, 3, 3)).to(dt), (0.1 * f(C, 3, 3)).to(dt)
    al, be, bias = torch.rand(C, device="cuda"), torch.rand(C, device="cuda"), torch.rand(C, device="cuda")
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    y = torch.empty(N, C, H, W, device="cuda", dtype=dt)
    win = torch.empty(N, C, H, W, device="cuda", dtype=torch.uint8)
    ws = torch.empty(tconv.tconv_dw_workspace_bytes(d, True), dtype=torch.uint8, device="cuda")
    gx = torch.empty_like(x)
    gw, gw2 = torch.empty(C, 3, 3, device="cuda"), torch.empty(C, 3, 3, device="cuda")
    ga, gb, gbi = (torch.empty(C, device="cuda") for _ in range(3))
    fa = (d, x, w, w2 if par else None, al if two else None, be if two else None, bias, y)
    calls = {"fwd": lambda: tconv.tconv_dw_forward(*fa, None),
             "fwd_winners": lambda: tconv.tconv_dw_forward(*fa, win),
             "bwd": lambda: tconv.tconv_dw_backward(d, x, w, w2 if par else None, al if two else None,
                                                    be if two else None, g, win, gx, gw, gw2 if par else None,
                                                    ga if two else None, gb if two else None, gbi, ws)}
    peaks_file = Path(__file__).parent / "MEASURED_PEAKS.json"
    hbm, src = (json.loads(peaks_file.read_text())["hbm_gbs"], "measured") if peaks_file.exists() else (6650.0, "fallback")
    n = N * C * H * W
    # algorithmic bytes: x once, y once (+ one code byte per output); backward: grad_y and codes for
    # grad_x plus grad_y, codes and x for the parameter gradients, grad_x written once
    nbytes = {"fwd": 2 * n * es, "fwd_winners": 2 * n * es + n, "bwd": (n * es + n + n * es) + (2 * n * es + n)}
    out = {"workload": f"depthwise {mode} {args.dtype}: N={N} C={C} {H}x{W} 3x3 s1 p1", "hbm_peak_GB_s": hbm,
           "hbm_peak_source": src}
    for name, fn in calls.items():
        assert fn() == 0, tconv.tconv_last_error()
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(args.steps, 5)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ms = float(np.median(ts))
        out[name] = {"ms": ms, "GB_s": nbytes[name] / ms / 1e6, "frac_of_hbm": nbytes[name] / ms / 1e6 / hbm,
                     "kernel": tconv.tconv_last_kernel()}
    print(json.dumps(out))


def run_conv3d(args):
    """The two tropical layers of the paper's 3-D LeNet (Table 1, configuration 3d: [5/6, 2] then
    [5/16] on the pooled volume) at both input sizes of the appendix (28^3 with batch 32, 64^3 with
    batch 2), mode --only (default compound), fp32 or bf16: forward, forward with winners and the
    full backward per layer, in ms and Ttap/s.  The layers are a few tens of Mtap: the times are
    close to launch latency, so no roofline fraction is claimed for them."""
    import torch
    from paper_2504_06881_b200 import inputs, tconv, tconv3d
    torch.cuda.set_device(0)
    mode = args.only or "compound"
    dt = tconv.TORCH_DTYPE[args.dtype]
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    layers = [("28^3 L1", inputs.layer3d(32, 1, 28, 28, 28, 6, T=5, R=5, S=5, stride=2, mode=mode, dtype=args.dtype)),
              ("28^3 L2", inputs.layer3d(32, 6, 6, 6, 6, 16, T=5, R=5, S=5, mode=mode, dtype=args.dtype)),
              ("64^3 L1", inputs.layer3d(2, 1, 64, 64, 64, 6, T=5, R=5, S=5, stride=2, mode=mode, dtype=args.dtype)),
              ("64^3 L2", inputs.layer3d(2, 6, 15, 15, 15, 16, T=5, R=5, S=5, mode=mode, dtype=args.dtype))]
    out = {"workload": f"3-D LeNet tropical layers, {mode} {args.dtype}", "layers": {}}
    l0 = tconv3d.tconv3d_launch_count()
    for name, d in layers:
        t = inputs.draw3d(d, 1070)
        dev = lambda a, ty=None: torch.from_numpy(a).cuda().to(ty) if ty else torch.from_numpy(a).cuda()
        x, w, w2, g = (dev(t[k], dt) for k in ("x", "w", "w2", "g"))
        al, be, bias = dev(t["alpha"]), dev(t["beta"]), dev(t["bias"])
        y = torch.empty(t["g"].shape, device="cuda", dtype=dt)
        win = tconv3d.winner_buffer(d, "cuda")
        ws = torch.empty(tconv3d.tconv3d_workspace_bytes(d, True), dtype=torch.uint8, device="cuda")
        gx, gw, gw2 = torch.empty_like(x), torch.empty_like(w, dtype=torch.float32), torch.empty_like(w, dtype=torch.float32)
        ga, gb, gbi = torch.empty_like(al), torch.empty_like(be), torch.empty_like(bias)
        fa = (d, x, w, w2 if par else None, al if two else None, be if two else None, bias, y)
        calls = {"fwd": lambda: tconv3d.tconv3d_forward(*fa, None),
                 "fwd_winners": lambda: tconv3d.tconv3d_forward(*fa, win),
                 "bwd": lambda: tconv3d.tconv3d_backward(d, x, w, w2 if par else None, al if two else None,
                                                         be if two else None, g, win, gx if d["C"] > 1 else None,
                                                         gw, gw2 if par else None, ga if two else None,
                                                         gb if two else None, gbi, ws)}
        od = tconv3d.tconv3d_output_shape(d)
        taps = d["N"] * d["K"] * od[0] * od[1] * od[2] * d["C"] * 125
        row = {"Mtap": taps / 1e6}
        for what, fn in calls.items():
            assert fn() == 0
            for _ in range(max(args.warmup, 3)):
                fn()
            torch.cuda.synchronize()
            ts = []
            for _ in range(max(args.steps, 5)):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            row[what + "_ms"] = float(np.median(ts))
        row["fwd_Ttap_s"] = taps / row["fwd_ms"] / 1e9
        out["layers"][name] = row
    out["gpu_launches"] = tconv3d.tconv3d_launch_count() - l0
    print(json.dumps(out))


def run_conv1d(args):
    """The opening layer of the paper's audio networks (appendix "One-dimensional data
    classification": one input channel, 128 output channels, window 80, stride 4, signals of 16000
    samples; batch --images, default 32) and a mid-network layer with a window of 3 (128 -> 128
    channels, length 1000), mode --only (default compound), fp32 or bf16: forward, forward with
    winners and the full backward, in ms and Ttap/s, and the forward's fraction of the mode's
    measured add+max/min peak."""
    import torch
    from paper_2504_06881_b200 import inputs, tconv, tconv3d
    from paper_2504_06881_b200.nn import TropicalConv1d
    torch.cuda.set_device(0)
    mode = args.only or "compound"
    dt = tconv.TORCH_DTYPE[args.dtype]
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    peaks, peaks16, _ = measure_alu_peak(torch, tconv)
    peak = (peaks16 if args.dtype == "bf16" else peaks)[mode]
    n = args.images if args.images != 128 else 32
    d = inputs.layer3d(n, 1, 1, 1, 16000, 128, T=1, R=1, S=80, stride=(1, 1, 4), mode=mode, dtype=args.dtype)
    out = {"workload": f"1-D audio layers, {mode} {args.dtype}, batch {n}", "peak_Ttap_s": peak / 1e12, "layers": {}}
    l0 = tconv3d.tconv3d_launch_count()
    t = inputs.draw3d(d, 1080)
    dev = lambda a, ty=None: torch.from_numpy(a).cuda().to(ty) if ty else torch.from_numpy(a).cuda()
    x, w, w2, g = (dev(t[k], dt) for k in ("x", "w", "w2", "g"))
    al, be, bias = dev(t["alpha"]), dev(t["beta"]), dev(t["bias"])
    y = torch.empty(t["g"].shape, device="cuda", dtype=dt)
    win = tconv3d.winner_buffer(d, "cuda")
    ws = torch.empty(tconv3d.tconv3d_workspace_bytes(d, True), dtype=torch.uint8, device="cuda")
    gx, gw, gw2 = torch.empty_like(x), torch.empty_like(w, dtype=torch.float32), torch.empty_like(w, dtype=torch.float32)
    ga, gb, gbi = torch.empty_like(al), torch.empty_like(be), torch.empty_like(bias)
    fa = (d, x, w, w2 if par else None, al if two else None, be if two else None, bias, y)
    calls = {"fwd": lambda: tconv3d.tconv3d_forward(*fa, None),
             "fwd_winners": lambda: tconv3d.tconv3d_forward(*fa, win),
             "bwd": lambda: tconv3d.tconv3d_backward(d, x, w, w2 if par else None, al if two else None,
                                                     be if two else None, g, win, gx, gw, gw2 if par else None,
                                                     ga if two else None, gb if two else None, gbi, ws)}
    od = tconv3d.tconv3d_output_shape(d)
    taps = d["N"] * d["K"] * od[2] * d["C"] * 80
    row = {"Mtap": taps / 1e6}
    for what, fn in calls.items():
        assert fn() == 0
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(args.steps, 5)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        row[what + "_ms"] = float(np.median(ts))
    row["fwd_Ttap_s"] = taps / row["fwd_ms"] / 1e9
    row["fwd_frac_of_alu_peak"] = taps / row["fwd_ms"] / 1e-3 / peak
    out["layers"]["k80 s4 1->128 L16000"] = row
    launches = tconv3d.tconv3d_launch_count() - l0
    # a mid-network layer (window 3, stride 1) through the module: the tiled 2-D kernels
    m = TropicalConv1d(128, 128, 3, padding=1, mode=mode, dtype=args.dtype).cuda()
    xm = torch.randn(n, 128, 1000, device="cuda", requires_grad=True)
    gm = torch.randn(n, 128, 1000, device="cuda")
    def step():
        xm.grad = None
        m(xm).backward(gm)
    l1 = tconv.tconv_launch_count()
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    ts = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); step(); e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    out["layers"]["k3 s1 128->128 L1000 (module, fwd+bwd)"] = {"Mtap": n * 128 * 128 * 1000 * 3 / 1e6,
                                                              "fwd_bwd_ms": float(np.median(ts))}
    out["gpu_launches"] = launches + tconv.tconv_launch_count() - l1
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--only", default=None, choices=["max_plus", "min_plus", "compound", "parallel"],
                    help="profile helper: run one layer's call instead of the benchmark step")
    ap.add_argument("--what", default="fwd", choices=["fwd", "fwd_winners", "bwd"])
    ap.add_argument("--images", type=int, default=128)
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16"])
    ap.add_argument("--fused-bn", action="store_true",
                    help="cfg5: batch-normalisation statistics from the tropical kernels' epilogue")
    ap.add_argument("--fuse-cast", action="store_true",
                    help="cfg5: the bf16 kernels read the float activations directly (x_dtype) instead of a converted copy")
    ap.add_argument("--no-headline", action="store_true",
                    help="skip the headline_layers section (cfg 3a / 3b / 4 timed after the step)")
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg5", "dw", "conv3d", "conv1d"],
                    help="cfg5: report the hybrid ResNet-18 training step instead (use --only compound|parallel); "
                         "dw: a depthwise (groups = C) layer against the HBM roofline; conv3d: the 3-D LeNet layers; conv1d: the 1-D audio layers")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "cfg5":
        run_cfg5(args)
    elif args.workload == "conv3d":
        run_conv3d(args)
    elif args.workload == "conv1d":
        run_conv1d(args)
    elif args.workload == "dw":
        run_dw(args)
    elif args.only:
        run_single(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
