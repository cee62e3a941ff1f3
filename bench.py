#!/usr/bin/env python
"""Benchmark of the linear-attention forward (Eq. 5 with the feature map of Eq. 6) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C]

One step = one `linattn_forward` over one batch of synthetic Wan-shaped input (default: the
Wan-1.3B 480p layer, B=1, H=12, n=32760, d=128, bf16).  Prints ONE JSON line on rank 0.
With N > 1 (under torchrun) every rank runs an independent replica on its own inputs: the
operator has no cross-GPU exchange, so there is no data-path collective (weak scaling).
`--impl reference` times the fp64 CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_08318_b200 import dist as ladist  # noqa: E402
from paper_2510_08318_b200 import synth  # noqa: E402

METRIC = "linear-attention fwd tokens/s"
UNIT = "tokens/s"
ROTATE = 3  # input sets cycled through, so that a step's inputs were last touched > 2 x L2 ago (config 5: all 30 layers)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


def source_digest(kernel: str = "linattn_fused_tc"):
    """Digest of the sources `kernel` is built from (the forward's tensor-core kernels, their PTX wrappers and the tensor
    maps; for the backward's kernels their own file as well): DRAM counters taken with ncu are only quoted for the code
    they were taken on."""
    import hashlib
    h = hashlib.sha256()
    names = ["sm100_kernels.cuh", "sm100_ptx.cuh", "tensor_map.hpp"] + (["sm100_backward.cuh"] if "bwd" in kernel else [])
    for name in names:
        h.update(open(os.path.join(ROOT, "paper_2510_08318_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(kernel):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` at the benchmark's workload, from the
    ncu summary under profiles/ (lines `kernel bytes digest`); None if absent or taken on other sources."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        f = line.split()
        if len(f) == 3 and f[0] == kernel and f[2] == source_digest(kernel):
            return float(f[1])
    return None


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons while the benchmark runs: NVML polled from a thread
    as fast as it answers (a few hundred microseconds per sample, so that even a timed region of a millisecond or two
    gets samples of its own), with `nvidia-smi -lms 50` as the fallback when the NVML binding is missing.  Read-only."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    BITS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.0002):
        self.index, self.rows, self.proc, self.nvml, self.stop_flag = index, [], None, None, False
        self.period_s = period_s

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll(self):
        n = self.nvml
        while not self.stop_flag:
            try:
                t = time.time()
                mhz = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                bits = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                self.rows.append((t, mhz, bits))
                time.sleep(self.period_s)   # leave the interpreter to the thread that launches the kernels
            except Exception:
                break

    def _read(self):
        for line in self.proc.stdout:
            f = [c.strip() for c in line.split(",")]
            if len(f) >= 6 and f[0].replace(".", "").isdigit():
                bits = sum(b for (nm, b), col in zip(self.BITS.items(), f[2:6]) if col == "Active")
                self.max_mhz = float(f[1]) if f[1].replace(".", "").isdigit() else None
                self.rows.append((time.time(), float(f[0]), bits))

    def stop(self, t0=None, t1=None):
        """Statistics over the samples taken inside [t0, t1] (the timed region) when there are any, else over all."""
        if self.nvml is None and not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no NVML binding and no nvidia-smi"], "samples": 0}
        self.stop_flag = True
        if self.proc:
            self.proc.terminate()
        self.thread.join(timeout=2)
        rows = list(self.rows)
        inside = [r for r in rows if t0 is not None and t0 <= r[0] <= t1]
        use, where = (inside, "timed region") if inside else (rows, "whole run of the benchmark's GPU passes")
        reasons = [nm for nm, b in self.BITS.items() if any(r[2] & b for r in use)]
        return {"sm_mhz": statistics.median(r[1] for r in use) if use else None, "sm_max_mhz": getattr(self, "max_mhz", None),
                "reasons": reasons, "samples": len(use), "samples_from": where, "samples_all_passes": len(rows),
                "source": "NVML" if self.nvml is not None else "nvidia-smi -lms 50"}


def time_oracle(x, budget_s: float):
    """Oracle (right-hand form of Eq. 5, fp64, as it stands) on a bounded sample: the first n_s tokens of
    every head.  Its cost is linear in tokens, so tokens/s on the sample stands for the workload."""
    import oracle
    B, H, n, d = x["q"].shape
    probe = min(n, 2048)

    def run(ns):
        sl = {k_: (x[k_][:, :, :ns].contiguous() if k_ in ("q", "k", "v") else x[k_]) for k_ in x}
        t0 = time.perf_counter()
        oracle.ref_linear(sl["q"], sl["k"], sl["v"], sl["Wq"], sl["Wk"])
        return time.perf_counter() - t0

    run(min(n, 256))  # builds / loads the oracle, warms the thread pool
    rate = probe / run(probe)
    ns = int(max(probe, min(n, rate * budget_s)))
    reps = int(max(1, min(50, round(budget_s * rate / ns))))  # whole workload fits the budget several times: repeat it
    secs = sum(run(ns) for _ in range(reps))
    return {"tokens": B * ns * reps, "seconds": secs, "value": B * ns * reps / secs, "cores": oracle.threads(),
            "sample": f"first {ns} of n={n} tokens of all {B}x{H} heads, {reps} runs, {secs:.2f} s"}


def reference_arm(args, wl):
    """--impl reference: the CPU oracle, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    x = synth.make_inputs(args.config)
    total = args.steps + args.warmup
    budget = min(10.0, 150.0 / max(1, total))   # seconds of oracle work per step: the whole run stays within minutes
    import oracle
    B, H, n, d = x["q"].shape
    probe = min(n, 1024)
    sl = lambda ns: [x[k_][:, :, :ns].contiguous() for k_ in ("q", "k", "v")] + [x["Wq"], x["Wk"]]
    oracle.ref_linear(*sl(64))  # builds / loads the oracle
    t0 = time.perf_counter(); oracle.ref_linear(*sl(probe)); rate = probe / (time.perf_counter() - t0)
    ns = int(max(256, min(n, rate * budget)))
    a = sl(ns)
    for _ in range(args.warmup):
        oracle.ref_linear(*a)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.ref_linear(*a)
    secs = time.perf_counter() - t0
    value = B * ns * args.steps / secs
    sample = f"first {ns} of n={n} tokens of all {B}x{H} heads per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(args, wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def wl_name(config, wl):
    return f"config {config}: {wl.name} B={wl.B} H={wl.H} n={wl.n} d={wl.d} {wl.dtype}"


def config_dict(args, wl):
    """The workload as both arms (ours and --impl reference) name it: identical keys and values, so that the two
    lines can be matched on it."""
    rotate = wl.layers if wl.layers > 1 else ROTATE
    return {"workload": wl_name(args.config, wl), "B": wl.B, "H": wl.H, "n": wl.n, "d": wl.d,
            "layout": "[B][n][H][d]" if getattr(args, "layout", 0) else "[B][H][n][d]",
            "l2": f"inputs larger than L2 and {rotate} input sets rotated (no set is re-read within {rotate - 1} steps)",
            "multi_gpu": "replicas only: independent inputs per rank, no collective on the data path"}


ALL_VARIANTS = [
    ("forward, config 2 (the metric's workload)", ["--config", "2"]),
    ("forward, config 3", ["--config", "3"]),
    ("forward, config 4", ["--config", "4"]),
    ("forward, config 5 (30 resident layers)", ["--config", "5"]),
    ("forward, config 6 (CogVideoX-2B-shaped, d = 64)", ["--config", "6"]),
    ("forward, config 2, token-major layout [B][n][H][d]", ["--config", "2", "--layout", "1"]),
    ("mixed attention (Eq. 8), r = 0.5, config 2", ["--config", "2", "--mixed", "0.5"]),
    ("ReLU kernel function, config 2", ["--config", "2", "--phi", "relu"]),
    ("backward, config 2", ["--config", "2", "--backward"]),
    ("training step (forward, then backward with the forward's S and z), config 2", ["--config", "2", "--train-step"]),
    ("backward, config 3", ["--config", "3", "--backward"]),
    ("backward, config 4", ["--config", "4", "--backward"]),
]


def run_all(args):
    """Child run of this script per variant (a fresh process each: fresh contexts, nothing resident from the previous
    one); prints each child's JSON line and writes a markdown table of them."""
    rows = []
    for title, extra in ALL_VARIANTS:
        steps = 300 if "--backward" not in extra and "--train-step" not in extra else 100
        cmd = [sys.executable, os.path.abspath(__file__), "--gpus", "1", "--steps", str(steps), "--warmup", "10", "--no-baselines"] + extra
        res = subprocess.run(cmd, capture_output=True, text=True)
        line = next((l for l in reversed(res.stdout.splitlines()) if l.startswith("{")), None)
        if res.returncode != 0 or line is None:
            rows.append((title, None, (res.stderr or res.stdout)[-300:].replace("\n", " ")))
            continue
        print(line, flush=True)
        rows.append((title, json.loads(line), ""))
    out = ["# Benchmark table: every workload and variant, one B200", "",
           f"Written by `python bench.py --all` (each row: `python bench.py --gpus 1 --steps 300 --warmup 10 --no-baselines <variant>`, "
           f"100 steps for the backward), source digest {source_digest()}.", "",
           "| variant | step (mean) | median / min | tokens/s | algorithmic GB/s | of measured peak | of nominal 8 TB/s | dominant kernel | SM clock (median), reasons |",
           "|---|---|---|---|---|---|---|---|---|"]
    for title, r, err in rows:
        if r is None:
            out.append(f"| {title} | failed: {err} | | | | | | | |")
            continue
        rf, ws, ck = r["roofline"], r["roofline"]["whole_step"], r.get("clocks") or {}
        sp = rf["step_spread"]
        out.append(f"| {title} | {1e3 * r['ms_per_step']:.1f} us | {1e3 * sp['median_ms']:.1f} / {1e3 * sp['min_ms']:.1f} us | {r['value']:.3e} | "
                   f"{ws['achieved']:.0f} | {ws['frac']:.3f} | {ws['frac_of_nominal_8TBs']:.3f} | {rf['kernel']} ({1e3 * rf['kernel_ms']:.1f} us) | "
                   f"{ck.get('sm_mhz')} MHz, {','.join(ck.get('reasons') or []) or 'none'} |")
    os.makedirs(os.path.dirname(args.table_out), exist_ok=True)
    with open(args.table_out, "w") as f:
        f.write("\n".join(out) + "\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=sorted(c_ for c_ in synth.CONFIGS if c_ >= 2))
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 CUDA-core kernels, 2 tensor-core kernels")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--no-baselines", action="store_true", help="skip the oracle and SDPA context baselines")
    ap.add_argument("--clock-period-ms", type=float, default=0.2, help="pause between two NVML samples of the SM clock (ms)")
    ap.add_argument("--mixed", type=float, default=None, metavar="R",
                    help="time mixed attention (Eq. 8) with score R instead: linattn_forward_mixed on a resident "
                         "softmax-branch output (5 tensors of traffic instead of 4)")
    ap.add_argument("--phi", default="hedgehog", choices=["hedgehog", "relu"],
                    help="kernel function: the Hedgehog feature map of Eq. 6 (the metric's) or the ReLU of the paper's ablation")
    ap.add_argument("--train-step", action="store_true",
                    help="time a training step of the layer: linattn_forward followed by linattn_backward on the same q, k, v, "
                         "with LINATTN_OPT_REUSE_STATE = 1 (the backward takes S and z over from the forward that just ran)")
    ap.add_argument("--backward", action="store_true",
                    help="time linattn_backward (gradients of the operator; the kernels --path selects) instead of the forward")
    ap.add_argument("--layout", type=int, default=0, choices=[0, 1],
                    help="memory order of q, k, v, out: 0 = [B][H][n][d] (the metric's), 1 = [B][n][H][d] (LINATTN_OPT_LAYOUT)")
    ap.add_argument("--source-digest", action="store_true",
                    help="print the digest of the forward kernels' sources (what profiles/dram_traffic.txt is keyed by) and exit")
    ap.add_argument("--all", action="store_true",
                    help="run every workload and variant (configs 2-5 and the CogVideoX-shaped one, mixed attention, ReLU, backward, "
                         "token-major layout) as child runs, print one JSON line each and write the table to --table-out")
    ap.add_argument("--table-out", default=os.path.join(ROOT, "profiles", "bench_table.md"))
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.source_digest:
        print(source_digest(), "(forward kernels)", source_digest("qside_bwd_tc"), "(backward kernels)")
        return
    if args.all:
        run_all(args)
        return
    wl = synth.CONFIGS[args.config]

    if args.impl == "reference":
        reference_arm(args, wl)
        return

    from paper_2510_08318_b200 import linattn

    rank, world, local = ladist.init_from_env("nccl")
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torchrun --nproc-per-node {args.gpus}"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    sampler = ClockSampler(local, args.clock_period_ms * 1e-3)   # started this early so that it is polling steadily by the time the timed region runs
    if rank == 0:
        sampler.start()

    # inputs: `rotate` independent sets per rank (different layers' seeds), resident in HBM; the 30-layer workload
    # keeps every layer resident and walks through them back to back on the one stream
    rotate = wl.layers if wl.layers > 1 else ROTATE
    B, H, n, d = wl.B, wl.H, wl.n, wl.d
    sets = []
    host0 = None
    for r in range(rotate):
        x = synth.make_inputs(args.config, layer=(rank * rotate + r) % max(wl.layers, 30))
        if r == 0:
            host0 = x
        sets.append({k_: t.to(dev) for k_, t in x.items()})
    outs = [torch.empty_like(s["q"]) for s in sets]
    softs = [torch.randn_like(s["q"]) for s in sets] if args.mixed is not None else None
    douts = [torch.randn_like(s["q"]) for s in sets] if (args.backward or args.train_step) else None
    ctxs = []
    for s in sets:  # one context per input set: its own feature map, as one layer would have
        c = linattn.LinAttn(H, d, max_B=B, max_n=n, device=local)
        c.set_option(linattn.OPT_PATH, args.path)
        c.set_option(linattn.OPT_SPLITS, args.splits)
        c.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_RELU if args.phi == "relu" else linattn.PHI_HEDGEHOG)
        c.set_option(linattn.OPT_LAYOUT, args.layout)   # i.i.d. synthetic values: the same storage read in the other order
        if args.train_step:
            c.set_option(linattn.OPT_REUSE_STATE, 1)
        c.set_feature_map(s["Wq"], s["Wk"])
        ctxs.append(c)
    stream = torch.cuda.current_stream()

    def step(i):
        j = i % rotate
        if args.train_step:
            ctxs[j].forward(sets[j]["q"], sets[j]["k"], sets[j]["v"], out=outs[j], stream=stream)
            ctxs[j].backward(sets[j]["q"], sets[j]["k"], sets[j]["v"], douts[j], stream=stream)
        elif douts is not None:
            ctxs[j].backward(sets[j]["q"], sets[j]["k"], sets[j]["v"], douts[j], stream=stream)
        elif softs is None:
            ctxs[j].forward(sets[j]["q"], sets[j]["k"], sets[j]["v"], out=outs[j], stream=stream)
        else:
            ctxs[j].forward_mixed(sets[j]["q"], sets[j]["k"], sets[j]["v"], softs[j], args.mixed, out=outs[j], stream=stream)

    # every context's first call (function attributes, the backward's workspace allocation) happens before the warm-up
    for i in range(rotate):
        step(i)
    ctxs[0].check()
    launches_per_step = ctxs[0].last_launch_count()
    if args.train_step:   # one more step on the first context, counting both calls (its very first backward also split S into hi + lo)
        ctxs[0].forward(sets[0]["q"], sets[0]["k"], sets[0]["v"], out=outs[0], stream=stream)
        launches_per_step = ctxs[0].last_launch_count()
        ctxs[0].backward(sets[0]["q"], sets[0]["k"], sets[0]["v"], douts[0], stream=stream)
        launches_per_step += ctxs[0].last_launch_count()

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the W warm-up steps run right before the timed region, with no host-side pause in between in which the GPU could
    # fall back to its idle clocks
    for i in range(args.warmup):
        step(i)
    ladist.barrier()
    torch.cuda.synchronize()
    t_region0 = time.time()
    ev0.record(stream)
    for i in range(args.steps):
        step(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    t_region1 = time.time()
    ladist.barrier()
    ms_total = ladist.max_over_ranks(ev0.elapsed_time(ev1))
    for c in ctxs:
        c.check()
    ms_step = ms_total / args.steps
    tokens_per_step = ladist.sum_over_ranks(float(B * n))
    value = tokens_per_step / (ms_step * 1e-3)

    # Second pass over the same steps, for the spread: an event pair around every step (around every block of 50 when
    # there are more than 400), median and minimum.  The events sit between launches, so these are a little above the
    # un-instrumented mean; `value` and `roofline.achieved` come from the first region only.
    block = 1 if args.steps <= 400 else 50
    nblk = max(1, args.steps // block)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(nblk + 1)]
    torch.cuda.synchronize()
    marks[0].record(stream)
    for bi in range(nblk):
        for i in range(bi * block, (bi + 1) * block):
            step(i)
        marks[bi + 1].record(stream)
    torch.cuda.synchronize()
    per_step = sorted(marks[bi].elapsed_time(marks[bi + 1]) / block for bi in range(nblk))
    spread = {"median_ms": statistics.median(per_step), "min_ms": per_step[0], "max_ms": per_step[-1],
              "events_around": f"every {'step' if block == 1 else f'{block} steps'}", "samples": nblk}
    clocks = sampler.stop(t_region0, t_region1) if rank == 0 else None
    if clocks is not None:
        clocks["timed_region_s"] = t_region1 - t_region0

    # per-kernel durations: a second pass of the same steps with events around every launch
    e = 2 if wl.dtype == "bf16" else 4
    # tensors of [B,H,n,d] one step must move: q, k, v in and o out; + the softmax branch for Eq. 8; for the
    # gradients q, k, v, dO in and dq, dk, dv out
    alg_total = (11.0 if args.train_step else 7.0 if douts is not None else 4.0 if softs is None else 5.0) * B * H * n * d * e
    for c in ctxs:
        c.set_option(linattn.OPT_PROFILE, 1)
    for i in range(min(args.steps, 300)):
        step(i)
    torch.cuda.synchronize()
    kernels = ctxs[0].kernel_times()  # [(name, mean ms, launches, algorithmic bytes per launch)]
    for c in ctxs:
        c.set_option(linattn.OPT_PROFILE, 0)
    peaks = load_peaks()
    dom = max(kernels, key=lambda kt: kt["ms"])
    if softs is not None:
        dom["bytes"] += 1.0 * B * H * n * d * e   # the softmax branch's output is read once more
    # Average launch duration of the dominant kernel.  When a step is ONE launch, that is the timed region itself (CUDA
    # events around it) divided by its launches: no event sits between launches and the clocks are those of the timed
    # region.  With several kernels per step it comes from the second pass, which has events around every launch.
    if launches_per_step == 1:
        kernel_ms = ms_step
        timing = "timed region (CUDA events around it) / launches in it; the step is this one kernel"
    else:
        kernel_ms = dom["ms"]
        timing = "mean over a second pass of the timed steps with CUDA events around each launch"
    achieved = dom["bytes"] / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom["name"], "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                "peak_nominal": 8000.0, "frac_of_nominal": achieved / 8000.0, "traffic": None,
                "kernel_ms": kernel_ms, "algorithmic_bytes_per_launch": dom["bytes"],
                "timing": timing, "step_spread": spread,
                "kernels": kernels,
                "whole_step": {"achieved": alg_total / (ms_step * 1e-3) / 1e9,
                               "frac": alg_total / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "frac_of_nominal_8TBs": alg_total / (ms_step * 1e-3) / 1e9 / 8000.0,
                               "algorithmic_bytes": alg_total}}
    # recorded at config 2, default layout, Eq. 6 feature map only
    plain = softs is None and args.phi == "hedgehog" and args.config == 2 and args.layout == 0
    roofline["traffic"] = recorded_traffic(dom["name"]) if plain else None

    # end to end through the host-buffer entry point: pinned host tensors in, pinned host tensor out
    pin = {k_: host0[k_].pin_memory() for k_ in ("q", "k", "v")}
    hout = torch.empty_like(host0["q"]).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    ctxs[0].forward_host(pin["q"], pin["k"], pin["v"], hout, stream=stream)  # allocates the staging buffers
    ladist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        ctxs[0].forward_host(pin["q"], pin["k"], pin["v"], hout, stream=stream)
    torch.cuda.synchronize()
    e2e_s = ladist.max_over_ranks(time.perf_counter() - t0) / e2e_steps
    nbytes = B * H * n * d * e
    e2e = {"value": tokens_per_step / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 3 * nbytes, "d2h_bytes_per_step": nbytes,
           "ms_per_step": 1e3 * e2e_s, "steps": e2e_steps, "entry_point": "linattn_forward_host (pinned host buffers)"}

    if douts is not None:
        e2e["note"] = "this is the forward's host-buffer entry point; the backward has no host-buffer form"
    result = {
        "metric": ("linear-attention fwd+bwd tokens/s" if args.train_step else "linear-attention bwd tokens/s" if douts is not None else "mixed-attention (Eq. 8) fwd tokens/s" if softs is not None
                   else "linear-attention (ReLU kernel function) fwd tokens/s" if args.phi == "relu" else METRIC), "value": value, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": config_dict(args, wl), "kernel_path": args.path,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
    }

    if rank == 0 and world == 1 and not args.no_baselines:
        cb = time_oracle(host0, budget_s=20.0)
        result["cpu_baseline"] = {"value": cb["value"], "unit": UNIT, "cores": cb["cores"], "kind": "oracle", "sample": cb["sample"]}
        # context only: softmax attention of the same shape through torch SDPA
        try:
            s = sets[0]
            for _ in range(2):
                torch.nn.functional.scaled_dot_product_attention(s["q"], s["k"], s["v"])
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            for _ in range(5):
                torch.nn.functional.scaled_dot_product_attention(s["q"], s["k"], s["v"])
            a1.record()
            torch.cuda.synchronize()
            sd = a0.elapsed_time(a1) / 5
            result["sdpa_baseline"] = {"ms_per_step": sd, "value": B * n / (sd * 1e-3), "unit": UNIT,
                                       "kind": "torch scaled_dot_product_attention, same [B,H,n,d] bf16, non-causal"}
        except Exception as exc:  # context number only
            result["sdpa_baseline"] = {"error": str(exc)[:200]}

    for c in ctxs:
        c.destroy()
    if rank == 0:
        print(json.dumps(result))
    ladist.shutdown()


if __name__ == "__main__":
    main()
