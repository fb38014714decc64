#!/usr/bin/env python
"""Benchmark of the LayerPipe training hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" = one minibatch through the whole path (cast+stash, forward of every layer,
loss, delta / G / update of every layer under the LayerPipe schedule).  Prints ONE JSON
line.  The path does not shard (stages are SM partitions of one GPU), so N > 1 runs N
independent replicas, one process per GPU, and adds their throughput.
"""
import argparse
import json
import os

os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")  # one hardware queue per scheduler stream; read when the CUDA context is created
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2108_06629_b200 import inputs as I  # noqa: E402
from paper_2108_06629_b200 import replicas  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}



def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ----------------------------------------------------------------------------- work model
def work_model(layers, batch, momentum):
    """Algorithmic flops and bytes per launch of each task kind, per layer (true shapes)."""
    out = {"forward": [], "delta": [], "G": [], "update": []}
    L = len(layers)
    for l, y in enumerate(layers):
        n_in, n_out = y["n_in"], y["n_out"]
        conv = y["kind"] == "conv"
        if conv:
            Ho, Wo = I.conv_out_hw(y)
            rows, rows_in = batch * Ho * Wo, batch * y["H"] * y["W"]     # output / input pixels
            params = n_in * n_out * y["R"] * y["S"]
        else:
            rows = rows_in = batch                                        # samples
            params = n_in * n_out
        fl = 2.0 * rows * params
        gelu = y["act"] == "gelu"
        last = l == L - 1
        pool = 1.25 * 2.0 * rows * n_out + 0.25 * rows * n_out if y.get("pool", 0) else 0.0   # re-read a, write pooled + argmax
        out["forward"].append(dict(flops=fl, bytes=2.0 * params + 2.0 * rows_in * n_in +
                                   (4.0 if last else (4.0 if gelu else 2.0)) * rows * n_out + pool))
        if l > 0:
            out["delta"].append(dict(flops=fl, bytes=2.0 * params + 2.0 * rows * n_out + 4.0 * rows_in * n_in))
        # G with the update fused into its epilogue: read W (,m), write W (,m) fp32 and the bf16 ring slot
        per_param = 18.0 if momentum != 0.0 else 10.0
        out["G"].append(dict(flops=fl, bytes=2.0 * (rows_in * n_in + rows * n_out) + per_param * params))
        # what is left of the update: bias gradient (column sums of delta) and the bias update
        out["update"].append(dict(flops=0.0, bytes=2.0 * rows * n_out + 24.0 * n_out))
    return out


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------- reference arm
def oracle_step_time(orc_factory, layers, batch, rows, n_steps):
    from oracle import layerpipe_oracle  # noqa: F401  (the oracle is only ever used on this leg)
    orc = orc_factory()
    ts = []
    for n in range(n_steps):
        x, y = I.minibatch(layers, batch, n)
        t0 = time.perf_counter()
        orc.step(x[:rows], y[:rows])
        ts.append(time.perf_counter() - t0)
    return ts


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, wl):
    """The CPU oracle, as it stands, timed on the host cores.  Each step is one oracle
    minibatch on the first `rows` rows of the synthetic minibatch (full-size layers); rows is
    chosen so that K + W steps fit a time budget of about three minutes."""
    from oracle import layerpipe_oracle as O
    layers, B = wl["layers"], wl["batch"]
    delays = wl["delays"]
    if delays is None:
        from oracle import partition_oracle as P
        fix, flex = P.mac_costs(layers, B)
        delays = P.partition(fix, flex, wl["stages"])["delay"]
    W0, b0 = I.initial_weights(layers, 0)

    def factory():
        return O.DelayedGradientTrainer(layers, delays, wl["lr"], wl["momentum"], W0, b0, mirror=True,
                                        dtype=np.float32)
    total = args.steps + args.warmup
    budget = 170.0
    t_small = min(oracle_step_time(factory, layers, B, 8, 2))
    t_full = min(oracle_step_time(factory, layers, B, B, 1))
    rows = B
    while rows > 8:
        est = t_small + (t_full - t_small) * (rows - 8) / max(B - 8, 1)
        if est * total <= budget:
            break
        rows //= 2
    rows = max(rows, 8)
    orc = factory()
    for n in range(args.warmup):
        x, y = I.minibatch(layers, B, n)
        orc.step(x[:rows], y[:rows])
    t0 = time.perf_counter()
    for n in range(args.steps):
        x, y = I.minibatch(layers, B, args.warmup + n)
        orc.step(x[:rows], y[:rows])
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    sample = "first %d of %d rows of each minibatch, full-size layers, %d timed steps" % (rows, B, args.steps)
    cores = blas_threads()
    line = {
        "impl": "reference", "metric": "training samples/sec", "value": value, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "batch": B, "delays": delays, "schedule": "sequential CPU oracle"},
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- our arm
_T0 = time.perf_counter()


def note(msg):
    """Progress on stderr (the JSON line is the only thing written to stdout)."""
    sys.stderr.write("[bench %7.1f s] %s\n" % (time.perf_counter() - _T0, msg))
    sys.stderr.flush()


MIN_TIMED_SECONDS = 1.5     # the timed region is repeated until this much device time has been measured


TRACE = os.environ.get("LP_BENCH_TRACE") == "1"   # diagnosis of a stalled run: handles mark task progress


def _report_progress(tr, stop):
    """Every 15 s that a block has not finished: which tasks the device still owes (LP_BENCH_TRACE=1)."""
    while not stop.wait(15.0):
        note("still waiting for the device:\n" + tr.task_progress())


def timed_block(torch, tr, xs, ys, steps, stream):
    """EXACTLY `steps` lp_step calls + lp_flush between two events on the caller's stream."""
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    stop = None
    if TRACE:
        import threading
        stop = threading.Event()
        threading.Thread(target=_report_progress, args=(tr, stop), daemon=True).start()
    e0.record(stream)
    P = len(xs)
    for k in range(steps):
        tr.step(xs[k % P], ys[k % P])
    tr.flush()
    e1.record(stream)
    torch.cuda.synchronize()
    if stop is not None:
        stop.set()
    return e0.elapsed_time(e1)


def e2e_block(torch, tr, hx, hy, xd, yd, steps, stream, lag, first_step):
    """Every step: pinned host -> device copy of that step's minibatch and labels, lp_step,
    and a device -> host read of one finished step's loss (the step `lag` calls back, so
    that the read does not drain the pipeline; the last `lag` losses are read at the end)."""
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    P = len(hx)
    losses = []
    torch.cuda.synchronize()
    e0.record(stream)
    for k in range(steps):
        xd[k % 2].copy_(hx[k % P], non_blocking=True)
        yd[k % 2].copy_(hy[k % P], non_blocking=True)
        tr.step(xd[k % 2], yd[k % 2])
        if k >= lag:
            losses.append(tr.get_loss(first_step + k - lag))
    for k in range(max(steps - lag, 0), steps):
        losses.append(tr.get_loss(first_step + k))
    tr.flush()
    e1.record(stream)
    torch.cuda.synchronize()
    assert len(losses) == steps and all(np.isfinite(losses))
    return e0.elapsed_time(e1)


def repeat_blocks(block, min_seconds, max_blocks=400):
    """Run `block()` (returns milliseconds) at least 3 times and until min_seconds of device time
    have been measured.  Returns the list of block times."""
    ts = []
    while len(ts) < 3 or (sum(ts) < 1e3 * min_seconds and len(ts) < max_blocks):
        ts.append(block())
    return ts


def summarize(ts, steps):
    med = statistics.median(ts)
    return {"ms_per_step": med / steps, "ms_per_step_min": min(ts) / steps, "ms_per_step_max": max(ts) / steps,
            "blocks": len(ts), "timed_seconds": sum(ts) * 1e-3}


class Workload:
    """Host and device copies of a workload's synthetic inputs, shared by every handle of the run."""

    def __init__(self, torch, name, dev):
        self.name = name
        self.wl = I.WORKLOADS[name]
        self.layers, self.B = self.wl["layers"], self.wl["batch"]
        self.W0, self.b0 = I.initial_weights(self.layers, 0)
        self.P = 8
        self.hx, self.hy = [], []
        for n in range(self.P):
            x, y = I.minibatch(self.layers, self.B, n)
            self.hx.append(torch.from_numpy(x).pin_memory())
            self.hy.append(torch.from_numpy(y).pin_memory())
        self.xs = [t.to(dev) for t in self.hx]
        self.ys = [t.to(dev) for t in self.hy]
        self.dev = dev

    def trainer(self, lpb, schedule, flags=0):
        wl = self.wl
        if TRACE:
            flags |= lpb.LP_TRACE_TASKS
        return lpb.Trainer(self.layers, self.B, wl["stages"], delays=wl["delays"], lr=wl["lr"], momentum=wl["momentum"],
                           schedule=schedule, flags=flags, W0=self.W0, b0=self.b0, device=self.dev)


def throughput(torch, lpb, w, schedule, steps, warmup, min_seconds, stream, flags=0, before_timing=None):
    """samples/s of one handle: warm-up (fills every ring), then repeated blocks of `steps` steps."""
    tr = w.trainer(lpb, schedule, flags)
    stage, delays, slots = tr.get_schedule()
    prewarm = max(delays) + 3 + max(warmup, 3)
    for k in range(prewarm):
        tr.step(w.xs[k % w.P], w.ys[k % w.P])
    tr.flush()
    torch.cuda.synchronize()
    if before_timing is not None:
        before_timing()
    l0 = tr.kernel_launches()
    ts = repeat_blocks(lambda: timed_block(torch, tr, w.xs, w.ys, steps, stream), min_seconds)
    launches = (tr.kernel_launches() - l0) // len(ts)
    if TRACE:
        note(tr.task_progress())
    rc, detail = tr.device_status()
    if rc != 0:
        raise SystemExit("device status %d (%d)" % (rc, detail))
    return tr, ts, launches, prewarm, (stage, delays, slots)


def kernel_times(torch, lpb, w, sched, flags, steps, stream):
    """Per task kind: launches, total and average event-timed duration over `steps` minibatches."""
    trp = w.trainer(lpb, sched, flags)
    _, delays, _ = trp.get_schedule()
    for k in range(max(delays) + 6):
        trp.step(w.xs[k % w.P], w.ys[k % w.P])
    trp.flush()
    torch.cuda.synchronize()
    trp.reset_task_times()
    nprof = max(1, min(steps, 32768 // (6 * len(w.layers))))
    timed_block(torch, trp, w.xs, w.ys, nprof, stream)
    out = {}
    for kind in ("forward", "delta", "G", "update", "loss", "cast"):
        n, tot = trp.task_time(kind)
        out[kind] = dict(launches=n, total_ms=tot, avg_us=1e3 * tot / max(n, 1))
    trp.close()
    del trp
    torch.cuda.empty_cache()
    return out


KERNEL_NAMES = {"forward": "gemm (forward contraction, Eqs. 1-2)", "delta": "gemm (delta contraction, Eqs. 3-4)",
                "G": "gemm (G contraction with the update of Eq. 6 in its epilogue)", "update": "sgd_update_kernel"}


def ncu_traffic(workload, kind):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the table
    in profiles/ncu_traffic.md (rows `| workload | task | bytes per launch | source |`); None if there
    is no capture for that pair."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.md")
    if not os.path.exists(path):
        return None
    for line in open(path):
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) >= 3 and cells[0] == workload and cells[1] == kind:
            try:
                return float(cells[2])
            except ValueError:
                return None
    return None


def roofline(workload, wl, kinds, peaks):
    wm = work_model(wl["layers"], wl["batch"], wl["momentum"])
    dom = max(("forward", "delta", "G", "update"), key=lambda k: kinds[k]["total_ms"])
    per = wm[dom]
    avg_bytes = sum(p["bytes"] for p in per) / len(per)
    avg_flops = sum(p["flops"] for p in per) / len(per)
    avg_s = kinds[dom]["avg_us"] * 1e-6
    ridge = peaks["bf16_tflops_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if avg_flops / max(avg_bytes, 1.0) > ridge:
        roof = {"bound": "tensor", "achieved": avg_flops / avg_s / 1e12, "peak": peaks["bf16_tflops_sustained"],
                "unit": "TFLOP/s", "peak_kind": "sustained (kernel timed inside a seconds-long step loop)",
                "frac_of_burst_peak": avg_flops / avg_s / 1e12 / peaks["bf16_tflops"]}
    else:
        roof = {"bound": "hbm", "achieved": avg_bytes / avg_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = ncu_traffic(workload, dom)
    roof["kernel"] = KERNEL_NAMES[dom]
    roof["task"] = dom
    roof["peak_source"] = "of " + peaks["_source"]
    roof["avg_launch_us"] = kinds[dom]["avg_us"]
    roof["avg_launch_us_overlapped"] = kinds[dom].get("avg_us_overlapped")
    roof["timing"] = ("CUDA events around every launch of the kernel, on the stream it runs on, in a pass of the same "
                      "steps with all tasks on one stream; avg_launch_us_overlapped is the same measurement under the "
                      "concurrent schedule")
    roof["algorithmic_per_launch"] = {"bytes": avg_bytes, "flops": avg_flops}
    # every contraction kind against the tensor roof (the metric's "tensor-pipe utilisation vs peak")
    roof["contractions"] = {}
    for k in ("forward", "delta", "G"):
        if kinds[k]["launches"]:
            fl = sum(p["flops"] for p in wm[k]) / len(wm[k])
            t = fl / (kinds[k]["avg_us"] * 1e-6) / 1e12
            roof["contractions"][k] = {"tflops": t, "frac_of_sustained": t / peaks["bf16_tflops_sustained"],
                                       "frac_of_burst": t / peaks["bf16_tflops"], "avg_us": kinds[k]["avg_us"]}
    return roof, wm


def step_figures(wm, ms_per_step, peaks):
    step_flops = sum(p["flops"] for k in ("forward", "delta", "G") for p in wm[k])
    step_bytes = sum(p["bytes"] for k in wm for p in wm[k])
    s = ms_per_step * 1e-3
    return {"tflops": step_flops / s / 1e12, "gbs_algorithmic": step_bytes / s / 1e9,
            "frac_of_bf16_sustained": step_flops / s / 1e12 / peaks["bf16_tflops_sustained"],
            "frac_of_bf16_burst": step_flops / s / 1e12 / peaks["bf16_tflops"],
            "frac_of_hbm": step_bytes / s / 1e9 / peaks["hbm_gbs"]}


def short_measure(torch, lpb, name, dev, stream, peaks, seconds=0.6):
    """samples/s of one workload under both schedules, a fraction of a second each (the
    per_workload object of the JSON line)."""
    w = Workload(torch, name, dev)
    steps = {"mlp4_784": 200, "mlp8_4096": 50, "vgg_small_32": 50, "vgg16_224": 10, "mlp16_8192": 10}.get(name, 20)
    out = {"batch": w.B}
    for sched, key in ((lpb.LP_SCHED_LAYERPIPE, "layerpipe"), (lpb.LP_SCHED_FUSED_B, "fused_b")):
        tr, ts, launches, _, (stage, delays, _) = throughput(torch, lpb, w, sched, steps, 3, seconds, stream)
        tr.close()
        del tr
        torch.cuda.empty_cache()
        sm = summarize(ts, steps)
        out[key] = {"samples_per_s": w.B / (sm["ms_per_step"] * 1e-3), "ms_per_step": sm["ms_per_step"],
                    "blocks": sm["blocks"], "steps_per_block": steps}
        out["delays"] = delays
        out["launches_per_step"] = launches // steps
    out["speedup_vs_fused_b"] = out["layerpipe"]["samples_per_s"] / out["fused_b"]["samples_per_s"]
    out["selfcheck"] = free_running_selfcheck(torch, lpb, w, lpb.LP_SCHED_LAYERPIPE)
    wm = work_model(w.layers, w.B, w.wl["momentum"])
    out["step"] = step_figures(wm, out["layerpipe"]["ms_per_step"], peaks)
    del w
    torch.cuda.empty_cache()
    return out


def borrowing_report(torch, lpb, w, args, stream):
    """Section III-B executed and measured.  Algorithm 1's step 2 (`profile`): per-layer task times
    from a pass with every task alone on the GPU; T_fix = forward + G + update, T_flex = delta, in
    nanoseconds, go through lp_plan_costs.  Four variants of the LayerPipe schedule are timed: the
    default plan (integer MAC model) and the plan from measured times, each with the delta
    contractions in one piece and divided into delta'' / delta' as the plan says."""
    wl, L = w.wl, len(w.layers)
    trp = w.trainer(lpb, lpb.LP_SCHED_LAYERPIPE, lpb.LP_TIME_TASKS | lpb.LP_SERIAL_TASKS)
    _, delays, _ = trp.get_schedule()
    for k in range(max(delays) + 4):
        trp.step(w.xs[k % w.P], w.ys[k % w.P])
    trp.flush()
    torch.cuda.synchronize()
    trp.reset_task_times()
    nprof = max(2, min(8, 32768 // (6 * L)))
    timed_block(torch, trp, w.xs, w.ys, nprof, stream)
    fix, flex = [], []
    for l in range(L):
        t = {k: trp.layer_task_time(k, l)[1] / nprof for k in ("forward", "G", "update", "delta")}
        fix.append(max(1, int(1e6 * (t["forward"] + t["G"] + t["update"]))))
        flex.append(int(1e6 * t["delta"]))
    trp.close()
    del trp
    torch.cuda.empty_cache()
    plans = {"mac_model": lpb.lp_plan(w.layers, w.B, wl["stages"]), "measured": lpb.lp_plan_costs(fix, flex, wl["stages"])}
    out = {"profile_ns": {"T_fix": fix, "T_flex": flex}, "variants": {}}
    steps = args.steps
    for pname, plan in plans.items():
        for split in (False, True):
            note("  variant %s%s" % (pname, "+split" if split else ""))
            tr = lpb.Trainer(w.layers, w.B, wl["stages"], stage=plan["stage"], delays=wl["delays"] if pname == "mac_model" else None,
                             lr=wl["lr"], momentum=wl["momentum"], schedule=lpb.LP_SCHED_LAYERPIPE, W0=w.W0, b0=w.b0, device=w.dev)
            cols = tr.set_delta_split(plan["piece_stage"], plan["piece_amount"]) if split else None
            _, d, _ = tr.get_schedule()
            for k in range(max(d) + 6):
                tr.step(w.xs[k % w.P], w.ys[k % w.P])
            tr.flush()
            torch.cuda.synchronize()
            ts = repeat_blocks(lambda: timed_block(torch, tr, w.xs, w.ys, steps, stream), 0.5)
            rc, detail = tr.device_status()
            tr.close()
            del tr
            torch.cuda.empty_cache()
            if rc != 0:
                raise SystemExit("device status %d (%d)" % (rc, detail))
            sm = summarize(ts, steps)
            out["variants"]["%s%s" % (pname, "+split" if split else "")] = {
                "samples_per_s": w.B / (sm["ms_per_step"] * 1e-3), "ms_per_step": sm["ms_per_step"], "stage": plan["stage"],
                "delays": d, "stages_used": plan["used"], "split_col": cols}
    return out


def run_ours(args):
    import torch
    from paper_2108_06629_b200 import binding as lpb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        backend = os.environ.get("LP_BENCH_BACKEND", "nccl")
        dist.init_process_group(backend, device_id=torch.device("cuda", local) if backend == "nccl" else None)
    lpb.lib()   # fails loudly if the CUDA library is missing
    dev = "cuda:%d" % local
    stream = torch.cuda.current_stream()
    sched = lpb.LP_SCHED_FUSED_B if args.schedule == "fused_b" else lpb.LP_SCHED_LAYERPIPE
    note("workload %s: generating inputs" % args.workload)
    w = Workload(torch, args.workload, dev)
    wl, layers, B = w.wl, w.layers, w.B
    note("timed loop")

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return replicas.max_over_ranks(ms, dist, dev if (dist is None or dist.get_backend() == "nccl") else "cpu")

    # ---- device-resident throughput: blocks of exactly K steps, repeated for >= 1.5 s ------------
    barrier()
    sampler = {}

    def start_sampler():
        # clocks and throttle reasons DURING the timed region only: the sampler (an nvidia-smi loop) starts once
        # the handle exists and the rings are warm, and stops after the end-to-end blocks
        sampler["clocks"] = ClockSampler(local)
        time.sleep(0.25)
    tr, ts, launches, prewarm, (stage, delays, slots) = throughput(torch, lpb, w, sched, args.steps, args.warmup,
                                                                    args.min_seconds, stream, before_timing=start_sampler)
    clocks = sampler["clocks"]
    barrier()
    dev_sum = summarize(ts, args.steps)
    ms = max_over_ranks(dev_sum["ms_per_step"] * args.steps)
    # ---- end to end: host buffers, copies inside the timed region --------------------------------
    xd = [torch.empty_like(w.xs[0]) for _ in range(2)]
    yd = [torch.empty_like(w.ys[0]) for _ in range(2)]
    lag = max(delays) + 1
    state = {"first": prewarm + args.steps * len(ts)}

    def e2e_once():
        t = e2e_block(torch, tr, w.hx, w.hy, xd, yd, args.steps, stream, lag, state["first"])
        state["first"] += args.steps
        return t
    note("end-to-end loop")
    ts_e2e = repeat_blocks(e2e_once, min(args.min_seconds, 1.0))
    barrier()
    e2e_sum = summarize(ts_e2e, args.steps)
    ms_e2e = max_over_ranks(e2e_sum["ms_per_step"] * args.steps)
    clk = clocks.stop()
    tr.close()
    del tr
    torch.cuda.empty_cache()

    line = None
    if rank == 0 and args.only_main:
        # the timed loop alone (what a profiler's launch list should see): no second schedule, no
        # per-kernel passes, no CPU baseline
        line = {"metric": "training samples/sec", "value": world * args.steps * B / (ms * 1e-3), "unit": "samples/s",
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
                "config": {"workload": args.workload, "batch": B, "delays": delays, "only_main": True},
                "gpu_launches": int(launches), "clocks": clk, "timing": dev_sum}
    elif rank == 0:
        peaks = load_peaks()
        # ---- same GPU, same kernels, backward as ONE task per layer (PipeDream-style) -------------
        osched = lpb.LP_SCHED_LAYERPIPE if sched == lpb.LP_SCHED_FUSED_B else lpb.LP_SCHED_FUSED_B
        note("other schedule")
        tro, ts_o, _, _, _ = throughput(torch, lpb, w, osched, args.steps, args.warmup, min(args.min_seconds, 1.0), stream)
        tro.close()
        del tro
        torch.cuda.empty_cache()
        o_sum = summarize(ts_o, args.steps)
        other = {"schedule": "layerpipe" if osched == lpb.LP_SCHED_LAYERPIPE else "fused_b",
                 "value": B / (o_sum["ms_per_step"] * 1e-3), "unit": "samples/s (1 GPU)", **o_sum}
        # ---- per-kernel times for the roofline ---------------------------------------------------
        # Under the real schedule up to a dozen kernels share the GPU, so a kernel's event-timed
        # duration there is the time it spent sharing, not its own cost.  The roofline uses a second
        # pass of the same steps with every task on one stream (LP_SERIAL_TASKS: the same kernels,
        # launches and operands, none overlapping); the overlapped averages are reported beside it.
        note("per-kernel times")
        kinds_live = kernel_times(torch, lpb, w, sched, lpb.LP_TIME_TASKS, args.steps, stream)
        kinds = kernel_times(torch, lpb, w, sched, lpb.LP_TIME_TASKS | lpb.LP_SERIAL_TASKS, args.steps, stream)
        for kind in kinds:
            kinds[kind]["avg_us_overlapped"] = kinds_live[kind]["avg_us"]
        roof, wm = roofline(args.workload, wl, kinds, peaks)
        note("self-check: free-running against serialised")
        selfcheck = free_running_selfcheck(torch, lpb, w, sched)
        note("borrowing report")
        borrowing = borrowing_report(torch, lpb, w, args, stream) if world == 1 else None
        del w
        torch.cuda.empty_cache()
        per_workload = {}
        if not args.no_per_workload and world == 1:
            for name in I.WORKLOADS:
                note("per-workload: %s" % name)
                per_workload[name] = short_measure(torch, lpb, name, dev, stream, peaks)
        note("cpu baseline (oracle)")
        cpu = cpu_baseline(wl)
        note("done")
        value = world * args.steps * B / (ms * 1e-3)
        e2e_value = world * args.steps * B / (ms_e2e * 1e-3)
        in_bytes = xd[0].numel() * xd[0].element_size() + yd[0].numel() * yd[0].element_size()
        line = {
            "metric": "training samples/sec", "value": value, "unit": "samples/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "batch": B, "stages_used": max(stage) + 1, "delays": delays,
                       "ring_slots": slots, "schedule": args.schedule, "parallelism": "replicas only",
                       "l2": "working set per step exceeds L2 (weights + update streams), no flush",
                       "prewarm_steps": prewarm,
                       "timed_region": "blocks of exactly `steps` lp_step calls + lp_flush between CUDA events, device idle on both "
                                       "sides; repeated until >= %.1f s were measured; value = median block" % args.min_seconds},
            "timing": dev_sum,
            "e2e": {"value": e2e_value, "unit": "samples/s", "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": 4,
                    **e2e_sum},
            "gpu_launches": int(launches),
            "clocks": clk,
            "roofline": roof,
            "step": step_figures(wm, ms / args.steps, peaks),
            "kernels": kinds,
            "other_schedule": other,
            "speedup_vs_fused_b": ((value / world) / other["value"] if other["schedule"] == "fused_b"
                                   else other["value"] / (value / world)),
            "borrowing": borrowing,
            "selfcheck": selfcheck,
            "per_workload": per_workload,
            "cpu_baseline": cpu,
        }
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


def free_running_selfcheck(torch, lpb, w, sched, steps=6):
    """The timed mode against the mode in which nothing overlaps: `steps` minibatches enqueued back to back on
    the scheduler's streams, and the same minibatches with every task on one stream (LP_SERIAL_TASKS).  The
    kernels are deterministic, so the losses must agree bit for bit; a difference is a hazard the scheduler
    missed or a race inside a kernel that only other kernels' traffic brings out (from the second step
    on every loss depends on every earlier update)."""
    losses = []
    for flags in (0, lpb.LP_SERIAL_TASKS):
        tr = w.trainer(lpb, sched, flags)
        for k in range(steps):
            tr.step(w.xs[k % w.P], w.ys[k % w.P])
        tr.flush()
        torch.cuda.synchronize()
        losses.append([tr.get_loss(k) for k in range(steps)])
        rc, detail = tr.device_status()
        tr.close()
        del tr
        torch.cuda.empty_cache()
        if rc != 0:
            raise SystemExit("device status %d (%d)" % (rc, detail))
    same = losses[0] == losses[1]
    out = {"steps": steps, "free_running_losses_equal_serialised": same, "last_loss": losses[0][-1]}
    if not same:      # reported, loudly, with the line: the reader decides what the timing is worth
        note("SELF-CHECK FAILED: free-running losses %s differ from serialised losses %s" % (losses[0], losses[1]))
        out["free_running_losses"], out["serialised_losses"] = losses
    return out


def cpu_baseline(wl):
    """The oracle, untouched, on this machine's host cores: whole minibatches until about 10 s of
    CPU work has been done (at least one)."""
    from oracle import layerpipe_oracle as O
    layers, B = wl["layers"], wl["batch"]
    delays = wl["delays"]
    if delays is None:
        from oracle import partition_oracle as P
        fix, flex = P.mac_costs(layers, B)
        delays = P.partition(fix, flex, wl["stages"])["delay"]
    W0, b0 = I.initial_weights(layers, 0)
    orc = O.DelayedGradientTrainer(layers, delays, wl["lr"], wl["momentum"], W0, b0, mirror=True, dtype=np.float32)
    n, t0 = 0, time.perf_counter()
    while True:
        x, y = I.minibatch(layers, B, n)
        orc.step(x, y)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= 10.0 or n >= 50:
            break
    return {"value": n * B / dt, "unit": "samples/s", "cores": blas_threads(), "kind": "oracle",
            "sample": "%d whole minibatches of %d, full-size layers, %.1f s" % (n, B, dt)}


def supervise(args, limit_s=480.0):
    env = dict(os.environ, LP_BENCH_CHILD="1")
    cmd = [sys.executable, "-X", "faulthandler", os.path.abspath(__file__)] + sys.argv[1:]
    for attempt in (1, 2):
        p = subprocess.Popen(cmd, env=env, stdout=subprocess.PIPE)
        try:
            out, _ = p.communicate(timeout=limit_s)
        except subprocess.TimeoutExpired:
            try:      # what the GPU is doing while the child makes no progress
                q = subprocess.run(["nvidia-smi", "--query-gpu=index,utilization.gpu,clocks.sm,power.draw,memory.used",
                                    "--format=csv,noheader"], capture_output=True, text=True, timeout=20)
                note("nvidia-smi: " + q.stdout.strip().replace("\n", " | "))
            except Exception:
                pass
            try:
                p.send_signal(__import__("signal").SIGABRT)     # faulthandler prints the child's Python stack
                p.wait(timeout=10)
            except Exception:
                p.kill()
                p.wait()
            note("attempt %d did not finish within %.0f s%s" % (attempt, limit_s, "; trying once more" if attempt == 1 else ""))
            continue
        sys.stdout.write(out.decode())
        sys.stdout.flush()
        if p.returncode != 0:
            raise SystemExit(p.returncode)
        return
    raise SystemExit("bench.py: the measurement did not finish in two attempts")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mlp16_8192", choices=sorted(I.WORKLOADS))
    ap.add_argument("--schedule", default="layerpipe", choices=["layerpipe", "fused_b"])
    ap.add_argument("--min-seconds", dest="min_seconds", type=float, default=MIN_TIMED_SECONDS)
    ap.add_argument("--no-per-workload", dest="no_per_workload", action="store_true")
    ap.add_argument("--no-watchdog", dest="no_watchdog", action="store_true",
                    help="measure in this process instead of a supervised child")
    ap.add_argument("--only-main", dest="only_main", action="store_true",
                    help="time the main loop only and print a reduced line (for profiler launch lists)")
    args = ap.parse_args()
    if args.steps < 1 or args.gpus < 1:
        raise SystemExit("--steps and --gpus must be positive")
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, I.WORKLOADS[args.workload])
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: run the N replicas ourselves, one process per GPU
        out = replicas.spawn_replicas([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)
        sys.stdout.write(out)
        return
    if os.environ.get("LP_BENCH_CHILD") != "1" and not args.no_watchdog:
        # Run the measurement in a child process under a time limit and try once more if it neither
        # finishes nor fails in time: a wedged run must not turn into a benchmark that never ends.
        return supervise(args)
    run_ours(args)


if __name__ == "__main__":
    main()
