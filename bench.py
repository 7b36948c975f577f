"""Benchmark: images/s of the fused + pruned ResNet forward through the C-ABI library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config C] [--batch B] [--prune P]
                    [--no-sweep] [--no-cpu] [--no-latency] [--per-op]

Headline workload (default `--config 5`): ResNet-50, batch 128, 40 % of the inner bottleneck filters pruned by
L1 norm - the largest of the workload list that one GPU holds.  One step = one fp_forward of the whole fused
graph over one batch of synthetic, seeded images that are already in HBM.  Between timed steps L2 is flushed by
writing a 256 MiB buffer; each step is timed with CUDA events on the launching stream and the K step times are
summed.  The same JSON line also carries
  configs     the other workloads of the list, each measured the same way with fewer steps,
  latency     ResNet-50 at batch 1: p50 / p99 over 1000 graph replays (the paper's protocol, Sec. V-C),
  sustained   the headline run back to back for about a second without flushes (clock / power state under load),
  side_kernels  the memory-bound kernels of the headline against the HBM peak.
`--impl reference` times the CPU oracle on the host cores instead (a deliberately plain program).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "images/s of fused+pruned ResNet forward on 1 B200; % of BF16 tensor/HBM roofline"
UNIT = "images/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0}     # HGX B200 data sheet: HBM3e, dense BF16
HEADLINE_CONFIG = 5
SWEEP = [(1, None), (2, 0.0), (2, None), (2, 0.5), (3, None), (4, None), (6, None), (7, None)]   # (config, prune)
KIND_NAMES = ("conv", "maxpool", "head", "input")


def recorded_traffic(workload, kernel):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, or None when the kernel source has
    changed since the counters were taken (or there is no summary for this workload)."""
    import hashlib
    rec = os.path.join(ROOT, "profiles", f"{kernel}_{workload}.traffic.txt")
    src = os.path.join(ROOT, "paper_2010_16165_b200", "csrc", kernel.replace("_kernel", "") + ".cu")
    try:
        kv = dict(l.split(":", 1) for l in open(rec) if ":" in l and not l.startswith("#"))
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
        if kv["workload"].strip() != workload or not sha.startswith(kv["kernel_sha256_prefix"].strip()):
            return None
        return float(kv["traffic_bytes_per_launch"])
    except Exception:
        return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------
# multi-process plumbing (one process per GPU; the path has no collective: replicas of the
# same batch-sharded work, timing reduced as max over ranks)
# ------------------------------------------------------------------------------------------

def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def init_dist(backend):
    import torch.distributed as dist
    rank, world, _ = dist_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms, units, device="cpu"):
    """Whole-job figures: time = max over ranks, units = sum over ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def window(self, t0, t1):
        """Summary of the samples taken between the host times t0 and t1."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        inside = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.06] or [r for (_, r) in self.rows][-1:]
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
                for n, v in zip(names, f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------

def oracle_images_per_s(w, n_images, min_seconds=10.0):
    """The oracle as it stands: fused + pruned forward in fp64 on the host cores, over the first `n_images`
    images of the workload, repeated until about `min_seconds` of CPU work have been timed."""
    from oracle import fpo
    gp, _, _, _ = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios)
    x = w.x[:n_images]
    passes, total = 0, 0.0
    while passes == 0 or total < min_seconds:
        t = time.perf_counter()
        fpo.fused_forward(gp, x)
        total += time.perf_counter() - t
        passes += 1
    return n_images * passes / total, fpo.num_threads(), total, passes


def run_reference(args):
    from paper_2010_16165_b200 import workloads as wl
    rank, world, _ = dist_env()
    if rank != 0:
        return
    from oracle import fpo
    w = wl.workload(args.config, batch=args.batch, prune=args.prune)
    cores = fpo.num_threads()
    n_img = min(w.batch, max(2 * cores, 8))
    gp, _, _, _ = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios)
    x = w.x[:n_img]
    # a bounded sample: one untimed pass gives the cost of a pass, the timed passes fill about 20 s
    t = time.perf_counter()
    fpo.fused_forward(gp, x)
    one = time.perf_counter() - t
    steps = max(1, min(args.steps, 20, int(20.0 / max(one, 1e-3))))
    t = time.perf_counter()
    for _ in range(steps):
        fpo.fused_forward(gp, x)
    dt = time.perf_counter() - t
    v = n_img * steps / dt
    sample = f"{n_img} of {w.batch} images per step, {steps} steps (per-image cost does not depend on batch)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": 1, "ms_per_step": 1e3 * dt / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "net": w.net.name, "batch": w.batch, "batch_per_gpu": w.batch, "prune": w.ratio_spec},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------
# the GPU arm
# ------------------------------------------------------------------------------------------

class Model:
    """One workload fused, pruned and resident on the device, with its buffers."""

    def __init__(self, torch, B, w, dev, no_prune=False):
        self.torch, self.B, self.w = torch, B, w
        self.dw, self.dbn = torch.from_numpy(w.weights).to(dev), torch.from_numpy(w.bn).to(dev)
        self.h = B.fp_fuse(w.net, self.dw, self.dbn, w.batch, B.FP_COMPUTE_BF16_TC,
                           B.FP_DTYPE_BF16 if w.in_bf16 else B.FP_DTYPE_F32, 1, 0)
        if not no_prune:
            B.fp_prune(self.h, w.ratios)
        self.n_classes = B.fp_query_int(self.h, B.FP_Q_N_CLASSES)
        x_host = torch.from_numpy(w.x)
        if w.in_bf16:
            x_host = x_host.to(torch.bfloat16)
        self.x_pinned = x_host.pin_memory()
        self.dx = x_host.to(dev)
        self.logits = torch.empty(w.batch, self.n_classes, device=dev)
        self.logits_pinned = torch.empty(w.batch, self.n_classes).pin_memory()

    def close(self):
        self.B.fp_destroy(self.h)


def timed_steps(torch, stream, flush, step, steps, warmup, sync_ranks=True):
    """`steps` steps, each bracketed by two events on `stream`, an L2 flush before each.  Returns the per-step
    milliseconds and the host times around the timed region."""
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            if flush is not None:
                flush.fill_(1)
            step()
        torch.cuda.synchronize()
        if sync_ranks:
            barrier()
        torch.cuda.synchronize()
        t0 = time.time()
        for a, b in ev:
            if flush is not None:
                flush.fill_(1)
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        if sync_ranks:
            barrier()
        torch.cuda.synchronize()
        t1 = time.time()
    return [a.elapsed_time(b) for a, b in ev], t0, t1


def percentile(v, q):
    s = sorted(v)
    return s[min(len(s) - 1, int(round(q * (len(s) - 1))))]


def kernel_report(B, m, peaks, peak_kind, reps):
    """Per-kernel-class figures of one forward from the library's per-operator times: the convolution class that
    takes more of the step (the `roofline` object), and the memory-bound side kernels."""
    w = m.w
    ops = B.op_infos(m.h)
    op_ms = B.fp_query_array(m.h, B.FP_Q_OP_TIMES, reps, np.float32, len(ops))
    # Convolution launches fall in two classes: fused runs of layers (one chain_tc_kernel launch per run,
    # its time reported at the run's first layer) and single layers (conv_tc_kernel).  Algorithmic bytes and
    # flops are the per-layer figures summed over the layers a launch executes.
    classes = {"chain_tc_kernel": [0, 0.0, 0.0, 0.0], "conv_tc_kernel": [0, 0.0, 0.0, 0.0]}
    side = {}
    seen_runs = set()
    for o, t in zip(ops, op_ms):
        if o.kind != 0:
            s = side.setdefault(KIND_NAMES[o.kind], [0, 0.0, 0.0])
            if t > 0:
                s[0] += 1
            s[1] += float(t)
            s[2] += o.bytes_per_image * w.batch + o.bytes_fixed
            continue
        c = classes["chain_tc_kernel" if o.chain >= 0 else "conv_tc_kernel"]
        if o.chain < 0 and t <= 0 and o.flops_per_image == 0:
            continue                   # a projection shortcut computed inside the layer that adds it: no launch of its own
        if o.chain < 0 or o.chain not in seen_runs:
            c[0] += 1
            seen_runs.add(o.chain)
        c[1] += float(t)
        c[2] += o.bytes_per_image * w.batch + o.bytes_fixed
        c[3] += o.flops_per_image * w.batch
    kernel = max(classes, key=lambda k: classes[k][1])
    n_conv, conv_ms, conv_bytes, conv_flops = classes[kernel]
    t_hbm = conv_bytes / (peaks["hbm_gbs"] * 1e9)
    t_flop = conv_flops / (peaks["bf16_tflops_sustained"] * 1e12)
    gbs = conv_bytes / (conv_ms * 1e-3) / 1e9
    tfs = conv_flops / (conv_ms * 1e-3) / 1e12
    if t_hbm >= t_flop:
        roof = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac_nominal": gbs / NOMINAL_PEAKS["hbm_gbs"], "nominal_peak": NOMINAL_PEAKS["hbm_gbs"]}
    else:
        roof = {"bound": "tensor", "achieved": tfs, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac_nominal": tfs / NOMINAL_PEAKS["bf16_tflops"], "nominal_peak": NOMINAL_PEAKS["bf16_tflops"]}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = recorded_traffic(w.name, kernel)
    roof["peak_source"] = peak_kind + (" (sustained BF16 figure: the kernel is timed inside a long step)" if roof["bound"] == "tensor" else "")
    roof["kernel"] = kernel
    roof["launches_per_step"] = n_conv
    roof["avg_launch_us"] = 1e3 * conv_ms / max(n_conv, 1)
    roof["algorithmic_bytes_per_step"] = conv_bytes
    roof["algorithmic_flops_per_step"] = conv_flops
    # both yardsticks for the same launches, whichever bounds them
    roof["hbm_frac"] = gbs / peaks["hbm_gbs"]
    roof["tensor_frac"] = tfs / peaks["bf16_tflops_sustained"]
    roof["share_of_step"] = conv_ms / float(sum(op_ms))
    roof["other_conv_class"] = {k: {"launches": v[0], "ms": v[1]} for k, v in classes.items() if k != kernel}
    side_out = []
    for name, (n, ms, by) in side.items():
        if n == 0 or ms <= 0:
            continue
        g = by / (ms * 1e-3) / 1e9
        side_out.append({"kernel": name, "launches": n, "us": 1e3 * ms, "algorithmic_bytes": by, "GBps": g,
                         "hbm_frac": g / peaks["hbm_gbs"], "hbm_frac_nominal": g / NOMINAL_PEAKS["hbm_gbs"]})
    return roof, side_out, ops, op_ms


def timed_queue(torch, stream, flush, step, steps, warmup, sync_ranks=True):
    """End to end: `steps` asynchronous calls queued back to back on `stream`, an L2 flush before each, between two events.
    The calls overlap one another where the library lets them (the next step's input crosses the bus while this step's
    network runs), so the time is that of the whole queue - flushes included - not a sum of per-step brackets.
    Returns the milliseconds of the whole queue."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            if flush is not None:
                flush.fill_(1)
            step()
        torch.cuda.synchronize()
        if sync_ranks:
            barrier()
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(steps):
            if flush is not None:
                flush.fill_(1)
            step()
        b.record(stream)
        torch.cuda.synchronize()
        if sync_ranks:
            barrier()
        # the flushes alone, for context (the reported time keeps them in)
        fa, fb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fa.record(stream)
        for _ in range(steps):
            if flush is not None:
                flush.fill_(1)
        fb.record(stream)
        torch.cuda.synchronize()
    return a.elapsed_time(b), fa.elapsed_time(fb)


def measure(torch, B, wl, dev, stream, flush, peaks, peak_kind, config, batch, prune, steps, warmup, args,
            headline=False, sampler=None):
    """One workload: device-resident throughput, end to end from pinned host buffers, kernel classes."""
    w = wl.workload(config, batch=batch, prune=prune, aggressive=args.aggressive if headline else False)
    m = Model(torch, B, w, dev, no_prune=args.no_prune if headline else False)
    try:
        step_dev = lambda: B.fp_forward(m.h, m.dx, w.batch, m.logits, stream)
        step_host = lambda: B.fp_forward_host_async(m.h, m.x_pinned, w.batch, m.logits_pinned, stream)
        per_step, t0, t1 = timed_steps(torch, stream, flush, step_dev, steps, warmup, sync_ranks=headline)
        assert B.fp_query_int(m.h, B.FP_Q_DEVICE_STATUS) == 0, "a device-side wait timed out"
        ms_e2e, ms_flushes = timed_queue(torch, stream, flush, step_host, steps, warmup, sync_ranks=headline)
        assert B.fp_query_int(m.h, B.FP_Q_DEVICE_STATUS) == 0, "a device-side wait timed out"
        ms = sum(per_step)
        roof, side, ops, op_ms = kernel_report(B, m, peaks, peak_kind, 20 if headline else 10)
        flops_img = B.fp_query_array(m.h, B.FP_Q_FLOPS, 0, np.float64, 1)[0]
        bytes2 = B.fp_query_array(m.h, B.FP_Q_BYTES, 0, np.float64, 2)
        n_launch = B.fp_query_int(m.h, B.FP_Q_N_LAUNCHES)
        whole_bytes = bytes2[0] * w.batch + bytes2[1]
        # compulsory traffic of a forward: the network input, every packed weight once, the logits
        compulsory = float(m.x_pinned.numel() * m.x_pinned.element_size()) + bytes2[1] + 4.0 * w.batch * m.n_classes
        step_ms = ms / steps
        r = {
            "workload": w.name, "net": w.net.name, "batch": w.batch, "prune": w.ratio_spec,
            "images_per_s": w.batch * steps / (ms * 1e-3), "ms_per_step": step_ms,
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_p99": percentile(per_step, 0.99),
            "steps": steps, "launches_per_step": int(n_launch),
            "e2e_images_per_s": w.batch * steps / (ms_e2e * 1e-3), "e2e_ms_per_step": ms_e2e / steps,
            "e2e_ms_per_step_without_flushes": (ms_e2e - ms_flushes) / steps,
            "h2d_bytes_per_step": int(m.x_pinned.numel() * m.x_pinned.element_size()),
            "d2h_bytes_per_step": int(m.logits_pinned.numel() * 4),
            "roofline": roof,
            "whole_step": {"flops": flops_img * w.batch, "algorithmic_bytes": whole_bytes, "compulsory_bytes": compulsory,
                           "hbm_frac": whole_bytes / (step_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                           "hbm_frac_nominal": whole_bytes / (step_ms * 1e-3) / 1e9 / NOMINAL_PEAKS["hbm_gbs"],
                           "compulsory_hbm_frac": compulsory / (step_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                           "tensor_frac": flops_img * w.batch / (step_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                           "tensor_frac_nominal": flops_img * w.batch / (step_ms * 1e-3) / 1e12 / NOMINAL_PEAKS["bf16_tflops"],
                           "sum_op_ms": float(sum(op_ms))},
            "side_kernels": side,
        }
        extra = {"ms": ms, "ms_e2e": ms_e2e, "ms_flushes": ms_flushes, "t0": t0, "t1": t1, "ops": ops, "op_ms": op_ms, "n_launch": n_launch}
        if headline:
            # the same forward back to back for about a second, no flush in between: the clock and power state of a
            # loaded GPU (the measured peaks were taken in that state); inputs + activations exceed L2 on this workload
            n = max(10, int(1200.0 / max(step_ms, 1e-3)))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                torch.cuda.synchronize()
                s0 = time.time()
                e0.record(stream)
                for _ in range(n):
                    step_dev()
                e1.record(stream)
                torch.cuda.synchronize()
                s1 = time.time()
            sus_ms = e0.elapsed_time(e1) / n
            r["sustained"] = {"steps": n, "ms_per_step": sus_ms, "images_per_s": w.batch / (sus_ms * 1e-3),
                              "l2": "not flushed; back-to-back graph launches",
                              "clocks": sampler.window(s0, s1) if sampler else None}
        if headline and args.soft_epochs > 0:
            # The loop body of Algorithm 1 on the device (not part of a forward step): update + score + select + zeroize
            # over all fused fp32 banks.  Algorithmic bytes per weight: 12 (W += dW) + 4 (score) + at most 4 (zeroize).
            n_w = sum(B.conv_bank_elems(m.h))
            upd = torch.randn(n_w, device=dev) * 0.01
            B.fp_soft_prune_epoch(m.h, w.ratios, upd)             # warm-up
            torch.cuda.synchronize()
            t = time.perf_counter()
            for _ in range(args.soft_epochs):
                B.fp_soft_prune_epoch(m.h, w.ratios, upd)
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t) / args.soft_epochs
            r["soft_prune_epoch"] = {"ms": 1e3 * dt, "weights": n_w, "convolutions": len([e for e in B.conv_bank_elems(m.h) if e]),
                                     "GBps": 16.0 * n_w / dt / 1e9, "timed": "host wall clock around the synchronous call"}
        return r, extra, w
    finally:
        m.close()


def measure_latency(torch, B, wl, dev, stream, flush, runs=1000):
    """ResNet-50 at batch 1 (the paper times single-batch inference, mean of 1000 runs): one CUDA-graph replay per
    run, an event on either side.  `warm`: runs back to back, weights stay in L2 as in a serving loop; `flushed`:
    a 256 MiB write before every run (200 runs)."""
    w = wl.workload(5, batch=1)
    m = Model(torch, B, w, dev)
    try:
        step = lambda: B.fp_forward(m.h, m.dx, 1, m.logits, stream)
        warm, _, _ = timed_steps(torch, stream, None, step, runs, 20, sync_ranks=False)
        cold, _, _ = timed_steps(torch, stream, flush, step, 200, 5, sync_ranks=False)
        assert B.fp_query_int(m.h, B.FP_Q_DEVICE_STATUS) == 0, "a device-side wait timed out"
        f = lambda v: {"runs": len(v), "mean_us": 1e3 * statistics.mean(v), "p50_us": 1e3 * percentile(v, 0.5),
                       "p99_us": 1e3 * percentile(v, 0.99), "min_us": 1e3 * min(v)}
        return {"workload": w.name, "launches_per_run": int(B.fp_query_int(m.h, B.FP_Q_N_LAUNCHES)), "cuda_graph": True,
                "warm_l2": f(warm), "flushed_l2": f(cold)}
    finally:
        m.close()


def run_gpu(args):
    import torch
    from paper_2010_16165_b200 import binding as B, workloads as wl
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    if world > 1:
        init_dist("nccl")
    dev = torch.device("cuda", local)
    peaks, peak_kind = load_peaks()
    stream = torch.cuda.Stream(device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than the 126 MB L2
    warmup = max(args.warmup, 3)

    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3 if sampler else 0.0)
    r, x, w = measure(torch, B, wl, dev, stream, flush, peaks, peak_kind, args.config, args.batch, args.prune, args.steps,
                      warmup, args, headline=True, sampler=sampler)
    clocks = sampler.window(x["t0"], x["t1"]) if sampler else None
    tot_ms, tot_units = aggregate(x["ms"], w.batch * args.steps, dev)
    tot_ms_e2e, _ = aggregate(x["ms_e2e"], w.batch * args.steps, dev)

    out = None
    if rank == 0:
        out = {
            "metric": METRIC, "value": tot_units / (tot_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": tot_ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "net": w.net.name, "batch": w.batch, "batch_per_gpu": w.batch, "prune": w.ratio_spec,
                       "norm": "l1", "pruned": not args.no_prune,
                       "fusion": ("bn folded, shortcut filters stacked into the convolutions (Sec. IV-B)" if args.aggressive
                                  else "bn folded, shortcut+relu in conv epilogue") + ", stages of 3x3 layers as one kernel", "cuda_graph": True,
                       "l2": "flushed between timed steps (256 MiB write)", "parallelism": f"replicas x{world}"},
            "ms_per_step_median": r["ms_per_step_median"], "ms_per_step_p99": r["ms_per_step_p99"],
            "e2e": {"value": tot_units / (tot_ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": r["h2d_bytes_per_step"],
                    "d2h_bytes_per_step": r["d2h_bytes_per_step"], "ms_per_step": tot_ms_e2e / args.steps,
                    "ms_per_step_without_flushes": r["e2e_ms_per_step_without_flushes"],
                    "call": "fp_forward_host_async, the steps queued back to back on one stream (pinned host input and "
                            "logits every step); timed as one queue between two events, L2 flushes included"},
            "gpu_launches": int(x["n_launch"] * args.steps),
            "clocks": clocks,
            "roofline": r["roofline"],
            "whole_step": r["whole_step"],
            "side_kernels": r["side_kernels"],
            "sustained": r.get("sustained"),
            "peaks": {"measured": peaks, "source": peak_kind, "nominal": NOMINAL_PEAKS},
        }
        if "soft_prune_epoch" in r:
            out["soft_prune_epoch"] = r["soft_prune_epoch"]
    if rank == 0 and args.per_op:
        groups = {}
        for o, t in zip(x["ops"], x["op_ms"]):
            key = (KIND_NAMES[o.kind], o.C, o.K, o.R, o.stride, o.H, o.res_mode)
            if o.kind == 0 and o.chain >= 0:
                key = ("fused_run", o.chain, 0, 3, 1, o.H, 0)
            g = groups.setdefault(key, [0, 0.0, 0.0, 0.0])
            g[0] += 1; g[1] += float(t) * 1e3
            g[2] += o.bytes_per_image * w.batch + o.bytes_fixed; g[3] += o.flops_per_image * w.batch
        out["per_op"] = [{"op": k[0], "C": k[1], "K": k[2], "R": k[3], "stride": k[4], "H": k[5], "res": k[6],
                          "launches": g[0], "us_per_launch": round(g[1] / g[0], 2),
                          "GBps": round(g[2] / g[1] * 1e6 / 1e9, 1) if g[1] > 0 else None,
                          "TFLOPs": round(g[3] / g[1] * 1e6 / 1e12, 2) if g[1] > 0 else None} for k, g in groups.items()]
    if rank == 0 and world == 1 and not args.no_sweep:
        # the other workloads of the list, same method, fewer steps
        rows = []
        for cfg, prune in SWEEP:
            rr, _, _ = measure(torch, B, wl, dev, stream, flush, peaks, peak_kind, cfg, None, prune, args.sweep_steps, 5, args)
            rows.append(rr)
        out["configs"] = rows
    if rank == 0 and world == 1 and not args.no_latency:
        out["latency"] = measure_latency(torch, B, wl, dev, stream, flush)
    if sampler:
        sampler.stop()
    if rank == 0:
        if world == 1 and not args.no_cpu:
            n_img = min(w.batch, max(2 * (os.cpu_count() or 8), 8))
            v, cores, secs, passes = oracle_images_per_s(w, n_img)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": f"the first {n_img} of {w.batch} images, {passes} passes, {secs:.1f} s of CPU work"}
        print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--config", type=int, default=HEADLINE_CONFIG)
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch size")
    ap.add_argument("--prune", type=float, default=None)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--no-sweep", action="store_true", help="skip the `configs` array (the other workloads)")
    ap.add_argument("--no-latency", action="store_true", help="skip the batch-1 latency measurement")
    ap.add_argument("--sweep-steps", type=int, default=50)
    ap.add_argument("--aggressive", action="store_true",
                    help="fuse every block the paper's way (Sec. IV-B: identity / shortcut filters stacked into the "
                         "convolutions, no add) instead of adding the shortcut in the epilogue")
    ap.add_argument("--soft-epochs", type=int, default=0,
                    help="after the benchmark, time this many passes of the dynamic pruning loop (fp_soft_prune_epoch)")
    ap.add_argument("--no-prune", action="store_true", help="run the fused graph without fp_prune (with --aggressive: "
                                                            "the fused, not yet pruned operators of Table VII)")
    ap.add_argument("--per-op", action="store_true", help="add per-operator-class times to the JSON line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
