#!/usr/bin/env python
"""Benchmark of the segment training step (samples/s) on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole path over one batch: a training step of every segment of the
workload (forward, loss against the intermediate labels or the class labels, backward, update).
Intermediate labels are generated once per cut before the timed region, as in the method (the
label matrix is produced once per training run); that launch is timed separately.

The headline workload is the largest one, `gemm_large` (both segments in flight on two streams, the
second one fed the first cut's label rows by class, i.e. the fully separate variant).  The timed
region is K steps between CUDA events on every stream in use; it is repeated (at least five times
and until half a second of device time has been spent) and the MEDIAN repeat is reported, all
repeats being listed.  Prints ONE JSON line.  `value` has every input resident in HBM; `e2e` goes
through the host-buffer entry point (pinned host batches in, loss out, every step); `roofline`
describes the kernel kind with the largest share of the step, timed with CUDA events around every
launch; `cpu_baseline` is the CPU oracle on this machine's host cores on a bounded sample.
"""
import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2403_11204_b200 import workloads as wl

L2_BYTES = 126 * 1024 * 1024

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum), mean over the launches of a kind in one step, from
# the ncu captures summarised under profiles/ (the file named beside each figure).  Workloads without a capture of
# their dominant kind report null.
NCU_TRAFFIC_BYTES = {("gemm_large", "fwd_gemm"): (469.9e6, "profiles/gemm_traffic_gemm_large.md"),
                     ("gemm_large", "dgrad_gemm"): (598.1e6, "profiles/gemm_traffic_gemm_large.md"),
                     ("gemm_large", "wgrad_gemm"): (451.6e6, "profiles/gemm_traffic_gemm_large.md"),
                     ("gemm_large", "update"): (1052.2e6, "profiles/gemm_traffic_gemm_large.md"),
                     ("paper_shaped", "fwd_gemm"): (2.614e+06, "profiles/gemm_traffic_paper_shaped.md"),
                     ("paper_shaped", "dgrad_gemm"): (2.955e+06, "profiles/gemm_traffic_paper_shaped.md"),
                     ("paper_shaped", "wgrad_gemm"): (1.340e+06, "profiles/gemm_traffic_paper_shaped.md")}

# Rows per oracle step in the CPU legs (full layer widths always): the oracle converts and rounds every weight
# matrix at each use, so a step of the largest segments costs seconds whatever the batch.
CPU_SAMPLE_BATCH = {"tiny": 64, "paper_net": 1410, "paper_shaped": 256, "bf16_wide": 256, "multi_cut": 128,
                    "gemm_large": 64}


# ---- peaks -----------------------------------------------------------------------------------
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def measure_tf32_peak(peaks):
    """TF32 dense peak, measured the way the bf16 figure of MEASURED_PEAKS.json was: torch.matmul on 8192^3
    with TF32 allowed, best of 10 (burst) and back to back for about a second (sustained).  A library product
    used as a yardstick only."""
    import torch
    try:
        old = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = True
        n = 8192
        a = torch.randn(n, n, device="cuda")
        b = torch.randn(n, n, device="cuda")
        flops = 2.0 * n ** 3
        for _ in range(3):
            a @ b
        best = 0.0
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); a @ b; e1.record()
            torch.cuda.synchronize()
            best = max(best, flops / (e0.elapsed_time(e1) * 1e-3) / 1e12)
        reps = max(10, int(1.0 / (flops / (best * 1e12))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            a @ b
        e1.record()
        torch.cuda.synchronize()
        sustained = reps * flops / (e0.elapsed_time(e1) * 1e-3) / 1e12
        torch.backends.cuda.matmul.allow_tf32 = old
        del a, b
        torch.cuda.empty_cache()
        peaks["tf32_tflops"], peaks["tf32_tflops_sustained"] = best, sustained
        peaks["tf32_source"] = "measured in this run: torch.matmul 8192^3 with TF32 allowed, best of 10 / back to back 1 s"
    except Exception as exc:                                   # keep the nominal ratio, and say so
        peaks["tf32_tflops"] = 0.5 * peaks["bf16_tflops"]
        peaks["tf32_tflops_sustained"] = 0.5 * peaks["bf16_tflops_sustained"]
        peaks["tf32_source"] = f"0.5 x bf16 (nominal ratio; measurement failed: {repr(exc)[:80]})"


def tensor_peak_tflops(precision, peaks, sustained=False):
    """Roofline denominator of the products: the burst figure (the machine's measured peak); the sustained one
    (a long library product under the power cap) is reported beside it."""
    if precision == "tf32":
        if "tf32_tflops" not in peaks:
            measure_tf32_peak(peaks)
        return peaks["tf32_tflops_sustained" if sustained else "tf32_tflops"]
    return peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"]


# ---- algorithmic work --------------------------------------------------------------------------
def segment_work(spec, batch, precision, optimizer):
    """FLOPs of the matrix products and bytes of the streaming kernels of one segment step."""
    w = spec.widths
    p_w = sum(w[i] * w[i + 1] for i in range(len(w) - 1))
    p_b = sum(w[1:])
    fwd = 2 * batch * p_w
    wgrad = 2 * batch * p_w
    dgrad = 2 * batch * (p_w - w[0] * w[1])            # no gradient into the segment input
    per_param = {"sgd": 12, "momentum": 20, "adam": 28}[optimizer] + ({"fp32": 0, "tf32": 4, "bf16": 2}[precision])
    es = 2 if precision == "bf16" else 4
    n_out = w[-1]
    loss_bytes = 2 * batch * n_out * es + 4 * batch
    bias_bytes = batch * sum(w[1:]) * es
    return {"fwd_gemm": fwd, "wgrad_gemm": wgrad, "dgrad_gemm": dgrad, "gemm_flops": fwd + wgrad + dgrad,
            "update_bytes": per_param * (p_w + p_b), "loss_bytes": loss_bytes, "bias_grad_bytes": bias_bytes,
            "params": p_w + p_b}


def step_fractions(work, ms, precision, peaks):
    """The two fractions of a (segment) step: the roofline sum (product FLOPs at the tensor peak plus update
    and loss bytes at the copy bandwidth) over the measured time, and the tensor-only one."""
    tp = tensor_peak_tflops(precision, peaks)
    tps = tensor_peak_tflops(precision, peaks, sustained=True)
    t_roof = work["gemm_flops"] / (tp * 1e12) + (work["update_bytes"] + work["loss_bytes"]) / (peaks["hbm_gbs"] * 1e9)
    tf = work["gemm_flops"] / (ms * 1e-3) / 1e12
    return {"roofline_ms": t_roof * 1e3, "roofline_frac": t_roof * 1e3 / ms, "gemm_tflops": tf,
            "tensor_only_frac": tf / tp, "tensor_only_frac_of_sustained_matmul": tf / tps}


# ---- clocks ------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index=0):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        num = lambda s: s.replace(".", "").isdigit()
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and num(r[0])]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and num(r[1])]
        pw = [float(r[6]) for r in self.rows if len(r) >= 7 and num(r[6])]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[2 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm), "sm_mhz_min": min(sm) if sm else None,
                "power_w_max": max(pw) if pw else None}


# ---- the CPU oracle leg --------------------------------------------------------------------------
def oracle_samples_per_s(workload, budget_s=20.0, max_steps=50, warmup=0):
    """Times the oracle's training step of every segment on a bounded sample of the workload: full layer
    widths, CPU_SAMPLE_BATCH rows per step (the workload's own batch where that is no larger)."""
    from oracle import rng as orng
    from oracle.segment import OracleSegment
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = len(os.sched_getaffinity(0))
    w = workload
    rows = min(w.batch, CPU_SAMPLE_BATCH.get(w.name, w.batch))
    segs = []
    for spec in w.segments:
        s = OracleSegment(spec.widths, w.n_classes, spec.is_final, precision=w.precision, optimizer=w.optimizer,
                          lr=w.lr, momentum=w.momentum, segment_id=spec.segment_id, init_seed=wl.INIT_SEED)
        if not spec.is_final:
            s.gen_labels(wl.LABEL_SEED, orng.DIST_NORMAL if w.label_dist == "normal" else orng.DIST_UNIFORM_KAPPA)
        segs.append(s)
    cls = wl.class_indices(w, rows)
    xs = [wl.features(w, rows, spec.widths[0], seed=spec.segment_id) for spec in w.segments]
    for _ in range(warmup):
        for s, x in zip(segs, xs):
            s.train_step(x, cls)
    t_total, steps = 0.0, 0
    while steps < max_steps and (t_total < budget_s or steps < 1):
        t0 = time.perf_counter()
        for s, x in zip(segs, xs):
            s.train_step(x, cls)
        t_total += time.perf_counter() - t0
        steps += 1
    what = "full-shape" if rows == w.batch else f"full-width, {rows}-row (of the workload's {w.batch})"
    return {"value": steps * rows / t_total, "unit": "samples/s", "cores": cores, "kind": "oracle",
            "sample": f"{steps} {what} step(s) of every segment ({t_total:.1f} s of NumPy fp64 on the host cores; "
                      f"samples/s = rows / time, the per-step cost of converting the weights included)"}, t_total / steps


# ---- our arm -----------------------------------------------------------------------------------
class Runner:
    def __init__(self, workload, device_index=0, host_data=True, n_samples=None):
        import torch
        from paper_2403_11204_b200.binding import Segment
        self.torch = torch
        self.w = workload
        w = workload
        torch.cuda.set_device(device_index)
        self.dt = torch.bfloat16 if w.precision == "bf16" else torch.float32
        self.n = n_samples or w.n_samples
        self.n -= self.n % w.batch
        self.streams = [torch.cuda.Stream() if w.concurrent else torch.cuda.current_stream() for _ in w.segments]
        self.segs = []
        for spec, st in zip(w.segments, self.streams):
            seg = Segment(spec.widths, w.n_classes, spec.is_final, precision=w.precision, optimizer=w.optimizer,
                          lr=w.lr, momentum=w.momentum, max_batch=w.batch, segment_id=spec.segment_id,
                          init_seed=wl.INIT_SEED, stream=st)
            self.segs.append(seg)
        # data: features and classes (seeded); host copies kept for the end-to-end leg
        self.host_x, self.host_cls = None, None
        if host_data:
            x = wl.features(w, self.n)
            cls = wl.class_indices(w, self.n)
            self.host_cls = torch.from_numpy(cls).pin_memory()
            hx = torch.from_numpy(x)
            self.host_x = [hx.to(self.dt).pin_memory()]
            self.cls = self.host_cls.cuda()
            self.x = [self.host_x[0].cuda()]
        else:
            g = torch.Generator(device="cuda").manual_seed(wl.DATA_SEED)
            n_feat = w.n_features
            if w.input_dist == "normal":
                x = torch.randn(self.n, n_feat, generator=g, device="cuda", dtype=torch.float32)
            else:
                x = torch.rand(self.n, n_feat, generator=g, device="cuda", dtype=torch.float32)
            self.x = [x.to(self.dt)]
            self.cls = torch.randint(0, w.n_classes, (self.n,), generator=g, device="cuda", dtype=torch.int32)
        self.sil_in = [None] * len(self.segs)
        torch.cuda.synchronize()

    def gen_labels(self):
        t0 = time.perf_counter()
        for seg in self.segs:
            if not seg.is_final:
                seg.gen_labels(wl.LABEL_SEED, self.w.label_dist)
        self.torch.cuda.synchronize()
        return (time.perf_counter() - t0) * 1e3

    def materialise_inputs(self):
        """Inputs of segment k > 0: the stored response of segment k-1 over the whole set (Section 2).
        Concurrently trained segments take the label row of each sample's class instead (the fully separate
        variant): nothing is materialised, seg_train_step_label_input gathers the rows inside the step."""
        torch, w = self.torch, self.w
        for k in range(1, len(self.segs)):
            prev = self.segs[k - 1]
            if w.concurrent:
                self.sil_in[k] = prev.labels()
                self.x.append(None)
                if self.host_x is not None:
                    self.host_x.append(None)
                continue
            xk = torch.empty(self.n, prev.widths[-1], dtype=prev.out_dtype, device="cuda")
            for i in range(0, self.n, w.batch):
                prev.forward(self.x[k - 1][i:i + w.batch], xk[i:i + w.batch])
            self.x.append(xk)
            if self.host_x is not None:
                self.host_x.append(xk.cpu().pin_memory())
        torch.cuda.synchronize()

    def batch_slice(self, step):
        i = (step * self.w.batch) % self.n
        return slice(i, i + self.w.batch)

    def step_segment(self, k, sl):
        seg = self.segs[k]
        if self.sil_in[k] is not None:
            seg.train_step_label_input(self.sil_in[k], self.cls[sl], self.loss[k])
        else:
            seg.train_step(self.x[k][sl], self.cls[sl], self.loss[k])

    def run_steps(self, first, count, which=None):
        for s in range(first, first + count):
            sl = self.batch_slice(s)
            for k in range(len(self.segs)):
                if which is None or k == which:
                    self.step_segment(k, sl)

    def timed(self, first, count, which=None):
        """Device time of `count` steps (ms): CUDA events on every stream in use, max over streams."""
        torch = self.torch
        torch.cuda.synchronize()
        used = [k for k in range(len(self.segs)) if which is None or k == which]
        streams = []
        for k in used:
            if all(self.streams[k].cuda_stream != s.cuda_stream for s in streams):
                streams.append(self.streams[k])
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in streams]
        for st, (e0, _) in zip(streams, evs):
            e0.record(st)
        self.run_steps(first, count, which)
        for st, (_, e1) in zip(streams, evs):
            e1.record(st)
        torch.cuda.synchronize()
        return max(e0.elapsed_time(e1) for e0, e1 in evs)

    def prepare(self):
        self.loss = [self.torch.zeros(1, device="cuda") for _ in self.segs]

    def launches(self):
        return sum(seg.launch_count() for seg in self.segs)

    def families(self):
        out = {}
        for seg in self.segs:
            for name, n in seg.product_launches().items():
                out[name] = out.get(name, 0) + n
        return out

    def close(self):
        for seg in self.segs:
            seg.close()


def unpartitioned_comparison(workload, steps=5):
    """End-to-end backprop of the unpartitioned network on the same GPU: one final segment spanning
    every layer (same precision, optimizer, batch).  Returns its device memory and step time."""
    import torch
    from paper_2403_11204_b200.binding import Segment
    w = workload
    widths = list(w.segments[0].widths)
    for spec in w.segments[1:]:
        widths += list(spec.widths[1:])
    dt = torch.bfloat16 if w.precision == "bf16" else torch.float32
    seg = Segment(widths, w.n_classes, True, precision=w.precision, optimizer=w.optimizer, lr=w.lr,
                  momentum=w.momentum, max_batch=w.batch, segment_id=0, init_seed=wl.INIT_SEED)
    g = torch.Generator(device="cuda").manual_seed(wl.DATA_SEED)
    x = torch.rand(w.batch, widths[0], generator=g, device="cuda").to(dt)
    cls = torch.randint(0, w.n_classes, (w.batch,), generator=g, device="cuda", dtype=torch.int32)
    loss = torch.zeros(1, device="cuda")
    for _ in range(3):
        seg.train_step(x, cls, loss)
    seg.poll()
    seg.timer_start()
    for _ in range(steps):
        seg.train_step(x, cls, loss)
    seg.timer_stop()
    ms = seg.timer_ms() / steps
    mem = seg.mem_bytes()[1]
    seg.close()
    return {"layers": len(widths) - 1, "mem_bytes_peak": mem, "ms_per_step": ms}


def _rank_barrier():
    """Barrier over the replicas when the run has more than one (a no-op otherwise)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def kernel_breakdown(r, steps, first, peaks):
    """Per-kind device time: the same steps again, one segment at a time, with CUDA events around every launch
    on the segment's stream (so the kinds add up to the serial time of the step).  Where weight-gradient
    products also apply the optimizer update (seg_profile_get kind 4), the weight-gradient and update kinds
    are reported as one kind, `wgrad_update`, with the products' FLOPs and the update's bytes beside its time.
    Returns (kernels dict, roofline dict of the dominant kind)."""
    w = r.w
    kinds = {}
    for k_seg, (spec, seg) in enumerate(zip(w.segments, r.segs)):
        seg.profile(True)
        r.run_steps(first, steps, which=k_seg)
        r.torch.cuda.synchronize()
        work = segment_work(spec, w.batch, w.precision, w.optimizer)
        prof = seg.profile_read()
        fused = prof.get("wgrad_update_gemm", (0, 0.0))[0] > 0
        for name, (n, tot) in prof.items():
            if fused and name in ("wgrad_gemm", "wgrad_update_gemm", "update"):
                name = "wgrad_update"
            elif name == "wgrad_update_gemm":
                continue
            k = kinds.setdefault(name, {"launches": 0, "ms": 0.0, "flops": 0.0, "bytes": 0.0, "seen": set()})
            k["launches"] += n
            k["ms"] += tot
            if (k_seg, name) in k["seen"]:
                continue
            k["seen"].add((k_seg, name))
            if name in ("fwd_gemm", "dgrad_gemm", "wgrad_gemm"):
                k["flops"] += work[name] * steps
            elif name == "fwd_loss_dgrad":  # first launch of a small fp32 segment's two-launch step
                k["flops"] += (work["fwd_gemm"] + work["dgrad_gemm"]) * steps
            elif name == "wgrad_update":
                k["flops"] += work["wgrad_gemm"] * steps
                k["bytes"] += (work["update_bytes"] + work["bias_grad_bytes"]) * steps
            elif name == "update":          # the update launch also reads dZ for the bias gradient
                k["bytes"] += (work["update_bytes"] + work["bias_grad_bytes"]) * steps
            elif name == "loss":
                k["bytes"] += work["loss_bytes"] * steps
        seg.profile(False)
    tp = tensor_peak_tflops(w.precision, peaks)
    tps = tensor_peak_tflops(w.precision, peaks, sustained=True)
    total_ms = sum(v["ms"] for v in kinds.values()) or 1.0
    kernels = {}
    for n, v in kinds.items():
        if v["launches"] == 0:
            continue
        e = {"launches": v["launches"], "ms_per_step": round(v["ms"] / steps, 5), "share": round(v["ms"] / total_ms, 4),
             "avg_us": round(1e3 * v["ms"] / v["launches"], 3)}
        if v["flops"] > 0:
            e["tflops"] = round(v["flops"] / (v["ms"] * 1e-3) / 1e12, 2)
            e["frac_of_peak"] = round(e["tflops"] / tp, 4)
        if v["bytes"] > 0:
            e["gbs"] = round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1)
            if v["flops"] > 0:       # products carrying the update: time against FLOPs at the tensor peak + bytes at the copy bandwidth
                e["frac_of_sum_roofline"] = round((v["flops"] / (tp * 1e12) + v["bytes"] / (peaks["hbm_gbs"] * 1e9)) / (v["ms"] * 1e-3), 4)
            else:
                e["frac_of_peak"] = round(e["gbs"] / peaks["hbm_gbs"], 4)
        kernels[n] = e
    dom = max(kinds, key=lambda n: kinds[n]["ms"])
    v = kinds[dom]
    timing = "CUDA events around every launch of this kind on the launching stream, same steps re-run after the timed region"
    traffic = NCU_TRAFFIC_BYTES.get((w.name, dom))
    if v["flops"] > 0:
        achieved = v["flops"] / (v["ms"] * 1e-3) / 1e12
        prec_note = (peaks.get("tf32_source", "") if w.precision == "tf32" else "bf16 torch.matmul burst figure")
        roof = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": tp, "unit": "TFLOP/s",
                "frac": achieved / tp, "frac_of_sustained_matmul": achieved / tps, "peak_sustained": tps,
                "traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None,
                "peak_source": f"{peaks['source']} ({prec_note})", "timing": timing,
                "launches": v["launches"], "avg_launch_us": 1e3 * v["ms"] / max(v["launches"], 1)}
        if v["bytes"] > 0:
            roof["note"] = ("these launches are weight-gradient products whose extra warps also stream the optimizer update "
                            f"({v['bytes'] / v['launches'] / 1e6:.1f} MB per launch on average, bias update launches included in "
                            "the time); achieved counts the products' FLOPs only")
    else:
        achieved = v["bytes"] / (v["ms"] * 1e-3) / 1e9
        roof = {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": traffic[0] if traffic else None,
                "traffic_source": traffic[1] if traffic else None,
                "peak_source": f"{peaks['source']}: copy bandwidth", "timing": timing,
                "launches": v["launches"], "avg_launch_us": 1e3 * v["ms"] / max(v["launches"], 1)}
    return kernels, roof


def measure(workload, steps, warmup, peaks, device_index=0, full=True, n_samples=None, extras=False):
    """Runs one workload.  full=True adds the end-to-end leg and the clock record; extras=True the training
    procedure and recovery legs (two sequential segments)."""
    import torch
    w = workload
    if n_samples is None and not full:
        n_samples = min(w.n_samples, 64 * w.batch)
    r = Runner(w, device_index, host_data=full, n_samples=n_samples)
    r.prepare()
    label_ms = r.gen_labels()
    r.materialise_inputs()
    data_bytes = sum(x.numel() * x.element_size() for x in r.x if x is not None)
    r.run_steps(0, max(warmup, 3))
    for seg in r.segs:
        seg.poll()
    sampler = ClockSampler(device_index)
    if full:
        sampler.start()
        time.sleep(0.25)
    # the timed region, repeated: exactly `steps` steps per repeat, at least 5 repeats and 0.5 s of device time
    l0, f0 = r.launches(), r.families()
    repeats, total_ms, pos = [], 0.0, warmup
    min_repeats, max_repeats = (5, 400) if full else (3, 20)
    while len(repeats) < min_repeats or (total_ms < (500.0 if full else 50.0) and len(repeats) < max_repeats):
        _rank_barrier()                       # replicas enter and leave every timed region together
        ms = r.timed(pos, steps)              # synchronises the device on both sides; CUDA events on every stream
        _rank_barrier()
        repeats.append(ms)
        total_ms += ms
        pos += steps
    launches = r.launches() - l0
    f1 = r.families()
    if full:
        time.sleep(0.15)
    clocks = sampler.stop() if full else None
    ms = float(np.median(repeats))
    out = {"ms_per_step": ms / steps, "samples_per_s": steps * w.batch / (ms * 1e-3), "launches": launches,
           "repeats": {"n": len(repeats), "steps_each": steps, "ms_per_step_median": ms / steps,
                       "ms_per_step_min": min(repeats) / steps, "ms_per_step_max": max(repeats) / steps,
                       "device_s_total": total_ms * 1e-3},
           "product_launches": {k: f1[k] - f0.get(k, 0) for k in f1},
           "label_gen_ms": label_ms, "data_bytes": data_bytes, "clocks": clocks, "segments": []}

    # per-segment timing (each segment alone on its stream) and the two fractions of the whole segment step
    whole = {"gemm_flops": 0, "update_bytes": 0, "loss_bytes": 0}
    for k, (spec, seg) in enumerate(zip(w.segments, r.segs)):
        work = segment_work(spec, w.batch, w.precision, w.optimizer)
        for key in whole:
            whole[key] += work[key]
        ms_k = float(np.median([r.timed(pos + i * steps, steps, which=k) for i in range(3)])) / steps
        pos += 3 * steps
        e = {"segment": k, "widths": spec.widths, "ms_per_step": ms_k, "samples_per_s": w.batch / (ms_k * 1e-3),
             "mem_bytes_peak": seg.mem_bytes()[1]}
        e.update(step_fractions(work, ms_k, w.precision, peaks))
        out["segments"].append(e)
    out["step"] = step_fractions(whole, out["ms_per_step"], w.precision, peaks)
    out["step"]["segments_alone_ms_sum"] = sum(s_["ms_per_step"] for s_ in out["segments"])
    out["kernels"], out["roofline"] = kernel_breakdown(r, max(3, min(steps, 20)), pos, peaks)
    if full:
        # end to end through the host-buffer entry points: every step reads its batch from pinned host memory
        # (host -> device inside the step) and writes its loss to pinned host memory (device -> host).
        # Timed twice: seg_train_step_host_async (steps enqueued back to back, one synchronisation at the end:
        # how a training loop calls it) and seg_train_step_host (waits for every loss).  A segment fed label rows
        # by class takes only the class indices from the host (a pinned -> device copy on its stream).
        e_steps = max(3, min(steps, 50))
        es = 2 if w.precision == "bf16" else 4
        h2d = sum(w.batch * ((spec.widths[0] * es if r.sil_in[k] is None else 0) + 4) for k, spec in enumerate(w.segments))
        loss_pin = torch.zeros(e_steps + 3, len(r.segs), dtype=torch.float32).pin_memory()
        cls_dev = [torch.empty(w.batch, dtype=torch.int32, device="cuda") for _ in r.segs]
        d2h = 0

        def e2e_loop(sync_every_step):
            nonlocal d2h
            d2h = 0
            for s in range(3 + e_steps):
                if s == 3:
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                sl = r.batch_slice(s)
                for k, seg in enumerate(r.segs):
                    if r.sil_in[k] is not None:
                        with torch.cuda.stream(r.streams[k]):
                            cls_dev[k].copy_(r.host_cls[sl], non_blocking=True)
                            seg.train_step_label_input(r.sil_in[k], cls_dev[k], r.loss[k])
                            loss_pin[s, k:k + 1].copy_(r.loss[k], non_blocking=True)
                        if sync_every_step:
                            r.streams[k].synchronize()
                    elif sync_every_step:
                        seg.train_step_host(r.host_x[k][sl], r.host_cls[sl])
                    else:
                        seg.train_step_host_async(r.host_x[k][sl], r.host_cls[sl], loss_pin[s, k:k + 1])
                    d2h += 4
            torch.cuda.synchronize()
            return time.perf_counter() - t0

        dt_sync = e2e_loop(True)
        dt_async = sorted(e2e_loop(False) for _ in range(3))[1]       # median of three passes
        assert bool(torch.isfinite(loss_pin[3:]).all()) and float(loss_pin[3:].abs().sum()) > 0.0
        out["e2e"] = {"value": e_steps * w.batch / dt_async, "unit": "samples/s", "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": 4 * len(w.segments), "steps": e_steps, "passes": 3,
                      "call": "seg_train_step_host_async per segment and step (pinned batch in, loss written to pinned "
                              "memory), one synchronisation after the last step"
                              + ("; the label-fed segment: pinned class indices copied in, seg_train_step_label_input, "
                                 "loss copied out" if any(s_ is not None for s_ in r.sil_in) else ""),
                      "waiting_for_every_loss": {"value": e_steps * w.batch / dt_sync, "unit": "samples/s",
                                                 "call": "seg_train_step_host"}}
    if extras and not w.concurrent:
        # the whole procedure of Section 2, one epoch per segment: train segment k over the resident set in
        # stored order (last partial batch included), store its response, hand it to segment k+1
        from paper_2403_11204_b200 import binding
        n_all = r.x[0].shape[0] + 0
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        binding.train_partitioned(r.segs, r.x[0], r.cls, w.batch, [1] * len(r.segs))
        e1.record()
        torch.cuda.synchronize()
        ms_proc = e0.elapsed_time(e1)
        out["procedure"] = {"what": "one epoch per segment over the resident set, in order, response of each segment "
                                    "stored for the next (seg_train_epochs + seg_forward_dataset)",
                            "samples": n_all, "ms": ms_proc,
                            "samples_per_s": n_all / (ms_proc * 1e-3)}
    if extras and not w.concurrent and len(w.segments) == 2:
        # recovery phase of Section 5: the left segment trained through the frozen right one, per step
        from paper_2403_11204_b200 import binding
        rec_loss = torch.zeros(1, device="cuda")
        n_rec = max(10, min(steps, 100))
        for s in range(5):
            sl = r.batch_slice(s)
            binding.recovery_step(r.segs[0], r.segs[1], r.x[0][sl], r.cls[sl], rec_loss)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in range(n_rec):
            sl = r.batch_slice(s + 5)
            binding.recovery_step(r.segs[0], r.segs[1], r.x[0][sl], r.cls[sl], rec_loss)
        e1.record()
        torch.cuda.synchronize()
        ms_rec = e0.elapsed_time(e1) / n_rec
        out["recovery"] = {"what": "seg_recovery_step: left segment trained through the frozen right segment "
                                   "(one replayed graph per step)", "steps": n_rec, "ms_per_step": ms_rec,
                           "samples_per_s": w.batch / (ms_rec * 1e-3)}
    r.close()
    del r
    torch.cuda.empty_cache()
    if len(w.segments) > 1:
        try:
            e2e_net = unpartitioned_comparison(w)
            seg_peak = max(s_["mem_bytes_peak"] for s_ in out["segments"])
            out["memory"] = {"largest_segment_bytes": seg_peak, "unpartitioned_bytes": e2e_net["mem_bytes_peak"],
                             "ratio": e2e_net["mem_bytes_peak"] / seg_peak,
                             "unpartitioned_ms_per_step": e2e_net["ms_per_step"],
                             "segments_ms_per_step_sum": sum(s_["ms_per_step"] for s_ in out["segments"]),
                             "note": "bytes held by the library per handle; segments trained one at a time need only the "
                                     "largest segment resident"}
        except Exception as exc:
            out["memory"] = {"error": repr(exc)[:200]}
    return out


def aggregate_over_ranks(ms_total, steps, batch, world, device="cuda"):
    """Replicas only: the job's time is the slowest rank's, its work the sum over ranks.
    Returns (samples/s of the whole job, ms of the timed region)."""
    if world > 1:
        import torch
        import torch.distributed as dist
        t = torch.tensor([ms_total], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    return world * steps * batch / (ms_total * 1e-3), ms_total


def short_segments(segs):
    keys = ("segment", "ms_per_step", "samples_per_s", "roofline_frac", "tensor_only_frac", "gemm_tflops")
    return [{k: (round(s[k], 5) if isinstance(s[k], float) else s[k]) for k in keys} for s in segs]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="gemm_large", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--others", default="multi_cut,bf16_wide,paper_shaped,tiny,paper_net",
                    help="further workloads summarised in the same line ('' for none)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--samples", type=int, default=0, help="size of the resident data set (0: the workload's own)")
    ap.add_argument("--quick", action="store_true",
                    help="warm-up and one timed region only (no end-to-end leg, breakdown, CPU leg or other workloads): "
                         "the command profilers are pointed at")
    ap.add_argument("--segment", type=int, default=-1, help="with --quick: run this segment only")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = wl.WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config = {"workload": f"{w.name}: " + " | ".join("-".join(map(str, s.widths)) for s in w.segments),
              "batch": w.batch, "optimizer": w.optimizer, "lr": w.lr, "n_classes": w.n_classes,
              "n_samples": w.n_samples, "label_dist": w.label_dist, "segments_per_step": len(w.segments),
              "segments_in_flight": "concurrently on two streams; segment 1 takes the label rows of the first cut by class "
                                    "(fully separate variant)" if w.concurrent else "one after another on one stream",
              "cache": ("inputs larger than L2: every step reads the next batch of a resident data set and streams "
                        "all weights and optimizer state") if w.n_samples * w.n_features * 2 > L2_BYTES else
                       "the workload's whole data set is smaller than L2 (no flush: that is its steady state)",
              "parallelism": "replicas only" if world > 1 else "single GPU"}

    if args.impl == "reference":
        if rank != 0:
            return
        base, _ = oracle_samples_per_s(w, budget_s=1e9, max_steps=max(args.steps, 1), warmup=min(args.warmup, 1))
        rows = min(w.batch, CPU_SAMPLE_BATCH.get(w.name, w.batch))
        line = {"impl": "reference", "metric": "segment train-step samples/sec", "value": base["value"],
                "unit": "samples/s", "n_gpus": 0, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": 1e3 * rows / base["value"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                "cpu_baseline": base,
                "e2e": {"value": base["value"], "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    from paper_2403_11204_b200 import build
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()                                   # in-tree library; a no-op when it is up to date
    if world > 1:
        dist.barrier()
    peaks = load_peaks()
    torch.cuda.set_device(local_rank)
    if args.quick:
        r = Runner(w, local_rank, host_data=False, n_samples=args.samples or min(w.n_samples, 16 * w.batch))
        r.prepare()
        r.gen_labels()
        r.materialise_inputs()
        which = args.segment if args.segment >= 0 else None
        r.run_steps(0, args.warmup, which)
        ms = r.timed(args.warmup, args.steps, which)
        print(json.dumps({"quick": True, "workload": w.name, "segment": which, "steps": args.steps,
                          "ms_per_step": ms / args.steps, "product_launches": r.families()}))
        r.close()
        return
    res = measure(w, args.steps, args.warmup, peaks, device_index=local_rank, full=True,
                  n_samples=args.samples or None, extras=not w.concurrent)
    ms_total = res["ms_per_step"] * args.steps
    value, ms_total = aggregate_over_ranks(ms_total, args.steps, w.batch, world)
    if world > 1:
        e = torch.tensor([res["e2e"]["value"]], device="cuda")
        dist.all_reduce(e, op=dist.ReduceOp.SUM)
        res["e2e"]["value"] = float(e.item())
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    line = {"metric": "segment train-step samples/sec", "value": value, "unit": "samples/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {"fp32": "f32", "tf32": "tf32", "bf16": "bf16"}[w.precision], "data": "synthetic",
            "config": config, "clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": res["launches"],
            "roofline": res.get("roofline"), "step": res["step"], "repeats": res["repeats"]}
    if not args.no_cpu_baseline:
        line["cpu_baseline"], _ = oracle_samples_per_s(w, budget_s=15.0)
    line["kernels"] = res.get("kernels")
    line["segments"] = short_segments(res["segments"])
    line["product_launches"] = res["product_launches"]
    others = {}
    for name in [n for n in args.others.split(",") if n and n != args.workload]:
        ow = wl.WORKLOADS[name]
        k = max(5, min(args.steps, 30))
        try:
            r = measure(ow, k, 3, peaks, device_index=local_rank, full=False, extras=(name == "paper_shaped"))
            o = {"ms_per_step": round(r["ms_per_step"], 5), "samples_per_s": round(r["samples_per_s"], 1),
                 "precision": ow.precision, "batch": ow.batch, "step": {kk: round(v, 4) for kk, v in r["step"].items()},
                 "segments": short_segments(r["segments"]),
                 "roofline": {kk: r["roofline"][kk] for kk in ("kernel", "bound", "achieved", "peak", "unit", "frac")},
                 "kernels": {kk: {k2: v[k2] for k2 in ("share", "avg_us", "tflops", "gbs", "frac_of_peak", "frac_of_sum_roofline")
                                  if k2 in v} for kk, v in r["kernels"].items()},
                 "product_launches": r["product_launches"]}
            if "memory" in r and "ratio" in r["memory"]:
                o["memory"] = {kk: r["memory"][kk] for kk in ("largest_segment_bytes", "unpartitioned_bytes", "ratio",
                                                              "unpartitioned_ms_per_step")}
            for extra in ("procedure", "recovery"):
                if extra in r:
                    o[extra] = {kk: v for kk, v in r[extra].items() if kk != "what"}
            if ow.n_samples * ow.n_features * 4 < L2_BYTES:
                o["cache"] = "the workload's whole data set is smaller than L2"
            others[name] = o
        except Exception as exc:                       # a secondary workload must not cost the headline
            others[name] = {"error": repr(exc)[:200]}
    line["others"] = others
    line["memory"] = res.get("memory")
    line["label_gen_ms"] = res["label_gen_ms"]
    for extra in ("procedure", "recovery"):
        if extra in res:
            line[extra] = res[extra]
    line["peaks"] = peaks
    # last, so that it survives a record that keeps only the end of the line: every workload in one compact object
    def brief(ms, step, segs):
        return {"ms": round(ms, 4), "sum_frac": round(step["roofline_frac"], 3), "tensor_frac": round(step["tensor_only_frac"], 3),
                "seg_ms": [round(s_["ms_per_step"], 4) for s_ in segs], "seg_sum_frac": [round(s_["roofline_frac"], 3) for s_ in segs],
                "seg_tensor_frac": [round(s_["tensor_only_frac"], 3) for s_ in segs]}
    summary = {}
    for name in reversed(list(others)):                 # the headline workload last, the largest others next to it
        if "error" not in others[name]:
            summary[name] = brief(others[name]["ms_per_step"], others[name]["step"], others[name]["segments"])
    summary[w.name] = brief(line["ms_per_step"], res["step"], res["segments"])
    line["summary"] = {"what": "ms per step; sum_frac = (product FLOPs / tensor peak + update and loss bytes / copy bandwidth) / step time; "
                               "tensor_frac = product FLOPs / step time / tensor peak; seg_* per segment",
                       **summary}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
