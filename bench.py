#!/usr/bin/env python
"""Benchmark of the segment training step (samples/s) on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole path over one batch: a training step of every segment of the
workload (forward, loss against the intermediate labels or the class labels, backward, update).
Intermediate labels are generated once per cut before the timed region, as in the method (the
label matrix is produced once per training run); that launch is timed separately.

Prints ONE JSON line.  `value` is timed with CUDA events with every input resident in HBM; `e2e`
goes through the host-buffer entry point (pinned host batches, loss read back every step);
`roofline` describes the kernel kind with the largest share of the step; `cpu_baseline` is the
CPU oracle timed on this machine's host cores on a bounded sample.
"""
import argparse
import json
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

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the product kernel kinds, from the
# ncu capture summarised in profiles/gemm_traffic_paper_shaped.md (every product launch of two steady-state
# steps of both segments; mean per kind).  Workloads without a capture of their dominant kind report null.
NCU_TRAFFIC_BYTES = {("paper_shaped", "fwd_gemm"): 2.621e6, ("paper_shaped", "dgrad_gemm"): 2.953e6,
                     ("paper_shaped", "wgrad_gemm"): 1.326e6}


# ---- peaks -----------------------------------------------------------------------------------
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


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


def tensor_peak_tflops(precision, peaks, sustained=True):
    base = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    return base * (0.5 if precision in ("tf32",) else 1.0)     # nominal TF32 : bf16 ratio is 1 : 2


# ---- clocks ------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

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
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ---- the CPU oracle leg --------------------------------------------------------------------------
def oracle_samples_per_s(workload, budget_s=20.0, max_steps=50):
    """Times the oracle's training step of every segment on batches of the workload."""
    from oracle import rng as orng
    from oracle.segment import OracleSegment
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = len(os.sched_getaffinity(0))
    w = workload
    segs = []
    for spec in w.segments:
        s = OracleSegment(spec.widths, w.n_classes, spec.is_final, precision=w.precision, optimizer=w.optimizer,
                          lr=w.lr, momentum=w.momentum, segment_id=spec.segment_id, init_seed=wl.INIT_SEED)
        if not spec.is_final:
            s.gen_labels(wl.LABEL_SEED, orng.DIST_NORMAL if w.label_dist == "normal" else orng.DIST_UNIFORM_KAPPA)
        segs.append(s)
    cls = wl.class_indices(w, w.batch)
    xs = [wl.features(w, w.batch, spec.widths[0], seed=spec.segment_id) for spec in w.segments]
    t_total, steps = 0.0, 0
    while steps < max_steps and (t_total < budget_s or steps < 1):
        t0 = time.perf_counter()
        for s, x in zip(segs, xs):
            s.train_step(x, cls)
        t_total += time.perf_counter() - t0
        steps += 1
    return {"value": steps * w.batch / t_total, "unit": "samples/s", "cores": cores, "kind": "oracle",
            "sample": f"{steps} full-shape step(s) of every segment at batch {w.batch} "
                      f"({t_total:.1f} s of NumPy fp64 on the host cores)"}, t_total / steps


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
        For concurrently trained segments the input is the label row of each sample's class."""
        torch, w = self.torch, self.w
        for k in range(1, len(self.segs)):
            prev = self.segs[k - 1]
            if w.concurrent:
                xk = prev.labels()[self.cls.long()].to(self.dt).contiguous()
            else:
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

    def run_steps(self, first, count, which=None):
        for s in range(first, first + count):
            sl = self.batch_slice(s)
            for k, seg in enumerate(self.segs):
                if which is not None and k != which:
                    continue
                seg.train_step(self.x[k][sl], self.cls[sl], self.loss[k])

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


def measure(workload, steps, warmup, peaks, device_index=0, full=True, n_samples=None):
    """Runs one workload.  full=True adds the end-to-end leg, per-kernel profile and clocks."""
    import torch
    w = workload
    if n_samples is None and not full:
        n_samples = min(w.n_samples, 64 * w.batch)
    r = Runner(w, device_index, host_data=full, n_samples=n_samples)
    r.prepare()
    label_ms = r.gen_labels()
    r.materialise_inputs()
    data_bytes = sum(x.numel() * x.element_size() for x in r.x)
    r.run_steps(0, max(warmup, 3))
    for seg in r.segs:
        seg.poll()
    sampler = ClockSampler(device_index)
    if full:
        sampler.start()
        time.sleep(0.25)
    l0 = r.launches()
    _rank_barrier()                       # replicas start the timed region together ...
    ms = r.timed(warmup, steps)           # (synchronises the device on both sides; CUDA events on every stream)
    _rank_barrier()                       # ... and leave it together
    launches = r.launches() - l0
    if full:
        time.sleep(0.15)
    clocks = sampler.stop() if full else None
    out = {"ms_per_step": ms / steps, "samples_per_s": steps * w.batch / (ms * 1e-3), "launches": launches,
           "label_gen_ms": label_ms, "data_bytes": data_bytes, "clocks": clocks, "segments": []}

    # per-segment timing and roofline of the whole segment step
    tp = tensor_peak_tflops(w.precision, peaks)
    for k, (spec, seg) in enumerate(zip(w.segments, r.segs)):
        work = segment_work(spec, w.batch, w.precision, w.optimizer)
        ms_k = r.timed(warmup + steps, steps, which=k) / steps
        t_roof = work["gemm_flops"] / (tp * 1e12) + (work["update_bytes"] + work["loss_bytes"]) / (peaks["hbm_gbs"] * 1e9)
        out["segments"].append({"segment": k, "widths": spec.widths, "ms_per_step": ms_k,
                                "samples_per_s": w.batch / (ms_k * 1e-3),
                                "roofline_ms": t_roof * 1e3, "roofline_frac": t_roof * 1e3 / ms_k,
                                "gemm_tflops": work["gemm_flops"] / (ms_k * 1e-3) / 1e12,
                                "mem_bytes_peak": seg.mem_bytes()[1]})
    if full:
        # per-kernel device time: the same steps again with events around every launch
        for seg in r.segs:
            seg.profile(True)
        r.run_steps(warmup, steps)
        torch.cuda.synchronize()
        kinds = {}
        for spec, seg in zip(w.segments, r.segs):
            work = segment_work(spec, w.batch, w.precision, w.optimizer)
            for name, (n, tot) in seg.profile_read().items():
                k = kinds.setdefault(name, {"launches": 0, "ms": 0.0, "flops": 0.0, "bytes": 0.0})
                k["launches"] += n
                k["ms"] += tot
                if name in ("fwd_gemm", "dgrad_gemm", "wgrad_gemm"):
                    k["flops"] += work[name] * steps
                elif name == "update":          # the update launch also reads dZ for the bias gradient
                    k["bytes"] += (work["update_bytes"] + work["bias_grad_bytes"]) * steps
                elif name == "loss":
                    k["bytes"] += work["loss_bytes"] * steps
            seg.profile(False)
        out["kernels"] = {n: {"launches": v["launches"], "ms_total": round(v["ms"], 4),
                              "avg_us": round(1e3 * v["ms"] / max(v["launches"], 1), 3)} for n, v in kinds.items()}
        dom = max(kinds, key=lambda n: kinds[n]["ms"])
        v = kinds[dom]
        if v["flops"] > 0:
            achieved = v["flops"] / (v["ms"] * 1e-3) / 1e12
            out["roofline"] = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": tp, "unit": "TFLOP/s",
                               "frac": achieved / tp, "traffic": NCU_TRAFFIC_BYTES.get((w.name, dom)),
                               "peak_source": f"{peaks['source']}: sustained bf16 {peaks['bf16_tflops_sustained']} TF/s"
                                              + (" x 0.5 nominal TF32 ratio" if w.precision == "tf32" else ""),
                               "timing": "CUDA events around every launch of this kind, same steps re-run after the timed region",
                               "launches": v["launches"], "avg_launch_us": 1e3 * v["ms"] / max(v["launches"], 1)}
        else:
            achieved = v["bytes"] / (v["ms"] * 1e-3) / 1e9
            out["roofline"] = {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                               "peak_source": f"{peaks['source']}: copy bandwidth",
                               "timing": "CUDA events around every launch of this kind, same steps re-run after the timed region",
                               "launches": v["launches"], "avg_launch_us": 1e3 * v["ms"] / max(v["launches"], 1)}
        # end to end through the host-buffer entry points: every step reads its batch from pinned host memory
        # (host -> device inside the step) and writes its loss to pinned host memory (device -> host).
        # Timed twice: seg_train_step_host_async (steps enqueued back to back, one synchronisation at the end:
        # how a training loop calls it) and seg_train_step_host (waits for every loss).
        e_steps = max(3, min(steps, 50))
        h2d = sum(w.batch * (spec.widths[0] * (2 if w.precision == "bf16" else 4) + 4) for spec in w.segments)
        loss_pin = torch.zeros(e_steps + 3, len(r.segs), dtype=torch.float32).pin_memory()

        def e2e_loop(sync_every_step):
            for s in range(3 + e_steps):
                if s == 3:
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                sl = r.batch_slice(s)
                for k, seg in enumerate(r.segs):
                    if sync_every_step:
                        seg.train_step_host(r.host_x[k][sl], r.host_cls[sl])
                    else:
                        seg.train_step_host_async(r.host_x[k][sl], r.host_cls[sl], loss_pin[s, k:k + 1])
            torch.cuda.synchronize()
            return time.perf_counter() - t0

        dt_sync = e2e_loop(True)
        dt_async = e2e_loop(False)
        assert bool(torch.isfinite(loss_pin[3:]).all()) and float(loss_pin[3:].abs().sum()) > 0.0
        out["e2e"] = {"value": e_steps * w.batch / dt_async, "unit": "samples/s", "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": 4 * len(w.segments), "steps": e_steps,
                      "call": "seg_train_step_host_async per segment and step, one synchronisation after the last step",
                      "waiting_for_every_loss": {"value": e_steps * w.batch / dt_sync, "unit": "samples/s",
                                                 "call": "seg_train_step_host"}}
    if full and not w.concurrent:
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
    if full and not w.concurrent and len(w.segments) == 2:
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
                             "note": "bytes held by the library per handle (parameters, gradients, optimizer state, "
                                     "operand copy, activations, dZ, staging); segments trained one at a time need only "
                                     "the largest segment resident"}
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="paper_shaped", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--others", default="bf16_wide,gemm_large,multi_cut,tiny,paper_net",
                    help="further workloads summarised in the same line ('' for none)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--samples", type=int, default=0, help="size of the resident data set (0: the workload's own)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = wl.WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config = {"workload": f"{w.name}: " + " | ".join("-".join(map(str, s.widths)) for s in w.segments),
              "batch": w.batch, "optimizer": w.optimizer, "lr": w.lr, "n_classes": w.n_classes,
              "n_samples": w.n_samples, "label_dist": w.label_dist, "segments_per_step": len(w.segments),
              "cache": "inputs larger than L2: every step reads the next batch of a resident data set",
              "parallelism": "replicas only" if world > 1 else "single GPU"}

    if args.impl == "reference":
        if rank != 0:
            return
        base, _ = oracle_samples_per_s(w, budget_s=20.0, max_steps=max(args.steps, 1))
        line = {"impl": "reference", "metric": "segment train-step samples/sec", "value": base["value"],
                "unit": "samples/s", "n_gpus": 0, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": 1e3 * w.batch / base["value"], "higher_is_better": True, "scaling": "weak",
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
    res = measure(w, args.steps, args.warmup, peaks, device_index=local_rank, full=True,
                  n_samples=args.samples or None)
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
            "roofline": res.get("roofline"), "kernels": res.get("kernels"), "segments": res["segments"],
            "label_gen_ms": res["label_gen_ms"], "memory": res.get("memory"), "procedure": res.get("procedure"),
            "recovery": res.get("recovery"), "peaks": peaks}
    if not args.no_cpu_baseline:
        line["cpu_baseline"], _ = oracle_samples_per_s(w, budget_s=15.0)
    others = {}
    for name in [n for n in args.others.split(",") if n and n != args.workload]:
        ow = wl.WORKLOADS[name]
        k = max(5, min(args.steps, 30))
        try:
            r = measure(ow, k, 3, peaks, device_index=local_rank, full=False)
            others[name] = {"samples_per_s": r["samples_per_s"], "ms_per_step": r["ms_per_step"], "steps": k,
                            "precision": ow.precision, "optimizer": ow.optimizer, "batch": ow.batch,
                            "concurrent_streams": ow.concurrent, "memory": r.get("memory"),
                            "segments": [{kk: s[kk] for kk in ("segment", "ms_per_step", "samples_per_s", "roofline_frac",
                                                               "gemm_tflops", "mem_bytes_peak")} for s in r["segments"]]}
        except Exception as exc:                       # a secondary workload must not cost the headline
            others[name] = {"error": repr(exc)[:200]}
    line["others"] = others
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
