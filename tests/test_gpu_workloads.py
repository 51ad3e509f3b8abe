"""The five synthetic workloads at full shape, in the launch configuration the benchmark times
(automatic backend: tcgen05 products for TF32 / bf16, FFMA for fp32), against the oracle:
one full training step per segment compared tensor by tensor, and 100-step loss curves.

Tolerances as in test_gpu_parity.py: fp32 1e-4, TF32 2e-3, bf16 2e-2; loss curves within 1 %.
The oracle runs the same step in NumPy (fp64 accumulation) with the same seeded arrays; its
weights come from its own initialisation, which the CUDA side must reproduce bit for bit."""
import os

import numpy as np
import pytest

from paper_2403_11204_b200 import workloads as wl
from parity_util import (batch_arrays, bits_equal, compare_step, make_oracle, make_pair, oracle_loss_curve,
                         segment_input, to_device)

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "tf32": 2e-3, "bf16": 2e-2}


CASES = [(name, k) for name in ("tiny", "paper_shaped", "bf16_wide", "gemm_large", "multi_cut")
         for k in range(len(wl.WORKLOADS[name].segments))]


@pytest.mark.parametrize("name,k", CASES)
def test_full_shape_single_step(name, k):
    w = wl.WORKLOADS[name]
    spec = w.segments[k]
    gpu, ora = make_pair(spec.widths, w.n_classes, spec.is_final, w.precision, w.optimizer, w.lr, w.batch,
                         segment_id=spec.segment_id, label_dist=w.label_dist, momentum=w.momentum)
    for l in range(ora.n_layers):                       # initialisation: bit-exact at full size
        W, b = gpu.params(l)
        assert bits_equal(W.cpu().numpy(), ora.W[l]) and bits_equal(b.cpu().numpy(), ora.b[l])
    if not spec.is_final:
        assert bits_equal(gpu.labels().cpu().numpy(), ora.sil)
    x, cls = segment_input(w, spec, w.batch)
    # the reduced-precision paths are held to the oracle's matching mode (tight) and to its plain fp32 mode
    plain = None
    if w.precision != "fp32":
        plain = make_oracle(spec.widths, w.n_classes, spec.is_final, "fp32", w.optimizer, w.lr,
                            segment_id=spec.segment_id, label_dist=w.label_dist, momentum=w.momentum)
    report = {}
    errs = compare_step(gpu, ora, x, cls, w.precision, TOL[w.precision], ora_plain=plain, report=report)
    print(name, k, {n: f"{v:.1e}" for n, v in errs.items()})
    for key, val in report.items():
        print("   ", key, {n: f"{v:.1e}" for n, v in val.items()} if isinstance(val, dict) else f"{val:.1e}")
    fam = gpu.product_launches()
    assert (fam["ffma"] == 0) == (w.precision != "fp32"), fam       # tensor cores for TF32 / bf16, FFMA for fp32
    gpu.close()


def test_paper_shaped_last_partial_batch():
    """112,800 = 440 * 256 + 160: the last batch of an epoch has 160 samples (means over 160)."""
    w = wl.WORKLOADS["paper_shaped"]
    spec = w.segments[0]
    gpu, ora = make_pair(spec.widths, w.n_classes, False, w.precision, w.optimizer, w.lr, w.batch)
    x, cls = segment_input(w, spec, w.n_samples % w.batch)
    assert x.shape[0] == 160
    compare_step(gpu, ora, x, cls, w.precision, TOL[w.precision])
    gpu.close()


def test_paper_network_batch_1410_uniform_kappa_labels():
    """The paper's own network and settings (Section 3): 784-80-60 | 60-60-60-47, kappa = 10,
    SGD momentum 0.9, batch 1410."""
    w = wl.WORKLOADS["paper_net"]
    for spec in w.segments:
        gpu, ora = make_pair(spec.widths, w.n_classes, spec.is_final, "fp32", "momentum", 0.01, w.batch,
                             segment_id=spec.segment_id, label_dist="uniform_kappa", kappa=10.0)
        x, cls = segment_input(w, spec, w.batch)
        compare_step(gpu, ora, x, cls, "fp32", 1e-4)
        x2, cls2 = segment_input(w, spec, w.batch, seed=9)
        compare_step(gpu, ora, x2, cls2, "fp32", 1e-4)
        gpu.close()


CURVES = [
    # workload, segment, batch (full widths everywhere; batch reduced where the oracle would take minutes)
    ("tiny", 0, 64), ("tiny", 1, 64),
    ("paper_shaped", 0, 256), ("paper_shaped", 1, 256),
    ("bf16_wide", 1, 256),
]
# Segments of 28 M to 143 M parameters: one oracle step costs seconds whatever the batch (every weight matrix
# is converted and rounded at each use), so their oracle curves are computed side by side in worker processes
# while this process only runs the CUDA side.
LARGE_CURVES = [("bf16_wide", 0, 64), ("multi_cut", 0, 64), ("multi_cut", 1, 64), ("multi_cut", 2, 64),
                ("multi_cut", 3, 256), ("gemm_large", 0, 32), ("gemm_large", 1, 32)]
STEPS = 100


def gpu_loss_curve(name, k, batch, steps=STEPS):
    import torch
    w = wl.WORKLOADS[name]
    spec = w.segments[k]
    n = min(w.n_samples, steps * batch)                # the first 100 batches of an epoch, in order
    from paper_2403_11204_b200.binding import Segment
    gpu = Segment(spec.widths, w.n_classes, spec.is_final, precision=w.precision, optimizer=w.optimizer, lr=w.lr,
                  momentum=w.momentum, max_batch=batch, segment_id=spec.segment_id, init_seed=wl.INIT_SEED)
    if not spec.is_final:
        gpu.gen_labels(wl.LABEL_SEED, w.label_dist)
    x, cls = segment_input(w, spec, n)
    xt, ct = to_device(x, cls, w.precision)
    losses = torch.zeros(steps, device="cuda")
    for s in range(steps):
        i = (s * batch) % n
        gpu.train_step(xt[i:i + batch], ct[i:i + batch], losses[s:s + 1])
    gpu.poll()
    got = losses.cpu().numpy().astype(np.float64)
    gpu.close()
    return got


@pytest.mark.parametrize("name,k,batch", CURVES)
def test_loss_curve_100_steps(name, k, batch):
    got = gpu_loss_curve(name, k, batch)
    ref = oracle_loss_curve((name, k, batch, STEPS, 0))
    rel = np.abs(got - ref) / np.abs(ref)
    print(name, k, "loss", ref[0], "->", ref[-1], "max rel diff", rel.max())
    assert rel.max() < 1e-2, (int(rel.argmax()), float(rel.max()))


def test_loss_curves_100_steps_of_the_large_segments():
    """bf16_wide segment 0, all four multi_cut segments and both gemm_large segments at full widths."""
    import multiprocessing as mp
    ctx = mp.get_context("spawn")                      # never fork a process that holds a CUDA context
    threads = max(1, (os.cpu_count() or 8) // len(LARGE_CURVES))
    with ctx.Pool(len(LARGE_CURVES)) as pool:
        pending = pool.map_async(oracle_loss_curve, [(n, k, b, STEPS, threads) for n, k, b in LARGE_CURVES])
        got = [gpu_loss_curve(n, k, b) for n, k, b in LARGE_CURVES]
        refs = pending.get(timeout=1500)
    worst = {}
    for (name, k, batch), g, ref in zip(LARGE_CURVES, got, refs):
        rel = np.abs(g - ref) / np.abs(ref)
        worst[(name, k)] = float(rel.max())
        print(name, k, "batch", batch, "loss", ref[0], "->", ref[-1], "max rel diff", rel.max())
    bad = {c: v for c, v in worst.items() if not v < 1e-2}
    assert not bad, bad
