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
from parity_util import batch_arrays, bits_equal, compare_step, make_pair, to_device

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "tf32": 2e-3, "bf16": 2e-2}


def segment_input(w, spec, n, seed=wl.DATA_SEED):
    """Features for segment 0; for later segments a stand-in for the previous segment's stored
    output: non-negative (post-ReLU-like) values of the right width, drawn from the same recipe."""
    x, cls = batch_arrays(w, n, spec.widths[0], seed=seed + 17 * spec.segment_id, precision=w.precision)
    if spec.segment_id > 0:
        x = np.abs(x)
    return x, cls


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
    errs = compare_step(gpu, ora, x, cls, w.precision, TOL[w.precision])
    print(name, k, {n: f"{v:.1e}" for n, v in errs.items()})
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
    ("bf16_wide", 0, 64), ("bf16_wide", 1, 256),
    ("multi_cut", 3, 256),
]
# The oracle converts and rounds every weight matrix at each use, which costs seconds per step on the
# 140 M-parameter segments whatever the batch; those curves run only when SEG_TEST_HEAVY=1.
HEAVY_CURVES = [("gemm_large", 1, 32), ("multi_cut", 1, 64)]
if os.environ.get("SEG_TEST_HEAVY") == "1":
    CURVES += HEAVY_CURVES


@pytest.mark.parametrize("name,k,batch", CURVES)
def test_loss_curve_100_steps(name, k, batch):
    import torch
    w = wl.WORKLOADS[name]
    spec = w.segments[k]
    steps = 100
    n = min(w.n_samples, steps * batch)                # the first 100 batches of an epoch, in order
    gpu, ora = make_pair(spec.widths, w.n_classes, spec.is_final, w.precision, w.optimizer, w.lr, batch,
                         segment_id=spec.segment_id, label_dist=w.label_dist, momentum=w.momentum)
    x, cls = segment_input(w, spec, n)
    xt, ct = to_device(x, cls, w.precision)
    losses = torch.zeros(steps, device="cuda")
    ref = np.zeros(steps)
    for s in range(steps):
        i = (s * batch) % n
        gpu.train_step(xt[i:i + batch], ct[i:i + batch], losses[s:s + 1])
        ref[s] = ora.train_step(x[i:i + batch], cls[i:i + batch])
    gpu.poll()
    got = losses.cpu().numpy().astype(np.float64)
    rel = np.abs(got - ref) / np.abs(ref)
    print(name, k, "loss", ref[0], "->", ref[-1], "max rel diff", rel.max())
    assert rel.max() < 1e-2, (int(rel.argmax()), float(rel.max()))
    gpu.close()
