"""Host-side arithmetic of the benchmark: the algorithmic FLOP / byte counts the roofline uses."""
import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench
from paper_2403_11204_b200 import workloads as wl


def test_gemm_flops_follow_6P_minus_first_layer_dgrad():
    # per sample: forward 2P + weight gradient 2P + dgrad 2(P - in0*out0), P = sum in*out
    w = wl.WORKLOADS["bf16_wide"]
    work = bench.segment_work(w.segments[0], w.batch, w.precision, w.optimizer)
    p = 784 * 4096 + 4096 * 4096 + 4096 * 2048
    assert p == 28_377_088
    assert work["gemm_flops"] == w.batch * (6 * p - 2 * 784 * 4096) == 167_772_160_000
    w4 = wl.WORKLOADS["gemm_large"]
    work4 = bench.segment_work(w4.segments[0], w4.batch, w4.precision, w4.optimizer)
    assert work4["gemm_flops"] == pytest.approx(3.436e12, rel=1e-3)


def test_update_bytes_per_parameter():
    w = wl.WORKLOADS["bf16_wide"]            # Adam, bf16 copy: 28 + 2 bytes per parameter
    work = bench.segment_work(w.segments[0], w.batch, w.precision, w.optimizer)
    assert work["update_bytes"] == 30 * work["params"]
    w2 = wl.WORKLOADS["paper_shaped"]        # Adam, TF32 copy: 28 + 4
    work2 = bench.segment_work(w2.segments[0], w2.batch, w2.precision, w2.optimizer)
    assert work2["update_bytes"] == 32 * work2["params"]
    w4 = wl.WORKLOADS["gemm_large"]          # momentum, bf16 copy: 20 + 2
    work4 = bench.segment_work(w4.segments[0], w4.batch, w4.precision, w4.optimizer)
    assert work4["update_bytes"] == 22 * work4["params"]


def test_workload_table_matches_the_configurations():
    t = wl.WORKLOADS
    assert [s.widths for s in t["tiny"].segments] == [[784, 128, 128, 64], [64, 64, 64, 47]]
    assert [s.widths for s in t["paper_shaped"].segments] == [[784, 1024, 1024, 512], [512, 512, 256, 47]]
    assert t["paper_shaped"].n_samples == 112800 and t["paper_shaped"].batch == 256
    assert t["paper_shaped"].n_samples % 256 == 160
    assert len(t["multi_cut"].segments) == 4 and all(len(s.widths) == 4 for s in t["multi_cut"].segments)
    assert t["paper_net"].n_samples // t["paper_net"].batch == 80          # Section 3: 80 steps per epoch
    for w in t.values():
        assert w.segments[-1].is_final and w.segments[-1].widths[-1] == w.n_classes
        for a, b in zip(w.segments, w.segments[1:]):
            assert a.widths[-1] == b.widths[0]


def test_class_distributions():
    import numpy as np
    w = t = wl.WORKLOADS["paper_shaped"]
    c = wl.class_indices(w, w.n_samples)
    assert np.bincount(c, minlength=47).tolist() == [2400] * 47           # balanced, as EMNIST balanced
    z = wl.WORKLOADS["bf16_wide"]
    cz = np.bincount(wl.class_indices(z, 200000), minlength=62)
    assert cz[0] > cz[10] > cz[61] > 0                                    # Zipf: frequent to rare
    assert abs(cz[0] / cz[1] - 2 ** 1.1) < 0.15
    x = wl.features(wl.WORKLOADS["tiny"], 1000)
    assert x.dtype == np.float32 and 0.0 <= x.min() and x.max() < 1.0
    b = wl.to_bf16_bits(x)
    assert np.max(np.abs(wl.from_bf16_bits(b) - x)) <= 2 ** -8


def test_step_fractions_follow_the_roofline_sum():
    """roofline time = product FLOPs at the tensor peak + update and loss bytes at the copy bandwidth; the step's fraction
    is that over the measured time, the tensor-only one counts the products alone."""
    peaks = {"hbm_gbs": 6000.0, "bf16_tflops": 1500.0, "bf16_tflops_sustained": 1200.0, "source": "test"}
    work = {"gemm_flops": 3.0e12, "update_bytes": 3.0e9, "loss_bytes": 0.0}
    f = bench.step_fractions(work, 4.0, "bf16", peaks)            # 2 ms of products + 0.5 ms of update in a 4 ms step
    assert f["roofline_ms"] == pytest.approx(2.5)
    assert f["roofline_frac"] == pytest.approx(0.625)
    assert f["gemm_tflops"] == pytest.approx(750.0)
    assert f["tensor_only_frac"] == pytest.approx(0.5)
    assert f["tensor_only_frac_of_sustained_matmul"] == pytest.approx(0.625)


def test_cpu_sample_rows_never_exceed_the_batch():
    for name, w in wl.WORKLOADS.items():
        assert 1 <= min(w.batch, bench.CPU_SAMPLE_BATCH.get(name, w.batch)) <= w.batch
