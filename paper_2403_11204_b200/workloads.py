"""Seeded synthetic workloads: shapes, hyper-parameters and input data only.

This module holds none of the method's arithmetic.  It describes the network
shapes the segment trainer is exercised on and draws the synthetic inputs
(features and class indices) that stand in for EMNIST-balanced-like data
(Section 3 of the paper: 784 features in [0,1], 47 balanced classes, 112,800
training samples).  Both the CUDA library's tests and the CPU oracle's tests
take their inputs from here, so that both sides see identical arrays.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

DATA_SEED = 0
LABEL_SEED = 1
INIT_SEED = 2


@dataclass(frozen=True)
class SegmentSpec:
    widths: List[int]            # input width, then each Linear layer's output width
    is_final: bool               # True: trained on class labels; False: on intermediate labels
    segment_id: int


@dataclass(frozen=True)
class Workload:
    name: str
    segments: List[SegmentSpec]
    n_classes: int
    n_samples: int
    batch: int
    precision: str               # "fp32" | "tf32" | "bf16"
    optimizer: str               # "sgd" | "momentum" | "adam"
    lr: float
    momentum: float = 0.9
    input_dist: str = "uniform"  # "uniform": U[0,1);  "normal": N(0,1)
    class_dist: str = "uniform"  # "uniform" | "balanced" | "zipf"
    zipf_s: float = 1.1
    label_dist: str = "normal"   # distribution of the intermediate labels in this workload
    epochs: int = 1
    concurrent: bool = False     # segments trained at the same time on separate streams
    note: str = ""

    @property
    def n_features(self) -> int:
        return self.segments[0].widths[0]


def _chain(widths_per_segment):
    segs = []
    for i, w in enumerate(widths_per_segment):
        segs.append(SegmentSpec(list(w), i == len(widths_per_segment) - 1, i))
    return segs


WORKLOADS = {
    # 6 Linear layers 784-128-128-64 | 64-64-47
    "tiny": Workload("tiny", _chain([[784, 128, 128, 64], [64, 64, 64, 47]]), 47, 2048, 64,
                     "fp32", "sgd", 0.01),
    # 784-1024-1024-512 | 512-256-47, EMNIST-balanced-sized
    "paper_shaped": Workload("paper_shaped", _chain([[784, 1024, 1024, 512], [512, 512, 256, 47]]),
                             47, 112800, 256, "tf32", "adam", 1e-3, class_dist="balanced", epochs=5),
    # 784-4096-4096-2048 | 2048-1024-62
    "bf16_wide": Workload("bf16_wide", _chain([[784, 4096, 4096, 2048], [2048, 2048, 1024, 62]]),
                          62, 262144, 1024, "bf16", "adam", 1e-3, class_dist="zipf"),
    # 1024-8192-8192-8192 | 8192-8192-1000
    "gemm_large": Workload("gemm_large", _chain([[1024, 8192, 8192, 8192], [8192, 8192, 8192, 1000]]),
                           1000, 65536, 4096, "bf16", "momentum", 0.01, input_dist="normal",
                           concurrent=True),
    # 12 Linear layers, hidden 4096, four segments of three layers
    "multi_cut": Workload("multi_cut", _chain([[784, 4096, 4096, 4096], [4096, 4096, 4096, 4096],
                                               [4096, 4096, 4096, 4096], [4096, 4096, 4096, 47]]),
                          47, 524288, 2048, "bf16", "adam", 1e-3),
    # the paper's own network (Section 3): 784-80-60 | 60-60-60-47, batch 1410, SGD momentum
    "paper_net": Workload("paper_net", _chain([[784, 80, 60], [60, 60, 60, 47]]), 47, 112800, 1410,
                          "fp32", "momentum", 0.01, class_dist="balanced", label_dist="uniform_kappa"),
}


def class_indices(wl: Workload, n: int, seed: int = DATA_SEED) -> np.ndarray:
    """int32 class index per sample, following the workload's class distribution."""
    g = np.random.Generator(np.random.PCG64(seed + 1000))
    m = wl.n_classes
    if wl.class_dist == "balanced":
        reps = -(-n // m)
        c = np.tile(np.arange(m, dtype=np.int32), reps)[:n]
        return g.permutation(c).astype(np.int32)
    if wl.class_dist == "zipf":
        p = 1.0 / np.arange(1, m + 1, dtype=np.float64) ** wl.zipf_s
        return g.choice(m, size=n, p=p / p.sum()).astype(np.int32)
    return g.integers(0, m, size=n, dtype=np.int32)


def features(wl: Workload, n: int, width: Optional[int] = None, seed: int = DATA_SEED) -> np.ndarray:
    """fp32 [n, width] inputs: U[0,1) (image-like) or N(0,1)."""
    g = np.random.Generator(np.random.PCG64(seed))
    width = wl.n_features if width is None else width
    if wl.input_dist == "normal":
        return g.standard_normal((n, width), dtype=np.float32)
    return g.random((n, width), dtype=np.float32)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Storage conversion of fp32 inputs to bf16 bit patterns (uint16), nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """fp32 values of bf16 bit patterns."""
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)
