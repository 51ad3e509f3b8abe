"""CUDA path against the oracle, through the C ABI.  Tolerances (max |diff| / max |ref| per tensor):
fp32 path 1e-4; bf16 path 2e-2; TF32 path 2e-3.  The reduced-precision paths quantise computed
values (activations, dZ) before the next product, so two correct implementations whose fp32/fp64
sums differ in the last bit can round one element to neighbouring grid points: half a TF32 ulp is
2^-11 = 4.9e-4 of that element, half a bf16 ulp 2^-9 = 2e-3.  The fp32 figure 1e-4 therefore
cannot hold for a TF32 path; 2e-3 leaves the same head-room over one flip that 2e-2 leaves bf16."""
import numpy as np
import pytest

from oracle import rng as orng
from paper_2403_11204_b200 import workloads as wl
import os

from parity_util import (batch_arrays, bits_equal, compare_step, make_oracle, make_pair, rel_err, sync_from_oracle,
                         to_device)

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "tf32": 2e-3, "bf16": 2e-2}


# ---- (1) label generation and initialisation: bit-exact -----------------------------------
@pytest.mark.parametrize("m,n_p", [(47, 64), (47, 60), (62, 2048), (3, 5), (1, 1), (1000, 1031)])
@pytest.mark.parametrize("dist", ["uniform_kappa", "normal"])
def test_labels_bit_exact(m, n_p, dist):
    gpu, ora = make_pair([16, n_p], m, False, "fp32", "sgd", 0.01, 4, segment_id=3, label_dist=dist,
                         label_seed=0x1234567890ABCDEF)
    assert bits_equal(gpu.labels().cpu().numpy(), ora.sil)
    gpu.close()


def test_label_values_do_not_depend_on_other_handles_or_order():
    a, ora = make_pair([8, 96], 10, False, "fp32", "sgd", 0.01, 4, segment_id=1)
    b, _ = make_pair([8, 96], 10, False, "bf16", "adam", 0.01, 4, segment_id=1, gemm_backend="simt")
    assert bits_equal(a.labels().cpu().numpy(), b.labels().cpu().numpy())
    assert bits_equal(a.labels().cpu().numpy(), ora.sil)
    a.close(); b.close()


@pytest.mark.parametrize("widths", [[784, 128, 128, 64], [64, 64, 64, 47], [60, 60, 60, 47], [5, 3]])
def test_initialisation_bit_exact(widths):
    gpu, ora = make_pair(widths, 47, widths[-1] == 47, "fp32", "sgd", 0.01, 4, segment_id=2)
    for l in range(ora.n_layers):
        W, b = gpu.params(l)
        assert bits_equal(W.cpu().numpy(), ora.W[l]) and bits_equal(b.cpu().numpy(), ora.b[l])
    gpu.close()


# ---- (2)-(4) one step: activations, loss, gradients, updated weights ----------------------------
SMALL = [
    # widths, final, precision, optimizer, batch
    ([784, 128, 128, 64], False, "fp32", "sgd", 64),
    ([64, 64, 64, 47], True, "fp32", "sgd", 64),
    ([784, 80, 60], False, "fp32", "momentum", 141),
    ([60, 60, 60, 47], True, "fp32", "momentum", 141),
    ([100, 72, 40], False, "fp32", "adam", 33),
    ([40, 24, 47], True, "fp32", "adam", 1),
    # wider than the two-launch step of small segments takes: the FFMA products, loss and update kernels
    ([200, 160, 96], False, "fp32", "adam", 50),
    ([96, 160, 47], True, "fp32", "momentum", 50),
    # four layers; a batch large enough for the 16-row slices, with a ragged last slice
    ([33, 128, 7, 128, 12], False, "fp32", "momentum", 77),
    ([60, 60, 47], True, "fp32", "sgd", 2405),
    ([1024, 47], True, "fp32", "adam", 9),
]


@pytest.mark.parametrize("widths,final,precision,optimizer,batch", SMALL)
def test_single_step_fp32(widths, final, precision, optimizer, batch):
    w = wl.WORKLOADS["tiny"]
    gpu, ora = make_pair(widths, 47, final, precision, optimizer, 0.01, batch)
    x, cls = batch_arrays(w, batch, widths[0])
    compare_step(gpu, ora, x, cls, precision, TOL[precision])
    x2, cls2 = batch_arrays(w, batch, widths[0], seed=7)
    if optimizer == "adam":
        sync_from_oracle(gpu, ora)
    compare_step(gpu, ora, x2, cls2, precision, TOL[precision])      # second step: optimizer state in play
    gpu.close()


def test_small_fp32_segment_steps_in_two_launches():
    """A small fp32 segment (the paper's 784-80-60 and 60-60-60-47) runs its whole step as two launches:
    the launch counter grows by two per step, eager, captured and replayed alike, both count as FFMA and one as a
    weight-gradient product that applied the update; a wider segment goes launch by launch."""
    import os
    if os.environ.get("SEG_NO_SMALL_FUSED") == "1":
        pytest.skip("the two-launch step is switched off in this process")
    w = wl.WORKLOADS["paper_net"]
    for widths, final, small in (([784, 80, 60], False, True), ([60, 60, 60, 47], True, True),
                                 ([784, 160, 60], False, False)):
        gpu, _ = make_pair(widths, 47, final, "fp32", "momentum", 0.01, 141)
        x, cls = batch_arrays(w, 141, widths[0])
        xt, ct = to_device(x, cls, "fp32")
        counts = []
        for _ in range(4):
            before = gpu.launch_count()
            gpu.train_step(xt, ct)
            counts.append(gpu.launch_count() - before)
        gpu.poll()
        fam = gpu.product_launches()
        if small:
            assert counts == [2, 2, 2, 2], counts
            assert (fam["ffma"], fam["fused_update"]) == (8, 4), fam
        else:
            assert min(counts) > 6 and fam["fused_update"] == 0, (counts, fam)
        gpu.close()


@pytest.mark.parametrize("label_dist", ["uniform_kappa", "normal"])
def test_tiny_workload_first_epoch_losses(label_dist):
    """The tiny workload, segment 1: every batch of one epoch, loss by loss (fp32, SGD)."""
    import torch
    w = wl.WORKLOADS["tiny"]
    spec = w.segments[0]
    gpu, ora = make_pair(spec.widths, w.n_classes, False, "fp32", "sgd", w.lr, w.batch, label_dist=label_dist)
    x, cls = batch_arrays(w, w.n_samples, spec.widths[0])
    xt, ct = to_device(x, cls, "fp32")
    losses = torch.zeros(w.n_samples // w.batch, device="cuda")
    ref = []
    for i in range(w.n_samples // w.batch):
        sl = slice(i * w.batch, (i + 1) * w.batch)
        gpu.train_step(xt[sl], ct[sl], losses[i:i + 1])
        ref.append(ora.train_step(x[sl], cls[sl]))
    gpu.poll()
    got = losses.cpu().numpy()
    assert np.max(np.abs(got - np.array(ref)) / np.abs(ref)) < 1e-4
    gpu.close()


REDUCED = [
    ([96, 80, 64, 48], False, "tf32", "adam", 40),
    ([48, 64, 32, 47], True, "tf32", "adam", 40),
    ([96, 80, 64, 48], False, "bf16", "adam", 40),
    ([48, 64, 32, 47], True, "bf16", "momentum", 40),
    ([784, 256, 128, 64], False, "bf16", "sgd", 200),
]


@pytest.mark.parametrize("widths,final,precision,optimizer,batch", REDUCED)
def test_single_step_reduced_precision_simt_backend(widths, final, precision, optimizer, batch):
    """Rounding points of the TF32 / bf16 modes, run on the FFMA kernels."""
    w = wl.WORKLOADS["tiny"]
    gpu, ora = make_pair(widths, 47, final, precision, optimizer, 1e-3, batch, gemm_backend="simt")
    x, cls = batch_arrays(w, batch, widths[0], precision=precision)
    compare_step(gpu, ora, x, cls, precision, TOL[precision])
    gpu.close()


def test_forward_only_and_set_params_route():
    import torch
    w = wl.WORKLOADS["tiny"]
    gpu, ora = make_pair([784, 128, 128, 64], 47, False, "fp32", "sgd", 0.01, 64, init_seed=11)
    g = np.random.default_rng(0)
    for l in range(ora.n_layers):                          # inject other weights on both sides
        ora.W[l] = (g.standard_normal(ora.W[l].shape) * 0.05).astype(np.float32)
        ora.b[l] = (g.standard_normal(ora.b[l].shape) * 0.05).astype(np.float32)
        gpu.set_params(l, torch.from_numpy(ora.W[l]).cuda(), torch.from_numpy(ora.b[l]).cuda())
    x, cls = batch_arrays(w, 50, 784)
    xt, _ = to_device(x, cls, "fp32")
    y = gpu.forward(xt)
    gpu.poll()
    assert rel_err(y.cpu().numpy(), ora.forward(x)[-1]) < 1e-4
    gpu.close()


@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_step_matches_device_step(pinned):
    """Page-locked batches are read by the staging kernel straight from host memory, pageable ones go
    through a device copy; both must give the oracle's step, two steps in a row (second batch differs)."""
    import torch
    w = wl.WORKLOADS["tiny"]
    a, ora = make_pair([784, 128, 128, 64], 47, False, "fp32", "sgd", 0.01, 64)
    x, cls = batch_arrays(w, 128, 784)
    for lo in (0, 64):
        xb, cb = x[lo:lo + 64].copy(), cls[lo:lo + 64].astype(np.int32)
        xt, ct = torch.from_numpy(xb), torch.from_numpy(cb)
        if pinned:
            xt, ct = xt.pin_memory(), ct.pin_memory()
        loss = a.train_step_host(xt, ct)
        ref = ora.train_step(xb, cls[lo:lo + 64])
        assert abs(loss - ref) / abs(ref) < 1e-4
    W, _ = a.params(0)
    assert rel_err(W.cpu().numpy(), ora.W[0]) < 1e-4
    a.close()


def test_host_buffer_step_without_wait():
    """seg_train_step_host_async: three steps enqueued back to back from pinned batches, losses read after
    one synchronisation; pageable buffers are refused."""
    import torch
    from paper_2403_11204_b200.binding import SegError
    w = wl.WORKLOADS["tiny"]
    a, ora = make_pair([784, 128, 128, 64], 47, False, "fp32", "sgd", 0.01, 64)
    x, cls = batch_arrays(w, 192, 784)
    xs = torch.from_numpy(x).pin_memory()
    cs = torch.from_numpy(cls.astype(np.int32)).pin_memory()
    losses = torch.zeros(3, dtype=torch.float32).pin_memory()
    for i in range(3):
        a.train_step_host_async(xs[64 * i:64 * (i + 1)], cs[64 * i:64 * (i + 1)], losses[i:i + 1])
    a.poll()
    for i in range(3):
        ref = ora.train_step(x[64 * i:64 * (i + 1)], cls[64 * i:64 * (i + 1)])
        assert abs(float(losses[i]) - ref) / abs(ref) < 1e-4
    W, _ = a.params(0)
    assert rel_err(W.cpu().numpy(), ora.W[0]) < 1e-4
    with pytest.raises(SegError) as e:
        a.train_step_host_async(torch.from_numpy(x[:64].copy()), cs[:64])
    assert e.value.status == 1
    a.close()


@pytest.mark.parametrize("widths,final,precision,batch", [([784, 80, 60], False, "fp32", 1410),
                                                          ([60, 60, 60, 47], True, "fp32", 1410),
                                                          ([784, 1024, 512], False, "tf32", 256),
                                                          ([512, 256, 47], True, "bf16", 200)])
def test_step_is_bit_reproducible(widths, final, precision, batch):
    """Every reduction of the step runs in a fixed order (loss partials, bias gradient, the K split of the
    FFMA and tensor-core products): two handles given the same batches end with identical bits."""
    import torch
    w = wl.WORKLOADS["paper_net"]
    x, cls = batch_arrays(w, batch, widths[0], precision=precision)
    results = []
    for _ in range(2):
        gpu, _ = make_pair(widths, 47, final, precision, "momentum", 0.01, batch)
        xt, ct = to_device(x, cls, precision)
        loss = torch.zeros(3, device="cuda")
        for i in range(3):
            gpu.train_step(xt, ct, loss[i:i + 1])
        gpu.poll()
        tensors = [loss.cpu().numpy()]
        for l in range(len(widths) - 1):
            W, b = gpu.params(l)
            dW, db = gpu.grads(l)
            tensors += [W.cpu().numpy(), b.cpu().numpy(), dW.cpu().numpy(), db.cpu().numpy()]
        results.append(tensors)
        gpu.close()
    for a, b in zip(*results):
        assert bits_equal(a, b)


def test_argument_errors_and_state():
    import torch
    from paper_2403_11204_b200.binding import SegError, Segment
    seg = Segment([16, 8], 4, False, max_batch=8)
    x = torch.zeros(4, 16, device="cuda")
    c = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(SegError) as e:
        seg.train_step(x, c)                               # labels never generated
    assert e.value.status == 6
    seg.gen_labels(1)
    with pytest.raises(SegError) as e:
        seg.train_step(torch.zeros(9, 16, device="cuda"), torch.zeros(9, dtype=torch.int32, device="cuda"))
    assert e.value.status == 2                             # batch > max_batch
    empty = torch.zeros(0, 16, device="cuda")
    with pytest.raises(SegError) as e:
        seg.train_step(empty, torch.zeros(0, dtype=torch.int32, device="cuda"))
    assert e.value.status in (1, 2)                        # an empty batch is refused (null pointer or shape), nothing is enqueued
    seg.train_step(x, c)
    seg.poll()
    cur, peak = seg.mem_bytes()
    assert 0 < cur <= peak
    assert seg.launch_count() > 0
    seg.close()
    fin = Segment([16, 4], 4, True, max_batch=8)
    with pytest.raises(SegError):
        fin.gen_labels(1)                                  # the final segment has no intermediate labels
    fin.close()


# ---- tensor-core products (tcgen05) against the oracle -----------------------------------------
TC_CASES = [
    # widths, final, precision, optimizer, batch   (shapes chosen to span several tiles + ragged tails)
    ([64, 128], False, "bf16", "sgd", 128),                 # one tile, forward + wgrad only
    ([128, 256, 128], False, "bf16", "sgd", 256),           # adds dgrad
    ([784, 320, 200, 72], False, "bf16", "adam", 300),      # K tail (784), ragged M / N
    ([72, 136, 264, 47], True, "bf16", "momentum", 129),    # final segment, 47 logits in fp32
    ([1024, 512, 512], False, "bf16", "adam", 1024),        # many tiles, several k blocks
    ([64, 128], False, "tf32", "sgd", 128),
    ([784, 320, 200, 72], False, "tf32", "adam", 300),
    ([72, 136, 264, 47], True, "tf32", "adam", 129),
    # the paper's own partitions (Section 3) on tensor cores: widths 80 / 60 / 47 are not multiples of 8 elements
    ([784, 80, 60], False, "bf16", "momentum", 1410),
    ([60, 60, 60, 47], True, "bf16", "momentum", 1410),
    ([784, 80, 60], False, "tf32", "momentum", 1410),
    ([60, 60, 60, 47], True, "tf32", "momentum", 1410),
    ([33, 17, 9], False, "bf16", "sgd", 5),                 # everything smaller than one tile, odd widths
    ([8, 8], False, "tf32", "sgd", 1),                      # a single sample
]


def expected_families(widths, batch):
    """Which product-kernel families a step of this shape must / must not launch, given the selection
    switches this process runs under (the forced-selection child runs set them)."""
    must, never = set(), {"ffma"}                     # SEG_GEMM_TCGEN05: never the FFMA kernels
    if os.environ.get("SEG_NO_SPLITK") == "1":
        never.add("tc_splitk")
    if os.environ.get("SEG_NO_PAIRS") == "1":
        never.add("tc_pair")
    if os.environ.get("SEG_NO_SPLITK") == "1" and os.environ.get("SEG_NO_PAIRS") == "1":
        must.add("tc_single")
    if os.environ.get("SEG_PAIR_MIN_TILES") == "1" and os.environ.get("SEG_NO_PAIRS") != "1":
        # pairs from one 256 x 256 tile on: the products of the 1024-512-512 case are too short to be split over K
        if batch >= 1024 and min(widths) >= 512:
            must.add("tc_pair")
    if os.environ.get("SEG_FUSED_UPDATE") != "1":
        never.add("fused_update")
    elif os.environ.get("SEG_NO_SPLITK") == "1":
        must.add("fused_update")                      # every weight gradient runs in a persistent kernel
    return must, never


@pytest.mark.parametrize("widths,final,precision,optimizer,batch", TC_CASES)
def test_single_step_tensor_core_backend(widths, final, precision, optimizer, batch):
    w = wl.WORKLOADS["tiny"]
    gpu, ora = make_pair(widths, 47, final, precision, optimizer, 1e-3, batch, gemm_backend="tcgen05")
    plain = make_oracle(widths, 47, final, "fp32", optimizer, 1e-3)
    x, cls = batch_arrays(w, batch, widths[0], precision=precision)
    report = {}
    compare_step(gpu, ora, x, cls, precision, TOL[precision], ora_plain=plain, report=report)
    print(widths, precision, {k: v for k, v in report.items() if k != "vs_plain_fp32_oracle"},
          "vs plain fp32 oracle:", {k: f"{v:.1e}" for k, v in report["vs_plain_fp32_oracle"].items()})
    x2, cls2 = batch_arrays(w, max(batch - 1, 1), widths[0], seed=5, precision=precision)
    if optimizer == "adam":
        sync_from_oracle(gpu, ora)
    compare_step(gpu, ora, x2, cls2, precision, TOL[precision])      # smaller batch on the same handle
    # which kernels ran: every product of both steps on tensor cores, in the family the switches allow
    fam = gpu.product_launches()
    n_products = 2 * (3 * len(widths) - 4)            # per step: L forward, L weight-gradient, L - 1 dgrad products
    assert sum(fam[f] for f in ("tc_single", "tc_splitk", "tc_pair", "ffma")) == n_products, fam
    must, never = expected_families(widths, batch)
    assert all(fam[f] == 0 for f in never), (fam, never)
    assert all(fam[f] > 0 for f in must), (fam, must)
    gpu.close()


def test_product_family_counters_tell_the_backends_apart():
    """seg_product_launches is what the tensor-core tests rely on to show that tcgen05 kernels ran, so it is
    checked from both sides: a bf16 handle on the automatic or the tensor-core backend counts its five
    products (2 forward, 2 weight-gradient, 1 dgrad) as tensor-core launches and none as FFMA; the same
    segment on the FFMA backend counts all five as FFMA.  (With SEG_GEMM_TCGEN05 a product the tensor-core
    path could not take would be SEG_ERR_UNSUPPORTED, never an FFMA launch; the handle's own buffers are
    always laid out so that it can.)"""
    import torch
    from paper_2403_11204_b200.binding import Segment
    x = torch.rand(8, 24, device="cuda").to(torch.bfloat16)
    cls = torch.zeros(8, dtype=torch.int32, device="cuda")
    for backend in ("auto", "tcgen05", "simt"):
        seg = Segment([24, 16, 8], 47, False, precision="bf16", max_batch=8, gemm_backend=backend)
        seg.gen_labels(1)
        for _ in range(4):                               # eager, captured and replayed steps all count
            seg.train_step(x, cls)
        seg.poll()
        fam = seg.product_launches()
        tc = fam["tc_single"] + fam["tc_splitk"] + fam["tc_pair"]
        assert (fam["ffma"], tc) == ((20, 0) if backend == "simt" else (0, 20)), (backend, fam)
        seg.close()


def test_replayed_step_reports_its_own_batch_size():
    """A step replayed from its captured graph must leave the handle knowing that step's batch size:
    seg_get_activation after it copies exactly that many rows (guard rows behind the buffer stay
    untouched), also when a forward pass at a larger batch ran in between."""
    import torch
    w = wl.WORKLOADS["tiny"]
    A, B = 24, 64
    gpu, ora = make_pair([784, 128, 64], 47, False, "fp32", "sgd", 0.01, B)
    x, cls = batch_arrays(w, B, 784)
    xt, ct = to_device(x, cls, "fp32")
    for _ in range(3):                                   # eager, capture, replay at batch A
        gpu.train_step(xt[:A], ct[:A])
        ora.train_step(x[:A], cls[:A])
    gpu.forward(xt)                                      # batch B in between
    gpu.train_step(xt[:A], ct[:A])                       # replayed
    ora.loss_and_grads(x[:A], cls[:A])
    buf = torch.full((A + 8, 64), -7.0, device="cuda")   # A rows for the call, 8 guard rows behind them
    st = gpu.lib.seg_get_activation(gpu.h, 2, buf.data_ptr())
    assert st == 0
    gpu.poll()
    got = buf.cpu().numpy()
    assert np.all(got[A:] == -7.0), "rows beyond the step's batch were written"
    assert rel_err(got[:A], ora.acts[2]) < 1e-4
    gpu.close()


def test_bounded_wait_runs_out_and_the_handle_stays_usable():
    """The product kernels' wait routine, given a barrier nothing arrives at and a limit of one millisecond,
    gives up, records it, and returns: seg_poll_status reports the time-out once, the next poll is clean,
    and a training step on the same handle afterwards still matches the oracle."""
    from paper_2403_11204_b200.binding import SegError
    w = wl.WORKLOADS["tiny"]
    gpu, ora = make_pair([64, 128], 47, False, "bf16", "sgd", 0.01, 128, gemm_backend="tcgen05")
    gpu.selftest_bounded_wait(1_000_000)
    with pytest.raises(SegError) as e:
        gpu.poll()
    assert e.value.status == 7
    gpu.poll()                                           # the record is cleared by the poll that reported it
    with pytest.raises(SegError) as e:
        gpu.selftest_bounded_wait(10)                    # limits outside [1 us, 1 s] are refused
    assert e.value.status == 1
    x, cls = batch_arrays(w, 128, 64, precision="bf16")
    compare_step(gpu, ora, x, cls, "bf16", TOL["bf16"])
    gpu.close()


def test_class_index_out_of_range_is_clamped_and_reported():
    import torch
    from paper_2403_11204_b200.binding import SegError
    w = wl.WORKLOADS["tiny"]
    gpu, ora = make_pair([64, 64, 32], 47, False, "fp32", "sgd", 0.01, 32)
    x, cls = batch_arrays(w, 32, 64)
    bad = cls.copy()
    bad[3], bad[17] = 47, -5                             # one past the end, one negative
    xt, ct = to_device(x, bad, "fp32")
    loss = torch.zeros(1, device="cuda")
    gpu.train_step(xt, ct, loss)
    with pytest.raises(SegError) as e:
        gpu.poll()
    assert e.value.status == 9
    clamped = np.clip(bad, 0, 46)
    ref = ora.train_step(x, clamped)                     # the step that ran is the step on the clamped indices
    assert abs(float(loss.item()) - ref) / abs(ref) < 1e-4
    gpu.poll()
    gpu.close()


def test_tie_ceiling_catches_a_widened_band():
    """The share of ReLU decisions the comparison may take from the CUDA path is bounded: with the band
    widened a hundredfold the same comparison must fail on that bound."""
    w = wl.WORKLOADS["tiny"]
    widths, batch = [784, 320, 200, 72], 300
    gpu, ora = make_pair(widths, 47, False, "bf16", "sgd", 1e-3, batch, gemm_backend="tcgen05")
    x, cls = batch_arrays(w, batch, widths[0], precision="bf16")
    with pytest.raises(AssertionError, match="tie band|large value at a tie|tie decisions"):
        compare_step(gpu, ora, x, cls, "bf16", TOL["bf16"], tie_scale=100.0)
    gpu.close()


def test_two_segments_hand_off_through_the_library_copy():
    """Section 2.1 deployment on the devices at hand: each segment is created on a device of its own when
    the machine has two, otherwise both on device 0 (same code path, the copy is then device-to-device):
    train the left segment, store its response, hand it to the right segment's device with
    seg_handoff_copy, train the right segment - against the oracle's procedure."""
    import torch
    from oracle import pnn
    from paper_2403_11204_b200 import binding
    from paper_2403_11204_b200.binding import Segment
    from parity_util import make_oracle
    w = wl.WORKLOADS["tiny"]
    devs = [0, 1] if torch.cuda.device_count() > 1 else [0, 0]
    specs = [([784, 64, 32], False), ([32, 32, 47], True)]
    segs, oras = [], []
    for k, (widths, final) in enumerate(specs):
        st = torch.cuda.Stream(device=devs[k])
        segs.append(Segment(widths, 47, final, precision="fp32", optimizer="momentum", lr=0.01, max_batch=64,
                            segment_id=k, stream=st, device=devs[k]))
        oras.append(make_oracle(widths, 47, final, "fp32", "momentum", 0.01, segment_id=k))
    segs[0].gen_labels(wl.LABEL_SEED, "normal")
    x, cls = batch_arrays(w, 200, 784)
    with torch.cuda.device(devs[0]):
        xt, ct = to_device(x, cls, "fp32")
    torch.cuda.synchronize()
    losses, _ = binding.train_partitioned(segs, xt, ct, 64, [2, 2])
    for s_ in segs:
        s_.poll()
    ref, _ = pnn.train_partitioned(oras, x, cls, 64, [2, 2])
    for got, want in zip(losses, ref):
        assert np.max(np.abs(got.cpu().numpy() - want) / np.abs(want)) < 1e-3
    for s_ in segs:
        s_.close()


def test_handles_created_and_used_from_two_threads():
    """Different handles may be created and used from different threads at the same time (the library's one-time set-up
    and per-device caches are synchronised): two threads each create a tensor-core segment on a stream of their own and
    run the same three steps; both must end with the bits a single-threaded run gives."""
    import threading
    import torch
    from paper_2403_11204_b200.binding import Segment
    w = wl.WORKLOADS["tiny"]
    widths, batch = [256, 384, 128], 192
    x, cls = batch_arrays(w, batch, widths[0], precision="bf16")
    xt, ct = to_device(x, cls, "bf16")

    def run(out, use_own_stream):
        st = torch.cuda.Stream() if use_own_stream else None
        seg = Segment(widths, 47, False, precision="bf16", optimizer="momentum", lr=0.01, max_batch=batch, stream=st)
        seg.gen_labels(wl.LABEL_SEED, "normal")
        loss = torch.zeros(3, device="cuda")
        for i in range(3):
            seg.train_step(xt, ct, loss[i:i + 1])
        seg.poll()
        W, b = seg.params(0)
        out.append((loss.cpu().numpy(), W.cpu().numpy(), b.cpu().numpy()))
        seg.close()

    ref = []
    run(ref, False)
    results = [[], []]
    threads = [threading.Thread(target=run, args=(results[i], True)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(120)
    for r in results:
        assert len(r) == 1, "a thread did not finish"
        for a, b in zip(r[0], ref[0]):
            assert bits_equal(a, b)
