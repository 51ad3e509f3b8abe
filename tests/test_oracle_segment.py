"""Pins for oracle/segment.py: finite differences, closed forms, invariants, the paper's
printed figures.  A dropped term, a wrong sign or a transposed operand fails one of them."""
import math
import os

import numpy as np
import pytest

from oracle import rng
from oracle.segment import OracleSegment, mse_loss, round_bf16, round_tf32, softmax_ce_loss

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_section3.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            k, v = line.split("=")
            out[k.strip()] = v.split()
    return out


def make(widths, final, precision="fp64", optimizer="sgd", n_classes=3, **kw):
    seg = OracleSegment(widths, n_classes, final, precision=precision, optimizer=optimizer, **kw)
    if not final:
        seg.gen_labels(1, rng.DIST_NORMAL)
    return seg


def data(seg, bsz, seed=0):
    g = np.random.default_rng(seed)
    return g.random((bsz, seg.widths[0])), g.integers(0, seg.n_classes, bsz)


# ---- the paper's printed bookkeeping (Section 3) ---------------------------------------
def test_parameter_counts_printed_in_the_paper():
    gold = read_golden()
    n_in = int(gold["input_width"][0])
    left = [n_in] + [int(v) for v in gold["left_widths"]]
    right = [left[-1]] + [int(v) for v in gold["right_widths"]]
    m = int(gold["n_classes"][0])
    assert OracleSegment(left, m, False).n_params() == int(gold["left_parameters"][0])
    assert OracleSegment(right, m, True).n_params() == int(gold["right_parameters"][0])
    # MACs = parameters + one op per ReLU output: only the network's last layer has no ReLU
    lseg, rseg = OracleSegment(left, m, False), OracleSegment(right, m, True)
    relu_l = sum(lseg.widths[1:]) if lseg.last_relu else sum(lseg.widths[1:-1])
    relu_r = sum(rseg.widths[1:]) if rseg.last_relu else sum(rseg.widths[1:-1])
    assert lseg.n_params() + relu_l == int(gold["left_macs"][0])
    assert rseg.n_params() + relu_r == int(gold["right_macs"][0])
    assert int(gold["train_images"][0]) // int(gold["batch"][0]) == 80
    sil = lseg.gen_labels(1, rng.DIST_UNIFORM_KAPPA, float(gold["kappa"][0]))
    assert sil.T.shape == (int(gold["sil_rows"][0]), int(gold["sil_cols"][0]))


# ---- finite differences (all-fp64 mode) --------------------------------------------------
@pytest.mark.parametrize("final", [False, True])
@pytest.mark.parametrize("widths", [[5, 4, 3], [6, 5, 4, 3], [4, 3]])
def test_gradients_match_central_differences(final, widths):
    seg = make(widths, final)
    x, cls = data(seg, 3, seed=len(widths))
    seg.loss_and_grads(x, cls)
    dW = [g.copy() for g in seg.dW]
    db = [g.copy() for g in seg.db]
    h = 1e-6
    for l in range(seg.n_layers):
        for arr, grad in ((seg.W[l], dW[l]), (seg.b[l], db[l])):
            it = np.nditer(arr, flags=["multi_index"])
            for _ in it:
                idx = it.multi_index
                keep = arr[idx]
                arr[idx] = keep + h
                lp = seg.loss_and_grads(x, cls)
                arr[idx] = keep - h
                lm = seg.loss_and_grads(x, cls)
                arr[idx] = keep
                fd = (lp - lm) / (2 * h)
                assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9, (l, idx, fd, grad[idx])


# ---- closed form: one Linear layer under MSE ---------------------------------------------
def test_single_linear_layer_mse_closed_form_and_sgd_step():
    seg = make([7, 5], False, n_classes=4, last_relu=False, lr=0.05)
    x, cls = data(seg, 6)
    W0, b0 = seg.W[0].copy(), seg.b[0].copy()
    T = seg.sil[cls].astype(np.float64)
    Y = x @ W0.T + b0
    loss = seg.train_step(x, cls)
    n = Y.size
    dW = 2.0 / n * (Y - T).T @ x
    db = 2.0 / n * (Y - T).sum(axis=0)
    assert math.isclose(loss, np.mean((Y - T) ** 2), rel_tol=1e-12)
    assert np.allclose(seg.dW[0], dW, rtol=1e-12, atol=0)
    assert np.allclose(seg.db[0], db, rtol=1e-12, atol=0)
    assert np.allclose(seg.W[0], W0 - 0.05 * dW, rtol=1e-12, atol=0)
    assert np.allclose(seg.b[0], b0 - 0.05 * db, rtol=1e-12, atol=0)


def test_relu_at_the_cut_masks_the_gradient():
    seg = make([7, 5], False, n_classes=4)          # non-final: ReLU on the cut layer
    x, cls = data(seg, 6)
    seg.loss_and_grads(x, cls)
    out = seg.acts[-1]
    assert (out >= 0).all() and (out == 0).any() and (out > 0).any()
    assert np.all(seg.dZ[-1][out == 0] == 0)


# ---- softmax cross-entropy ------------------------------------------------------------
@pytest.mark.parametrize("m", [47, 62, 1000])
def test_softmax_ce_zero_logits_is_log_m(m):
    cls = np.arange(5) % m
    loss, dz = softmax_ce_loss(np.zeros((5, m)), cls)
    assert math.isclose(loss, math.log(m), rel_tol=1e-14)
    assert np.allclose(dz.sum(axis=1), 0.0, atol=1e-15)
    want = np.full((5, m), 1.0 / m)
    want[np.arange(5), cls] -= 1.0
    assert np.allclose(dz, want / 5, rtol=1e-13)


def test_softmax_ce_shift_invariance_and_row_sums():
    g = np.random.default_rng(1)
    z = g.normal(size=(4, 9)) * 5
    cls = g.integers(0, 9, 4)
    l0, d0 = softmax_ce_loss(z, cls)
    l1, d1 = softmax_ce_loss(z + np.array([[100.0], [-50.0], [3.0], [0.0]]), cls)
    assert math.isclose(l0, l1, rel_tol=1e-12) and np.allclose(d0, d1, atol=1e-14)
    assert np.allclose(d0.sum(axis=1), 0, atol=1e-15)
    # brute force, sample by sample
    brute = -np.mean([z[i, cls[i]] - math.log(sum(math.exp(v) for v in z[i])) for i in range(4)])
    assert math.isclose(l0, brute, rel_tol=1e-12)


def test_mse_matches_elementwise_brute_force():
    g = np.random.default_rng(2)
    a, t = g.normal(size=(3, 4)), g.normal(size=(3, 4))
    loss, da = mse_loss(a, t)
    assert math.isclose(loss, sum((a[i, j] - t[i, j]) ** 2 for i in range(3) for j in range(4)) / 12)
    assert np.allclose(da, (a - t) / 6.0)


# ---- training sanity -----------------------------------------------------------------
@pytest.mark.parametrize("final,opt,lr", [(False, "sgd", 0.05), (True, "sgd", 0.05),
                                           (False, "momentum", 0.01), (True, "adam", 1e-3)])
def test_loss_decreases_on_a_fixed_batch(final, opt, lr):
    seg = make([10, 8, 6], final, precision="fp32", optimizer=opt, lr=lr, n_classes=6)
    x, cls = data(seg, 16)
    losses = [seg.train_step(x.astype(np.float32), cls) for _ in range(8)]
    assert all(b < a for a, b in zip(losses, losses[1:])), losses


def test_target_equal_to_output_gives_zero_loss_and_no_update():
    seg = make([6, 5, 4], False, precision="fp32", n_classes=1)
    x = np.tile(np.random.default_rng(3).random((1, 6)).astype(np.float32), (4, 1))
    cls = np.zeros(4, dtype=np.int64)
    seg.sil = seg.forward(x)[-1][:1].copy()          # the single class's target = current output
    before = [p.copy() for p in seg.W + seg.b]
    assert seg.train_step(x, cls) == 0.0
    assert all(np.array_equal(a.view(np.uint32), b.view(np.uint32)) for a, b in zip(before, seg.W + seg.b))


# ---- optimizers -----------------------------------------------------------------------
def _one_step(opt, **kw):
    seg = make([6, 5, 4], False, optimizer=opt, **kw)
    x, cls = data(seg, 5)
    before = [p.copy() for p in seg.W + seg.b]
    seg.train_step(x, cls)
    return seg, before


def test_momentum_first_step_equals_sgd_and_mu_zero_is_sgd():
    a, _ = _one_step("sgd", lr=0.1)
    b, _ = _one_step("momentum", lr=0.1, momentum=0.9)
    assert all(np.array_equal(p, q) for p, q in zip(a.W + a.b, b.W + b.b))
    c = make([6, 5, 4], False, optimizer="momentum", lr=0.1, momentum=0.0)
    d = make([6, 5, 4], False, optimizer="sgd", lr=0.1)
    x, cls = data(c, 5)
    for _ in range(3):
        c.train_step(x, cls)
        d.train_step(x, cls)
    assert all(np.array_equal(p, q) for p, q in zip(c.W + c.b, d.W + d.b))


def test_momentum_second_step_by_hand():
    seg = make([6, 5, 4], False, optimizer="momentum", lr=0.1, momentum=0.9)
    x, cls = data(seg, 5)
    w0 = seg.W[0].copy()
    seg.train_step(x, cls)
    g1 = seg.dW[0].copy()
    w1 = seg.W[0].copy()
    seg.train_step(x, cls)
    g2 = seg.dW[0]
    assert np.allclose(w1, w0 - 0.1 * g1, rtol=1e-14)
    assert np.allclose(seg.W[0], w1 - 0.1 * (0.9 * g1 + g2), rtol=1e-13)


def test_adam_first_step_is_lr_times_normalised_gradient():
    seg, before = _one_step("adam", lr=1e-3, eps=1e-8)
    for p0, p1, g in zip(before, seg.W + seg.b, seg.dW + seg.db):
        assert np.allclose(p1 - p0, -1e-3 * g / (np.abs(g) + 1e-8), rtol=1e-9, atol=1e-16)


def test_adam_two_steps_by_hand_scalar():
    seg = make([3, 2], False, optimizer="adam", lr=1e-2, n_classes=2, last_relu=False)
    x, cls = data(seg, 4)
    p = float(seg.W[0][1, 2])
    m = v = 0.0
    for t in (1, 2):
        seg.loss_and_grads(x, cls)
        g = float(seg.dW[0][1, 2])
        m = 0.9 * m + 0.1 * g
        v = 0.999 * v + 0.001 * g * g
        p = p - 1e-2 * (m / (1 - 0.9 ** t)) / (math.sqrt(v / (1 - 0.999 ** t)) + 1e-8)
        seg.apply_update()
        assert math.isclose(float(seg.W[0][1, 2]), p, rel_tol=1e-12)


# ---- gather by class (Section 3: the label of an image is its class's SIL column) -----------
def test_same_class_same_target_and_permutation_invariance():
    seg = make([8, 6, 5], False, n_classes=4)
    x, cls = data(seg, 9, seed=5)
    cls[3] = cls[7]
    seg.loss_and_grads(x, cls)
    t = seg.sil[cls]
    assert np.array_equal(t[3], t[7])
    g = [a.copy() for a in seg.dW + seg.db]
    perm = np.random.default_rng(0).permutation(9)
    seg.loss_and_grads(x[perm], cls[perm])
    assert all(np.allclose(a, b, rtol=1e-12, atol=1e-18) for a, b in zip(g, seg.dW + seg.db))


# ---- segments are independent; the unpartitioned network is one long final segment -----------
def test_chained_segments_reproduce_the_unpartitioned_forward():
    left = make([9, 7, 5], False, n_classes=4, segment_id=0)
    right = make([5, 6, 4], True, n_classes=4, segment_id=1)
    whole = OracleSegment([9, 7, 5, 6, 4], 4, True, precision="fp64")
    whole.W = [w.copy() for w in left.W + right.W]
    whole.b = [b.copy() for b in left.b + right.b]
    x, _ = data(left, 5)
    assert np.array_equal(right.forward(left.forward(x)[-1])[-1], whole.forward(x)[-1])
    snapshot = [p.copy() for p in right.W + right.b]
    left.train_step(x, np.zeros(5, dtype=np.int64))
    assert all(np.array_equal(a, b) for a, b in zip(snapshot, right.W + right.b))


# ---- reduced-precision roundings ------------------------------------------------------
def test_rounding_helpers():
    a = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -9, -3.14159, 1e-30, 0.0], dtype=np.float32)
    b = round_bf16(a)
    assert float(b[0]) == 1.0 and float(b[2]) == 1.0 + 2 ** -7 and float(b[3]) == 1.0 + 2 ** -7
    assert b[1] == 1.0                                  # tie goes to the even mantissa
    assert float(round_bf16(np.float32(1.0 + 3 * 2 ** -8))) == 1.0 + 2 ** -6   # tie, odd -> up
    assert np.all(np.abs(b - a) <= np.abs(a) * 2 ** -8)
    t = round_tf32(a)
    assert np.all(np.abs(t - a) <= np.abs(a) * 2 ** -11)
    assert np.all((t.view(np.uint32) & 0x1FFF) == 0) and np.all((b.view(np.uint32) & 0xFFFF) == 0)
    assert float(round_tf32(np.float32(1.0 + 2 ** -11))) == 1.0               # tie to even
    assert float(round_tf32(np.float32(1.0 + 3 * 2 ** -11))) == 1.0 + 2 ** -9


def test_reduced_precision_modes_stay_close_to_fp32_mode():
    ref = make([32, 24, 16], False, precision="fp32", n_classes=5)
    x, cls = data(ref, 12)
    x = round_bf16(x.astype(np.float32))
    ref.loss_and_grads(x, cls)
    for prec, tol in (("tf32", 2e-3), ("bf16", 2e-2)):
        seg = make([32, 24, 16], False, precision=prec, n_classes=5)
        seg.loss_and_grads(x, cls)
        for a, b in zip(ref.dW + ref.db + ref.acts[1:], seg.dW + seg.db + seg.acts[1:]):
            assert np.max(np.abs(a.astype(np.float64) - b)) <= tol * np.max(np.abs(a))


def test_tie_break_only_acts_where_the_caller_flips_and_matches_a_perturbed_network():
    """Choosing relu' = 0 on one barely-positive unit equals the gradient of the same network with that
    unit's bias lowered by more than its pre-activation (the unit is then off, the forward output of
    everything else unchanged up to that tiny amount)."""
    seg = make([6, 5, 4], False, n_classes=3)
    x, cls = data(seg, 4, seed=11)
    seg.forward(x)
    z = seg.preact[0]
    b_idx, j = np.unravel_index(np.argmin(np.where(z > 0, z, np.inf)), z.shape)   # smallest positive unit
    eps = float(z[b_idx, j])
    base = seg.loss_and_grads(x, cls)
    g_plain = [g.copy() for g in seg.dW + seg.db]
    same = seg.loss_and_grads(x, cls, tie_break=lambda l, zz, m: m)
    assert same == base and all(np.array_equal(a, b) for a, b in zip(g_plain, seg.dW + seg.db))

    def flip(l, zz, m):
        m = m.copy()
        if l == 1:
            m[b_idx, j] = False
        return m
    seg.loss_and_grads(x, cls, tie_break=flip)
    g_flip = [g.copy() for g in seg.dW + seg.db]
    other = make([6, 5, 4], False, n_classes=3)
    xs = x.copy()
    # switch the unit off for that sample only: subtract from the sample's input what lowers z by 2*eps
    w = other.W[0][j]
    xs[b_idx] = xs[b_idx] - 2 * eps * w / float(w @ w)
    other.loss_and_grads(xs, cls)
    assert (other.preact[0][b_idx, j] < 0) and np.sum((other.preact[0] > 0) != (z > 0)) == 1
    for a, b in zip(g_flip, other.dW + other.db):
        assert np.allclose(a, b, atol=20 * eps * (1 + np.abs(b).max()) + 1e-12)
    assert any(not np.array_equal(a, b) for a, b in zip(g_flip, g_plain))
