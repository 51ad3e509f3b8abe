"""Pins for WHERE the oracle's reduced-precision modes round (bf16 and TF32).

The reading being pinned: master weights are fp32 and enter every product through a rounded copy;
the segment input is rounded once; hidden activations and every dZ are rounded when they are stored
(fp32 first, then to the operand grid); the loss and dZ of the last layer are taken from the STORED
output; the bias gradient is the sum of the STORED dZ; the final segment's logits stay fp32.

The reference here is a scalar re-derivation that shares nothing with the oracle: nested Python loops
over lists, and "round to s significant bits, ties to even" done arithmetically (frexp, a power-of-two
quantum and Python's round-half-even), not by bit tricks.  All inputs are small dyadic rationals, so
every fp64 sum on either side is exact and the comparison can be equality, bit for bit.  For each
rounding point the same scalar network is also evaluated with that one rounding left out; the result
must differ in a named tensor, which shows that an oracle that dropped or moved that rounding would
fail the equality above.
"""
import math

import numpy as np
import pytest

from oracle import pnn
from oracle.segment import OracleSegment

SIG = {"bf16": 8, "tf32": 11}          # significant bits of the operand grids


def rnd(x, bits):
    """Nearest value with `bits` significant bits, ties to even (x a Python float)."""
    if x == 0.0:
        return 0.0
    _, e = math.frexp(x)                # |x| = m 2^e, 0.5 <= m < 1
    q = math.ldexp(1.0, e - bits)
    return round(x / q) * q             # x / q is exact; round() is half-to-even


def f32(x):
    return rnd(x, 24)                   # fp32 storage (no subnormals or overflow in these examples)


class Scalar:
    """The segment step written out with loops.  `drop` names one rounding to leave out."""

    def __init__(self, W, b, prec, is_final, last_relu, drop=None):
        self.W = [[list(map(float, r)) for r in w] for w in W]
        self.b = [list(map(float, v)) for v in b]
        self.s, self.is_final, self.last_relu, self.drop = SIG[prec], is_final, last_relu, drop

    def op(self, v, what):              # operand rounding of weights / the segment input
        return v if self.drop == what else rnd(v, self.s)

    def store(self, v, what):           # fp32 store, then the operand grid
        v = f32(v)
        return v if self.drop == what else rnd(v, self.s)

    def forward(self, x):
        n = len(self.W)
        acts = [[[self.op(float(v), "x") for v in row] for row in x]]
        for l in range(n):
            last = l == n - 1
            out = []
            for row in acts[-1]:
                zrow = []
                for j, wj in enumerate(self.W[l]):
                    z = sum(a * self.op(w, "w") for a, w in zip(row, wj)) + self.b[l][j]
                    if (not last) or self.last_relu:
                        z = max(z, 0.0)
                    zrow.append(f32(z) if (last and self.is_final) else self.store(z, "act"))
                out.append(zrow)
            acts.append(out)
        return acts

    def backward(self, acts, dz_last):
        n, B = len(self.W), len(dz_last)
        dz = [[self.store(v, "dz") for v in row] for row in dz_last]
        dW, db, dZ = [None] * n, [None] * n, [None] * n
        for l in reversed(range(n)):
            dZ[l] = dz
            n_out, n_in = len(self.W[l]), len(self.W[l][0])
            dW[l] = [[f32(sum(dz[b][j] * acts[l][b][i] for b in range(B))) for i in range(n_in)] for j in range(n_out)]
            if self.drop == "db":       # the mutation: bias gradient from the unrounded dZ of the last layer
                src = dz_last if l == n - 1 else dz
                db[l] = [f32(sum(f32(src[b][j]) for b in range(B))) for j in range(n_out)]
            else:
                db[l] = [f32(sum(dz[b][j] for b in range(B))) for j in range(n_out)]
            if l > 0:
                nxt = []
                for b in range(B):
                    row = []
                    for i in range(n_in):
                        v = sum(dz[b][j] * self.op(self.W[l][j][i], "w") for j in range(n_out))
                        row.append(self.store(v if acts[l][b][i] > 0 else 0.0, "dz"))
                    nxt.append(row)
                dz = nxt
        return dW, db, dZ

    def mse_step(self, x, target):
        acts = self.forward(x)
        out = acts[-1]
        n = len(out) * len(out[0])
        loss = sum((a - t) ** 2 for ro, rt in zip(out, target) for a, t in zip(ro, rt)) / n
        dz = [[(2.0 * (a - t) / n) * (1.0 if (a > 0 or not self.last_relu) else 0.0) for a, t in zip(ro, rt)]
              for ro, rt in zip(out, target)]
        return (loss, acts) + self.backward(acts, dz)


def dyadic(g, shape, bits, lo, hi):
    """Random multiples of 2^-bits in [lo, hi)."""
    q = 2.0 ** -bits
    return g.integers(int(lo / q), int(hi / q), size=shape).astype(np.float64) * q


def example(prec, seed=0):
    g = np.random.default_rng(seed)
    widths = [3, 4, 2]
    W = [dyadic(g, (widths[l + 1], widths[l]), 12, -1.0, 1.0) for l in range(2)]     # fp32 masters off the operand grid
    b = [dyadic(g, (widths[l + 1],), 12, -0.25, 0.5) for l in range(2)]
    x = dyadic(g, (4, 3), 7 if prec == "bf16" else 15, 0.0, 2.0)   # bf16 inputs arrive in bf16; TF32 inputs are fp32
    sil = dyadic(g, (3, 2), 12, -1.0, 2.0)        # targets finer than the operand grid, so that dZ needs rounding
    cls = np.array([2, 0, 1, 0])
    return widths, W, b, x, sil, cls


def oracle_for(prec, widths, W, b, sil, is_final=False, n_classes=3):
    o = OracleSegment(widths, n_classes, is_final, precision=prec, optimizer="sgd", lr=0.125)
    o.W = [w.astype(np.float32) for w in W]
    o.b = [v.astype(np.float32) for v in b]
    o.sil = None if sil is None else sil.astype(np.float32)
    return o


@pytest.mark.parametrize("prec", ["bf16", "tf32"])
def test_mse_step_rounds_exactly_where_the_reading_says(prec):
    widths, W, b, x, sil, cls = example(prec)
    o = oracle_for(prec, widths, W, b, sil)
    loss_o = o.loss_and_grads(x.astype(np.float32), cls)
    ref = Scalar(W, b, prec, False, True)
    loss, acts, dW, db, dZ = ref.mse_step(x.tolist(), sil[cls].tolist())
    assert loss_o == loss
    for l in range(1, 3):
        assert np.array_equal(o.acts[l].astype(np.float64), np.array(acts[l])), f"A{l}"
    for l in range(2):
        assert np.array_equal(o.dZ[l].astype(np.float64), np.array(dZ[l])), f"dZ{l}"
        assert np.array_equal(o.dW[l].astype(np.float64), np.array(dW[l])), f"dW{l}"
        assert np.array_equal(o.db[l].astype(np.float64), np.array(db[l])), f"db{l}"
    # the update acts on the fp32 master, not on the rounded copy
    o.apply_update()
    for l in range(2):
        want = [[f32(w - 0.125 * g) for w, g in zip(rw, rg)] for rw, rg in zip(W[l].tolist(), dW[l])]
        assert np.array_equal(o.W[l].astype(np.float64), np.array(want)), f"W{l}"

    # every rounding point matters on this input: leaving one out changes a named tensor
    def variant(drop):
        return Scalar(W, b, prec, False, True, drop=drop).mse_step(x.tolist(), sil[cls].tolist())
    changed = {"w": ("acts", 1), "act": ("acts", 1), "dz": ("dZ", 1), "db": ("db", 1)}
    if prec == "tf32":
        changed["x"] = ("acts", 1)
    for drop, (name, l) in changed.items():
        v_loss, v_acts, v_dW, v_db, v_dZ = variant(drop)
        got = {"acts": v_acts, "dZ": v_dZ, "db": v_db}[name][l]
        full = {"acts": acts, "dZ": dZ, "db": db}[name][l]
        assert got != full, f"dropping the '{drop}' rounding does not change {name}[{l}]: the example is too weak"
    # stored-output reading of the loss: with unrounded activations the loss itself moves
    assert variant("act")[0] != loss


@pytest.mark.parametrize("prec", ["bf16", "tf32"])
def test_final_segment_keeps_fp32_logits_and_rounds_dz(prec):
    g = np.random.default_rng(3)
    widths = [3, 4, 3]
    W = [dyadic(g, (widths[l + 1], widths[l]), 12, -1.0, 1.0) for l in range(2)]
    b = [dyadic(g, (widths[l + 1],), 12, -0.25, 0.5) for l in range(2)]
    x = dyadic(g, (4, 3), 7, 0.0, 2.0)
    cls = np.array([2, 0, 1, 0])
    o = oracle_for(prec, widths, W, b, None, is_final=True)
    loss_o = o.loss_and_grads(x.astype(np.float32), cls)
    ref = Scalar(W, b, prec, True, False)
    acts = ref.forward(x.tolist())
    logits = acts[-1]
    assert np.array_equal(o.acts[2].astype(np.float64), np.array(logits))          # fp32, not on the operand grid
    assert any(rnd(v, SIG[prec]) != v for row in logits for v in row)
    # softmax cross-entropy by hand on those logits (exp is not exact arithmetic: compare to 1e-12, far below
    # the 2^-9 / 2^-12 a misplaced rounding moves things by)
    B = len(logits)
    dz, loss = [], 0.0
    for row, c in zip(logits, cls):
        m = max(row)
        e = [math.exp(v - m) for v in row]
        s = sum(e)
        loss += -(row[c] - m - math.log(s)) / B
        dz.append([(ei / s - (1.0 if j == c else 0.0)) / B for j, ei in enumerate(e)])
    dW, db, dZ = ref.backward(acts, dz)
    assert abs(loss_o - loss) < 1e-12
    for l in range(2):
        assert np.allclose(o.dZ[l], np.array(dZ[l]), rtol=1e-9, atol=0)
        assert np.allclose(o.dW[l], np.array(dW[l]), rtol=1e-6, atol=1e-12)
        assert np.allclose(o.db[l], np.array(db[l]), rtol=1e-6, atol=1e-12)
    # the stored dZ of the last layer sits on the operand grid, and an unrounded one would differ
    assert all(rnd(v, SIG[prec]) == v for row in dZ[1] for v in row)
    assert any(rnd(f32(v), SIG[prec]) != f32(v) for row in dz for v in row)


@pytest.mark.parametrize("prec", ["bf16", "tf32"])
def test_recovery_step_rounds_at_the_same_points(prec):
    """Section 5 (recovery): forward through both partitions, cross-entropy, dgrad through the frozen right
    partition, then the left partition's backward pass - every stored dZ on the operand grid, the frozen
    weights through their rounded copy."""
    g = np.random.default_rng(10)
    wl_, wr_, B = [3, 6, 4], [4, 5, 3], 16    # large enough that every rounding point shifts some stored value
    Wl = [dyadic(g, (wl_[l + 1], wl_[l]), 12, -1.0, 1.0) for l in range(2)]
    bl = [dyadic(g, (wl_[l + 1],), 12, 0.0, 0.5) for l in range(2)]
    Wr = [dyadic(g, (wr_[l + 1], wr_[l]), 12, -1.0, 1.0) for l in range(2)]
    br = [dyadic(g, (wr_[l + 1],), 12, 0.0, 0.5) for l in range(2)]
    x = dyadic(g, (B, 3), 7, 0.0, 2.0)
    cls = g.integers(0, 3, B)
    left = oracle_for(prec, wl_, Wl, bl, dyadic(g, (3, 4), 6, 0.0, 1.0))
    right = oracle_for(prec, wr_, Wr, br, None, is_final=True)
    loss_o = pnn.recovery_step(left, right, x.astype(np.float32), cls)

    def scalar(drop=None):
        sl = Scalar(Wl, bl, prec, False, True, drop=drop)
        sr = Scalar(Wr, br, prec, True, False, drop=drop)
        al = sl.forward(x.tolist())
        ar = sr.forward(al[-1])
        logits = ar[-1]
        dz, loss = [], 0.0
        for row, c in zip(logits, cls):
            m = max(row)
            e = [math.exp(v - m) for v in row]
            s = sum(e)
            loss += -(row[c] - m - math.log(s)) / B
            dz.append([(ei / s - (1.0 if j == c else 0.0)) / B for j, ei in enumerate(e)])
        # right partition: activations' gradient only
        dz = [[sr.store(v, "dz") for v in row] for row in dz]
        for l in (1, 0):
            n_out, n_in = len(Wr[l]), len(Wr[l][0])
            da = [[sum(dz[b][j] * sr.op(float(Wr[l][j][i]), "w") for j in range(n_out)) for i in range(n_in)] for b in range(B)]
            if l > 0:
                dz = [[sr.store(da[b][i] if ar[l][b][i] > 0 else 0.0, "dz") for i in range(n_in)] for b in range(B)]
        into_left = [[da[b][i] if al[-1][b][i] > 0 else 0.0 for i in range(len(da[0]))] for b in range(B)]
        return (loss,) + sl.backward(al, into_left)

    loss, dW, db, dZ = scalar()
    assert abs(loss_o - loss) < 1e-12
    for l in range(2):
        assert np.allclose(left.dZ[l], np.array(dZ[l]), rtol=1e-9, atol=0), f"dZ{l}"
        assert np.allclose(left.dW[l], np.array(dW[l]), rtol=1e-6, atol=1e-12), f"dW{l}"
        assert np.allclose(left.db[l], np.array(db[l]), rtol=1e-6, atol=1e-12), f"db{l}"
    flat = lambda r: np.concatenate([[r[0]]] + [np.ravel(t) for part in r[1:] for t in part])
    full = flat((loss, dW, db, dZ))
    for drop in ("w", "act", "dz"):               # each rounding moves the loss or some gradient of this example
        assert not np.allclose(flat(scalar(drop)), full, rtol=1e-6, atol=1e-12), drop
