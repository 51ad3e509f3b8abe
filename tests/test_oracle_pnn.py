"""Pins for oracle/pnn.py, the paper's training procedure (Section 2)."""
import numpy as np

from oracle import pnn, rng
from oracle.segment import OracleSegment


def make_net(seed=2):
    left = OracleSegment([12, 10, 8], 4, False, precision="fp64", optimizer="momentum", lr=0.05, segment_id=0, init_seed=seed)
    right = OracleSegment([8, 9, 4], 4, True, precision="fp64", optimizer="momentum", lr=0.05, segment_id=1, init_seed=seed)
    left.gen_labels(1, rng.DIST_UNIFORM_KAPPA, 2.0)
    return left, right


def data(n=50):
    g = np.random.default_rng(0)
    return g.random((n, 12)), g.integers(0, 4, n)


def test_step_count_and_no_shuffle_order():
    # Section 3: 112,800 images at batch 1410 = 80 steps per epoch; here 50 samples at batch 16 = 4 steps
    left, _ = make_net()
    x, cls = data()
    losses = pnn.train_epochs(left, x, cls, 16, 3)
    assert len(losses) == 3 * 4
    # same thing by hand, batch by batch in stored order, last batch of 2 samples
    ref, _ = make_net()
    by_hand = []
    for _ in range(3):
        for lo, hi in ((0, 16), (16, 32), (32, 48), (48, 50)):
            by_hand.append(ref.train_step(x[lo:hi], cls[lo:hi]))
    assert np.array_equal(losses, np.array(by_hand))
    assert all(np.array_equal(a, b) for a, b in zip(left.W + left.b, ref.W + ref.b))


def test_phases_are_separate_and_right_input_is_the_final_left_response():
    left, right = make_net()
    x, cls = data()
    right_before = [p.copy() for p in right.W + right.b]
    # phase 1 only: the right partition is not used at all (Section 2)
    pnn.train_epochs(left, x, cls, 16, 2)
    assert all(np.array_equal(a, b) for a, b in zip(right_before, right.W + right.b))
    left_after = [p.copy() for p in left.W + left.b]
    stored = pnn.forward_dataset(left, x, 16)
    assert np.array_equal(stored, left.forward(x)[-1])            # chunking does not change the response
    # the whole procedure from scratch gives the same stored response and leaves the left part alone in phase 2
    l2, r2 = make_net()
    losses, right_in = pnn.train_partitioned([l2, r2], x, cls, 16, [2, 3])
    assert np.array_equal(right_in, stored)
    assert all(np.array_equal(a, b) for a, b in zip(left_after, l2.W + l2.b))
    assert len(losses[0]) == 8 and len(losses[1]) == 12
    assert losses[1][-1] < losses[1][0]                            # the right partition learns the labels
    pred = pnn.predict([l2, r2], x, 16)
    whole = OracleSegment([12, 10, 8, 9, 4], 4, True, precision="fp64")
    whole.W, whole.b = [w.copy() for w in l2.W + r2.W], [b.copy() for b in l2.b + r2.b]
    assert np.array_equal(pred, np.argmax(whole.forward(x)[-1], axis=1))   # joined network = one network


def test_three_partitions_use_one_label_set_per_cut():
    segs = [OracleSegment([12, 9, 7], 4, False, precision="fp64", segment_id=0),
            OracleSegment([7, 7, 6], 4, False, precision="fp64", segment_id=1),
            OracleSegment([6, 5, 4], 4, True, precision="fp64", segment_id=2)]
    segs[0].gen_labels(1, rng.DIST_UNIFORM_KAPPA, 10.0)
    segs[1].gen_labels(1, rng.DIST_UNIFORM_KAPPA, 10.0)
    assert segs[0].sil.shape == (4, 7) and segs[1].sil.shape == (4, 6)
    assert not np.array_equal(segs[0].sil[:, :6], segs[1].sil)     # distinct streams per cut
    x, cls = data(40)
    losses, _ = pnn.train_partitioned(segs, x, cls, 8, [1, 1, 2])
    assert [len(l) for l in losses] == [5, 5, 10]


def test_recovery_step_equals_end_to_end_gradients_of_the_joined_network():
    """Section 5: the left part is trained through the frozen right part.  Its gradients must be the
    joined network's own (already pinned by finite differences), the right part must not move, and
    the update must be the left optimizer's."""
    left, right = make_net()
    x, cls = data(20)
    whole = OracleSegment([12, 10, 8, 9, 4], 4, True, precision="fp64", optimizer="momentum", lr=0.05)
    whole.W, whole.b = [w.copy() for w in left.W + right.W], [b.copy() for b in left.b + right.b]
    loss_whole = whole.loss_and_grads(x, cls)
    right_before = [p.copy() for p in right.W + right.b]
    left_before = [p.copy() for p in left.W + left.b]
    loss = pnn.recovery_step(left, right, x, cls)
    assert abs(loss - loss_whole) < 1e-14
    for l in range(2):
        assert np.allclose(left.dW[l], whole.dW[l], rtol=1e-12, atol=1e-16)
        assert np.allclose(left.db[l], whole.db[l], rtol=1e-12, atol=1e-16)
    assert all(np.array_equal(a, b) for a, b in zip(right_before, right.W + right.b))
    for p0, p1, g in zip(left_before, left.W + left.b, left.dW + left.db):
        assert np.allclose(p1, p0 - 0.05 * g, rtol=1e-13, atol=1e-18)     # first momentum step = SGD step
    losses = [pnn.recovery_step(left, right, x, cls) for _ in range(5)]
    assert losses[-1] < loss                                               # recovery lowers the joined loss
