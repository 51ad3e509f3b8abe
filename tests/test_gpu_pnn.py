"""The paper's training procedure end to end (Section 2): train the left partition on the
intermediate labels, store its response, train the right partition on it, join - through
seg_train_epochs / seg_forward_dataset, against oracle/pnn.py, loss by loss."""
import numpy as np
import pytest

from oracle import pnn
from paper_2403_11204_b200 import workloads as wl
from parity_util import make_pair, rel_err, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,epochs,label_dist", [("tiny", [1, 1], "normal"), ("tiny", [2, 1], "uniform_kappa")])
def test_two_partition_training_matches_the_oracle(name, epochs, label_dist):
    import torch
    from paper_2403_11204_b200 import binding
    w = wl.WORKLOADS[name]
    n = 1000                                             # 15 full batches of 64 and one of 40
    pairs = [make_pair(s.widths, w.n_classes, s.is_final, w.precision, w.optimizer, w.lr, w.batch,
                       segment_id=s.segment_id, label_dist=label_dist, kappa=10.0) for s in w.segments]
    gpu = [p[0] for p in pairs]
    ora = [p[1] for p in pairs]
    x = wl.features(w, n)
    cls = wl.class_indices(w, n)
    xt, ct = to_device(x, cls, w.precision)
    losses_g, right_in_g = binding.train_partitioned(gpu, xt, ct, w.batch, epochs)
    for seg in gpu:
        seg.poll()
    losses_o, right_in_o = pnn.train_partitioned(ora, x, cls.astype(np.int64), w.batch, epochs)
    for lg, lo in zip(losses_g, losses_o):
        got = lg.cpu().numpy().astype(np.float64)
        assert got.shape == lo.shape
        assert np.max(np.abs(got - lo) / np.abs(lo)) < 1e-3
    assert rel_err(right_in_g.cpu().numpy(), right_in_o) < 1e-3
    for g, o in zip(gpu, ora):
        for l in range(o.n_layers):
            W, b = g.params(l)
            assert rel_err(W.cpu().numpy(), o.W[l]) < 1e-3 and rel_err(b.cpu().numpy(), o.b[l]) < 1e-3
    pred_g = binding.predict(gpu, xt, w.batch).cpu().numpy()
    pred_o = pnn.predict(ora, x, w.batch)
    assert np.mean(pred_g == pred_o) > 0.99              # argmax may differ only on near-ties
    for seg in gpu:
        seg.close()
