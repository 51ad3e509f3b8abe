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


@pytest.mark.parametrize("precision,backend,tol", [("fp32", "auto", 1e-4), ("bf16", "tcgen05", 2e-2), ("tf32", "tcgen05", 2e-3)])
def test_recovery_step_matches_the_oracle(precision, backend, tol):
    """Section 5 (recovery epochs): the left segment trained through the frozen right segment."""
    import torch
    from paper_2403_11204_b200 import binding
    from parity_util import batch_arrays, bits_equal
    w = wl.WORKLOADS["tiny"]
    batch = 200
    gl, ol = make_pair([784, 256, 136], 47, False, precision, "momentum", 0.01, batch, segment_id=0, gemm_backend=backend)
    gr, orr = make_pair([136, 72, 47], 47, True, precision, "momentum", 0.01, batch, segment_id=1, gemm_backend=backend)
    x, cls = batch_arrays(w, batch, 784, precision=precision)
    xt, ct = to_device(x, cls, precision)
    right_before = [t.clone() for l in range(2) for t in gr.params(l)]
    for step in range(4):                                   # eager, captured, replayed twice
        loss_t = torch.zeros(1, device="cuda")
        binding.recovery_step(gl, gr, xt, ct, loss_t)
        gl.poll()
        loss_o = pnn.recovery_step(ol, orr, x, cls.astype(np.int64))
        assert abs(float(loss_t.item()) - loss_o) <= tol * abs(loss_o)
        if step >= 2:
            continue          # two trajectories in reduced precision drift apart: later steps are held to the loss only
        for l in range(2):
            dW, db = gl.grads(l)
            assert rel_err(dW.cpu().numpy(), ol.dW[l]) <= tol and rel_err(db.cpu().numpy(), ol.db[l]) <= tol
            W, b = gl.params(l)
            assert rel_err(W.cpu().numpy(), ol.W[l]) <= tol and rel_err(b.cpu().numpy(), ol.b[l]) <= tol
    right_after = [t for l in range(2) for t in gr.params(l)]
    assert all(torch.equal(a, b) for a, b in zip(right_before, right_after))       # frozen: bit-identical
    gl.close(); gr.close()


@pytest.mark.parametrize("precision,backend,tol,hidden", [("fp32", "auto", 1e-4, 200), ("fp32", "auto", 1e-4, 96),
                                                          ("bf16", "tcgen05", 2e-2, 200)])
def test_fully_separate_variant_label_rows_as_input(precision, backend, tol, hidden):
    """Section 2, last flowchart: a middle partition trained with the previous cut's labels as input and
    its own cut's labels as target; the input rows are gathered by class on the device (by the staging
    kernel, or, hidden = 96, inside the first launch of a small fp32 segment's two-launch step)."""
    import torch
    from oracle import rng as orng
    from parity_util import compare_step, bits_equal
    w = wl.WORKLOADS["tiny"]
    m, batch = 47, 150
    prev_labels = orng.gen_labels(wl.LABEL_SEED, 0, m, 136, orng.DIST_UNIFORM_KAPPA, 10.0)     # cut 0: 47 x 136
    gpu, ora = make_pair([136, hidden, 72], m, False, precision, "momentum", 0.01, batch, segment_id=1,
                         gemm_backend=backend, label_dist="uniform_kappa")
    cls = wl.class_indices(w, batch)
    sil_t = torch.from_numpy(prev_labels).cuda()
    ct = torch.from_numpy(cls).cuda()
    for step in range(3):                                   # eager, captured, replayed
        loss_t = torch.zeros(1, device="cuda")
        gpu.train_step_label_input(sil_t, ct, loss_t)
        gpu.poll()
        loss_o = ora.train_step(prev_labels[cls], cls.astype(np.int64))
        assert abs(float(loss_t.item()) - loss_o) <= tol * abs(loss_o)
        for l in range(2):
            dW, db = gpu.grads(l)
            assert rel_err(dW.cpu().numpy(), ora.dW[l]) <= tol and rel_err(db.cpu().numpy(), ora.db[l]) <= tol
            W, b = gpu.params(l)
            assert rel_err(W.cpu().numpy(), ora.W[l]) <= tol
    # an ordinary step on the same handle afterwards still reads the caller's x
    x = prev_labels[cls]
    if precision == "bf16":
        x = wl.from_bf16_bits(wl.to_bf16_bits(x))
    compare_step(gpu, ora, x, cls, precision, tol)
    gpu.close()
