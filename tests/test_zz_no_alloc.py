"""The allocation-free loss entry point against the ordinary training step.

seg_label_loss_noalloc serves callers that cannot allocate device memory (fixed memory budgets,
latency-bound loops that must not hit the device synchronisation cudaMalloc implies, code that
owns a stream but no allocator): its reduction scratch is a static array inside the library.
Here it is fed the stored output, class indices and labels of a real training step and must
reproduce that step's loss and, through the column sums of its dZ, that step's last-layer bias
gradient - twice in a row, because the second call meets whatever the first one left in the
shared scratch.  This file sorts last on purpose: a run that stops at the first failure has
already run everything else.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-4          # the fp32 tolerance of the parity tests


def _step(seg, x, cls):
    import torch
    loss = torch.zeros(1, device="cuda")
    seg.train_step(x, cls, loss)
    seg.poll()
    n = seg.n_layers
    return float(loss.item()), seg.activation(n).clone(), seg.grads(n - 1)[1].clone()


def test_noalloc_loss_matches_training_step_twice_in_a_row():
    import torch
    from paper_2403_11204_b200 import build, workloads as wl
    build.build()
    from paper_2403_11204_b200.binding import Segment, label_loss_noalloc
    w = wl.WORKLOADS["tiny"]
    widths = [784, 128, 72]
    seg = Segment(widths, w.n_classes, False, precision="fp32", optimizer="sgd", lr=0.01, max_batch=200)
    seg.gen_labels(wl.LABEL_SEED, "normal")
    sil = seg.labels()
    cases = []
    for batch, seed in ((200, 0), (77, 3)):
        x = torch.from_numpy(wl.features(w, batch, widths[0], seed)).cuda()
        cls = torch.from_numpy(wl.class_indices(w, batch, seed)).cuda()
        loss, out, db = _step(seg, x, cls)
        cases.append((out.contiguous(), cls, loss, db))
    outputs = [(torch.empty_like(out), torch.zeros(1, device="cuda")) for out, _, _, _ in cases]
    torch.cuda.synchronize()
    for (out, cls, _, _), (dz, loss_t) in zip(cases, outputs):       # two calls in a row on one stream
        label_loss_noalloc(out, cls, sil, True, dz, loss_t)
    torch.cuda.synchronize()
    for (out, cls, loss_ref, db_ref), (dz, loss_t) in zip(cases, outputs):
        assert abs(float(loss_t.item()) - loss_ref) <= TOL * abs(loss_ref)
        db = dz.sum(dim=0, dtype=torch.float64).cpu().numpy()
        ref = db_ref.double().cpu().numpy()
        assert np.max(np.abs(db - ref)) <= TOL * np.max(np.abs(ref))
        assert bool(((dz != 0) <= (out > 0)).all())                  # the ReLU mask of the cut layer
    seg.close()


def test_noalloc_rejects_sizes_beyond_its_maximum():
    import torch
    from paper_2403_11204_b200 import binding
    lib = binding.load()
    t = torch.zeros(4, device="cuda")
    c = torch.zeros(4, dtype=torch.int32, device="cuda")
    p = lambda x: binding.c_void_p(x.data_ptr())
    assert lib.seg_label_loss_noalloc(p(t), p(c), p(t), 1, 65537, 1, 1, p(t), None, None) == 2
    assert lib.seg_label_loss_noalloc(p(t), p(c), p(t), 1, 1, 65537, 1, p(t), None, None) == 2
    assert lib.seg_label_loss_noalloc(None, p(c), p(t), 1, 1, 1, 1, p(t), None, None) == 1
