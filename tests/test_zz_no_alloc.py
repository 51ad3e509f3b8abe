"""The allocation-free loss entry point against the ordinary training step.

seg_label_loss_noalloc serves callers that cannot allocate device memory (fixed memory budgets,
latency-bound loops that must not hit the device synchronisation cudaMalloc implies, code that
owns a stream but no allocator): its reduction scratch is a static array inside the library.
Here it is fed the stored output, class indices and labels of a real training step and must
reproduce that step's loss and, through the column sums of its dZ, that step's last-layer bias
gradient - twice in a row, because the second call meets whatever the first one left in the
shared scratch.  A second test checks the loss and every element of dZ against the three-line
formula of the header, written out in NumPy float64, with and without the ReLU mask and for a
width that the wide (16-byte) code path cannot take.  This file sorts last on purpose: a run that
stops at the first failure has already run everything else.
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


@pytest.mark.parametrize("n_p,batch", [(72, 200), (61, 77), (8, 1)])
@pytest.mark.parametrize("relu_mask", [1, 0])
def test_noalloc_loss_matches_its_definition_element_by_element(n_p, batch, relu_mask):
    """loss = mean (out - sil[cls])^2 and dz = 2 (out - sil[cls]) / (batch n_p) [out > 0 if masked], every
    element, on two calls in a row; class indices outside [0, n_classes) are clamped, not read out of bounds."""
    import torch
    from paper_2403_11204_b200 import build
    build.build()
    from paper_2403_11204_b200.binding import label_loss_noalloc
    g = np.random.default_rng(n_p * 1000 + batch)
    n_classes = 47
    sil = g.standard_normal((n_classes, n_p)).astype(np.float32)
    for call in range(2):
        out = g.standard_normal((batch, n_p)).astype(np.float32)
        cls = g.integers(0, n_classes, batch).astype(np.int32)
        if batch > 2 and call == 1:
            cls[0], cls[1] = n_classes + 3, -1                       # clamped to the last / first class
        t = sil[np.clip(cls, 0, n_classes - 1)].astype(np.float64)
        d = out.astype(np.float64) - t
        loss_ref = float(np.mean(d * d))
        dz_ref = 2.0 * d / (batch * n_p) * ((out > 0) if relu_mask else 1.0)
        out_t, cls_t, sil_t = (torch.from_numpy(a).cuda() for a in (out, cls, sil))
        dz_t, loss_t = torch.full_like(out_t, 7.0), torch.zeros(1, device="cuda")
        label_loss_noalloc(out_t, cls_t, sil_t, relu_mask, dz_t, loss_t)
        torch.cuda.synchronize()
        assert abs(float(loss_t.item()) - loss_ref) <= TOL * abs(loss_ref)
        err = np.max(np.abs(dz_t.cpu().numpy().astype(np.float64) - dz_ref))
        assert err <= TOL * np.max(np.abs(dz_ref)), (call, err)


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
