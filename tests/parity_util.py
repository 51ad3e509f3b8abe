"""Helpers shared by the GPU parity tests: build the CUDA segment and the oracle segment from
one description, feed both the same seeded arrays, and compare tensor by tensor."""
import numpy as np

from oracle import rng as orng
from oracle.segment import OracleSegment
from paper_2403_11204_b200 import workloads as wl


def rel_err(got, ref):
    """max |got - ref| / max |ref|  (element-wise ratios are meaningless next to ReLU zeros)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(got - ref)) / max(float(np.max(np.abs(ref))), 1e-30))


DIST_CODE = {"uniform_kappa": orng.DIST_UNIFORM_KAPPA, "normal": orng.DIST_NORMAL}


def make_pair(widths, n_classes, is_final, precision, optimizer, lr, max_batch, segment_id=0,
              oracle_precision=None, gemm_backend="auto", label_dist="normal", kappa=10.0,
              label_seed=wl.LABEL_SEED, init_seed=wl.INIT_SEED, momentum=0.9, last_relu=None):
    from paper_2403_11204_b200.binding import Segment
    gpu = Segment(widths, n_classes, is_final, precision=precision, optimizer=optimizer, lr=lr,
                  momentum=momentum, max_batch=max_batch, segment_id=segment_id, init_seed=init_seed,
                  gemm_backend=gemm_backend, last_relu=last_relu)
    ora = OracleSegment(widths, n_classes, is_final, precision=oracle_precision or precision,
                        optimizer=optimizer, lr=lr, momentum=momentum, segment_id=segment_id,
                        init_seed=init_seed, last_relu=last_relu)
    if not is_final:
        gpu.gen_labels(label_seed, label_dist, kappa)
        ora.gen_labels(label_seed, DIST_CODE[label_dist], kappa)
    return gpu, ora


def batch_arrays(workload, n, width, seed=wl.DATA_SEED, precision="fp32"):
    x = wl.features(workload, n, width, seed)
    cls = wl.class_indices(workload, n, seed)
    if precision == "bf16":
        x = wl.from_bf16_bits(wl.to_bf16_bits(x))      # both sides see bf16-representable inputs
    return x, cls


def to_device(x, cls, precision):
    import torch
    xt = torch.from_numpy(x).cuda()
    if precision == "bf16":
        xt = xt.to(torch.bfloat16)                       # exact: values are bf16-representable
    return xt.contiguous(), torch.from_numpy(cls.astype(np.int32)).cuda()


def sync_from_oracle(gpu, ora):
    """Copies the oracle's parameters, optimizer state and step counter into the CUDA segment, so
    that a following step is compared from identical state (used between Adam steps, whose
    trajectories otherwise separate at the ill-conditioned elements described in compare_step)."""
    import torch
    n = ora.n_layers
    for l in range(n):
        gpu.set_params(l, torch.from_numpy(ora.W[l]).cuda(), torch.from_numpy(ora.b[l]).cuda())
        if ora.optimizer != "sgd":
            gpu.set_opt_state(l, 0, torch.from_numpy(ora.state1[l]).cuda(), torch.from_numpy(ora.state1[n + l]).cuda())
        if ora.optimizer == "adam":
            gpu.set_opt_state(l, 1, torch.from_numpy(ora.state2[l]).cuda(), torch.from_numpy(ora.state2[n + l]).cuda())
    gpu.set_step(ora.t)


def bits_equal(a, b):
    a = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    b = np.ascontiguousarray(b, dtype=np.float32).view(np.uint32)
    return bool(np.array_equal(a, b))


def compare_step(gpu, ora, x, cls, precision, tol, check_state=True):
    """Runs one training step on both sides and returns {tensor name: relative error};
    asserts every entry is within tol.

    Updated parameters under Adam: the update  -lr * m_hat / (sqrt(v_hat) + eps)  is a normalised
    (sign-like) function of the gradient, so wherever |g| is not larger than the gradient's own
    error the updated weight is ill-conditioned: two correct gradients within tolerance of each
    other give updates that differ by up to 2 lr.  There the comparison is made on the elements
    whose reference gradient is at least ten times the measured gradient error (same tolerance),
    and every other element is held to the absolute bound 3 lr that Adam's step size implies.

    ReLU ties: relu' is a decision taken from a floating-point value.  Where the oracle's own
    pre-activation is within 5 % of the activation tolerance of zero, both derivatives are correct
    answers (an output within tolerance may sit on either side of zero), so there the oracle's
    backward pass follows the sign the CUDA path stored (which must itself be that small); everywhere
    else the oracle decides alone and the stored signs must agree with it."""
    import torch
    xt, ct = to_device(x, cls, precision)
    loss_t = torch.zeros(1, device="cuda")
    gpu.train_step(xt, ct, loss_t)
    gpu.poll()
    acts_gpu = {l: gpu.activation(l).cpu().numpy() for l in range(1, ora.n_layers + 1)}
    ties = {}

    def tie_break(l, z, m):
        thr = 0.05 * tol * max(float(np.max(z)), 1e-30)
        amb = np.abs(z) <= thr
        g_on = acts_gpu[l] > 0
        assert float(np.max(np.abs(acts_gpu[l][amb]), initial=0.0)) <= 2.0 * thr, f"A{l}: large value at a tie"
        assert np.array_equal(g_on[~amb], m[~amb]), f"A{l}: ReLU sign differs away from zero"
        ties[l] = float(np.mean(amb & (g_on != m)))
        return np.where(amb, g_on, m)

    loss_o = ora.train_step(x, cls, tie_break)
    errs = {"loss": abs(float(loss_t.item()) - loss_o) / max(abs(loss_o), 1e-30)}
    for l in range(1, ora.n_layers + 1):
        errs[f"A{l}"] = rel_err(acts_gpu[l], ora.acts[l])
    for l in range(ora.n_layers):
        dW, db = (t.cpu().numpy() for t in gpu.grads(l))
        errs[f"dW{l}"] = rel_err(dW, ora.dW[l])
        errs[f"db{l}"] = rel_err(db, ora.db[l])
        if not check_state:
            continue
        W, b = (t.cpu().numpy() for t in gpu.params(l))
        for name, got, ref, g_got, g_ref in ((f"W{l}", W, ora.W[l], dW, ora.dW[l]),
                                             (f"b{l}", b, ora.b[l], db, ora.db[l])):
            if ora.optimizer != "adam":
                errs[name] = rel_err(got, ref)
                continue
            g_err = float(np.max(np.abs(g_got.astype(np.float64) - g_ref)))
            well = (np.abs(g_ref) >= 10.0 * g_err + 10.0 * ora.eps) | ((g_ref == 0) & (g_got == 0))
            diff = np.abs(got.astype(np.float64) - ref)
            scale = max(float(np.max(np.abs(ref))), 1e-30)
            errs[name] = float(diff[well].max() / scale) if well.any() else 0.0
            assert float(diff.max()) <= 3.0 * ora.lr + tol * scale, (name, float(diff.max()))
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, f"beyond tolerance {tol}: {bad}  (all: {errs})"
    return errs
