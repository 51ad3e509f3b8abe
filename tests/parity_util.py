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
    ora = make_oracle(widths, n_classes, is_final, oracle_precision or precision, optimizer, lr, segment_id,
                      label_dist, kappa, label_seed, init_seed, momentum, last_relu)
    if not is_final:
        gpu.gen_labels(label_seed, label_dist, kappa)
    return gpu, ora


def make_oracle(widths, n_classes, is_final, precision, optimizer, lr, segment_id=0, label_dist="normal",
                kappa=10.0, label_seed=wl.LABEL_SEED, init_seed=wl.INIT_SEED, momentum=0.9, last_relu=None):
    """The oracle of a segment alone (e.g. a second one in plain fp32 mode for compare_step's ora_plain)."""
    ora = OracleSegment(widths, n_classes, is_final, precision=precision, optimizer=optimizer, lr=lr,
                        momentum=momentum, segment_id=segment_id, init_seed=init_seed, last_relu=last_relu)
    if not is_final:
        ora.gen_labels(label_seed, DIST_CODE[label_dist], kappa)
    return ora


def batch_arrays(workload, n, width, seed=wl.DATA_SEED, precision="fp32"):
    x = wl.features(workload, n, width, seed)
    cls = wl.class_indices(workload, n, seed)
    if precision == "bf16":
        x = wl.from_bf16_bits(wl.to_bf16_bits(x))      # both sides see bf16-representable inputs
    return x, cls


def segment_input(w, spec, n, seed=wl.DATA_SEED):
    """Features for segment 0; for later segments a stand-in for the previous segment's stored
    output: non-negative (post-ReLU-like) values of the right width, drawn from the same recipe."""
    x, cls = batch_arrays(w, n, spec.widths[0], seed=seed + 17 * spec.segment_id, precision=w.precision)
    if spec.segment_id > 0:
        x = np.abs(x)
    return x, cls


def oracle_loss_curve(args):
    """The oracle's losses over the first `steps` batches of a workload segment, in order.  A plain
    function of its arguments so that it can run in a worker process (threads > 0 limits the worker's
    BLAS threads so that several workers share the host cores)."""
    name, k, batch, steps, threads = args
    w = wl.WORKLOADS[name]
    spec = w.segments[k]

    def run():
        n = min(w.n_samples, steps * batch)
        ora = make_oracle(spec.widths, w.n_classes, spec.is_final, w.precision, w.optimizer, w.lr,
                          segment_id=spec.segment_id, label_dist=w.label_dist, momentum=w.momentum)
        x, cls = segment_input(w, spec, n)
        ref = np.zeros(steps)
        for s in range(steps):
            i = (s * batch) % n
            ref[s] = ora.train_step(x[i:i + batch], cls[i:i + batch])
        return ref
    if threads > 0:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=threads):
            return run()
    return run()


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


# Share of a layer's units whose ReLU derivative the comparison may take from the CUDA path (see compare_step):
# the band is 5 % of the activation tolerance around zero, i.e. 1e-3 (bf16) / 1e-4 (TF32) of the largest
# pre-activation, so for a layer whose pre-activations spread over their range the expected share is of
# that order; ten times that is the ceiling.  fp32 comparisons take nothing from the CUDA path.
TIE_CEILING = {"fp32": 0.0, "tf32": 1e-3, "bf16": 1e-2}      # measured: up to 3.5e-4 / 4.6e-3
# Units per layer whose decision may actually differ from the oracle's own: a share of the layer, at least 2.
TIE_FLIPS = {"tf32": 2e-5, "bf16": 2e-4}
TIE_FLIPS_MIN = 2
# Tolerances of the reduced-precision CUDA paths against the oracle's PLAIN fp32 mode (fp32 storage, fp64
# accumulation, no operand rounding): the figures stated for those paths, 2e-2 (bf16) and 2e-3 (TF32).
PLAIN_TOL = {"tf32": 2e-3, "bf16": 2e-2}
# Share of units within the observed activation deviation of zero in the plain-oracle comparison.
PLAIN_TIE_CEILING = {"tf32": 0.005, "bf16": 0.05}       # measured: up to 2.1e-3 / 2.4e-2
# Adam: smallest share of a tensor's elements that must be in the well-conditioned set (compared at tol).
ADAM_WELL_FLOOR = 0.4        # measured: 0.58 to 1.0 over all Adam cases


def compare_step(gpu, ora, x, cls, precision, tol, check_state=True, ora_plain=None, report=None, tie_scale=1.0):
    """Runs one training step on both sides and returns {tensor name: relative error};
    asserts every entry is within tol.  `report`, a dict, receives the side figures (share of ReLU
    decisions taken from the CUDA path per layer, what those decisions move in the oracle's own
    gradients, Adam's well-conditioned share, errors against the plain fp32 oracle).

    ora_plain: an oracle of the same segment in plain fp32 mode and the same (initial) state.  The CUDA
    path's activations, loss and gradients are then ALSO compared with it, at PLAIN_TOL[precision].  A
    reduced-precision path's pre-activations differ from the plain ones by up to the deviation the
    activation comparison itself measures (dev_l = max |A_l(CUDA) - A_l(plain)|, asserted within
    tolerance); a unit whose plain pre-activation lies within dev_l of zero can therefore be on either
    side of zero in a correct reduced-precision path, and one such unit moves a whole sample's
    contribution in or out of dW and db (at batch 128 that alone is 2-3 % of the largest gradient
    element).  For those units the plain oracle's backward pass follows the sign the CUDA path stored;
    all other signs must agree.  The share of such units is reported and bounded by PLAIN_TIE_CEILING.

    Updated parameters under Adam: the update  -lr * m_hat / (sqrt(v_hat) + eps)  is a normalised
    (sign-like) function of the gradient, so wherever |g| is not larger than the gradient's own
    error the updated weight is ill-conditioned: two correct gradients within tolerance of each
    other give updates that differ by up to 2 lr.  There the comparison is made on the elements
    whose reference gradient is at least ten times the measured gradient error (same tolerance),
    and every other element is held to the absolute bound 3 lr that Adam's step size implies.  The
    share of elements in the first set is reported and must be at least ADAM_WELL_FLOOR.

    ReLU ties (reduced precisions only): relu' is a decision taken from a floating-point value.  Where the
    oracle's own pre-activation is within 5 % of the activation tolerance of zero, both derivatives are
    correct answers (an output within tolerance may sit on either side of zero), so there the oracle's
    backward pass follows the sign the CUDA path stored (which must itself be that small); everywhere
    else the oracle decides alone and the stored signs must agree with it.  The share of units decided
    that way is bounded by TIE_CEILING per layer, the number of units whose decision actually differs
    from the oracle's own by TIE_FLIPS per layer, and what those decisions move in the oracle's own
    gradients is reported (one flipped unit moves one sample's contribution: at batch 300 that alone
    exceeds the TF32 tolerance, which is why the rule exists).  fp32 comparisons install no such rule.
    tie_scale widens the band (a test of the ceiling uses it)."""
    import torch
    xt, ct = to_device(x, cls, precision)
    loss_t = torch.zeros(1, device="cuda")
    gpu.train_step(xt, ct, loss_t)
    gpu.poll()
    acts_gpu = {l: gpu.activation(l).cpu().numpy() for l in range(1, ora.n_layers + 1)}
    grads_gpu = [tuple(t.cpu().numpy() for t in gpu.grads(l)) for l in range(ora.n_layers)]
    report = {} if report is None else report
    ties, flipped = {}, {}

    def tie_break(l, z, m):
        thr = tie_scale * 0.05 * tol * max(float(np.max(z)), 1e-30)
        amb = np.abs(z) <= thr
        g_on = acts_gpu[l] > 0
        assert float(np.max(np.abs(acts_gpu[l][amb]), initial=0.0)) <= 2.0 * thr, f"A{l}: large value at a tie"
        assert np.array_equal(g_on[~amb], m[~amb]), f"A{l}: ReLU sign differs away from zero"
        ties[l] = float(np.mean(amb))
        flipped[l] = float(np.mean(amb & (g_on != m)))
        return np.where(amb, g_on, m)

    if ora_plain is not None:
        plain_share = {}

        def plain_tie(l, z, m):
            dev = float(np.max(np.abs(acts_gpu[l] - np.maximum(z, 0.0))))
            amb = np.abs(z) <= dev
            g_on = acts_gpu[l] > 0
            assert np.array_equal(g_on[~amb], m[~amb]), f"A{l}: ReLU sign differs from the plain oracle beyond the deviation"
            plain_share[l] = float(np.mean(amb))
            return np.where(amb, g_on, m)

        loss_p = ora_plain.loss_and_grads(x, cls, plain_tie)
        report["plain_tie_share"] = plain_share
        for l, share in plain_share.items():
            assert share <= PLAIN_TIE_CEILING[precision], f"A{l}: {share:.2e} of the units within the deviation of zero"
        plain = {"loss": abs(float(loss_t.item()) - loss_p) / max(abs(loss_p), 1e-30)}
        for l in range(1, ora.n_layers + 1):
            plain[f"A{l}"] = rel_err(acts_gpu[l], ora_plain.acts[l])
        for l in range(ora.n_layers):
            plain[f"dW{l}"] = rel_err(grads_gpu[l][0], ora_plain.dW[l])
            plain[f"db{l}"] = rel_err(grads_gpu[l][1], ora_plain.db[l])
        report["vs_plain_fp32_oracle"] = plain
        bad = {k: v for k, v in plain.items() if not (v <= PLAIN_TOL[precision])}
        assert not bad, f"against the plain fp32 oracle, beyond {PLAIN_TOL[precision]}: {bad}  (all: {plain})"

    use_ties = precision != "fp32"
    if use_ties:
        ora.loss_and_grads(x, cls)                      # the oracle left alone: its own ReLU decisions
        own = [g.copy() for g in ora.dW + ora.db]
    loss_o = ora.train_step(x, cls, tie_break if use_ties else None)
    if use_ties:
        report["tie_share"] = dict(ties)
        report["tie_flipped"] = dict(flipped)
        report["tie_effect"] = max(rel_err(a, b) for a, b in zip(ora.dW + ora.db, own))
        for l, share in ties.items():
            assert share <= TIE_CEILING[precision], f"A{l}: {share:.2e} of the units lie in the tie band (ceiling {TIE_CEILING[precision]})"
        for l, share in flipped.items():
            n_units = ora.acts[l].size
            assert share * n_units <= max(TIE_FLIPS_MIN, TIE_FLIPS[precision] * n_units), \
                f"A{l}: {share * n_units:.0f} ReLU decisions differ from the oracle's own"
    errs = {"loss": abs(float(loss_t.item()) - loss_o) / max(abs(loss_o), 1e-30)}
    for l in range(1, ora.n_layers + 1):
        errs[f"A{l}"] = rel_err(acts_gpu[l], ora.acts[l])
    well_share = {}
    for l in range(ora.n_layers):
        dW, db = grads_gpu[l]
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
            well_share[name] = float(np.mean(well))
            assert float(diff.max()) <= 3.0 * ora.lr + tol * scale, (name, float(diff.max()))
            assert well_share[name] >= ADAM_WELL_FLOOR, f"{name}: only {well_share[name]:.2f} of the elements are compared at tolerance"
    if well_share:
        report["adam_well_conditioned_share"] = well_share
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, f"beyond tolerance {tol}: {bad}  (all: {errs})"
    return errs
