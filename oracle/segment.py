"""Oracle for one training step of a fully connected network segment.

TEST INFRASTRUCTURE ONLY: plain NumPy, every contraction and reduction accumulated in
float64, no blocking, no fusion; the formulas are written as the definitions read.
Shares no code with the CUDA library.

What is computed (paper: Section 2 for the procedure, Section 3 for the network):
  * a segment is a stack of Linear layers  Z_l = A_{l-1} W_l^T + b_l,  A_l = relu(Z_l);
    only the network's final layer is left without ReLU (Section 3);
  * a non-final segment regresses its output on the synthetic intermediate label of
    the sample's class: target T_b = SIL[class_b] (Section 2, Eq. 1; Section 3: each
    image's label is one column of the SIL matrix).  The paper does not name the loss;
    mean squared error over all B*N_P elements is used;
  * the final segment is trained on the original class labels (Section 2, second
    phase); softmax cross-entropy averaged over the batch is used;
  * gradients stay inside the segment (Section 1: nothing is exchanged between
    partitions), so no gradient with respect to the segment input is formed;
  * optimizer: SGD with momentum as in Section 3 (buf = mu*buf + g; p -= lr*buf), plain
    SGD, and Adam (bias-corrected, no weight decay) for the synthetic workloads.

Precision modes
  "fp64": everything float64 (finite-difference checks).
  "fp32": fp32 storage of parameters/activations/gradients, float64 accumulation.
  "tf32": fp32 storage; matrix-product operands are TF32 (10-bit mantissa, round to
          nearest even): weights through a rounded copy, hidden activations and
          back-propagated dZ rounded when they are stored; final logits stay fp32.
  "bf16": fp32 master parameters; matrix-product operands are bf16: weights are rounded
          to bf16 copies, hidden activations and back-propagated dZ are stored in bf16;
          the final segment's logits stay fp32.
ReLU ties.  relu'(z) is taken as 1 for z > 0 and 0 otherwise, decided on the oracle's own
pre-activation.  A caller comparing against another implementation may pass `tie_break`
to loss_and_grads: for elements whose |z| is below the caller's ambiguity threshold (both
signs are correct answers within the stated tolerance of the activations) it may choose
the derivative; everywhere else the oracle's own decision stands.  The forward values
are never altered.
Pins live in tests/test_oracle_segment.py (finite differences, closed forms, invariants).
"""
import numpy as np

from . import rng


def round_bf16(a):
    """Round fp32 values to the nearest bf16 (ties to even); result held in fp32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(np.shape(a))


def round_tf32(a):
    """Round fp32 values to TF32 (8-bit exponent, 10-bit mantissa; ties to even)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x0FFF) + ((u >> np.uint64(13)) & np.uint64(1))) & np.uint64(0xFFFFE000)
    return u.astype(np.uint32).view(np.float32).reshape(np.shape(a))


def mse_loss(a, target):
    """loss = mean over all B*N elements of (a - t)^2;  dloss/da = 2 (a - t) / (B*N)."""
    d = a.astype(np.float64) - target.astype(np.float64)
    n = d.size
    return float(np.sum(d * d) / n), 2.0 * d / n


def softmax_ce_loss(z, cls):
    """loss = -mean_b log softmax(z_b)[cls_b];  dloss/dz = (softmax(z) - onehot) / B."""
    z = z.astype(np.float64)
    bsz = z.shape[0]
    zs = z - z.max(axis=1, keepdims=True)
    ez = np.exp(zs)
    p = ez / ez.sum(axis=1, keepdims=True)
    logp = zs - np.log(ez.sum(axis=1, keepdims=True))
    loss = float(-np.sum(logp[np.arange(bsz), cls]) / bsz)
    dz = p.copy()
    dz[np.arange(bsz), cls] -= 1.0
    return loss, dz / bsz


class OracleSegment:
    """State and one-step arithmetic of one segment."""

    def __init__(self, widths, n_classes, is_final, last_relu=None, precision="fp32",
                 optimizer="sgd", lr=0.01, momentum=0.9, beta1=0.9, beta2=0.999, eps=1e-8,
                 segment_id=0, init_seed=2):
        assert precision in ("fp64", "fp32", "tf32", "bf16")
        assert optimizer in ("sgd", "momentum", "adam")
        self.widths = [int(w) for w in widths]
        self.n_layers = len(self.widths) - 1
        self.n_classes = int(n_classes)
        self.is_final = bool(is_final)
        self.last_relu = (not self.is_final) if last_relu is None else bool(last_relu)
        self.precision = precision
        self.optimizer = optimizer
        self.lr, self.momentum = float(lr), float(momentum)
        self.beta1, self.beta2, self.eps = float(beta1), float(beta2), float(eps)
        self.segment_id = int(segment_id)
        self.store = np.float64 if precision == "fp64" else np.float32
        self.W, self.b = [], []
        for l in range(self.n_layers):
            W, b = rng.init_linear(init_seed, self.segment_id, l, self.widths[l], self.widths[l + 1])
            self.W.append(W.astype(self.store))
            self.b.append(b.astype(self.store))
        zeros = lambda: [np.zeros_like(p) for p in self.W + self.b]
        self.state1 = zeros()        # momentum buffer, or Adam first moment
        self.state2 = zeros()        # Adam second moment
        self.t = 0                   # optimizer step counter
        self.sil = None
        self.acts = self.dZ = self.dW = self.db = None

    # -- Eq. 1 -----------------------------------------------------------------------
    def gen_labels(self, seed, dist=rng.DIST_UNIFORM_KAPPA, kappa=10.0):
        self.sil = rng.gen_labels(seed, self.segment_id, self.n_classes, self.widths[-1], dist, kappa)
        return self.sil

    # -- rounding points of the reduced-precision modes --------------------------------
    def _operand(self, a):
        if self.precision == "tf32":
            return round_tf32(a)
        if self.precision == "bf16":
            return round_bf16(a)
        return a

    def _store_act(self, a64):
        a = a64.astype(self.store)
        if self.precision == "bf16":
            return round_bf16(a)
        if self.precision == "tf32":
            return round_tf32(a)
        return a

    # -- forward (Section 3: Linear + ReLU, identity on the network's last layer) -------
    def forward(self, x):
        acts = [np.asarray(x, dtype=self.store)]
        self.preact = []
        for l in range(self.n_layers):
            a_op = self._operand(acts[-1]).astype(np.float64)
            w_op = self._operand(self.W[l]).astype(np.float64)
            z = a_op @ w_op.T + self.b[l].astype(np.float64)
            last = l == self.n_layers - 1
            self.preact.append(z)
            if (not last) or self.last_relu:
                z = np.maximum(z, 0.0)
            if last and self.is_final:
                acts.append(z.astype(self.store))          # logits stay fp32
            else:
                acts.append(self._store_act(z))
        return acts

    # -- loss + backward -------------------------------------------------------------
    def loss_and_grads(self, x, cls, tie_break=None):
        """tie_break(layer, z, mask) -> mask: optional choice of relu' on near-zero pre-activations
        (layer = 1-based index of the activation A_layer, z = fp64 pre-activation, mask = z > 0)."""
        cls = np.asarray(cls, dtype=np.int64)
        acts = self.forward(x)
        out = acts[-1]
        masks = [None] * (self.n_layers + 1)
        for l in range(1, self.n_layers + 1):
            if l < self.n_layers or self.last_relu:
                m = acts[l] > 0
                masks[l] = tie_break(l, self.preact[l - 1], m) if tie_break is not None else m
        if self.is_final:
            loss, dz = softmax_ce_loss(out, cls)
            if self.last_relu:
                dz = dz * masks[-1]
        else:
            target = self.sil[cls]                          # gather: one SIL row per sample
            loss, da = mse_loss(out, target)
            dz = da * masks[-1] if self.last_relu else da   # relu'(0) taken as 0
        dZ = [None] * self.n_layers
        dW = [None] * self.n_layers
        db = [None] * self.n_layers
        dz = self._store_act(dz)
        for l in reversed(range(self.n_layers)):
            dZ[l] = dz
            dz_op = self._operand(dz).astype(np.float64)
            a_prev = self._operand(acts[l]).astype(np.float64)
            dW[l] = (dz_op.T @ a_prev).astype(self.store)
            db[l] = dz.astype(np.float64).sum(axis=0).astype(self.store)
            if l > 0:
                w_op = self._operand(self.W[l]).astype(np.float64)
                da_prev = dz_op @ w_op
                dz = self._store_act(da_prev * masks[l])
        self.acts, self.dZ, self.dW, self.db = acts, dZ, dW, db
        return loss

    # -- optimizer ---------------------------------------------------------------------
    def apply_update(self):
        params = self.W + self.b
        grads = self.dW + self.db
        self.t += 1
        for i, (p, g) in enumerate(zip(params, grads)):
            p64, g64 = p.astype(np.float64), g.astype(np.float64)
            if self.optimizer == "sgd":
                new = p64 - self.lr * g64
            elif self.optimizer == "momentum":
                buf = self.momentum * self.state1[i].astype(np.float64) + g64
                self.state1[i] = buf.astype(self.store)
                new = p64 - self.lr * self.state1[i].astype(np.float64)
            else:
                m = self.beta1 * self.state1[i].astype(np.float64) + (1.0 - self.beta1) * g64
                v = self.beta2 * self.state2[i].astype(np.float64) + (1.0 - self.beta2) * g64 * g64
                self.state1[i], self.state2[i] = m.astype(self.store), v.astype(self.store)
                mhat = self.state1[i].astype(np.float64) / (1.0 - self.beta1 ** self.t)
                vhat = self.state2[i].astype(np.float64) / (1.0 - self.beta2 ** self.t)
                new = p64 - self.lr * mhat / (np.sqrt(vhat) + self.eps)
            p[...] = new.astype(self.store)

    def train_step(self, x, cls, tie_break=None):
        """One step: forward, loss, backward, update.  Returns the loss before the update."""
        loss = self.loss_and_grads(x, cls, tie_break)
        self.apply_update()
        return loss

    def n_params(self):
        return sum(w.size for w in self.W) + sum(b.size for b in self.b)
