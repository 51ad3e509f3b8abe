"""Oracle for the paper's training procedure around the segment step (Section 2, Figs. 3 and 4).

TEST INFRASTRUCTURE ONLY.  Plain loops over OracleSegment.train_step, in the order the paper
states: segment k is trained for its own number of epochs on the stored response of segment k-1
(segment 0 on the original inputs), without shuffling, against its own intermediate labels (the
last segment against the class labels); after its training ends its response over the whole set
is stored and becomes the input of segment k+1.  "The response at the last epoch" is read as one
inference pass with the final weights.
"""
import numpy as np


def train_epochs(seg, x, cls, batch, epochs):
    """epochs passes over (x, cls) in stored order; a last partial batch is a smaller step."""
    losses = []
    n = x.shape[0]
    for _ in range(epochs):
        for i in range(0, n, batch):
            losses.append(seg.train_step(x[i:i + batch], cls[i:i + batch]))
    return np.array(losses)


def forward_dataset(seg, x, batch):
    return np.concatenate([seg.forward(x[i:i + batch])[-1] for i in range(0, x.shape[0], batch)], axis=0)


def train_partitioned(segments, x, cls, batch, epochs):
    losses, cur = [], x
    for k, (seg, n_ep) in enumerate(zip(segments, epochs)):
        losses.append(train_epochs(seg, cur, cls, batch, n_ep))
        if k + 1 < len(segments):
            cur = forward_dataset(seg, cur, batch)
    return losses, cur


def predict(segments, x, batch):
    cur = x
    for seg in segments:
        cur = forward_dataset(seg, cur, batch)
    return np.argmax(cur, axis=1)


def recovery_step(left, right, x, cls):
    """One step of the recovery phase (Section 5): the left partition is trained further through the
    right one, whose weights are frozen.  Forward through both, softmax cross-entropy on the class
    labels, back-propagation through the right partition down to its input, then the left partition's
    own backward pass and optimizer update.  Returns the joined network's loss before the update."""
    from .segment import softmax_ce_loss
    cls = np.asarray(cls, dtype=np.int64)
    acts_l = left.forward(x)
    acts_r = right.forward(acts_l[-1])
    loss, dz = softmax_ce_loss(acts_r[-1], cls)
    dz = right._store_act(dz)
    for l in reversed(range(right.n_layers)):                 # right: gradient w.r.t. activations only
        da = right._operand(dz).astype(np.float64) @ right._operand(right.W[l]).astype(np.float64)
        if l > 0:
            dz = right._store_act(da * (acts_r[l] > 0))
    dz = da * (acts_l[-1] > 0) if left.last_relu else da       # into the left partition's last layer
    dz = left._store_act(dz)
    n = left.n_layers
    dW, db, dZ = [None] * n, [None] * n, [None] * n
    for l in reversed(range(n)):
        dZ[l] = dz
        dz_op = left._operand(dz).astype(np.float64)
        dW[l] = (dz_op.T @ left._operand(acts_l[l]).astype(np.float64)).astype(left.store)
        db[l] = dz.astype(np.float64).sum(axis=0).astype(left.store)
        if l > 0:
            dz = left._store_act((dz_op @ left._operand(left.W[l]).astype(np.float64)) * (acts_l[l] > 0))
    left.acts, left.dZ, left.dW, left.db = acts_l, dZ, dW, db
    right.acts = acts_r
    left.apply_update()
    return loss
