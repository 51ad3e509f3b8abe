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
