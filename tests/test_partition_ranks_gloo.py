"""One partition per process (Section 2.1): rank k trains segment k and hands its stored response to rank
k + 1 in a single point-to-point message.  The orchestration (`binding.train_partitioned_ranks`) is run
here as three gloo ranks on CPU; each rank's segment is the CPU oracle behind the small interface the
function needs, so what is under test is the order of training and hand-off, the shapes and dtypes of the
messages, and that nothing else is exchanged.  The result must equal the single-process procedure exactly.
"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
WIDTHS = [[12, 10, 8], [8, 7, 6], [6, 5, 4]]


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _oracles():
    from oracle import rng
    from oracle.segment import OracleSegment
    segs = []
    for k, w in enumerate(WIDTHS):
        s = OracleSegment(w, 4, k == len(WIDTHS) - 1, precision="fp32", optimizer="momentum", lr=0.05, segment_id=k)
        if k < len(WIDTHS) - 1:
            s.gen_labels(1, rng.DIST_UNIFORM_KAPPA, 2.0)
        segs.append(s)
    return segs


def _data(n=50):
    g = np.random.default_rng(0)
    return g.random((n, 12)).astype(np.float32), g.integers(0, 4, n).astype(np.int32)


class OracleBehindTheSegmentInterface:
    """What train_partitioned_ranks needs of a segment, served by the CPU oracle on torch CPU tensors."""

    def __init__(self, ora):
        from oracle import pnn
        self.ora, self.pnn = ora, pnn
        self.widths, self.act_dtype = ora.widths, torch.float32

    def train_epochs(self, x, cls, batch, epochs, losses):
        out = self.pnn.train_epochs(self.ora, x.numpy(), cls.numpy(), batch, epochs)
        losses[:len(out)] = torch.from_numpy(out.astype(np.float32))

    def forward_dataset(self, x, batch):
        return torch.from_numpy(self.pnn.forward_dataset(self.ora, x.numpy(), batch))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2403_11204_b200 import binding
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x, cls = _data()
    seg = OracleBehindTheSegmentInterface(_oracles()[rank])
    losses, cur = binding.train_partitioned_ranks(seg, torch.from_numpy(x) if rank == 0 else None,
                                                  torch.from_numpy(cls), 16, 2, rank, world)
    out.put((rank, losses.numpy().copy(), cur.numpy().copy()))
    dist.barrier()
    dist.destroy_process_group()


def test_three_ranks_reproduce_the_single_process_procedure():
    from oracle import pnn
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 3, port, out)) for r in range(3)]
    for p in procs:
        p.start()
    got = {}
    for _ in procs:
        r, losses, cur = out.get()
        got[r] = (losses, cur)
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    x, cls = _data()
    segs = _oracles()
    ref_losses, _ = pnn.train_partitioned(segs, x, cls, 16, [2, 2, 2])
    inputs = [x]
    segs2 = _oracles()
    for k in range(2):                                   # the input every later rank must have received
        pnn.train_epochs(segs2[k], inputs[-1], cls, 16, 2)
        inputs.append(pnn.forward_dataset(segs2[k], inputs[-1], 16))
    for r in range(3):
        assert np.array_equal(got[r][0], ref_losses[r].astype(np.float32)), r
        assert np.array_equal(got[r][1], inputs[r]), r
        assert got[r][1].shape == (50, WIDTHS[r][0])
