"""The sequence-sharded forward's exchange on CPU: two and three `gloo` ranks gather their summaries
in rank order, and the per-rank driver hands the library the right rank, world size and gathered
arrays (the library is replaced by a recorder here: the kernels need a GPU, the plumbing does not)."""
import os
import socket
import types

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_06938_b200 import sharded


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class Recorder:
    """Stands in for the binding module: the summary of rank r is filled with r + 1 (state) and
    1 / (r + 2) (decay); finish records what it was given."""

    def __init__(self, rank):
        self.rank = rank
        self.finish_args = None

    def swimba_shard_summary(self, h, w, u, x, dt, B, L, state, decay, idx, wt, workspace, stream=None):
        state.fill_(float(self.rank + 1))
        decay.fill_(1.0 / (self.rank + 2))

    def swimba_shard_finish(self, h, w, x, h0, all_state, all_decay, rank, world, B, L, y, h_end, workspace,
                            stream=None):
        self.finish_args = (rank, world, all_state.clone(), all_decay.clone())
        y.zero_()


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, L, H, P, N = 2, 5, 3, 4, 8
        rec = Recorder(rank)
        handle = types.SimpleNamespace(cfg=types.SimpleNamespace(d_state=N))
        x = torch.zeros(B, L, H, P)
        y = torch.ones(B, L, H, P)
        all_state, all_decay = sharded.sequence_sharded_forward(rec, handle, None, None, x, None, None, B, L, y,
                                                                None, None, dist=dist)
        r_, w_, st, dc = rec.finish_args
        out[rank] = (r_, w_, tuple(st.shape), tuple(dc.shape), [float(st[i].mean()) for i in range(world)],
                     [float(dc[i].mean()) for i in range(world)], float(y.abs().sum()),
                     bool(torch.equal(st, all_state)))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_summaries_arrive_in_rank_order_on_every_rank(world):
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == set(range(world))
    for rank in range(world):
        r_, w_, st_shape, dc_shape, st_means, dc_means, ysum, same = res[rank]
        assert (r_, w_) == (rank, world)
        assert st_shape == (world, 2, 3, 4, 8) and dc_shape == (world, 2, 3)
        assert st_means == [float(i + 1) for i in range(world)]
        assert all(abs(dc_means[i] - 1.0 / (i + 2)) < 1e-7 for i in range(world))
        assert ysum == 0.0 and same


def test_single_process_needs_no_group():
    st, dc = torch.ones(1, 2, 3, 4), torch.ones(1, 2)
    a, d = sharded.gather_summaries(st, dc)
    assert tuple(a.shape) == (1, 1, 2, 3, 4) and tuple(d.shape) == (1, 1, 2)
