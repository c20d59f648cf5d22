"""The multi-GPU path on CPU: two `gloo` ranks run the replica plumbing of the benchmark (the path
has no exchange step, so ranks share only the barrier and the maximum of their step times)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_06938_b200 import replicas, synth


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.rank_env() == (rank, world, rank)
        cfg = synth.LayerConfig("replica", "bf16", 2, 64, 64, 2, 64, 128, 1, 4, 2, 128)
        inp = synth.make_inputs(cfg, seed=replicas.replica_seed(rank, 0))
        # each replica has its own batch; a checksum travels to rank 0 through the timing channel
        checksum = float(inp["u"].float().abs().sum())
        ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        dist.barrier()
        ms = replicas.max_over_ranks(ms_local, dist)
        value = replicas.whole_job_throughput(world, cfg.tokens, ms)
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, torch.tensor([checksum], dtype=torch.float64))
        out[rank] = (ms, value, [float(s) for s in sums])
    finally:
        dist.destroy_process_group()


def test_two_replicas_share_only_the_timing():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    tokens = 2 * 64
    for rank in (0, 1):
        ms, value, sums = res[rank]
        assert ms == 15.0                                   # the maximum over ranks, on every rank
        assert abs(value - world * tokens / 15e-3) < 1e-6   # whole-job figure
        assert sums[0] != sums[1]                           # the replicas worked on different batches


def test_single_process_defaults():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.rank_env() == (0, 1, 0)
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.replica_seed(0, 3) != replicas.replica_seed(1, 3)
