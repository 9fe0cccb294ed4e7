"""bench.py --gpus N runs independent replicas: every rank draws its own batch and the ranks only
exchange their elapsed times (MAX) and meet at barriers.  This covers that host-side logic with
two gloo ranks on CPU."""
import os
import socket

import numpy as np
import pytest

import wersa_inputs as wi


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # the per-rank batch of bench.py: same shape, seed shifted by 1000 per rank
    _, inp = wi.make_config("cfg1_single_head_fp32", seed=wi.CONFIGS["cfg1_single_head_fp32"]["seed"] + 1000 * rank)
    digest = float(np.abs(inp["Q"]).sum())
    dist.barrier()
    t = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)      # pretend elapsed ms of this rank
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    d = torch.tensor([digest], dtype=torch.float64)
    gathered = [torch.zeros_like(d) for _ in range(world)]
    dist.all_gather(gathered, d)
    out[rank] = (float(t.item()), [float(g.item()) for g in gathered])
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_reduce_max_time_and_draw_different_batches():
    import torch.multiprocessing as mp
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        t_max, digests = res[rank]
        assert t_max == 15.0                      # max over ranks, seen by every rank
        assert digests[0] != digests[1]           # different seeds -> different batches
    assert res[0][1] == res[1][1]
