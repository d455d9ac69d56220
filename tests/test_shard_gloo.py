"""The N > 1 launch path on CPU: two gloo ranks, independent shards, max-over-ranks timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_19758_b200 import inputs, shard


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = shard.shard_spec(inputs.config_spec(2, scale_down=64), rank, world)
    case = inputs.make_case(spec)
    shard.barrier(dist)
    ms_local = 10.0 + 5.0 * rank              # rank 1 is the slow one
    units_local = float(case.total_q)
    value, ms, units = shard.aggregate(dist, ms_local, units_local)
    out[rank] = (value, ms, units, spec.config_id, float(case.q.float().abs().sum()))
    dist.destroy_process_group()


def test_two_ranks_take_independent_shards_and_report_the_slowest_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert len(out) == 2
    v0, ms0, u0, id0, sum0 = out[0]
    v1, ms1, u1, id1, sum1 = out[1]
    assert ms0 == ms1 == 15.0                 # max over ranks
    assert u0 == u1 == 2 * 512                # units of the whole job
    assert v0 == v1 == (2 * 512) / 15e-3
    assert id0 != id1 and sum0 != sum1        # different seeds: different data, same shape


def test_single_rank_is_the_plain_benchmark():
    spec = inputs.config_spec(3)
    assert shard.shard_spec(spec, 0, 1).config_id == spec.config_id
    value, ms, units = shard.aggregate(None, 20.0, 1000.0)
    assert (value, ms, units) == (1000.0 / 20e-3, 20.0, 1000.0)
