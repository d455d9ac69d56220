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


# ------------------------------------------------------------------------------------------------------
# one workload split by KV head (strong scaling): the union of the ranks' results is the unsplit result
# ------------------------------------------------------------------------------------------------------

def _head_worker(rank, world, port, out, dtype):
    import numpy as np
    from oracle import fp2_oracle as O
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    whole = inputs.small_spec(seqs=[(700, 100), (300, 0)], num_q_heads=8, num_kv_heads=4, page_size=16,
                              dtype=dtype, config_id=33)
    whole.alpha = 0.2
    spec = shard.shard_spec_by_heads(whole, rank, world)
    case = inputs.make_case(spec)
    # the rank's planner geometry and oracle run on its head slice alone
    wl = O.Workload(O.Params.from_dict(case.params()), **inputs.oracle_args(case))
    sel = O.oracle_select(wl)
    lists = {k: v[0] for k, v in sel.items()}
    o, lse = O.scatter_output(wl, O.oracle_attend(wl, lists), case.total_q)
    o_all = shard.gather_heads(dist, torch.from_numpy(o), head_dim=1)
    lse_all = shard.gather_heads(dist, torch.from_numpy(lse), head_dim=0)
    counts = torch.tensor([len(lists[s.seg]) for s in wl.segs], dtype=torch.int64)
    parts = [torch.empty_like(counts) for _ in range(world)]
    dist.all_gather(parts, counts)
    if rank == 0:
        out["o"], out["lse"], out["counts"] = o_all.numpy(), lse_all.numpy(), [p.tolist() for p in parts]
        out["q_rank0"] = case.q.float().numpy() if dtype == "bf16" else case.q.numpy()
    dist.destroy_process_group()


def _whole_reference(dtype):
    import numpy as np
    from oracle import fp2_oracle as O
    whole = inputs.small_spec(seqs=[(700, 100), (300, 0)], num_q_heads=8, num_kv_heads=4, page_size=16,
                              dtype=dtype, config_id=33)
    whole.alpha = 0.2
    case = inputs.make_case(whole)
    wl = O.Workload(O.Params.from_dict(case.params()), **inputs.oracle_args(case))
    sel = O.oracle_select(wl)
    lists = {k: v[0] for k, v in sel.items()}
    o, lse = O.scatter_output(wl, O.oracle_attend(wl, lists), case.total_q)
    return case, wl, lists, o, lse


def test_head_sharded_ranks_reproduce_the_unsplit_result_bit_for_bit():
    import numpy as np
    for dtype in ("bf16", "fp8"):
        world = 2
        mgr = mp.Manager()
        out = mgr.dict()
        mp.spawn(_head_worker, args=(world, _free_port(), out, dtype), nprocs=world, join=True)
        case, wl, lists, o, lse = _whole_reference(dtype)
        assert np.array_equal(out["o"], o) and np.array_equal(out["lse"], lse)      # fp64, bit for bit
        # list lengths: rank r's segments are the whole workload's segments of its heads, in the same order
        hkv = case.spec.num_kv_heads
        for r in range(world):
            mine = [len(lists[s.seg]) for s in wl.segs if r * hkv // world <= s.h < (r + 1) * hkv // world]
            assert mine == out["counts"][r]
        # the rank draws exactly the head slice of the whole workload's tensors
        sl = shard.slice_case_heads(case, 0, hkv // world)
        q0 = sl.q.float().numpy() if dtype == "bf16" else sl.q.numpy()
        assert np.array_equal(q0, out["q_rank0"])


def test_slice_case_heads_matches_a_rank_drawn_shard():
    whole = inputs.small_spec(seqs=[(500, 0)], num_q_heads=12, num_kv_heads=4, page_size=32, dtype="fp8", config_id=34)
    case = inputs.make_case(whole)
    for world in (2, 4):
        for r in range(world):
            mine = inputs.make_case(shard.shard_spec_by_heads(whole, r, world))
            per = 4 // world
            sl = shard.slice_case_heads(case, r * per, (r + 1) * per)
            for a, b in ((mine.q, sl.q), (mine.k_cache, sl.k_cache), (mine.v_cache, sl.v_cache),
                         (mine.q_scale, sl.q_scale), (mine.k_scale, sl.k_scale), (mine.v_scale, sl.v_scale),
                         (mine.page_table, sl.page_table)):
                assert torch.equal(a, b)
            assert mine.params() == sl.params()
