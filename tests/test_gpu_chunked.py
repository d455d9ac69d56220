"""Chunked prefill with pooled statistics carried from chunk to chunk (Sec. 4.3 "Compatibility with Chunked
Prefill"): the lists, the pooled arrays and the attention output of a chunk must not depend on whether its prefix
was pooled again or carried over."""
import numpy as np
import pytest
import torch

from oracle import fp2_oracle as O
from paper_2608_19758_b200 import binding, inputs
from test_gpu_parity import check_attention, check_lists

pytestmark = pytest.mark.gpu


def chunk_case(case, lens_k, lens_q):
    """The same batch seen at an earlier point of its prefill: sequence b has lens_k[b] KV tokens of which the
    last lens_q[b] are new.  Shares the KV pool and page table of `case`; queries are the matching rows."""
    import copy
    c = copy.copy(case)
    cu_full = case.cu_seqlens_q.numpy()
    pre_full = (case.seqlens_k.numpy() - np.diff(cu_full))
    rows = []
    for b, (lk, lq) in enumerate(zip(lens_k, lens_q)):
        first = cu_full[b] + (lk - lq) - pre_full[b]
        rows.append(torch.arange(first, first + lq))
    c.q = case.q[torch.cat(rows)].contiguous()
    c.cu_seqlens_q = torch.tensor(np.concatenate([[0], np.cumsum(lens_q)]), dtype=torch.int32)
    c.seqlens_k = torch.tensor(lens_k, dtype=torch.int32)
    return c


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_carried_pooled_means_give_identical_lists_and_outputs(dtype):
    spec = inputs.small_spec(seqs=[(3000, 0), (900, 0), (257, 0)], num_q_heads=8, num_kv_heads=2, page_size=16,
                             dtype=dtype, config_id=90)
    spec.alpha = 0.1
    full = inputs.make_case(spec)
    c1 = chunk_case(full, [1700, 500, 128], [1700, 500, 128])          # first chunk of every sequence
    c2 = chunk_case(full, [3000, 900, 257], [1300, 400, 129])          # second chunk: the rest
    d1, d2, d2f = binding.DeviceCase(c1), binding.DeviceCase(c2), binding.DeviceCase(c2)
    d1.select(); d1.status()
    assert binding.fp2_pool_carry_count(d2.plan, d1.plan, [0, 1, 2]) == [13, 3, 1]
    binding.fp2_pool_carry(d2.plan, d2.workspace, d1.plan, d1.workspace, [0, 1, 2])
    assert d2.plan.last_launch_count() == 1
    d2.select(); d2.status()
    d2f.select(); d2f.status()                                         # the same chunk, pooled from scratch
    assert torch.equal(d2.seg_count, d2f.seg_count) and torch.equal(d2.blk_idx, d2f.blk_idx)
    # pooled arrays (everything between the 128-byte header and the work order is pooled statistics)
    a, b = d2.workspace.view(torch.uint8), d2f.workspace.view(torch.uint8)
    nb = sum(-(-l // 128) for l in [3000, 900, 257])
    pooled_bytes = 1024 + 3 * ((nb * 2 * 128 * 2 + 1023) // 1024 * 1024)
    assert torch.equal(a[1024:pooled_bytes], b[1024:pooled_bytes])
    d2.sparse(); d2.status()
    d2f.sparse(); d2f.status()
    assert torch.equal(d2.out, d2f.out) and torch.equal(d2.lse, d2f.lse)
    # and against the oracle
    prm = dict(c2.params())
    wl = O.Workload(O.Params.from_dict(prm), **inputs.oracle_args(c2))
    check_lists(d2, wl)
    check_attention(d2, wl, d2.lists_host(), dtype=dtype)
    # a second select on the same plan pools everything again (the carry is used once) -- same result
    d2.select(); d2.status()
    assert torch.equal(d2.blk_idx, d2f.blk_idx)


def test_carry_with_new_and_reordered_sequences():
    spec = inputs.small_spec(seqs=[(2000, 0), (1000, 0)], num_q_heads=4, num_kv_heads=2, page_size=64, config_id=91)
    full = inputs.make_case(spec)
    c1 = chunk_case(full, [1000, 600], [1000, 600])
    d1 = binding.DeviceCase(c1)
    d1.select(); d1.status()
    # next step: the batch now lists the second sequence first, and a carry from "nowhere" for the other
    spec2 = inputs.small_spec(seqs=[(1000, 600), (2000, 1000)], num_q_heads=4, num_kv_heads=2, page_size=64,
                              config_id=91)
    c2 = inputs.make_case(spec2)
    # same KV contents as `full`, sequences swapped: rebuild the page table rows accordingly
    c2.k_cache, c2.v_cache = full.k_cache, full.v_cache
    c2.page_table = full.page_table[[1, 0]].contiguous()
    d2, d2f = binding.DeviceCase(c2), binding.DeviceCase(c2)
    assert binding.fp2_pool_carry_count(d2.plan, d1.plan, [1, -1]) == [4, 0]
    binding.fp2_pool_carry(d2.plan, d2.workspace, d1.plan, d1.workspace, [1, -1])
    d2.select(); d2.status()
    d2f.select(); d2f.status()
    assert torch.equal(d2.seg_count, d2f.seg_count) and torch.equal(d2.blk_idx, d2f.blk_idx)
