"""KV splitting (Eq. 18): the attention path with segments cut into parts and merged must give the oracle's
result within the same gates, whatever the number of parts."""
import numpy as np
import pytest
import torch

from oracle import fp2_oracle as O
from paper_2608_19758_b200 import binding, inputs
from test_gpu_parity import check_attention, check_lists, make

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("target", [1, 2, 5, 0, -1])
@pytest.mark.parametrize("dtype,g,hkv,p,seqs", [
    ("bf16", 4, 2, 16, [(1500, 300), (700, 0), (129, 128), (40, 0)]),
    ("bf16", 7, 1, 64, [(3000, 0)]),
    ("fp8", 4, 2, 32, [(2500, 500), (257, 0)]),
])
def test_split_attention_matches_oracle(target, dtype, g, hkv, p, seqs):
    spec = inputs.small_spec(seqs=seqs, num_q_heads=g * hkv, num_kv_heads=hkv, page_size=p, dtype=dtype,
                             config_id=70 + g)
    spec.alpha = 0.2
    case, dc, wl = make(spec)
    dc.plan.set_split(target)
    dc.select(); dc.status()
    lists = dc.lists_host()
    dc.sparse(); dc.status()
    if target != 0:                                    # automatic: the host may see that nothing can be split
        assert dc.plan.last_launch_count() == (4 if target < 0 else 6)
    check_attention(dc, wl, lists, dtype=dtype)
    dc.dense(); dc.status()
    check_attention(dc, wl, None, dense=True, dtype=dtype)


def test_split_without_correction_and_with_caller_lists():
    """Lists of one block per segment (every part but the first is empty at target 1 ... no: one iteration, one
    part) and long hand-made lists that are cut into many parts."""
    spec = inputs.small_spec(seqs=[(4096, 0)], num_q_heads=4, num_kv_heads=2, page_size=64, config_id=77)
    case, dc, wl = make(spec, use_correction=0)
    dc.plan.set_split(1)
    dc.select(); dc.status()
    off = dc.seg_offset.cpu().numpy()
    cnt = np.zeros(dc.plan.num_segments, dtype=np.int32)
    idx = dc.blk_idx.cpu().numpy().copy()
    lists = {}
    for s in wl.segs:                                   # every second candidate, always the diagonal band
        L = sorted(set(range(0, s.J_hi + 1, 2)) | set(range(s.J_lo, s.J_hi + 1)))
        lists[s.seg] = np.asarray(L, dtype=np.int32)
        cnt[s.seg] = len(L)
        idx[off[s.seg]:off[s.seg] + len(L)] = L
    dc.sparse(seg_count=torch.from_numpy(cnt).cuda(), blk_idx=torch.from_numpy(idx).cuda())
    dc.status()
    check_attention(dc, wl, lists)


def test_split_is_deterministic_and_equals_unsplit_within_rounding():
    spec = inputs.config_spec(1)
    case, dc, wl = make(spec)
    dc.select(); dc.status()
    dc.plan.set_split(2)
    dc.sparse(); torch.cuda.synchronize()
    a, la = dc.out.clone(), dc.lse.clone()
    dc.sparse(); torch.cuda.synchronize()
    assert torch.equal(a, dc.out) and torch.equal(la, dc.lse)
    dc.plan.set_split(-1)
    dc.sparse(); torch.cuda.synchronize()
    dc.status()
    assert (a.float() - dc.out.float()).abs().max().item() <= 2e-2
    assert torch.allclose(la, dc.lse, rtol=1e-5, atol=1e-5)


def test_large_plans_are_not_split():
    spec = inputs.config_spec(2, scale_down=2)           # 16K tokens: 4096 segments, more than 4 per worker
    case, dc, wl = make(spec)
    dc.plan.set_split(1)
    dc.select(); dc.sparse(); dc.status()
    assert dc.plan.last_launch_count() == 4
