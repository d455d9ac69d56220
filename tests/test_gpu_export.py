"""GPU parity of the index export (Algorithm 1 line 5; Sec. 3.4) against the oracle: integer work, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import fp2_oracle as O
from paper_2608_19758_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def make(spec, **over):
    case = inputs.make_case(spec)
    dc = binding.DeviceCase(case, **over)
    prm = dict(case.params())
    prm.update(over)
    wl = O.Workload(O.Params.from_dict(prm), **inputs.oracle_args(case))
    return case, dc, wl


def check_export(dc, wl, tile):
    lists = dc.lists_host()
    cu, idx = dc.export_csr(tile)
    dc.status()
    assert dc.plan.last_launch_count() == 3
    want_cu, want_idx = O.export_csr(wl, lists, tile)
    got_cu = cu.cpu().numpy().astype(np.int64)
    assert (got_cu == want_cu).all()
    assert (idx.cpu().numpy()[:want_cu[-1]] == want_idx).all()
    return int(want_cu[-1])


@pytest.mark.parametrize("tile", [16, 32, 64, 128])
@pytest.mark.parametrize("seqs,g,hkv,p", [
    ([(2300, 0)], 7, 2, 64),                                    # tiles straddle positions
    ([(1500, 300), (700, 0), (129, 128), (64, 0), (1, 0)], 4, 2, 16),   # ragged last blocks of every kind
    ([(8192 + 65, 4096)], 1, 2, 128),
])
def test_export_matches_oracle(tile, seqs, g, hkv, p):
    spec = inputs.small_spec(seqs=seqs, num_q_heads=g * hkv, num_kv_heads=hkv, page_size=p, config_id=60 + g)
    spec.alpha = 0.05
    case, dc, wl = make(spec)
    dc.select(); dc.status()
    n = check_export(dc, wl, tile)
    assert n > 0


def test_export_of_dense_lists_config2():
    """All candidates listed at 32K: 2 tiles per block, 2 x 1 052 672 entries."""
    spec = inputs.config_spec(2)
    spec.alpha = 0.0                       # alpha <= 0 selects every candidate
    case, dc, wl = make(spec)
    dc.select(); dc.status()
    cu, idx = dc.export_csr(64)
    dc.status()
    cuh = cu.cpu().numpy().astype(np.int64)
    assert cuh[-1] == 2 * dc.plan.idx_capacity == 2 * 8 * 131584
    rng = np.random.default_rng(1)
    ih = idx.cpu().numpy()
    for seg in rng.choice(dc.plan.num_segments, 64, replace=False):
        s = wl.segs[seg]
        assert (ih[cuh[seg]:cuh[seg + 1]] == np.arange(2 * (s.J_hi + 1))).all()


def test_export_flags_malformed_lists():
    spec = inputs.small_spec(seqs=[(1000, 0)], num_q_heads=4, num_kv_heads=2, page_size=16, config_id=66)
    case, dc, wl = make(spec)
    dc.select(); dc.status()
    bad = dc.blk_idx.clone()
    off = int(dc.seg_offset[3].item())
    bad[off] = 10 ** 6                     # far outside 0..J_hi
    cu = torch.empty(dc.plan.num_segments + 1, dtype=torch.int32, device="cuda")
    idx = torch.empty(dc.plan.idx_capacity * 2, dtype=torch.int32, device="cuda")
    binding.fp2_export_csr(dc.plan, dc.seg_count, bad, 64, cu, idx, dc.workspace)
    code, words = dc.status(raise_on_error=False)
    assert code == 1 and words[2] & 1
    with pytest.raises(binding.Fp2Error):   # output buffer too small: refused on the host
        binding.fp2_export_csr(dc.plan, dc.seg_count, dc.blk_idx, 64, cu, idx[:5], dc.workspace)


@pytest.mark.parametrize("p", [16, 64])
def test_page_table_from_token_map(p):
    spec = inputs.small_spec(seqs=[(1500, 300), (700, 0), (129, 128), (17, 0)], num_q_heads=4, num_kv_heads=2,
                             page_size=p, config_id=67)
    case, dc, wl = make(spec)
    pt = case.page_table.numpy()
    lens = case.seqlens_k.numpy()
    tok = np.full((len(lens), int(lens.max())), -1, dtype=np.int32)
    for b, L in enumerate(lens):
        j = np.arange(L)
        tok[b, :L] = pt[b, j // p] * p + j % p                  # Eq. 22
    want, bad = O.page_table_from_token_map(tok, lens, p, pt.shape[1])
    assert not bad
    tok_d = torch.from_numpy(tok).cuda()
    out = torch.full_like(dc.page_table, -5)
    binding.fp2_page_table_from_token_map(dc.plan, tok_d, dc.seqlens_k, out, dc.workspace)
    dc.status()
    assert (out.cpu().numpy() == want).all()
    # and the derived table drives the path to the same result as the original one
    dc.select(); dc.status()
    a = dc.lists_host()
    dc.page_table = out
    dc.select(); dc.status()
    b = dc.lists_host()
    assert all((a[s] == b[s]).all() for s in a)
    tok[0, p] += 1                                               # not the first slot of a page
    binding.fp2_page_table_from_token_map(dc.plan, torch.from_numpy(tok).cuda(), dc.seqlens_k, out, dc.workspace)
    code, words = dc.status(raise_on_error=False)
    assert code == 1 and words[2] & 4
