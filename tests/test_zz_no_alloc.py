"""fp2_dense_prefill_static: the dense path for callers that cannot hand in (or create) a device workspace --
for instance a plug-in that was handed fixed buffers, or code on a path where the allocator must not be entered.  Its scratch is a device array inside
the library; the call itself allocates nothing.

The file name sorts last on purpose: a run that stops at the first failure has then already run every other
test.  The check: two calls in a row (the second one meets the scratch as the first left it) must both
reproduce what fp2_dense_prefill writes with a caller workspace, within the tolerances of the parity tests.
"""
import numpy as np
import pytest
import torch

from paper_2608_19758_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _run_static(dc, out, lse):
    binding.fp2_dense_prefill_static(dc.plan, dc.q, dc.k_cache, dc.v_cache, dc.page_table, dc.cu_seqlens_q,
                                     dc.seqlens_k, dc.q_scale, dc.k_scale, dc.v_scale, out, lse)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_static_scratch_dense_matches_workspace_dense_twice(dtype):
    spec = inputs.small_spec(seqs=[(1900, 300), (700, 0), (129, 128)], num_q_heads=8, num_kv_heads=2,
                             page_size=16, config_id=95, dtype=dtype)
    case = inputs.make_case(spec)
    dc = binding.DeviceCase(case)
    dc.dense()
    dc.status()
    ref_o = dc.out.float().clone()
    ref_l = dc.lse.clone()
    tol = 2e-2 if dtype == "bf16" else 6e-2
    for call in range(2):
        out = torch.full_like(dc.out, float("nan"))
        lse = torch.full_like(dc.lse, float("nan"))
        torch.cuda.synchronize()
        # "allocates nothing": neither the driver's free memory nor torch's own pool may move across the call
        free_before, _ = torch.cuda.mem_get_info()
        torch_before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        _run_static(dc, out, lse)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, (call, free_before, free_after)
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == torch_before
        # the status block of this variant lives in the library's own array: read through the NULL workspace
        code, words = binding.fp2_read_status(dc.plan, None, raise_on_error=False)
        assert code == 0 and not any(words), (call, code, words)
        assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all(), f"call {call}"
        err_o = (out.float() - ref_o).abs().max().item()
        err_l = ((lse - ref_l).abs() / ref_l.abs().clamp_min(1.0)).max().item()
        assert err_o <= tol, (call, err_o)
        assert err_l <= 1e-3, (call, err_l)


def test_static_scratch_reports_a_skipped_page_id():
    """A page id outside the pool in a live page-table entry is skipped and flagged; the flag of the static
    variant is read through fp2_read_status with a NULL workspace, and the next call is clean again."""
    spec = inputs.small_spec(seqs=[(600, 0)], num_q_heads=4, num_kv_heads=2, page_size=16, config_id=96)
    case = inputs.make_case(spec)
    dc = binding.DeviceCase(case)
    out = torch.full_like(dc.out, float("nan"))
    good = dc.page_table.clone()
    dc.page_table[0, 3] = dc.prm["num_pages"] + 7
    _run_static(dc, out, None)
    code, words = binding.fp2_read_status(dc.plan, None, raise_on_error=False)
    assert code == 1 and (words[2] & 2) and words[0] == 0, (code, words)
    dc.page_table.copy_(good)
    _run_static(dc, out, None)
    code, words = binding.fp2_read_status(dc.plan, None, raise_on_error=False)
    assert code == 0 and not any(words)
    assert torch.isfinite(out.float()).all()


def test_static_scratch_rejects_plans_beyond_its_capacity():
    # 33 KV heads exceed the 32 the built-in scratch is sized for: refused on the host, nothing is launched
    prm = dict(num_seqs=1, total_q=256, num_q_heads=33, num_kv_heads=33, head_dim=128, block_size=128,
               tile_rows=128, page_size=64, num_pages=8, max_pages_per_seq=4, sink_tokens=256, window_tokens=512,
               use_correction=1, alpha=0.1, softmax_scale=0.0, dtype=0)
    plan = binding.Plan(prm, [0, 256], [256])
    t = torch.zeros(256 * 33 * 128, dtype=torch.bfloat16, device="cuda")
    pt = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.Fp2Error) as e:
        binding.fp2_dense_prefill_static(plan, t, t, t, pt, pt, pt, None, None, None, t, None)
    assert e.value.code == 3
    plan.close()
