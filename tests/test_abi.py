"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, validates arguments on
the host, and its planner agrees with the oracle's geometry.  No kernel is launched here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import fp2_oracle as O
from paper_2608_19758_b200 import binding, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fp2.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fp2_[a-z_0-9]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_symbols()
    assert "fp2_select_blocks" in names and "fp2_sparse_prefill" in names and "fp2_dense_prefill" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_status_strings():
    assert binding.fp2_status_string(0) == "ok"
    assert "wait" in binding.fp2_status_string(5)


def base_params(**kw):
    p = dict(num_seqs=1, total_q=300, num_q_heads=8, num_kv_heads=2, head_dim=128, block_size=128, tile_rows=128,
             page_size=16, num_pages=64, max_pages_per_seq=32, sink_tokens=256, window_tokens=512,
             use_correction=1, alpha=0.1, softmax_scale=0.0, dtype=0)
    p.update(kw)
    return p


@pytest.mark.parametrize("kw,cu,lk,code", [
    (dict(head_dim=64), [0, 300], [400], 2),
    (dict(block_size=64), [0, 300], [400], 2),
    (dict(page_size=48), [0, 300], [400], 2),
    (dict(dtype=7), [0, 300], [400], 2),
    (dict(num_q_heads=7), [0, 300], [400], 1),
    (dict(), [0, 300], [200], 1),                 # Lq > Lk
    (dict(), [0, 299], [400], 1),                 # sum Lq != total_q
    (dict(), [0, 300], [16 * 32 + 1], 1),         # more pages than max_pages_per_seq
    (dict(max_pages_per_seq=1 << 20, num_pages=1 << 20), [0, 300], [128 * 4096 + 1], 3),   # over compiled capacity
    (dict(alpha=float("nan")), [0, 300], [400], 1),
])
def test_plan_rejects_bad_arguments_on_the_host(kw, cu, lk, code):
    with pytest.raises(binding.Fp2Error) as e:
        binding.Plan(base_params(**kw), cu, lk)
    assert e.value.code == code


def test_null_pointers_are_rejected():
    lib = binding.load()
    assert lib.fp2_plan_create(None, None, None, None) == 1
    assert lib.fp2_plan_sizes(None, None, None, None) == 1
    assert lib.fp2_select_blocks(None, *([None] * 14)) == 1
    assert lib.fp2_dense_prefill(None, *([None] * 13)) == 1
    assert lib.fp2_sparse_prefill(None, *([None] * 15), 0, None) == 1
    lib.fp2_plan_destroy(None)


@pytest.mark.parametrize("spec", [
    inputs.config_spec(1), inputs.config_spec(2), inputs.config_spec(4, scale_down=8), inputs.config_spec(5),
    inputs.small_spec(seqs=[(777, 123), (129, 128), (5, 0)], num_q_heads=14, num_kv_heads=2, page_size=8),
])
def test_planner_matches_oracle_geometry(spec):
    cu = np.concatenate([[0], np.cumsum([lk - pre for lk, pre in spec.seqs])]).astype(np.int64)
    lk = [s[0] for s in spec.seqs]
    need = max(-(-x // spec.page_size) for x in lk)
    prm = base_params(num_seqs=len(lk), total_q=int(cu[-1]), num_q_heads=spec.num_q_heads,
                      num_kv_heads=spec.num_kv_heads, page_size=spec.page_size, num_pages=1 << 20,
                      max_pages_per_seq=need)
    plan = binding.Plan(prm, cu.tolist(), lk)
    segs = O.segments(O.Params.from_dict(prm), cu, lk)
    assert plan.num_segments == len(segs)
    assert plan.idx_capacity == sum(s.J_hi + 1 for s in segs)
    assert plan.workspace_bytes % 1024 == 0 and plan.workspace_bytes > 0
    rng = np.random.default_rng(0)
    probe = set(rng.integers(0, len(segs), size=min(300, len(segs))).tolist()) | {0, len(segs) - 1}
    off = np.concatenate([[0], np.cumsum([s.J_hi + 1 for s in segs])])
    blk_off = np.concatenate([[0], np.cumsum([-(-x // 128) for x in lk])])
    for i in probe:
        s, d = segs[i], plan.segment(i)
        assert (d["b"], d["h"], d["t"], d["r0"], d["nrows"], d["pre"], d["J_lo"], d["J_hi"]) == \
               (s.b, s.h, s.t, s.r0, s.r1 - s.r0, s.pre, s.J_lo, s.J_hi)
        assert d["off"] == off[i] and d["Lk"] == lk[s.b] and d["blk_off"] == blk_off[s.b]
    plan.close()


def test_stage_calls_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    plan = binding.Plan(base_params(), [0, 300], [400])
    lib = binding.load()
    dummy = C.c_void_p(1024)
    code = lib.fp2_dense_prefill(plan.handle, dummy, dummy, dummy, dummy, dummy, dummy, None, None, None, dummy,
                                 None, dummy, None)
    assert code == 4            # FP2_ERR_CUDA: no kernel ran, nothing fell back to the CPU
    plan.close()


def test_pool_carry_count_is_host_only_and_counts_complete_blocks():
    """Blocks carried between chunks = blocks complete in both (floor(min(Lk) / 128)); needs no device."""
    from paper_2608_19758_b200 import binding
    def plan(seqs):
        prm = dict(num_seqs=len(seqs), total_q=sum(l - p for l, p in seqs), num_q_heads=4, num_kv_heads=2, head_dim=128,
                   block_size=128, tile_rows=128, page_size=16, num_pages=4096, max_pages_per_seq=1024,
                   sink_tokens=256, window_tokens=512, use_correction=1, alpha=0.1, softmax_scale=0.0, dtype=0)
        cu = [0]
        for l, p in seqs:
            cu.append(cu[-1] + l - p)
        return binding.Plan(prm, cu, [l for l, _ in seqs])
    src = plan([(1000, 0), (300, 0), (128, 0)])
    dst = plan([(1500, 1000), (4000, 0), (700, 300), (129, 128)])
    assert binding.fp2_pool_carry_count(dst, src, [0, -1, 1, 2]) == [7, 0, 2, 1]
    with pytest.raises(binding.Fp2Error):
        binding.fp2_pool_carry_count(dst, src, [5, -1, 1, 2])          # no such source sequence
