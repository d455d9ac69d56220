"""ctypes binding of libfp2.so: argument marshalling only (every step of the path runs in the CUDA kernels).

The functions carry the names of the C ABI (include/fp2.h).  torch is used for device memory and streams.
There is no CPU fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

FP2_OK = 0
STATUS_NAMES = {0: "FP2_OK", 1: "FP2_ERR_INVALID_ARG", 2: "FP2_ERR_UNSUPPORTED", 3: "FP2_ERR_CAPACITY",
                4: "FP2_ERR_CUDA", 5: "FP2_ERR_TIMEOUT"}

EXPORTS = ["fp2_plan_create", "fp2_plan_sizes", "fp2_plan_destroy", "fp2_plan_segment", "fp2_select_blocks",
           "fp2_pool_blocks",
           "fp2_sparse_prefill", "fp2_dense_prefill", "fp2_dense_prefill_static", "fp2_export_csr",
           "fp2_page_table_from_token_map", "fp2_plan_set_split", "fp2_pool_carry", "fp2_pool_carry_count",
           "fp2_read_status", "fp2_selftest_bounded_wait", "fp2_last_launch_count", "fp2_status_string"]


class Fp2Error(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")
        self.code = code


class fp2_params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("num_seqs", "total_q", "num_q_heads", "num_kv_heads", "head_dim",
                                         "block_size", "tile_rows", "page_size", "num_pages", "max_pages_per_seq",
                                         "sink_tokens", "window_tokens", "use_correction")] + \
               [("alpha", C.c_float), ("softmax_scale", C.c_float), ("dtype", C.c_int32)]


_lib = None


def lib_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> C.CDLL:
    """Loads (building first if the sources are newer) the shared library; raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing and _build.needs_build():
        _build.build()
    if not os.path.exists(_build.LIB):
        raise RuntimeError("libfp2.so is missing: run `python -m paper_2608_19758_b200.build`")
    lib = C.CDLL(_build.LIB)
    vp, i32p, i64p, f32p = C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p
    lib.fp2_plan_create.argtypes = [C.POINTER(fp2_params), C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                    C.POINTER(C.c_void_p)]
    lib.fp2_plan_create.restype = C.c_int
    lib.fp2_plan_sizes.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.fp2_plan_sizes.restype = C.c_int
    lib.fp2_plan_destroy.argtypes = [C.c_void_p]
    lib.fp2_plan_destroy.restype = None
    lib.fp2_plan_segment.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    lib.fp2_plan_segment.restype = C.c_int
    lib.fp2_select_blocks.argtypes = [C.c_void_p, vp, vp, vp, i32p, i32p, i32p, f32p, f32p, f32p, i64p, i32p, i32p,
                                      vp, C.c_void_p]
    lib.fp2_select_blocks.restype = C.c_int
    lib.fp2_pool_blocks.argtypes = [C.c_void_p, vp, vp, i32p, i32p, f32p, f32p, vp, C.c_void_p]
    lib.fp2_pool_blocks.restype = C.c_int
    lib.fp2_sparse_prefill.argtypes = [C.c_void_p, vp, vp, vp, i32p, i32p, i32p, i64p, i32p, i32p, f32p, f32p, f32p,
                                       vp, f32p, vp, C.c_int32, C.c_void_p]
    lib.fp2_sparse_prefill.restype = C.c_int
    lib.fp2_dense_prefill.argtypes = [C.c_void_p, vp, vp, vp, i32p, i32p, i32p, f32p, f32p, f32p, vp, f32p, vp,
                                      C.c_void_p]
    lib.fp2_dense_prefill.restype = C.c_int
    lib.fp2_dense_prefill_static.argtypes = [C.c_void_p, vp, vp, vp, i32p, i32p, i32p, f32p, f32p, f32p, vp, f32p,
                                             C.c_void_p]
    lib.fp2_dense_prefill_static.restype = C.c_int
    lib.fp2_export_csr.argtypes = [C.c_void_p, i32p, i32p, C.c_int32, i32p, i32p, C.c_int64, vp, C.c_void_p]
    lib.fp2_export_csr.restype = C.c_int
    lib.fp2_page_table_from_token_map.argtypes = [C.c_void_p, i32p, C.c_int32, i32p, i32p, vp, C.c_void_p]
    lib.fp2_page_table_from_token_map.restype = C.c_int
    lib.fp2_pool_carry.argtypes = [C.c_void_p, vp, C.c_void_p, vp, C.POINTER(C.c_int32), C.c_void_p]
    lib.fp2_pool_carry.restype = C.c_int
    lib.fp2_pool_carry_count.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.fp2_pool_carry_count.restype = C.c_int
    lib.fp2_plan_set_split.argtypes = [C.c_void_p, C.c_int32]
    lib.fp2_plan_set_split.restype = C.c_int
    lib.fp2_selftest_bounded_wait.argtypes = [C.c_void_p, vp, C.c_void_p]
    lib.fp2_selftest_bounded_wait.restype = C.c_int
    lib.fp2_read_status.argtypes = [C.c_void_p, vp, C.POINTER(C.c_int32), C.c_void_p]
    lib.fp2_read_status.restype = C.c_int
    lib.fp2_last_launch_count.argtypes = [C.c_void_p]
    lib.fp2_last_launch_count.restype = C.c_int32
    lib.fp2_status_string.argtypes = [C.c_int]
    lib.fp2_status_string.restype = C.c_char_p
    _lib = lib
    return lib


def _check(code: int, where: str):
    if code != FP2_OK:
        raise Fp2Error(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def fp2_status_string(code: int) -> str:
    return load().fp2_status_string(code).decode()


class Plan:
    """Owner of an fp2_plan handle (host-side metadata + one small device table)."""

    def __init__(self, params: dict, h_cu_seqlens_q, h_seqlens_k):
        lib = load()
        self.params = fp2_params(**params)
        ns = int(params["num_seqs"])
        cu = (C.c_int32 * (ns + 1))(*[int(x) for x in h_cu_seqlens_q])
        lk = (C.c_int32 * ns)(*[int(x) for x in h_seqlens_k])
        h = C.c_void_p()
        _check(lib.fp2_plan_create(C.byref(self.params), cu, lk, C.byref(h)), "fp2_plan_create")
        self.handle = h
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        _check(lib.fp2_plan_sizes(h, C.byref(a), C.byref(b), C.byref(c)), "fp2_plan_sizes")
        self.num_segments, self.idx_capacity, self.workspace_bytes = a.value, b.value, c.value

    def segment(self, seg: int) -> dict:
        out = (C.c_int32 * 10)()
        off = C.c_int64()
        _check(load().fp2_plan_segment(self.handle, seg, out, C.byref(off)), "fp2_plan_segment")
        keys = ("b", "h", "t", "r0", "nrows", "pre", "Lk", "J_lo", "J_hi", "blk_off")
        d = dict(zip(keys, list(out)))
        d["off"] = off.value
        return d

    def set_split(self, target: int):
        """KV splitting (Eq. 18): < 0 off, 0 automatic, > 0 requested iterations per part."""
        _check(load().fp2_plan_set_split(self.handle, target), "fp2_plan_set_split")

    def last_launch_count(self) -> int:
        return int(load().fp2_last_launch_count(self.handle))

    def new_workspace(self, device="cuda") -> torch.Tensor:
        """Zeroed device workspace (torch's allocator returns 512-byte aligned blocks; 1024 is required,
        so over-allocate and slice)."""
        raw = torch.zeros(self.workspace_bytes + 1024, dtype=torch.uint8, device=device)
        shift = (-raw.data_ptr()) % 1024
        ws = raw[shift:shift + self.workspace_bytes]
        ws._fp2_keepalive = raw
        return ws

    def new_lists(self, device="cuda"):
        seg_offset = torch.zeros(self.num_segments + 1, dtype=torch.int64, device=device)
        seg_count = torch.zeros(max(self.num_segments, 1), dtype=torch.int32, device=device)
        blk_idx = torch.zeros(max(self.idx_capacity, 1), dtype=torch.int32, device=device)
        return seg_offset, seg_count, blk_idx

    def close(self):
        if getattr(self, "handle", None):
            load().fp2_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def fp2_select_blocks(plan: Plan, q, k_cache, v_cache, page_table, cu_seqlens_q, seqlens_k, q_scale, k_scale,
                      v_scale, seg_offset, seg_count, blk_idx, workspace, stream=None):
    _check(load().fp2_select_blocks(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(page_table),
                                    _ptr(cu_seqlens_q), _ptr(seqlens_k), _ptr(q_scale), _ptr(k_scale),
                                    _ptr(v_scale), _ptr(seg_offset), _ptr(seg_count), _ptr(blk_idx),
                                    _ptr(workspace), _stream(stream)), "fp2_select_blocks")


def fp2_pool_blocks(plan: Plan, k_cache, v_cache, page_table, seqlens_k, k_scale, v_scale, workspace, stream=None):
    """Block-mean pooling alone: the pooled statistics of `workspace` are refreshed, no list is written."""
    _check(load().fp2_pool_blocks(plan.handle, _ptr(k_cache), _ptr(v_cache), _ptr(page_table), _ptr(seqlens_k),
                                  _ptr(k_scale), _ptr(v_scale), _ptr(workspace), _stream(stream)), "fp2_pool_blocks")


def fp2_sparse_prefill(plan: Plan, q, k_cache, v_cache, page_table, cu_seqlens_q, seqlens_k, seg_offset, seg_count,
                       blk_idx, q_scale, k_scale, v_scale, out, lse, workspace, pooled_valid: bool = True,
                       stream=None):
    _check(load().fp2_sparse_prefill(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(page_table),
                                     _ptr(cu_seqlens_q), _ptr(seqlens_k), _ptr(seg_offset), _ptr(seg_count),
                                     _ptr(blk_idx), _ptr(q_scale), _ptr(k_scale), _ptr(v_scale), _ptr(out),
                                     _ptr(lse), _ptr(workspace), 1 if pooled_valid else 0, _stream(stream)),
           "fp2_sparse_prefill")


def fp2_dense_prefill(plan: Plan, q, k_cache, v_cache, page_table, cu_seqlens_q, seqlens_k, q_scale, k_scale,
                      v_scale, out, lse, workspace, stream=None):
    _check(load().fp2_dense_prefill(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(page_table),
                                    _ptr(cu_seqlens_q), _ptr(seqlens_k), _ptr(q_scale), _ptr(k_scale),
                                    _ptr(v_scale), _ptr(out), _ptr(lse), _ptr(workspace), _stream(stream)),
           "fp2_dense_prefill")


def fp2_dense_prefill_static(plan: Plan, q, k_cache, v_cache, page_table, cu_seqlens_q, seqlens_k, q_scale, k_scale,
                             v_scale, out, lse, stream=None):
    """Dense prefill without a caller workspace: the library's built-in device scratch is used."""
    _check(load().fp2_dense_prefill_static(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(page_table),
                                           _ptr(cu_seqlens_q), _ptr(seqlens_k), _ptr(q_scale), _ptr(k_scale),
                                           _ptr(v_scale), _ptr(out), _ptr(lse), _stream(stream)),
           "fp2_dense_prefill_static")


def fp2_export_csr(plan: Plan, seg_count, blk_idx, tile_tokens: int, cu, idx, workspace, stream=None):
    """Compact CSR of physical tiles (cu int32 [nseg + 1], idx int32) from the padded block lists."""
    _check(load().fp2_export_csr(plan.handle, _ptr(seg_count), _ptr(blk_idx), tile_tokens, _ptr(cu), _ptr(idx),
                                 idx.numel(), _ptr(workspace), _stream(stream)), "fp2_export_csr")


def fp2_page_table_from_token_map(plan: Plan, token_to_slot, seqlens_k, page_table, workspace, stream=None):
    """Page-level table [num_seqs, max_pages_per_seq] from a token-level slot map [num_seqs, max_tokens]."""
    _check(load().fp2_page_table_from_token_map(plan.handle, _ptr(token_to_slot), token_to_slot.shape[1],
                                                _ptr(seqlens_k), _ptr(page_table), _ptr(workspace),
                                                _stream(stream)), "fp2_page_table_from_token_map")


def fp2_pool_carry_count(dst: Plan, src: Plan, src_seq):
    """Blocks per sequence of `dst` whose pooled means would be carried over from `src` (host only)."""
    ns = len(src_seq)
    a = (C.c_int32 * max(ns, 1))(*src_seq)
    out = (C.c_int32 * max(ns, 1))()
    _check(load().fp2_pool_carry_count(dst.handle, src.handle, a, out), "fp2_pool_carry_count")
    return list(out)[:ns]


def fp2_pool_carry(dst: Plan, dst_workspace, src: Plan, src_workspace, src_seq, stream=None):
    """Copies the pooled means of the blocks complete in both chunks from src_workspace to dst_workspace; the next
    fp2_select_blocks on `dst` pools only the rest."""
    a = (C.c_int32 * max(len(src_seq), 1))(*src_seq)
    _check(load().fp2_pool_carry(dst.handle, _ptr(dst_workspace), src.handle, _ptr(src_workspace), a,
                                 _stream(stream)), "fp2_pool_carry")


def fp2_selftest_bounded_wait(plan: Plan, workspace, stream=None):
    """Launches the library's bounded-wait probe: a wait that runs out, recorded in the status block of `workspace`."""
    _check(load().fp2_selftest_bounded_wait(plan.handle, _ptr(workspace), _stream(stream)), "fp2_selftest_bounded_wait")


def fp2_read_status(plan: Plan, workspace, stream=None, raise_on_error: bool = True):
    words = (C.c_int32 * 8)()
    code = load().fp2_read_status(plan.handle, _ptr(workspace), words, _stream(stream))
    if raise_on_error:
        _check(code, f"fp2_read_status words={list(words)}")
    return code, list(words)


class DeviceCase:
    """A workload's tensors moved to the GPU, with a plan, workspace and list buffers (test / bench helper)."""

    def __init__(self, case, device="cuda", **param_overrides):
        self.case = case
        prm = case.params()
        prm.update(param_overrides)
        self.prm = prm
        self.plan = Plan(prm, case.cu_seqlens_q.tolist(), case.seqlens_k.tolist())
        dev = torch.device(device)
        self.q = case.q.to(dev)
        self.k_cache = case.k_cache.to(dev)
        self.v_cache = case.v_cache.to(dev)
        self.page_table = case.page_table.to(dev)
        self.cu_seqlens_q = case.cu_seqlens_q.to(dev)
        self.seqlens_k = case.seqlens_k.to(dev)
        self.q_scale = None if case.q_scale is None else case.q_scale.to(dev)
        self.k_scale = None if case.k_scale is None else case.k_scale.to(dev)
        self.v_scale = None if case.v_scale is None else case.v_scale.to(dev)
        self.workspace = self.plan.new_workspace(dev)
        self.seg_offset, self.seg_count, self.blk_idx = self.plan.new_lists(dev)
        self.out = torch.empty(case.total_q, prm["num_q_heads"], prm["head_dim"], dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty(prm["num_q_heads"], case.total_q, dtype=torch.float32, device=dev)
        # Tests set this: every stage call then first overwrites the buffers it is about to fill (lists with -1,
        # outputs with NaN), so that a row or an entry the call fails to write cannot pass on an earlier call's values.
        self.poison = False

    def _poison_lists(self):
        if self.poison:
            self.seg_count.fill_(-1)
            self.blk_idx.fill_(-1)

    def _poison_outputs(self):
        if self.poison:
            self.out.fill_(float("nan"))
            self.lse.fill_(float("nan"))

    def select(self):
        self._poison_lists()
        fp2_select_blocks(self.plan, self.q, self.k_cache, self.v_cache, self.page_table, self.cu_seqlens_q,
                          self.seqlens_k, self.q_scale, self.k_scale, self.v_scale, self.seg_offset, self.seg_count,
                          self.blk_idx, self.workspace)

    def pool(self):
        fp2_pool_blocks(self.plan, self.k_cache, self.v_cache, self.page_table, self.seqlens_k, self.k_scale,
                        self.v_scale, self.workspace)

    def sparse(self, pooled_valid=True, seg_count=None, blk_idx=None):
        self._poison_outputs()
        fp2_sparse_prefill(self.plan, self.q, self.k_cache, self.v_cache, self.page_table, self.cu_seqlens_q,
                           self.seqlens_k, self.seg_offset, self.seg_count if seg_count is None else seg_count,
                           self.blk_idx if blk_idx is None else blk_idx, self.q_scale, self.k_scale, self.v_scale,
                           self.out, self.lse, self.workspace, pooled_valid)

    def dense(self):
        self._poison_outputs()
        fp2_dense_prefill(self.plan, self.q, self.k_cache, self.v_cache, self.page_table, self.cu_seqlens_q,
                          self.seqlens_k, self.q_scale, self.k_scale, self.v_scale, self.out, self.lse,
                          self.workspace)

    def export_csr(self, tile_tokens=64):
        """(cu, idx) device tensors of the lists currently in the buffers."""
        cu = torch.empty(self.plan.num_segments + 1, dtype=torch.int32, device=self.q.device)
        idx = torch.empty(max(self.plan.idx_capacity * (128 // tile_tokens), 1), dtype=torch.int32, device=self.q.device)
        fp2_export_csr(self.plan, self.seg_count, self.blk_idx, tile_tokens, cu, idx, self.workspace)
        return cu, idx

    def status(self, raise_on_error=True):
        return fp2_read_status(self.plan, self.workspace, raise_on_error=raise_on_error)

    def lists_host(self):
        """{seg: ascending int32 array} of the lists currently in the buffers."""
        off = self.seg_offset.cpu().numpy()
        cnt = self.seg_count.cpu().numpy()
        idx = self.blk_idx.cpu().numpy()
        return {s: idx[off[s]:off[s] + cnt[s]].copy() for s in range(self.plan.num_segments)}
