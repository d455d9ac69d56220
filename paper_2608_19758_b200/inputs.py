"""Seeded synthetic inputs for the block-sparse prefill path.

This module only *draws* inputs (queries, a paged KV cache, page tables, lengths, FP8
scales).  It holds none of the method's arithmetic: no pooling, scoring, thresholding or
attention happens here, so both the CUDA path and the CPU oracle can be fed from it.

The inputs stand in for long-context "needle in a haystack" activations (Sec. 4.1 setup:
B = 128, 256 sink tokens, 512-token window, alpha = 0.1): every (sequence, KV head) carries

* a *locality* signal  a * u(pos)  added to queries and keys, where each of the 128
  components of u is a sum of 8 sinusoids whose periods (256..4096 tokens, log-uniform)
  are shared by all components and whose phases are drawn per component, so that the
  q.k logit has a Toeplitz ("slash") structure with a local peak;
* an *attention sink*: keys at absolute positions 0..3 get  +4 * w  and every query gets
  +0.5 * w, for one Gaussian direction w with ||w|| = sqrt(d);
* optional *vertical* keys: a few key positions per head get  +3 * w.

All values are rounded once to BF16 (or quantised once to FP8 e4m3 with per-head scales);
those bits are what every consumer reads.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

SEED_BASE = 20260819
HEAD_DIM = 128
E4M3_MAX = 448.0


@dataclass
class CaseSpec:
    """Shape of one synthetic workload (one call of the hot path)."""

    name: str
    config_id: int                      # enters the seed
    seqs: List[Tuple[int, int]]         # per sequence: (Lk total KV tokens, pre cached prefix)
    num_q_heads: int
    num_kv_heads: int
    page_size: int
    dtype: str = "bf16"                 # "bf16" | "fp8"
    shuffle_pages: bool = True
    spare_page_frac: float = 0.0        # extra unused pages in the pool
    n_vertical: int = 16
    sink: bool = True
    locality_a: float = 1.5
    block_size: int = 128
    tile_rows: int = 128
    sink_tokens: int = 256
    window_tokens: int = 512
    alpha: float = 0.1
    use_correction: int = 1
    head_dim: int = HEAD_DIM
    kv_head_offset: int = 0             # this workload holds KV heads [offset, offset + num_kv_heads) of a larger one
                                        # (enters the per-head seeds only: a head-sharded rank draws its own heads)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads


@dataclass
class Case:
    """Concrete tensors of one workload (all on the CPU; callers move them)."""

    spec: CaseSpec
    q: torch.Tensor                     # [total_q, Hq, d]  bf16, or uint8 (e4m3 bits)
    k_cache: torch.Tensor               # [num_pages, p, Hkv, d]
    v_cache: torch.Tensor
    page_table: torch.Tensor            # int32 [ns, max_pages_per_seq]; unused entries = -1
    cu_seqlens_q: torch.Tensor          # int32 [ns+1]
    seqlens_k: torch.Tensor             # int32 [ns]
    q_scale: Optional[torch.Tensor] = None   # fp32 [Hq]   (fp8 only)
    k_scale: Optional[torch.Tensor] = None   # fp32 [Hkv]
    v_scale: Optional[torch.Tensor] = None   # fp32 [Hkv]
    meta: dict = field(default_factory=dict)

    @property
    def num_pages(self) -> int:
        return int(self.k_cache.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.q.shape[0])

    def params(self) -> dict:
        s = self.spec
        return dict(
            num_seqs=len(s.seqs), total_q=self.total_q, num_q_heads=s.num_q_heads,
            num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, block_size=s.block_size,
            tile_rows=s.tile_rows, page_size=s.page_size, num_pages=self.num_pages,
            max_pages_per_seq=int(self.page_table.shape[1]), sink_tokens=s.sink_tokens,
            window_tokens=s.window_tokens, use_correction=s.use_correction, alpha=s.alpha,
            softmax_scale=0.0, dtype=0 if s.dtype == "bf16" else 1)


# --------------------------------------------------------------------------------------
# bit-level views handed to consumers that do not speak torch dtypes
# --------------------------------------------------------------------------------------

def as_bits(t: torch.Tensor) -> np.ndarray:
    """BF16 tensor -> uint16 array of its bit patterns; uint8 (e4m3 bits) passes through."""
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.uint8:
        return t.contiguous().numpy()
    raise TypeError(f"unsupported dtype {t.dtype}")


def _np_or_none(t):
    return None if t is None else t.numpy()


def oracle_args(case: Case) -> dict:
    """Keyword arguments (plain numpy) describing `case` for a CPU consumer."""
    return dict(
        q_bits=as_bits(case.q), k_bits=as_bits(case.k_cache), v_bits=as_bits(case.v_cache),
        page_table=case.page_table.numpy(), cu_seqlens_q=case.cu_seqlens_q.numpy(),
        seqlens_k=case.seqlens_k.numpy(), q_scale=_np_or_none(case.q_scale),
        k_scale=_np_or_none(case.k_scale), v_scale=_np_or_none(case.v_scale))


# --------------------------------------------------------------------------------------
# drawing
# --------------------------------------------------------------------------------------

def _locality_features(pos: torch.Tensor, periods: torch.Tensor, phases: torch.Tensor) -> torch.Tensor:
    """u[pos, c] = 8^-1/2 * sum_m cos(2 pi pos / T_m + phi[c, m]); fp32 [len(pos), d]."""
    ang = (2.0 * math.pi) * pos.to(torch.float64)[:, None] / periods.to(torch.float64)[None, :]
    c, s = torch.cos(ang), torch.sin(ang)                              # [n, 8]
    cp, sp = torch.cos(phases.to(torch.float64)), torch.sin(phases.to(torch.float64))   # [d, 8]
    u = (c @ cp.T - s @ sp.T) / math.sqrt(periods.numel())
    return u.to(torch.float32)


def _draw_seq_head(spec: CaseSpec, seq: int, kv_head: int, Lk: int, pre: int):
    """Float32 q [Lq, g, d], k [Lk, d], v [Lk, d] of one (sequence, KV head)."""
    d, g = spec.head_dim, spec.group
    Lq = Lk - pre
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED_BASE + 1000 * spec.config_id + 17 * seq + kv_head)
    periods = torch.exp(torch.rand(8, generator=gen, dtype=torch.float64)
                        * (math.log(4096.0) - math.log(256.0)) + math.log(256.0))
    phases = torch.rand(d, 8, generator=gen, dtype=torch.float64) * (2.0 * math.pi)
    w = torch.randn(d, generator=gen, dtype=torch.float64)
    w = (w / w.norm() * math.sqrt(d)).to(torch.float32)
    vert = torch.randint(0, max(Lk, 1), (max(spec.n_vertical, 1),), generator=gen)
    k = torch.randn(Lk, d, generator=gen, dtype=torch.float32)
    v = torch.randn(Lk, d, generator=gen, dtype=torch.float32)
    q = torch.randn(Lq, g, d, generator=gen, dtype=torch.float32)
    if spec.locality_a != 0.0:
        u = _locality_features(torch.arange(Lk), periods, phases)
        k += spec.locality_a * u
        q += spec.locality_a * u[pre:, None, :]
    if spec.sink:
        k[: min(4, Lk)] += 4.0 * w
        q += 0.5 * w
    if spec.n_vertical > 0:
        k[vert.unique()] += 3.0 * w
    return q, k, v


def _page_layout(spec: CaseSpec):
    """Page ids for every sequence: list of int64 tensors, and the pool size."""
    p = spec.page_size
    need = [-(-Lk // p) for Lk, _ in spec.seqs]
    total = sum(need)
    pool = total + int(math.ceil(total * spec.spare_page_frac))
    if spec.shuffle_pages:
        gen = torch.Generator(device="cpu")
        gen.manual_seed(SEED_BASE + 1000 * spec.config_id + 999)
        ids = torch.randperm(pool, generator=gen)[:total]
    else:
        ids = torch.arange(total)
    out, o = [], 0
    for n in need:
        out.append(ids[o:o + n].clone())
        o += n
    return out, pool


def quantize_e4m3(x: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
    """Round x/scale to FP8 e4m3 (nearest-even, saturating at +-448); returns uint8 bits."""
    y = (x / scale).clamp_(-E4M3_MAX, E4M3_MAX)
    return y.to(torch.float8_e4m3fn).view(torch.uint8)


def make_case(spec: CaseSpec) -> Case:
    d, Hq, Hkv, g, p = spec.head_dim, spec.num_q_heads, spec.num_kv_heads, spec.group, spec.page_size
    assert Hq % Hkv == 0 and spec.block_size % p == 0
    ns = len(spec.seqs)
    pages, pool = _page_layout(spec)
    max_pages = max(int(x.numel()) for x in pages)
    page_table = torch.full((ns, max_pages), -1, dtype=torch.int32)
    for b, ids in enumerate(pages):
        page_table[b, : ids.numel()] = ids.to(torch.int32)
    lq = [Lk - pre for Lk, pre in spec.seqs]
    cu = torch.zeros(ns + 1, dtype=torch.int32)
    cu[1:] = torch.tensor(lq, dtype=torch.int32).cumsum(0)
    total_q = int(cu[-1])
    seqlens_k = torch.tensor([Lk for Lk, _ in spec.seqs], dtype=torch.int32)

    fp8 = spec.dtype == "fp8"
    store = torch.float32 if fp8 else torch.bfloat16
    qf = torch.zeros(total_q, Hq, d, dtype=store)
    kf = torch.zeros(pool * p, Hkv, d, dtype=store)
    vf = torch.zeros(pool * p, Hkv, d, dtype=store)
    for b, (Lk, pre) in enumerate(spec.seqs):
        tok = torch.arange(Lk)
        slots = pages[b][tok // p] * p + tok % p
        for h in range(Hkv):
            q, k, v = _draw_seq_head(spec, b, h + spec.kv_head_offset, Lk, pre)
            qf[int(cu[b]):int(cu[b + 1]), h * g:(h + 1) * g] = q.to(store)
            kf[slots, h] = k.to(store)
            vf[slots, h] = v.to(store)
    case_kw = {}
    if fp8:
        q_scale = (qf.abs().amax(dim=(0, 2)) / E4M3_MAX).clamp_min(1e-12).to(torch.float32)
        k_scale = (kf.abs().amax(dim=(0, 2)) / E4M3_MAX).clamp_min(1e-12).to(torch.float32)
        v_scale = (vf.abs().amax(dim=(0, 2)) / E4M3_MAX).clamp_min(1e-12).to(torch.float32)
        qf = quantize_e4m3(qf, q_scale[None, :, None])
        kf = quantize_e4m3(kf, k_scale[None, :, None])
        vf = quantize_e4m3(vf, v_scale[None, :, None])
        case_kw = dict(q_scale=q_scale, k_scale=k_scale, v_scale=v_scale)
    return Case(spec=spec, q=qf.contiguous(), k_cache=kf.view(pool, p, Hkv, d).contiguous(),
                v_cache=vf.view(pool, p, Hkv, d).contiguous(), page_table=page_table,
                cu_seqlens_q=cu, seqlens_k=seqlens_k, **case_kw)


# --------------------------------------------------------------------------------------
# the five named workloads, and scaled-down relatives for parity tests
# --------------------------------------------------------------------------------------

def _c5_lengths(ns: int = 16, total: int = 262144, lo: int = 1024, hi: int = 65536, config_id: int = 5):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED_BASE + 1000 * config_id + 998)
    ln = torch.rand(ns, generator=gen, dtype=torch.float64) * (math.log(hi) - math.log(lo)) + math.log(lo)
    L = torch.exp(ln)
    L = torch.clamp((L * (total / L.sum())).round(), lo, hi).to(torch.int64)
    frac = torch.rand(ns, generator=gen, dtype=torch.float64) * 0.75
    pre = torch.floor(L.to(torch.float64) * frac).to(torch.int64)
    return [(int(a), int(b)) for a, b in zip(L, pre)]


def config_spec(i: int, dtype: Optional[str] = None, scale_down: int = 1) -> CaseSpec:
    """Workload `i` (1..5).  `scale_down` divides the sequence lengths (parity-test relatives)."""
    if i == 1:
        return CaseSpec("C1", 1, [(2048 // scale_down, 0)], 4, 1, 128, "bf16", shuffle_pages=False,
                        n_vertical=0)
    if i == 2:
        return CaseSpec("C2", 2, [(32768 // scale_down, 0)], 32, 8, 64, dtype or "bf16")
    if i == 3:
        return CaseSpec("C3", 3, [(131072 // scale_down, 0)], 32, 8, 64, dtype or "bf16")
    if i == 4:
        return CaseSpec("C4", 4, [(131072 // scale_down, 0)], 28, 4, 64, dtype or "fp8")
    if i == 5:
        seqs = _c5_lengths(total=262144 // scale_down, lo=max(64, 1024 // scale_down),
                           hi=max(256, 65536 // scale_down))
        return CaseSpec("C5", 5, seqs, 32, 8, 16, dtype or "bf16", spare_page_frac=0.10)
    raise ValueError(i)


def small_spec(name: str = "small", config_id: int = 90, seqs: Sequence[Tuple[int, int]] = ((1000, 0),),
               num_q_heads: int = 4, num_kv_heads: int = 2, page_size: int = 16, dtype: str = "bf16",
               **kw) -> CaseSpec:
    return CaseSpec(name, config_id, list(seqs), num_q_heads, num_kv_heads, page_size, dtype, **kw)
