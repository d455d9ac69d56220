"""CPU oracle for the block-sparse prefill path -- TEST INFRASTRUCTURE, not the product.

A plain, slow, fp64 restatement of what the path computes, written from the paper:
block-mean pooling (Eq. 5), block energies (Eq. 19), max-based threshold with forced
sink / window / diagonal blocks (Eq. 3, Eq. 20), and block-sparse causal attention with
the mean-correction term (Eq. 4, Eq. 6) over a paged KV cache (Eq. 22) with PackGQA row
packing (Eq. 13).  It shares no code with the CUDA path and is imported only by the tests,
the smoke check and the benchmark's CPU-baseline leg.

Inputs are the exact bit patterns the GPU reads: BF16 as uint16, FP8 e4m3 as uint8 with
per-head fp32 scales; they are widened to fp64 here and everything after is fp64.
Library steps used: numpy matmul / exp / max.  No blocking or fusion beyond the paper's
definitions: every tile is handled whole, every softmax is evaluated with one max shift.

Readings of the paper taken here (each is a choice where the text is silent or has two
forms):
  * logits carry 1/sqrt(d) everywhere, as Eq. 19 writes them (Eq. 1 omits the factor);
  * a query tile is `tile_rows` consecutive *packed* rows of one KV head (Eq. 13), and all
    rows of the tile enter the block energy (Eq. 19 sums over q_i in I);
  * candidates of a tile are the blocks 0..J_hi with J_hi the block of the tile's last row;
    the energy carries no per-row causal mask and the max in Eq. 20 runs over all
    candidates, forced ones included;
  * "sink" = blocks below ceil(sink_tokens/B); "window" = blocks at or above
    J_lo - ceil(window_tokens/B), which contains the diagonal band J_lo..J_hi
    ("most recent" and "diag" name the same blocks);
  * only blocks J < J_lo (entirely visible to every row of the tile) may be corrected
    (Sec. 3.2, implementation paragraph); they are always full, so |B_J| = B there;
  * comparison is ">=": equality selects;
  * LSE is the natural log of the corrected denominator, softmax scale included.

Index export (Algorithm 1 line 5; Sec. 3.3 "Index-Driven Sparse Traversal", Eq. 17; Sec. 3.4
"Serving Integration"): the block lists as a compact CSR of physical tiles, and the
page-level table taken from a token-level slot map by striding.  Readings: a logical block
expands to the physical tiles that hold at least one real token of it (B / tile_tokens of
them except in a ragged last block); `cu` is the running count in segment order.

KV splitting (Eq. 18; Sec. 3.3 "Sparsity-Aware Load Balancing"): the iteration sequence of a
segment -- its list backwards (Eq. 17), then its correction terms -- cut into U contiguous
parts of ceil(n / U) iterations, each part reduced to (O_u, LSE_u) on its own, the parts merged
by their log-sum-exp weights.  Reading: a correction term belongs to exactly one part (here:
they follow the listed blocks in the sequence).

Parity pins: every function here is pinned by tests that do not go through this file's
own formulae (dense limit against a naive loop and torch SDPA, the block-constant closed
form, brute force on tiny inputs, Eq. 1-3 against Eq. 19-20, invariants).  What is NOT
pinned, by design: how well Eq. 6 approximates full attention on real activations --
"parity unpinned" for that claim only.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

# --------------------------------------------------------------------------------------
# widening of the stored bit patterns
# --------------------------------------------------------------------------------------


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """BF16 is the upper half of an IEEE fp32 word."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _e4m3_table() -> np.ndarray:
    """Value of each of the 256 e4m3 ("fn": no infinities, 0x7f/0xff = NaN) bit patterns."""
    t = np.zeros(256, dtype=np.float64)
    for b in range(256):
        sign = -1.0 if b & 0x80 else 1.0
        e = (b >> 3) & 0xF
        m = b & 0x7
        if e == 0xF and m == 0x7:
            val = float("nan")
        elif e == 0:
            val = (m / 8.0) * 2.0 ** (-6)
        else:
            val = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[b] = sign * val
    return t


_E4M3 = _e4m3_table()


def e4m3_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return _E4M3[bits]


def widen(bits: np.ndarray, scale: Optional[np.ndarray], head_axis: int) -> np.ndarray:
    """Stored tensor -> fp64 values.  `scale` (per head, fp32) applies to FP8 only."""
    if bits.dtype == np.uint16:
        return bf16_bits_to_f64(bits)
    if bits.dtype == np.uint8:
        x = e4m3_bits_to_f64(bits)
        shape = [1] * x.ndim
        shape[head_axis] = -1
        return x * scale.astype(np.float64).reshape(shape)
    raise TypeError(bits.dtype)


def _widen_head(bits: np.ndarray, scale_h) -> np.ndarray:
    """Tokens of a single head -> fp64 (FP8 values times that head's scale)."""
    if bits.dtype == np.uint16:
        return bf16_bits_to_f64(bits)
    return e4m3_bits_to_f64(bits) * float(scale_h)


# --------------------------------------------------------------------------------------
# geometry: PackGQA tiles (Eq. 13), KV blocks, paging (Eq. 22)
# --------------------------------------------------------------------------------------


@dataclass
class Params:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int = 128
    block_size: int = 128          # B
    tile_rows: int = 128           # M, packed rows per query tile
    page_size: int = 128           # p
    sink_tokens: int = 256
    window_tokens: int = 512
    use_correction: int = 1
    alpha: float = 0.1
    softmax_scale: float = 0.0     # 0 -> 1/sqrt(d)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def scale(self) -> float:
        return self.softmax_scale if self.softmax_scale > 0 else 1.0 / math.sqrt(self.head_dim)

    @classmethod
    def from_dict(cls, d: dict) -> "Params":
        keys = cls.__dataclass_fields__.keys()
        return cls(**{k: d[k] for k in keys if k in d})


@dataclass
class Segment:
    """One (sequence b, KV head h, tile t): the unit the block lists are defined on."""

    seg: int
    b: int
    h: int
    t: int
    r0: int          # first packed row (inclusive)
    r1: int          # last packed row (exclusive)
    pre: int         # cached prefix length of the sequence
    J_lo: int        # block of the first row's absolute position
    J_hi: int        # block of the last row's absolute position


def num_tiles(p: Params, Lq: int) -> int:
    return -(-(p.group * Lq) // p.tile_rows)


def segments(p: Params, cu_seqlens_q: Sequence[int], seqlens_k: Sequence[int]) -> List[Segment]:
    """All segments in list order: seg = Hkv*tile_off[b] + h*ntiles_b + t."""
    out: List[Segment] = []
    g, M, B = p.group, p.tile_rows, p.block_size
    tile_off = 0
    for b in range(len(seqlens_k)):
        Lq = int(cu_seqlens_q[b + 1]) - int(cu_seqlens_q[b])
        Lk = int(seqlens_k[b])
        pre = Lk - Lq
        nt = num_tiles(p, Lq)
        for h in range(p.num_kv_heads):
            for t in range(nt):
                r0, r1 = t * M, min((t + 1) * M, g * Lq)
                p_lo = pre + r0 // g               # Eq. 13: pos(r) = floor(r / g)
                p_hi = pre + (r1 - 1) // g
                out.append(Segment(p.num_kv_heads * tile_off + h * nt + t, b, h, t, r0, r1, pre,
                                   p_lo // B, p_hi // B))
        tile_off += nt
    return out


def candidate_pairs(p: Params, cu_seqlens_q, seqlens_k) -> int:
    return sum(s.J_hi + 1 for s in segments(p, cu_seqlens_q, seqlens_k))


def gather_kv(cache: np.ndarray, page_table_row: np.ndarray, Lk: int, h: int, page_size: int) -> np.ndarray:
    """Tokens 0..Lk-1 of one sequence and KV head through the page table (Eq. 22)."""
    j = np.arange(Lk)
    slot = page_table_row[j // page_size].astype(np.int64) * page_size + (j % page_size)
    flat = cache.reshape(-1, cache.shape[2], cache.shape[3])
    return flat[slot, h, :]


def tile_queries(q_seq: np.ndarray, p: Params, s: Segment) -> np.ndarray:
    """Rows r0..r1-1 of the packed matrix Q' of KV head s.h (Eq. 12-13): [rows, d]."""
    r = np.arange(s.r0, s.r1)
    return q_seq[r // p.group, s.h * p.group + (r % p.group), :]


def row_positions(p: Params, s: Segment) -> np.ndarray:
    """Absolute position of each row of the tile (bottom-right aligned causal mask)."""
    return s.pre + np.arange(s.r0, s.r1) // p.group


# --------------------------------------------------------------------------------------
# Eq. 5: pooled block means
# --------------------------------------------------------------------------------------


def pooled_means(x: np.ndarray, B: int) -> np.ndarray:
    """Mean over the real tokens of every block of `B` tokens: [ceil(L/B), d]."""
    L = x.shape[0]
    nblk = -(-L // B)
    out = np.empty((nblk, x.shape[1]), dtype=np.float64)
    for J in range(nblk):
        out[J] = x[J * B:min((J + 1) * B, L)].mean(axis=0)
    return out


def block_token_counts(L: int, B: int) -> np.ndarray:
    nblk = -(-L // B)
    return np.array([min((J + 1) * B, L) - J * B for J in range(nblk)], dtype=np.int64)


# --------------------------------------------------------------------------------------
# Eq. 19: block energies; Eq. 20 / Eq. 3: selection
# --------------------------------------------------------------------------------------


def block_energies(q_tile: np.ndarray, kbar_cand: np.ndarray, scale: float):
    """E_J = sum_{i in I} exp(s_iJ - M),  s_iJ = scale * q_i . kbar_J,  M = max_{i,J} s_iJ."""
    s = scale * (q_tile @ kbar_cand.T)
    M = s.max()
    E = np.exp(s - M).sum(axis=0)
    return E, M


def forced_mask(J_lo: int, J_hi: int, B: int, sink_tokens: int, window_tokens: int) -> np.ndarray:
    J = np.arange(J_hi + 1)
    sink_blocks = -(-sink_tokens // B)
    window_blocks = -(-window_tokens // B)
    return (J < sink_blocks) | (J >= J_lo - window_blocks)


def select_blocks(E: np.ndarray, alpha: float, forced: np.ndarray):
    """Ascending selected block ids, and each candidate's relative distance to the threshold."""
    thr = alpha * E.max()
    keep = (E >= thr) | forced
    margin = np.abs(E - thr) / thr if thr > 0 else np.full_like(E, np.inf)
    return np.nonzero(keep)[0].astype(np.int32), margin


# --------------------------------------------------------------------------------------
# Eq. 4 / Eq. 6: attention over the selected blocks with mean correction
# --------------------------------------------------------------------------------------


def attend_tile(q_tile, pos, K, V, kbar, vbar, n_tok, selected, J_lo, B, scale, use_correction):
    """Rows of one tile -> (O [rows, d], LSE [rows]).

    numerator   = sum_{J in S} sum_{j in B_J, j <= pos_i} e^{s_ij} v_j + sum_{J in F \\ S} n_J e^{sbar_iJ} vbar_J
    denominator = the same with v -> 1;  F = {J < J_lo}.
    """
    Lk = K.shape[0]
    tok = np.concatenate([np.arange(J * B, min((J + 1) * B, Lk)) for J in selected]) \
        if len(selected) else np.zeros(0, dtype=np.int64)
    logits = scale * (q_tile @ K[tok].T)
    logits = np.where(tok[None, :] <= pos[:, None], logits, -np.inf)
    values = V[tok]
    if use_correction:
        sel = np.zeros(max(J_lo, 0), dtype=bool)
        s_in = np.asarray(selected)
        sel[s_in[s_in < J_lo]] = True
        corr = np.nonzero(~sel)[0]
        if corr.size:
            lbar = scale * (q_tile @ kbar[corr].T) + np.log(n_tok[corr].astype(np.float64))[None, :]
            logits = np.concatenate([logits, lbar], axis=1)
            values = np.concatenate([values, vbar[corr]], axis=0)
    m = logits.max(axis=1, keepdims=True)
    w = np.exp(logits - m)
    den = w.sum(axis=1)
    return (w @ values) / den[:, None], m[:, 0] + np.log(den)


# --------------------------------------------------------------------------------------
# whole-stage drivers over a batch
# --------------------------------------------------------------------------------------


class Workload:
    """Widened views of one batch; per-(sequence, head) gathers are cached on demand."""

    def __init__(self, params: Params, q_bits, k_bits, v_bits, page_table, cu_seqlens_q, seqlens_k,
                 q_scale=None, k_scale=None, v_scale=None):
        self.p = params
        self.q_bits, self.k_bits, self.v_bits = q_bits, k_bits, v_bits
        self.page_table = page_table
        self.cu = np.asarray(cu_seqlens_q).astype(np.int64)
        self.lk = np.asarray(seqlens_k).astype(np.int64)
        self.q_scale, self.k_scale, self.v_scale = q_scale, k_scale, v_scale
        self.segs = segments(params, self.cu, self.lk)
        self._kv = {}

    def q_seq(self, b: int) -> np.ndarray:
        return widen(self.q_bits[self.cu[b]:self.cu[b + 1]], self.q_scale, head_axis=1)

    def kv(self, b: int, h: int):
        """(K, V, kbar, vbar, n_tok) of one sequence and KV head, fp64."""
        key = (b, h)
        if key not in self._kv:
            if len(self._kv) > 4:
                self._kv.clear()
            p = self.p
            Lk = int(self.lk[b])
            K = gather_kv(self.k_bits, self.page_table[b], Lk, h, p.page_size)
            V = gather_kv(self.v_bits, self.page_table[b], Lk, h, p.page_size)
            K = _widen_head(K, None if self.k_scale is None else self.k_scale[h])
            V = _widen_head(V, None if self.v_scale is None else self.v_scale[h])
            self._kv[key] = (K, V, pooled_means(K, p.block_size), pooled_means(V, p.block_size),
                             block_token_counts(Lk, p.block_size))
        return self._kv[key]


def oracle_select(wl: Workload, seg_ids: Optional[Sequence[int]] = None):
    """Stage 1 for the given segments (default: all).

    Returns {seg: (idx int32 ascending, E float64[J_hi+1], margin float64[J_hi+1])}.
    """
    p = wl.p
    out = {}
    todo = wl.segs if seg_ids is None else [wl.segs[i] for i in seg_ids]
    qcache = {}
    for s in todo:
        if s.b not in qcache:
            qcache = {s.b: wl.q_seq(s.b)}
        _, _, kbar, _, _ = wl.kv(s.b, s.h)
        qt = tile_queries(qcache[s.b], p, s)
        E, _ = block_energies(qt, kbar[:s.J_hi + 1], p.scale)
        idx, margin = select_blocks(E, p.alpha, forced_mask(s.J_lo, s.J_hi, p.block_size,
                                                            p.sink_tokens, p.window_tokens))
        out[s.seg] = (idx, E, margin)
    return out


def oracle_attend(wl: Workload, lists, seg_ids: Optional[Sequence[int]] = None, dense: bool = False):
    """Stage 2 for the given segments.  `lists[seg]` = ascending selected block ids (ignored
    when `dense`, where every candidate block is attended exactly and nothing is corrected).

    Returns {seg: (O float64 [rows, d], LSE float64 [rows])}; row k of a segment is packed row
    r0 + k, i.e. position floor(r/g), query head h*g + r mod g.
    """
    p = wl.p
    out = {}
    todo = wl.segs if seg_ids is None else [wl.segs[i] for i in seg_ids]
    qcache = {}
    for s in todo:
        if s.b not in qcache:
            qcache = {s.b: wl.q_seq(s.b)}
        K, V, kbar, vbar, n_tok = wl.kv(s.b, s.h)
        qt = tile_queries(qcache[s.b], p, s)
        sel = np.arange(s.J_hi + 1) if dense else np.asarray(lists[s.seg])
        out[s.seg] = attend_tile(qt, row_positions(p, s), K, V, kbar, vbar, n_tok, sel, s.J_lo,
                                 p.block_size, p.scale, 0 if dense else p.use_correction)
    return out


def scatter_output(wl: Workload, results, total_q: int):
    """Segment results -> O [total_q, Hq, d] and LSE [Hq, total_q] (NaN where not computed)."""
    p = wl.p
    O = np.full((total_q, p.num_q_heads, p.head_dim), np.nan)
    L = np.full((p.num_q_heads, total_q), np.nan)
    for s in wl.segs:
        if s.seg not in results:
            continue
        o, lse = results[s.seg]
        r = np.arange(s.r0, s.r1)
        tok = wl.cu[s.b] + r // p.group
        head = s.h * p.group + r % p.group
        O[tok, head] = o
        L[head, tok] = lse
    return O, L


# ------------------------------------------------------------------------------------------
# Index export
# ------------------------------------------------------------------------------------------

def export_csr(wl: Workload, lists, tile_tokens: int = 64):
    """Algorithm 1 line 5: (cu, idx) with every listed logical block J of a segment replaced by the
    physical tiles (tile_tokens tokens each) that intersect its real tokens [J B, min((J+1) B, Lk)).
    cu: int64 [nseg + 1] (exclusive running count, Eq. 17's cu[g]); idx: int32 ascending per segment."""
    B = wl.p.block_size
    cu = [0]
    idx: List[int] = []
    for s in wl.segs:
        Lk = int(wl.lk[s.b])
        for J in lists[s.seg]:
            first, last = int(J) * B, min((int(J) + 1) * B, Lk)      # real tokens of the block
            t = first // tile_tokens
            while t * tile_tokens < last:
                idx.append(t)
                t += 1
        cu.append(len(idx))
    return np.asarray(cu, dtype=np.int64), np.asarray(idx, dtype=np.int32)


def page_table_from_token_map(token_to_slot: np.ndarray, seqlens_k: Sequence[int], page_size: int,
                              max_pages: int):
    """Sec. 3.4: the page-level table is the token-level slot map read every page_size entries.
    token_to_slot [ns, max_tokens]: global slot of token j of sequence b (Eq. 22's addr(b, j)).
    Returns (page_table int32 [ns, max_pages] with -1 past the last page, misaligned) where misaligned
    says some sampled slot was not the first slot of a page."""
    ns = len(seqlens_k)
    pt = np.full((ns, max_pages), -1, dtype=np.int32)
    misaligned = False
    for b in range(ns):
        for k in range(max_pages):
            if k * page_size >= int(seqlens_k[b]):
                break
            slot = int(token_to_slot[b, k * page_size])
            misaligned |= slot % page_size != 0
            pt[b, k] = slot // page_size
    return pt, misaligned


# ------------------------------------------------------------------------------------------
# KV splitting (Eq. 18) and the merge of partial results
# ------------------------------------------------------------------------------------------

def split_ranges(n: int, U: int):
    """Eq. 18: part u of U takes iterations [u ceil(n / U), min((u + 1) ceil(n / U), n))."""
    step = -(-n // U) if n > 0 else 0
    return [(min(u * step, n), min((u + 1) * step, n)) for u in range(U)]


def merge_partials(parts):
    """parts: [(O_u [rows, d], LSE_u [rows])], LSE_u = -inf (and O_u arbitrary) for an empty part.
    O = sum_u w_u O_u / sum_u w_u, LSE = log sum_u e^{LSE_u}, w_u = e^{LSE_u - max_u LSE_u}."""
    lse = np.stack([l for _, l in parts])                       # [U, rows]
    top = lse.max(axis=0)
    safe = np.where(np.isfinite(top), top, 0.0)
    w = np.exp(lse - safe[None, :])                             # e^{-inf} = 0 for empty parts
    den = w.sum(axis=0)
    num = sum(w[u][:, None] * np.where(np.isfinite(lse[u])[:, None], parts[u][0], 0.0) for u in range(len(parts)))
    with np.errstate(divide="ignore", invalid="ignore"):
        return num / den[:, None], safe + np.log(den)


def attend_tile_split(q_tile, pos, K, V, kbar, vbar, n_tok, selected, J_lo, B, scale, use_correction, U):
    """attend_tile evaluated part by part (Eq. 18) and merged.  The iteration sequence is the listed blocks
    in descending order (Eq. 17) followed by the corrected blocks in ascending order."""
    sel = [int(J) for J in selected][::-1]
    corr = []
    if use_correction:
        listed = set(sel)
        corr = [J for J in range(max(J_lo, 0)) if J not in listed]
    seq = [("x", J) for J in sel] + [("c", J) for J in corr]
    Lk = K.shape[0]
    parts = []
    for a, b in split_ranges(len(seq), U):
        logits, values = [], []
        for kind, J in seq[a:b]:
            if kind == "x":
                tok = np.arange(J * B, min((J + 1) * B, Lk))
                lg = scale * (q_tile @ K[tok].T)
                logits.append(np.where(tok[None, :] <= pos[:, None], lg, -np.inf))
                values.append(V[tok])
            else:
                logits.append(scale * (q_tile @ kbar[J][:, None]) + math.log(float(n_tok[J])))
                values.append(vbar[J][None, :])
        if not logits:
            parts.append((np.zeros((q_tile.shape[0], V.shape[1])), np.full(q_tile.shape[0], -np.inf)))
            continue
        lg = np.concatenate(logits, axis=1)
        vv = np.concatenate(values, axis=0)
        m = lg.max(axis=1, keepdims=True)
        m = np.where(np.isfinite(m), m, 0.0)
        w = np.exp(lg - m)
        den = w.sum(axis=1)
        with np.errstate(divide="ignore", invalid="ignore"):
            parts.append((np.where(den[:, None] > 0, (w @ vv) / den[:, None], 0.0), m[:, 0] + np.log(den)))
    return merge_partials(parts)
