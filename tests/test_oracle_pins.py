"""Pins for the CPU oracle: each test fixes the oracle to something other than itself --
a closed form, a library routine, a brute-force enumeration written differently, an
invariant the mathematics gives, or a figure the paper prints."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import fp2_oracle as O
from paper_2608_19758_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------------------------------
# helpers: tiny random workloads in fp64-exact BF16 values
# ------------------------------------------------------------------------------------------

def bf16_bits(x: np.ndarray) -> np.ndarray:
    return inputs.as_bits(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def tiny_workload(seed, seqs, Hq, Hkv, d, B, M, p, alpha=0.1, sink_tokens=None, window_tokens=None,
                  use_correction=1, shuffle=True, kv_override=None):
    """Random small workload.  seqs = [(Lk, pre)].  Returns (Workload, raw dict)."""
    rng = np.random.default_rng(seed)
    ns = len(seqs)
    need = [-(-Lk // p) for Lk, _ in seqs]
    pool = sum(need) + 3
    ids = rng.permutation(pool) if shuffle else np.arange(pool)
    pt = np.full((ns, max(need)), -1, dtype=np.int32)
    o = 0
    for b, n in enumerate(need):
        pt[b, :n] = ids[o:o + n]
        o += n
    total_q = sum(Lk - pre for Lk, pre in seqs)
    cu = np.zeros(ns + 1, dtype=np.int32)
    cu[1:] = np.cumsum([Lk - pre for Lk, pre in seqs])
    q = rng.standard_normal((total_q, Hq, d)) * 1.5
    kc = rng.standard_normal((pool, p, Hkv, d))
    vc = rng.standard_normal((pool, p, Hkv, d))
    if kv_override is not None:
        kv_override(kc, vc, pt, seqs, p, rng)
    prm = O.Params(num_q_heads=Hq, num_kv_heads=Hkv, head_dim=d, block_size=B, tile_rows=M, page_size=p,
                   sink_tokens=B if sink_tokens is None else sink_tokens,
                   window_tokens=B if window_tokens is None else window_tokens,
                   use_correction=use_correction, alpha=alpha)
    raw = dict(q_bits=bf16_bits(q), k_bits=bf16_bits(kc), v_bits=bf16_bits(vc), page_table=pt,
               cu_seqlens_q=cu, seqlens_k=np.array([Lk for Lk, _ in seqs], dtype=np.int32))
    return O.Workload(prm, **raw), raw


def vals(bits):
    return O.bf16_bits_to_f64(bits)


# ------------------------------------------------------------------------------------------
# an independent brute force: token-by-token Python loops, full weight matrix with one
# surrogate column per block (Eq. 6), written without any of the oracle's helpers
# ------------------------------------------------------------------------------------------

def brute_force(prm: O.Params, raw, alpha):
    q = vals(raw["q_bits"]); kc = vals(raw["k_bits"]); vc = vals(raw["v_bits"])
    pt, cu, lk = raw["page_table"], raw["cu_seqlens_q"], raw["seqlens_k"]
    Hq, Hkv, d, B, M, p = prm.num_q_heads, prm.num_kv_heads, prm.head_dim, prm.block_size, prm.tile_rows, prm.page_size
    g = Hq // Hkv
    sc = 1.0 / math.sqrt(d)
    sinkb = -(-prm.sink_tokens // B)
    winb = -(-prm.window_tokens // B)
    lists, outs, lses = {}, {}, {}
    seg = 0
    for b in range(len(lk)):
        Lk = int(lk[b]); Lq = int(cu[b + 1] - cu[b]); pre = Lk - Lq
        nblk = -(-Lk // B)
        ntile = -(-(g * Lq) // M)
        for h in range(Hkv):
            K = [[kc[pt[b][j // p], j % p, h, c] for c in range(d)] for j in range(Lk)]
            V = [[vc[pt[b][j // p], j % p, h, c] for c in range(d)] for j in range(Lk)]
            nJ = [min(B, Lk - J * B) for J in range(nblk)]
            kbar = [[math.fsum(K[j][c] for j in range(J * B, J * B + nJ[J])) / nJ[J] for c in range(d)]
                    for J in range(nblk)]
            vbar = [[math.fsum(V[j][c] for j in range(J * B, J * B + nJ[J])) / nJ[J] for c in range(d)]
                    for J in range(nblk)]
            for t in range(ntile):
                rows = list(range(t * M, min((t + 1) * M, g * Lq)))
                qrow = {r: q[cu[b] + r // g, h * g + r % g] for r in rows}
                apos = {r: pre + r // g for r in rows}
                p_first, p_last = apos[rows[0]], apos[rows[-1]]
                cand = [J for J in range(nblk) if J * B <= p_last]
                s = {(r, J): sc * math.fsum(qrow[r][c] * kbar[J][c] for c in range(d)) for r in rows for J in cand}
                mx = max(s.values())
                E = {J: math.fsum(math.exp(s[r, J] - mx) for r in rows) for J in cand}
                thr = alpha * max(E.values())
                fully_visible = [J for J in cand if J * B + B - 1 < (p_first // B) * B]
                keep = [J for J in cand if E[J] >= thr or J < sinkb or J >= p_first // B - winb]
                lists[seg] = keep
                o_rows, l_rows = [], []
                for r in rows:
                    w, val = [], []
                    for J in keep:
                        for j in range(J * B, J * B + nJ[J]):
                            if j <= apos[r]:
                                w.append(sc * math.fsum(qrow[r][c] * K[j][c] for c in range(d)))
                                val.append(V[j])
                    if prm.use_correction:
                        for J in fully_visible:
                            if J not in keep:
                                w.append(s[r, J] + math.log(nJ[J]))
                                val.append(vbar[J])
                    m = max(w)
                    e = [math.exp(x - m) for x in w]
                    den = math.fsum(e)
                    o_rows.append([math.fsum(e[i] * val[i][c] for i in range(len(e))) / den for c in range(d)])
                    l_rows.append(m + math.log(den))
                outs[seg] = np.array(o_rows); lses[seg] = np.array(l_rows)
                seg += 1
    return lists, outs, lses


@pytest.mark.parametrize("g,pre,p", [(1, 0, 4), (2, 5, 2), (3, 0, 4), (3, 5, 1), (2, 0, 4)])
def test_brute_force_tiny(g, pre, p):
    """Whole oracle (geometry, paging, pooling, energies, selection, Eq. 6) == enumeration."""
    Hkv = 2
    for alpha in (0.9, 0.4, 0.05):
        wl, raw = tiny_workload(11 + g, [(24, pre), (13, 0)], Hkv * g, Hkv, 8, 4, 4, p, alpha=alpha,
                                sink_tokens=4, window_tokens=4)
        lists, outs, lses = brute_force(wl.p, raw, alpha)
        sel = O.oracle_select(wl)
        assert len(sel) == len(lists)
        for s in wl.segs:
            assert list(sel[s.seg][0]) == lists[s.seg], (s, alpha)
        att = O.oracle_attend(wl, {k: v[0] for k, v in sel.items()})
        for k in att:
            np.testing.assert_allclose(att[k][0], outs[k], rtol=0, atol=1e-12)
            np.testing.assert_allclose(att[k][1], lses[k], rtol=0, atol=1e-12)


def test_brute_force_no_correction():
    wl, raw = tiny_workload(5, [(24, 3)], 4, 2, 8, 4, 4, 4, alpha=0.6, sink_tokens=4, window_tokens=0,
                            use_correction=0)
    lists, outs, lses = brute_force(wl.p, raw, 0.6)
    sel = O.oracle_select(wl)
    att = O.oracle_attend(wl, {k: v[0] for k, v in sel.items()})
    assert any(len(lists[k]) < wl.segs[k].J_hi + 1 for k in lists)      # something was pruned
    for k in att:
        np.testing.assert_allclose(att[k][0], outs[k], atol=1e-12)


# ------------------------------------------------------------------------------------------
# dense limit: selecting everything is textbook causal softmax attention
# ------------------------------------------------------------------------------------------

def naive_causal(q, K, V, pre, sc):
    """q [Lq, d]; plain double loop."""
    out = np.zeros_like(q); lse = np.zeros(q.shape[0])
    for i in range(q.shape[0]):
        n = pre + i + 1
        l = sc * (K[:n] @ q[i])
        m = l.max(); e = np.exp(l - m)
        out[i] = (e[:, None] * V[:n]).sum(0) / e.sum()
        lse[i] = m + math.log(e.sum())
    return out, lse


@pytest.mark.parametrize("g,pre", [(1, 0), (4, 0), (4, 37), (3, 11)])
def test_dense_limit_vs_naive_and_sdpa(g, pre):
    Hkv, d, B, M, p, Lk = 2, 16, 16, 16, 8, 150
    wl, raw = tiny_workload(3, [(Lk, pre)], Hkv * g, Hkv, d, B, M, p, alpha=0.0)
    sel = O.oracle_select(wl)
    for s in wl.segs:                                   # alpha = 0 keeps every candidate
        assert list(sel[s.seg][0]) == list(range(s.J_hi + 1))
    a1 = O.oracle_attend(wl, {k: v[0] for k, v in sel.items()})
    a2 = O.oracle_attend(wl, None, dense=True)
    Oo, Ll = O.scatter_output(wl, a1, Lk - pre)
    Od, Ld = O.scatter_output(wl, a2, Lk - pre)
    np.testing.assert_allclose(Oo, Od, atol=1e-13)
    q = vals(raw["q_bits"])
    for h in range(Hkv):
        K, V, *_ = wl.kv(0, h)
        for hq in range(h * g, (h + 1) * g):
            ref, lref = naive_causal(q[:, hq], K, V, pre, 1 / math.sqrt(d))
            np.testing.assert_allclose(Oo[:, hq], ref, atol=1e-12)
            np.testing.assert_allclose(Ll[hq], lref, atol=1e-12)
            if pre == 0:                                # library routine, top-left == bottom-right
                tq = torch.from_numpy(q[:, hq])[None, None]
                tk = torch.from_numpy(K)[None, None]; tv = torch.from_numpy(V)[None, None]
                sd = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
                np.testing.assert_allclose(Oo[:, hq], sd[0, 0].numpy(), atol=1e-12)


# ------------------------------------------------------------------------------------------
# Eq. 6 closed form: block-constant K and V make the correction exact for ANY selection
# ------------------------------------------------------------------------------------------

def _block_constant(B):
    def f(kc, vc, pt, seqs, p, rng):
        for b, (Lk, _) in enumerate(seqs):
            for J in range(-(-Lk // B)):
                kk = rng.standard_normal(kc.shape[2:]); vv = rng.standard_normal(vc.shape[2:])
                for j in range(J * B, min((J + 1) * B, Lk)):
                    kc[pt[b, j // p], j % p] = kk
                    vc[pt[b, j // p], j % p] = vv
    return f


@pytest.mark.parametrize("alpha", [0.9, 0.3, 0.01])
def test_block_constant_correction_is_exact(alpha):
    B = 8
    wl, raw = tiny_workload(7, [(96, 0), (50, 13)], 4, 2, 16, B, 8, 4, alpha=alpha, sink_tokens=0,
                            window_tokens=0, kv_override=_block_constant(B))
    sel = O.oracle_select(wl)
    lists = {k: v[0] for k, v in sel.items()}
    pruned = sum(s.J_hi + 1 - len(lists[s.seg]) for s in wl.segs)
    if alpha >= 0.3:
        assert pruned > 0
    corr = O.oracle_attend(wl, lists)
    dense = O.oracle_attend(wl, None, dense=True)
    for k in corr:
        np.testing.assert_allclose(corr[k][0], dense[k][0], atol=1e-12)
        np.testing.assert_allclose(corr[k][1], dense[k][1], atol=1e-12)
    # and without the correction the truncated result must differ (the term is not a no-op)
    wl.p.use_correction = 0
    trunc = O.oracle_attend(wl, lists)
    if pruned:
        assert max(np.abs(trunc[k][0] - dense[k][0]).max() for k in trunc) > 1e-6


def test_lse_ordering_truncated_le_corrected_le_dense():
    """Jensen: |B| e^{mean s} <= sum e^{s}; all terms positive."""
    wl, _ = tiny_workload(9, [(200, 20)], 6, 2, 16, 8, 8, 8, alpha=0.5, sink_tokens=8, window_tokens=8)
    sel = O.oracle_select(wl)
    lists = {k: v[0] for k, v in sel.items()}
    corr = O.oracle_attend(wl, lists)
    dense = O.oracle_attend(wl, None, dense=True)
    wl.p.use_correction = 0
    trunc = O.oracle_attend(wl, lists)
    strict = 0
    for k in corr:
        assert np.all(trunc[k][1] <= corr[k][1] + 1e-12)
        assert np.all(corr[k][1] <= dense[k][1] + 1e-12)
        strict += int(np.any(trunc[k][1] < corr[k][1] - 1e-9))
    assert strict > 0


def test_taylor_orders_of_the_surrogate():
    """Eq. 7: mass error of a corrected block is O(delta^2), numerator error O(delta)."""
    rng = np.random.default_rng(0)
    d, B = 16, 32
    q = rng.standard_normal((1, d))
    k0 = rng.standard_normal(d); noise = rng.standard_normal((B, d)); noise -= noise.mean(0)
    V = rng.standard_normal((B, d))
    errs_den, errs_num = [], []
    for eps in (1e-2, 1e-3):
        K = k0 + eps * noise
        kbar, vbar = O.pooled_means(K, B), O.pooled_means(V, B)
        s = (q @ K.T)[0] / math.sqrt(d)
        sbar = float((q @ kbar.T)[0, 0]) / math.sqrt(d)
        errs_den.append(abs(np.exp(s).sum() - B * math.exp(sbar)))
        errs_num.append(np.abs(np.exp(s) @ V - B * math.exp(sbar) * vbar[0]).max())
    assert 1.8 < math.log10(errs_den[0] / errs_den[1]) < 2.2
    assert 0.8 < math.log10(errs_num[0] / errs_num[1]) < 1.2


# ------------------------------------------------------------------------------------------
# Eq. 1-3 (per-block max / sum, global rescale, normalised score) == Eq. 19-20 (energies)
# ------------------------------------------------------------------------------------------

def test_normalised_score_form_equals_energy_form():
    rng = np.random.default_rng(4)
    d = 32
    for trial in range(20):
        nrow, ncand = int(rng.integers(1, 40)), int(rng.integers(1, 30))
        qt = rng.standard_normal((nrow, d)) * 2.0
        kb = rng.standard_normal((ncand, d))
        sc = 1 / math.sqrt(d)
        alpha = float(rng.choice([0.5, 0.1, 0.01]))
        # Eq. 1-3 literally
        s = sc * qt @ kb.T
        m_IJ = s.max(axis=0)
        S_IJ = np.exp(s - m_IJ[None, :]).sum(axis=0)
        M_I = m_IJ.max()
        unnorm = S_IJ * np.exp(m_IJ - M_I)
        keep_sets = []
        for eps in (0.0, 1e-6, 1.0):
            score = unnorm / (unnorm.sum() + eps)
            keep_sets.append(set(np.nonzero(score >= alpha * score.max())[0]))
        E, M = O.block_energies(qt, kb, sc)
        idx, margin = O.select_blocks(E, alpha, np.zeros(ncand, dtype=bool))
        np.testing.assert_allclose(M, M_I)
        np.testing.assert_allclose(E, unnorm, rtol=1e-12)
        near = set(np.nonzero(margin < 1e-9)[0])
        for ks in keep_sets:
            assert (ks ^ set(idx.tolist())) <= near


# ------------------------------------------------------------------------------------------
# selection invariants
# ------------------------------------------------------------------------------------------

def test_selection_invariants():
    wl, _ = tiny_workload(21, [(700, 0), (300, 123)], 8, 2, 16, 16, 16, 8, alpha=0.2, sink_tokens=32,
                          window_tokens=48)
    prev = None
    for alpha in (1.5, 1.0, 0.2, 0.01, 0.0):
        wl.p.alpha = alpha
        sel = O.oracle_select(wl)
        for s in wl.segs:
            idx, E, _ = sel[s.seg]
            assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] <= s.J_hi       # ascending, unique, candidates
            assert set(range(s.J_lo, s.J_hi + 1)) <= set(idx)                            # diagonal band always kept
            assert set(range(min(2, s.J_hi + 1))) <= set(idx)                            # 32 sink tokens = 2 blocks
            assert set(range(max(0, s.J_lo - 3), s.J_hi + 1)) <= set(idx)                # 48-token window = 3 blocks
            if alpha <= 1.0:
                assert int(np.argmax(E)) in set(idx)
            if alpha == 0.0:
                assert len(idx) == s.J_hi + 1
            if alpha > 1.0:
                forced = O.forced_mask(s.J_lo, s.J_hi, 16, 32, 48)
                assert list(idx) == list(np.nonzero(forced)[0])
            if prev is not None:
                assert set(prev[s.seg][0]) <= set(idx)                                    # S(a2) subset S(a1), a1 < a2
        prev = sel


def test_margin_by_hand():
    """The distance to the threshold that decides which list mismatches are excused: |E_J - alpha max E| divided
    by alpha max E (the threshold of Eq. 20), worked by hand.  E = [1, 0.1005, 0.0999, 0.05], alpha = 0.1: the
    threshold is 0.1, so the distances are 0.9 / 0.1, 0.0005 / 0.1, 0.0001 / 0.1 and 0.05 / 0.1.  Dividing by
    max E instead of the threshold would give a tenth of these; dividing by E_J would give 0.9, ~0.005, ~0.001, 1."""
    E = np.array([1.0, 0.1005, 0.0999, 0.05])
    idx, margin = O.select_blocks(E, 0.1, np.zeros(4, dtype=bool))
    assert idx.tolist() == [0, 1]
    np.testing.assert_allclose(margin, [9.0, 5e-3, 1e-3, 0.5], rtol=0, atol=1e-12)
    # forced blocks enter the list but their margin is still their energy's distance to the threshold
    idx, margin = O.select_blocks(E, 0.1, np.array([False, False, False, True]))
    assert idx.tolist() == [0, 1, 3]
    np.testing.assert_allclose(margin, [9.0, 5e-3, 1e-3, 0.5], rtol=0, atol=1e-12)
    # scale invariance: multiplying every energy by a constant changes neither the list nor the margins
    idx2, margin2 = O.select_blocks(E * 1024.0, 0.1, np.zeros(4, dtype=bool))
    assert idx2.tolist() == [0, 1]
    np.testing.assert_allclose(margin2, margin, rtol=1e-12)
    # alpha = 1: only the maximum reaches the threshold, and it sits on it
    idx, margin = O.select_blocks(E, 1.0, np.zeros(4, dtype=bool))
    assert idx.tolist() == [0]
    np.testing.assert_allclose(margin, [0.0, 0.8995, 0.9001, 0.95], rtol=0, atol=1e-12)


def test_margin_is_zero_exactly_on_the_threshold():
    """margin_J == 0  <=>  E_J == alpha max E, on exactly representable numbers (powers of two), and the margin
    of a candidate is the relative perturbation of its energy that would flip its membership."""
    E = np.array([8.0, 2.0, 1.0, 0.5, 2.0])
    for alpha, on_thr in ((0.25, [1, 4]), (0.125, [2]), (1.0, [0]), (0.3, [])):
        idx, margin = O.select_blocks(E, alpha, np.zeros(5, dtype=bool))
        assert sorted(np.nonzero(margin == 0.0)[0].tolist()) == on_thr
        assert sorted(np.nonzero(E == alpha * E.max())[0].tolist()) == on_thr
        assert set(on_thr) <= set(idx.tolist())                   # ">=": equality selects
    rng = np.random.default_rng(11)
    E = rng.uniform(0.01, 1.0, 200)
    alpha = 0.3
    idx, margin = O.select_blocks(E, alpha, np.zeros(200, dtype=bool))
    thr = alpha * E.max()
    kept = set(idx.tolist())
    for J in range(200):
        if J == int(np.argmax(E)):
            continue                                              # moving the maximum moves the threshold itself
        for sign in (-1.0, 1.0):
            for f, flips in ((0.5, False), (1.5, True)):
                Ep = E.copy()
                Ep[J] = E[J] + sign * f * margin[J] * thr         # move E_J by f x margin x threshold
                in_now = Ep[J] >= thr
                moved_across = in_now != (J in kept)
                toward = (sign > 0) != (J in kept)                # toward the threshold
                assert moved_across == (flips and toward), (J, sign, f)


def test_pooled_means_closed_form():
    B = 8
    x = np.arange(27, dtype=np.float64)[:, None] * np.array([[1.0, -2.0]])
    m = O.pooled_means(x, B)
    # mean of an arithmetic progression = midpoint; ragged tail averages its 3 real tokens only
    np.testing.assert_allclose(m[:, 0], [3.5, 11.5, 19.5, 25.0])
    np.testing.assert_allclose(m[:, 1], [-7.0, -23.0, -39.0, -50.0])
    assert list(O.block_token_counts(27, B)) == [8, 8, 8, 3]


def test_widening_of_bit_patterns():
    x = torch.tensor([1.0, -2.5, 3.140625, 1e-3, 65280.0], dtype=torch.bfloat16)
    np.testing.assert_array_equal(O.bf16_bits_to_f64(inputs.as_bits(x)), x.to(torch.float64).numpy())
    allb = torch.arange(256, dtype=torch.uint8)
    ref = allb.view(torch.float8_e4m3fn).to(torch.float64).numpy()           # library decode
    got = O.e4m3_bits_to_f64(allb.numpy())
    np.testing.assert_array_equal(np.isnan(got), np.isnan(ref))
    np.testing.assert_array_equal(got[~np.isnan(ref)], ref[~np.isnan(ref)])


# ------------------------------------------------------------------------------------------
# geometry / counting
# ------------------------------------------------------------------------------------------

def test_candidate_pair_counts_of_the_configs():
    for L, Hq, Hkv, per_head in ((2048, 4, 1, 544), (32768, 32, 8, 131584), (131072, 32, 8, 2099200)):
        p = O.Params(num_q_heads=Hq, num_kv_heads=Hkv)
        n = O.candidate_pairs(p, [0, L], [L])
        g = Hq // Hkv
        nblk = L // 128
        assert n == Hkv * per_head == Hkv * g * nblk * (nblk + 1) // 2


def _golden():
    out = {}
    for line in open(os.path.join(GOLDEN, "paper_figures.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def test_paper_index_memory_arithmetic():
    """The paper's table: dense mask 8 / 32 MB, CSR about 3 / 6 MB at 9% / 5% density
    (batch 1, 32 query heads, 4 KV heads, 64-token physical tiles, int32)."""
    gold = _golden()
    for L, key_mask, key_csr, key_rho in ((65536, "dense_mask_mb_64k", "csr_mb_64k", "csr_density_64k"),
                                          (131072, "dense_mask_mb_128k", "csr_mb_128k", "csr_density_128k")):
        nblk = L // 128
        assert 32 * nblk * nblk / 2 ** 20 == gold[key_mask]
        p = O.Params(num_q_heads=32, num_kv_heads=4)
        segs = O.segments(p, [0, L], [L])
        assert len(segs) == 4 * (8 * L // 128)
        pairs = sum(s.J_hi + 1 for s in segs)
        csr_mb = pairs * gold[key_rho] * 2 * 4 / 1e6           # 2 physical tiles per logical block
        assert abs(csr_mb - gold[key_csr]) / gold[key_csr] < 0.2


def test_paper_overhead_ratio():
    gold = _golden()
    rho, B = gold["aux_ratio_rho"], gold["aux_ratio_B"]
    assert abs((2 - rho) / (2 * rho * B) - gold["aux_over_attn_ratio"]) < 0.005


def test_segment_order_and_rows_g7():
    """g = 7 tiles straddle positions: rows, positions and blocks must be row-based."""
    p = O.Params(num_q_heads=14, num_kv_heads=2, block_size=128, tile_rows=128)
    segs = O.segments(p, [0, 100, 300], [400, 200])
    nt0, nt1 = -(-700 // 128), -(-1400 // 128)
    assert len(segs) == 2 * (nt0 + nt1)
    for i, s in enumerate(segs):
        assert s.seg == i
    s = segs[nt0 + 2]                       # sequence 0, head 1, tile 2
    assert (s.b, s.h, s.t, s.r0, s.r1, s.pre) == (0, 1, 2, 256, 384, 300)
    assert s.J_lo == (300 + 256 // 7) // 128 and s.J_hi == (300 + 383 // 7) // 128
    last = segs[nt0 - 1]
    assert last.r1 == 700 and last.J_hi == (300 + 99) // 128
    pos = O.row_positions(p, s)
    assert pos[0] == 300 + 36 and pos[-1] == 300 + 54 and len(pos) == 128


# ------------------------------------------------------------------------------------------
# invariances: paging, batching, GQA packing, chunked dense
# ------------------------------------------------------------------------------------------

def _rebuild(raw, prm, **over):
    kw = dict(raw); kw.update(over)
    return O.Workload(prm, **kw)


def test_page_permutation_is_bit_invariant():
    wl, raw = tiny_workload(31, [(130, 10)], 4, 2, 16, 16, 16, 4, alpha=0.3, shuffle=True)
    # same tokens laid out contiguously
    p = 4
    Lk = 130
    npg = -(-Lk // p)
    kc = raw["k_bits"]; vc = raw["v_bits"]
    kc2 = np.zeros_like(kc); vc2 = np.zeros_like(vc)
    kc2[:npg] = kc[raw["page_table"][0, :npg]]; vc2[:npg] = vc[raw["page_table"][0, :npg]]
    pt2 = np.arange(npg, dtype=np.int32)[None, :]
    wl2 = _rebuild(raw, wl.p, k_bits=kc2, v_bits=vc2, page_table=pt2)
    s1, s2 = O.oracle_select(wl), O.oracle_select(wl2)
    a1 = O.oracle_attend(wl, {k: v[0] for k, v in s1.items()})
    a2 = O.oracle_attend(wl2, {k: v[0] for k, v in s2.items()})
    for k in a1:
        assert np.array_equal(s1[k][0], s2[k][0]) and np.array_equal(s1[k][1], s2[k][1])
        assert np.array_equal(a1[k][0], a2[k][0]) and np.array_equal(a1[k][1], a2[k][1])


def test_sequence_in_batch_equals_sequence_alone():
    seqs = [(90, 0), (130, 40), (33, 5)]
    wl, raw = tiny_workload(32, seqs, 4, 2, 16, 16, 16, 4, alpha=0.3)
    sel = O.oracle_select(wl)
    att = O.oracle_attend(wl, {k: v[0] for k, v in sel.items()})
    Ob, Lb = O.scatter_output(wl, att, int(raw["cu_seqlens_q"][-1]))
    for b, (Lk, pre) in enumerate(seqs):
        cu = raw["cu_seqlens_q"]
        one = dict(raw, q_bits=raw["q_bits"][cu[b]:cu[b + 1]], page_table=raw["page_table"][b:b + 1],
                   cu_seqlens_q=np.array([0, Lk - pre], dtype=np.int32), seqlens_k=np.array([Lk], dtype=np.int32))
        w1 = O.Workload(wl.p, **one)
        s1 = O.oracle_select(w1)
        a1 = O.oracle_attend(w1, {k: v[0] for k, v in s1.items()})
        O1, L1 = O.scatter_output(w1, a1, Lk - pre)
        assert np.array_equal(O1, Ob[cu[b]:cu[b + 1]])
        assert np.array_equal(L1, Lb[:, cu[b]:cu[b + 1]])


def test_gqa_packing_equals_replicated_heads():
    """Attention at (g, M) == a g=1 run with the KV head replicated g times, M/g rows per
    tile and each replica given the packed tile's list."""
    g, Hkv, M, B, d, p, Lk, pre = 4, 1, 16, 16, 16, 8, 112, 16
    wl, raw = tiny_workload(33, [(Lk, pre)], g, Hkv, d, B, M, p, alpha=0.4)
    sel = O.oracle_select(wl)
    lists = {k: v[0] for k, v in sel.items()}
    att = O.oracle_attend(wl, lists)
    Og, Lg = O.scatter_output(wl, att, Lk - pre)
    kc = np.repeat(raw["k_bits"], g, axis=2); vc = np.repeat(raw["v_bits"], g, axis=2)
    prm1 = O.Params(num_q_heads=g, num_kv_heads=g, head_dim=d, block_size=B, tile_rows=M // g, page_size=p,
                    sink_tokens=wl.p.sink_tokens, window_tokens=wl.p.window_tokens, alpha=0.4)
    w1 = O.Workload(prm1, **dict(raw, k_bits=kc, v_bits=vc))
    nt = len(wl.segs)
    assert len(w1.segs) == g * nt
    lists1 = {s.seg: lists[s.t] for s in w1.segs}
    a1 = O.oracle_attend(w1, lists1)
    O1, L1 = O.scatter_output(w1, a1, Lk - pre)
    np.testing.assert_allclose(O1, Og, atol=1e-13)
    np.testing.assert_allclose(L1, Lg, atol=1e-13)


def test_chunked_dense_equals_rows_of_single_shot():
    Lk, pre = 140, 60
    wl, raw = tiny_workload(34, [(Lk, 0)], 4, 2, 16, 16, 16, 4)
    full = O.oracle_attend(wl, None, dense=True)
    Of, Lf = O.scatter_output(wl, full, Lk)
    chunk = dict(raw, q_bits=raw["q_bits"][pre:], cu_seqlens_q=np.array([0, Lk - pre], dtype=np.int32))
    wc = O.Workload(wl.p, **chunk)
    part = O.oracle_attend(wc, None, dense=True)
    Oc, Lc = O.scatter_output(wc, part, Lk - pre)
    np.testing.assert_allclose(Oc, Of[pre:], atol=1e-13)
    np.testing.assert_allclose(Lc, Lf[:, pre:], atol=1e-13)


def test_fp8_inputs_are_dequantised_per_head():
    spec = inputs.small_spec(seqs=[(300, 44)], num_q_heads=6, num_kv_heads=2, page_size=16, dtype="fp8")
    case = inputs.make_case(spec)
    wl = O.Workload(O.Params.from_dict(case.params()), **inputs.oracle_args(case))
    K, V, *_ = wl.kv(0, 1)
    pt = case.page_table[0].numpy()
    j = 123
    raw = case.k_cache[pt[j // 16], j % 16, 1].view(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(K[j], raw * float(case.k_scale[1]))
    q = wl.q_seq(0)
    rawq = case.q[5, 4].view(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(q[5, 4], rawq * float(case.q_scale[4]))
    # dense attention on the dequantised values equals the naive loop
    den = O.oracle_attend(wl, None, dense=True)
    Oo, _ = O.scatter_output(wl, den, 256)
    ref, _ = naive_causal(q[:, 4], K, V, 44, 1 / math.sqrt(128))
    np.testing.assert_allclose(Oo[:, 4], ref, atol=1e-12)


def test_generator_density_matches_forced_fraction_on_config1():
    """Config 1 at alpha = 0.1: every selected block is a forced one (sink 2 + window 4 + diag)."""
    case = inputs.make_case(inputs.config_spec(1))
    wl = O.Workload(O.Params.from_dict(case.params()), **inputs.oracle_args(case))
    sel = O.oracle_select(wl)
    nsel = sum(len(v[0]) for v in sel.values())
    forced = sum(int(O.forced_mask(s.J_lo, s.J_hi, 128, 256, 512).sum()) for s in wl.segs)
    assert forced == 364 and nsel >= forced and nsel <= 544


# ------------------------------------------------------------------------------------------
# index export (Algorithm 1 line 5; Sec. 3.4): pinned by token coverage, by the paper's
# "B / 64 physical tiles per logical block" and its index-memory figure, and by the round trip
# through Eq. 22
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("tile", [16, 32, 64, 128])
def test_export_csr_covers_exactly_the_listed_tokens(tile):
    wl, raw = tiny_workload(31, [(500, 100), (129, 0), (64, 0), (333, 300)], Hq=4, Hkv=2, d=8, B=128, M=128, p=16)
    sel = O.oracle_select(wl)
    lists = {seg: v[0] for seg, v in sel.items()}
    cu, idx = O.export_csr(wl, lists, tile)
    assert cu[0] == 0 and len(cu) == len(wl.segs) + 1 and cu[-1] == len(idx)
    assert (np.diff(cu) >= 0).all()
    for s in wl.segs:
        Lk = int(wl.lk[s.b])
        tiles = idx[cu[s.seg]:cu[s.seg + 1]]
        assert (np.diff(tiles) > 0).all()                      # ascending, unique
        want = np.zeros(Lk, dtype=bool)                        # tokens of the listed blocks, one by one
        for J in lists[s.seg]:
            want[J * 128:min((J + 1) * 128, Lk)] = True
        got = np.zeros(Lk + tile, dtype=bool)
        for t in tiles:
            assert t * tile < Lk                               # every tile holds a real token
            got[t * tile:(t + 1) * tile] = True
        # a tile may reach past its block only inside the same block's padding (tile <= B divides B)
        assert (got[:Lk] == want).all()


def test_export_csr_two_tiles_per_full_block_and_paper_index_memory():
    """B / 64 = 2 physical tiles per logical block (Sec. 3.3, implementation details); with every block
    listed at 128K (32 query heads, 4 KV heads) the index holds 2 x pairs int32 entries, and at the paper's
    5 % density that is its 6 MB figure."""
    gold = _golden()
    p = O.Params(num_q_heads=32, num_kv_heads=4)
    L = 4096

    class W:   # geometry only: export_csr touches segments and lengths, never the tensors
        pass
    wl = W()
    wl.p, wl.lk = p, np.array([L])
    wl.segs = O.segments(p, [0, L], [L])
    lists = {s.seg: np.arange(s.J_hi + 1) for s in wl.segs}
    cu, idx = O.export_csr(wl, lists, 64)
    pairs = sum(s.J_hi + 1 for s in wl.segs)
    assert cu[-1] == 2 * pairs
    s0 = wl.segs[5]
    assert list(idx[cu[5]:cu[6]]) == [t for J in range(s0.J_hi + 1) for t in (2 * J, 2 * J + 1)]
    # scale the count to 128K (pairs grow with L^2) and apply the paper's density
    pairs_128k = sum(s.J_hi + 1 for s in O.segments(p, [0, 131072], [131072]))
    mb = 2 * pairs_128k * gold["csr_density_128k"] * 4 / 1e6
    assert abs(mb - gold["csr_mb_128k"]) / gold["csr_mb_128k"] < 0.2


def test_export_csr_ragged_last_block():
    p = O.Params(num_q_heads=1, num_kv_heads=1)

    class W:
        pass
    for Lk, n_last in ((128 + 1, 1), (128 + 64, 1), (128 + 65, 2), (256, 2)):
        wl = W()
        wl.p, wl.lk = p, np.array([Lk])
        wl.segs = O.segments(p, [0, Lk], [Lk])
        last = wl.segs[-1]
        cu, idx = O.export_csr(wl, {s.seg: np.arange(s.J_hi + 1) for s in wl.segs}, 64)
        assert cu[last.seg + 1] - cu[last.seg] == 2 * last.J_hi + n_last


def test_page_table_from_token_map_round_trip():
    """Eq. 22 forwards (slot of every token from the page table), then the strided read backwards."""
    rng = np.random.default_rng(5)
    p, lens = 16, [500, 17, 16, 129]
    need = [-(-L // p) for L in lens]
    ids = rng.permutation(sum(need) + 5)
    pt = np.full((len(lens), max(need)), -1, dtype=np.int32)
    o = 0
    for b, n in enumerate(need):
        pt[b, :n] = ids[o:o + n]
        o += n
    tok = np.full((len(lens), max(lens)), -7, dtype=np.int32)
    for b, L in enumerate(lens):
        for j in range(L):
            tok[b, j] = pt[b, j // p] * p + j % p            # Eq. 22
    got, bad = O.page_table_from_token_map(tok, lens, p, pt.shape[1])
    assert not bad and (got == pt).all()
    tok[3, 32] += 3                                            # a slot that does not start a page
    got, bad = O.page_table_from_token_map(tok, lens, p, pt.shape[1])
    assert bad


# ------------------------------------------------------------------------------------------
# KV splitting (Eq. 18): the partition is checked against its definition, the merge against
# the single-pass result and against a two-part case worked by hand
# ------------------------------------------------------------------------------------------

def test_split_ranges_partition_the_sequence_by_count():
    for n in range(0, 40):
        for U in range(1, 9):
            r = O.split_ranges(n, U)
            assert len(r) == U
            covered = [t for a, b in r for t in range(a, b)]
            assert covered == list(range(n))                    # contiguous, in order, nothing twice
            sizes = [b - a for a, b in r]
            assert max(sizes) == -(-n // U)                     # the ceil of Eq. 18
            assert sizes == sorted(sizes, reverse=True)         # full parts first, then the short one, then empty


def test_merge_of_two_parts_by_hand():
    """Two keys, one per part: weights e^{s0}, e^{s1}; the merge must give the softmax average."""
    s0, s1 = 0.3, -1.2
    v0, v1 = np.array([[1.0, 2.0]]), np.array([[-3.0, 0.5]])
    o, lse = O.merge_partials([(v0, np.array([s0])), (v1, np.array([s1]))])
    w0, w1 = math.exp(s0), math.exp(s1)
    assert np.allclose(o, (w0 * v0 + w1 * v1) / (w0 + w1), rtol=0, atol=1e-15)
    assert abs(lse[0] - math.log(w0 + w1)) < 1e-15
    o, lse = O.merge_partials([(v0, np.array([s0])), (np.zeros((1, 2)), np.array([-np.inf]))])   # an empty part
    assert np.allclose(o, v0) and abs(lse[0] - s0) < 1e-15


@pytest.mark.parametrize("U", [1, 2, 3, 5, 16])
@pytest.mark.parametrize("use_correction", [0, 1])
def test_split_attention_equals_single_pass(U, use_correction):
    wl, raw = tiny_workload(41, [(700, 200), (130, 0)], Hq=4, Hkv=2, d=16, B=128, M=128, p=16, alpha=0.3,
                            use_correction=use_correction)
    sel = O.oracle_select(wl)
    p = wl.p
    for s in wl.segs[::3]:
        K, V, kbar, vbar, n_tok = wl.kv(s.b, s.h)
        qt = O.tile_queries(wl.q_seq(s.b), p, s)
        args = (qt, O.row_positions(p, s), K, V, kbar, vbar, n_tok, sel[s.seg][0], s.J_lo, p.block_size, p.scale,
                use_correction)
        o1, l1 = O.attend_tile(*args)
        o2, l2 = O.attend_tile_split(*args, U)
        assert np.allclose(o1, o2, rtol=0, atol=1e-12) and np.allclose(l1, l2, rtol=0, atol=1e-12)
