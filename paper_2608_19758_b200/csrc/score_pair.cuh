// Fused block scoring and selection (Eq. 19, Eq. 20; Algorithm 1 lines 3-5) for BF16 plans whose packed query tile
// is a TMA box (group size divides 128): score_select_kernel with TWO adjacent query tiles of a KV head per unit.
//
// At long sequences score_select_kernel is bound by the traffic of the pooled keys from L2 into shared memory: every
// chunk of 128 pooled keys (hi + lo: 64 KB) is fetched once per query tile, 35 bytes per cycle and SM at 131072
// tokens, before the tensor pipe (1024 cycles per chunk) or the exponentials (1024) are busy.  Adjacent tiles of one
// KV head have the same candidates (the later one at most one block more), so here a chunk of pooled keys, once in
// shared memory, is multiplied with both tiles in one MMA of N = 256 (A = 128 pooled keys on the TMEM lanes,
// B = the two query tiles back to back): half the bytes per tile, half the MMA instructions.
//
// Units (built by the planner, heaviest first): a pair of tiles (t-1, t) of one (sequence, KV head) when the later
// tile has at most 1024 candidate blocks, else a single tile.  CTA b takes units b, b + grid, b + 2 grid, ...
// Everything else is as in score_select_kernel: the contraction runs transposed, kbar enters as a BF16 (hi, lo) pair
// accumulated into one fp32 accumulator, two consumer warpgroups alternate over the chunks (two TMEM accumulators
// of 256 columns) and each takes, per pooled key, maximum and exponential sum over the rows of the first tile and
// then of the second, log2 energies go to shared memory, and a selection warp applies threshold and forced sets and
// writes the ordered lists of unit u beside the scoring of unit u+1.
//
// Roles: warps 0-3 / 4-7 consumer warpgroups; warp 8 TMA producer of kbar pieces (16 KB: 128 keys x 64 elements, four
// per chunk: hi | lo x the two halves of d); warp 9 UMMA issuer and TMEM owner; warp 10 unit set-up and query tiles by
// TMA (two units in flight); warp 11 selection.
// Shared memory: 2 x 64 KB query pairs + 4 x 16 KB pieces + 16 KB energies.  TMEM: 2 x 256 columns.
#pragma once
#include "score_select.cuh"

namespace fp2 {

constexpr int kPairThreads = 384;
constexpr int kPairInfoSlots = 4;        // unit descriptors in flight
constexpr int kPairQBufs = 2;            // 64 KB query-pair buffers
constexpr int kPairPieces = 4;           // ring of 16 KB kbar pieces
constexpr int kPairPieceBytes = 16384;
constexpr int kPairMaxCand = 1024;       // a tile is paired only if it has at most this many candidate blocks
constexpr int kPairSmemBytes = 1024 /*align*/ + kPairQBufs * 65536 + kPairPieces * kPairPieceBytes + kMaxBlocks * 4;

struct PairInfo {
  SegInfo sg[2];
  int32_t nt;       // tiles in the unit: 1 or 2
  int32_t valid;    // 0: no more work
};

// One pooled key (= this thread's TMEM lane) against the 128 query rows of one tile (= 128 TMEM columns at
// lane_addr): m = max_j x_j, sum = sum_j 2^(x_j - m), x_j = s_j * cs.  PARTIAL: only the first nrows columns are real
// query rows.  With `release` the accumulator is handed back as soon as it is in registers.
template <bool PARTIAL>
__device__ __forceinline__ void score_cols(uint32_t lane_addr, float cs, int nrows, uint64_t* release, float& m_out,
                                           float& sum_out) {
  uint32_t xv[128];
#pragma unroll
  for (int k = 0; k < 4; ++k) tmem_ld32(lane_addr + k * 32, reinterpret_cast<uint32_t(&)[32]>(xv[k * 32]));
  tmem_wait_ld();
  if (release != nullptr) {
    tc_fence_before();
    mbar_arrive(release);
  }
  float x[128];
#pragma unroll
  for (int j = 0; j < 128; ++j) {
    x[j] = __uint_as_float(xv[j]);
    if constexpr (PARTIAL) x[j] = (j < nrows) ? x[j] : -INFINITY;
  }
  float m8[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const float* v = &x[c * 16];
    m8[c] = max3(max3(max3(v[0], v[1], v[2]), max3(v[3], v[4], v[5]), max3(v[6], v[7], v[8])),
                 max3(v[9], v[10], v[11]), max3(max3(v[12], v[13], v[14]), v[15], v[15]));
  }
  // the multiplier is positive: the maximum is taken over the raw logits and the scaling rides in the fused
  // multiply-add that subtracts it
  float m = fmaxf(max3(m8[0], m8[1], m8[2]), max3(max3(m8[3], m8[4], m8[5]), m8[6], m8[7])) * cs;
  const uint64_t nm2 = f2_pack(-m, -m), mul2 = f2_pack(cs, cs);
  uint64_t s4[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
  for (int j = 0; j < 128; j += 2) {
    float d0, d1;
    f2_unpack(f2_fma(f2_pack(x[j], x[j + 1]), mul2, nm2), d0, d1);
    s4[(j >> 1) & 3] = f2_add(s4[(j >> 1) & 3], f2_pack(ex2(d0), ex2(d1)));
  }
  float t0, t1;
  f2_unpack(f2_add(f2_add(s4[0], s4[1]), f2_add(s4[2], s4[3])), t0, t1);
  m_out = m;
  sum_out = t0 + t1;
}

__global__ void __launch_bounds__(kPairThreads, 1)
score_pair_kernel(const __grid_constant__ CUtensorMap map_khi, const __grid_constant__ CUtensorMap map_klo,
                  const __grid_constant__ CUtensorMap map_q, const SegInfo* __restrict__ segs,
                  const int2* __restrict__ units, int nunits, DevParams P, int64_t* __restrict__ seg_offset,
                  int32_t* __restrict__ seg_count, int32_t* __restrict__ blk_idx, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // query pair buffer: [half of d][tile][128 rows x 128 bytes] -- the two tiles of a half are 256 consecutive rows of
  // one swizzled K-major operand
  uint8_t* sQ = smem;
  uint8_t* sStage = smem + kPairQBufs * 65536;                                  // ring of kbar pieces
  float* sE = reinterpret_cast<float*>(sStage + kPairPieces * kPairPieceBytes); // log2 energies: unit parity x 2048,
                                                                                // second tile of a pair 1024 further

  __shared__ PairInfo info[kPairInfoSlots];
  __shared__ uint64_t info_full[kPairInfoSlots], info_empty[kPairInfoSlots], q_full[kPairQBufs], q_empty[kPairQBufs];
  __shared__ uint64_t full[kPairPieces], empty[kPairPieces], acc_full[2], acc_empty[2];
  __shared__ uint64_t e_full[2], sel_done[2];   // [unit & 1] energies of the unit are complete / its lists are written
  __shared__ uint64_t drain_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float red[2][2][8];                // [unit & 1][tile][consumer warp] maxima of the log2 energies

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  WaitCtx ctx{status, &abort_flag};

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < kPairInfoSlots; ++i) {
      mbar_init(&info_full[i], 1);
      mbar_init(&info_empty[i], 2 + 256 + 1);   // producer, issuer, consumers, selection warp
    }
    for (int i = 0; i < kPairQBufs; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&e_full[i], 256);
      mbar_init(&sel_done[i], 1);
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 256);
    }
    for (int i = 0; i < kPairPieces; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(&drain_bar, 1);
    fence_barrier_init();
  }
  if (warp == 9) {
    tmem_alloc(&tmem_base_s, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  // chunks of a unit: those of its last tile (the later tile of a pair has the larger candidate range)
  auto unit_chunks = [](const PairInfo& pi) { return (pi.sg[pi.nt - 1].J_hi + 128) >> 7; };

  if (warp == 10) {
    // ---------------- set-up: unit k of this CTA is number blockIdx.x + k * gridDim.x of the planner's table
    // (heaviest first; a static round-robin, no atomic on the critical path).  Query tiles by TMA: under PackGQA
    // (Eq. 13) a tile is 128 / g consecutive tokens x g consecutive heads, one box per 64-element half.
    const uint64_t pol = l2_policy_evict_first();
    for (int k = 0;; ++k) {
      const int slot = k % kPairInfoSlots, qb = k % kPairQBufs;
      if (k >= kPairInfoSlots) mbar_wait(&info_empty[slot], ((k / kPairInfoSlots) - 1) & 1, ctx, 111);
      const int u = (int)blockIdx.x + k * (int)gridDim.x;
      bool valid = u < nunits && !*ctx.abort;   // after a wait has run out no further unit is started
      valid = __shfl_sync(0xffffffffu, valid, 0);
      if (lane == 0) {
        PairInfo& pi = info[slot];
        pi.valid = valid;
        if (valid) {
          const int2 un = units[u];
          pi.sg[0] = segs[un.x];
          pi.nt = un.y >= 0 ? 2 : 1;
          if (un.y >= 0) pi.sg[1] = segs[un.y];
        }
        __threadfence_block();
        mbar_arrive(&info_full[slot]);
      }
      __syncwarp();
      if (!valid) break;
      if (k >= kPairQBufs) mbar_wait(&q_empty[qb], ((k / kPairQBufs) - 1) & 1, ctx, 112);
      if (lane == 0) {
        const PairInfo& pi = info[slot];
        uint8_t* dst = sQ + qb * 65536;
        mbar_arrive_expect_tx(&q_full[qb], (uint32_t)pi.nt * 32768u);
        for (int tt = 0; tt < pi.nt; ++tt) {
          const SegInfo& sg = pi.sg[tt];
          const int tok = sg.q_tok0 + sg.r0 / P.group;
          tma_load_3d_hint(dst + tt * 16384, &map_q, &q_full[qb], 0, sg.h * P.group, tok, pol);
          tma_load_3d_hint(dst + 32768 + tt * 16384, &map_q, &q_full[qb], 64, sg.h * P.group, tok, pol);
        }
      }
      __syncwarp();
    }
  } else if (warp == 11) {
    // ---------------- selection: threshold, forced blocks, ordered compaction of the tiles of unit `it` ----------------
    for (int it = 0;; ++it) {
      const int slot = it % kPairInfoSlots, eb = it & 1;
      mbar_wait(&info_full[slot], (it / kPairInfoSlots) & 1, ctx, 151);
      const PairInfo& pi = info[slot];
      if (!pi.valid) break;
      mbar_wait(&e_full[eb], (it >> 1) & 1, ctx, 152);
      for (int tt = 0; tt < pi.nt; ++tt) {
        const SegInfo sg = pi.sg[tt];
        const int ncand = sg.J_hi + 1;
        const float* e = sE + (ncand > kMaxBlocks / 2 ? 0 : eb * (kMaxBlocks / 2) + tt * kPairMaxCand);
        float maxE = red[eb][tt][0];
#pragma unroll
        for (int i = 1; i < 8; ++i) maxE = fmaxf(maxE, red[eb][tt][i]);
        // J selected  <=>  E_J >= alpha max E  <=>  e_J >= log2(alpha) + max e   (alpha <= 0 selects everything)
        const float thr = P.alpha > 0.f ? maxE + log2f(P.alpha) : -INFINITY;
        const int win_lo = sg.J_lo - P.window_blocks;
        int pos = 0;
        for (int J0 = 0; J0 < ncand; J0 += 32) {
          const int J = J0 + lane;
          const bool keep = J < ncand && (e[J] >= thr || J < P.sink_blocks || J >= win_lo);
          const unsigned bal = __ballot_sync(0xffffffffu, keep);
          if (keep) blk_idx[sg.off + pos + __popc(bal & ((1u << lane) - 1u))] = J;
          pos += __popc(bal);
        }
        __syncwarp();
        if (lane == 0) {
          seg_count[sg.seg] = pos;
          seg_offset[sg.seg] = sg.off;
          if (sg.seg == P.nseg - 1) seg_offset[P.nseg] = sg.off + ncand;
        }
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&sel_done[eb]);
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else if (warp == 8) {
    // ---------------- producer: kbar pieces of every 128-block chunk (hi then lo, each in its two halves of d) ----------------
    if (lane == 0) {
      tma_prefetch_desc(&map_khi);
      tma_prefetch_desc(&map_klo);
      const uint64_t keep = l2_policy_evict_last();
      uint32_t pc = 0;
      for (int it = 0;; ++it) {
        const int slot = it % kPairInfoSlots;
        mbar_wait(&info_full[slot], (it / kPairInfoSlots) & 1, ctx, 121);
        const PairInfo& pi = info[slot];
        if (!pi.valid) break;
        const int h = pi.sg[0].h, blk_off = pi.sg[0].blk_off;
        const int nchunks = unit_chunks(pi);
        for (int c = 0; c < nchunks; ++c) {
#pragma unroll
          for (int p = 0; p < 4; ++p, ++pc) {
            const int s = pc % kPairPieces;
            if (pc >= kPairPieces) mbar_wait(&empty[s], ((pc / kPairPieces) - 1) & 1, ctx, 122);
            mbar_arrive_expect_tx(&full[s], kPairPieceBytes);
            tma_load_3d_hint(sStage + s * kPairPieceBytes, p < 2 ? &map_khi : &map_klo, &full[s], (p & 1) * 64, h,
                             blk_off + c * 128, keep);
          }
        }
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else if (warp == 9) {
    // ---------------- UMMA issuer: acc[chunk & 1] = kbar_hi Q^T + kbar_lo Q^T over the unit's one or two tiles ----------------
    if (lane == 0) {
      uint32_t pc = 0, ac0 = 0, ac1 = 0, gc0 = 0;   // gc0: chunks of all earlier units
      for (int it = 0;; ++it) {
        const int slot = it % kPairInfoSlots, qb = it % kPairQBufs;
        mbar_wait(&info_full[slot], (it / kPairInfoSlots) & 1, ctx, 131);
        const PairInfo& pi = info[slot];
        if (!pi.valid) break;
        const int nchunks = unit_chunks(pi);
        const uint32_t idesc = make_idesc(128, 128 * pi.nt, 1, 1, 0, 0);
        mbar_wait(&q_full[qb], (it / kPairQBufs) & 1, ctx, 132);
        const uint32_t q_addr = smem_u32(sQ + qb * 65536);
        for (int c = 0; c < nchunks; ++c) {
          const int a = (gc0 + c) & 1;
          uint32_t& ac = a ? ac1 : ac0;
          if (ac >= 1) mbar_wait(&acc_empty[a], (ac - 1) & 1, ctx, 133);
          ++ac;
#pragma unroll
          for (int p = 0; p < 4; ++p, ++pc) {
            const int s = pc % kPairPieces;
            mbar_wait(&full[s], (pc / kPairPieces) & 1, ctx, 134);
            tc_fence_after();
            const uint32_t a_addr = smem_u32(sStage + s * kPairPieceBytes);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t ad = make_smem_desc_sw128(a_addr + ks * 32, 16, 1024);
              const uint64_t bd = make_smem_desc_sw128(q_addr + (p & 1) * 32768 + ks * 32, 16, 1024);
              umma_f16_ss(tmem + a * 256, ad, bd, idesc, (p | ks) != 0);
            }
            umma_commit(&empty[s]);
          }
          umma_commit(&acc_full[a]);
        }
        umma_commit(&q_empty[qb]);
        mbar_arrive(&info_empty[slot]);
        gc0 += nchunks;
      }
    }
  } else {
    // ---------------- consumers: per pooled key and tile, maximum and exponential sum over the tile's rows ----------------
    const int wg = warp >> 2;
    const int key = (warp & 3) * 32 + lane;  // TMEM lane = pooled key within the chunk
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const float cs = P.scale_log2;
    uint32_t uc0 = 0, uc1 = 0;   // uses of the two accumulators
    uint32_t gc0 = 0;  // chunks of all earlier units
    bool prev_big = false;
    for (int it = 0;; ++it) {
      const int slot = it % kPairInfoSlots;
      mbar_wait(&info_full[slot], (it / kPairInfoSlots) & 1, ctx, 141);
      const PairInfo& pi = info[slot];
      if (!pi.valid) break;
      const int nt = pi.nt;
      const int nchunks = unit_chunks(pi);
      const int ncand0 = pi.sg[0].J_hi + 1, ncand1 = nt > 1 ? pi.sg[1].J_hi + 1 : 0;
      const int nrows0 = pi.sg[0].nrows, nrows1 = nt > 1 ? pi.sg[1].nrows : 0;
      // per candidate: log2 of its energy, e_J = m_J + log2(S_J)  (Eq. 1-2 / Eq. 20 in the log domain: the common
      // factor 2^-M of Eq. 20 cancels in the comparison with alpha * max)
      float lmax0 = -INFINITY;
      const int eb = it & 1;
      const bool big = ncand0 > kMaxBlocks / 2;    // a single tile that takes the whole energy buffer
      float* e0 = sE + (big ? 0 : eb * (kMaxBlocks / 2));
      float* e1 = e0 + kPairMaxCand;
      // the part of the energy buffer this unit writes must have been read by the selection of unit it-2, and a unit
      // that takes (or follows one that took) the whole buffer also waits for unit it-1
      if (it >= 2) mbar_wait(&sel_done[eb], ((it >> 1) - 1) & 1, ctx, 143);
      if (it >= 1 && (big || prev_big)) mbar_wait(&sel_done[eb ^ 1], ((it - 1) >> 1) & 1, ctx, 144);
      prev_big = big;
      // Accumulators alternate by a chunk count that runs across units.  In a pair, warpgroup w takes tile w of
      // every chunk, and both hand the accumulator back as soon as their columns are in registers, so the MMAs of
      // the chunk after next start at once.  In a single-tile unit the warpgroups alternate over the chunks (the
      // one whose turn it is not only passes the accumulator on).
      for (int c = 0; c < nchunks; ++c) {
        const int a = (int)((gc0 + (uint32_t)c) & 1u);
        uint32_t& ua = a ? uc1 : uc0;
        mbar_wait(&acc_full[a], ua & 1, ctx, 142);
        ++ua;
        tc_fence_after();
        const int J = c * 128 + key;
        float m, sum;
        if (nt > 1) {
          const uint32_t lane_addr = lane_base + a * 256 + wg * 128;
          const int nrows = wg ? nrows1 : nrows0;
          if (nrows == kTileRows) score_cols<false>(lane_addr, cs, kTileRows, &acc_empty[a], m, sum);
          else score_cols<true>(lane_addr, cs, nrows, &acc_empty[a], m, sum);
          if (J < (wg ? ncand1 : ncand0)) {
            const float e = m + log2f(sum);
            (wg ? e1 : e0)[J] = e;
            lmax0 = fmaxf(lmax0, e);
          }
        } else if (a == wg) {
          if (nrows0 == kTileRows) score_cols<false>(lane_base + a * 256, cs, kTileRows, &acc_empty[a], m, sum);
          else score_cols<true>(lane_base + a * 256, cs, nrows0, &acc_empty[a], m, sum);
          if (J < ncand0) {
            const float e = m + log2f(sum);
            e0[J] = e;
            lmax0 = fmaxf(lmax0, e);
          }
        } else {
          mbar_arrive(&acc_empty[a]);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lmax0 = fmaxf(lmax0, __shfl_xor_sync(0xffffffffu, lmax0, o));
      // hand the unit to the selection warp and go on: in a pair the warps of warpgroup w hold maxima of tile w
      if (lane == 0) {
        const int tt = nt > 1 ? wg : 0;
        red[eb][tt][warp] = lmax0;
        red[eb][tt ^ 1][warp] = -INFINITY;
      }
      __syncwarp();
      mbar_arrive(&e_full[eb]);
      mbar_arrive(&info_empty[slot]);
      gc0 += (uint32_t)nchunks;
    }
  }
  if (abort_flag) {   // MMAs and bulk copies may still be in flight: let them finish before tensor memory goes
    if (warp == 9 && lane == 0) {
      umma_commit(&drain_bar);
      mbar_wait_drain(&drain_bar, 0, 200000000ll);
    }
    __nanosleep(2000000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, 512);
}

}  // namespace fp2
