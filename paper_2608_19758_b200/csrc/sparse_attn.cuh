// Block-sparse causal flash attention with mean correction (Eq. 4, Eq. 6; Algorithm 1 lines 6-11),
// persistent, warp-specialised, tcgen05 / TMEM / TMA.  The same kernel runs the dense path (implicit list
// 0..J_hi, no correction).
//
// CTAs loop over work units (sequence, KV head, packed query tile) taken from a work order (KV-head-major,
// heaviest first) through a global counter.  For a unit with selected list idx[0..T) the iteration sequence
// is the list traversed backwards (Eq. 17) followed by the non-empty correction chunks: a correction chunk
// stages 128 consecutive pooled (kbar, vbar) rows exactly like a KV block, its logits are shifted by log2(128)
// (every corrected block is full) and masked by todo = fully-visible & ~selected.
//
// TWO small CTAs per SM.  Per 128x128 block the tensor pipe (two GEMMs) and the MUFU pipe (16384
// exponentials) are each busy 1024 cycles, and a softmax step has several hundred cycles of latency around its
// exponentials (TMEM load, row maximum, TMEM store, barrier hand-overs).  Two warpgroups that share one tile must
// exchange row maxima and so move in lockstep: both are in their latency phase at the same time and the MUFU
// pipe idles (that layout, one CTA of 12 warps per SM, measured 42-48 % tensor-pipe activity on the dense
// path; this one 59 %).  Here every CTA has ONE softmax warpgroup that owns whole rows (thread = row, 128 logits
// in registers), nothing crosses between the two CTAs of an SM, and they drift out of phase by themselves: while
// one CTA's warps stream exponentials the other's wait for the tensor pipe, load logits or hand over P.
//
// One CTA: 256 threads, 96 KB of tile memory (Q, one K stage, one V stage), 256 TMEM columns:
//   S [0,128)  logits of the iteration; P (16-bit pairs) overwrites its first 64 columns in place
//   O [128,256)
// Everything is single-buffered: S = Q K^T of iteration i+1 is issued behind O += P V of iteration i (which
// reads P out of the S columns), the K tile of i+1 is requested when S = Q K^T (i) has completed and the V tile
// when O += P V (i) has.  The other CTA of the SM fills the bubbles this leaves.  P is handed to the issuer in
// kPParts column slices, so O += P V runs its first k-steps under the remaining exponentials.
//
// Roles: warps 0..3 softmax + epilogue; warp 4 TMA producer (Eq. 22); warp 5 UMMA issuer (and TMEM owner);
// warps 6, 7 unit set-up (fetch the next unit, validate its list, build the correction masks, stage Q).
//
// FP8 inputs (Eq. 15; template parameter FP8): S = Q K^T runs as a kind::f8f6f4 MMA straight on the raw e4m3
// tiles (Q and K both K-major, 128-byte rows, as cp.async / TMA write them), at twice the BF16 rate.  The
// probabilities stay 16-bit -- a single e4m3 probability tile costs ~0.06 max-abs output error by itself -- so
// O += P V is a kind::f16 MMA on F16 operands: P packed as F16, V widened (exactly) from its raw e4m3 tile into
// the F16 V stage by the softmax warpgroup itself at the top of the iteration.  The per-head scales never touch
// the operands: q_scale * k_scale multiplies the logits of a row, v_scale multiplies the output.  Correction
// chunks: the pooled keys come as an e4m3 hi + lo pair in raw units (two accumulating MMA groups, ~8 mantissa
// bits together), the pooled values as F16.  Tile memory: Q 16 KB, K 32 KB (one raw tile, or hi | lo of a
// chunk), raw V 16 KB, F16 V 32 KB.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"
#include "ptx.cuh"
#include "score_select.cuh"  // load_q_tile_async
#include "split_kv.cuh"

namespace fp2 {

constexpr int kTileBytes = 32768;   // one 128 x 128 tile of 16-bit elements
constexpr int kRawBytes = 16384;    // one 128 x 128 tile of FP8 elements as TMA delivers it

struct TileInfo {
  SegInfo sg;
  int32_t valid;     // 0: no more work
  int32_t T;         // exact iterations (listed blocks)
  int32_t nchunk;    // non-empty correction chunks
  int32_t ndiag;     // listed blocks J >= J_lo: the first ndiag iterations (the list is traversed backwards)
  int32_t dense;
  int32_t it_begin, it_end;   // this unit's part of the iteration sequence [0, T + nchunk) (Eq. 18); all of it unless split
  int32_t parts;              // parts the segment is split into (1: the unit writes the final output)
  int32_t slot;               // partial-result slot of this unit when parts > 1
  int32_t chunk_id[kMaxChunks];
  uint32_t todo[kMaxChunks][4];
};

struct AttnArgs {
  const uint8_t* q;
  const int32_t* page_table;
  const SegInfo* segs;
  const int32_t* order;      // work order
  const int32_t* seg_count;  // NULL => dense
  const int32_t* blk_idx;
  const float* q_scale;
  const float* k_scale;
  const float* v_scale;
  __nv_bfloat16* out;
  float* lse;
  int* work_counter;
  int* status;
  // KV splitting (Eq. 18).  unit_split == NULL: one unit per segment, `order` lists the segments.  Otherwise
  // `order` lists the segment of every unit, unit_split its part (see pack_split), *n_units their number, and a
  // unit of a split segment leaves (O, m, l) unnormalised in part_o [slot][128][128] / part_ml [slot][128].
  const int32_t* unit_split;
  const int32_t* n_units;
  float* part_o;
  float2* part_ml;
#ifdef FP2_PROFILE
  long long* prof;   // [grid][16] cycle counters of the softmax warpgroup (development builds only)
#endif
};

#ifdef FP2_PROFILE
#define PF_BEGIN() pf_a = clock64()
#define PF_END(k) (pf_b = clock64(), pf[k] += pf_b - pf_a, pf_a = pf_b)
#else
#define PF_BEGIN()
#define PF_END(k)
#endif

constexpr int kPParts = 4;   // P is handed to the issuer in this many column slices (4 or 8)

template <bool FP8>
struct AttnCfg {
  static constexpr int kThreads = 256;
  static constexpr int kCtasPerSm = 2;
  static constexpr int kBiasBytes = 4096;                    // one 128 x 32 e5m2 operand without swizzle
  static constexpr int kSmemBytes = 1024 + 3 * kTileBytes + 2 * kBiasBytes;   // both dtypes: 96 KB of tiles + the mask operands
  // Registers: two CTAs share the file, 128 per thread at launch; setmaxnreg moves them from the service warps
  // to the softmax warps.  The move waits without bound for registers the CTA does not own, so the sum is
  // checked here and the compiled register count is checked on the host before the first launch.
  static constexpr int kRegsBase = 128;
  static constexpr int kRegsService = 56;
  static constexpr int kRegsSoftmax = 200;
  static constexpr int kRegsAfterMove = (kThreads - 128) * kRegsService + 128 * kRegsSoftmax;
  static_assert(kRegsAfterMove <= kThreads * kRegsBase, "register budget: setmaxnreg.inc would wait forever");
  static_assert(kThreads * kRegsBase * kCtasPerSm <= 65536, "two CTAs must fit the register file");
};

// Masked iterations (diagonal blocks, correction chunks -- the minority): overwrite the hidden logits of this
// thread's row with -inf in TMEM, so that the softmax step itself carries no mask logic.  Column j stays
// visible iff j <= tok_lim and bit j of the 128-bit mask (32 bits per word) is set.  Not inlined: it is off the
// common path and four times 32 unrolled selects are a lot of code.
__device__ __noinline__ void mask_row(uint32_t s_addr, int tok_lim, uint32_t cm0, uint32_t cm1, uint32_t cm2,
                                      uint32_t cm3) {
#pragma unroll 1
  for (int k = 0; k < 4; ++k) {
    const uint32_t cmk = k == 0 ? cm0 : k == 1 ? cm1 : k == 2 ? cm2 : cm3;
    const bool all_vis = (k * 32 + 31 <= tok_lim) && (cmk == 0xffffffffu);
    if (__all_sync(0xffffffffu, all_vis)) continue;   // TMEM accesses are warp-wide: decide per warp
    uint32_t rr[32];
    tmem_ld32(s_addr + k * 32, rr);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const bool vis = (k * 32 + j <= tok_lim) && ((cmk >> j) & 1u);
      rr[j] = vis ? rr[j] : 0xff800000u;  // -inf
    }
    tmem_st32(s_addr + k * 32, rr);
  }
  tmem_wait_st();
}

// The thread's whole logit row (raw, unscaled) into registers, and its maximum: all four TMEM loads in flight,
// chains of three-input maxima.
__device__ __forceinline__ float row_load_max(uint32_t s_addr, uint32_t (&x)[128]) {
#pragma unroll
  for (int k = 0; k < 4; ++k) tmem_ld32(s_addr + k * 32, reinterpret_cast<uint32_t(&)[32]>(x[k * 32]));
  tmem_wait_ld();
  float mx8[16];
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    const float* v = reinterpret_cast<const float*>(&x[c * 8]);
    mx8[c] = fmaxf(max3(max3(v[0], v[1], v[2]), v[3], v[4]), max3(v[5], v[6], v[7]));
  }
#pragma unroll
  for (int c = 0; c < 5; ++c) mx8[c] = max3(mx8[3 * c], mx8[3 * c + 1], mx8[3 * c + 2]);
  return fmaxf(max3(mx8[0], mx8[1], mx8[2]), max3(mx8[3], mx8[4], mx8[15]));
}

// p = 2^(x * cs + neg_m) for the 128 logits in registers, written as BF16 (F16) pairs to the 64 columns at p_addr.
// Scaling and row sum use packed fp32x2 instructions.  After the first 64 probabilities the thread arrives on
// half_ready.  Returns the row sum.
template <bool F16>
__device__ __forceinline__ float row_exp(const uint32_t (&x)[128], uint32_t p_addr, float cs, float neg_m,
                                         uint64_t* part_ready) {
  const uint64_t cs2 = f2_pack(cs, cs), nm2 = f2_pack(neg_m, neg_m);
  uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};   // four independent (lo, hi) accumulators, +0.0f bit patterns
#pragma unroll
  for (int k = 0; k < kPParts; ++k) {
    constexpr int W = 64 / kPParts;   // packed registers (= P columns) per part
    uint32_t pk[W];
#pragma unroll
    for (int j = 0; j < W; ++j) {
      const int c = k * 2 * W + 2 * j;
      const uint64_t x2 = f2_fma(f2_pack(__uint_as_float(x[c]), __uint_as_float(x[c + 1])), cs2, nm2);
      float x0, x1;
      f2_unpack(x2, x0, x1);
      const float p0 = ex2(x0), p1 = ex2(x1);
      sum2[j & 3] = f2_add(sum2[j & 3], f2_pack(p0, p1));
      pk[j] = F16 ? pack_f16x2(p0, p1) : pack_bf16x2(p0, p1);
    }
    tmem_st_cols(p_addr + k * W, pk);
    if (k + 1 < kPParts) {   // a part of P: O += P V may run its next k-steps
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&part_ready[k]);
    }
  }
  float a0, a1;
  f2_unpack(f2_add(f2_add(sum2[0], sum2[1]), f2_add(sum2[2], sum2[3])), a0, a1);
  return a0 + a1;
}

// map_kbar / map_kbar_lo: pooled keys of the correction chunks -- BF16: one BF16 array (map_kbar_lo unused);
// FP8: the e4m3 hi and lo arrays.  map_vbar: pooled values, 16-bit.  map_q: packed query tiles (DevParams::q_tma).
template <bool FP8>
__global__ void __launch_bounds__(AttnCfg<FP8>::kThreads, AttnCfg<FP8>::kCtasPerSm)
sparse_attn_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const __grid_constant__ CUtensorMap map_kbar, const __grid_constant__ CUtensorMap map_kbar_lo,
                    const __grid_constant__ CUtensorMap map_vbar, const __grid_constant__ CUtensorMap map_q,
                    AttnArgs A, DevParams P) {
  constexpr int kSetupThreads = 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                                  // 32 KB (BF16) / 16 KB (raw e4m3)
  uint8_t* sK = smem + (FP8 ? kRawBytes : kTileBytes); // 32 KB
  uint8_t* sV = sK + kTileBytes;                       // 32 KB, 16-bit
  uint8_t* sVraw = sV + kTileBytes;                    // FP8 only: 16 KB raw e4m3 V tile
  (void)sVraw;
  // Masks enter the logits through the tensor core: one more k-step S += hot . bias^T (kind::f8f6f4, e5m2 x e5m2,
  // K = 32), which costs 64 cycles of the tensor pipe instead of a TMEM round trip of the softmax warpgroup.
  //   sHot [128 rows x 32]: row i holds 57344 (the largest e5m2) in column c(i) and zeros elsewhere, c(i) = the
  //     row's position minus the tile's first position (Eq. 13: floor((r0 + i) / g) - floor(r0 / g)); written by the
  //     set-up warps with the query tile.  Group sizes with more than 32 positions per tile (g < 4) use i mod 32.
  //   sBias [128 columns x 32], written by the producer warp per masked iteration:
  //     diagonal block: bias[j][c] = -57344 where column j is hidden from position c (j > t0 + c), else 0;
  //     correction chunk: bias[j][c] = -57344 for every c where block j is not to be corrected (selected, or past
  //       the fully visible range), else 0 -- the todo mask is the same for all rows.
  // A hidden logit thus carries -3.3e9 (raw units), which the exponential turns into an exact zero.
  // Both operands are K-major without swizzle: 8-row x 16-byte core matrices, row r at (r / 8) * 256 + (r % 8) * 16,
  // bytes 16..31 of the row 128 bytes further.
  uint8_t* sHot = smem + 3 * kTileBytes;
  uint8_t* sBias = sHot + AttnCfg<FP8>::kBiasBytes;

  __shared__ TileInfo info[2];
  __shared__ uint32_t sel_bits[kMaxBlocks / 32];
  __shared__ uint64_t info_full[2], info_empty[2], q_full, q_empty;
  // Every barrier below completes exactly once per iteration; with G the iteration's index counted over the
  // whole kernel, the phase that belongs to iteration G has parity G & 1.
  __shared__ uint64_t k_full, v_full;
  __shared__ uint64_t s_done;    // S = Q K^T (G) has completed: the logits are in TMEM, the K stage is free --
                                 // and, MMAs completing in issue order, O += P V (G-1) is in O
  __shared__ uint64_t pv_done[2];  // [G & 1], phase (G >> 1) & 1: O += P V (G) has completed -- the V stage is free,
                                   // O holds iteration G.  Two barriers so that a waiter may be two iterations
                                   // behind the issuer without mistaking one phase for another.
  __shared__ uint64_t vraw_full, vraw_empty;   // FP8: the raw V tile has landed / has been widened
  __shared__ uint64_t p_ready[kPParts];   // slice q (128 / kPParts probabilities of every row) of P (G) is in TMEM
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ int ndiag_s;
  __shared__ uint64_t drain_bar;   // teardown after an abort: every MMA issued by this CTA has completed

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  WaitCtx ctx{A.status, &abort_flag};

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(&info_full[i], 1);
      mbar_init(&info_empty[i], 2 + 128);   // producer, issuer, softmax threads
    }
    mbar_init(&q_full, kSetupThreads);
    mbar_init(&vraw_full, 1);
    mbar_init(&vraw_empty, 1);
    mbar_init(&q_empty, 1);
    mbar_init(&k_full, 1);
    mbar_init(&v_full, 1);
    mbar_init(&s_done, 1);
    mbar_init(&pv_done[0], 1);
    mbar_init(&pv_done[1], 1);
    mbar_init(&drain_bar, 1);
    for (int i = 0; i < kPParts; ++i) mbar_init(&p_ready[i], 128);
    fence_barrier_init();
  }
  // K / V stages start zeroed: rows of pages past the end of a sequence are never loaded, and whatever sits
  // there is multiplied by probabilities that are exactly zero, so it must be finite.
  for (int i = tid; i < (2 * kTileBytes + (FP8 ? kRawBytes : 0)) / 16; i += AttnCfg<FP8>::kThreads)
    reinterpret_cast<uint4*>(sK)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 5) {
    tmem_alloc(&tmem_base_s, 256);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const int g = P.group;

  // O += P V (G) has completed.  Safe for a waiter that is at most two iterations behind the issuer.
  auto wait_pv = [&](uint32_t G, int where) { mbar_wait(&pv_done[G & 1], (G >> 1) & 1, ctx, where); };

  if (warp >= 6) {
    // =============================== unit set-up + Q staging ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    const int t64 = tid - 32 * 6;
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      if (it >= 2) mbar_wait(&info_empty[slot], ((it >> 1) - 1) & 1, ctx, 201);
      TileInfo& ti = info[slot];
      if (t64 == 0) {
        const int w = atomicAdd(A.work_counter, 1);
        const int n_units = A.unit_split ? *A.n_units : P.nseg;
        // after a wait has run out somewhere in this CTA no further unit is started: the terminating descriptor
        // makes every role leave its loop the ordinary way
        if (w < n_units && !*ctx.abort) {
          const int seg = A.order[w];
          const int32_t split = A.unit_split ? A.unit_split[w] : pack_split(0, 1, 0);
          ti.parts = (split >> 8) & 0xff;
          ti.slot = ((split >> 16) & 0xffff) + (split & 0xff);
          ti.it_begin = split & 0xff;   // the part index for now; turned into a range once T + nchunk is known
          ti.sg = A.segs[seg];
          ti.valid = 1;
          ti.dense = (A.seg_count == nullptr);
          int T = ti.dense ? ti.sg.J_hi + 1 : A.seg_count[seg];
          if (T < 0 || T > ti.sg.J_hi + 1) {  // malformed count: clamp so every loop stays bounded
            atomicOr(A.status + ST_BAD_LIST, 1);
            T = max(0, min(T, ti.sg.J_hi + 1));
          }
          ti.T = T;
          ti.nchunk = 0;
          ti.ndiag = ti.dense ? min(T, ti.sg.J_hi - ti.sg.J_lo + 1) : 0;
          ndiag_s = 0;
        } else {
          ti.valid = 0;
        }
      }
      named_bar_sync(2, kSetupThreads);
      const bool valid = ti.valid != 0;
      if (valid && !ti.dense) {
        const SegInfo& sg = ti.sg;
        const int32_t* list = A.blk_idx + sg.off;
        const int T = ti.T;
        const int nwords = (sg.J_lo + 31) >> 5;
        const bool corr = P.use_correction != 0;
        if (corr)
          for (int w = t64; w < nwords; w += kSetupThreads) sel_bits[w] = 0u;
        named_bar_sync(2, kSetupThreads);
        bool bad = false;
        int nd = 0;
        for (int k = t64; k < T; k += kSetupThreads) {
          const int J = list[k];
          if (J < 0 || J > sg.J_hi || (k > 0 && list[k - 1] >= J)) bad = true;
          if (corr && J >= 0 && J < sg.J_lo) atomicOr(&sel_bits[J >> 5], 1u << (J & 31));
          nd += J >= sg.J_lo;
        }
        if (bad) atomicOr(A.status + ST_BAD_LIST, 1);
        if (nd) atomicAdd(&ndiag_s, nd);
        named_bar_sync(2, kSetupThreads);
        if (t64 == 0) ti.ndiag = ndiag_s;
        if (corr) {
          const int nch = (sg.J_lo + 127) >> 7;
          for (int c = t64; c < nch; c += kSetupThreads) {
#pragma unroll
            for (int w = 0; w < 4; ++w) {
              const int first = c * 128 + w * 32;
              uint32_t validm = 0u;
              if (first + 32 <= sg.J_lo) validm = 0xffffffffu;
              else if (first < sg.J_lo) validm = (1u << (sg.J_lo - first)) - 1u;
              ti.todo[c][w] = (first < sg.J_lo ? ~sel_bits[first >> 5] : 0u) & validm;
            }
          }
          named_bar_sync(2, kSetupThreads);
          if (t64 == 0) {
            int n = 0;
            for (int c = 0; c < nch; ++c)
              if (ti.todo[c][0] | ti.todo[c][1] | ti.todo[c][2] | ti.todo[c][3]) ti.chunk_id[n++] = c;
            ti.nchunk = n;
          }
        }
      }
      named_bar_sync(2, kSetupThreads);
      if (t64 == 0 && valid) {   // Eq. 18: part u of U takes iterations [u ceil(n / U), min((u + 1) ceil(n / U), n))
        const int n = ti.T + ti.nchunk, u = ti.it_begin;
        const int step = (n + ti.parts - 1) / ti.parts;
        ti.it_begin = min(u * step, n);
        ti.it_end = min((u + 1) * step, n);
      }
      named_bar_sync(2, kSetupThreads);
      if (t64 == 0) mbar_arrive(&info_full[slot]);
      if (!valid) break;
      // Q tile: wait until every S = Q K^T of the previous unit has completed, then overwrite
      if (it >= 1) mbar_wait(&q_empty, (it - 1) & 1, ctx, 202);
      {   // sHot: rows 2 t64 and 2 t64 + 1
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int row = 2 * t64 + u;
          const int c = P.diag_mma ? (ti.sg.r0 + row) / g - ti.sg.r0 / g : (row & 31);
          uint32_t w[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
          for (int k = 0; k < 8; ++k) w[k] = (c >> 2) == k ? 0x7bu << ((c & 3) * 8) : 0u;   // e5m2 57344
          uint8_t* dst = sHot + (row >> 3) * 256 + (row & 7) * 16;
          *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(dst + 128) = make_uint4(w[4], w[5], w[6], w[7]);
        }
        fence_proxy_async();
      }
      if (P.q_tma) {
        // PackGQA (Eq. 13) with a group size that divides 128: the tile is 128 / g tokens x g heads, one TMA box
        // per 128 bytes of a row (two 64-element halves for BF16, the whole row for e4m3), landing in the swizzled
        // layout the MMA reads.  Rows past the end of a short last tile get whatever follows; nothing reads them.
        if (t64 == 0) {
          const SegInfo& sg = ti.sg;
          const uint64_t pol = l2_policy_evict_first();
          mbar_arrive_expect_tx(&q_full, FP8 ? kRawBytes : kTileBytes);
          tma_load_3d_hint(sQ, &map_q, &q_full, 0, sg.h * g, sg.q_tok0 + sg.r0 / g, pol);
          if constexpr (!FP8)
            tma_load_3d_hint(sQ + 16384, &map_q, &q_full, 64, sg.h * g, sg.q_tok0 + sg.r0 / g, pol);
        } else {
          mbar_arrive(&q_full);
        }
        continue;
      }
      if constexpr (FP8) {
        load_q_raw_async(sQ, A.q, ti.sg, P, t64, kSetupThreads);
        cp_async_wait_all();
      }
      else load_q_tile_async(sQ, A.q, ti.sg, P, t64, kSetupThreads);
      fence_proxy_async();
      mbar_arrive(&q_full);
    }
  } else if (warp == 4) {
    // =============================== TMA producer ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    if (lane == 0) {
      tma_prefetch_desc(&map_k);
      tma_prefetch_desc(&map_v);
      tma_prefetch_desc(&map_kbar);
      tma_prefetch_desc(&map_vbar);
    }
    uint32_t G = 0, rc = 0;
    (void)rc;
    const uint64_t keep = l2_policy_evict_last();   // K / V pages and pooled means: shared by many tiles
    const int ppb = P.pages_per_block, psz = P.page_size;
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 301);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const SegInfo& sg = ti.sg;
      const int T = ti.T;
      const int32_t* list = A.blk_idx + sg.off;
      const int32_t* pt = A.page_table + (size_t)sg.b * P.max_pages_per_seq;
      // page id of this lane's page of exact iteration i (-1: past the end of the sequence, or not an exact
      // iteration).  Fetched one iteration ahead: list entry -> page-table entry are two dependent global loads.
      int J_fetched = 0;   // block id of the iteration fetch_pid was last asked for (warp-uniform)
      auto fetch_pid = [&](int i) -> int {
        if (i >= T) return -1;
        int J = ti.dense ? sg.J_hi - i : list[T - 1 - i];
        J = max(0, min(J, sg.J_hi));
        J_fetched = J;
        if (lane >= ppb) return -1;
        if (J * kBlock + lane * psz >= sg.Lk) return -1;
        int pid = pt[J * ppb + lane];
        if (pid < 0 || pid >= P.num_pages) {
          atomicOr(A.status + ST_BAD_LIST, 2);
          pid = -1;
        }
        return pid;
      };
      // hidden columns of a masked iteration -> sBias (see there); row j = lane * 4 + u gets 32 bytes of which the
      // first nh[u] are -57344 (e5m2 0xfb).  The S = Q K^T that last read sBias has completed (wait 302).
      auto write_bias = [&](const int (&nh)[4]) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = lane * 4 + u;
          uint32_t w[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int n = nh[u] - 4 * k;   // hidden bytes in this word
            w[k] = n >= 4 ? 0xfbfbfbfbu : n <= 0 ? 0u : (0xfbfbfbfbu >> (32 - 8 * n));
          }
          uint8_t* dst = sBias + (j >> 3) * 256 + (j & 7) * 16;
          *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(dst + 128) = make_uint4(w[4], w[5], w[6], w[7]);
        }
        fence_proxy_async();
        __syncwarp();
      };
      int pid_next = fetch_pid(ti.it_begin);
      for (int i = ti.it_begin; i < ti.it_end; ++i, ++G) {
        const int pid = pid_next;
        const int J_cur = J_fetched;
        pid_next = fetch_pid(i + 1);
        if (G >= 1) mbar_wait(&s_done, (G - 1) & 1, ctx, 302);   // K stage free
        if (i < ti.ndiag && P.diag_mma) {
          // diagonal block: column j is hidden from the tile's position c iff J * 128 + j > pre + r0 / g + c
          const int t0 = sg.pre + sg.r0 / g - J_cur * kBlock;
          int nh[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) nh[u] = max(0, min(32, lane * 4 + u - t0));
          write_bias(nh);
        }
        if (i < T) {
          const int nvalid = __popc(__ballot_sync(0xffffffffu, pid >= 0));
          if constexpr (FP8) {
            // raw e4m3 tiles, 128 bytes per token row: K straight into the K stage (the MMA reads it as it
            // lands), V into the raw slot for the widening warp
            const uint32_t bytes = (uint32_t)nvalid * psz * 128u;
            if (lane == 0) mbar_arrive_expect_tx(&k_full, bytes);
            __syncwarp();
            if (pid >= 0) tma_load_3d_hint(sK + lane * psz * 128, &map_k, &k_full, 0, sg.h, pid * psz, keep);
            if (rc >= 1) mbar_wait(&vraw_empty, (rc - 1) & 1, ctx, 306);
            if (lane == 0) mbar_arrive_expect_tx(&vraw_full, bytes);
            __syncwarp();
            if (pid >= 0) tma_load_3d_hint(sVraw + lane * psz * 128, &map_v, &vraw_full, 0, sg.h, pid * psz, keep);
            ++rc;
          } else {
            const uint32_t bytes = (uint32_t)nvalid * psz * 256u;
            if (lane == 0) mbar_arrive_expect_tx(&k_full, bytes);
            __syncwarp();
            if (pid >= 0) {
              tma_load_3d_hint(sK + lane * psz * 128, &map_k, &k_full, 0, sg.h, pid * psz, keep);
              tma_load_3d_hint(sK + 16384 + lane * psz * 128, &map_k, &k_full, 64, sg.h, pid * psz, keep);
            }
            if (G >= 1) wait_pv(G - 1, 303);  // V stage free
            if (lane == 0) mbar_arrive_expect_tx(&v_full, bytes);
            __syncwarp();
            if (pid >= 0) {
              tma_load_3d_hint(sV + lane * psz * 128, &map_v, &v_full, 0, sg.h, pid * psz, keep);
              tma_load_3d_hint(sV + 16384 + lane * psz * 128, &map_v, &v_full, 64, sg.h, pid * psz, keep);
            }
          }
        } else {
          const int cid = ti.chunk_id[i - T];
          const int row0 = sg.blk_off + cid * 128;
          {
            const uint32_t w = ti.todo[cid][lane >> 3];
            int nh[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) nh[u] = ((w >> ((lane * 4 + u) & 31)) & 1u) ? 0 : 32;
            write_bias(nh);
          }
          if (lane == 0) {
            mbar_arrive_expect_tx(&k_full, kTileBytes);
            if constexpr (FP8) {   // e4m3 hi | lo, 16 KB each
              tma_load_3d_hint(sK, &map_kbar, &k_full, 0, sg.h, row0, keep);
              tma_load_3d_hint(sK + 16384, &map_kbar_lo, &k_full, 0, sg.h, row0, keep);
            } else {
              tma_load_3d_hint(sK, &map_kbar, &k_full, 0, sg.h, row0, keep);
              tma_load_3d_hint(sK + 16384, &map_kbar, &k_full, 64, sg.h, row0, keep);
            }
          }
          if (G >= 1) wait_pv(G - 1, 305);    // V stage free
          if (lane == 0) {
            mbar_arrive_expect_tx(&v_full, kTileBytes);
            tma_load_3d_hint(sV, &map_vbar, &v_full, 0, sg.h, row0, keep);
            tma_load_3d_hint(sV + 16384, &map_vbar, &v_full, 64, sg.h, row0, keep);
          }
          __syncwarp();
        }
      }
      if (lane == 0) mbar_arrive(&info_empty[slot]);
    }
  } else if (warp == 5) {
    // =============================== UMMA issuer ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    if (lane == 0) {
      constexpr int kFmt = FP8 ? 0 : 1;   // kind::f16 operand format of O += P V: 0 = F16, 1 = BF16
      constexpr uint32_t idesc_qk = FP8 ? make_idesc(128, 128, 0, 0, 0, 0)    // kind::f8f6f4, E4M3 x E4M3
                                        : make_idesc(128, 128, 1, 1, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(128, 128, kFmt, kFmt, 0, 1);
      const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
      uint32_t G = 0;
      for (int it = 0;; ++it) {
        const int slot = it & 1;
        mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 403);
        const TileInfo& ti = info[slot];
        if (!ti.valid) break;
        const int T = ti.T;
        (void)T;
        mbar_wait(&q_full, it & 1, ctx, 404);
        const int i0 = ti.it_begin, i1 = ti.it_end;
        for (int i = i0; i < i1; ++i, ++G) {
          // S = Q K^T (G).  The S columns are free: O += P V (G-1), which read P out of them, was issued before.
          mbar_wait(&k_full, G & 1, ctx, 405);
          tc_fence_after();
          if constexpr (FP8) {
            // raw e4m3 operands, 32 elements (= 32 bytes of the swizzled row) per MMA; a correction chunk adds
            // the lo part of the pooled keys on top of the hi part
            const int parts = i < T ? 1 : 2;
            for (int part = 0; part < parts; ++part) {
#pragma unroll
              for (int ks = 0; ks < 4; ++ks) {
                const uint64_t ad = make_smem_desc_sw128(q_addr + ks * 32, 16, 1024);
                const uint64_t bd = make_smem_desc_sw128(k_addr + part * 16384 + ks * 32, 16, 1024);
                umma_f8_ss(tmem, ad, bd, idesc_qk, (part > 0) || ks > 0);
              }
            }
          } else {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
              const uint64_t ad = make_smem_desc_sw128(q_addr + off, 16, 1024);
              const uint64_t bd = make_smem_desc_sw128(k_addr + off, 16, 1024);
              umma_f16_ss(tmem, ad, bd, idesc_qk, ks > 0);
            }
          }
          if (i >= T || (i < ti.ndiag && P.diag_mma)) {   // masked iteration: the mask as one more k-step (see sBias)
            constexpr uint32_t idesc_bias = make_idesc(128, 128, 1, 1, 0, 0);   // e5m2 x e5m2
            umma_f8_ss(tmem, make_smem_desc_plain(smem_u32(sHot), 128, 256),
                       make_smem_desc_plain(smem_u32(sBias), 128, 256), idesc_bias, 1u);
          }
          umma_commit(&s_done);
          if (i == i1 - 1) umma_commit(&q_empty);
          // O += P V (G)
          mbar_wait(&v_full, G & 1, ctx, 402);
#pragma unroll
          for (int h = 0; h < kPParts; ++h) {   // as each slice of P arrives
            mbar_wait(&p_ready[h], G & 1, ctx, 401);
            tc_fence_after();
#pragma unroll
            for (int ks = (8 / kPParts) * h; ks < (8 / kPParts) * (h + 1); ++ks) {
              const uint64_t bd = make_smem_desc_sw128(v_addr + ks * 2048, 16384, 1024);
              umma_f16_ts(tmem + 128, tmem + ks * 8, bd, idesc_pv, (i > i0) || ks > 0);
            }
          }
          umma_commit(&pv_done[G & 1]);
        }
        if (i1 == i0) umma_commit(&q_empty);  // nothing to do for this unit: nothing read Q, release it at once
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else {
    // =============================== softmax warpgroup + epilogue ===============================
    setmaxnreg_inc<AttnCfg<FP8>::kRegsSoftmax>();
    const int row = warp * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t s_addr = lane_base;         // S; P overwrites its first 64 columns
    const uint32_t o_addr = lane_base + 128;
    uint32_t G = 0, rc = 0;   // rc: exact iterations so far (uses of the raw V slot)
    (void)rc;
    const uint64_t stream_pol = l2_policy_evict_first();   // outputs are written once and not read here
#ifdef FP2_PROFILE
    long long pf[16];
    for (int i = 0; i < 16; ++i) pf[i] = 0;
    const long long pf_t0 = clock64();
    long long pf_a, pf_b;
#endif
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      PF_BEGIN();
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 501);
      PF_END(0);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const int T = ti.T;
      const bool dense = ti.dense != 0;
      const int J_hi = ti.sg.J_hi, J_lo = ti.sg.J_lo;
      const int32_t* list = A.blk_idx + ti.sg.off;
      const int r = ti.sg.r0 + row;
      const int pos = ti.sg.pre + r / g;
      // logit multiplier in log2 units.  FP8 (Eq. 15): the MMAs see raw e4m3 values (pooled keys included), so
      // every logit of a row carries q_scale * k_scale; the output carries v_scale.
      float cs_all = P.scale_log2, out_scale = 1.0f;
      if constexpr (FP8) {
        cs_all *= A.q_scale[ti.sg.h * g + r % g] * A.k_scale[ti.sg.h];
        out_scale = A.v_scale[ti.sg.h];
      }
      // The mask bias is -3.3e9 in raw units; with FP8 scales so small that this is no longer far below every
      // visible logit of the row, the warp masks in TMEM as well.
      bool weak_bias = false;
      if constexpr (FP8) weak_bias = __any_sync(0xffffffffu, !(cs_all * 3.0e9f > 256.f));
      float m = -INFINITY, l = 0.f;
      // block id of the next exact iteration, fetched one iteration ahead
      const int i0 = ti.it_begin, i1 = ti.it_end;
      int J_next = (!dense && i0 < T) ? list[T - 1 - i0] : 0;
      for (int i = i0; i < i1; ++i, ++G) {
        // iteration kind and masks
        bool need_mask = false;
        int tok_lim = 1 << 30;     // exact block: columns j with j <= tok_lim are visible
        uint32_t cm0 = 0xffffffffu, cm1 = 0xffffffffu, cm2 = 0xffffffffu, cm3 = 0xffffffffu;
        float shift = 0.f;
        if (i < T) {
          int J = dense ? J_hi - i : J_next;
          if (!dense && i + 1 < T) J_next = list[T - 2 - i];
          J = max(0, min(J, J_hi));
          need_mask = J >= J_lo && (!P.diag_mma || weak_bias);   // else the causal mask is in the logits already
          tok_lim = pos - J * kBlock;
        } else {
          shift = 7.0f;  // log2(128): one pooled row stands for a full block (Eq. 6); the todo mask is in the logits already
          if (weak_bias) {
            const int c = ti.chunk_id[i - T];
            cm0 = ti.todo[c][0];
            cm1 = ti.todo[c][1];
            cm2 = ti.todo[c][2];
            cm3 = ti.todo[c][3];
            need_mask = true;
          }
        }
        if constexpr (FP8) {
          // Exact iteration: widen this iteration's raw e4m3 V tile (exactly) into the F16 V stage before looking
          // at the logits.  128 threads take ~900 cycles (the copy is bound by shared-memory bandwidth next to the
          // other CTA's MMAs); one or two dedicated warps were slower than the time they have, between
          // O += P V (G-1) freeing the stage and the first slice of P (G) needing it.
          if (i < T) {
            mbar_wait(&vraw_full, rc & 1, ctx, 603);
            if (G >= 1) wait_pv(G - 1, 602);
            widen_tile_f16(sVraw, sV, tid, 128);
            fence_proxy_async();
            named_bar_sync(1, 128);
            if (tid == 0) {
              mbar_arrive(&vraw_empty);
              mbar_arrive(&v_full);
            }
            ++rc;
          }
        }
        PF_BEGIN();
        mbar_wait(&s_done, G & 1, ctx, 502);
        PF_END(i == i0 ? 1 : (i < T ? 2 : 3));
#ifdef FP2_PROFILE
        pf[i == i0 ? 8 : (i < T ? 9 : 10)] += 1;
#endif
        tc_fence_after();
        if (need_mask) mask_row(s_addr, tok_lim, cm0, cm1, cm2, cm3);
        PF_END(4);
        uint32_t x[128];
        const float mx = fmaf(row_load_max(s_addr, x), cs_all, shift);  // cs > 0: scaling commutes with the maximum
        const float m_new = fmaxf(m, mx);
        // lazy rescale: only when some row of the warp moved its maximum by more than 2^8.  O is at rest: the
        // MMAs complete in issue order, so S (G) in TMEM means O += P V (G-1) has been added.
        if (__any_sync(0xffffffffu, m_new > m + 8.0f)) {
          const float f = (m == -INFINITY) ? 0.f : ex2(m - m_new);
          if (i > i0) {
#pragma unroll 1
            for (int k = 0; k < 4; ++k) {
              uint32_t rr[32];
              tmem_ld32(o_addr + k * 32, rr);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) rr[j] = __float_as_uint(__uint_as_float(rr[j]) * f);
              tmem_st32(o_addr + k * 32, rr);
            }
          }
          l *= f;
          m = m_new;
        }
        // a row with nothing visible so far has m = -inf and only -inf logits: exponent against 0 -> zeros
        const float neg_m = (m == -INFINITY) ? shift : shift - m;
        l += row_exp<FP8>(x, s_addr, cs_all, neg_m, &p_ready[0]);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&p_ready[kPParts - 1]);
        PF_END(5);
      }
      // ------------------------------ epilogue ------------------------------
      PF_BEGIN();
      const SegInfo& sg = ti.sg;
      const float inv = l > 0.f ? out_scale / l : 0.f;
      const bool have_o = i1 > i0;
      const bool row_ok = row < sg.nrows;
      const size_t tok = (size_t)sg.q_tok0 + r / g;
      const int head = sg.h * g + r % g;
      __nv_bfloat16* orow = A.out + (tok * P.num_q_heads + head) * kHeadDim;
      if (have_o) {
        wait_pv(G - 1, 503);   // O += P V of the unit's last iteration
        tc_fence_after();
      }
      PF_END(6);
      if (ti.parts > 1) {
        // one part of a split segment (Eq. 18): leave (O, m, l) unnormalised for the merge kernel
        float* prow = A.part_o + ((size_t)ti.slot * 128 + row) * 128;
        if (have_o) {
#pragma unroll 1
          for (int k = 0; k < 4; ++k) {
            uint32_t a0[32];
            tmem_ld32(o_addr + k * 32, a0);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 4; ++j) st_global_v8(prow + k * 32 + j * 8, &a0[j * 8], stream_pol);
          }
        }
        A.part_ml[(size_t)ti.slot * 128 + row] = make_float2(have_o ? m : -INFINITY, have_o ? l : 0.f);
        tc_fence_before();
        mbar_arrive(&info_empty[slot]);
        continue;
      }
#pragma unroll 1
      for (int k = 0; k < 4; ++k) {
        uint32_t a0[32];
        if (have_o) {
          tmem_ld32(o_addr + k * 32, a0);
          tmem_wait_ld();
        }
        uint32_t o[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float v0 = have_o ? __uint_as_float(a0[2 * j]) * inv : 0.f;
          const float v1 = have_o ? __uint_as_float(a0[2 * j + 1]) * inv : 0.f;
          o[j] = pack_bf16x2(v0, v1);
        }
        if (row_ok) {   // 32-byte stores: every instruction writes whole sectors
          st_global_v8(orow + k * 32, &o[0], stream_pol);
          st_global_v8(orow + k * 32 + 16, &o[8], stream_pol);
        }
      }
      if (row_ok && A.lse != nullptr)
        A.lse[(size_t)head * P.total_q + tok] = (m + log2f(l)) * 0.6931471805599453f;
      tc_fence_before();
      mbar_arrive(&info_empty[slot]);
      PF_END(7);
    }
#ifdef FP2_PROFILE
    pf[15] = clock64() - pf_t0;
    if (tid == 0 && A.prof)
      for (int i = 0; i < 16; ++i) A.prof[(size_t)blockIdx.x * 16 + i] = pf[i];
#endif
  }
  // teardown: on the normal path every barrier has been consumed and every MMA has completed (the epilogue waited
  // for the last one).  After an abort MMAs and bulk copies may still be in flight: the issuing thread waits (bounded)
  // for its MMAs, everyone gives the copies time, and only then is tensor memory released.
  if (abort_flag) {
    if (warp == 5 && lane == 0) {
      umma_commit(&drain_bar);
      mbar_wait_drain(&drain_bar, 0, 200000000ll);
    }
    __nanosleep(2000000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 256);
}

}  // namespace fp2
