// Block-sparse causal flash attention with mean correction (Eq. 4, Eq. 6; Algorithm 1 lines 6-11),
// persistent, warp-specialised, tcgen05 / TMEM / TMA.  The same kernel runs the dense path (implicit list
// 0..J_hi, no correction).
//
// One CTA per SM loops over work units (sequence, KV head, packed query tile) taken from a work order
// (KV-head-major, heaviest first) through a global counter.  For a unit with selected list idx[0..T) the
// iteration sequence is the list traversed backwards (Eq. 17) followed by the non-empty correction chunks:
// a correction chunk stages 128 consecutive pooled (kbar, vbar) rows exactly like a KV block, its logits are
// shifted by log2(128) (every corrected block is full) and masked by todo = fully-visible & ~selected.
//
// Roles:
//   warps 0..4W-1   W = kWG softmax warpgroups (2 by default).  All work on EVERY iteration: warpgroup w owns
//              logit columns [w 128/W, (w+1) 128/W) of all 128 rows (thread = row).  They exchange the row maximum
//              through shared memory once per iteration; one accumulator O serves the whole tile (no merge at the
//              end).  W = 4 (four warps per scheduler, 104 registers each) builds and passes parity but measured
//              3 % (dense) to 10 % (sparse) slower at 32K than W = 2 with 224 registers.
//   warp 4W    TMA producer: K / V pages through the page table into two rings (Eq. 22)
//   warp 4W+1  UMMA issuer: S = Q K^T (SS), O += P V (P read from TMEM, V MN-major from shared memory)
//   warps 4W+2, 4W+3  tile set-up: fetch the next unit, validate its list, build the correction masks, stage Q
//   warps 4W+4..4W+7  (FP8 inputs only) widen raw e4m3 K / V tiles to F16 into the K / V rings
//
// TMEM columns: S0 [0,128) S1 [128,256) O [256,384) P0 [384,448) P1 [448,512).  P (BF16 pairs) has its own
// columns, so S = Q K^T of iteration i+2 may start as soon as the softmax of iteration i has read S -- it does
// not wait for O += P V of iteration i.  Issue order: QK(0) QK(1) PV(0) QK(2) PV(1) ...  Per 128x128 block
// the tensor pipe and the MUFU pipe are each busy 1024 cycles (ncu); how far the two overlap is what the
// schedule decides.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"
#include "ptx.cuh"
#include "score_select.cuh"  // load_q_tile_bf16

namespace fp2 {

constexpr int kTileBytes = 32768;   // one 128 x 128 tile of 16-bit elements
constexpr int kRawBytes = 16384;    // one 128 x 128 tile of FP8 elements as TMA delivers it

// FP8 inputs (Eq. 15) run through the same 16-bit pipeline: the producer lands raw e4m3 K / V tiles in a small
// ring, a fourth warpgroup widens them to F16 (exact) into the K / V rings, and both GEMMs run as kind::f16
// with F16 operands (Q widened when staged, P packed as F16).  The per-head scales never touch the operands:
// q_scale * k_scale multiplies the logits of a row, v_scale multiplies the output.  A single e4m3 probability
// tile, the other way to feed FP8 V to the tensor core, costs ~0.06 max-abs output error by itself.
#ifndef FP2_SOFTMAX_WGS
#define FP2_SOFTMAX_WGS 2
#endif
constexpr int kWG = FP2_SOFTMAX_WGS;      // softmax warpgroups; each owns 128 / kWG logit columns of every row
constexpr int kCW = 128 / kWG;            // columns per warpgroup (64 or 32)
constexpr int kSW = 4 * kWG;              // softmax warps; the service warps follow them
static_assert(kWG == 2 || kWG == 4, "two or four softmax warpgroups");

template <bool FP8>
struct AttnCfg {
  static constexpr int kThreads = 128 * kWG + 128 + (FP8 ? 128 : 0);
  static constexpr int kNQ = FP8 ? 1 : 2;   // Q tiles in shared memory: two let the next unit's queries land while
                                            // this unit is still being multiplied (FP8 has no room for a second)
  static constexpr int kNK = 2;             // K ring stages (32 KB each).  Must stay 2: stage i % 2 is released by the
                                            // same commit that publishes S buffer i % 2
  static constexpr int kNV = 2;             // V ring stages
  static constexpr int kNRaw = FP8 ? 3 : 0; // raw FP8 tile ring (16 KB each), K and V tiles alternate
  static constexpr int kSmemBytes = 1024 + kTileBytes * (kNQ + kNK + kNV) + kNRaw * kRawBytes + 2048 * kWG;
  // Registers.  The CTA is launched with kRegsBase registers per thread (what __launch_bounds__(kThreads, 1)
  // lets ptxas use); setmaxnreg then moves registers from the service warps (kRegsService) to the softmax warps
  // (kRegsSoftmax).  setmaxnreg.inc waits -- without bound -- until the CTA's own pool has the registers, so the
  // total after the move must not exceed the launch allocation; the host checks the compiled register count
  // against kRegsAfterMove before the first launch and refuses to launch otherwise.
  static constexpr int kRegsBase = (65536 / kThreads) / 8 * 8;
  static constexpr int kRegsService = (kWG == 4) ? 48 : 56;
  static constexpr int kRegsSoftmax = (kWG == 4) ? (FP8 ? 96 : 104) : (FP8 ? 200 : 224);
  static constexpr int kRegsAfterMove = (kThreads - 128 * kWG) * kRegsService + 128 * kWG * kRegsSoftmax;
  static_assert(kRegsAfterMove <= kThreads * kRegsBase, "register budget: setmaxnreg.inc would wait forever");
  static constexpr int kFmt = FP8 ? 0 : 1;  // UMMA kind::f16 operand format: 0 = F16, 1 = BF16
};

struct TileInfo {
  SegInfo sg;
  int32_t valid;     // 0: no more work
  int32_t T;         // exact iterations (listed blocks)
  int32_t nchunk;    // non-empty correction chunks
  int32_t dense;
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
};

// Masked iterations (diagonal blocks, correction chunks -- the minority): overwrite the hidden logits of this
// thread's row with -inf in TMEM, so that the softmax step itself carries no mask logic (predicating the mask
// into the softmax body cost 2.5x on every iteration, masked or not).  The thread owns kCW columns starting at
// block column col0; column j stays visible iff j <= tok_lim and bit (j - col0) of cm (32 bits per word) is set.
__device__ __forceinline__ void mask_cols(uint32_t s_addr, int col0, int tok_lim, const uint32_t* cm) {
#pragma unroll
  for (int k = 0; k < kCW / 32; ++k) {
    const bool all_vis = (col0 + k * 32 + 31 <= tok_lim) && (cm[k] == 0xffffffffu);
    if (__all_sync(0xffffffffu, all_vis)) continue;   // TMEM accesses are warp-wide: decide per warp
    uint32_t rr[32];
    tmem_ld32(s_addr + k * 32, rr);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const bool vis = (col0 + k * 32 + j <= tok_lim) && ((cm[k] >> j) & 1u);
      rr[j] = vis ? rr[j] : 0xff800000u;  // -inf
    }
    tmem_st32(s_addr + k * 32, rr);
  }
  tmem_wait_st();
}

// This thread's kCW logit columns (raw, unscaled) into registers, and their maximum: all TMEM loads in flight,
// chains of three-input maxima.
__device__ __forceinline__ float cols_row_max(uint32_t s_addr, uint32_t (&sv)[kCW]) {
#pragma unroll
  for (int k = 0; k < kCW / 32; ++k) tmem_ld32(s_addr + k * 32, reinterpret_cast<uint32_t(&)[32]>(sv[k * 32]));
  tmem_wait_ld();
  float mx8[kCW / 8];
#pragma unroll
  for (int c = 0; c < kCW / 8; ++c) {
    const float* v = reinterpret_cast<const float*>(&sv[c * 8]);
    mx8[c] = fmaxf(max3(max3(v[0], v[1], v[2]), v[3], v[4]), max3(v[5], v[6], v[7]));
  }
  float r = fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3]));
  if constexpr (kCW == 64) r = fmaxf(r, fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
  return r;
}

// p = 2^(s * cs + neg_m) for this thread's kCW logits (still in the registers the maximum pass loaded them into),
// written as 16-bit pairs to kCW / 2 columns at p_addr.  One TMEM read per logit: besides the latency, TMEM
// loads of the softmax warps lengthen the time the tensor pipe takes to accept each MMA of the issuing thread.
// Scaling and row sum use packed fp32x2 instructions.  Returns the row's partial sum.
template <bool F16>
__device__ __forceinline__ float cols_row_exp(const uint32_t (&sv)[kCW], uint32_t p_addr, float cs, float neg_m) {
  const uint64_t cs2 = f2_pack(cs, cs), nm2 = f2_pack(neg_m, neg_m);
  uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};   // four independent (lo, hi) accumulators, +0.0f bit patterns
#pragma unroll
  for (int k = 0; k < kCW / 32; ++k) {
    uint32_t pk[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint64_t x2 =
          f2_fma(f2_pack(__uint_as_float(sv[k * 32 + 2 * j]), __uint_as_float(sv[k * 32 + 2 * j + 1])), cs2, nm2);
      float x0, x1;
      f2_unpack(x2, x0, x1);
      const float p0 = ex2(x0), p1 = ex2(x1);
      sum2[j & 3] = f2_add(sum2[j & 3], f2_pack(p0, p1));
      pk[j] = F16 ? pack_f16x2(p0, p1) : pack_bf16x2(p0, p1);
    }
    tmem_st16(p_addr + k * 16, pk);
  }
  float a0, a1;
  f2_unpack(f2_add(f2_add(sum2[0], sum2[1]), f2_add(sum2[2], sum2[3])), a0, a1);
  return a0 + a1;
}

// FP8 query tile -> shared memory as F16 (exact), same K-major swizzled layout as the BF16 tile.
__device__ __forceinline__ void load_q_tile_f16(uint8_t* sQ, const uint8_t* __restrict__ q, const SegInfo& sg,
                                                const DevParams& P, int t, int nthr) {
  const int g = P.group;
  constexpr int BATCH = 8;
  for (int i0 = t; i0 < kTileRows * 16; i0 += nthr * BATCH) {
    uint2 v[BATCH];
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int i = i0 + u * nthr;
      const int row = i >> 4, ch = i & 15;   // 16 chunks of 8 elements per row
      v[u] = make_uint2(0, 0);
      if (i < kTileRows * 16 && row < sg.nrows) {
        const int r = sg.r0 + row;
        const size_t tok = (size_t)sg.q_tok0 + r / g;
        const size_t head = (size_t)sg.h * g + r % g;
        v[u] = __ldg(reinterpret_cast<const uint2*>(q + (tok * P.num_q_heads + head) * kHeadDim + ch * 8));
      }
    }
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int i = i0 + u * nthr;
      const int row = i >> 4, ch = i & 15;
      if (i < kTileRows * 16) {
        const uint4 o = make_uint4(e4m3x2_to_f16x2(v[u].x), e4m3x2_to_f16x2(v[u].x >> 16),
                                   e4m3x2_to_f16x2(v[u].y), e4m3x2_to_f16x2(v[u].y >> 16));
        *reinterpret_cast<uint4*>(sQ + (ch >> 3) * 16384 + sw128_offset(row, ch & 7)) = o;
      }
    }
  }
}

template <bool FP8>
__global__ void __launch_bounds__(AttnCfg<FP8>::kThreads, 1)
sparse_attn_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const __grid_constant__ CUtensorMap map_kbar, const __grid_constant__ CUtensorMap map_vbar,
                   AttnArgs A, DevParams P) {
  constexpr int kNQ = AttnCfg<FP8>::kNQ, kNK = AttnCfg<FP8>::kNK, kNV = AttnCfg<FP8>::kNV, kNRaw = AttnCfg<FP8>::kNRaw;
  constexpr int kAttnThreads = AttnCfg<FP8>::kThreads;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + kNQ * kTileBytes;
  uint8_t* sV = sK + kNK * kTileBytes;
  uint8_t* sRaw = sV + kNV * kTileBytes;                          // FP8 only: raw tile ring
  float* sX = reinterpret_cast<float*>(sRaw + kNRaw * kRawBytes);  // [2 parity][kWG][128] row-max exchange, then the same for row sums

  __shared__ TileInfo info[2];
  __shared__ uint32_t sel_bits[2][kMaxBlocks / 32];
  __shared__ uint64_t info_full[2], info_empty[2], q_full[2], q_empty[2], tile_done;
  // One tcgen05.commit costs the issuing thread ~70 cycles, so barriers that would be signalled by the same
  // commit are merged: s_full[a] also releases K stage a (k_empty), v_empty[b] also says that O += P V of an
  // iteration with parity b has completed (what the lazy rescale waits for).
  static_assert(kNK == 2 && kNV == 2, "merged barriers assume two K stages and two V stages");
  __shared__ uint64_t k_full[kNK], v_full[kNV], v_empty[kNV];
  __shared__ uint64_t s_full[2], p_ready[2];
  uint64_t* const k_empty = s_full;
  __shared__ uint64_t raw_full[kNRaw > 0 ? kNRaw : 1], raw_empty[kNRaw > 0 ? kNRaw : 1];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  WaitCtx ctx{A.status, &abort_flag};

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(&info_full[i], 1);
      mbar_init(&info_empty[i], 2 + 128 * kWG + (FP8 ? 1 : 0));
      mbar_init(&s_full[i], 1);
      mbar_init(&p_ready[i], 128 * kWG);
    }
    for (int i = 0; i < 2; ++i) { mbar_init(&q_full[i], 64); mbar_init(&q_empty[i], 1); }
    mbar_init(&tile_done, 1);
    for (int i = 0; i < kNK; ++i) mbar_init(&k_full[i], 1);
    for (int i = 0; i < kNV; ++i) { mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1); }
    for (int i = 0; i < kNRaw; ++i) { mbar_init(&raw_full[i], 1); mbar_init(&raw_empty[i], 1); }
    fence_barrier_init();
  }
  // K / V rings start zeroed: rows of pages past the end of a sequence are never loaded, and whatever sits
  // there is multiplied by probabilities that are exactly zero, so it must be finite.
  for (int i = tid; i < ((kNK + kNV) * kTileBytes + kNRaw * kRawBytes) / 16; i += kAttnThreads)
    reinterpret_cast<uint4*>(sK)[i] = make_uint4(0, 0, 0, 0);
  if (warp == kSW + 1) {
    tmem_alloc(&tmem_base_s, 512);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const int g = P.group;

  if (FP8 && warp >= kSW + 4) {
    // =============================== FP8 -> F16 widening warpgroup ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    if constexpr (FP8) {
      const int t128 = tid - 32 * (kSW + 4);
      uint32_t kc = 0, vc = 0, rc = 0;
      for (int it = 0;; ++it) {
        const int slot = it & 1;
        mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 601);
        const TileInfo& ti = info[slot];
        if (!ti.valid) break;
        const int T = ti.T, n_it = T + ti.nchunk;
        for (int i = 0; i < n_it; ++i, ++kc, ++vc) {
          if (i >= T) continue;   // correction chunks arrive as F16 straight into the K / V rings
#pragma unroll
          for (int kv = 0; kv < 2; ++kv, ++rc) {
            const int rs = rc % kNRaw;
            const int ds = kv ? (int)(vc % kNV) : (int)(kc % kNK);
            const uint32_t dc = kv ? vc : kc;
            const int dn = kv ? kNV : kNK;
            uint64_t* d_empty = kv ? &v_empty[ds] : &k_empty[ds];
            uint64_t* d_full = kv ? &v_full[ds] : &k_full[ds];
            if (dc >= (uint32_t)dn) mbar_wait(d_empty, ((dc / dn) - 1) & 1, ctx, 602);
            mbar_wait(&raw_full[rs], (rc / kNRaw) & 1, ctx, 603);
            widen_tile_f16(sRaw + rs * kRawBytes, (kv ? sV : sK) + ds * kTileBytes, t128, 128);
            fence_proxy_async();
            named_bar_sync(3, 128);
            if (t128 == 0) {
              mbar_arrive(&raw_empty[rs]);
              mbar_arrive(d_full);
            }
          }
        }
        if (t128 == 0) mbar_arrive(&info_empty[slot]);
      }
    }
  } else if (warp >= kSW + 2) {
    // =============================== tile set-up + Q staging ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    const int t64 = tid - 32 * (kSW + 2);
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      if (it >= 2) mbar_wait(&info_empty[slot], ((it >> 1) - 1) & 1, ctx, 201);
      TileInfo& ti = info[slot];
      if (t64 == 0) {
        const int w = atomicAdd(A.work_counter, 1);
        if (w < P.nseg) {
          const int seg = A.order[w];
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
        } else {
          ti.valid = 0;
        }
      }
      named_bar_sync(2, 64);
      const bool valid = ti.valid != 0;
      if (valid && !ti.dense) {
        const SegInfo& sg = ti.sg;
        const int32_t* list = A.blk_idx + sg.off;
        const int T = ti.T;
        const int nwords = (sg.J_lo + 31) >> 5;
        const bool corr = P.use_correction != 0;
        if (corr)
          for (int w = t64; w < nwords; w += 64) sel_bits[slot][w] = 0u;
        named_bar_sync(2, 64);
        bool bad = false;
        for (int k = t64; k < T; k += 64) {
          const int J = list[k];
          if (J < 0 || J > sg.J_hi || (k > 0 && list[k - 1] >= J)) bad = true;
          if (corr && J >= 0 && J < sg.J_lo) atomicOr(&sel_bits[slot][J >> 5], 1u << (J & 31));
        }
        if (bad) atomicOr(A.status + ST_BAD_LIST, 1);
        named_bar_sync(2, 64);
        if (corr) {
          const int nch = (sg.J_lo + 127) >> 7;
          for (int c = t64; c < nch; c += 64) {
#pragma unroll
            for (int w = 0; w < 4; ++w) {
              const int first = c * 128 + w * 32;
              uint32_t validm = 0u;
              if (first + 32 <= sg.J_lo) validm = 0xffffffffu;
              else if (first < sg.J_lo) validm = (1u << (sg.J_lo - first)) - 1u;
              ti.todo[c][w] = (first < sg.J_lo ? ~sel_bits[slot][first >> 5] : 0u) & validm;
            }
          }
          named_bar_sync(2, 64);
          if (t64 == 0) {
            int n = 0;
            for (int c = 0; c < nch; ++c)
              if (ti.todo[c][0] | ti.todo[c][1] | ti.todo[c][2] | ti.todo[c][3]) ti.chunk_id[n++] = c;
            ti.nchunk = n;
          }
        }
      }
      named_bar_sync(2, 64);
      if (t64 == 0) mbar_arrive(&info_full[slot]);
      if (!valid) break;
      // Q tile: wait until every S = Q K^T of the unit that last used this buffer has completed, then overwrite
      const int qb = it % kNQ;
      if (it >= kNQ) mbar_wait(&q_empty[qb], ((it / kNQ) - 1) & 1, ctx, 202);
      if constexpr (FP8) load_q_tile_f16(sQ + qb * kTileBytes, A.q, ti.sg, P, t64, 64);
      else load_q_tile_async(sQ + qb * kTileBytes, A.q, ti.sg, P, t64, 64);
      fence_proxy_async();
      mbar_arrive(&q_full[qb]);
    }
  } else if (warp == kSW) {
    // =============================== TMA producer ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    if (lane == 0) {
      tma_prefetch_desc(&map_k);
      tma_prefetch_desc(&map_v);
      tma_prefetch_desc(&map_kbar);
      tma_prefetch_desc(&map_vbar);
    }
    uint32_t kc = 0, vc = 0, rc = 0;
    (void)rc;
    const uint64_t keep = l2_policy_evict_last();   // K / V pages and pooled means: shared by many tiles
    const int ppb = P.pages_per_block, psz = P.page_size;
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 301);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const SegInfo& sg = ti.sg;
      const int T = ti.T, n_it = T + ti.nchunk;
      const int32_t* list = A.blk_idx + sg.off;
      const int32_t* pt = A.page_table + (size_t)sg.b * P.max_pages_per_seq;
      // page id of this lane's page of exact iteration i (-1: past the end of the sequence, or not an exact
      // iteration).  Fetched one iteration ahead: list entry -> page-table entry are two dependent global loads.
      auto fetch_pid = [&](int i) -> int {
        if (i >= T || lane >= ppb) return -1;
        int J = ti.dense ? sg.J_hi - i : list[T - 1 - i];
        J = max(0, min(J, sg.J_hi));
        if (J * kBlock + lane * psz >= sg.Lk) return -1;
        int pid = pt[J * ppb + lane];
        if (pid < 0 || pid >= P.num_pages) {
          atomicOr(A.status + ST_BAD_LIST, 2);
          pid = -1;
        }
        return pid;
      };
      int pid_next = fetch_pid(0);
      for (int i = 0; i < n_it; ++i) {
        const int ks = kc % kNK, vs = vc % kNV;
        uint8_t* dK = sK + ks * kTileBytes;
        uint8_t* dV = sV + vs * kTileBytes;
        const int pid = pid_next;
        pid_next = fetch_pid(i + 1);
        if (i < T) {
          const int nvalid = __popc(__ballot_sync(0xffffffffu, pid >= 0));
          if constexpr (FP8) {
            // raw e4m3 tiles (128 bytes per token row) into the raw ring; the widening warpgroup fills the K / V rings
            const uint32_t rbytes = (uint32_t)nvalid * psz * 128u;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv, ++rc) {
              const int rs = rc % kNRaw;
              if (rc >= (uint32_t)kNRaw) mbar_wait(&raw_empty[rs], ((rc / kNRaw) - 1) & 1, ctx, 306);
              if (lane == 0) mbar_arrive_expect_tx(&raw_full[rs], rbytes);
              __syncwarp();
              if (pid >= 0)
                tma_load_3d_hint(sRaw + rs * kRawBytes + lane * psz * 128, kv ? &map_v : &map_k, &raw_full[rs], 0, sg.h,
                            pid * psz, keep);
            }
            ++kc;
            ++vc;
            continue;
          }
          const uint32_t bytes = (uint32_t)nvalid * psz * 256u;
          if (kc >= kNK) mbar_wait(&k_empty[ks], ((kc / kNK) - 1) & 1, ctx, 302);
          if (lane == 0) mbar_arrive_expect_tx(&k_full[ks], bytes);
          __syncwarp();
          if (pid >= 0) {
            tma_load_3d_hint(dK + lane * psz * 128, &map_k, &k_full[ks], 0, sg.h, pid * psz, keep);
            tma_load_3d_hint(dK + 16384 + lane * psz * 128, &map_k, &k_full[ks], 64, sg.h, pid * psz, keep);
          }
          if (vc >= kNV) mbar_wait(&v_empty[vs], ((vc / kNV) - 1) & 1, ctx, 303);
          if (lane == 0) mbar_arrive_expect_tx(&v_full[vs], bytes);
          __syncwarp();
          if (pid >= 0) {
            tma_load_3d_hint(dV + lane * psz * 128, &map_v, &v_full[vs], 0, sg.h, pid * psz, keep);
            tma_load_3d_hint(dV + 16384 + lane * psz * 128, &map_v, &v_full[vs], 64, sg.h, pid * psz, keep);
          }
        } else {
          const int row0 = sg.blk_off + ti.chunk_id[i - T] * 128;
          if (kc >= kNK) mbar_wait(&k_empty[ks], ((kc / kNK) - 1) & 1, ctx, 304);
          if (lane == 0) {
            mbar_arrive_expect_tx(&k_full[ks], kTileBytes);
            tma_load_3d_hint(dK, &map_kbar, &k_full[ks], 0, sg.h, row0, keep);
            tma_load_3d_hint(dK + 16384, &map_kbar, &k_full[ks], 64, sg.h, row0, keep);
          }
          if (vc >= kNV) mbar_wait(&v_empty[vs], ((vc / kNV) - 1) & 1, ctx, 305);
          if (lane == 0) {
            mbar_arrive_expect_tx(&v_full[vs], kTileBytes);
            tma_load_3d_hint(dV, &map_vbar, &v_full[vs], 0, sg.h, row0, keep);
            tma_load_3d_hint(dV + 16384, &map_vbar, &v_full[vs], 64, sg.h, row0, keep);
          }
          __syncwarp();
        }
        ++kc;
        ++vc;
      }
      if (lane == 0) mbar_arrive(&info_empty[slot]);
    }
  } else if (warp == kSW + 1) {
    // =============================== UMMA issuer ===============================
    setmaxnreg_dec<AttnCfg<FP8>::kRegsService>();
    if (lane == 0) {
      constexpr int kFmt = AttnCfg<FP8>::kFmt;
      constexpr uint32_t idesc_qk = make_idesc(128, 128, kFmt, kFmt, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(128, 128, kFmt, kFmt, 0, 1);
      uint32_t kc = 0, vc = 0, pc0 = 0, pc1 = 0;
      auto issue_pv = [&](int j) {
        const int b = vc & 1;   // P buffer / V stage: parity of the iteration counted over the whole kernel
        if (b) { mbar_wait(&p_ready[1], pc1 & 1, ctx, 401); ++pc1; }
        else { mbar_wait(&p_ready[0], pc0 & 1, ctx, 401); ++pc0; }
        const int vs = vc % kNV;
        mbar_wait(&v_full[vs], (vc / kNV) & 1, ctx, 402);
        tc_fence_after();
        const uint32_t v_addr = smem_u32(sV + vs * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t bd = make_smem_desc_sw128(v_addr + ks * 2048, 16384, 1024);
          umma_f16_ts(tmem + 256, tmem + 384 + b * 64 + ks * 8, bd, idesc_pv, (j > 0) || ks > 0);
        }
        umma_commit(&v_empty[vs]);   // V stage vs (== iteration parity) is free and O holds this iteration
        ++vc;
      };
      for (int it = 0;; ++it) {
        const int slot = it & 1;
        mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 403);
        const TileInfo& ti = info[slot];
        if (!ti.valid) break;
        const int n_it = ti.T + ti.nchunk;
        const int qb = it % kNQ;
        mbar_wait(&q_full[qb], (it / kNQ) & 1, ctx, 404);
        const uint32_t q_addr = smem_u32(sQ + qb * kTileBytes);
        for (int i = 0; i < n_it; ++i) {
          const int ks_ = kc % kNK;
          const int a = ks_;   // S buffer = K stage = parity of the iteration counted over the whole kernel
          mbar_wait(&k_full[ks_], (kc / kNK) & 1, ctx, 405);
          tc_fence_after();
          const uint32_t k_addr = smem_u32(sK + ks_ * kTileBytes);
          // S_a is free: the softmax of iteration i-2 signalled p_ready[a] (waited for in issue_pv(i-2))
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
            const uint64_t ad = make_smem_desc_sw128(q_addr + off, 16, 1024);
            const uint64_t bd = make_smem_desc_sw128(k_addr + off, 16, 1024);
            umma_f16_ss(tmem + a * 128, ad, bd, idesc_qk, ks > 0);
          }
          umma_commit(&s_full[a]);   // S_a is ready and K stage ks_ (== a) is free
          ++kc;
          if (i == n_it - 1) umma_commit(&q_empty[qb]);
          if (i >= 1) issue_pv(i - 1);
        }
        if (n_it >= 1) issue_pv(n_it - 1);
        else umma_commit(&q_empty[qb]);  // empty list: nothing read Q, release it at once
        umma_commit(&tile_done);
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else {
    // =============================== softmax warpgroups + epilogue ===============================
    setmaxnreg_inc<AttnCfg<FP8>::kRegsSoftmax>();
    const int wg = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t o_addr = lane_base + 256 + wg * kCW;   // this thread's kCW columns of O
    uint32_t sc0 = 0, sc1 = 0;   // completed uses of S0 / S1 (phases of s_full)
    uint32_t pv_base = 0;        // iterations (= UMMA groups O += P V = V stage uses) before this tile
    const uint64_t stream_pol = l2_policy_evict_first();   // outputs are written once and not read here
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 501);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const SegInfo sg = ti.sg;
      const int T = ti.T, n_it = T + ti.nchunk;
      const int32_t* list = A.blk_idx + sg.off;
      const int r = sg.r0 + row;
      const int pos = sg.pre + r / g;
      // logit multipliers in log2 units.  FP8 (Eq. 15): the MMAs see raw e4m3 values, so exact blocks carry
      // q_scale * k_scale and pooled chunks (kbar is stored de-scaled) carry q_scale only.
      float cs_exact = P.scale_log2, cs_chunk = P.scale_log2, out_scale = 1.0f;
      if constexpr (FP8) {
        const float qs = A.q_scale[sg.h * g + r % g];
        cs_chunk *= qs;
        cs_exact *= qs * A.k_scale[sg.h];
        out_scale = A.v_scale[sg.h];
      }
      float m = -INFINITY, l = 0.f;
      // block id of the next exact iteration, fetched one iteration ahead
      int J_next = (!ti.dense && T > 0) ? list[T - 1] : 0;
      for (int i = 0; i < n_it; ++i) {
        const int a = (pv_base + i) & 1;   // S / P buffer: parity of the iteration counted over the whole kernel
        const uint32_t s_addr = lane_base + a * 128 + wg * kCW;
        const uint32_t p_addr = lane_base + 384 + a * 64 + wg * (kCW / 2);
        // iteration kind and masks
        bool need_mask = false;
        int tok_lim = 1 << 30;     // exact block: columns j with j <= tok_lim are visible
        uint32_t cm[kCW / 32];
#pragma unroll
        for (int w = 0; w < kCW / 32; ++w) cm[w] = 0xffffffffu;
        float shift = 0.f, cs = cs_exact;
        if (i < T) {
          int J = ti.dense ? sg.J_hi - i : J_next;
          if (!ti.dense && i + 1 < T) J_next = list[T - 2 - i];
          J = max(0, min(J, sg.J_hi));
          need_mask = J >= sg.J_lo;
          tok_lim = pos - J * kBlock;
        } else {
          const int c = ti.chunk_id[i - T];
#pragma unroll
          for (int w = 0; w < kCW / 32; ++w) cm[w] = ti.todo[c][wg * (kCW / 32) + w];
          shift = 7.0f;  // log2(128): one pooled row stands for a full block (Eq. 6)
          cs = cs_chunk;
          need_mask = true;
        }
        if (a) { mbar_wait(&s_full[1], sc1 & 1, ctx, 502); ++sc1; }
        else { mbar_wait(&s_full[0], sc0 & 1, ctx, 502); ++sc0; }
        tc_fence_after();
        if (need_mask) mask_cols(s_addr, wg * kCW, tok_lim, cm);
        // row maximum over all 128 columns: own half, then the other warpgroup's through shared memory
        uint32_t sv[kCW];
        float mx = cols_row_max(s_addr, sv);
        float* xch = sX + (i & 1) * (kWG * 128);
        xch[wg * 128 + row] = mx;
        named_bar_sync(1, 128 * kWG);
#pragma unroll
        for (int w = 1; w < kWG; ++w) mx = fmaxf(mx, xch[((wg + w) % kWG) * 128 + row]);
        mx = fmaf(mx, cs, shift);  // cs > 0: scaling commutes with the maximum
        const float m_new = fmaxf(m, mx);
        // lazy rescale: only when some row of the warp moved its maximum by more than 2^8.  Both warpgroups
        // hold the same rows in the same warps and the same m, so they take the same decision.
        const bool need = m_new > m + 8.0f;
        if (__any_sync(0xffffffffu, need)) {
          const float f = (m == -INFINITY) ? 0.f : ex2(m - m_new);
          if (i > 0) {
            // O must be at rest: wait for O += P V of iteration i-1, the ((pv_base + i - 1) / 2)-th use of V stage
            // (pv_base + i - 1) % 2 counted over the whole kernel (iterations and V stages advance together)
            mbar_wait(&v_empty[(pv_base + i - 1) & 1], ((pv_base + i - 1) >> 1) & 1, ctx, 504);
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < kCW / 32; ++k) {
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
        l += cols_row_exp<FP8>(sv, p_addr, cs, neg_m);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&p_ready[a]);
      }
      pv_base += (uint32_t)n_it;
      // ------------------------------ epilogue ------------------------------
      mbar_wait(&tile_done, it & 1, ctx, 503);
      tc_fence_after();
      float* xch = sX + 2 * kWG * 128 + (it & 1) * (kWG * 128);   // by tile parity: no barrier before its next use
      xch[wg * 128 + row] = l;
      named_bar_sync(1, 128 * kWG);
      float L = l;
#pragma unroll
      for (int w = 1; w < kWG; ++w) L += xch[((wg + w) % kWG) * 128 + row];
      const float inv = L > 0.f ? out_scale / L : 0.f;
      const bool have_o = n_it >= 1;
      const bool row_ok = row < sg.nrows;
      const size_t tok = (size_t)sg.q_tok0 + r / g;
      const int head = sg.h * g + r % g;
      __nv_bfloat16* orow = A.out + (tok * P.num_q_heads + head) * kHeadDim + wg * kCW;
#pragma unroll
      for (int k = 0; k < kCW / 32; ++k) {
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
      if (wg == 0 && row_ok && A.lse != nullptr)
        A.lse[(size_t)head * P.total_q + tok] = (m + log2f(L)) * 0.6931471805599453f;
      tc_fence_before();
      mbar_arrive(&info_empty[slot]);
    }
  }
  // teardown: on the normal path every barrier has been consumed; after an abort give in-flight copies time
  if (abort_flag) __nanosleep(2000000);
  tc_fence_before();
  __syncthreads();
  if (warp == kSW + 1) tmem_dealloc(tmem, 512);
}

}  // namespace fp2
