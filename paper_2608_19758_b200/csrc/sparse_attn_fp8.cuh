// Block-sparse causal flash attention with mean correction (Eq. 4, Eq. 6; Algorithm 1 lines 6-11) for FP8 e4m3
// inputs with per-head scales (Eq. 15): same work units, iteration sequence and outputs as sparse_attn_kernel.
//
// Every contraction runs on the raw e4m3 tiles as a kind::f8f6f4 MMA, at twice the BF16 rate:
//   S = Q K^T           Q and K as TMA / cp.async deliver them (K-major, 128-byte rows);
//   O += P V            V consumed raw and MN-major straight from its TMA tile (no transpose, no widening), and the
//                       probabilities as a PAIR of 8-bit tiles,  P = P_hi + P_lo,  P_hi = e4m3(p),
//                       P_lo = e5m2(p - P_hi),  two accumulating MMA groups.  A single e4m3 tile -- the paper's
//                       P~ = e4m3(2^8 p) -- costs ~0.06 max-abs output error by itself, at the parity gate; the pair
//                       carries ~7 mantissa bits, and the e5m2 low part keeps probabilities down to 2^-24 of the
//                       row maximum (an e4m3 low part would drop everything below 2^-18).
// The per-head scales never touch the operands: q_scale * k_scale multiplies the logits of a row, v_scale the output.
// p is computed as 2^(x - m + 4) with the lazy rescale threshold at 2^4, so p <= 2^8 (e4m3 reaches 448) and the
// row maximum contributes at least 2^4; the offset comes out again in the LSE.
//
// P leaves the softmax warpgroup through SHARED memory (4 slices of 32 key columns, hi and lo: 8 slots of 4 KB,
// unswizzled K-major operands), not through tensor memory as in sparse_attn_kernel.  The FP8 tiles are half the
// size of the BF16 ones, which is what pays for the 32 KB.  The S columns are therefore free as soon as every
// softmax thread has its logit row in registers (barrier s_free): S (i+1) is issued at the START of softmax (i)
// and waits in tensor memory when softmax (i) ends, so the warpgroup goes from one iteration straight into the next
// instead of idling while the tensor pipe works for it.  A whole iteration of P is buffered, so O += P V (i) may
// trail softmax (i) by up to an iteration without stalling anybody.
// K and V have a producer warp each, because their stages free at different times (K when S (i) completes, early in
// softmax (i); V in two halves of 64 tokens as the k-steps of O += P V (i) complete).
//
// Correction chunks: pooled keys as an e4m3 hi + lo pair in raw units (two MMA groups), pooled values as e4m3 in raw
// units.  Masks (todo mask of a chunk, causal mask of a diagonal block) enter the logits as one more k-step, see
// sparse_attn_kernel.
//
// One CTA: 256 threads, 16 KB Q + 32 KB K stage + 16 KB V stage + 32 KB P + 8 KB mask operands, 256 TMEM columns
// (S [0,128), O [128,256)).  Two CTAs per SM.
// Roles: warps 0..3 softmax + epilogue; warp 4 K producer; warp 5 UMMA issuer (and TMEM owner); warp 6 V producer;
// warp 7 unit set-up (next unit, list validation, correction masks, Q staging).
// The issuer keeps two cursors over the same sequence of iterations -- the next S to issue and the O += P V
// being fed -- and polls: while it waits for the next slice of P it issues the next S as soon as its K tile has
// landed and the S columns are free.  The S cursor runs at most one iteration ahead, also across unit boundaries.
//
// Every wait is bounded (see ptx.cuh); the polling loops of the issuer carry their own cycle budget.
#pragma once
#include "sparse_attn.cuh"

namespace fp2 {

struct AttnFp8Cfg {
  static constexpr int kThreads = 256;
  static constexpr int kCtasPerSm = 2;
  static constexpr int kSlices = 4;          // slices of P per iteration: 32 key columns = one K = 32 step, hi and lo
  static constexpr int kSlotBytes = 4096;    // 128 rows x 32 bytes
  static constexpr int kQBytes = kRawBytes, kKBytes = 2 * kRawBytes, kVBytes = kRawBytes;
  static constexpr int kPBytes = 2 * kSlices * kSlotBytes;
  static constexpr int kBiasBytes = 4096;
  static constexpr int kSmemBytes = 1024 + kQBytes + kKBytes + kVBytes + kPBytes + 2 * kBiasBytes;
  static constexpr int kSetupThreads = 32;
  static constexpr int kRegsBase = 128;
  static constexpr int kRegsService = 56;
  static constexpr int kRegsSoftmax = 200;
  static constexpr int kRegsAfterMove = (kThreads - 128) * kRegsService + 128 * kRegsSoftmax;
  static_assert(kRegsAfterMove <= kThreads * kRegsBase, "register budget: setmaxnreg.inc would wait forever");
  static_assert(kThreads * kRegsBase * kCtasPerSm <= 65536, "two CTAs must fit the register file");
};

// A polling loop's cycle budget (mbar_wait carries its own; a thread that watches several barriers polls them with
// mbar_test and asks this whether to give up).
struct PollBudget {
  long long t0;
  int spins;
  __device__ __forceinline__ void start() { t0 = 0; spins = 0; }
  // false: keep polling; true: give up (abort flag seen, or the budget ran out and was recorded)
  __device__ __forceinline__ bool expired(const WaitCtx& ctx, int where) {
    if (((++spins) & 63) != 0) return false;
    if (t0 == 0) t0 = clock64();
    if (*ctx.abort) {
      if (where >= 200 && where < 700) ctx.status[3 + (where / 100 - 2)] = where;
      return true;
    }
    if (clock64() - t0 > ctx.budget) {
      *ctx.abort = 1;
      if (atomicCAS(ctx.status + ST_TIMEOUT, 0, 1) == 0) ctx.status[ST_WHERE] = where;
      return true;
    }
    return false;
  }
};

// (p0, p1) -> two e4m3 bytes (hi) and two e5m2 bytes (lo) with p ~ hi + lo (Eq. 15 with a second term).
__device__ __forceinline__ void split_p_pair(float p0, float p1, uint32_t& hi2, uint32_t& lo2) {
  asm("{\n .reg .b16 h, l;\n .reg .b32 hh, ph, d;\n"
      " cvt.rn.satfinite.e4m3x2.f32 h, %3, %2;\n"
      " cvt.rn.f16x2.e4m3x2 hh, h;\n"
      " cvt.rn.f16x2.f32 ph, %3, %2;\n"
      " sub.rn.f16x2 d, ph, hh;\n"
      " cvt.rn.satfinite.e5m2x2.f16x2 l, d;\n"
      " cvt.u32.u16 %0, h;\n cvt.u32.u16 %1, l;\n}"
      : "=r"(hi2), "=r"(lo2)
      : "f"(p0), "f"(p1));
}

__global__ void __launch_bounds__(AttnFp8Cfg::kThreads, AttnFp8Cfg::kCtasPerSm)
sparse_attn_fp8_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                       const __grid_constant__ CUtensorMap map_kbar, const __grid_constant__ CUtensorMap map_kbar_lo,
                       const __grid_constant__ CUtensorMap map_vbar, const __grid_constant__ CUtensorMap map_q,
                       AttnArgs A, DevParams P) {
  using Cfg = AttnFp8Cfg;
  constexpr int kSetupThreads = Cfg::kSetupThreads;
  constexpr int NS = Cfg::kSlices;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                      // 16 KB raw e4m3, K-major, 128-byte swizzle
  uint8_t* sK = sQ + Cfg::kQBytes;         // 32 KB: one raw K tile, or hi | lo of a chunk of pooled keys
  uint8_t* sV = sK + Cfg::kKBytes;         // 16 KB raw e4m3 [128 tokens][128 d]: MN-major operand as TMA writes it
  uint8_t* sP = sV + Cfg::kVBytes;         // slice s: hi at s * 8 KB, lo 4 KB further; row r of a slot at
                                           // (r / 8) * 256 + (r % 8) * 16, bytes 16..31 of the row 128 bytes on
  uint8_t* sHot = sP + Cfg::kPBytes;       // mask operands, see sparse_attn_kernel
  uint8_t* sBias = sHot + Cfg::kBiasBytes;

  __shared__ TileInfo info[2];
  __shared__ uint32_t sel_bits[kMaxBlocks / 32];
  __shared__ uint64_t info_full[2], info_empty[2], q_full, q_empty;
  // With G the iteration's index counted over the whole kernel: the barriers below complete once per iteration
  // (the phase of iteration G has parity G & 1), except pv_done, which alternates between two barriers.
  __shared__ uint64_t k_full, v_full[2];   // v_full[h]: tokens [64 h, 64 h + 64) of the V tile have landed
  __shared__ uint64_t s_done;      // S = Q K^T (G) has completed: the logits are in TMEM, the K stage and sBias are free
  __shared__ uint64_t s_free;      // every softmax thread has the logits of iteration G in registers: S may be overwritten
  __shared__ uint64_t p_full[NS];  // slice s of P (G) is in shared memory (128 arrivals)
  __shared__ uint64_t p_done[NS - 1];   // the MMAs of slices 0..s of O += P V (G) have completed: their slots are free, after
                                        // slice 1 so is the first half of the V stage; the last slice reports on pv_done
  __shared__ uint64_t pv_done[2];  // [G & 1], phase (G >> 1) & 1: O += P V (G) has completed -- V stage free, O at rest
  __shared__ uint64_t drain_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ int ndiag_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  WaitCtx ctx{A.status, &abort_flag};

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(&info_full[i], 1);
      mbar_init(&info_empty[i], 3 + 128);   // K producer, V producer, issuer, softmax threads
    }
    mbar_init(&q_full, kSetupThreads);
    mbar_init(&q_empty, 1);
    mbar_init(&k_full, 1);
    mbar_init(&v_full[0], 1);
    mbar_init(&v_full[1], 1);
    mbar_init(&s_done, 1);
    mbar_init(&s_free, 128);
    mbar_init(&pv_done[0], 1);
    mbar_init(&pv_done[1], 1);
    mbar_init(&drain_bar, 1);
    for (int i = 0; i < NS; ++i) mbar_init(&p_full[i], 128);
    for (int i = 0; i < NS - 1; ++i) mbar_init(&p_done[i], 1);
    fence_barrier_init();
  }
  // K / V stages start zeroed: rows of pages past the end of a sequence are never loaded, and whatever sits
  // there is multiplied by probabilities that are exactly zero, so it must be finite.
  for (int i = tid; i < (Cfg::kKBytes + Cfg::kVBytes) / 16; i += Cfg::kThreads)
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

  auto wait_pv = [&](uint32_t G, int where) { mbar_wait(&pv_done[G & 1], (G >> 1) & 1, ctx, where); };

  if (warp == 7) {
    // =============================== unit set-up + Q staging ===============================
    setmaxnreg_dec<Cfg::kRegsService>();
    const int t32 = lane;
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      if (it >= 2) mbar_wait(&info_empty[slot], ((it >> 1) - 1) & 1, ctx, 201);
      TileInfo& ti = info[slot];
      if (t32 == 0) {
        const int w = atomicAdd(A.work_counter, 1);
        const int n_units = A.unit_split ? *A.n_units : P.nseg;
        // after a wait has run out somewhere in this CTA no further unit is started
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
        } else {
          ti.valid = 0;
        }
      }
      __syncwarp();
      const bool valid = ti.valid != 0;
      if (valid && !ti.dense) {
        const SegInfo& sg = ti.sg;
        const int32_t* list = A.blk_idx + sg.off;
        const int T = ti.T;
        const int nwords = (sg.J_lo + 31) >> 5;
        const bool corr = P.use_correction != 0;
        if (corr)
          for (int w = t32; w < nwords; w += kSetupThreads) sel_bits[w] = 0u;
        __syncwarp();
        bool bad = false;
        int nd = 0;
        for (int k = t32; k < T; k += kSetupThreads) {
          const int J = list[k];
          if (J < 0 || J > sg.J_hi || (k > 0 && list[k - 1] >= J)) bad = true;
          if (corr && J >= 0 && J < sg.J_lo) atomicOr(&sel_bits[J >> 5], 1u << (J & 31));
          nd += J >= sg.J_lo;
        }
        if (bad) atomicOr(A.status + ST_BAD_LIST, 1);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) nd += __shfl_xor_sync(0xffffffffu, nd, o);
        if (t32 == 0) ti.ndiag = nd;
        __syncwarp();
        if (corr) {
          const int nch = (sg.J_lo + 127) >> 7;
          for (int c = t32; c < nch; c += kSetupThreads) {
#pragma unroll
            for (int w = 0; w < 4; ++w) {
              const int first = c * 128 + w * 32;
              uint32_t validm = 0u;
              if (first + 32 <= sg.J_lo) validm = 0xffffffffu;
              else if (first < sg.J_lo) validm = (1u << (sg.J_lo - first)) - 1u;
              ti.todo[c][w] = (first < sg.J_lo ? ~sel_bits[first >> 5] : 0u) & validm;
            }
          }
          __syncwarp();
          if (t32 == 0) {
            int n = 0;
            for (int c = 0; c < nch; ++c)
              if (ti.todo[c][0] | ti.todo[c][1] | ti.todo[c][2] | ti.todo[c][3]) ti.chunk_id[n++] = c;
            ti.nchunk = n;
          }
        }
      }
      __syncwarp();
      if (t32 == 0 && valid) {   // Eq. 18: part u of U takes iterations [u ceil(n / U), min((u + 1) ceil(n / U), n))
        const int n = ti.T + ti.nchunk, u = ti.it_begin;
        const int step = (n + ti.parts - 1) / ti.parts;
        ti.it_begin = min(u * step, n);
        ti.it_end = min((u + 1) * step, n);
        __threadfence_block();
      }
      __syncwarp();
      if (t32 == 0) mbar_arrive(&info_full[slot]);
      if (!valid) break;
      // Q tile and the one-hot mask operand: wait until every S = Q K^T of the previous unit has completed
      if (it >= 1) mbar_wait(&q_empty, (it - 1) & 1, ctx, 202);
#pragma unroll
      for (int u = 0; u < 4; ++u) {   // sHot: rows 4 t32 .. 4 t32 + 3
        const int row = 4 * t32 + u;
        const int c = P.diag_mma ? (ti.sg.r0 + row) / g - ti.sg.r0 / g : (row & 31);
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) w[k] = (c >> 2) == k ? 0x7bu << ((c & 3) * 8) : 0u;   // e5m2 57344
        uint8_t* dst = sHot + (row >> 3) * 256 + (row & 7) * 16;
        *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(dst + 128) = make_uint4(w[4], w[5], w[6], w[7]);
      }
      fence_proxy_async();
      if (P.q_tma) {
        // PackGQA (Eq. 13) with a group size that divides 128: the tile is 128 / g tokens x g heads, one TMA box of
        // whole 128-byte rows, landing in the swizzled layout the MMA reads.
        if (t32 == 0) {
          const SegInfo& sg = ti.sg;
          const uint64_t pol = l2_policy_evict_first();
          mbar_arrive_expect_tx(&q_full, kRawBytes);
          tma_load_3d_hint(sQ, &map_q, &q_full, 0, sg.h * g, sg.q_tok0 + sg.r0 / g, pol);
        } else {
          mbar_arrive(&q_full);
        }
        continue;
      }
      load_q_raw_async(sQ, A.q, ti.sg, P, t32, kSetupThreads);
      cp_async_wait_all();
      fence_proxy_async();
      mbar_arrive(&q_full);
    }
  } else if (warp == 4) {
    // =============================== K producer (Eq. 22) + mask bias ===============================
    setmaxnreg_dec<Cfg::kRegsService>();
    if (lane == 0) {
      tma_prefetch_desc(&map_k);
      tma_prefetch_desc(&map_kbar);
      tma_prefetch_desc(&map_kbar_lo);
    }
    uint32_t G = 0;
    const uint64_t keep = l2_policy_evict_last();   // K / V pages and pooled means: shared by many tiles
    const int psz = P.page_size, ppb = P.pages_per_block;
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 301);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const SegInfo& sg = ti.sg;
      const int T = ti.T;
      int J_fetched = 0;   // block id of the iteration fetch_pid was last asked for (warp-uniform)
      auto fetch_pid = [&](int i) -> int {
        if (i >= T) return -1;
        int J = ti.dense ? sg.J_hi - i : A.blk_idx[sg.off + T - 1 - i];
        J = max(0, min(J, sg.J_hi));
        J_fetched = J;
        if (lane >= ppb || J * kBlock + lane * psz >= sg.Lk) return -1;
        int pid = A.page_table[(size_t)sg.b * P.max_pages_per_seq + J * ppb + lane];
        if (pid < 0 || pid >= P.num_pages) {
          atomicOr(A.status + ST_BAD_LIST, 2);
          pid = -1;
        }
        return pid;
      };
      // hidden columns of a masked iteration -> sBias; row j = lane * 4 + u gets 32 bytes of which the first nh[u]
      // are -57344 (e5m2 0xfb).  The S = Q K^T that last read sBias has completed (wait 302).
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
        if (G >= 1) mbar_wait(&s_done, (G - 1) & 1, ctx, 302);   // K stage and sBias free
        if (i < T) {
          if (i < ti.ndiag && P.diag_mma) {
            // diagonal block: column j is hidden from the tile's position c iff J * 128 + j > pre + r0 / g + c
            const int t0 = sg.pre + sg.r0 / g - J_cur * kBlock;
            int nh[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) nh[u] = max(0, min(32, lane * 4 + u - t0));
            write_bias(nh);
          }
          const int nvalid = __popc(__ballot_sync(0xffffffffu, pid >= 0));
          if (lane == 0) mbar_arrive_expect_tx(&k_full, (uint32_t)nvalid * psz * 128u);
          __syncwarp();
          if (pid >= 0) tma_load_3d_hint(sK + lane * psz * 128, &map_k, &k_full, 0, sg.h, pid * psz, keep);
        } else {
          const int cid = ti.chunk_id[i - T];
          const uint32_t w = ti.todo[cid][lane >> 3];
          int nh[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) nh[u] = ((w >> ((lane * 4 + u) & 31)) & 1u) ? 0 : 32;
          write_bias(nh);
          if (lane == 0) {
            const int row0 = sg.blk_off + cid * 128;
            mbar_arrive_expect_tx(&k_full, 2 * kRawBytes);
            tma_load_3d_hint(sK, &map_kbar, &k_full, 0, sg.h, row0, keep);
            tma_load_3d_hint(sK + kRawBytes, &map_kbar_lo, &k_full, 0, sg.h, row0, keep);
          }
        }
        __syncwarp();
      }
      if (lane == 0) mbar_arrive(&info_empty[slot]);
    }
  } else if (warp == 6) {
    // =============================== V producer ===============================
    // Boxes of vrows = min(page size, 64) token rows; lane b loads box b of the block (tokens [b vrows, (b+1) vrows)),
    // which lies in half (b vrows) / 64 of the stage.  A chunk of pooled values comes in two boxes of 64 rows.
    setmaxnreg_dec<Cfg::kRegsService>();
    if (lane == 0) {
      tma_prefetch_desc(&map_v);
      tma_prefetch_desc(&map_vbar);
    }
    uint32_t G = 0;
    const uint64_t keep = l2_policy_evict_last();
    const int psz = P.page_size;
    const int vrows = psz < 64 ? psz : 64;
    const int tok0 = lane * vrows;            // first token of this lane's box within the block
    const int half = tok0 >> 6;
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 311);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const SegInfo& sg = ti.sg;
      const int T = ti.T;
      auto fetch_row = [&](int i) -> int {   // first cache slot of this lane's box, or -1
        if (i >= T || tok0 >= kBlock) return -1;
        int J = ti.dense ? sg.J_hi - i : A.blk_idx[sg.off + T - 1 - i];
        J = max(0, min(J, sg.J_hi));
        if (J * kBlock + tok0 >= sg.Lk) return -1;
        const int pid = A.page_table[(size_t)sg.b * P.max_pages_per_seq + J * P.pages_per_block + tok0 / psz];
        if (pid < 0 || pid >= P.num_pages) {
          atomicOr(A.status + ST_BAD_LIST, 2);
          return -1;
        }
        return pid * psz + tok0 % psz;
      };
      int row_next = fetch_row(ti.it_begin);
      for (int i = ti.it_begin; i < ti.it_end; ++i, ++G) {
        const int vrow = row_next;
        row_next = fetch_row(i + 1);
        const bool exact = i < T;
        const int t0 = exact ? tok0 : lane * 64;
        const int crow = sg.blk_off + (exact ? 0 : ti.chunk_id[i - T] * 128) + t0;
        const bool mine0 = exact ? (vrow >= 0 && half == 0) : lane == 0;
        const bool mine1 = exact ? (vrow >= 0 && half == 1) : lane == 1;
        const uint32_t box_bytes = (uint32_t)(exact ? vrows : 64) * 128u;
        const int n0 = __popc(__ballot_sync(0xffffffffu, mine0)), n1 = __popc(__ballot_sync(0xffffffffu, mine1));
        const CUtensorMap* mp = exact ? &map_v : &map_vbar;
        const int rr = exact ? vrow : crow;
        // first half: free when the MMAs of slices 0 and 1 of O += P V (G-1) have completed
        if (G >= 1) mbar_wait(&p_done[1], (G - 1) & 1, ctx, 312);
        if (lane == 0) mbar_arrive_expect_tx(&v_full[0], n0 * box_bytes);
        __syncwarp();
        if (mine0) tma_load_3d_hint(sV + t0 * 128, mp, &v_full[0], 0, sg.h, rr, keep);
        // second half: free when all of O += P V (G-1) has completed
        if (G >= 1) wait_pv(G - 1, 313);
        if (lane == 0) mbar_arrive_expect_tx(&v_full[1], n1 * box_bytes);
        __syncwarp();
        if (mine1) tma_load_3d_hint(sV + t0 * 128, mp, &v_full[1], 0, sg.h, rr, keep);
        __syncwarp();
      }
      if (lane == 0) mbar_arrive(&info_empty[slot]);
    }
  } else if (warp == 5) {
    // =============================== UMMA issuer ===============================
    setmaxnreg_dec<Cfg::kRegsService>();
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(128, 128, 0, 0, 0, 0);      // e4m3 x e4m3, both K-major
      constexpr uint32_t idesc_pv_hi = make_idesc(128, 128, 0, 0, 0, 1);   // A = P_hi e4m3 K-major, B = V e4m3 MN-major
      constexpr uint32_t idesc_pv_lo = make_idesc(128, 128, 1, 0, 0, 1);   // A = P_lo e5m2
      constexpr uint32_t idesc_bias = make_idesc(128, 128, 1, 1, 0, 0);    // e5m2 x e5m2
      const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV), p_addr = smem_u32(sP);
      const uint64_t hot_desc = make_smem_desc_plain(smem_u32(sHot), 128, 256);
      const uint64_t bias_desc = make_smem_desc_plain(smem_u32(sBias), 128, 256);
      // ---- S cursor: the next S = Q K^T to issue is iteration iS of unit itS, global index GS ----
      uint32_t GS = 0;
      int itS = 0, iS = 0, i1S = 0, TS = 0, ndS = 0;
      bool s_open = false;   // info and Q of unit itS have been seen
      bool s_end = false;    // the S cursor has met the terminating (invalid) unit
      // Tries to issue the next S; with `block` it waits (bounded) for whatever is missing.  Returns true if an S
      // was issued.
      auto issue_next_s = [&](bool block) -> bool {
        while (!s_end) {
          if (!s_open) {
            const int slot = itS & 1;
            if (block) mbar_wait(&info_full[slot], (itS >> 1) & 1, ctx, 403);
            else if (!mbar_test(&info_full[slot], (itS >> 1) & 1)) return false;
            if (*ctx.abort) return false;
            const TileInfo& t = info[slot];
            if (!t.valid) {
              s_end = true;
              return false;
            }
            if (block) mbar_wait(&q_full, itS & 1, ctx, 404);
            else if (!mbar_test(&q_full, itS & 1)) return false;
            if (t.it_end == t.it_begin) {   // nothing to do for this unit: nothing reads Q, release it at once
              umma_commit(&q_empty);
              ++itS;
              continue;
            }
            iS = t.it_begin;
            i1S = t.it_end;
            TS = t.T;
            ndS = P.diag_mma ? t.ndiag : 0;
            s_open = true;
          }
          if (block) {
            mbar_wait(&k_full, GS & 1, ctx, 405);
            if (GS >= 1) mbar_wait(&s_free, (GS - 1) & 1, ctx, 406);
          } else {
            if (!mbar_test(&k_full, GS & 1)) return false;
            if (GS >= 1 && !mbar_test(&s_free, (GS - 1) & 1)) return false;
          }
          if (*ctx.abort) return false;
          tc_fence_after();
          // raw e4m3 operands, 32 elements (= 32 bytes of the swizzled row) per MMA; a correction chunk adds the lo
          // part of the pooled keys on top of the hi part
          const int parts = iS < TS ? 1 : 2;
          for (int part = 0; part < parts; ++part) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              umma_f8_ss(tmem, make_smem_desc_sw128(q_addr + ks * 32, 16, 1024),
                         make_smem_desc_sw128(k_addr + part * kRawBytes + ks * 32, 16, 1024), idesc_qk, (part | ks) != 0);
          }
          if (iS >= TS || iS < ndS) umma_f8_ss(tmem, hot_desc, bias_desc, idesc_bias, 1u);   // masked iteration
          umma_commit(&s_done);
          ++GS;
          if (++iS == i1S) {
            umma_commit(&q_empty);   // every S = Q K^T of the unit has been issued: Q is free when they complete
            s_open = false;
            ++itS;
          }
          return true;
        }
        return false;
      };
      // ---- O += P V cursor ----
      uint32_t GP = 0;
      for (int it = 0; !*ctx.abort; ++it) {
        const int slot = it & 1;
        mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 407);
        const TileInfo& ti = info[slot];
        if (!ti.valid) break;
        const int i0 = ti.it_begin, i1 = ti.it_end;
        for (int i = i0; i < i1 && !*ctx.abort; ++i, ++GP) {
          while (GS <= GP && !*ctx.abort)   // the logits of this iteration must be on their way
            if (!issue_next_s(true)) break;
#pragma unroll 1
          for (int s = 0; s < NS; ++s) {
            uint64_t* vbar = &v_full[s >> 1];
            PollBudget pb;
            pb.start();
            // this k-step needs its slice of P and its half of V; meanwhile: the next iteration's logits, as soon
            // as they can go
            while (!(mbar_test(&p_full[s], GP & 1) && mbar_test(vbar, GP & 1))) {
              if (GS == GP + 1) issue_next_s(false);
              if (pb.expired(ctx, 401)) break;
            }
            if (*ctx.abort) break;
            tc_fence_after();
            const uint64_t vd = make_smem_desc_sw128(v_addr + s * 4096, 4096, 1024);
            umma_f8_ss(tmem + 128, make_smem_desc_plain(p_addr + s * 2 * Cfg::kSlotBytes, 128, 256), vd, idesc_pv_hi,
                       (i > i0) || s > 0);
            umma_f8_ss(tmem + 128, make_smem_desc_plain(p_addr + (s * 2 + 1) * Cfg::kSlotBytes, 128, 256), vd,
                       idesc_pv_lo, 1u);
            if (s < NS - 1) umma_commit(&p_done[s]);
          }
          umma_commit(&pv_done[GP & 1]);
        }
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else {
    // =============================== softmax warpgroup + epilogue ===============================
    setmaxnreg_inc<Cfg::kRegsSoftmax>();
    const int row = warp * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t s_addr = lane_base;
    const uint32_t o_addr = lane_base + 128;
    const uint32_t p_row = smem_u32(sP) + (row >> 3) * 256 + (row & 7) * 16;   // this row inside a slot
    uint32_t G = 0;
    const uint64_t stream_pol = l2_policy_evict_first();   // outputs are written once and not read here
    for (int it = 0;; ++it) {
      const int slot = it & 1;
      mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 501);
      const TileInfo& ti = info[slot];
      if (!ti.valid) break;
      const int T = ti.T;
      const bool dense = ti.dense != 0;
      const int J_hi = ti.sg.J_hi, J_lo = ti.sg.J_lo;
      const int32_t* list = A.blk_idx + ti.sg.off;
      const int r = ti.sg.r0 + row;
      const int pos = ti.sg.pre + r / g;
      // logit multiplier in log2 units (Eq. 15): the MMAs see raw e4m3 values (pooled keys included), so every
      // logit of a row carries q_scale * k_scale; the output carries v_scale
      const float cs_all = P.scale_log2 * A.q_scale[ti.sg.h * g + r % g] * A.k_scale[ti.sg.h];
      const float out_scale = A.v_scale[ti.sg.h];
      // The mask bias is -3.3e9 in raw units; with scales so small that this is no longer far below every visible
      // logit of the row, the warp masks in TMEM as well.
      const bool weak_bias = __any_sync(0xffffffffu, !(cs_all * 3.0e9f > 256.f));
      float m = -INFINITY, l = 0.f;
      const int i0 = ti.it_begin, i1 = ti.it_end;
      int J_next = (!dense && i0 < T) ? list[T - 1 - i0] : 0;   // block id of the next exact iteration, fetched ahead
      for (int i = i0; i < i1; ++i, ++G) {
        bool need_mask = false;
        int tok_lim = 1 << 30;     // exact block: columns j with j <= tok_lim are visible
        uint32_t cm0 = 0xffffffffu, cm1 = 0xffffffffu, cm2 = 0xffffffffu, cm3 = 0xffffffffu;
        float shift = 4.0f;        // p = 2^(x - m + 4): see the head of the file
        if (i < T) {
          int J = dense ? J_hi - i : J_next;
          if (!dense && i + 1 < T) J_next = list[T - 2 - i];
          J = max(0, min(J, J_hi));
          need_mask = J >= J_lo && (!P.diag_mma || weak_bias);   // else the causal mask is in the logits already
          tok_lim = pos - J * kBlock;
        } else {
          shift = 11.0f;  // + log2(128): one pooled row stands for a full block (Eq. 6); the todo mask is in the logits
          if (weak_bias) {
            const int c = ti.chunk_id[i - T];
            cm0 = ti.todo[c][0];
            cm1 = ti.todo[c][1];
            cm2 = ti.todo[c][2];
            cm3 = ti.todo[c][3];
            need_mask = true;
          }
        }
        mbar_wait(&s_done, G & 1, ctx, 502);
        tc_fence_after();
        if (need_mask) mask_row(s_addr, tok_lim, cm0, cm1, cm2, cm3);
        uint32_t x[128];
        // row maximum in the frame of m: scaled logit + (shift - 4)
        const float mx = fmaf(row_load_max(s_addr, x), cs_all, shift - 4.0f);  // cs > 0: scaling commutes with the maximum
        tc_fence_before();
        mbar_arrive(&s_free);   // the logits are in registers: the next S may overwrite the columns
        const float m_new = fmaxf(m, mx);
        // lazy rescale: only when some row of the warp moved its maximum by more than 2^4 (so p <= 2^8).  O must be at
        // rest: S (G) was issued ahead of O += P V (G-1), so wait for that one explicitly.
        if (__any_sync(0xffffffffu, m_new > m + 4.0f)) {
          const float f = (m == -INFINITY) ? 0.f : ex2(m - m_new);
          if (i > i0) {
            wait_pv(G - 1, 505);
            tc_fence_after();
#pragma unroll 1
            for (int k = 0; k < 4; ++k) {
              uint32_t rr[32];
              tmem_ld32(o_addr + k * 32, rr);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) rr[j] = __float_as_uint(__uint_as_float(rr[j]) * f);
              tmem_st32(o_addr + k * 32, rr);
            }
            tmem_wait_st();
            tc_fence_before();
          }
          l *= f;
          m = m_new;
        }
        // a row with nothing visible so far has m = -inf and only -inf logits: exponent against 0 -> zeros
        const float neg_m = (m == -INFINITY) ? shift : shift - m;
        const uint64_t cs2 = f2_pack(cs_all, cs_all), nm2 = f2_pack(neg_m, neg_m);
        uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
        for (int s = 0; s < NS; ++s) {
          // the slot was last read by the MMAs of slice s of the previous iteration
          if (G >= 1) {
            if (s < NS - 1) mbar_wait(&p_done[s], (G - 1) & 1, ctx, 504);
            else wait_pv(G - 1, 506);
          }
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {   // four columns -> one word of hi, one of lo
            uint32_t h2[2], l2[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const int c = s * 32 + 4 * j + 2 * u;
              const uint64_t x2 = f2_fma(f2_pack(__uint_as_float(x[c]), __uint_as_float(x[c + 1])), cs2, nm2);
              float x0, x1;
              f2_unpack(x2, x0, x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              sum2[(2 * j + u) & 3] = f2_add(sum2[(2 * j + u) & 3], f2_pack(p0, p1));
              split_p_pair(p0, p1, h2[u], l2[u]);
            }
            hi[j] = h2[0] | (h2[1] << 16);
            lo[j] = l2[0] | (l2[1] << 16);
          }
          const uint32_t dst = p_row + s * 2 * Cfg::kSlotBytes;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + 128), "r"(hi[4]), "r"(hi[5]), "r"(hi[6]), "r"(hi[7]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + Cfg::kSlotBytes), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + Cfg::kSlotBytes + 128), "r"(lo[4]), "r"(lo[5]), "r"(lo[6]), "r"(lo[7]) : "memory");
          fence_proxy_async();
          mbar_arrive(&p_full[s]);
        }
        float a0, a1;
        f2_unpack(f2_add(f2_add(sum2[0], sum2[1]), f2_add(sum2[2], sum2[3])), a0, a1);
        l += a0 + a1;
      }
      // ------------------------------ epilogue ------------------------------
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
      if (ti.parts > 1) {
        // one part of a split segment (Eq. 18): leave (O, m, l) unnormalised for the merge kernel; l and O carry the
        // 2^4 of the probabilities, which cancels in O / l, and m is reported in the frame of l
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
        A.part_ml[(size_t)ti.slot * 128 + row] = make_float2(have_o ? m - 4.0f : -INFINITY, have_o ? l : 0.f);
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
        A.lse[(size_t)head * P.total_q + tok] = (m - 4.0f + log2f(l)) * 0.6931471805599453f;
      tc_fence_before();
      mbar_arrive(&info_empty[slot]);
    }
  }
  // teardown: on the normal path every barrier has been consumed and every MMA has completed.  After an abort MMAs
  // and bulk copies may still be in flight: wait (bounded) for the MMAs, give the copies time, then release TMEM.
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
