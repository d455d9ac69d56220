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
// Roles (12 warps):
//   warps 0-3  softmax warpgroup 0: iterations 0, 2, 4, ...  (TMEM: S0 / P0, O0)
//   warps 4-7  softmax warpgroup 1: iterations 1, 3, 5, ...  (TMEM: S1 / P1, O1)
//       each keeps its own running (max, sum) and its own O accumulator; the two are merged in the epilogue,
//       so the warpgroups never synchronise inside the main loop and one's exponentials overlap the other's MMAs.
//   warp 8     TMA producer: K / V pages through the page table into two rings (Eq. 22)
//   warp 9     UMMA issuer: S = Q K^T (SS), O += P V (P read from TMEM, V MN-major from shared memory)
//   warps 10-11 tile set-up: fetch the next unit, validate its list, build the correction masks, stage Q
//
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P (BF16 pairs) overwrites the first 64
// columns of its S buffer.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"
#include "ptx.cuh"
#include "score_select.cuh"  // load_q_tile_bf16

namespace fp2 {

constexpr int kAttnThreads = 384;
constexpr int kNK = 3;  // K ring stages (32 KB each)
constexpr int kNV = 2;  // V ring stages
constexpr int kTileBytes = 32768;
constexpr int kAttnSmemBytes = 1024 + kTileBytes * (1 + kNK + kNV) + 2048;

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
// thread's row with -inf in TMEM, so that the softmax step itself carries no mask logic.  Column j stays
// visible iff j <= tok_lim and bit j of cm is set.  (Predicating the mask into the softmax body cost 2.5x on
// every iteration, masked or not.)
__device__ __forceinline__ void mask_tile(uint32_t s_addr, int tok_lim, const uint32_t* cm) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const bool all_vis = (k * 32 + 31 <= tok_lim) && (cm[k] == 0xffffffffu);
    if (__all_sync(0xffffffffu, all_vis)) continue;
    uint32_t rr[32];
    tmem_ld32(s_addr + k * 32, rr);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const bool vis = (k * 32 + j <= tok_lim) && ((cm[k] >> j) & 1u);
      rr[j] = vis ? rr[j] : 0xff800000u;  // -inf
    }
    tmem_st32(s_addr + k * 32, rr);
  }
  tmem_wait_st();
}

// Online-softmax step of one thread (= one query row) over a 128-column logit tile held in TMEM at s_addr:
// updates the running maximum m (log2 units) and sum l, rescales the row of the O accumulator at o_addr when
// the maximum moved by more than 2^8 (lazy rescale; decided per warp because TMEM accesses are warp-wide),
// and overwrites the first 64 columns of the tile with P = 2^(x - m) as BF16 pairs (the A operand of P V).
//   x_j = s_j * cs + shift
__device__ __forceinline__ void softmax_tile(uint32_t s_addr, uint32_t o_addr, float cs, float shift, bool have_o,
                                             float& m, float& l) {
  // pass 1: row maximum.  Four TMEM loads in flight behind one wait, eight independent max chains.
  float mx;
  {
    uint32_t sv[128];
#pragma unroll
    for (int k = 0; k < 4; ++k) tmem_ld32(s_addr + k * 32, reinterpret_cast<uint32_t(&)[32]>(sv[k * 32]));
    tmem_wait_ld();
    float mx8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) mx8[c] = __uint_as_float(sv[c]);
#pragma unroll
    for (int j = 8; j < 128; ++j) mx8[j & 7] = fmaxf(mx8[j & 7], __uint_as_float(sv[j]));
    mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
               fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
  }
  mx = fmaf(mx, cs, shift);  // cs > 0: scaling commutes with the maximum
  const float m_new = fmaxf(m, mx);
  const bool need = m_new > m + 8.0f;
  if (__any_sync(0xffffffffu, need)) {
    const float f = (m == -INFINITY) ? 0.f : ex2(m - m_new);
    if (have_o) {
#pragma unroll
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
  // pass 2: p = 2^(x - m).  Chunk k of P lands on columns [16k, 16k+16), which pass 2 has already read; the
  // load of chunk k+1 is in flight while chunk k is exponentiated.  A row with nothing visible so far has
  // m = -inf and only -inf logits: its exponent is taken against 0 and gives exact zeros.
  const float neg_m = (m == -INFINITY) ? shift : shift - m;
  float sum4[4] = {0.f, 0.f, 0.f, 0.f};
  uint32_t buf[2][32];
  tmem_ld32(s_addr, buf[0]);
  tmem_wait_ld();
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if (k < 3) tmem_ld32(s_addr + (k + 1) * 32, buf[(k + 1) & 1]);
    uint32_t pk[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float p0 = ex2(fmaf(__uint_as_float(buf[k & 1][2 * j]), cs, neg_m));
      const float p1 = ex2(fmaf(__uint_as_float(buf[k & 1][2 * j + 1]), cs, neg_m));
      sum4[j & 3] += p0 + p1;
      pk[j] = pack_bf16x2(p0, p1);
    }
    if (k < 3) tmem_wait_ld();
    tmem_st16(s_addr + k * 16, pk);
  }
  l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
}

template <bool FP8>
__global__ void __launch_bounds__(kAttnThreads, 1)
sparse_attn_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const __grid_constant__ CUtensorMap map_kbar, const __grid_constant__ CUtensorMap map_vbar,
                   AttnArgs A, DevParams P) {
  static_assert(!FP8, "FP8 path is built separately");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + kTileBytes;
  uint8_t* sV = sK + kNK * kTileBytes;
  float* sML = reinterpret_cast<float*>(sV + kNV * kTileBytes);  // [2 wg][2 (m,l)][128]

  __shared__ TileInfo info[2];
  __shared__ uint32_t sel_bits[2][kMaxBlocks / 32];
  __shared__ uint64_t info_full[2], info_empty[2], q_full, q_empty, tile_done;
  __shared__ uint64_t k_full[kNK], k_empty[kNK], v_full[kNV], v_empty[kNV];
  __shared__ uint64_t s_full[2], p_ready[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  WaitCtx ctx{A.status, &abort_flag};

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(&info_full[i], 1);
      mbar_init(&info_empty[i], 2 + 256);
      mbar_init(&s_full[i], 1);
      mbar_init(&p_ready[i], 128);
    }
    mbar_init(&q_full, 64);
    mbar_init(&q_empty, 1);
    mbar_init(&tile_done, 1);
    for (int i = 0; i < kNK; ++i) { mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < kNV; ++i) { mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1); }
    fence_barrier_init();
  }
  // K / V rings start zeroed: rows of pages past the end of a sequence are never loaded, and whatever sits
  // there is multiplied by probabilities that are exactly zero, so it must be finite.
  for (int i = tid; i < (kNK + kNV) * kTileBytes / 16; i += kAttnThreads)
    reinterpret_cast<uint4*>(sK)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 9) {
    tmem_alloc(&tmem_base_s, 512);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const int g = P.group;

  if (warp >= 10) {
    // =============================== tile set-up + Q staging ===============================
    setmaxnreg_dec<56>();
    const int t64 = tid - 320;
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
      // Q tile: wait until every S = Q K^T of the previous unit has completed, then overwrite
      if (it >= 1) mbar_wait(&q_empty, (it - 1) & 1, ctx, 202);
      load_q_tile_bf16<FP8, 4>(sQ, A.q, ti.sg, P, t64, 64);
      fence_proxy_async();
      mbar_arrive(&q_full);
    }
  } else if (warp == 8) {
    // =============================== TMA producer ===============================
    setmaxnreg_dec<56>();
    if (lane == 0) {
      tma_prefetch_desc(&map_k);
      tma_prefetch_desc(&map_v);
      tma_prefetch_desc(&map_kbar);
      tma_prefetch_desc(&map_vbar);
    }
    uint32_t kc = 0, vc = 0;
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
      for (int i = 0; i < n_it; ++i) {
        const int ks = kc % kNK, vs = vc % kNV;
        uint8_t* dK = sK + ks * kTileBytes;
        uint8_t* dV = sV + vs * kTileBytes;
        if (i < T) {
          int J = ti.dense ? sg.J_hi - i : list[T - 1 - i];
          J = max(0, min(J, sg.J_hi));
          int pid = -1;
          if (lane < ppb) {
            const int tok0 = J * kBlock + lane * psz;
            if (tok0 < sg.Lk) {
              pid = pt[J * ppb + lane];
              if (pid < 0 || pid >= P.num_pages) {
                atomicOr(A.status + ST_BAD_LIST, 2);
                pid = -1;
              }
            }
          }
          const int nvalid = __popc(__ballot_sync(0xffffffffu, pid >= 0));
          const uint32_t bytes = (uint32_t)nvalid * psz * 256u;
          if (kc >= kNK) mbar_wait(&k_empty[ks], ((kc / kNK) - 1) & 1, ctx, 302);
          if (lane == 0) mbar_arrive_expect_tx(&k_full[ks], bytes);
          __syncwarp();
          if (pid >= 0) {
            tma_load_3d(dK + lane * psz * 128, &map_k, &k_full[ks], 0, sg.h, pid * psz);
            tma_load_3d(dK + 16384 + lane * psz * 128, &map_k, &k_full[ks], 64, sg.h, pid * psz);
          }
          if (vc >= kNV) mbar_wait(&v_empty[vs], ((vc / kNV) - 1) & 1, ctx, 303);
          if (lane == 0) mbar_arrive_expect_tx(&v_full[vs], bytes);
          __syncwarp();
          if (pid >= 0) {
            tma_load_3d(dV + lane * psz * 128, &map_v, &v_full[vs], 0, sg.h, pid * psz);
            tma_load_3d(dV + 16384 + lane * psz * 128, &map_v, &v_full[vs], 64, sg.h, pid * psz);
          }
        } else {
          const int row0 = sg.blk_off + ti.chunk_id[i - T] * 128;
          if (kc >= kNK) mbar_wait(&k_empty[ks], ((kc / kNK) - 1) & 1, ctx, 304);
          if (lane == 0) {
            mbar_arrive_expect_tx(&k_full[ks], kTileBytes);
            tma_load_3d(dK, &map_kbar, &k_full[ks], 0, sg.h, row0);
            tma_load_3d(dK + 16384, &map_kbar, &k_full[ks], 64, sg.h, row0);
          }
          if (vc >= kNV) mbar_wait(&v_empty[vs], ((vc / kNV) - 1) & 1, ctx, 305);
          if (lane == 0) {
            mbar_arrive_expect_tx(&v_full[vs], kTileBytes);
            tma_load_3d(dV, &map_vbar, &v_full[vs], 0, sg.h, row0);
            tma_load_3d(dV + 16384, &map_vbar, &v_full[vs], 64, sg.h, row0);
          }
          __syncwarp();
        }
        ++kc;
        ++vc;
      }
      if (lane == 0) mbar_arrive(&info_empty[slot]);
    }
  } else if (warp == 9) {
    // =============================== UMMA issuer ===============================
    setmaxnreg_dec<56>();
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(128, 128, 1, 1, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(128, 128, 1, 1, 0, 1);
      const uint32_t q_addr = smem_u32(sQ);
      uint32_t kc = 0, vc = 0, pc[2] = {0, 0};
      auto issue_pv = [&](int j) {
        const int b = j & 1;
        mbar_wait(&p_ready[b], pc[b] & 1, ctx, 401);
        ++pc[b];
        const int vs = vc % kNV;
        mbar_wait(&v_full[vs], (vc / kNV) & 1, ctx, 402);
        tc_fence_after();
        const uint32_t v_addr = smem_u32(sV + vs * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t bd = make_smem_desc_sw128(v_addr + ks * 2048, 16384, 1024);
          umma_f16_ts(tmem + 256 + b * 128, tmem + b * 128 + ks * 8, bd, idesc_pv, (j >= 2) || ks > 0);
        }
        umma_commit(&v_empty[vs]);
        ++vc;
      };
      for (int it = 0;; ++it) {
        const int slot = it & 1;
        mbar_wait(&info_full[slot], (it >> 1) & 1, ctx, 403);
        const TileInfo& ti = info[slot];
        if (!ti.valid) break;
        const int n_it = ti.T + ti.nchunk;
        mbar_wait(&q_full, it & 1, ctx, 404);
        for (int i = 0; i < n_it; ++i) {
          const int a = i & 1;
          const int ks_ = kc % kNK;
          mbar_wait(&k_full[ks_], (kc / kNK) & 1, ctx, 405);
          tc_fence_after();
          const uint32_t k_addr = smem_u32(sK + ks_ * kTileBytes);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
            const uint64_t ad = make_smem_desc_sw128(q_addr + off, 16, 1024);
            const uint64_t bd = make_smem_desc_sw128(k_addr + off, 16, 1024);
            umma_f16_ss(tmem + a * 128, ad, bd, idesc_qk, ks > 0);
          }
          umma_commit(&k_empty[ks_]);
          umma_commit(&s_full[a]);
          ++kc;
          if (i == n_it - 1) umma_commit(&q_empty);
          if (i >= 1) issue_pv(i - 1);
        }
        if (n_it >= 1) issue_pv(n_it - 1);
        else umma_commit(&q_empty);  // empty list: nothing read Q, release it at once
        umma_commit(&tile_done);
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else {
    // =============================== softmax warpgroups + epilogue ===============================
    setmaxnreg_inc<224>();
    const int wg = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_base + wg * 128;
    const uint32_t o_addr = lane_base + 256 + wg * 128;
    uint32_t sc = 0;  // uses of this warpgroup's S buffer so far (phase of s_full[wg])
    const float cs = P.scale_log2;
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
      float m = -INFINITY, l = 0.f;
      int used = 0;
      // block id of this warpgroup's next exact iteration, fetched one iteration ahead
      int J_next = (!ti.dense && wg < T) ? list[T - 1 - wg] : 0;
      for (int i = wg; i < n_it; i += 2, ++used) {
        // iteration kind and masks
        bool need_mask = false;
        int tok_lim = 0;           // exact block: columns j with j <= tok_lim are visible
        uint32_t cm[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
        float shift = 0.f;
        if (i < T) {
          int J = ti.dense ? sg.J_hi - i : J_next;
          if (!ti.dense && i + 2 < T) J_next = list[T - 3 - i];
          J = max(0, min(J, sg.J_hi));
          need_mask = J >= sg.J_lo;
          tok_lim = pos - J * kBlock;
        } else {
          const int c = ti.chunk_id[i - T];
#pragma unroll
          for (int w = 0; w < 4; ++w) cm[w] = ti.todo[c][w];
          shift = 7.0f;  // log2(128): one pooled row stands for a full block (Eq. 6)
          need_mask = true;
          tok_lim = 1 << 30;
        }
        mbar_wait(&s_full[wg], sc & 1, ctx, 502);
        ++sc;
        tc_fence_after();
        if (need_mask) mask_tile(s_addr, tok_lim, cm);
        softmax_tile(s_addr, o_addr, cs, shift, used > 0, m, l);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&p_ready[wg]);
      }
      // ------------------------------ epilogue ------------------------------
      mbar_wait(&tile_done, it & 1, ctx, 503);
      tc_fence_after();
      sML[(wg * 2 + 0) * 128 + row] = m;
      sML[(wg * 2 + 1) * 128 + row] = l;
      named_bar_sync(1, 256);
      const float m0 = sML[0 * 128 + row], l0 = sML[1 * 128 + row];
      const float m1 = sML[2 * 128 + row], l1 = sML[3 * 128 + row];
      const float mm = fmaxf(m0, m1);
      const float f0 = (m0 == -INFINITY) ? 0.f : ex2(m0 - mm);
      const float f1 = (m1 == -INFINITY) ? 0.f : ex2(m1 - mm);
      const float L = l0 * f0 + l1 * f1;
      const float inv = L > 0.f ? 1.0f / L : 0.f;
      const bool have0 = n_it >= 1, have1 = n_it >= 2;
      const bool row_ok = row < sg.nrows;
      const size_t tok = (size_t)sg.q_tok0 + r / g;
      const int head = sg.h * g + r % g;
      __nv_bfloat16* orow = A.out + (tok * P.num_q_heads + head) * kHeadDim + wg * 64;
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        uint32_t a0[32], a1[32];
        if (have0) tmem_ld32(lane_base + 256 + wg * 64 + k * 32, a0);
        if (have1) tmem_ld32(lane_base + 384 + wg * 64 + k * 32, a1);
        tmem_wait_ld();
        uint32_t o[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float v0 = 0.f, v1 = 0.f;
          if (have0) {
            v0 = __uint_as_float(a0[2 * j]) * f0;
            v1 = __uint_as_float(a0[2 * j + 1]) * f0;
          }
          if (have1) {
            v0 = fmaf(__uint_as_float(a1[2 * j]), f1, v0);
            v1 = fmaf(__uint_as_float(a1[2 * j + 1]), f1, v1);
          }
          o[j] = pack_bf16x2(v0 * inv, v1 * inv);
        }
        if (row_ok) {
          uint4* dst = reinterpret_cast<uint4*>(orow + k * 32);
#pragma unroll
          for (int j = 0; j < 4; ++j) dst[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        }
      }
      if (wg == 0 && row_ok && A.lse != nullptr)
        A.lse[(size_t)head * P.total_q + tok] = (mm + log2f(L)) * 0.6931471805599453f;
      tc_fence_before();
      named_bar_sync(1, 256);
      mbar_arrive(&info_empty[slot]);
    }
  }
  // teardown: on the normal path every barrier has been consumed; after an abort give in-flight copies time
  if (abort_flag) __nanosleep(2000000);
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, 512);
}

}  // namespace fp2
