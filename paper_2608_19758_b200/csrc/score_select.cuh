// Fused block scoring and selection (Eq. 19, Eq. 20; Algorithm 1 lines 3-5); persistent, one CTA per SM,
// segments dealt round-robin in heaviest-first order.
//
// For the packed query tile I (128 rows of one KV head) and every candidate block J <= J_hi:
//     s_iJ = scale * q_i . kbar_J,   m_J = max_i s_iJ,   S_J = sum_i 2^{(s_iJ - m_J) log2 e}
// (the per-block max / sum of Eq. 1), then the energy in the log domain  e_J = m_J log2 e + log2 S_J  (the
// global rescale of Eq. 2 / Eq. 20 only adds a constant), threshold  e_J >= log2 alpha + max_J e_J, forced
// sink / window / diagonal blocks, and an ordered compaction of the survivors into the segment's list.
//
// The contraction runs on the tensor cores TRANSPOSED: A = a chunk of 128 pooled keys (rows = TMEM lanes),
// B = the query tile (columns), so that each consumer thread owns one pooled key and the sum over the tile's
// rows is a sum over its own TMEM columns -- no cross-thread reduction in the main loop.  kbar enters as a
// BF16 (hi, lo) pair accumulated into the same fp32 accumulator, which keeps the energies accurate to ~1e-5
// relative; a single BF16 kbar would move them by ~3e-3 and flip list entries.  FP8 inputs: the query tile is
// widened to F16 (exact) and kbar is an F16 (hi, lo) pair.
//
// Roles: warps 0-3 / 4-7 = two consumer warpgroups alternating over chunks (TMEM accumulators 0 / 1); warp 8 = TMA
// producer of kbar pieces; warp 9 = UMMA issuer; warp 10 fetches the next segments and stages their query tiles into
// free Q buffers (by TMA when the tile is a box -- BF16, group size divides 128 --, else with cp.async, widening FP8
// to F16), so that the next tile's MMAs start while the current tile is still being exponentiated; warp 11 applies
// threshold and forced sets and writes the ordered list of tile t beside the scoring of tile t+1.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include "common.cuh"
#include "ptx.cuh"

namespace fp2 {

#ifdef FP2_PROFILE
__device__ long long* g_score_prof = nullptr;   // development builds: [cta][warpgroup][8] cycle counters
#endif
constexpr int kScoreThreads = 384;
constexpr int kScoreInfoSlots = 4;       // segment descriptors in flight
constexpr int kScoreQSlots = 3;           // 32 KB query slots.  BF16: three tiles in flight (two loading while one is
                                         // multiplied; one tile in flight per SM cannot cover the HBM latency-
                                         // bandwidth product).  FP8: two F16 tiles + two raw 16 KB staging tiles.
constexpr int kScoreStages = 3;          // ring of 32 KB pieces: the kbar_hi or the kbar_lo half of a 128-block chunk
constexpr int kScoreRawBytes = 20480;     // FP8: one raw e4m3 box of a query tile (up to 160 rows of 128 bytes)
constexpr int kScoreSmemBytes = 1024 /*align*/ + kScoreQSlots * 32768 + kScoreStages * 32768 + kMaxBlocks * 4 + 2048 +
                                (2 * kScoreRawBytes - 32768);   // the two raw boxes take the third Q slot and 8 KB more

// Query tile -> shared memory in the K-major 128-byte-swizzled layout the UMMA descriptors expect:
// BF16: two 64-column halves of [128 rows x 128 B]; FP8 is widened to BF16 on the way (exact).
// Rows >= nrows are zero-filled.  Called by `nthr` threads with local index `t`.
template <bool FP8, int BATCH = 8>
__device__ __forceinline__ void load_q_tile_bf16(uint8_t* sQ, const uint8_t* __restrict__ q, const SegInfo& sg,
                                                 const DevParams& P, int t, int nthr) {
  const int g = P.group;
  for (int i0 = t; i0 < kTileRows * 16; i0 += nthr * BATCH) {
    uint4 v[BATCH];
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int i = i0 + u * nthr;
      const int row = i >> 4, ch = i & 15;  // 16 chunks of 8 elements per row
      v[u] = make_uint4(0, 0, 0, 0);
      if (i < kTileRows * 16 && row < sg.nrows) {
        const int r = sg.r0 + row;
        const size_t tok = (size_t)sg.q_tok0 + r / g;
        const size_t head = (size_t)sg.h * g + r % g;
        const size_t e = (tok * P.num_q_heads + head) * kHeadDim + ch * 8;
        if constexpr (!FP8) {
          v[u] = __ldg(reinterpret_cast<const uint4*>(q + e * 2));
        } else {
          uint2 raw = __ldg(reinterpret_cast<const uint2*>(q + e));
          const __nv_fp8x2_storage_t* p2 = reinterpret_cast<const __nv_fp8x2_storage_t*>(&raw);
          uint32_t o[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            __half2_raw hh = __nv_cvt_fp8x2_to_halfraw2(p2[k], __NV_E4M3);
            float2 f = __half22float2(*reinterpret_cast<__half2*>(&hh));
            o[k] = pack_bf16x2(f.x, f.y);
          }
          v[u] = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int i = i0 + u * nthr;
      const int row = i >> 4, ch = i & 15;
      if (i < kTileRows * 16)
        *reinterpret_cast<uint4*>(sQ + (ch >> 3) * 16384 + sw128_offset(row, ch & 7)) = v[u];
    }
  }
}

// One raw FP8 tile (128 rows x 128 bytes, 128-byte swizzle as TMA wrote it) -> one F16 tile in the two-halves
// layout of the K / V rings.  nthr threads (a multiple of 8); eight consecutive threads take one row, so every quarter-warp reads
// one whole 128-byte row (conflict-free).  Element order inside a row is preserved, so the same routine
// serves K (K-major operand) and V (MN-major operand).
__device__ __forceinline__ void widen_chunk_f16(const uint4& v, uint8_t* dst, int row, int c) {
  const uint4 lo = make_uint4(e4m3x2_to_f16x2(v.x), e4m3x2_to_f16x2(v.x >> 16), e4m3x2_to_f16x2(v.y),
                              e4m3x2_to_f16x2(v.y >> 16));
  const uint4 hi = make_uint4(e4m3x2_to_f16x2(v.z), e4m3x2_to_f16x2(v.z >> 16), e4m3x2_to_f16x2(v.w),
                              e4m3x2_to_f16x2(v.w >> 16));
  uint8_t* half = dst + (c >> 2) * 16384;   // d < 64 -> first half
  const int oc = (c & 3) * 2;               // chunk index inside the half (8 f16 per 16 bytes)
  *reinterpret_cast<uint4*>(half + sw128_offset(row, oc)) = lo;
  *reinterpret_cast<uint4*>(half + sw128_offset(row, oc + 1)) = hi;
}
// Loads go in batches of eight ahead of the stores: raw and dst are both shared memory, and a load the compiler
// cannot prove independent of the previous store waits for it (measured: 1260 cycles per tile with 128 threads
// against 885 with the loads hoisted).
// row_off: the tile's first row inside the raw buffer (a TMA box may start a few packed rows before the tile).
__device__ __forceinline__ void widen_tile_f16(const uint8_t* __restrict__ raw, uint8_t* __restrict__ dst, int t,
                                               int nthr, int row_off = 0) {
  for (int i0 = t; i0 < kTileRows * 8; i0 += 8 * nthr) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * nthr;
      if (i < kTileRows * 8) v[u] = *reinterpret_cast<const uint4*>(raw + sw128_offset((i >> 3) + row_off, i & 7));
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * nthr;   // row = i >> 3; c = i & 7: 16-byte chunk = 16 elements d = 16c .. 16c+15
      if (i < kTileRows * 8) widen_chunk_f16(v[u], dst, i >> 3, i & 7);
    }
  }
}

// Raw FP8 query tile -> shared memory with cp.async in the layout widen_tile_f16 reads (128-byte rows, swizzled).
__device__ __forceinline__ void load_q_raw_async(uint8_t* sRaw, const uint8_t* __restrict__ q, const SegInfo& sg,
                                                 const DevParams& P, int t, int nthr) {
  const int g = P.group;
  const uint32_t base = smem_u32(sRaw);
  const uint64_t pol = l2_policy_evict_first();
  for (int i = t; i < kTileRows * 8; i += nthr) {
    const int row = i >> 3, ch = i & 7;
    const uint8_t* src = q;
    uint32_t nbytes = 0;
    if (row < sg.nrows) {
      const int r = sg.r0 + row;
      const size_t tok = (size_t)sg.q_tok0 + r / g;
      const size_t head = (size_t)sg.h * g + r % g;
      src = q + (tok * P.num_q_heads + head) * kHeadDim + ch * 16;
      nbytes = 16;
    }
    cp_async16(base + sw128_offset(row, ch), src, nbytes, pol);
  }
}

// One pooled key (= this thread's TMEM lane) against the 128 query rows of the tile (= TMEM columns):
// m = max_j x_j, sum = sum_j 2^(x_j - m), x_j = s_j * (scale log2 e [* q_scale of row j]).  PARTIAL: only the
// first nrows columns are real query rows.  Releases the accumulator as soon as it is in registers.
template <bool FP8, bool PARTIAL>
__device__ __forceinline__ void score_chunk(uint32_t lane_addr, float cs, const float* sC, int nrows,
                                            uint64_t* acc_empty_bar, float& m_out, float& sum_out) {
  uint32_t xv[128];
#pragma unroll
  for (int k = 0; k < 4; ++k) tmem_ld32(lane_addr + k * 32, reinterpret_cast<uint32_t(&)[32]>(xv[k * 32]));
  tmem_wait_ld();
  tc_fence_before();
  mbar_arrive(acc_empty_bar);
  // x_j = s_j * multiplier, rows past nrows masked to -inf.  BF16: one multiplier for all rows, which commutes
  // with the maximum (it is positive): the maximum is taken over the raw logits and the scaling rides in the
  // fused multiply-add that subtracts it.  FP8: a multiplier per row (q_scale), applied first.
  float x[128];
#pragma unroll
  for (int j = 0; j < 128; j += 2) {
    if constexpr (FP8) {
      const uint64_t mult2 = f2_pack(sC[j], sC[j + 1]);
      f2_unpack(f2_mul(f2_pack(__uint_as_float(xv[j]), __uint_as_float(xv[j + 1])), mult2), x[j], x[j + 1]);
    } else {
      x[j] = __uint_as_float(xv[j]);
      x[j + 1] = __uint_as_float(xv[j + 1]);
    }
    if constexpr (PARTIAL) {
      x[j] = (j < nrows) ? x[j] : -INFINITY;
      x[j + 1] = (j + 1 < nrows) ? x[j + 1] : -INFINITY;
    }
  }
  float m8[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const float* v = &x[c * 16];
    m8[c] = max3(max3(max3(v[0], v[1], v[2]), max3(v[3], v[4], v[5]), max3(v[6], v[7], v[8])),
                 max3(v[9], v[10], v[11]), max3(max3(v[12], v[13], v[14]), v[15], v[15]));
  }
  float m = fmaxf(max3(m8[0], m8[1], m8[2]), max3(max3(m8[3], m8[4], m8[5]), m8[6], m8[7]));
  const float mul = FP8 ? 1.0f : cs;
  m *= mul;
  const uint64_t nm2 = f2_pack(-m, -m), mul2 = f2_pack(mul, mul);
  uint64_t s4[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
  for (int j = 0; j < 128; j += 2) {
    float d0, d1;
    if constexpr (FP8) f2_unpack(f2_add(f2_pack(x[j], x[j + 1]), nm2), d0, d1);
    else f2_unpack(f2_fma(f2_pack(x[j], x[j + 1]), mul2, nm2), d0, d1);
    s4[(j >> 1) & 3] = f2_add(s4[(j >> 1) & 3], f2_pack(ex2(d0), ex2(d1)));
  }
  float t0, t1;
  f2_unpack(f2_add(f2_add(s4[0], s4[1]), f2_add(s4[2], s4[3])), t0, t1);
  m_out = m;
  sum_out = t0 + t1;
}

// BF16 query tile -> shared memory with cp.async: every 16-byte piece of the tile is in flight at once (the
// register-staged variant above keeps only a few loads per thread in flight and was latency-bound at one tile
// per ~12 us).  Same layout and zero fill as load_q_tile_bf16; with `wait` it returns after the copies have landed,
// otherwise the caller closes a cp.async group and waits for it later.
__device__ __forceinline__ void load_q_tile_async(uint8_t* sQ, const uint8_t* __restrict__ q, const SegInfo& sg,
                                                  const DevParams& P, int t, int nthr, bool wait = true) {
  const int g = P.group;
  const uint32_t base = smem_u32(sQ);
  const uint64_t pol = l2_policy_evict_first();   // queries are read once
  for (int i = t; i < kTileRows * 16; i += nthr) {
    const int row = i >> 4, ch = i & 15;
    const uint8_t* src = q;
    uint32_t nbytes = 0;
    if (row < sg.nrows) {
      const int r = sg.r0 + row;
      const size_t tok = (size_t)sg.q_tok0 + r / g;
      const size_t head = (size_t)sg.h * g + r % g;
      src = q + ((tok * P.num_q_heads + head) * kHeadDim + ch * 8) * 2;
      nbytes = 16;
    }
    cp_async16(base + (ch >> 3) * 16384 + sw128_offset(row, ch & 7), src, nbytes, pol);
  }
  if (wait) cp_async_wait_all();
}

template <bool FP8>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_select_kernel(const __grid_constant__ CUtensorMap map_khi, const __grid_constant__ CUtensorMap map_klo,
                    const __grid_constant__ CUtensorMap map_q, const uint8_t* __restrict__ q, const SegInfo* __restrict__ segs, const float* __restrict__ q_scale,
                    DevParams P, int64_t* __restrict__ seg_offset, int32_t* __restrict__ seg_count,
                    int32_t* __restrict__ blk_idx, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int kScoreQBufs = FP8 ? 2 : 3;
  uint8_t* sQ = smem;                                    // kScoreQBufs x 32 KB query tiles (+ raw staging, FP8)
  uint8_t* sQraw = smem + 2 * 32768;                     // FP8: two raw e4m3 boxes of kScoreRawBytes
  uint8_t* sStage = smem + kScoreQSlots * 32768 + (2 * kScoreRawBytes - 32768);   // kScoreStages x 32 KB pieces (kbar_hi or kbar_lo chunk)
  float* sE = reinterpret_cast<float*>(sStage + kScoreStages * 32768);  // per candidate: log2 of its energy
  float* sC = sE + kMaxBlocks;                                          // [kScoreInfoSlots][128] per-row multiplier (FP8); a slot is
                                                                        // rewritten only after every consumer has released its descriptor

  __shared__ SegInfo info[kScoreInfoSlots];
  __shared__ int info_valid[kScoreInfoSlots];
  __shared__ uint64_t info_full[kScoreInfoSlots], info_empty[kScoreInfoSlots], q_full[kScoreQSlots], q_empty[kScoreQSlots];
  __shared__ uint64_t full[kScoreStages], empty[kScoreStages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float red[2][8];
  __shared__ uint64_t e_full[2], sel_done[2];   // [tile & 1] energies of the tile are complete / its list is written
  __shared__ uint64_t raw_full[2];              // FP8, raw boxes by TMA: box k & 1 has landed
  __shared__ uint64_t drain_bar;                // teardown after an abort: every MMA issued by this CTA has completed

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  WaitCtx ctx{status, &abort_flag};
  // When the query tiles come by TMA, one set-up warp is enough and the other (warp 11) takes the selection off
  // the consumers: they only leave the tile's energies (and their maxima) in shared memory and go on with the next
  // tile's chunks; threshold, forced blocks and the ordered compaction of tile t run beside the scoring of tile
  // t+1.  The energy buffer is used in two halves by tile parity; a tile with more than kMaxBlocks / 2 candidates
  // takes both and waits for its neighbours.  In this mode the two warpgroups also share the chunks by a count
  // that runs across tiles, so a tile with an odd number of chunks leaves neither of them short.
  const bool q_by_tma = !FP8 && P.q_tma;   // else warp 10 stages the tile with cp.async (and widens FP8 to F16)

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < kScoreInfoSlots; ++i) {
      mbar_init(&info_full[i], 1);
      mbar_init(&info_empty[i], 2 + 256 + 1);   // producer, issuer, consumers, selection warp
    }
    for (int i = 0; i < kScoreQBufs; ++i) {
      mbar_init(&q_full[i], q_by_tma ? 1 : 32);
      mbar_init(&q_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&e_full[i], 256);
      mbar_init(&sel_done[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 128);
    }
    for (int i = 0; i < kScoreStages; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(&drain_bar, 1);
    mbar_init(&raw_full[0], 1);
    mbar_init(&raw_full[1], 1);
    fence_barrier_init();
  }
  if (warp == 9) {
    tmem_alloc(&tmem_base_s, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;

  if (warp == 10) {
    // ---------------- set-up (warp 10): segment k of this CTA is number blockIdx.x + k * gridDim.x in heaviest-first order
    // (a static round-robin: no atomic on the critical path).  The loop is software-pipelined: the copies of
    // tile k+1 are issued before the copies of tile k are waited for, so two query tiles are in flight.
    const int t64 = lane;
    auto seg_of = [&](int k) { return P.nseg - 1 - ((int)blockIdx.x + k * (int)gridDim.x); };
    auto issue = [&](int k) -> bool {   // publishes tile k's descriptor and starts its query copies
      const int slot = k % kScoreInfoSlots, qb = k % kScoreQBufs;
      if (k >= kScoreInfoSlots) mbar_wait(&info_empty[slot], ((k / kScoreInfoSlots) - 1) & 1, ctx, 111);
      const int sgi = seg_of(k);
      // after a wait has run out somewhere in this CTA no further tile is started
      if (t64 == 0) info_valid[slot] = sgi >= 0 && !*ctx.abort;
      __syncwarp();
      const bool valid = info_valid[slot] != 0;
      if (t64 == 0 && valid) info[slot] = segs[sgi];
      __syncwarp();
      if (t64 == 0) {
        __threadfence_block();
        mbar_arrive(&info_full[slot]);
      }
      if (!valid) return false;
      const SegInfo sg = info[slot];
      if constexpr (FP8) {
        // raw e4m3 rows into the staging slot (its previous content was widened two tiles ago by these threads).
        // Under PackGQA (Eq. 13) the tile's rows are consecutive (token, head) pairs of the KV head's group: the box
        // [128 bytes, g heads, q_box_tok tokens] that starts at the tile's first token holds them all, in packed
        // order, the tile's first row sg.r0 % g rows into it.  One TMA copy instead of 1024 address computations.
        if (P.q_raw_tma) {
          if (t64 == 0) {
            mbar_arrive_expect_tx(&raw_full[k & 1], (uint32_t)(P.group * P.q_box_tok * 128));
            tma_load_3d_hint(sQraw + (k & 1) * kScoreRawBytes, &map_q, &raw_full[k & 1], 0, sg.h * P.group,
                             sg.q_tok0 + sg.r0 / P.group, l2_policy_evict_first());
          }
        } else {
          load_q_raw_async(sQraw + (k & 1) * kScoreRawBytes, q, sg, P, t64, 32);
        }
      } else {
        // the Q buffer is free once every MMA of the tile that used it kScoreQBufs tiles ago has completed
        if (k >= kScoreQBufs) mbar_wait(&q_empty[qb], ((k / kScoreQBufs) - 1) & 1, ctx, 112);
        load_q_tile_async(sQ + qb * 32768, q, sg, P, t64, 32, false);
      }
      cp_async_commit();
      return true;
    };
    if (q_by_tma) {
      // Under PackGQA (Eq. 13) packed row r is (token r / g, head r % g): when g divides 128 a tile is 128 / g
      // consecutive tokens x g consecutive heads, i.e. one TMA box per 64-element half, landing in exactly the
      // swizzled layout the MMA reads.  No thread touches the data; the tile's barrier carries the byte count.
      // Rows past the end of a short last tile read the tokens that follow (or zeros past the tensor's end) and are
      // never used.  Three tiles in flight.
      const uint64_t pol = l2_policy_evict_first();
      for (int k = 0;; ++k) {
        const int slot = k % kScoreInfoSlots, qb = k % kScoreQBufs;
        if (k >= kScoreInfoSlots) mbar_wait(&info_empty[slot], ((k / kScoreInfoSlots) - 1) & 1, ctx, 111);
        const int sgi = seg_of(k);
        bool valid = sgi >= 0 && !*ctx.abort;   // after a wait has run out no further tile is started
        valid = __shfl_sync(0xffffffffu, valid, 0);
        if (t64 == 0) {
          info_valid[slot] = valid;
          if (valid) info[slot] = segs[sgi];
          __threadfence_block();
          mbar_arrive(&info_full[slot]);
        }
        __syncwarp();
        if (!valid) break;
        if (k >= kScoreQBufs) mbar_wait(&q_empty[qb], ((k / kScoreQBufs) - 1) & 1, ctx, 112);
        if (t64 == 0) {
          const SegInfo& sg = info[slot];
          uint8_t* dst = sQ + qb * 32768;
          mbar_arrive_expect_tx(&q_full[qb], 32768);
          tma_load_3d_hint(dst, &map_q, &q_full[qb], 0, sg.h * P.group, sg.q_tok0 + sg.r0 / P.group, pol);
          tma_load_3d_hint(dst + 16384, &map_q, &q_full[qb], 64, sg.h * P.group, sg.q_tok0 + sg.r0 / P.group, pol);
        }
        __syncwarp();
      }
    } else {
#ifdef FP2_PROFILE
    long long sp[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long sa = clock64(), sb;
    const long long st0 = sa;
#define STP(k) (sb = clock64(), sp[k] += sb - sa, sa = sb)
#else
#define STP(k)
#endif
    bool have = issue(0);
    int k = 0;
    for (; have; ++k) {
      STP(4);
      const bool next = issue(k + 1);
      STP(0);
      if (next) cp_async_wait_group<1>(); else cp_async_wait_group<0>();
      STP(1);
      const int qb = k % kScoreQBufs;
      if constexpr (FP8) {
        const SegInfo& sgw = info[k % kScoreInfoSlots];
        if (P.q_raw_tma) mbar_wait(&raw_full[k & 1], (k >> 1) & 1, ctx, 114);
        __syncwarp();   // every thread's copies of tile k have landed
        if (k >= kScoreQBufs) mbar_wait(&q_empty[qb], ((k / kScoreQBufs) - 1) & 1, ctx, 113);
        STP(2);
        widen_tile_f16(sQraw + (k & 1) * kScoreRawBytes, sQ + qb * 32768, t64, 32, P.q_raw_tma ? sgw.r0 % P.group : 0);
        STP(3);
        const SegInfo& sgk = info[k % kScoreInfoSlots];
        for (int j = t64; j < kTileRows; j += 32)
          sC[(k % kScoreInfoSlots) * 128 + j] = P.scale_log2 * q_scale[sgk.h * P.group + (sgk.r0 + j) % P.group];
      }
      fence_proxy_async();
      mbar_arrive(&q_full[qb]);
      have = next;
    }
#ifdef FP2_PROFILE
    if (g_score_prof && t64 == 0) {
      sp[5] = k;
      sp[7] = clock64() - st0;
      for (int i = 0; i < 8; ++i) g_score_prof[((size_t)gridDim.x * 2 + blockIdx.x) * 8 + i] = sp[i];
    }
#endif
    }
  } else if (warp == 11) {
    // ---------------- selection warp: threshold, forced blocks, ordered compaction of tile `it` ----------------
    for (int it = 0;; ++it) {
      const int slot = it % kScoreInfoSlots, eb = it & 1;
      mbar_wait(&info_full[slot], (it / kScoreInfoSlots) & 1, ctx, 151);
      if (!info_valid[slot]) break;
      const SegInfo sg = info[slot];
      const int ncand = sg.J_hi + 1;
      const float* e = sE + (ncand > kMaxBlocks / 2 ? 0 : eb * (kMaxBlocks / 2));
      mbar_wait(&e_full[eb], (it >> 1) & 1, ctx, 152);
      float maxE = red[eb][0];
#pragma unroll
      for (int i = 1; i < 8; ++i) maxE = fmaxf(maxE, red[eb][i]);
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
        mbar_arrive(&sel_done[eb]);
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else if (warp == 8) {
    // ---------------- producer: kbar pieces (hi, lo of every 128-block chunk) via TMA ----------------
    if (lane == 0) {
      tma_prefetch_desc(&map_khi);
      tma_prefetch_desc(&map_klo);
      const uint64_t keep = l2_policy_evict_last();
      uint32_t pc = 0;
      for (int it = 0;; ++it) {
        const int slot = it % kScoreInfoSlots;
        mbar_wait(&info_full[slot], (it / kScoreInfoSlots) & 1, ctx, 121);
        if (!info_valid[slot]) break;
        const int h = info[slot].h, blk_off = info[slot].blk_off;
        const int nchunks = (info[slot].J_hi + 128) >> 7;
        for (int c = 0; c < nchunks; ++c) {
#pragma unroll
          for (int part = 0; part < 2; ++part, ++pc) {
            const int s = pc % kScoreStages;
            if (pc >= kScoreStages) mbar_wait(&empty[s], ((pc / kScoreStages) - 1) & 1, ctx, 122);
            uint8_t* dst = sStage + s * 32768;
            mbar_arrive_expect_tx(&full[s], 32768);
            const CUtensorMap* mp = part ? &map_klo : &map_khi;
            tma_load_3d_hint(dst, mp, &full[s], 0, h, blk_off + c * 128, keep);
            tma_load_3d_hint(dst + 16384, mp, &full[s], 64, h, blk_off + c * 128, keep);
          }
        }
        mbar_arrive(&info_empty[slot]);
      }
    }
  } else if (warp == 9) {
    // ---------------- UMMA issuer: acc[c & 1] = kbar_hi Q^T + kbar_lo Q^T ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = FP8 ? make_idesc(128, 128, 0, 0, 0, 0) : make_idesc(128, 128, 1, 1, 0, 0);
      uint32_t pc = 0, ac0 = 0, ac1 = 0, gc0 = 0;   // gc0: chunks of all earlier tiles
      for (int it = 0;; ++it) {
        const int slot = it % kScoreInfoSlots, qb = it % kScoreQBufs;
        mbar_wait(&info_full[slot], (it / kScoreInfoSlots) & 1, ctx, 131);
        if (!info_valid[slot]) break;
        const int nchunks = (info[slot].J_hi + 128) >> 7;
        mbar_wait(&q_full[qb], (it / kScoreQBufs) & 1, ctx, 132);
        const uint32_t q_addr = smem_u32(sQ + qb * 32768);
        for (int c = 0; c < nchunks; ++c) {
          const int a = (gc0 + c) & 1;
          uint32_t& ac = a ? ac1 : ac0;
          if (ac >= 1) mbar_wait(&acc_empty[a], (ac - 1) & 1, ctx, 133);
          ++ac;
#pragma unroll
          for (int part = 0; part < 2; ++part, ++pc) {
            const int s = pc % kScoreStages;
            mbar_wait(&full[s], (pc / kScoreStages) & 1, ctx, 134);
            tc_fence_after();
            const uint32_t a_addr = smem_u32(sStage + s * 32768);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
              const uint64_t ad = make_smem_desc_sw128(a_addr + off, 16, 1024);
              const uint64_t bd = make_smem_desc_sw128(q_addr + off, 16, 1024);
              umma_f16_ss(tmem + a * 128, ad, bd, idesc, (part | ks) != 0);
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
    // ---------------- consumers: per pooled key, max and exp-sum over the tile's rows; then selection ----------------
    const int wg = warp >> 2;
    const int key = (warp & 3) * 32 + lane;  // TMEM lane = pooled key within the chunk
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + wg * 128;
    const float cs = P.scale_log2;
    uint32_t uc = 0;  // uses of this warpgroup's accumulator
    uint32_t gc0 = 0;  // chunks of all earlier tiles
    bool prev_big = false;
#ifdef FP2_PROFILE
    long long pf[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const long long pf_t0 = clock64();
    long long pf_a = pf_t0, pf_b;
#define SPF(k) (pf_b = clock64(), pf[k] += pf_b - pf_a, pf_a = pf_b)
#else
#define SPF(k)
#endif
    for (int it = 0;; ++it) {
      const int slot = it % kScoreInfoSlots;
      SPF(3);
      mbar_wait(&info_full[slot], (it / kScoreInfoSlots) & 1, ctx, 141);
      SPF(0);
#ifdef FP2_PROFILE
      if (!info_valid[slot] && g_score_prof && lane == 0 && (warp & 3) == 0) {
        pf[7] = clock64() - pf_t0;
        for (int i = 0; i < 8; ++i) g_score_prof[((size_t)blockIdx.x * 2 + wg) * 8 + i] = pf[i];
      }
#endif
      if (!info_valid[slot]) break;
      const SegInfo sg = info[slot];
      const int ncand = sg.J_hi + 1;
      const int nchunks = (ncand + 127) >> 7;
      // per candidate: log2 of its energy, e_J = m_J + log2(S_J)  (Eq. 1-2 / Eq. 20 in the log domain: the
      // common factor 2^-M of Eq. 20 cancels in the comparison with alpha * max)
      float lmax = -INFINITY;
      const int eb = it & 1;
      const bool big = ncand > kMaxBlocks / 2;
      float* e_out = sE + (!big ? eb * (kMaxBlocks / 2) : 0);
      // the half of the energy buffer this tile writes must have been read by the selection of tile it-2, and a
      // tile that takes (or follows one that took) the whole buffer also waits for tile it-1
      if (it >= 2) mbar_wait(&sel_done[eb], ((it >> 1) - 1) & 1, ctx, 143);
      if (it >= 1 && (big || prev_big)) mbar_wait(&sel_done[eb ^ 1], ((it - 1) >> 1) & 1, ctx, 144);
      prev_big = big;
      for (int c = (int)((gc0 ^ (uint32_t)wg) & 1u); c < nchunks; c += 2, ++uc) {
        SPF(3);
        mbar_wait(&acc_full[wg], uc & 1, ctx, 142);
        SPF(1);
#ifdef FP2_PROFILE
        pf[5] += 1;
#endif
        tc_fence_after();
        float m, sum;
        if (sg.nrows == kTileRows) score_chunk<FP8, false>(lane_addr, cs, sC + slot * 128, kTileRows, &acc_empty[wg], m, sum);
        else score_chunk<FP8, true>(lane_addr, cs, sC + slot * 128, sg.nrows, &acc_empty[wg], m, sum);
        const int J = c * 128 + key;
        if (J < ncand) {
          const float e = m + log2f(sum);
          e_out[J] = e;
          lmax = fmaxf(lmax, e);
        }
        SPF(2);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lmax = fmaxf(lmax, __shfl_xor_sync(0xffffffffu, lmax, o));
      // hand the tile to the selection warp and go on
      if (lane == 0) red[eb][warp] = lmax;
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
  if (warp == 9) tmem_dealloc(tmem, 256);
}

}  // namespace fp2
