// Count-balanced KV splitting (Eq. 18; Sec. 3.3 "Sparsity-Aware Load Balancing") for launches with fewer work
// units than workers: a segment's iteration sequence -- its list backwards (Eq. 17), then its correction chunks
// -- is cut into U contiguous parts of ceil(n / U) iterations, every part becomes a work unit of its own that
// leaves an unnormalised partial (O_u, m_u, l_u), and a second kernel merges the parts of a segment by their
// log-sum-exp weights.  A correction chunk is one iteration, so it belongs to exactly one part.
//
// The plan is made on the device (the lists are): one CTA reads the work order (KV-head-major, heaviest first),
// estimates every segment's iteration count n = listed blocks + chunks that may be needed, picks
//   L = max(requested or kMinPartLen, ceil(sum n / workers)),   U = min(kMaxSplits, max(1, round(n / L))),
// (one round of parts of about the mean load per worker; a part never much shorter than L, so that it outweighs
// its share of the merge and its own start-up: set-up, Q tile, first K/V tiles), and writes the units in the
// same order, the parts of a segment next to each other.  sum round(n / L) is at most nseg / 2 + workers, within
// the nseg + 2 workers the unit arrays and the partial buffers are sized for when the plan is created.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace fp2 {

constexpr int kMaxSplits = 16;
constexpr int kMinPartLen = 12;     // iterations per part below which splitting costs more than it gains

// unit_split word: part index u (bits 0..7), parts U (bits 8..15), first partial slot of the segment (bits 16..31)
__host__ __device__ inline int32_t pack_split(int u, int U, int slot) { return u | (U << 8) | (slot << 16); }

__global__ void __launch_bounds__(1024, 1)
split_plan_kernel(const SegInfo* __restrict__ segs, const int32_t* __restrict__ order,
                  const int32_t* __restrict__ seg_count, int nseg, int use_correction, int workers, int target,
                  int32_t* __restrict__ unit_seg, int32_t* __restrict__ unit_split, int32_t* __restrict__ seg_split,
                  int32_t* __restrict__ split_list, int32_t* __restrict__ n_units, int32_t* __restrict__ n_split) {
  __shared__ int32_t part_a[1024], part_b[1024], part_c[1024];
  __shared__ int s_total;
  const int t = threadIdx.x;
  const int per = (nseg + 1023) / 1024;
  const int beg = min(t * per, nseg), end = min(beg + per, nseg);
  auto est = [&](int w) {   // iterations of the segment at position w of the work order (chunks: upper bound)
    const SegInfo& sg = segs[order[w]];
    int T = seg_count ? seg_count[sg.seg] : sg.J_hi + 1;
    T = max(0, min(T, sg.J_hi + 1));
    const int chunks = (seg_count && use_correction) ? (sg.J_lo + 127) >> 7 : 0;
    return T + chunks;
  };
  if (t == 0) s_total = 0;
  __syncthreads();
  int mine = 0;
  for (int w = beg; w < end; ++w) mine += est(w);
  atomicAdd(&s_total, mine);
  __syncthreads();
  const int total = s_total;
  const int floor_len = (total + workers - 1) / workers;
  const int L = max(max(target > 0 ? target : kMinPartLen, floor_len), 1);
  // units and partial slots before this thread's segments
  int units = 0, slots = 0, nsplit = 0;
  for (int w = beg; w < end; ++w) {
    const int U = min(kMaxSplits, max(1, (est(w) + L / 2) / L));
    units += U;
    slots += U > 1 ? U : 0;
    nsplit += U > 1;
  }
  part_a[t] = units;
  part_b[t] = slots;
  part_c[t] = nsplit;
  __syncthreads();
  for (int d = 1; d < 1024; d <<= 1) {
    const int a = t >= d ? part_a[t - d] : 0, b = t >= d ? part_b[t - d] : 0, c = t >= d ? part_c[t - d] : 0;
    __syncthreads();
    part_a[t] += a;
    part_b[t] += b;
    part_c[t] += c;
    __syncthreads();
  }
  int uoff = part_a[t] - units, soff = part_b[t] - slots, loff = part_c[t] - nsplit;
  for (int w = beg; w < end; ++w) {
    const int seg = order[w];
    const int U = min(kMaxSplits, max(1, (est(w) + L / 2) / L));
    const int slot = U > 1 ? soff : 0;
    for (int u = 0; u < U; ++u) {
      unit_seg[uoff + u] = seg;
      unit_split[uoff + u] = pack_split(u, U, slot);
    }
    seg_split[seg] = U > 1 ? pack_split(0, U, slot) : 0;
    if (U > 1) split_list[loff++] = seg;
    uoff += U;
    soff += U > 1 ? U : 0;
  }
  if (t == 1023) {
    *n_units = part_a[1023];
    *n_split = part_c[1023];
  }
}

// Merge of the parts of the split segments.  CTAs loop over (split segment, group of kMergeRows rows).  Threads
// 0 .. kMergeRows-1 first compute the rows' weights 2^(m_u - m) and 1 / sum; then thread = output column, all
// rows of the group loaded before the first use (every partial row is one 512-byte line).
constexpr int kMergeRows = 8;

__global__ void __launch_bounds__(128)
split_combine_kernel(const SegInfo* __restrict__ segs, const int32_t* __restrict__ seg_split,
                     const int32_t* __restrict__ split_list, const int32_t* __restrict__ n_split,
                     const float* __restrict__ part_o, const float2* __restrict__ part_ml,
                     const float* __restrict__ v_scale, DevParams P, __nv_bfloat16* __restrict__ out,
                     float* __restrict__ lse) {
  constexpr int kGroups = 128 / kMergeRows;
  const int n_items = *n_split * kGroups;
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
  const int seg = split_list[item / kGroups];
  const int32_t word = seg_split[seg];
  const int U = (word >> 8) & 0xff, slot = (word >> 16) & 0xffff;
  const SegInfo sg = segs[seg];
  const int row0 = (item % kGroups) * kMergeRows;
  if (row0 >= sg.nrows) continue;
  __syncthreads();   // the shared arrays of the previous item are no longer read
  __shared__ float w_s[kMergeRows][kMaxSplits];
  __shared__ float inv_s[kMergeRows];
  const int t = threadIdx.x, g = P.group;
  if (t < kMergeRows) {
    const int row = row0 + t;
    float mv[kMaxSplits], lv[kMaxSplits];
    float m = -INFINITY;
    for (int u = 0; u < U; ++u) {
      const float2 ml = part_ml[(size_t)(slot + u) * 128 + row];
      mv[u] = ml.x;
      lv[u] = ml.y;
      m = fmaxf(m, ml.x);
    }
    float L = 0.f;
    for (int u = 0; u < U; ++u) {
      const float w = (mv[u] == -INFINITY) ? 0.f : exp2f(mv[u] - m);   // an empty part has m = -inf, l = 0
      w_s[t][u] = w;
      L += w * lv[u];
    }
    const float out_scale = v_scale ? v_scale[sg.h] : 1.0f;
    inv_s[t] = L > 0.f ? out_scale / L : 0.f;
    if (row < sg.nrows && lse != nullptr) {
      const int r = sg.r0 + row;
      const size_t tok = (size_t)sg.q_tok0 + r / g;
      const int head = sg.h * g + r % g;
      lse[(size_t)head * P.total_q + tok] = (m + log2f(L)) * 0.6931471805599453f;
    }
  }
  __syncthreads();
  const int c = t;
  float acc[kMergeRows];
#pragma unroll
  for (int i = 0; i < kMergeRows; ++i) acc[i] = 0.f;
  for (int u = 0; u < U; ++u) {
    float v[kMergeRows];
#pragma unroll
    for (int i = 0; i < kMergeRows; ++i)
      v[i] = (row0 + i < sg.nrows && w_s[i][u] != 0.f) ? part_o[((size_t)(slot + u) * 128 + row0 + i) * 128 + c] : 0.f;
#pragma unroll
    for (int i = 0; i < kMergeRows; ++i) acc[i] = fmaf(w_s[i][u], v[i], acc[i]);
  }
#pragma unroll
  for (int i = 0; i < kMergeRows; ++i) {
    const int row = row0 + i;
    if (row >= sg.nrows) break;
    const int r = sg.r0 + row;
    const size_t tok = (size_t)sg.q_tok0 + r / g;
    const int head = sg.h * g + r % g;
    out[(tok * P.num_q_heads + head) * kHeadDim + c] = __float2bfloat16_rn(acc[i] * inv_s[i]);
  }
  }
}

}  // namespace fp2
