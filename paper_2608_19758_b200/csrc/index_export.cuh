// Index export (Algorithm 1 line 5; Sec. 3.3 "Index-Driven Sparse Traversal", Eq. 17; Sec. 3.4 "Serving
// Integration"): the padded block lists of the selector as a compact CSR (cu, idx) of physical tiles of
// tile_tokens tokens, per segment in segment order (that is: per KV head under PackGQA), and the page-level
// table read out of a token-level slot map by striding.
//
// A logical block J of 128 tokens becomes the tiles J tpb .. J tpb + tpb - 1 (tpb = 128 / tile_tokens) that hold
// at least one real token; only the last block of a sequence can be short, and a list is ascending, so only a
// segment's last entry can produce fewer than tpb tiles -- entry k of a segment always starts at cu + k tpb.
// Integer work throughout; launch-latency- and HBM-bound (reads the lists once, writes tpb entries per block).
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace fp2 {

// tiles of block J that hold a real token of a sequence of Lk tokens
__device__ __forceinline__ int tiles_in_block(int J, int Lk, int tile_tokens) {
  const int ntok = min(kBlock, Lk - J * kBlock);
  return ntok <= 0 ? 0 : (ntok + tile_tokens - 1) / tile_tokens;
}

// count and list entries as the attention kernel reads them: out-of-range values are clamped (and flagged)
__device__ __forceinline__ int clamped_count(const SegInfo& sg, const int32_t* seg_count, int* status) {
  int T = seg_count[sg.seg];
  if (T < 0 || T > sg.J_hi + 1) {
    atomicOr(status + ST_BAD_LIST, 1);
    T = max(0, min(T, sg.J_hi + 1));
  }
  return T;
}

// cu[g + 1] = number of tiles of segment g; cu[0] = 0.  One thread per segment.
__global__ void csr_count_kernel(const SegInfo* __restrict__ segs, const int32_t* __restrict__ seg_count,
                                 const int32_t* __restrict__ blk_idx, int nseg, int tile_tokens,
                                 int32_t* __restrict__ cu, int* __restrict__ status) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g == 0) cu[0] = 0;
  if (g >= nseg) return;
  const SegInfo sg = segs[g];
  const int T = clamped_count(sg, seg_count, status);
  const int tpb = kBlock / tile_tokens;
  int n = 0;
  if (T > 0) {
    const int J = max(0, min(blk_idx[sg.off + T - 1], sg.J_hi));
    n = (T - 1) * tpb + tiles_in_block(J, sg.Lk, tile_tokens);
  }
  cu[g + 1] = n;
}

// single CTA of 1024 threads: inclusive scan of cu[1 .. n] in place (cu[g + 1] = tiles of segments 0..g).
// Tiles of kScanTile = 1024 x 8 elements: every thread loads its 8 consecutive values at once, scans them in
// registers, the CTA scans the 1024 thread totals through shared memory, and a running carry links the tiles.
constexpr int kScanPerThread = 8;
__global__ void __launch_bounds__(1024, 1) csr_scan_kernel(int32_t* __restrict__ cu, int n) {
  __shared__ int32_t warp_tot[32];
  __shared__ int32_t s_carry;
  int32_t* v = cu + 1;
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  if (t == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < n; base += 1024 * kScanPerThread) {
    const int i0 = base + t * kScanPerThread;
    int32_t x[kScanPerThread];
#pragma unroll
    for (int j = 0; j < kScanPerThread; ++j) x[j] = i0 + j < n ? v[i0 + j] : 0;
#pragma unroll
    for (int j = 1; j < kScanPerThread; ++j) x[j] += x[j - 1];
    // exclusive prefix of the thread totals: warp scan, then the 32 warp totals
    int32_t incl = x[kScanPerThread - 1];
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    if (lane == 31) warp_tot[w] = incl;
    __syncthreads();
    if (w == 0) {
      int32_t wt = warp_tot[lane];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, wt, d);
        if (lane >= d) wt += y;
      }
      warp_tot[lane] = wt;   // inclusive over warps
    }
    __syncthreads();
    const int32_t carry = s_carry;
    const int32_t before = carry + (w > 0 ? warp_tot[w - 1] : 0) + incl - x[kScanPerThread - 1];
#pragma unroll
    for (int j = 0; j < kScanPerThread; ++j)
      if (i0 + j < n) v[i0 + j] = x[j] + before;
    __syncthreads();
    if (t == 1023) s_carry = carry + warp_tot[31];
    __syncthreads();
  }
}

// one warp per segment: entry k of the list -> its tiles at cu[g] + k tpb
__global__ void csr_fill_kernel(const SegInfo* __restrict__ segs, const int32_t* __restrict__ seg_count,
                                const int32_t* __restrict__ blk_idx, int nseg, int tile_tokens,
                                const int32_t* __restrict__ cu, int32_t* __restrict__ idx, int* __restrict__ status) {
  const int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (g >= nseg) return;
  const SegInfo sg = segs[g];
  int T = seg_count[sg.seg];
  T = max(0, min(T, sg.J_hi + 1));   // flagged by the counting kernel
  const int tpb = kBlock / tile_tokens;
  const int32_t* list = blk_idx + sg.off;
  int32_t* out = idx + cu[g];
  bool bad = false;
  for (int k = lane; k < T; k += 32) {
    int J = list[k];
    if (J < 0 || J > sg.J_hi || (k > 0 && list[k - 1] >= J)) bad = true;
    J = max(0, min(J, sg.J_hi));
    const int n = k + 1 < T ? tpb : tiles_in_block(J, sg.Lk, tile_tokens);
    for (int j = 0; j < n; ++j) out[k * tpb + j] = J * tpb + j;
  }
  if (bad) atomicOr(status + ST_BAD_LIST, 1);
}

// page_table[b][k] = token_to_slot[b][k p] / p for the pages that hold a token, -1 beyond (Sec. 3.4).  A sampled
// slot that is not the first of a page is flagged in the status block.
__global__ void page_table_from_token_map_kernel(const int32_t* __restrict__ token_to_slot, int max_tokens,
                                                 const int32_t* __restrict__ seqlens_k, int ns, int p, int max_pages,
                                                 int32_t* __restrict__ page_table, int* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= ns * max_pages) return;
  const int b = i / max_pages, k = i % max_pages;
  int32_t v = -1;
  if ((int64_t)k * p < seqlens_k[b] && (int64_t)k * p < max_tokens) {
    const int32_t slot = token_to_slot[(size_t)b * max_tokens + (size_t)k * p];
    if (slot < 0 || slot % p != 0) atomicOr(status + ST_BAD_LIST, 4);
    v = slot < 0 ? -1 : slot / p;
  }
  page_table[i] = v;
}

}  // namespace fp2
