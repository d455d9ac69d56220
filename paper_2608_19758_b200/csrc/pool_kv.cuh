// Block-mean pooling (Eq. 5; Algorithm 1 line 2): kbar_J, vbar_J = mean over the real tokens of KV block J,
// read through the page table (Eq. 22).  HBM-bound: K and V are read exactly once with 16-byte loads,
// 256-byte (BF16) or 128-byte (FP8) contiguous per token row, fp32 accumulation.
//
// Outputs, all BF16 [nblk_tot, Hkv, 128]:
//   kbar_hi = bf16(mean k), kbar_lo = bf16(mean k - kbar_hi)   (hi + lo carries ~16 mantissa bits for the scorer)
//   vbar    = bf16(mean v)
// kbar_hi and vbar double as the operands of the correction chunks in the attention kernel.
// FP8 inputs: the three arrays hold F16 instead of BF16: kbar_hi / kbar_lo = F16 pair of the de-scaled mean (mean
// of raw values x k_scale) for the scorer, vbar = f16(mean of RAW v) -- v_scale is applied to the attention
// output.  Two more arrays, e4m3 [nblk_tot, Hkv, 128] each, hold the mean of the RAW keys as a hi + lo pair
// (hi = e4m3(mean), lo = e4m3(mean - hi): ~8 mantissa bits together) for the correction chunks of the attention
// kernel, whose S = Q K^T runs on raw e4m3 operands.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include "common.cuh"
#include "ptx.cuh"

namespace fp2 {

template <bool FP8>
__device__ __forceinline__ void accum16(const uint4& v, float* acc) {
  if constexpr (!FP8) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(p[i]);
      acc[2 * i] += f.x;
      acc[2 * i + 1] += f.y;
    }
  } else {
    const __nv_fp8x2_storage_t* p = reinterpret_cast<const __nv_fp8x2_storage_t*>(&v);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(p[i], __NV_E4M3);
      float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
      acc[2 * i] += f.x;
      acc[2 * i + 1] += f.y;
    }
  }
}

// One pooled mean -> the operand formats the scorer and the correction chunks read (see the head of the file).
template <bool FP8>
__device__ __forceinline__ void write_pooled(int which, float mean, size_t o, int h, const float* __restrict__ k_scale,
                                             __nv_bfloat16* __restrict__ kbar_hi, __nv_bfloat16* __restrict__ kbar_lo,
                                             __nv_bfloat16* __restrict__ vbar, uint8_t* __restrict__ kbar8_hi,
                                             uint8_t* __restrict__ kbar8_lo) {
  if constexpr (FP8) {
    if (which == 0) {
      // the attention kernel multiplies raw e4m3 queries with this pair in one FP8 MMA group each
      const __nv_fp8_storage_t hi8 = __nv_cvt_float_to_fp8(mean, __NV_SATFINITE, __NV_E4M3);
      const float hi8f = __half2float(__half(__nv_cvt_fp8_to_halfraw(hi8, __NV_E4M3)));
      kbar8_hi[o] = hi8;
      kbar8_lo[o] = __nv_cvt_float_to_fp8(mean - hi8f, __NV_SATFINITE, __NV_E4M3);
      mean *= k_scale[h];
    }
    const __half hi16 = __float2half_rn(mean);
    if (which == 0) {
      reinterpret_cast<__half*>(kbar_hi)[o] = hi16;
      reinterpret_cast<__half*>(kbar_lo)[o] = __float2half_rn(mean - __half2float(hi16));
    } else {
      reinterpret_cast<__half*>(vbar)[o] = hi16;
    }
  } else {
    const __nv_bfloat16 hi16 = __float2bfloat16_rn(mean);
    if (which == 0) {
      kbar_hi[o] = hi16;
      kbar_lo[o] = __float2bfloat16_rn(mean - __bfloat162float(hi16));
    } else {
      vbar[o] = hi16;
    }
  }
}

// 1-D grid of nblk_tot * Hkv * 2 CTAs: (K or V) fastest, then the KV head, then the block, so CTAs that run
// together read neighbouring pieces of the same token rows.  One CTA pools one operand of one (block, head):
// 128 token rows of 256 B (BF16) / 128 B (FP8).  256 threads, every load of a thread issued before the first
// use; small enough in registers for four CTAs per SM, which is what hides the page-table -> data dependency.
template <bool FP8>
__global__ void __launch_bounds__(256, 4) pool_kv_kernel(const uint8_t* __restrict__ k_cache,
                                                         const uint8_t* __restrict__ v_cache,
                                                         const int32_t* __restrict__ page_table,
                                                         const int32_t* __restrict__ plan_lk,  // [ns], the plan's copy
                                                         const int32_t* __restrict__ blk_off,  // [ns+1]
                                                         const float* __restrict__ k_scale,
                                                         const float* __restrict__ v_scale, DevParams P,
                                                         __nv_bfloat16* __restrict__ kbar_hi,
                                                         __nv_bfloat16* __restrict__ kbar_lo,
                                                         __nv_bfloat16* __restrict__ vbar,
                                                         uint8_t* __restrict__ kbar8_hi,
                                                         uint8_t* __restrict__ kbar8_lo,
                                                         const int32_t* __restrict__ carry,
                                                         int* __restrict__ status) {
  constexpr int ROW_BYTES = FP8 ? 128 : 256;
  constexpr int CHUNKS = ROW_BYTES / 16;       // 16-byte chunks per token row
  constexpr int EPC = FP8 ? 16 : 8;            // elements per chunk
  constexpr int ROWS_PER_PASS = 256 / CHUNKS;  // 16 (bf16) or 32 (fp8)
  constexpr int PASSES = kBlock / ROWS_PER_PASS;

  __shared__ float red[ROWS_PER_PASS][kHeadDim + 4];

  const int which = blockIdx.x & 1;            // 0: K, 1: V
  const int bh = blockIdx.x >> 1;
  const int gblk = bh / P.num_kv_heads, h = bh % P.num_kv_heads;
  // sequence of this pooled block: binary search in blk_off
  int lo = 0, hi = P.num_seqs;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (blk_off[mid] <= gblk) lo = mid; else hi = mid;
  }
  const int b = lo, J = gblk - blk_off[b];
  // chunked prefill: the means of the first carry[3 b + 2] blocks of this sequence were carried over from the
  // previous chunk's workspace (pool_carry_kernel) and are not computed again
  if (carry != nullptr && J < carry[3 * b + 2]) return;
  // The length comes from the plan's table (validated on the host when the plan was made), like every other piece
  // of geometry: a block of the pooled arrays always has between 1 and 128 real tokens.
  const int Lk = plan_lk[b];
  const int ntok = min(kBlock, Lk - J * kBlock);
  const int chunk = threadIdx.x % CHUNKS, rg = threadIdx.x / CHUNKS;
  const int32_t* pt = page_table + (size_t)b * P.max_pages_per_seq;
  const size_t row_stride = (size_t)P.num_kv_heads * ROW_BYTES;
  const uint8_t* cache = which ? v_cache : k_cache;

  uint4 dv[PASSES];
#pragma unroll
  for (int ps = 0; ps < PASSES; ++ps) {
    const int tl = ps * ROWS_PER_PASS + rg;
    dv[ps] = make_uint4(0, 0, 0, 0);   // zero bit patterns add 0 in both encodings
    if (tl < ntok) {
      const int j = J * kBlock + tl;
      const int pid = pt[j / P.page_size];
      if (pid < 0 || pid >= P.num_pages) {
        // a page id outside the pool: nothing is read for this token (it counts as zeros) and the call is flagged
        atomicOr(status + ST_BAD_LIST, 2);
      } else {
        const size_t slot = (size_t)pid * P.page_size + (j % P.page_size);
        dv[ps] = __ldg(reinterpret_cast<const uint4*>(cache + slot * row_stride + (size_t)h * ROW_BYTES + chunk * 16));
      }
    }
  }
  float acc[EPC];
#pragma unroll
  for (int i = 0; i < EPC; ++i) acc[i] = 0.f;
#pragma unroll
  for (int ps = 0; ps < PASSES; ++ps) accum16<FP8>(dv[ps], acc);
#pragma unroll
  for (int i = 0; i < EPC; ++i) red[rg][chunk * EPC + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < kHeadDim) {
    const int c = threadIdx.x;
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < ROWS_PER_PASS; ++r) s += red[r][c];
    const size_t o = ((size_t)gblk * P.num_kv_heads + h) * kHeadDim + c;
    write_pooled<FP8>(which, s / (float)ntok, o, h, k_scale, kbar_hi, kbar_lo, vbar, kbar8_hi, kbar8_lo);
  }
}

// The same pooling with one CTA per (block, K or V) over ALL KV heads: a token's row of the cache is
// Hkv x 128 elements contiguous, so the CTA streams 128 whole rows (256 KB for 8 BF16 heads) behind ONE look-up of
// the block's page ids instead of one dependent look-up per 32 KB.  Used when the row's 16-byte chunks divide 256
// (Hkv a power of two, at most 16 BF16 / 32 FP8 heads).  Thread t owns chunk t mod C of the row and the tokens
// t / C, t / C + G, ... (G = 256 / C token groups): four 16-byte loads in flight per thread and batch, four CTAs per
// SM, fp32 accumulation, one shared-memory reduction over the G groups.  Page sizes are powers of two, so the slot
// of a token takes a shift and a mask (a division per load made the kernel ALU-bound: 143 -> 110 us at 128K).
// Measured at 131072 tokens, 8 BF16 heads: 93 us for 537 MB = 5.8 TB/s; a bare streaming read reaches 6.8 TB/s.
template <bool FP8>
__global__ void __launch_bounds__(256, 4) pool_rows_kernel(const uint8_t* __restrict__ k_cache,
                                                           const uint8_t* __restrict__ v_cache,
                                                           const int32_t* __restrict__ page_table,
                                                           const int32_t* __restrict__ plan_lk,
                                                           const int32_t* __restrict__ blk_off,
                                                           const float* __restrict__ k_scale,
                                                           const float* __restrict__ v_scale, DevParams P,
                                                           __nv_bfloat16* __restrict__ kbar_hi,
                                                           __nv_bfloat16* __restrict__ kbar_lo,
                                                           __nv_bfloat16* __restrict__ vbar,
                                                           uint8_t* __restrict__ kbar8_hi,
                                                           uint8_t* __restrict__ kbar8_lo,
                                                           const int32_t* __restrict__ carry,
                                                           int* __restrict__ status) {
  constexpr int CH = FP8 ? 8 : 16;             // 16-byte chunks per head row
  constexpr int EPC = FP8 ? 16 : 8;            // elements per chunk
  constexpr int BATCH = 4;                     // loads in flight per thread; four CTAs per SM overlap each other's set-up and reduction
  __shared__ float red[256 * EPC];             // [token group][chunk][element]
  __shared__ int32_t pids[kBlock / 8];         // page ids of the block (page size >= 8)

  const int which = blockIdx.x & 1;            // 0: K, 1: V
  const int gblk = blockIdx.x >> 1;
  int lo = 0, hi = P.num_seqs;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (blk_off[mid] <= gblk) lo = mid; else hi = mid;
  }
  const int b = lo, J = gblk - blk_off[b];
  if (carry != nullptr && J < carry[3 * b + 2]) return;   // carried over from the previous chunk (pool_carry_kernel)
  const int Lk = plan_lk[b];
  const int ntok = min(kBlock, Lk - J * kBlock);
  const int psz = P.page_size, ppb = P.pages_per_block;
  const int psz_log2 = 31 - __clz(psz);        // page sizes are powers of two: shifts and masks, no divisions per load
  if ((int)threadIdx.x < ppb) {
    int pid = -1;
    if ((int)threadIdx.x * psz < ntok) {
      pid = page_table[(size_t)b * P.max_pages_per_seq + J * ppb + threadIdx.x];
      if (pid < 0 || pid >= P.num_pages) {   // outside the pool: its tokens count as zeros, the call is flagged
        atomicOr(status + ST_BAD_LIST, 2);
        pid = -1;
      }
    }
    pids[threadIdx.x] = pid;
  }
  __syncthreads();

  const int C = P.num_kv_heads * CH;           // chunks per token row; divides 256
  const int G = 256 / C;
  const int chunk = threadIdx.x % C, tg = threadIdx.x / C;
  const int per = kBlock / G;                  // tokens of this thread
  const size_t row_bytes = (size_t)C * 16;
  const uint8_t* cache = which ? v_cache : k_cache;
  float acc[EPC];
#pragma unroll
  for (int i = 0; i < EPC; ++i) acc[i] = 0.f;
  for (int i0 = 0; i0 < per; i0 += BATCH) {
    // every load of the batch is issued unconditionally (a token that is not there reads the start of the cache
    // instead and is replaced by zeros afterwards), so that all of them are in flight before the first use
    uint4 dv[BATCH];
    bool ok[BATCH];
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int tl = tg + (i0 + u) * G;        // consecutive token groups interleave: the CTA reads G rows at a time
      const int pid = pids[min(tl, kBlock - 1) >> psz_log2];
      ok[u] = i0 + u < per && tl < ntok && pid >= 0;
      const size_t off = ok[u] ? (((size_t)pid << psz_log2) + (size_t)(tl & (psz - 1))) * row_bytes + chunk * 16 : 0;
      dv[u] = __ldg(reinterpret_cast<const uint4*>(cache + off));
    }
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      if (!ok[u]) dv[u] = make_uint4(0, 0, 0, 0);   // zero bit patterns add 0 in both encodings
      accum16<FP8>(dv[u], acc);
    }
  }
#pragma unroll
  for (int i = 0; i < EPC; ++i) red[(tg * C + chunk) * EPC + i] = acc[i];
  __syncthreads();
  const int nout = C * EPC;                    // Hkv x 128 means
  for (int o = threadIdx.x; o < nout; o += 256) {
    float sum = 0.f;
    for (int r = 0; r < G; ++r) sum += red[r * nout + o];
    const int h = o / kHeadDim;
    write_pooled<FP8>(which, sum / (float)ntok, (size_t)gblk * nout + o, h, k_scale, kbar_hi, kbar_lo, vbar, kbar8_hi,
                      kbar8_lo);
  }
}

// ----------------------------------------------------------------------------------------
// Work ordering (Sec. 3.3 "Sparsity-Aware Load Balancing", Eq. 21): segments sorted KV-head-major, then by
// descending block count (capped), by a counting sort on the device.  Order among equal keys is arbitrary;
// it only changes which CTA runs a segment, never a result.
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ int order_bucket(int h, int count) {
  int c = count < kCountBuckets - 1 ? count : kCountBuckets - 1;
  return h * kCountBuckets + (kCountBuckets - 1 - c);
}

__global__ void order_hist_kernel(const SegInfo* __restrict__ segs, const int32_t* __restrict__ count, int nseg,
                                  int32_t* __restrict__ hist) {
  int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= nseg) return;
  int c = count ? count[s] : segs[s].J_hi + 1;
  atomicAdd(&hist[order_bucket(segs[s].h, c)], 1);
}

// single CTA of 1024 threads: exclusive scan of nb = Hkv * kCountBuckets counters, in place.
__global__ void order_scan_kernel(int32_t* __restrict__ hist, int nb) {
  __shared__ int32_t part[1024];
  const int per = (nb + 1023) / 1024;
  const int beg = threadIdx.x * per, end = min(beg + per, nb);
  int s = 0;
  for (int i = beg; i < end; ++i) s += hist[i];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int d = 1; d < 1024; d <<= 1) {
    int v = threadIdx.x >= d ? part[threadIdx.x - d] : 0;
    __syncthreads();
    part[threadIdx.x] += v;
    __syncthreads();
  }
  int run = part[threadIdx.x] - s;
  for (int i = beg; i < end; ++i) {
    int v = hist[i];
    hist[i] = run;
    run += v;
  }
}

__global__ void order_scatter_kernel(const SegInfo* __restrict__ segs, const int32_t* __restrict__ count, int nseg,
                                     int32_t* __restrict__ cursor, int32_t* __restrict__ order) {
  int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= nseg) return;
  int c = count ? count[s] : segs[s].J_hi + 1;
  int pos = atomicAdd(&cursor[order_bucket(segs[s].h, c)], 1);
  order[pos] = s;
}

// ----------------------------------------------------------------------------------------
// Pooled statistics carried from one chunk of a chunked prefill to the next (Sec. 4.3, "Compatibility with Chunked Prefill": the index stage runs once
// per chunk; without this every chunk pools the whole cached prefix again).  The means of a block that was
// complete in the previous chunk are the same numbers in this one: rows are copied from the previous workspace's
// layout to this plan's.  carry[3 b + {0, 1, 2}] = first source row, first destination row, rows to copy of
// sequence b.  grid (sequences, row groups of 8); a row of one array is Hkv x 128 elements.
// ----------------------------------------------------------------------------------------
__global__ void pool_carry_kernel(const int32_t* __restrict__ carry, int row_bytes16, int row_bytes8,
                                  const uint8_t* __restrict__ s_khi, const uint8_t* __restrict__ s_klo,
                                  const uint8_t* __restrict__ s_vbar, const uint8_t* __restrict__ s_k8hi,
                                  const uint8_t* __restrict__ s_k8lo, uint8_t* __restrict__ d_khi,
                                  uint8_t* __restrict__ d_klo, uint8_t* __restrict__ d_vbar,
                                  uint8_t* __restrict__ d_k8hi, uint8_t* __restrict__ d_k8lo) {
  const int b = blockIdx.x;
  const int src0 = carry[3 * b], dst0 = carry[3 * b + 1], n = carry[3 * b + 2];
  for (int j = blockIdx.y * 8; j < n; j += gridDim.y * 8) {
    const int rows = min(8, n - j);
    auto copy = [&](const uint8_t* s, uint8_t* d, int rb) {
      if (rb == 0) return;
      const uint4* sp = reinterpret_cast<const uint4*>(s + (size_t)(src0 + j) * rb);
      uint4* dp = reinterpret_cast<uint4*>(d + (size_t)(dst0 + j) * rb);
      for (int i = threadIdx.x; i < rows * rb / 16; i += blockDim.x) dp[i] = sp[i];
    };
    copy(s_khi, d_khi, row_bytes16);
    copy(s_klo, d_klo, row_bytes16);
    copy(s_vbar, d_vbar, row_bytes16);
    copy(s_k8hi, d_k8hi, row_bytes8);
    copy(s_k8lo, d_k8lo, row_bytes8);
  }
}

}  // namespace fp2
