// Shared device-side definitions: segment table entries, kernel parameter block, compile-time shape.
#pragma once
#include <stdint.h>

namespace fp2 {

constexpr int kHeadDim = 128;     // d
constexpr int kBlock = 128;       // B: KV tokens per selection block (Sec. 4.1)
constexpr int kTileRows = 128;    // packed query rows per tile (kBlockM, Sec. 4.1)
constexpr int kMaxBlocks = 4096;  // KV blocks per sequence the kernels are compiled for (512K tokens)
constexpr int kMaxChunks = kMaxBlocks / 128;
constexpr int kCountBuckets = 1024;  // work-order histogram resolution (selected-block count, capped)

// One (sequence, KV head, tile) segment; built on the host by the planner.
struct SegInfo {
  int32_t b, h, t;
  int32_t nrows;    // real packed rows in the tile (<= 128)
  int32_t q_tok0;   // cu_seqlens_q[b]
  int32_t r0;       // first packed row of the tile
  int32_t pre;      // cached prefix length Lk - Lq
  int32_t Lk;
  int32_t J_lo;     // block of the first row's absolute position
  int32_t J_hi;     // block of the last row's absolute position (candidates are 0..J_hi)
  int32_t blk_off;  // first row of this sequence in the pooled-mean arrays
  int32_t seg;      // index of this segment in segment order
  int64_t off;      // seg_offset: start of this segment's list in blk_idx
  __host__ __device__ int h_seg() const { return seg; }
};
static_assert(sizeof(SegInfo) == 56, "SegInfo layout");

struct DevParams {
  int32_t num_q_heads, num_kv_heads, group;
  int32_t page_size, pages_per_block, max_pages_per_seq, num_pages;
  int32_t sink_blocks, window_blocks, use_correction;
  int32_t num_seqs, nseg, nblk_tot, total_q;
  int32_t fp8;
  int32_t q_tma;     // 1: the group size divides 128, so a packed query tile is a TMA box [128 bytes, g heads, 128 / g tokens]
                     //    (x 2 for BF16); used by the attention kernel (both dtypes) and the BF16 scorer
  int32_t q_box_tok; // tokens of the box that holds a packed tile's rows: 128 / g, or floor((g - 1 + 127) / g) + 1 when g does not
                     // divide 128 (the tile then starts r0 % g rows into the box)
  int32_t q_raw_tma; // 1: FP8 plans whose box fits the scorer's raw staging slot: the scorer fetches query tiles by TMA
  int32_t diag_mma;  // 1: a tile spans at most 32 positions (g >= 4), so the causal mask of a diagonal block can ride
                     //    on a K = 32 one-hot MMA step in the attention kernel
  float alpha;
  float scale_log2;  // softmax scale * log2(e)
};

}  // namespace fp2
