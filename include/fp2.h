/* fp2 -- block-sparse causal prefill attention for B200 (sm_100a): C ABI.
 *
 * Two stages (Algorithm 1 of the paper):
 *   stage 1  fp2_select_blocks   block-mean pooling (Eq. 5), block energies of every (KV head, packed query
 *                                tile, KV block) (Eq. 19), max-based threshold plus forced sink / window /
 *                                diagonal blocks (Eq. 3, Eq. 20) -> per-(sequence, KV head, tile) block lists;
 *   stage 2  fp2_sparse_prefill  flash attention over the listed blocks, the unlisted fully visible blocks
 *                                entering through their pooled means (mean correction, Eq. 6), over a paged
 *                                KV cache (Eq. 22) in a continuous batch with PackGQA row packing (Eq. 13).
 *   fp2_dense_prefill is stage 2 with every candidate block attended exactly.
 *
 * Conventions common to all calls
 *   - Every tensor pointer is a DEVICE pointer unless its name starts with h_ (host).  The caller owns all
 *     tensors, list buffers and the workspace; the library owns only the plan object.  Stage calls allocate
 *     and free nothing, enqueue their kernels on the given stream and return without synchronising.
 *   - Layouts (row-major, innermost last):
 *       q, out        [total_q, num_q_heads, 128]        BF16 (out always BF16; q BF16 or FP8 e4m3)
 *       k_cache, v_cache [num_pages, page_size, num_kv_heads, 128]   BF16 or FP8 e4m3
 *       page_table    int32 [num_seqs, max_pages_per_seq]; token j of sequence b lives in slot
 *                     page_table[b][j / page_size] * page_size + j % page_size  (Eq. 22)
 *       cu_seqlens_q  int32 [num_seqs + 1]  offsets of the sequences' new tokens in q / out
 *       seqlens_k     int32 [num_seqs]      total KV tokens (cached prefix + new tokens)
 *       q_scale [num_q_heads], k_scale / v_scale [num_kv_heads]  fp32 de-quantisation scales, FP8 only
 *                     (NULL for BF16); per-tensor scaling (Eq. 15) is the case of equal entries
 *       lse           fp32 [num_q_heads, total_q], natural log of the softmax denominator (may be NULL)
 *     Query i of sequence b sits at absolute position (seqlens_k[b] - Lq_b) + i: the causal mask is aligned
 *     to the end of the KV sequence, so cached prefixes (chunked prefill) are visible to every new token.
 *   - Segments.  With g = num_q_heads / num_kv_heads, packed row r of a KV head's query matrix is position
 *     r / g, query head h_kv * g + r % g (Eq. 13); tile t holds packed rows [128 t, 128 (t+1)).  Segment
 *     seg = num_kv_heads * tile_off[b] + h_kv * ntiles_b + t, ntiles_b = ceil(g * Lq_b / 128), tile_off the
 *     exclusive scan of ntiles.  Lists are a padded CSR: seg_offset[seg] (fixed by the plan: exclusive scan
 *     of the candidate counts J_hi + 1), seg_count[seg] selected blocks, blk_idx[seg_offset[seg] + k]
 *     ascending ids of 128-token KV blocks.
 *   - Lengths.  Every kernel takes its geometry (lengths, prefixes, tiles, block ranges) from the plan, i.e. from
 *     the HOST copies given to fp2_plan_create, which are validated there.  The device arrays cu_seqlens_q and
 *     seqlens_k of the stage calls must hold the same values; the current kernels do not read them, so a
 *     disagreement cannot move an access out of bounds.
 *   - Errors.  Every call returns an fp2_status.  Problems visible on the host (null pointers, unsupported
 *     shapes, inconsistent lengths in fp2_plan_create) are reported before anything is launched.  The device
 *     never traps: waits inside the kernels are bounded; list entries outside 0..J_hi are clamped; a page id
 *     outside [0, num_pages) in a live page-table entry is not dereferenced (pooling reads zeros for its tokens,
 *     the attention kernel skips the page).  Each of these conditions is recorded in a status block that
 *     fp2_read_status returns.
 */
#ifndef FP2_H_
#define FP2_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FP2_OK = 0,
  FP2_ERR_INVALID_ARG = 1,  /* null pointer, inconsistent lengths, malformed list seen on the device */
  FP2_ERR_UNSUPPORTED = 2,  /* head_dim != 128, block_size != 128, page_size not dividing 128, ...    */
  FP2_ERR_CAPACITY = 3,     /* sequence longer than the compiled maximum                              */
  FP2_ERR_CUDA = 4,         /* a CUDA runtime / driver call failed                                    */
  FP2_ERR_TIMEOUT = 5       /* a bounded wait inside a kernel expired                                 */
} fp2_status;

typedef enum { FP2_BF16 = 0, FP2_FP8_E4M3 = 1 } fp2_dtype;

typedef struct fp2_plan fp2_plan; /* opaque */
typedef void* fp2_stream;         /* a cudaStream_t passed as an address-sized handle; NULL = default */

/* Shapes and method parameters (Sec. 4.1: B = 128, 256 sink tokens, 512-token window, alpha = 0.1). */
typedef struct {
  int32_t num_seqs, total_q, num_q_heads, num_kv_heads;
  int32_t head_dim;       /* must be 128                                                              */
  int32_t block_size;     /* B, KV tokens per selection block; must be 128                            */
  int32_t tile_rows;      /* packed query rows per tile; must be 128                                  */
  int32_t page_size;      /* p; 8, 16, 32, 64 or 128                                                  */
  int32_t num_pages, max_pages_per_seq;
  int32_t sink_tokens;    /* blocks J < ceil(sink_tokens / B) are always selected                     */
  int32_t window_tokens;  /* blocks J >= J_lo - ceil(window_tokens / B) are always selected           */
  int32_t use_correction; /* 1: Eq. 6 (mean correction); 0: Eq. 4 (plain truncation)                  */
  float alpha;            /* threshold factor of Eq. 3 / Eq. 20                                       */
  float softmax_scale;    /* 0 selects 1 / sqrt(head_dim)                                             */
  int32_t dtype;          /* fp2_dtype of q, k_cache, v_cache                                         */
} fp2_params;

/* Planner (host side; the per-step metadata of Sec. 3.4 "Serving Integration").  Takes HOST copies of the
 * lengths, builds the segment table and uploads it to the current device (one small allocation owned by the
 * plan, freed by fp2_plan_destroy).  h_cu_seqlens_q has num_seqs + 1 entries, h_seqlens_k num_seqs.
 * Returns FP2_ERR_INVALID_ARG for null / inconsistent input (Lq_b < 0, Lq_b > Lk_b, sum Lq != total_q, pages
 * needed > max_pages_per_seq), FP2_ERR_UNSUPPORTED / FP2_ERR_CAPACITY for shapes outside the compiled
 * kernels (see fp2_status).  *out is written only on FP2_OK.  If no CUDA device is usable the plan is still
 * returned -- sizes and the segment table can be queried -- but stage calls on it return FP2_ERR_CUDA. */
fp2_status fp2_plan_create(const fp2_params* params, const int32_t* h_cu_seqlens_q, const int32_t* h_seqlens_k,
                           fp2_plan** out);

/* Sizes the caller needs: number of segments, capacity of blk_idx in entries (worst case = all candidate
 * pairs), bytes of device workspace (pooled statistics, work order, status block).  Any output may be NULL. */
fp2_status fp2_plan_sizes(const fp2_plan* plan, int64_t* num_segments, int64_t* idx_capacity,
                          int64_t* workspace_bytes);

void fp2_plan_destroy(fp2_plan* plan);

/* Host-side view of one row of the segment table (PackGQA geometry, Eq. 13; candidates 0..J_hi):
 * out10 = {b, h_kv, t, first packed row, real rows, prefix length, Lk, J_lo, J_hi, first pooled-block row of
 * the sequence}; *list_offset = seg_offset[seg] (may be NULL).  Host memory; needs no device. */
fp2_status fp2_plan_segment(const fp2_plan* plan, int64_t seg, int32_t* out10, int64_t* list_offset);

/* Stage 1 (Algorithm 1, lines 1-5).  Pools K and V into per-block means kept in `workspace`, scores every
 * candidate block of every segment and writes the lists.
 *   out: seg_offset int64 [num_segments + 1], seg_count int32 [num_segments], blk_idx int32 [idx_capacity].
 * v_cache is read here because the pooled V means (used by stage 2's correction) are produced in the same
 * pass.  The workspace must be at least workspace_bytes and 1024-byte aligned, and must be passed unchanged to
 * the following fp2_sparse_prefill.  Its first 128 bytes hold the status block and the work counter and
 * must be zero before the first stage call (fp2_read_status clears the status block again). */
fp2_status fp2_select_blocks(fp2_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                             const int32_t* page_table, const int32_t* cu_seqlens_q, const int32_t* seqlens_k,
                             const float* q_scale, const float* k_scale, const float* v_scale,
                             int64_t* seg_offset, int32_t* seg_count, int32_t* blk_idx, void* workspace,
                             fp2_stream stream);

/* Block-mean pooling alone (Eq. 5; Algorithm 1 line 2): the first kernel of fp2_select_blocks as a call of its own.
 * Reads K and V once through the page table and leaves the per-block means (kbar, vbar of every 128-token block
 * and KV head, in the operand formats the scorer and the correction chunks read) in `workspace`, exactly as
 * fp2_select_blocks does.  For callers that refresh the pooled statistics without re-running the selection (lists
 * supplied by the caller, then fp2_sparse_prefill with pooled_valid = 1), and for timing the pooling pass by
 * itself.  k_scale / v_scale are read for FP8 plans only.  One kernel on `stream`; nothing is allocated. */
fp2_status fp2_pool_blocks(fp2_plan* plan, const void* k_cache, const void* v_cache, const int32_t* page_table,
                           const int32_t* seqlens_k, const float* k_scale, const float* v_scale, void* workspace,
                           fp2_stream stream);

/* Stage 2 (Algorithm 1, lines 6-11; Eq. 4, Eq. 6).  Attends exactly over the listed blocks; with
 * use_correction = 1 every unlisted block J < J_lo (fully visible to the whole tile) contributes
 * |B_J| e^{q.kbar_J / sqrt(d)} (vbar_J, 1) to numerator and denominator.  The lists may come from
 * fp2_select_blocks or from the caller (ascending, unique, within 0..J_hi; entries outside are clamped and
 * flagged in the status block).  `pooled_valid` != 0 says the workspace still holds the pooled means of a
 * preceding fp2_select_blocks on the same inputs; 0 makes this call recompute them.
 *   out: out BF16 [total_q, num_q_heads, 128]; lse fp32 [num_q_heads, total_q] or NULL. */
fp2_status fp2_sparse_prefill(fp2_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* page_table, const int32_t* cu_seqlens_q, const int32_t* seqlens_k,
                              const int64_t* seg_offset, const int32_t* seg_count, const int32_t* blk_idx,
                              const float* q_scale, const float* k_scale, const float* v_scale, void* out,
                              float* lse, void* workspace, int32_t pooled_valid, fp2_stream stream);

/* Dense causal attention through the same kernel: every candidate block 0..J_hi of every tile is attended
 * exactly, nothing is pooled or corrected (the paper's own dense baseline, Sec. 3.3). */
fp2_status fp2_dense_prefill(fp2_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                             const int32_t* page_table, const int32_t* cu_seqlens_q, const int32_t* seqlens_k,
                             const float* q_scale, const float* k_scale, const float* v_scale, void* out,
                             float* lse, void* workspace, fp2_stream stream);

/* (No counterpart in the paper.)  fp2_dense_prefill for callers that have no device workspace to hand in and
 * may not create one: a plug-in whose host passes it fixed input and output buffers and forbids device
 * allocation, or code on a path where the memory allocator must not be entered (a framework callback, a
 * latency-critical loop that may not take the allocator's lock).  The scratch
 * of the dense path (status block, work counter, work order, counting-sort histogram) lives in a device array
 * that is part of the library image: about 0.4 MB on every GPU that loads the library, held until exit.
 *   - Limits: at most 65536 segments and 32 KV heads; larger plans are rejected with FP2_ERR_CAPACITY.
 *     BF16 and FP8 plans alike (the dense path of an FP8 plan needs no more scratch than that of a BF16 plan).
 *   - The call allocates and frees nothing.  The first call on a device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current); that first call should come before any stream
 *     capture.
 *   - All calls on a device share the one array, and it keeps what the previous call left: the entry point
 *     clears the words that must start at zero, on `stream`.  Two calls whose kernels overlap on the GPU
 *     (different streams, no dependency) race on it -- serialise them.
 *   - The status block of this variant sits in the same array: fp2_read_status(plan, NULL, ...) reads and clears
 *     it (bounded waits that ran out, page ids that were skipped), like it does for a caller's workspace.
 * Arguments and results as fp2_dense_prefill, without `workspace`. */
fp2_status fp2_dense_prefill_static(fp2_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                                    const int32_t* page_table, const int32_t* cu_seqlens_q,
                                    const int32_t* seqlens_k, const float* q_scale, const float* k_scale,
                                    const float* v_scale, void* out, float* lse, fp2_stream stream);

/* Pooled statistics carried over between the chunks of a chunked prefill (Sec. 4.3 "Compatibility with Chunked
 * Prefill": the index stage is re-run for every chunk; pooling the cached prefix again each time is avoidable work).  `src` /
 * `src_workspace` are the plan and workspace of the previous chunk after its fp2_select_blocks; `dst` is this
 * chunk's plan.  h_src_seq (HOST, dst.num_seqs entries) names for every sequence of `dst` its index in `src`, or
 * -1 for a sequence that was not there.  For every block that was complete then and is complete now
 * (floor(min(Lk_src, Lk_dst) / 128) per sequence) the pooled means are copied from src_workspace to
 * dst_workspace, and the next fp2_select_blocks on `dst` -- only that one -- pools just the remaining blocks.
 * The caller guarantees that those blocks hold the same K / V (and, for FP8, the same scales) as before, which is
 * what a paged prefix cache does.  Plans must agree in KV heads and dtype.  One copy kernel on `stream`; the
 * stream must be ordered after the previous chunk's fp2_select_blocks and before dst's.  Nothing is allocated.
 * fp2_pool_carry_count is the host-side half alone: h_blocks[b] = blocks that would be carried (needs no device). */
fp2_status fp2_pool_carry(fp2_plan* dst, void* dst_workspace, const fp2_plan* src, const void* src_workspace,
                          const int32_t* h_src_seq, fp2_stream stream);
fp2_status fp2_pool_carry_count(const fp2_plan* dst, const fp2_plan* src, const int32_t* h_src_seq,
                                int32_t* h_blocks);

/* KV splitting (Eq. 18; Sec. 3.3 "Sparsity-Aware Load Balancing"), off by default.  Plans with few segments
 * (fewer than four per worker CTA of the attention kernel) can cut the iteration sequence of a heavy segment --
 * its list backwards, then its correction chunks -- into up to 16 contiguous parts of about equal count, run the
 * parts as separate work units and merge their partial results by log-sum-exp weights; fp2_sparse_prefill and
 * fp2_dense_prefill then enqueue two more kernels (the device-side split plan and the merge).  The result is the
 * same up to rounding.
 *   target < 0 (default): never split;  0: automatic, parts of about the mean load per worker and at least 12
 *   iterations;  > 0: parts of about `target` iterations (never more than nseg + 2 workers parts in all, which
 *   is what the workspace is sized for).
 * Larger plans are never split and ignore the setting; so do calls in which no segment could yield two parts.
 * On B200 the split did not pay in any case measured (the attention kernel already keeps two independent CTAs per
 * SM, and the two extra launches cost ~10 us), hence the default.  Host-side, takes effect at the next stage call. */
fp2_status fp2_plan_set_split(fp2_plan* plan, int32_t target);

/* Index export (Algorithm 1 line 5; Sec. 3.3 "Index-Driven Sparse Traversal", Eq. 17).  Turns the padded lists
 * (seg_count, blk_idx as fp2_select_blocks writes them or as a caller supplies them) into a compact CSR over
 * physical tiles of `tile_tokens` tokens (16, 32, 64 or 128; the paper's kernels use 64): every listed logical
 * block J becomes the tiles J*(128/tile_tokens) ... that hold at least one token of the sequence, ascending.
 *   out: cu  int32 [num_segments + 1]   cu[g] = first entry of segment g, cu[num_segments] = total entries;
 *        idx int32 [idx_len]            idx_len must be at least idx_capacity * (128 / tile_tokens).
 * Segments are in segment order (KV-head-major inside a sequence), i.e. the index is organised per KV head.
 * Malformed list entries are clamped as in fp2_sparse_prefill and flagged in the status block of `workspace`.
 * FP2_ERR_UNSUPPORTED if the worst-case entry count does not fit int32, FP2_ERR_CAPACITY if idx_len is too
 * small.  All pointers device memory; three small kernels on `stream`; nothing is allocated. */
fp2_status fp2_export_csr(fp2_plan* plan, const int32_t* seg_count, const int32_t* blk_idx, int32_t tile_tokens,
                          int32_t* cu, int32_t* idx, int64_t idx_len, void* workspace, fp2_stream stream);

/* Page-level table from a token-level slot map (Sec. 3.4 "Serving Integration": the page index is the token-level
 * mapping read every page_size entries; Eq. 22 is the inverse).  token_to_slot int32 [num_seqs, max_tokens] holds
 * the global slot (page * page_size + offset) of token j of sequence b; entries past seqlens_k[b] are not read.
 *   out: page_table int32 [num_seqs, max_pages_per_seq], -1 for pages past the end of a sequence.
 * A sampled slot that is negative or not the first slot of a page is flagged in the status block
 * (fp2_read_status returns FP2_ERR_INVALID_ARG).  Device pointers; one kernel on `stream`. */
fp2_status fp2_page_table_from_token_map(fp2_plan* plan, const int32_t* token_to_slot, int32_t max_tokens,
                                         const int32_t* seqlens_k, int32_t* page_table, void* workspace,
                                         fp2_stream stream);

/* Synchronises `stream`, reads the status block of `workspace` and clears it.  Returns FP2_ERR_TIMEOUT if a
 * bounded wait expired, FP2_ERR_INVALID_ARG if a list entry had to be clamped or a page id was out of range, else
 * FP2_OK.  If h_status_words is not NULL it receives the 8 raw int32 words (host memory).  workspace == NULL
 * selects the status block of fp2_dense_prefill_static on the plan's device, which must be the current one. */
fp2_status fp2_read_status(fp2_plan* plan, void* workspace, int32_t* h_status_words, fp2_stream stream);

/* (No counterpart in the paper: a self-test of the library's failure handling.)  Every wait inside the kernels --
 * on a bulk copy, an MMA, another warp -- is bounded: after a cycle budget it gives up, records the fact (status
 * word 0) and the place (word 1) in the status block, and the CTA leaves the ordinary way, releasing its tensor
 * memory.  This call proves that mechanism on the device without involving the attention path: it launches one
 * 64-thread CTA that allocates tensor memory and waits, with a budget of 10^6 cycles (under a millisecond), on a
 * barrier that nobody ever arrives on.  The kernel returns by itself; the following fp2_read_status on the same
 * workspace returns FP2_ERR_TIMEOUT with words {1, 901 or 902, ...} and clears the block, and later stage calls on
 * the same plan and workspace are unaffected.  Nothing is allocated; one kernel on `stream`. */
fp2_status fp2_selftest_bounded_wait(fp2_plan* plan, void* workspace, fp2_stream stream);

/* Number of kernels the last stage call on this plan enqueued (host counter). */
int32_t fp2_last_launch_count(const fp2_plan* plan);

const char* fp2_status_string(fp2_status s);

#ifdef __cplusplus
}
#endif
#endif /* FP2_H_ */
