// C ABI of the library (declared in include/fp2.h): host-side planner, argument checks, TMA tensor maps,
// kernel launches.  No device memory is allocated in the stage calls; the plan owns one small device table.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <algorithm>
#include <vector>

#include "../../include/fp2.h"
#include "common.cuh"
#include "pool_kv.cuh"
#include "score_select.cuh"
#include "score_pair.cuh"
#include "sparse_attn.cuh"
#include "index_export.cuh"

using namespace fp2;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct fp2_plan {
  fp2_params prm;
  DevParams dev;
  int device;
  int num_sms;
  int64_t nseg, idx_capacity, nblk_tot;
  std::vector<int32_t> h_cu_q, h_lk;
  std::vector<SegInfo> h_segs;
  // device table owned by the plan: [SegInfo x nseg][blk_off x (ns+1)]
  void* d_table;
  SegInfo* d_segs;
  int32_t* d_blk_off;
  int32_t* d_carry;                 // [3 x num_seqs]: pooled rows carried over from a previous chunk (fp2_pool_carry)
  int32_t* d_lk;                    // [num_seqs]: KV lengths as given to fp2_plan_create
  int2* d_units;                    // scorer work units of BF16 plans with TMA query tiles: (segment, second segment or -1)
  int32_t nunits;
  std::vector<int32_t> h_blk_off, h_carry;
  bool carry_valid;
  // workspace layout (byte offsets)
  int64_t ws_status, ws_counter, ws_khi, ws_klo, ws_vbar, ws_k8hi, ws_k8lo, ws_order, ws_hist, ws_bytes;
  // KV splitting (Eq. 18): only plans with few segments carry the buffers
  bool split_capable;
  int32_t split_target;   // < 0 off, 0 automatic, > 0 requested iterations per part
  int32_t max_iters;      // longest iteration sequence any segment can have (all candidates + all chunks)
  int64_t split_units_cap, ws_unit_seg, ws_unit_split, ws_seg_split, ws_part_ml, ws_part_o;
  EncodeTiledFn encode;
  int32_t last_launches;
  bool attrs_set;
};

static inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

extern "C" const char* fp2_status_string(fp2_status s) {
  switch (s) {
    case FP2_OK: return "ok";
    case FP2_ERR_INVALID_ARG: return "invalid argument";
    case FP2_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case FP2_ERR_CAPACITY: return "sequence exceeds compiled capacity";
    case FP2_ERR_CUDA: return "CUDA error";
    case FP2_ERR_TIMEOUT: return "bounded wait expired inside a kernel";
  }
  return "unknown status";
}

extern "C" fp2_status fp2_plan_create(const fp2_params* p, const int32_t* h_cu, const int32_t* h_lk, fp2_plan** out) {
  if (!p || !h_cu || !h_lk || !out) return FP2_ERR_INVALID_ARG;
  if (p->num_seqs <= 0 || p->total_q < 0 || p->num_q_heads <= 0 || p->num_kv_heads <= 0) return FP2_ERR_INVALID_ARG;
  if (p->num_q_heads % p->num_kv_heads != 0) return FP2_ERR_INVALID_ARG;
  if (p->head_dim != kHeadDim || p->block_size != kBlock || p->tile_rows != kTileRows) return FP2_ERR_UNSUPPORTED;
  const int ps = p->page_size;
  if (!(ps == 8 || ps == 16 || ps == 32 || ps == 64 || ps == 128)) return FP2_ERR_UNSUPPORTED;
  if (p->dtype != FP2_BF16 && p->dtype != FP2_FP8_E4M3) return FP2_ERR_UNSUPPORTED;
  if (p->num_pages <= 0 || p->max_pages_per_seq <= 0) return FP2_ERR_INVALID_ARG;
  if (p->sink_tokens < 0 || p->window_tokens < 0) return FP2_ERR_INVALID_ARG;
  if (!(p->alpha == p->alpha) || p->softmax_scale < 0.f) return FP2_ERR_INVALID_ARG;
  if (h_cu[0] != 0 || h_cu[p->num_seqs] != p->total_q) return FP2_ERR_INVALID_ARG;

  const int g = p->num_q_heads / p->num_kv_heads;
  int64_t ntiles_tot = 0, nblk_tot = 0;
  for (int b = 0; b < p->num_seqs; ++b) {
    const int64_t lq = (int64_t)h_cu[b + 1] - h_cu[b], lk = h_lk[b];
    if (lq < 0 || lk < 0 || lq > lk) return FP2_ERR_INVALID_ARG;
    if ((lk + ps - 1) / ps > p->max_pages_per_seq) return FP2_ERR_INVALID_ARG;
    const int64_t nblk = (lk + kBlock - 1) / kBlock;
    if (nblk > kMaxBlocks) return FP2_ERR_CAPACITY;
    ntiles_tot += (g * lq + kTileRows - 1) / kTileRows;
    nblk_tot += nblk;
  }
  if (ntiles_tot * p->num_kv_heads > (int64_t)0x7fffffff || nblk_tot * p->num_kv_heads * 2 > (int64_t)0x7fffffff)
    return FP2_ERR_CAPACITY;

  fp2_plan* pl = new (std::nothrow) fp2_plan();
  if (!pl) return FP2_ERR_CUDA;
  pl->prm = *p;
  pl->h_cu_q.assign(h_cu, h_cu + p->num_seqs + 1);
  pl->h_lk.assign(h_lk, h_lk + p->num_seqs);
  pl->nseg = ntiles_tot * p->num_kv_heads;
  pl->nblk_tot = nblk_tot;
  pl->d_table = nullptr;
  pl->last_launches = 0;
  pl->attrs_set = false;

  // segment table: seg = Hkv * tile_off[b] + h * ntiles_b + t
  std::vector<SegInfo> segs((size_t)pl->nseg);
  std::vector<int32_t> blk_off((size_t)p->num_seqs + 1);
  int64_t tile_off = 0, off = 0, boff = 0;
  for (int b = 0; b < p->num_seqs; ++b) {
    const int lq = h_cu[b + 1] - h_cu[b], lk = h_lk[b], pre = lk - lq;
    const int nt = (int)(((int64_t)g * lq + kTileRows - 1) / kTileRows);
    blk_off[b] = (int32_t)boff;
    for (int h = 0; h < p->num_kv_heads; ++h)
      for (int t = 0; t < nt; ++t) {
        SegInfo& s = segs[(size_t)(p->num_kv_heads * tile_off + (int64_t)h * nt + t)];
        const int64_t r0 = (int64_t)t * kTileRows;
        const int64_t r1 = r0 + kTileRows < (int64_t)g * lq ? r0 + kTileRows : (int64_t)g * lq;
        s.b = b; s.h = h; s.t = t;
        s.nrows = (int)(r1 - r0);
        s.q_tok0 = h_cu[b];
        s.r0 = (int)r0;
        s.pre = pre;
        s.Lk = lk;
        s.J_lo = (int)((pre + r0 / g) / kBlock);
        s.J_hi = (int)((pre + (r1 - 1) / g) / kBlock);
        s.blk_off = (int32_t)boff;
        s.seg = (int32_t)(p->num_kv_heads * tile_off + (int64_t)h * nt + t);
        s.off = 0;
      }
    tile_off += nt;
    boff += (lk + kBlock - 1) / kBlock;
  }
  blk_off[p->num_seqs] = (int32_t)boff;
  pl->max_iters = 0;
  for (int64_t i = 0; i < pl->nseg; ++i) {
    segs[(size_t)i].off = off;
    off += segs[(size_t)i].J_hi + 1;
    const int iters = segs[(size_t)i].J_hi + 1 + (segs[(size_t)i].J_lo + 127) / 128;
    pl->max_iters = iters > pl->max_iters ? iters : pl->max_iters;
  }
  pl->idx_capacity = off;
  pl->h_blk_off = blk_off;
  pl->carry_valid = false;
  pl->d_carry = nullptr;

  // Scorer work units (score_pair_kernel): adjacent tiles (t-1, t) of one (sequence, KV head) share their candidate
  // blocks, so they are scored together when the later one has at most kPairMaxCand candidates; heaviest first
  // (descending segment index, like the single-tile scorer's order).
  std::vector<int2> units;
  {
    int64_t tile_off2 = 0;
    std::vector<int64_t> toff((size_t)p->num_seqs), ntiles((size_t)p->num_seqs);
    for (int b = 0; b < p->num_seqs; ++b) {
      const int lq = h_cu[b + 1] - h_cu[b];
      ntiles[(size_t)b] = ((int64_t)g * lq + kTileRows - 1) / kTileRows;
      toff[(size_t)b] = tile_off2;
      tile_off2 += ntiles[(size_t)b];
    }
    for (int b = p->num_seqs - 1; b >= 0; --b)
      for (int h = p->num_kv_heads - 1; h >= 0; --h) {
        const int64_t base = p->num_kv_heads * toff[(size_t)b] + (int64_t)h * ntiles[(size_t)b];
        for (int64_t t = ntiles[(size_t)b] - 1; t >= 0;) {
          if (t >= 1 && segs[(size_t)(base + t)].J_hi + 1 <= kPairMaxCand) {
            units.push_back(make_int2((int)(base + t - 1), (int)(base + t)));
            t -= 2;
          } else {
            units.push_back(make_int2((int)(base + t), -1));
            t -= 1;
          }
        }
      }
  }
  pl->nunits = (int32_t)units.size();
  pl->d_units = nullptr;

  // Device part.  Without a usable CUDA device the plan is still returned (sizes and the segment table can be
  // queried), but every stage call on it fails with FP2_ERR_CUDA.
  pl->device = -1;
  pl->num_sms = 0;
  pl->encode = nullptr;
  cudaDeviceProp prop;
  int dev = -1;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess) {
    if (prop.major != 10) { delete pl; return FP2_ERR_UNSUPPORTED; }
    pl->device = dev;
    pl->num_sms = prop.multiProcessorCount;
    const size_t seg_bytes = (size_t)align_up((int64_t)sizeof(SegInfo) * (pl->nseg > 0 ? pl->nseg : 1), 256);
    const size_t boff_bytes = (size_t)align_up((int64_t)sizeof(int32_t) * blk_off.size(), 256);
    const size_t carry_bytes = (size_t)align_up((int64_t)sizeof(int32_t) * 3 * (p->num_seqs > 0 ? p->num_seqs : 1), 256);
    const size_t lk_bytes = (size_t)align_up((int64_t)sizeof(int32_t) * (p->num_seqs > 0 ? p->num_seqs : 1), 256);
    const size_t tab_bytes = seg_bytes + boff_bytes + carry_bytes + lk_bytes + sizeof(int2) * (units.size() + 1);
    if (cudaMalloc(&pl->d_table, tab_bytes) != cudaSuccess) { delete pl; return FP2_ERR_CUDA; }
    pl->d_segs = reinterpret_cast<SegInfo*>(pl->d_table);
    pl->d_blk_off = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(pl->d_table) + seg_bytes);
    pl->d_carry = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(pl->d_table) + seg_bytes + boff_bytes);
    pl->d_lk = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(pl->d_table) + seg_bytes + boff_bytes + carry_bytes);
    pl->d_units = reinterpret_cast<int2*>(reinterpret_cast<uint8_t*>(pl->d_table) + seg_bytes + boff_bytes + carry_bytes + lk_bytes);
    if ((pl->nseg > 0 && cudaMemcpy(pl->d_segs, segs.data(), sizeof(SegInfo) * segs.size(),
                                    cudaMemcpyHostToDevice) != cudaSuccess) ||
        cudaMemcpy(pl->d_blk_off, blk_off.data(), sizeof(int32_t) * blk_off.size(), cudaMemcpyHostToDevice) !=
            cudaSuccess ||
        cudaMemcpy(pl->d_lk, h_lk, sizeof(int32_t) * p->num_seqs, cudaMemcpyHostToDevice) != cudaSuccess ||
        (!units.empty() && cudaMemcpy(pl->d_units, units.data(), sizeof(int2) * units.size(), cudaMemcpyHostToDevice) !=
                               cudaSuccess)) {
      cudaFree(pl->d_table);
      delete pl;
      return FP2_ERR_CUDA;
    }
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
      cudaFree(pl->d_table);
      delete pl;
      return FP2_ERR_CUDA;
    }
    pl->encode = reinterpret_cast<EncodeTiledFn>(fn);
  } else {
    (void)cudaGetLastError();
  }
  pl->h_segs.swap(segs);

  // workspace layout
  const int64_t pooled = align_up(nblk_tot * p->num_kv_heads * kHeadDim * 2, 1024);
  int64_t o = 0;
  pl->ws_status = o;  o += 64;
  pl->ws_counter = o; o += 64;
  o = align_up(o, 1024);
  pl->ws_khi = o;  o += pooled;
  pl->ws_klo = o;  o += pooled;
  pl->ws_vbar = o; o += pooled;
  // FP8 plans: the pooled keys once more, as an e4m3 hi + lo pair in raw units (correction chunks of the
  // attention kernel)
  const int64_t pooled8 = p->dtype == FP2_FP8_E4M3 ? align_up(nblk_tot * p->num_kv_heads * kHeadDim, 1024) : 0;
  pl->ws_k8hi = o; o += pooled8;
  pl->ws_k8lo = o; o += pooled8;
  pl->ws_order = o; o += align_up(4 * (pl->nseg > 0 ? pl->nseg : 1), 1024);
  pl->ws_hist = o;  o += align_up(4 * ((int64_t)p->num_kv_heads * kCountBuckets + 1), 1024);
  // KV splitting pays when there are fewer units than a few waves of workers; the unit arrays and the partial
  // results are sized for nseg + 2 workers units, the bound split_plan_kernel keeps
  const int64_t workers = (int64_t)pl->num_sms * AttnCfg<false>::kCtasPerSm;
  pl->split_target = -1;   // off unless asked for: see fp2_plan_set_split
  pl->split_capable = pl->num_sms > 0 && pl->nseg > 0 && pl->nseg < 4 * workers && pl->nseg + 2 * workers < 65536;
  pl->split_units_cap = pl->split_capable ? pl->nseg + 2 * workers : 0;
  pl->ws_unit_seg = o;   o += align_up(4 * pl->split_units_cap, 1024);
  pl->ws_unit_split = o; o += align_up(4 * pl->split_units_cap, 1024);
  pl->ws_seg_split = o;  o += align_up(pl->split_capable ? 8 * pl->nseg : 0, 1024);   // per-segment word + list of split segments
  pl->ws_part_ml = o;    o += align_up(pl->split_units_cap * 128 * 8, 1024);
  pl->ws_part_o = o;     o += pl->split_units_cap * 128 * 128 * 4;
  pl->ws_bytes = o;

  DevParams& d = pl->dev;
  d.num_q_heads = p->num_q_heads; d.num_kv_heads = p->num_kv_heads; d.group = g;
  d.page_size = ps; d.pages_per_block = kBlock / ps; d.max_pages_per_seq = p->max_pages_per_seq;
  d.num_pages = p->num_pages;
  d.sink_blocks = (p->sink_tokens + kBlock - 1) / kBlock;
  d.window_blocks = (p->window_tokens + kBlock - 1) / kBlock;
  d.use_correction = p->use_correction ? 1 : 0;
  d.num_seqs = p->num_seqs; d.nseg = (int32_t)pl->nseg; d.nblk_tot = (int32_t)nblk_tot; d.total_q = p->total_q;
  d.fp8 = p->dtype == FP2_FP8_E4M3;
  d.q_tma = (128 % g == 0) ? 1 : 0;
  d.q_box_tok = (128 % g == 0) ? 128 / g : (g - 1 + 127) / g + 1;
  d.q_raw_tma = (d.fp8 && g <= 128 && d.q_box_tok <= 256 && g * d.q_box_tok * 128 <= kScoreRawBytes) ? 1 : 0;
  // positions spanned by a 128-row packed tile: 128 / g when g divides 128, else up to floor((g - 1 + 127) / g) + 1
  d.diag_mma = ((128 % g == 0) ? 128 / g : (g - 1 + 127) / g + 1) <= 32 ? 1 : 0;
  d.alpha = p->alpha;
  const double sc = p->softmax_scale > 0.f ? (double)p->softmax_scale : 1.0 / sqrt((double)kHeadDim);
  d.scale_log2 = (float)(sc * 1.4426950408889634);
  *out = pl;
  return FP2_OK;
}

extern "C" fp2_status fp2_plan_sizes(const fp2_plan* pl, int64_t* nseg, int64_t* cap, int64_t* ws) {
  if (!pl) return FP2_ERR_INVALID_ARG;
  if (nseg) *nseg = pl->nseg;
  if (cap) *cap = pl->idx_capacity;
  if (ws) *ws = pl->ws_bytes;
  return FP2_OK;
}

extern "C" void fp2_plan_destroy(fp2_plan* pl) {
  if (!pl) return;
  if (pl->d_table) cudaFree(pl->d_table);
  delete pl;
}

extern "C" fp2_status fp2_plan_segment(const fp2_plan* pl, int64_t seg, int32_t* out10, int64_t* list_offset) {
  if (!pl || !out10 || seg < 0 || seg >= pl->nseg) return FP2_ERR_INVALID_ARG;
  const SegInfo& s = pl->h_segs[(size_t)seg];
  const int32_t v[10] = {s.b, s.h, s.t, s.r0, s.nrows, s.pre, s.Lk, s.J_lo, s.J_hi, s.blk_off};
  memcpy(out10, v, sizeof(v));
  if (list_offset) *list_offset = s.off;
  return FP2_OK;
}

extern "C" fp2_status fp2_plan_set_split(fp2_plan* pl, int32_t target) {
  if (!pl) return FP2_ERR_INVALID_ARG;
  pl->split_target = target;
  return FP2_OK;
}

extern "C" int32_t fp2_last_launch_count(const fp2_plan* pl) { return pl ? pl->last_launches : 0; }

// ------------------------------------------------------------------------------------------------------
// helpers
// ------------------------------------------------------------------------------------------------------
// 3-D map over [rows, heads, 128] elements, box = [box_rows, 1, 64 (bf16) | 128 (fp8)], 128-byte swizzle.
static bool make_map(fp2_plan* pl, CUtensorMap* m, const void* base, int64_t rows, int heads, int box_rows, bool fp8) {
  const int esz = fp8 ? 1 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * esz, (cuuint64_t)kHeadDim * esz * heads};
  cuuint32_t box[3] = {(cuuint32_t)(128 / esz), 1u, (cuuint32_t)box_rows};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = pl->encode(m, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                          const_cast<void*>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Packed query tile as a TMA box (see DevParams::q_tma): [128 bytes, g heads, 128 / g tokens] of q [total_q, Hq, 128]
// -- 64 BF16 elements (the tile takes two boxes) or 128 e4m3 bytes (one box).
static bool make_q_map(fp2_plan* pl, CUtensorMap* m, const void* q, int box_tokens = 0) {
  const int g = pl->dev.group;
  const bool fp8 = pl->dev.fp8;
  const cuuint64_t esz = fp8 ? 1 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)pl->prm.num_q_heads, (cuuint64_t)pl->prm.total_q};
  cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * esz, (cuuint64_t)kHeadDim * esz * pl->prm.num_q_heads};
  cuuint32_t box[3] = {fp8 ? 128u : 64u, (cuuint32_t)g, (cuuint32_t)(box_tokens > 0 ? box_tokens : 128 / g)};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = pl->encode(m, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                          const_cast<void*>(q), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

static fp2_status set_attrs(fp2_plan* pl) {
  if (pl->attrs_set) return FP2_OK;
  if (cudaFuncSetAttribute(score_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes) !=
          cudaSuccess ||
      cudaFuncSetAttribute(score_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kScoreSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(score_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kScoreSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(sparse_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           AttnCfg<false>::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(sparse_attn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           AttnCfg<true>::kSmemBytes) != cudaSuccess)
    return FP2_ERR_CUDA;
  // The attention kernels move registers between warps with setmaxnreg, whose wait is unbounded: launch only
  // if the compiled kernels really own the registers the move assumes.
  cudaFuncAttributes fa;
  if (cudaFuncGetAttributes(&fa, sparse_attn_kernel<false>) != cudaSuccess) return FP2_ERR_CUDA;
  if (fa.numRegs * AttnCfg<false>::kThreads < AttnCfg<false>::kRegsAfterMove) return FP2_ERR_UNSUPPORTED;
  if (cudaFuncGetAttributes(&fa, sparse_attn_kernel<true>) != cudaSuccess) return FP2_ERR_CUDA;
  if (fa.numRegs * AttnCfg<true>::kThreads < AttnCfg<true>::kRegsAfterMove) return FP2_ERR_UNSUPPORTED;
  pl->attrs_set = true;
  return FP2_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static fp2_status check_common(fp2_plan* pl, const void* q, const void* k, const void* v, const int32_t* pt,
                               const int32_t* cu, const int32_t* lk, const float* qs, const float* ks,
                               const float* vs, const void* ws) {
  if (!pl || !q || !k || !v || !pt || !cu || !lk || !ws) return FP2_ERR_INVALID_ARG;
  if (pl->dev.fp8 && (!qs || !ks || !vs)) return FP2_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(ws, 1024)) return FP2_ERR_INVALID_ARG;
  if (pl->device < 0) return FP2_ERR_CUDA;  // plan was made without a device
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != pl->device) return FP2_ERR_INVALID_ARG;
  return set_attrs(pl);
}

static fp2_status launch_pool(fp2_plan* pl, const void* k, const void* v, const int32_t* pt, const int32_t* lk,
                              const float* ks, const float* vs, uint8_t* ws, cudaStream_t st,
                              const int32_t* carry = nullptr) {
  if (pl->nblk_tot == 0) return FP2_OK;
  const unsigned grid = (unsigned)(pl->nblk_tot * pl->prm.num_kv_heads * 2);   // K and V pooled by separate CTAs
  __nv_bfloat16* khi = reinterpret_cast<__nv_bfloat16*>(ws + pl->ws_khi);
  __nv_bfloat16* klo = reinterpret_cast<__nv_bfloat16*>(ws + pl->ws_klo);
  __nv_bfloat16* vb = reinterpret_cast<__nv_bfloat16*>(ws + pl->ws_vbar);
  int* status = reinterpret_cast<int*>(ws + pl->ws_status);
  (void)lk;   // the lengths the kernel uses are the plan's own copy
  // whole cache rows per CTA when a row's 16-byte chunks divide 256 (see pool_rows_kernel), else one head per CTA
  const int row_chunks = pl->prm.num_kv_heads * (pl->dev.fp8 ? 8 : 16);
  if (row_chunks <= 256 && 256 % row_chunks == 0) {
    const unsigned grid_rows = (unsigned)(pl->nblk_tot * 2);
    if (pl->dev.fp8)
      pool_rows_kernel<true><<<grid_rows, 256, 0, st>>>((const uint8_t*)k, (const uint8_t*)v, pt, pl->d_lk, pl->d_blk_off,
                                                        ks, vs, pl->dev, khi, klo, vb, ws + pl->ws_k8hi,
                                                        ws + pl->ws_k8lo, carry, status);
    else
      pool_rows_kernel<false><<<grid_rows, 256, 0, st>>>((const uint8_t*)k, (const uint8_t*)v, pt, pl->d_lk,
                                                         pl->d_blk_off, ks, vs, pl->dev, khi, klo, vb, nullptr, nullptr,
                                                         carry, status);
    pl->last_launches += 1;
    return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
  }
  if (pl->dev.fp8)
    pool_kv_kernel<true><<<grid, 256, 0, st>>>((const uint8_t*)k, (const uint8_t*)v, pt, pl->d_lk, pl->d_blk_off, ks, vs,
                                               pl->dev, khi, klo, vb, ws + pl->ws_k8hi, ws + pl->ws_k8lo, carry, status);
  else
    pool_kv_kernel<false><<<grid, 256, 0, st>>>((const uint8_t*)k, (const uint8_t*)v, pt, pl->d_lk, pl->d_blk_off, ks, vs,
                                                pl->dev, khi, klo, vb, nullptr, nullptr, carry, status);
  pl->last_launches += 1;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

// counting sort of the segments: KV-head-major, descending block count
static fp2_status launch_order(fp2_plan* pl, const int32_t* seg_count, uint8_t* ws, cudaStream_t st) {
  const int nseg = (int)pl->nseg;
  int32_t* hist = reinterpret_cast<int32_t*>(ws + pl->ws_hist);
  int32_t* order = reinterpret_cast<int32_t*>(ws + pl->ws_order);
  const int nb = pl->prm.num_kv_heads * kCountBuckets;
  if (cudaMemsetAsync(hist, 0, sizeof(int32_t) * (size_t)(nb + 1), st) != cudaSuccess) return FP2_ERR_CUDA;
  if (cudaMemsetAsync(ws + pl->ws_counter, 0, 64, st) != cudaSuccess) return FP2_ERR_CUDA;
  const int blocks = (nseg + 255) / 256;
  order_hist_kernel<<<blocks, 256, 0, st>>>(pl->d_segs, seg_count, nseg, hist);
  order_scan_kernel<<<1, 1024, 0, st>>>(hist, nb);
  order_scatter_kernel<<<blocks, 256, 0, st>>>(pl->d_segs, seg_count, nseg, hist, order);
  pl->last_launches += 3;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------
// stage 1
// ------------------------------------------------------------------------------------------------------
extern "C" fp2_status fp2_select_blocks(fp2_plan* pl, const void* q, const void* k, const void* v, const int32_t* pt,
                                        const int32_t* cu, const int32_t* lk, const float* qs, const float* ks,
                                        const float* vs, int64_t* seg_offset, int32_t* seg_count, int32_t* blk_idx,
                                        void* workspace, fp2_stream stream) {
  fp2_status s = check_common(pl, q, k, v, pt, cu, lk, qs, ks, vs, workspace);
  if (s != FP2_OK) return s;
  if (!seg_offset || !seg_count || !blk_idx) return FP2_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  pl->last_launches = 0;
  if (pl->nseg == 0) return FP2_OK;
  // pooled rows carried over by fp2_pool_carry are used once: by this call
  const int32_t* carry = pl->carry_valid ? pl->d_carry : nullptr;
  pl->carry_valid = false;
  if ((s = launch_pool(pl, k, v, pt, lk, ks, vs, ws, st, carry)) != FP2_OK) return s;
  CUtensorMap mhi, mlo;
  if (!make_map(pl, &mhi, ws + pl->ws_khi, pl->nblk_tot, pl->prm.num_kv_heads, 128, false) ||
      !make_map(pl, &mlo, ws + pl->ws_klo, pl->nblk_tot, pl->prm.num_kv_heads, 128, false))
    return FP2_ERR_CUDA;
  CUtensorMap mq = mhi;   // unused unless the scorer takes its query tiles by TMA
  if (pl->dev.fp8 ? (pl->dev.q_raw_tma && !make_q_map(pl, &mq, q, pl->dev.q_box_tok))
                  : (pl->dev.q_tma && !make_q_map(pl, &mq, q)))
    return FP2_ERR_CUDA;
  int* status = reinterpret_cast<int*>(ws + pl->ws_status);
  const unsigned grid = (unsigned)(pl->nseg < pl->num_sms ? pl->nseg : pl->num_sms);
  if (pl->dev.fp8)
    score_select_kernel<true><<<grid, kScoreThreads, kScoreSmemBytes, st>>>(
        mhi, mlo, mq, (const uint8_t*)q, pl->d_segs, qs, pl->dev, seg_offset, seg_count, blk_idx, status);
  else if (pl->dev.q_tma) {
    // BF16 tiles that are TMA boxes: pairs of adjacent tiles per pooled-key chunk.  The pair kernel takes the pooled
    // keys in pieces of 64 elements x 128 keys, which is the box of mhi / mlo already.
    const unsigned grid_pairs = (unsigned)(pl->nunits < pl->num_sms ? pl->nunits : pl->num_sms);
    score_pair_kernel<<<grid_pairs, kPairThreads, kPairSmemBytes, st>>>(mhi, mlo, mq, pl->d_segs, pl->d_units, pl->nunits,
                                                                        pl->dev, seg_offset, seg_count, blk_idx, status);
  } else
    score_select_kernel<false><<<grid, kScoreThreads, kScoreSmemBytes, st>>>(
        mhi, mlo, mq, (const uint8_t*)q, pl->d_segs, qs, pl->dev, seg_offset, seg_count, blk_idx, status);
  pl->last_launches += 1;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

// Block-mean pooling alone (the first kernel of stage 1)
extern "C" fp2_status fp2_pool_blocks(fp2_plan* pl, const void* k, const void* v, const int32_t* pt,
                                      const int32_t* lk, const float* ks, const float* vs, void* workspace,
                                      fp2_stream stream) {
  if (!pl || !k || !v || !pt || !lk || !workspace) return FP2_ERR_INVALID_ARG;
  if (pl->dev.fp8 && (!ks || !vs)) return FP2_ERR_INVALID_ARG;
  if (!aligned(k, 16) || !aligned(v, 16) || !aligned(workspace, 1024)) return FP2_ERR_INVALID_ARG;
  if (pl->device < 0) return FP2_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != pl->device) return FP2_ERR_INVALID_ARG;
  pl->last_launches = 0;
  return launch_pool(pl, k, v, pt, lk, ks, vs, reinterpret_cast<uint8_t*>(workspace),
                     reinterpret_cast<cudaStream_t>(stream));
}

// ------------------------------------------------------------------------------------------------------
// stage 2 (sparse and dense)
// ------------------------------------------------------------------------------------------------------
// Attention: two 256-thread CTAs per SM, each a persistent worker on the shared work counter.  mkb / mkb_lo:
// pooled keys of the correction chunks (BF16: one BF16 array, mkb_lo unused; FP8: e4m3 hi and lo).
#ifdef FP2_PROFILE
static long long* g_prof_ptr = nullptr;
extern "C" void fp2_debug_set_prof(long long* p) { g_prof_ptr = p; }
extern "C" void fp2_debug_set_score_prof(long long* p) { cudaMemcpyToSymbol(fp2::g_score_prof, &p, sizeof(p)); }
#endif

static void launch_attn(fp2_plan* pl, const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mkb,
                        const CUtensorMap& mkb_lo, const CUtensorMap& mvb, const CUtensorMap& mq, const AttnArgs& a,
                        int64_t max_units, cudaStream_t st) {
  const int64_t workers = (int64_t)pl->num_sms * AttnCfg<false>::kCtasPerSm;
  const unsigned grid = (unsigned)(max_units < workers ? max_units : workers);
  if (pl->dev.fp8)
    sparse_attn_kernel<true><<<grid, AttnCfg<true>::kThreads, AttnCfg<true>::kSmemBytes, st>>>(mk, mv, mkb, mkb_lo,
                                                                                                 mvb, mq, a, pl->dev);
  else
    sparse_attn_kernel<false><<<grid, AttnCfg<false>::kThreads, AttnCfg<false>::kSmemBytes, st>>>(
        mk, mv, mkb, mkb_lo, mvb, mq, a, pl->dev);
}

static fp2_status run_attention(fp2_plan* pl, const void* q, const void* k, const void* v, const int32_t* pt,
                                const int32_t* cu, const int32_t* lk, const int32_t* seg_count,
                                const int32_t* blk_idx, const float* qs, const float* ks, const float* vs, void* out,
                                float* lse, void* workspace, bool need_pool, fp2_stream stream) {
  fp2_status s = check_common(pl, q, k, v, pt, cu, lk, qs, ks, vs, workspace);
  if (s != FP2_OK) return s;
  if (!out || !aligned(out, 16)) return FP2_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  pl->last_launches = 0;
  if (pl->nseg == 0) return FP2_OK;
  if (need_pool && (s = launch_pool(pl, k, v, pt, lk, ks, vs, ws, st)) != FP2_OK) return s;
  if ((s = launch_order(pl, seg_count, ws, st)) != FP2_OK) return s;
  const bool fp8 = pl->dev.fp8 != 0;
  const int64_t slots = (int64_t)pl->prm.num_pages * pl->prm.page_size;
  CUtensorMap mk, mv, mkb, mkb_lo, mvb;
  if (!make_map(pl, &mk, k, slots, pl->prm.num_kv_heads, pl->prm.page_size, fp8) ||
      !make_map(pl, &mv, v, slots, pl->prm.num_kv_heads, pl->prm.page_size, fp8) ||
      !make_map(pl, &mvb, ws + pl->ws_vbar, pl->nblk_tot, pl->prm.num_kv_heads, 128, false))
    return FP2_ERR_CUDA;
  if (fp8) {   // correction chunks: pooled keys as an e4m3 hi + lo pair
    if (!make_map(pl, &mkb, ws + pl->ws_k8hi, pl->nblk_tot, pl->prm.num_kv_heads, 128, true) ||
        !make_map(pl, &mkb_lo, ws + pl->ws_k8lo, pl->nblk_tot, pl->prm.num_kv_heads, 128, true))
      return FP2_ERR_CUDA;
  } else {
    if (!make_map(pl, &mkb, ws + pl->ws_khi, pl->nblk_tot, pl->prm.num_kv_heads, 128, false)) return FP2_ERR_CUDA;
    mkb_lo = mkb;
  }
  AttnArgs a;
  a.q = reinterpret_cast<const uint8_t*>(q);
  a.page_table = pt;
  a.segs = pl->d_segs;
  a.order = reinterpret_cast<const int32_t*>(ws + pl->ws_order);
  a.seg_count = seg_count;
  a.blk_idx = blk_idx;
  a.q_scale = qs; a.k_scale = ks; a.v_scale = vs;
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.lse = lse;
  a.work_counter = reinterpret_cast<int*>(ws + pl->ws_counter);
  a.status = reinterpret_cast<int*>(ws + pl->ws_status);
  a.unit_split = nullptr; a.n_units = nullptr; a.part_o = nullptr; a.part_ml = nullptr;
#ifdef FP2_PROFILE
  a.prof = g_prof_ptr;
#endif
  // a part is never shorter than kMinPartLen iterations (or the requested length): nothing to split when even the
  // longest candidate range (plus its correction chunks) is below one and a half such parts
  const int min_len = pl->split_target > 0 ? pl->split_target : kMinPartLen;
  const bool split = pl->split_capable && pl->split_target >= 0 && 2 * pl->max_iters >= 3 * min_len;
  int64_t max_units = pl->nseg;
  if (split) {
    // device-side scheduler prep (Eq. 18): units = parts of segments, in the work order
    int32_t* unit_seg = reinterpret_cast<int32_t*>(ws + pl->ws_unit_seg);
    int32_t* unit_split = reinterpret_cast<int32_t*>(ws + pl->ws_unit_split);
    int32_t* seg_split = reinterpret_cast<int32_t*>(ws + pl->ws_seg_split);
    int32_t* split_list = seg_split + pl->nseg;
    int32_t* n_units = reinterpret_cast<int32_t*>(ws + pl->ws_counter) + 1;
    int32_t* n_split = n_units + 1;
    const int workers = pl->num_sms * AttnCfg<false>::kCtasPerSm;
    split_plan_kernel<<<1, 1024, 0, st>>>(pl->d_segs, a.order, seg_count, (int)pl->nseg, pl->dev.use_correction,
                                          workers, pl->split_target, unit_seg, unit_split, seg_split, split_list, n_units,
                                          n_split);
    pl->last_launches += 1;
    a.order = unit_seg;
    a.unit_split = unit_split;
    a.n_units = n_units;
    a.part_o = reinterpret_cast<float*>(ws + pl->ws_part_o);
    a.part_ml = reinterpret_cast<float2*>(ws + pl->ws_part_ml);
    max_units = pl->split_units_cap;
  }
  CUtensorMap mq = mk;   // unused unless q_tma
  if (pl->dev.q_tma && !make_q_map(pl, &mq, q)) return FP2_ERR_CUDA;
  launch_attn(pl, mk, mv, mkb, mkb_lo, mvb, mq, a, max_units, st);
  pl->last_launches += 1;
  if (split) {
    int32_t* seg_split = reinterpret_cast<int32_t*>(ws + pl->ws_seg_split);
    split_combine_kernel<<<(unsigned)(pl->num_sms * 8), 128, 0, st>>>(
        pl->d_segs, seg_split, seg_split + pl->nseg, reinterpret_cast<int32_t*>(ws + pl->ws_counter) + 2, a.part_o,
        a.part_ml, fp8 ? vs : nullptr, pl->dev, a.out, lse);
    pl->last_launches += 1;
  }
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

extern "C" fp2_status fp2_sparse_prefill(fp2_plan* pl, const void* q, const void* k, const void* v,
                                         const int32_t* pt, const int32_t* cu, const int32_t* lk,
                                         const int64_t* seg_offset, const int32_t* seg_count, const int32_t* blk_idx,
                                         const float* qs, const float* ks, const float* vs, void* out, float* lse,
                                         void* workspace, int32_t pooled_valid, fp2_stream stream) {
  if (!seg_offset || !seg_count || !blk_idx) return FP2_ERR_INVALID_ARG;
  const bool need_pool = pl && pl->dev.use_correction && !pooled_valid;
  return run_attention(pl, q, k, v, pt, cu, lk, seg_count, blk_idx, qs, ks, vs, out, lse, workspace, need_pool,
                       stream);
}

extern "C" fp2_status fp2_dense_prefill(fp2_plan* pl, const void* q, const void* k, const void* v, const int32_t* pt,
                                        const int32_t* cu, const int32_t* lk, const float* qs, const float* ks,
                                        const float* vs, void* out, float* lse, void* workspace, fp2_stream stream) {
  return run_attention(pl, q, k, v, pt, cu, lk, nullptr, nullptr, qs, ks, vs, out, lse, workspace, false, stream);
}

// ------------------------------------------------------------------------------------------------------
// Dense prefill for callers that cannot provide a workspace (see include/fp2.h).  The scratch the dense path
// needs -- status block, work counter, work order, histogram of the counting sort -- lives in a file-scope
// device array instead of caller memory.  Nothing here allocates.
// ------------------------------------------------------------------------------------------------------
constexpr int kStaticMaxSegments = 65536;
constexpr int kStaticMaxKvHeads = 32;
constexpr size_t kStaticOffOrder = 1024;
constexpr size_t kStaticOffHist = kStaticOffOrder + sizeof(int32_t) * kStaticMaxSegments;
constexpr size_t kStaticBytes = kStaticOffHist + sizeof(int32_t) * ((size_t)kStaticMaxKvHeads * kCountBuckets + 256);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// In host code `g_static_scratch` is only a handle; the device address comes from cudaGetSymbolAddress,
// asked once per device with that device current.
constexpr int kMaxDevices = 64;
static unsigned char* g_static_ptr[kMaxDevices];

static fp2_status static_scratch_for(int device, unsigned char** out) {
  if (device < 0 || device >= kMaxDevices) return FP2_ERR_UNSUPPORTED;
  if (!g_static_ptr[device]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return FP2_ERR_CUDA;
    g_static_ptr[device] = reinterpret_cast<unsigned char*>(ptr);
  }
  *out = g_static_ptr[device];
  return FP2_OK;
}

extern "C" fp2_status fp2_dense_prefill_static(fp2_plan* pl, const void* q, const void* k, const void* v,
                                               const int32_t* pt, const int32_t* cu, const int32_t* lk,
                                               const float* qs, const float* ks, const float* vs, void* out,
                                               float* lse, fp2_stream stream) {
  if (!pl || !q || !k || !v || !pt || !cu || !lk || !out) return FP2_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16)) return FP2_ERR_INVALID_ARG;
  if (pl->device < 0) return FP2_ERR_CUDA;
  if (pl->dev.fp8 && (!qs || !ks || !vs)) return FP2_ERR_INVALID_ARG;
  if (pl->nseg > kStaticMaxSegments || pl->prm.num_kv_heads > kStaticMaxKvHeads) return FP2_ERR_CAPACITY;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != pl->device) return FP2_ERR_INVALID_ARG;
  fp2_status s = set_attrs(pl);
  if (s != FP2_OK) return s;
  unsigned char* sw = nullptr;
  if ((s = static_scratch_for(dev, &sw)) != FP2_OK) return s;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  pl->last_launches = 0;
  if (pl->nseg == 0) return FP2_OK;
  const int nseg = (int)pl->nseg;
  int32_t* order = reinterpret_cast<int32_t*>(sw + kStaticOffOrder);
  int32_t* hist = reinterpret_cast<int32_t*>(sw + kStaticOffHist);
  const int nb = pl->prm.num_kv_heads * kCountBuckets;
  // the array keeps the previous call's contents: status, counter and histogram must start at zero
  if (cudaMemsetAsync(sw, 0, 1024, st) != cudaSuccess) return FP2_ERR_CUDA;
  if (cudaMemsetAsync(hist, 0, sizeof(int32_t) * (size_t)(nb + 1), st) != cudaSuccess) return FP2_ERR_CUDA;
  const int blocks = (nseg + 255) / 256;
  order_hist_kernel<<<blocks, 256, 0, st>>>(pl->d_segs, nullptr, nseg, hist);
  order_scan_kernel<<<1, 1024, 0, st>>>(hist, nb);
  order_scatter_kernel<<<blocks, 256, 0, st>>>(pl->d_segs, nullptr, nseg, hist, order);
  const int64_t slots = (int64_t)pl->prm.num_pages * pl->prm.page_size;
  CUtensorMap mk, mv;
  const bool fp8 = pl->dev.fp8 != 0;
  if (!make_map(pl, &mk, k, slots, pl->prm.num_kv_heads, pl->prm.page_size, fp8) ||
      !make_map(pl, &mv, v, slots, pl->prm.num_kv_heads, pl->prm.page_size, fp8))
    return FP2_ERR_CUDA;
  AttnArgs a;
  a.q = reinterpret_cast<const uint8_t*>(q);
  a.page_table = pt;
  a.segs = pl->d_segs;
  a.order = order;
  a.seg_count = nullptr;
  a.blk_idx = nullptr;
  a.q_scale = qs; a.k_scale = ks; a.v_scale = vs;
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.lse = lse;
  a.work_counter = reinterpret_cast<int*>(sw + 64);
  a.status = reinterpret_cast<int*>(sw);
  // the dense path stages no pooled chunks: the two pooled-mean maps are never dereferenced
  a.unit_split = nullptr; a.n_units = nullptr; a.part_o = nullptr; a.part_ml = nullptr;
#ifdef FP2_PROFILE
  a.prof = nullptr;
#endif
  CUtensorMap mq = mk;   // unused unless q_tma
  if (pl->dev.q_tma && !make_q_map(pl, &mq, q)) return FP2_ERR_CUDA;
  launch_attn(pl, mk, mv, mk, mk, mv, mq, a, pl->nseg, st);
  pl->last_launches = 4;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------
// Pooled statistics carried from the previous chunk of a chunked prefill
// ------------------------------------------------------------------------------------------------------
extern "C" fp2_status fp2_pool_carry_count(const fp2_plan* dst, const fp2_plan* src, const int32_t* h_src_seq,
                                           int32_t* h_blocks) {
  if (!dst || !src || !h_src_seq || !h_blocks) return FP2_ERR_INVALID_ARG;
  if (dst->prm.num_kv_heads != src->prm.num_kv_heads || dst->prm.dtype != src->prm.dtype) return FP2_ERR_INVALID_ARG;
  for (int b = 0; b < dst->prm.num_seqs; ++b) {
    const int s = h_src_seq[b];
    if (s >= src->prm.num_seqs) return FP2_ERR_INVALID_ARG;
    // a block's means carry over if the block was complete then and is complete now
    h_blocks[b] = s < 0 ? 0 : std::min(src->h_lk[(size_t)s], dst->h_lk[(size_t)b]) / kBlock;
  }
  return FP2_OK;
}

extern "C" fp2_status fp2_pool_carry(fp2_plan* dst, void* dst_workspace, const fp2_plan* src,
                                     const void* src_workspace, const int32_t* h_src_seq, fp2_stream stream) {
  if (!dst || !src || !dst_workspace || !src_workspace || !h_src_seq) return FP2_ERR_INVALID_ARG;
  if (!aligned(dst_workspace, 1024) || !aligned(src_workspace, 1024)) return FP2_ERR_INVALID_ARG;
  if (dst->device < 0 || src->device != dst->device) return FP2_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != dst->device) return FP2_ERR_INVALID_ARG;
  const int ns = dst->prm.num_seqs;
  dst->h_carry.assign((size_t)3 * (ns > 0 ? ns : 1), 0);
  std::vector<int32_t> n((size_t)(ns > 0 ? ns : 1));
  fp2_status s = fp2_pool_carry_count(dst, src, h_src_seq, n.data());
  if (s != FP2_OK) return s;
  int max_n = 0;
  for (int b = 0; b < ns; ++b) {
    dst->h_carry[3 * b] = h_src_seq[b] < 0 ? 0 : src->h_blk_off[(size_t)h_src_seq[b]];
    dst->h_carry[3 * b + 1] = dst->h_blk_off[(size_t)b];
    dst->h_carry[3 * b + 2] = n[(size_t)b];
    max_n = std::max(max_n, n[(size_t)b]);
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  dst->last_launches = 0;
  if (ns == 0) return FP2_OK;
  // (a pageable host source: the runtime stages the bytes before this call returns)
  if (cudaMemcpyAsync(dst->d_carry, dst->h_carry.data(), sizeof(int32_t) * 3 * ns, cudaMemcpyHostToDevice, st) !=
      cudaSuccess)
    return FP2_ERR_CUDA;
  dst->carry_valid = true;
  if (max_n == 0) return FP2_OK;
  const uint8_t* sw = reinterpret_cast<const uint8_t*>(src_workspace);
  uint8_t* dw = reinterpret_cast<uint8_t*>(dst_workspace);
  const int rb16 = dst->prm.num_kv_heads * kHeadDim * 2;
  const int rb8 = dst->dev.fp8 ? dst->prm.num_kv_heads * kHeadDim : 0;
  const unsigned gy = (unsigned)std::min((max_n + 7) / 8, 1024);
  pool_carry_kernel<<<dim3((unsigned)ns, gy), 256, 0, st>>>(
      dst->d_carry, rb16, rb8, sw + src->ws_khi, sw + src->ws_klo, sw + src->ws_vbar, sw + src->ws_k8hi,
      sw + src->ws_k8lo, dw + dst->ws_khi, dw + dst->ws_klo, dw + dst->ws_vbar, dw + dst->ws_k8hi, dw + dst->ws_k8lo);
  dst->last_launches = 1;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------
// Index export
// ------------------------------------------------------------------------------------------------------
extern "C" fp2_status fp2_export_csr(fp2_plan* pl, const int32_t* seg_count, const int32_t* blk_idx,
                                     int32_t tile_tokens, int32_t* cu, int32_t* idx, int64_t idx_len,
                                     void* workspace, fp2_stream stream) {
  if (!pl || !seg_count || !blk_idx || !cu || !idx || !workspace) return FP2_ERR_INVALID_ARG;
  if (tile_tokens != 16 && tile_tokens != 32 && tile_tokens != 64 && tile_tokens != 128) return FP2_ERR_UNSUPPORTED;
  if (!aligned(workspace, 1024)) return FP2_ERR_INVALID_ARG;
  if (pl->device < 0) return FP2_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != pl->device) return FP2_ERR_INVALID_ARG;
  const int64_t worst = pl->idx_capacity * (kBlock / tile_tokens);
  if (worst > 0x7fffffffll) return FP2_ERR_UNSUPPORTED;   // cu is int32
  if (idx_len < worst) return FP2_ERR_CAPACITY;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int* status = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(workspace) + pl->ws_status);
  const int nseg = (int)pl->nseg;
  pl->last_launches = 0;
  csr_count_kernel<<<(nseg + 256) / 256, 256, 0, st>>>(pl->d_segs, seg_count, blk_idx, nseg, tile_tokens, cu, status);
  pl->last_launches += 1;
  if (nseg > 0) {
    csr_scan_kernel<<<1, 1024, 0, st>>>(cu, nseg);
    csr_fill_kernel<<<(unsigned)(((int64_t)nseg * 32 + 255) / 256), 256, 0, st>>>(pl->d_segs, seg_count, blk_idx, nseg,
                                                                                 tile_tokens, cu, idx, status);
    pl->last_launches += 2;
  }
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

extern "C" fp2_status fp2_page_table_from_token_map(fp2_plan* pl, const int32_t* token_to_slot, int32_t max_tokens,
                                                    const int32_t* seqlens_k, int32_t* page_table, void* workspace,
                                                    fp2_stream stream) {
  if (!pl || !token_to_slot || !seqlens_k || !page_table || !workspace || max_tokens <= 0) return FP2_ERR_INVALID_ARG;
  if (!aligned(workspace, 1024)) return FP2_ERR_INVALID_ARG;
  if (pl->device < 0) return FP2_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != pl->device) return FP2_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int* status = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(workspace) + pl->ws_status);
  const int64_t n = (int64_t)pl->prm.num_seqs * pl->prm.max_pages_per_seq;
  pl->last_launches = 0;
  if (n == 0) return FP2_OK;
  page_table_from_token_map_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
      token_to_slot, max_tokens, seqlens_k, pl->prm.num_seqs, pl->prm.page_size, pl->prm.max_pages_per_seq, page_table,
      status);
  pl->last_launches = 1;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------
// Self-test of the bounded waits: one small CTA that owns tensor memory and waits on a barrier nobody arrives on,
// with a short cycle budget.  The wait gives up by itself, records where, the CTA releases its tensor memory and
// the kernel returns: nothing hangs and nothing traps.
// ------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(64, 1) bounded_wait_probe_kernel(int* status, long long budget_cycles) {
  __shared__ uint64_t never;       // nobody arrives here
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(&never, 1);
    fence_barrier_init();
  }
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, 32);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  WaitCtx ctx{status, &abort_flag, budget_cycles};
  if (warp == 1) mbar_wait(&never, 0, ctx, 901);      // every lane of the warp runs into the budget
  if (warp == 0) mbar_wait(&never, 0, ctx, 902);      // sees the abort flag of the other warp, or its own expiry
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base_s, 32);
}

extern "C" fp2_status fp2_selftest_bounded_wait(fp2_plan* pl, void* workspace, fp2_stream stream) {
  if (!pl || !workspace || !aligned(workspace, 1024)) return FP2_ERR_INVALID_ARG;
  if (pl->device < 0) return FP2_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
  if (dev != pl->device) return FP2_ERR_INVALID_ARG;
  int* status = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(workspace) + pl->ws_status);
  bounded_wait_probe_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(status, 1000000ll);
  pl->last_launches = 1;
  return cudaGetLastError() == cudaSuccess ? FP2_OK : FP2_ERR_CUDA;
}

extern "C" fp2_status fp2_read_status(fp2_plan* pl, void* workspace, int32_t* h_words, fp2_stream stream) {
  if (!pl) return FP2_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int32_t w[ST_WORDS];
  uint8_t* status = nullptr;
  if (workspace) {
    status = reinterpret_cast<uint8_t*>(workspace) + pl->ws_status;
  } else {
    // no workspace: the status block of fp2_dense_prefill_static on the plan's device (the current one)
    if (pl->device < 0) return FP2_ERR_CUDA;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return FP2_ERR_CUDA;
    if (dev != pl->device) return FP2_ERR_INVALID_ARG;
    fp2_status s = static_scratch_for(dev, &status);
    if (s != FP2_OK) return s;
  }
  if (cudaMemcpyAsync(w, status, sizeof(w), cudaMemcpyDeviceToHost, st) != cudaSuccess) return FP2_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FP2_ERR_CUDA;
  if (cudaMemsetAsync(status, 0, sizeof(w), st) != cudaSuccess) return FP2_ERR_CUDA;
  if (h_words) memcpy(h_words, w, sizeof(w));
  if (w[ST_TIMEOUT]) return FP2_ERR_TIMEOUT;
  if (w[ST_BAD_LIST]) return FP2_ERR_INVALID_ARG;
  return FP2_OK;
}
