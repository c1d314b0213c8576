// C-ABI entry points: argument checks, context, pool bookkeeping (host side), tensor maps.
// Every device-side step lives in the other translation units; nothing here computes.
#include <string.h>

#include <new>

#include "wk_internal.cuh"

namespace wk {

PoolLayout pool_layout(const wk_config& c) {
  PoolLayout p;
  const size_t D = static_cast<size_t>(c.n_heads) * c.head_dim;
  const size_t C = static_cast<size_t>(c.tokens_per_frame) + c.n_keep;
  const size_t kv = align_up(static_cast<size_t>(c.n_layers) * c.pool_slots * C * D * 2, 256);
  p.k_off = 0;
  p.v_off = kv;
  p.pose_off = 2 * kv;
  p.valid_off = p.pose_off + align_up(static_cast<size_t>(c.pool_slots) * 8 * sizeof(float), 256);
  p.status_off = p.valid_off + align_up(static_cast<size_t>(c.pool_slots) * sizeof(int32_t), 256);
  p.total = p.status_off + 256;
  return p;
}

ScratchLayout scratch_layout(const wk_config& c, int max_batch, int max_lq, int max_splits) {
  ScratchLayout s;
  const size_t D = static_cast<size_t>(c.n_heads) * c.head_dim;
  const size_t NA = static_cast<size_t>(c.frames_per_chunk - 1) * c.tokens_per_frame;
  // per-head scoring makes n_heads problems of 128 columns out of every chunk: the column-sized arrays keep their
  // size, the per-problem ones grow by n_heads
  const size_t Bc = static_cast<size_t>(max_batch > 0 ? max_batch : 1);
  const size_t B = Bc * (c.score_mode == WK_SCORE_PER_HEAD ? c.n_heads : 1);
  s.anchor_parts = 32;
  size_t off = 0;
  s.m32_off = off;   off += align_up(Bc * D * sizeof(float), 256);
  s.m64_off = off;   off += align_up(Bc * D * sizeof(double), 256);
  s.s32_off = off;   off += align_up(B * NA * sizeof(float), 256);
  s.mnorm_off = off; off += align_up(B * 32 * sizeof(double), 256);   // up to 32 shares of |m|^2 per problem
  s.part_off = off;  off += align_up(Bc * s.anchor_parts * D * sizeof(double), 256);
  s.inv_off = off;   off += align_up(B * c.tokens_per_frame * sizeof(double), 256);
  s.cnt_off = off;   off += align_up((3 * Bc + 4) * sizeof(uint32_t), 256);   // tickets of the anchor and the score pass, ready words, work queue
  s.dist_off = off;  off += align_up(static_cast<size_t>(c.pool_slots) * 2 * sizeof(double), 256);
  const size_t slots = static_cast<size_t>(attention_partial_slots(c.n_heads, max_lq > 0 ? max_lq : 1, max_splits));
  s.opart_off = off;   off += align_up(slots * 2 * kTileQ * kHeadDim * sizeof(float), 256);
  s.lsepart_off = off; off += align_up(slots * 2 * kTileQ * sizeof(float), 256);
  // query-based retrieval: per-slot log-sum-exp of the query [slot][H][max_lq], identity slot ids, per-block masses
  const size_t lq1 = static_cast<size_t>(max_lq > 0 ? max_lq : 1);
  s.qr_blocks = static_cast<int>((static_cast<size_t>(c.n_heads) * lq1 + 255) / 256);
  s.qr_lse_off = off;  off += align_up(static_cast<size_t>(c.pool_slots) * c.n_heads * lq1 * sizeof(float), 256);
  s.qr_ids_off = off;  off += align_up(static_cast<size_t>(c.pool_slots) * sizeof(int32_t), 256);
  s.qr_part_off = off; off += align_up(static_cast<size_t>(s.qr_blocks) * c.pool_slots * sizeof(double), 256);
  s.total = off;
  return s;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    cudaDriverEntryPointQueryResult qr;
    void* p = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(p);
    }
  }
  return fn;
}

wk_status encode_rows_map(wk_ctx* ctx, const void* base, int64_t rows, int box_rows, CUtensorMap* out) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return cuda_fail(ctx, cudaErrorNotSupported);
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(ctx->D), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ctx->D) * 2};
  cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t es[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    ctx->last_cuda_error = static_cast<int32_t>(r);
    return WK_ERR_CUDA;
  }
  return WK_OK;
}

wk_status encode_pool_map(wk_ctx* ctx, const void* base, int64_t rows, int64_t n_mats, int box_rows, CUtensorMap* out) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return cuda_fail(ctx, cudaErrorNotSupported);
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(ctx->D), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(n_mats)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(ctx->D) * 2, static_cast<cuuint64_t>(ctx->D) * 2 * rows};
  cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    ctx->last_cuda_error = static_cast<int32_t>(r);
    return WK_ERR_CUDA;
  }
  return WK_OK;
}

// Small round-robin cache: steady-state callers pass the same window buffers every step.
const CUtensorMap* cached_rows_map(wk_ctx* ctx, const void* base, int32_t rows, wk_status* st) {
  *st = WK_OK;
  for (auto& e : ctx->tmap_cache) {
    if (e.ptr == base && e.rows == rows) return &e.map;
  }
  TmapKey k;
  k.ptr = base;
  k.rows = rows;
  *st = encode_rows_map(ctx, base, rows, kTileKV, &k.map);
  if (*st != WK_OK) return nullptr;
  const size_t cap = 256;
  if (ctx->tmap_cache.size() < cap) {
    ctx->tmap_cache.push_back(k);
    return &ctx->tmap_cache.back().map;
  }
  size_t i = ctx->tmap_cache_next++ % cap;
  ctx->tmap_cache[i] = k;
  return &ctx->tmap_cache[i].map;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static wk_status check_config(const wk_config* c) {
  if (!c) return WK_ERR_ARG;
  if (c->head_dim != kHeadDim) return WK_ERR_ARG;
  if (c->n_layers < 1 || c->n_heads < 1 || c->tokens_per_frame < 1 || c->frames_per_chunk < 2) return WK_ERR_ARG;
  if (c->n_keep < 0 || c->n_keep > (c->frames_per_chunk - 1) * c->tokens_per_frame) return WK_ERR_ARG;
  if (c->pool_slots < 1 || c->max_k < 0) return WK_ERR_ARG;
  if (c->max_dense_segments < 1 || c->max_dense_segments > kMaxDenseSegs) return WK_ERR_ARG;
  if ((c->score_mode != WK_SCORE_WHOLE_KEY && c->score_mode != WK_SCORE_PER_HEAD) || !(c->softmax_scale >= 0.f))
    return WK_ERR_ARG;
  if (static_cast<int64_t>(c->n_layers) * c->pool_slots > 0x7fffffffLL) return WK_ERR_ARG;
  return WK_OK;
}

// Every entry point that touches the device runs on the context's own device, whatever the caller had current.
static wk_status use_device(wk_ctx* ctx) {
  int dev = -1;
  WK_CUDA_TRY(ctx, cudaGetDevice(&dev));
  if (dev != ctx->cfg.device) WK_CUDA_TRY(ctx, cudaSetDevice(ctx->cfg.device));
  return WK_OK;
}
#define WK_USE_DEVICE(ctx)                                  \
  do {                                                      \
    wk_status st__ = ::wk::use_device(ctx);                 \
    if (st__ != WK_OK) return st__;                         \
  } while (0)

}  // namespace wk

using namespace wk;

extern "C" {

wk_status wk_create(const wk_config* cfg, wk_ctx** out) {
  if (!out) return WK_ERR_ARG;
  *out = nullptr;
  wk_status st = check_config(cfg);
  if (st != WK_OK) return st;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) return WK_ERR_NO_DEVICE;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return WK_ERR_NO_DEVICE;
  if (prop.major != 10) return WK_ERR_NO_DEVICE;  // the kernels are sm_100a only; there is no fallback
  if (cudaSetDevice(cfg->device) != cudaSuccess) return WK_ERR_NO_DEVICE;
  wk_ctx* ctx = new (std::nothrow) wk_ctx();
  if (!ctx) return WK_ERR_ARG;
  ctx->cfg = *cfg;
  ctx->D = cfg->n_heads * cfg->head_dim;
  ctx->C = cfg->tokens_per_frame + cfg->n_keep;
  ctx->FT = cfg->frames_per_chunk * cfg->tokens_per_frame;
  ctx->NA = (cfg->frames_per_chunk - 1) * cfg->tokens_per_frame;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 0.08838834764831845f;  // 1/sqrt(128)
  ctx->slots.resize(cfg->pool_slots);
  for (auto& s : ctx->slots) s.layer_mask.assign(cfg->n_layers, 0);
  ctx->tmap_cache.reserve(256);
  *out = ctx;
  return WK_OK;
}

void wk_destroy(wk_ctx* ctx) { delete ctx; }

size_t wk_pool_bytes(const wk_config* cfg) {
  if (check_config(cfg) != WK_OK) return 0;
  return pool_layout(*cfg).total;
}

size_t wk_scratch_bytes(const wk_config* cfg, int32_t max_batch, int32_t max_lq, int32_t max_splits) {
  if (check_config(cfg) != WK_OK || max_batch < 0 || max_lq < 0 || max_splits < 0) return 0;
  return scratch_layout(*cfg, max_batch, max_lq, max_splits).total;
}

wk_status wk_bind(wk_ctx* ctx, void* pool_dev, size_t pool_bytes, void* scratch_dev, size_t scratch_bytes,
                  int32_t max_batch, int32_t max_lq, int32_t max_splits) {
  if (!ctx || !pool_dev || !scratch_dev) return WK_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(pool_dev) & 255u) || (reinterpret_cast<uintptr_t>(scratch_dev) & 255u)) return WK_ERR_ARG;
  if (max_batch < 0 || max_lq < 0 || max_splits < 0) return WK_ERR_ARG;
  WK_USE_DEVICE(ctx);
  PoolLayout pl = pool_layout(ctx->cfg);
  ScratchLayout sl = scratch_layout(ctx->cfg, max_batch, max_lq, max_splits);
  if (pool_bytes < pl.total || scratch_bytes < sl.total) return WK_ERR_SHAPE;
  ctx->pl = pl;
  ctx->sl = sl;
  ctx->pool_base = static_cast<uint8_t*>(pool_dev);
  ctx->scratch_base = static_cast<uint8_t*>(scratch_dev);
  ctx->Kpool = reinterpret_cast<__nv_bfloat16*>(ctx->pool_base + pl.k_off);
  ctx->Vpool = reinterpret_cast<__nv_bfloat16*>(ctx->pool_base + pl.v_off);
  ctx->poses_dev = reinterpret_cast<float*>(ctx->pool_base + pl.pose_off);
  ctx->valid_dev = reinterpret_cast<int32_t*>(ctx->pool_base + pl.valid_off);
  ctx->status_dev = reinterpret_cast<uint32_t*>(ctx->pool_base + pl.status_off);
  ctx->max_batch = max_batch;
  ctx->max_lq = max_lq;
  ctx->max_splits = max_splits;
  const int64_t n_mats = static_cast<int64_t>(ctx->cfg.n_layers) * ctx->cfg.pool_slots;
  wk_status st = encode_pool_map(ctx, ctx->Kpool, ctx->C, n_mats, kTileKV, &ctx->tm_kpool);
  if (st != WK_OK) return st;
  st = encode_pool_map(ctx, ctx->Vpool, ctx->C, n_mats, kTileKV, &ctx->tm_vpool);
  if (st != WK_OK) return st;
  // the anchor pass counts finished CTAs per problem in scratch; the counters must start at zero
  WK_CUDA_TRY(ctx, cudaMemset(ctx->scratch_base + sl.cnt_off, 0, sl.dist_off - sl.cnt_off));
  {
    std::vector<int32_t> ids(ctx->cfg.pool_slots);
    for (int i = 0; i < ctx->cfg.pool_slots; ++i) ids[i] = i;
    WK_CUDA_TRY(ctx, cudaMemcpy(ctx->scratch_base + sl.qr_ids_off, ids.data(), ids.size() * sizeof(int32_t),
                                cudaMemcpyHostToDevice));
  }
  ctx->bound = true;
  return WK_OK;
}

wk_status wk_compress_chunk(wk_ctx* ctx, const void* K_chunks, int64_t batch_stride_elems, int32_t batch,
                            int32_t* keep_idx_out, float* scores_out, void* stream) {
  if (!ctx || !K_chunks || !keep_idx_out || batch < 0) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (!aligned16(K_chunks) || (batch_stride_elems & 7) != 0) return WK_ERR_ARG;
  if (batch > 1 && batch_stride_elems < static_cast<int64_t>(ctx->FT) * ctx->D) return WK_ERR_ARG;
  if (batch > ctx->max_batch) return WK_ERR_SHAPE;
  if (batch == 0) return WK_OK;
  return launch_compress(ctx, static_cast<const __nv_bfloat16*>(K_chunks), batch_stride_elems, batch, keep_idx_out,
                         scores_out, static_cast<cudaStream_t>(stream));
}

// Shared by wk_pool_append and wk_pool_compress_append: slot choice and bookkeeping around the gather kernel.
static wk_status append_checked(wk_ctx* ctx, int32_t layer0, int32_t n, const void* K_chunks, const void* V_chunks,
                                int64_t batch_stride_elems, const int32_t* keep_idx_dev, const float* pose_host,
                                int64_t chunk_tag, int32_t* slot_io_host, cudaStream_t s, bool after_selection) {
  int slot = *slot_io_host;
  if (slot < 0) {
    if (slot != -1) return WK_ERR_BAD_SLOT;
    for (int i = 0; i < ctx->cfg.pool_slots; ++i) {
      if (ctx->slots[i].state == SLOT_FREE) { slot = i; break; }
    }
    if (slot < 0) return WK_ERR_POOL_FULL;
  } else {
    if (slot >= ctx->cfg.pool_slots || ctx->slots[slot].state != SLOT_OPEN) return WK_ERR_BAD_SLOT;
  }
  SlotInfo& si = ctx->slots[slot];
  for (int l = layer0; l < layer0 + n; ++l) {
    if (si.state == SLOT_OPEN && si.layer_mask[l]) return WK_ERR_BAD_SLOT;  // layer stored twice
  }
  wk_status st = launch_append(ctx, layer0, n, slot, static_cast<const __nv_bfloat16*>(K_chunks),
                               static_cast<const __nv_bfloat16*>(V_chunks), batch_stride_elems, keep_idx_dev, s,
                               after_selection);
  if (st != WK_OK) return st;
  if (si.state == SLOT_FREE) {
    si.state = SLOT_OPEN;
    si.layers_done = 0;
    si.layer_mask.assign(ctx->cfg.n_layers, 0);
    si.tag = chunk_tag;
    memcpy(si.pose, pose_host, sizeof(si.pose));
  }
  for (int l = layer0; l < layer0 + n; ++l) si.layer_mask[l] = 1;
  si.layers_done += n;
  if (si.layers_done == ctx->cfg.n_layers) {
    st = launch_slot_mark(ctx, slot, 1, si.pose, s);
    if (st != WK_OK) return st;
    si.state = SLOT_VALID;
    si.seq = ctx->next_seq++;
  }
  *slot_io_host = slot;
  return WK_OK;
}

wk_status wk_pool_append(wk_ctx* ctx, int32_t layer0, int32_t n, const void* K_chunks, const void* V_chunks,
                         int64_t batch_stride_elems, const int32_t* keep_idx_dev, const float* pose_host,
                         int64_t chunk_tag, int32_t* slot_io_host, void* stream) {
  if (!ctx || !K_chunks || !V_chunks || !keep_idx_dev || !pose_host || !slot_io_host) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (!aligned16(K_chunks) || !aligned16(V_chunks) || (batch_stride_elems & 7) != 0) return WK_ERR_ARG;
  if (layer0 < 0 || n < 1 || layer0 + n > ctx->cfg.n_layers) return WK_ERR_SHAPE;
  if (n > 1 && batch_stride_elems < static_cast<int64_t>(ctx->FT) * ctx->D) return WK_ERR_ARG;
  return append_checked(ctx, layer0, n, K_chunks, V_chunks, batch_stride_elems, keep_idx_dev, pose_host, chunk_tag,
                        slot_io_host, static_cast<cudaStream_t>(stream), false);
}

wk_status wk_pool_compress_append(wk_ctx* ctx, int32_t layer0, int32_t n, const void* K_chunks, const void* V_chunks,
                                  int64_t batch_stride_elems, int32_t* keep_idx_dev, const float* pose_host,
                                  int64_t chunk_tag, int32_t evict_oldest_if_full, int32_t* slot_io_host,
                                  int32_t* evicted_slot_host, void* stream) {
  if (!ctx || !K_chunks || !V_chunks || !keep_idx_dev || !pose_host || !slot_io_host) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (!aligned16(K_chunks) || !aligned16(V_chunks) || (batch_stride_elems & 7) != 0) return WK_ERR_ARG;
  if (layer0 < 0 || n < 1 || layer0 + n > ctx->cfg.n_layers || n > ctx->max_batch) return WK_ERR_SHAPE;
  if (n > 1 && batch_stride_elems < static_cast<int64_t>(ctx->FT) * ctx->D) return WK_ERR_ARG;
  if (evicted_slot_host) *evicted_slot_host = -1;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // everything that can fail on the host is settled before the first launch
  int slot = *slot_io_host;
  if (slot < -1 || slot >= ctx->cfg.pool_slots) return WK_ERR_BAD_SLOT;
  if (slot >= 0) {
    if (ctx->slots[slot].state != SLOT_OPEN) return WK_ERR_BAD_SLOT;
    for (int l = layer0; l < layer0 + n; ++l)
      if (ctx->slots[slot].layer_mask[l]) return WK_ERR_BAD_SLOT;
  } else {
    bool have_free = false;
    for (const auto& si : ctx->slots) have_free = have_free || si.state == SLOT_FREE;
    if (!have_free) {
      const int victim = wk_pool_oldest(ctx);
      if (!evict_oldest_if_full || victim < 0) return WK_ERR_POOL_FULL;
      wk_status st = wk_pool_evict(ctx, victim, stream);
      if (st != WK_OK) return st;
      if (evicted_slot_host) *evicted_slot_host = victim;
    }
  }
  wk_status st = launch_compress(ctx, static_cast<const __nv_bfloat16*>(K_chunks), batch_stride_elems, n, keep_idx_dev,
                                 nullptr, s);
  if (st != WK_OK) return st;
  return append_checked(ctx, layer0, n, K_chunks, V_chunks, batch_stride_elems, keep_idx_dev, pose_host, chunk_tag,
                        slot_io_host, s, true);
}

size_t wk_host_chunk_bytes(const wk_ctx* ctx) {
  if (!ctx) return 0;
  return 2 * static_cast<size_t>(ctx->cfg.n_layers) * ctx->C * ctx->D * sizeof(__nv_bfloat16);
}

wk_status wk_pool_store_host(wk_ctx* ctx, int32_t slot, void* host_dst, void* stream) {
  if (!ctx || !host_dst) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (slot < 0 || slot >= ctx->cfg.pool_slots || ctx->slots[slot].state != SLOT_VALID) return WK_ERR_BAD_SLOT;
  // one layer of one slot is contiguous (C * D elements); the layers of a slot are pool_slots such blocks apart
  const size_t row = static_cast<size_t>(ctx->C) * ctx->D * sizeof(__nv_bfloat16);
  const size_t pitch = row * ctx->cfg.pool_slots;
  const int L = ctx->cfg.n_layers;
  uint8_t* dst = static_cast<uint8_t*>(host_dst);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  WK_CUDA_TRY(ctx, cudaMemcpy2DAsync(dst, row, reinterpret_cast<const uint8_t*>(ctx->Kpool) + slot * row, pitch, row, L,
                                     cudaMemcpyDeviceToHost, s));
  WK_CUDA_TRY(ctx, cudaMemcpy2DAsync(dst + row * L, row, reinterpret_cast<const uint8_t*>(ctx->Vpool) + slot * row, pitch,
                                     row, L, cudaMemcpyDeviceToHost, s));
  return WK_OK;
}

wk_status wk_pool_load_host(wk_ctx* ctx, int32_t layer0, int32_t n, const void* host_src, const float* pose_host,
                            int64_t chunk_tag, int32_t* slot_io_host, void* stream) {
  if (!ctx || !host_src || !pose_host || !slot_io_host) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (layer0 < 0 || n < 1 || layer0 + n > ctx->cfg.n_layers) return WK_ERR_SHAPE;
  int slot = *slot_io_host;
  if (slot < 0) {
    if (slot != -1) return WK_ERR_BAD_SLOT;
    for (int s = 0; s < ctx->cfg.pool_slots; ++s) {
      if (ctx->slots[s].state == SLOT_FREE) { slot = s; break; }
    }
    if (slot < 0) return WK_ERR_POOL_FULL;
  } else {
    if (slot >= ctx->cfg.pool_slots || ctx->slots[slot].state != SLOT_OPEN) return WK_ERR_BAD_SLOT;
  }
  SlotInfo& si = ctx->slots[slot];
  for (int l = layer0; l < layer0 + n; ++l) {
    if (si.state == SLOT_OPEN && si.layer_mask[l]) return WK_ERR_BAD_SLOT;  // layer loaded twice
  }
  const size_t row = static_cast<size_t>(ctx->C) * ctx->D * sizeof(__nv_bfloat16);
  const size_t pitch = row * ctx->cfg.pool_slots;
  const int L = ctx->cfg.n_layers;
  const uint8_t* src = static_cast<const uint8_t*>(host_src);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  WK_CUDA_TRY(ctx, cudaMemcpy2DAsync(reinterpret_cast<uint8_t*>(ctx->Kpool) + layer0 * pitch + slot * row, pitch,
                                     src + layer0 * row, row, row, n, cudaMemcpyHostToDevice, s));
  WK_CUDA_TRY(ctx, cudaMemcpy2DAsync(reinterpret_cast<uint8_t*>(ctx->Vpool) + layer0 * pitch + slot * row, pitch,
                                     src + (static_cast<size_t>(L) + layer0) * row, row, row, n, cudaMemcpyHostToDevice, s));
  if (si.state == SLOT_FREE) {
    si.state = SLOT_OPEN;
    si.layers_done = 0;
    si.layer_mask.assign(ctx->cfg.n_layers, 0);
    si.tag = chunk_tag;
    memcpy(si.pose, pose_host, sizeof(si.pose));
  }
  for (int l = layer0; l < layer0 + n; ++l) si.layer_mask[l] = 1;
  si.layers_done += n;
  if (si.layers_done == ctx->cfg.n_layers) {
    wk_status st = launch_slot_mark(ctx, slot, 1, si.pose, s);
    if (st != WK_OK) return st;
    si.state = SLOT_VALID;
    si.seq = ctx->next_seq++;
  }
  *slot_io_host = slot;
  return WK_OK;
}

wk_status wk_pool_evict(wk_ctx* ctx, int32_t slot, void* stream) {
  if (!ctx) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (slot < 0 || slot >= ctx->cfg.pool_slots || ctx->slots[slot].state != SLOT_VALID) return WK_ERR_BAD_SLOT;
  wk_status st = launch_slot_mark(ctx, slot, 0, ctx->slots[slot].pose, static_cast<cudaStream_t>(stream));
  if (st != WK_OK) return st;
  ctx->slots[slot].state = SLOT_FREE;
  ctx->slots[slot].tag = -1;
  return WK_OK;
}

int32_t wk_pool_oldest(const wk_ctx* ctx) {
  if (!ctx) return -1;
  int best = -1;
  for (int s = 0; s < ctx->cfg.pool_slots; ++s) {
    if (ctx->slots[s].state == SLOT_VALID && (best < 0 || ctx->slots[s].seq < ctx->slots[best].seq)) best = s;
  }
  return best;
}

int32_t wk_pool_count(const wk_ctx* ctx) {
  if (!ctx) return 0;
  int n = 0;
  for (const auto& s : ctx->slots) n += (s.state == SLOT_VALID);
  return n;
}

int64_t wk_pool_tag(const wk_ctx* ctx, int32_t slot) {
  if (!ctx || slot < 0 || slot >= ctx->cfg.pool_slots || ctx->slots[slot].state != SLOT_VALID) return -1;
  return ctx->slots[slot].tag;
}

wk_status wk_retrieve(wk_ctx* ctx, const float* cur_pose_host, int32_t k, int32_t* slots_out_dev, double* dist_out_dev,
                      int32_t* n_out_host, void* stream) {
  if (!ctx || !cur_pose_host || !slots_out_dev || !n_out_host) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (k < 0 || k > ctx->cfg.max_k) return WK_ERR_SHAPE;
  const int M = wk_pool_count(ctx);
  *n_out_host = k < M ? k : M;
  return launch_retrieve(ctx, cur_pose_host, k, slots_out_dev, dist_out_dev, static_cast<cudaStream_t>(stream));
}

size_t wk_retrieve_scan_scratch_bytes(void) { return retrieve_scan_scratch_bytes(); }

wk_status wk_retrieve_scan(wk_ctx* ctx, const float* poses_dev, const int32_t* valid_dev, int64_t n,
                           const float* cur_pose_host, int32_t k, int32_t* ids_out_dev, double* dist_out_dev,
                           int32_t out_capacity, void* scratch_dev, size_t scratch_bytes, void* stream) {
  if (!ctx || !cur_pose_host || !ids_out_dev || !scratch_dev || (n > 0 && !poses_dev)) return WK_ERR_ARG;
  if (!aligned16(poses_dev) || !aligned16(scratch_dev)) return WK_ERR_ARG;
  if (k < 0 || k > 64 || k > out_capacity || n < 0 || n >= (int64_t(1) << 31)) return WK_ERR_SHAPE;
  if (scratch_bytes < retrieve_scan_scratch_bytes()) return WK_ERR_SHAPE;
  WK_USE_DEVICE(ctx);
  return launch_retrieve_scan(ctx, poses_dev, valid_dev, n, cur_pose_host, k, ids_out_dev, dist_out_dev, out_capacity,
                              scratch_dev, static_cast<cudaStream_t>(stream));
}

wk_status wk_retrieve_query(wk_ctx* ctx, int32_t layer, const void* Q, int32_t lq, int32_t k, int32_t* slots_out_dev,
                            float* score_out_dev, int32_t* n_out_host, void* stream) {
  if (!ctx || !Q || !slots_out_dev || !n_out_host || lq < 1) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (!aligned16(Q)) return WK_ERR_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers || lq > ctx->max_lq || k < 0 || k > ctx->cfg.max_k) return WK_ERR_SHAPE;
  if (ctx->cfg.pool_slots > 1024) return WK_ERR_SHAPE;
  const int M = wk_pool_count(ctx);
  *n_out_host = k < M ? k : M;
  return launch_retrieve_query(ctx, layer, static_cast<const __nv_bfloat16*>(Q), lq, k, slots_out_dev, score_out_dev,
                               static_cast<cudaStream_t>(stream));
}

wk_status wk_memory_attention(wk_ctx* ctx, int32_t layer, const void* Q, int32_t lq, const wk_dense_seg* segs_host,
                              int32_t n_segs, const int32_t* slots_dev, int32_t n_slots, void* O, float* lse_out,
                              int32_t kv_splits, void* stream) {
  if (!ctx || !Q || !O || lq < 1 || n_segs < 0 || n_slots < 0) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  if (n_segs == 0 && n_slots == 0) return WK_ERR_ARG;
  if ((n_segs > 0 && !segs_host) || (n_slots > 0 && !slots_dev)) return WK_ERR_ARG;
  if (!aligned16(Q) || !aligned16(O)) return WK_ERR_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers) return WK_ERR_SHAPE;
  if (lq > ctx->max_lq || n_slots > ctx->cfg.max_k || n_segs > ctx->cfg.max_dense_segments) return WK_ERR_SHAPE;
  if (kv_splits > (ctx->max_splits > 1 ? ctx->max_splits : 1)) return WK_ERR_SHAPE;
  for (int i = 0; i < n_segs; ++i) {
    if (!segs_host[i].K || !segs_host[i].V || segs_host[i].n_tokens < 1) return WK_ERR_ARG;
    if (!aligned16(segs_host[i].K) || !aligned16(segs_host[i].V)) return WK_ERR_ARG;
  }
  return launch_attention(ctx, layer, static_cast<const __nv_bfloat16*>(Q), lq, segs_host, n_segs, slots_dev, n_slots,
                          static_cast<__nv_bfloat16*>(O), lse_out, kv_splits, static_cast<cudaStream_t>(stream));
}

wk_status wk_poll_status(wk_ctx* ctx, uint32_t* device_flags, void* stream) {
  if (!ctx) return WK_ERR_ARG;
  if (!ctx->bound) return WK_ERR_UNBOUND;
  WK_USE_DEVICE(ctx);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint32_t flags = 0;
  WK_CUDA_TRY(ctx, cudaMemcpyAsync(&flags, ctx->status_dev, sizeof(flags), cudaMemcpyDeviceToHost, s));
  WK_CUDA_TRY(ctx, cudaMemsetAsync(ctx->status_dev, 0, sizeof(flags), s));
  WK_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  if (device_flags) *device_flags = flags;
  if (flags & WK_DEV_TIMEOUT) return WK_ERR_TIMEOUT;
  if (flags & WK_DEV_NONFINITE) return WK_ERR_NONFINITE;
  if (flags & WK_DEV_BAD_SLOT) return WK_ERR_BAD_SLOT;
  return WK_OK;
}

const char* wk_status_string(wk_status s) {
  switch (s) {
    case WK_OK: return "ok";
    case WK_ERR_ARG: return "bad argument";
    case WK_ERR_SHAPE: return "size outside the context's limits";
    case WK_ERR_POOL_FULL: return "chunk pool is full";
    case WK_ERR_BAD_SLOT: return "slot is not valid";
    case WK_ERR_CUDA: return "CUDA call failed";
    case WK_ERR_TIMEOUT: return "a bounded device wait ran out";
    case WK_ERR_NONFINITE: return "non-finite score";
    case WK_ERR_UNBOUND: return "wk_bind has not been called";
    case WK_ERR_NO_DEVICE: return "no sm_100-class CUDA device";
    default: return "unknown status";
  }
}

int32_t wk_last_cuda_error(const wk_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
int64_t wk_launch_count(const wk_ctx* ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
