// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/wk.h"

namespace wk {

constexpr int kHeadDim = 128;
constexpr int kMaxDenseSegs = 8;
constexpr int kTileKV = 128;   // KV rows per attention tile
constexpr int kTileQ = 128;    // Q rows per MMA tile (two per CTA)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct PoolLayout {
  size_t k_off, v_off, pose_off, valid_off, status_off, total;
};
PoolLayout pool_layout(const wk_config& c);

struct ScratchLayout {
  size_t m32_off, m64_off, s32_off, mnorm_off, part_off, inv_off, cnt_off;   // compression
  size_t dist_off;                                                  // retrieval
  size_t opart_off, lsepart_off;                                    // split-KV partials
  size_t qr_lse_off, qr_ids_off, qr_part_off;                       // query-based retrieval
  int qr_blocks;
  size_t total;
  int anchor_parts;  // partial-sum slices per problem written by the anchor pass
};
ScratchLayout scratch_layout(const wk_config& c, int max_batch, int max_lq, int max_splits);

enum SlotState : uint8_t { SLOT_FREE = 0, SLOT_OPEN = 1, SLOT_VALID = 2 };
struct SlotInfo {
  SlotState state = SLOT_FREE;
  int32_t layers_done = 0;
  std::vector<uint8_t> layer_mask;
  int64_t seq = 0;
  int64_t tag = -1;
  float pose[8] = {0, 0, 0, 0, 1, 0, 0, 0};
};

struct TmapKey {
  const void* ptr;
  int32_t rows;
  CUtensorMap map;
};

}  // namespace wk

struct wk_ctx {
  wk_config cfg;
  int D, C, FT, NA;  // row width, rows per stored chunk, rows per chunk, non-anchor rows per chunk
  int sm_count;
  float scale;
  // bound buffers
  bool bound = false;
  uint8_t* pool_base = nullptr;
  uint8_t* scratch_base = nullptr;
  wk::PoolLayout pl;
  wk::ScratchLayout sl;
  int max_batch = 0, max_lq = 0, max_splits = 0;
  __nv_bfloat16* Kpool = nullptr;
  __nv_bfloat16* Vpool = nullptr;
  float* poses_dev = nullptr;
  int32_t* valid_dev = nullptr;
  uint32_t* status_dev = nullptr;
  // host bookkeeping of the pool
  std::vector<wk::SlotInfo> slots;
  int64_t next_seq = 0;
  // tensor maps
  CUtensorMap tm_kpool, tm_vpool;
  std::vector<wk::TmapKey> tmap_cache;
  size_t tmap_cache_next = 0;
  // per-context (hence per-device) one-time kernel attributes: opt-ins to large dynamic shared memory
  bool attn_attr_set = false;
  uint32_t compress_epoch = 0;   // call counter of the one-launch compression: its `ready` words compare against it
  // diagnostics
  int32_t last_cuda_error = 0;
  int64_t launches = 0;
};

namespace wk {

// Records a CUDA error in the context and maps it to WK_ERR_CUDA.
inline wk_status cuda_fail(wk_ctx* ctx, cudaError_t e) {
  ctx->last_cuda_error = static_cast<int32_t>(e);
  return WK_ERR_CUDA;
}
#define WK_CUDA_TRY(ctx, expr)                                 \
  do {                                                         \
    cudaError_t e__ = (expr);                                  \
    if (e__ != cudaSuccess) return ::wk::cuda_fail(ctx, e__);  \
  } while (0)

inline wk_status after_launch(wk_ctx* ctx, int n = 1) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  ctx->launches += n;
  return WK_OK;
}

// Tensor-map helpers (implemented in wk_api.cu).
// rows x D bf16 matrix, box = 64 columns x box_rows rows, 128-byte swizzle, zero fill out of bounds.
wk_status encode_rows_map(wk_ctx* ctx, const void* base, int64_t rows, int box_rows, CUtensorMap* out);
// [n_mats][rows][D] bf16, box = 64 x box_rows x 1.
wk_status encode_pool_map(wk_ctx* ctx, const void* base, int64_t rows, int64_t n_mats, int box_rows, CUtensorMap* out);
const CUtensorMap* cached_rows_map(wk_ctx* ctx, const void* base, int32_t rows, wk_status* st);

// Number of fp32 partial-result slots (256 rows x 128 each) the attention kernel may need.
int attention_partial_slots(int n_heads, int max_lq, int max_splits);

// Kernel launchers (one per translation unit).
wk_status launch_compress(wk_ctx* ctx, const __nv_bfloat16* K, int64_t stride, int batch, int32_t* keep_idx,
                          float* scores_out, cudaStream_t s);
// after_selection: the launch is chained to the selection kernel that writes keep_idx (same stream, issued just before)
// and walks the layers last to first.
wk_status launch_append(wk_ctx* ctx, int layer0, int n, int slot, const __nv_bfloat16* K, const __nv_bfloat16* V,
                        int64_t stride, const int32_t* keep_idx, cudaStream_t s, bool after_selection = false);
wk_status launch_slot_mark(wk_ctx* ctx, int slot, int valid, const float* pose, cudaStream_t s);
wk_status launch_retrieve(wk_ctx* ctx, const float* cur_pose, int k, int32_t* slots_out, double* dist_out, cudaStream_t s);
// Kernels of one call that depend on each other in a chain are launched so that a kernel may be scheduled while its
// predecessor drains (programmatic dependent launch): dep_wait() at the top of a kernel returns once the predecessor
// has completed and its writes are visible; dep_release() lets the successor's launch proceed.  A kernel launched the
// ordinary way after a chained one still waits for its full completion.
#ifdef __CUDACC__
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline void launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // errors surface in after_launch
}
#endif

size_t retrieve_scan_scratch_bytes();
wk_status launch_retrieve_scan(wk_ctx* ctx, const float* poses, const int32_t* valid, int64_t n, const float* cur_pose,
                               int k, int32_t* ids_out, double* dist_out, int out_capacity, void* scratch, cudaStream_t s);
wk_status launch_attention(wk_ctx* ctx, int layer, const __nv_bfloat16* Q, int lq, const wk_dense_seg* segs, int n_segs,
                           const int32_t* slots_dev, int n_slots, __nv_bfloat16* O, float* lse, int kv_splits,
                           cudaStream_t s, bool lse_only = false);
wk_status launch_retrieve_query(wk_ctx* ctx, int layer, const __nv_bfloat16* Q, int lq, int k, int32_t* slots_out,
                                float* score_out, cudaStream_t s);

}  // namespace wk
