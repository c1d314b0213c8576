// Chunk pool (Section 4.2): device side of append (row-gather compaction of K and V into a slot) and of the
// slot table (validity flag + pose).  Slot allocation and FIFO bookkeeping are host side (wk_api.cu).
#include "wk_internal.cuh"

namespace wk {
namespace {

constexpr int kAppendThreads = 256;

// grid = (ceil(C / rows_per_cta), n_layers_in_call, 2 [K|V]); one warp per kept row, 16-byte vectors.  With per-head
// keep-sets (hs = n_heads index lists per layer) every 128-column block of a stored row has its own source token.
__global__ void __launch_bounds__(kAppendThreads)
append_rows(const __nv_bfloat16* __restrict__ Ksrc, const __nv_bfloat16* __restrict__ Vsrc, int64_t stride,
            const int32_t* __restrict__ keep_idx, int hs, int C, int FT, int D, __nv_bfloat16* __restrict__ Kdst,
            __nv_bfloat16* __restrict__ Vdst, int64_t dst_layer_stride, int rows_per_cta, int reverse,
            uint32_t* __restrict__ status) {
  dep_wait();   // returns at once unless the launch was chained to the selection that writes keep_idx
  // reverse: walk the layers last to first, so that the layers whose keys the scoring pass touched last (and L2 still
  // holds) are gathered first
  const int l = reverse ? static_cast<int>(gridDim.y) - 1 - static_cast<int>(blockIdx.y) : static_cast<int>(blockIdx.y);
  const int which = blockIdx.z, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const __nv_bfloat16* src = (which ? Vsrc : Ksrc) + static_cast<int64_t>(l) * stride;
  __nv_bfloat16* dst = (which ? Vdst : Kdst) + static_cast<int64_t>(l) * dst_layer_stride;
  const int32_t* idx = keep_idx + static_cast<int64_t>(l) * hs * C;
  const int vecs = D >> 3, vecs_per_list = vecs / hs;
  const int r0 = blockIdx.x * rows_per_cta, r1 = min(C, r0 + rows_per_cta);
  for (int r = r0 + warp; r < r1; r += kAppendThreads / 32) {
    uint4* d = reinterpret_cast<uint4*>(dst + static_cast<int64_t>(r) * D);
    // four 16-byte loads of the row in flight per lane before the first store
    for (int v0 = lane; v0 < vecs; v0 += 128) {
      uint4 q[4];
      bool ok[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        ok[u] = v < vecs;
        if (ok[u]) {
          const int j = idx[(v / vecs_per_list) * C + r];
          if (j < 0 || j >= FT) {                   // never dereference a bad index
            atomicOr(status, WK_DEV_BAD_SLOT);
            ok[u] = false;
          } else {
            q[u] = __ldg(reinterpret_cast<const uint4*>(src + static_cast<int64_t>(j) * D) + v);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (ok[u]) d[v0 + 32 * u] = q[u];
    }
  }
}

struct Pose8 { float v[8]; };

__global__ void slot_mark(int32_t* __restrict__ valid, float* __restrict__ poses, int slot, int is_valid, Pose8 pose) {
  if (threadIdx.x < 8) poses[slot * 8 + threadIdx.x] = pose.v[threadIdx.x];
  if (threadIdx.x == 0) valid[slot] = is_valid;
}

}  // namespace

wk_status launch_append(wk_ctx* ctx, int layer0, int n, int slot, const __nv_bfloat16* K, const __nv_bfloat16* V,
                        int64_t stride, const int32_t* keep_idx, cudaStream_t s, bool after_selection) {
  const int C = ctx->C, D = ctx->D;
  const int64_t slot_elems = static_cast<int64_t>(C) * D;
  const int64_t layer_stride = slot_elems * ctx->cfg.pool_slots;
  __nv_bfloat16* Kdst = ctx->Kpool + layer0 * layer_stride + slot * slot_elems;
  __nv_bfloat16* Vdst = ctx->Vpool + layer0 * layer_stride + slot * slot_elems;
  const int rows_per_cta = 32;
  const dim3 grid((C + rows_per_cta - 1) / rows_per_cta, n, 2);
  const int hs = ctx->cfg.score_mode == WK_SCORE_PER_HEAD ? ctx->cfg.n_heads : 1;
  if (after_selection)
    launch_chained(append_rows, grid, dim3(kAppendThreads), 0, s, K, V, stride, keep_idx, hs, C, ctx->FT, D, Kdst, Vdst,
                   layer_stride, rows_per_cta, 1, ctx->status_dev);
  else
    append_rows<<<grid, kAppendThreads, 0, s>>>(K, V, stride, keep_idx, hs, C, ctx->FT, D, Kdst, Vdst, layer_stride,
                                                rows_per_cta, 0, ctx->status_dev);
  return after_launch(ctx);
}

wk_status launch_slot_mark(wk_ctx* ctx, int slot, int valid, const float* pose, cudaStream_t s) {
  Pose8 p;
  for (int i = 0; i < 8; ++i) p.v[i] = pose[i];
  slot_mark<<<1, 32, 0, s>>>(ctx->valid_dev, ctx->poses_dev, slot, valid, p);
  return after_launch(ctx);
}

}  // namespace wk
