// World Retrieval (Section 4.2, Eq. 4) with the camera distance of Section 5.1: squared-L2 translation
// distance and geodesic rotation angle to the current pose, each divided by its maximum over the stored
// chunks, summed; the k smallest win, ties to the lowest slot.  The whole pool is a few KB of poses, so one
// CTA does everything in fp64 in a single launch and the result stays in device memory for the attention call.
#include "wk_internal.cuh"

namespace wk {
namespace {

constexpr int kRetrieveThreads = 1024;

struct Pose8 { float v[8]; };

__device__ __forceinline__ double block_max(double v, double* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  double r = red[0];
  for (int w = 1; w < kRetrieveThreads / 32; ++w) r = fmax(r, red[w]);
  return r;
}

__global__ void __launch_bounds__(kRetrieveThreads)
retrieve_kernel(const float* __restrict__ poses, const int32_t* __restrict__ valid, int n_slots, Pose8 cur, int k,
                int max_k, double* __restrict__ dist /*[2][n_slots]*/, int32_t* __restrict__ slots_out,
                double* __restrict__ dist_out, uint32_t* __restrict__ status /*may be null*/) {
  __shared__ double red[kRetrieveThreads / 32];
  const int tid = threadIdx.x;
  double* dt = dist;
  double* dr = dist + n_slots;
  double mt = 0.0, mr = 0.0;
  for (int s = tid; s < n_slots; s += kRetrieveThreads) {
    if (!valid[s]) { dt[s] = -1.0; continue; }     // negative marks "not a candidate"
    const float* p = poses + s * 8;
    const double dx = static_cast<double>(p[0]) - static_cast<double>(cur.v[0]);
    const double dy = static_cast<double>(p[1]) - static_cast<double>(cur.v[1]);
    const double dz = static_cast<double>(p[2]) - static_cast<double>(cur.v[2]);
    const double t = dx * dx + dy * dy + dz * dz;
    const double dot = static_cast<double>(p[4]) * cur.v[4] + static_cast<double>(p[5]) * cur.v[5] +
                       static_cast<double>(p[6]) * cur.v[6] + static_cast<double>(p[7]) * cur.v[7];
    if (!isfinite(t) || !isfinite(dot)) {          // a NaN/Inf pose (stored or current) is not a candidate
      dt[s] = -1.0;
      if (status) atomicOr(status, WK_DEV_NONFINITE);
      continue;
    }
    const double r = 2.0 * acos(fmin(1.0, fabs(dot)));    // q and -q are the same rotation
    dt[s] = t;
    dr[s] = r;
    mt = fmax(mt, t);
    mr = fmax(mr, r);
  }
  mt = block_max(mt, red);
  mr = block_max(mr, red);
  __syncthreads();
  // combined distance, each term normalised by its maximum over the candidates (a zero maximum drops the term)
  for (int s = tid; s < n_slots; s += kRetrieveThreads) {
    if (dt[s] < 0.0) continue;
    const double a = mt > 0.0 ? dt[s] / mt : 0.0;
    const double b = mr > 0.0 ? dr[s] / mr : 0.0;
    dr[s] = a + b;
  }
  for (int i = tid; i < max_k; i += kRetrieveThreads) {
    slots_out[i] = -1;
    if (dist_out) dist_out[i] = 0.0;
  }
  __syncthreads();
  // rank by counting: position of slot s = number of candidates that precede it under (distance, slot)
  for (int s = tid; s < n_slots; s += kRetrieveThreads) {
    if (dt[s] < 0.0) continue;
    const double d = dr[s];
    int rank = 0;
    for (int u = 0; u < n_slots; ++u) {
      if (dt[u] < 0.0) continue;
      const double du = dr[u];
      rank += (du < d) || (du == d && u < s);
    }
    if (rank < k) {
      slots_out[rank] = s;
      if (dist_out) dist_out[rank] = d;
    }
  }
}

// ---- query-based retrieval (Appendix C) --------------------------------------------------------------------------
// lse[slot][h][r] holds, for every valid slot, the log-sum-exp of query row r of head h over that slot's stored keys.
// The softmax mass of a slot for (h, r) is exp(lse[slot] - logsumexp over slots); a slot's score is the mean mass.
// query_mass: one thread per (h, r); the masses are added over the warp by shuffles, over the block in a fixed order,
// and every block leaves one partial per slot -- no floating-point atomics, so the ranking is reproducible.
constexpr int kMassThreads = 256;

__global__ void __launch_bounds__(kMassThreads)
query_mass(const float* __restrict__ lse, const int32_t* __restrict__ valid, int n_slots, int n_hr,
           double* __restrict__ block_part /*[gridDim.x][n_slots]*/) {
  extern __shared__ float warp_part[];   // [8 warps][n_slots]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int i = blockIdx.x * kMassThreads + tid;
  const bool live = i < n_hr;
  float mx = -INFINITY;
  for (int s = 0; s < n_slots; ++s)
    if (valid[s] && live) mx = fmaxf(mx, lse[static_cast<int64_t>(s) * n_hr + i]);
  float den = 0.f;
  for (int s = 0; s < n_slots; ++s)
    if (valid[s] && live) den += expf(lse[static_cast<int64_t>(s) * n_hr + i] - mx);
  const float inv = (live && den > 0.f) ? 1.f / den : 0.f;
  for (int s = 0; s < n_slots; ++s) {
    float m = 0.f;
    if (valid[s] && live) m = expf(lse[static_cast<int64_t>(s) * n_hr + i] - mx) * inv;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
    if (lane == 0) warp_part[warp * n_slots + s] = m;
  }
  __syncthreads();
  for (int s = tid; s < n_slots; s += kMassThreads) {
    double t = 0.0;
    for (int w = 0; w < kMassThreads / 32; ++w) t += static_cast<double>(warp_part[w * n_slots + s]);
    block_part[static_cast<int64_t>(blockIdx.x) * n_slots + s] = t;
  }
}

// One CTA: adds the blocks' partials in order, ranks the valid slots by (score descending, slot ascending).
__global__ void __launch_bounds__(1024)
query_topk(const double* __restrict__ block_part, int n_blocks, const int32_t* __restrict__ valid, int n_slots, int n_hr,
           int k, int max_k, int32_t* __restrict__ slots_out, float* __restrict__ score_out) {
  __shared__ double score[1024];
  const int tid = threadIdx.x;
  for (int s = tid; s < n_slots; s += 1024) {
    double t = 0.0;
    for (int b = 0; b < n_blocks; ++b) t += block_part[static_cast<int64_t>(b) * n_slots + s];
    score[s] = valid[s] ? t / static_cast<double>(n_hr) : -1.0;   // negative marks "not a candidate"
  }
  for (int i = tid; i < max_k; i += 1024) {
    slots_out[i] = -1;
    if (score_out) score_out[i] = 0.f;
  }
  __syncthreads();
  for (int s = tid; s < n_slots; s += 1024) {
    const double v = score[s];
    if (v < 0.0) continue;
    int rank = 0;
    for (int u = 0; u < n_slots; ++u) {
      const double w = score[u];
      if (w < 0.0) continue;
      rank += (w > v) || (w == v && u < s);
    }
    if (rank < k) {
      slots_out[rank] = s;
      if (score_out) score_out[rank] = static_cast<float>(v);
    }
  }
}

// Scratch of the allocation-free entry point: two doubles per slot, held by every GPU that loads the library.
constexpr int kStaticMaxSlots = 4096;
static __device__ __align__(256) double g_retrieve_scratch[2 * kStaticMaxSlots];

}  // namespace

wk_status launch_retrieve(wk_ctx* ctx, const float* cur_pose, int k, int32_t* slots_out, double* dist_out,
                          cudaStream_t s) {
  Pose8 cur;
  for (int i = 0; i < 8; ++i) cur.v[i] = cur_pose[i];
  double* dist = reinterpret_cast<double*>(ctx->scratch_base + ctx->sl.dist_off);
  retrieve_kernel<<<1, kRetrieveThreads, 0, s>>>(ctx->poses_dev, ctx->valid_dev, ctx->cfg.pool_slots, cur, k,
                                                 ctx->cfg.max_k, dist, slots_out, dist_out, ctx->status_dev);
  return after_launch(ctx);
}

wk_status launch_retrieve_query(wk_ctx* ctx, int layer, const __nv_bfloat16* Q, int lq, int k, int32_t* slots_out,
                                float* score_out, cudaStream_t s) {
  const int H = ctx->cfg.n_heads, S = ctx->cfg.pool_slots, n_hr = H * lq;
  float* lse = reinterpret_cast<float*>(ctx->scratch_base + ctx->sl.qr_lse_off);
  const int32_t* ids = reinterpret_cast<const int32_t*>(ctx->scratch_base + ctx->sl.qr_ids_off);
  double* part = reinterpret_cast<double*>(ctx->scratch_base + ctx->sl.qr_part_off);
  // log-sum-exp of the query over each stored chunk alone: the attention kernel in its LSE-only mode, every pool slot a
  // problem of its own in one launch (slots that hold nothing come back as -inf and are masked by the valid flags)
  wk_status st = launch_attention(ctx, layer, Q, lq, nullptr, 0, ids, S, nullptr, lse, 1, s, true);
  if (st != WK_OK) return st;
  const int blocks = (n_hr + kMassThreads - 1) / kMassThreads;
  query_mass<<<blocks, kMassThreads, static_cast<size_t>(kMassThreads / 32) * S * sizeof(float), s>>>(lse, ctx->valid_dev, S,
                                                                                                     n_hr, part);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  query_topk<<<1, 1024, 0, s>>>(part, blocks, ctx->valid_dev, S, n_hr, k, ctx->cfg.max_k, slots_out, score_out);
  return after_launch(ctx);
}

}  // namespace wk

extern "C" wk_status wk_retrieve_noalloc(const float* poses_dev, const int32_t* valid_dev, int32_t n_slots,
                                         const float* cur_pose_host, int32_t k, int32_t max_k, int32_t* slots_out_dev,
                                         double* dist_out_dev, void* stream) {
  using namespace wk;
  if (!poses_dev || !valid_dev || !cur_pose_host || !slots_out_dev) return WK_ERR_ARG;
  if (n_slots < 0 || k < 0 || max_k < 1 || k > max_k) return WK_ERR_ARG;
  if (n_slots > kStaticMaxSlots) return WK_ERR_SHAPE;   // the built-in scratch holds 4096 slots and cannot grow
  // Set-up, once per device and with that device current: in host code the array's name is only a stand-in, the
  // device address has to be asked for.
  static double* scratch_of_device[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return WK_ERR_NO_DEVICE;
  if (!scratch_of_device[dev]) {
    double* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_retrieve_scratch) != cudaSuccess || !ptr) return WK_ERR_CUDA;
    scratch_of_device[dev] = ptr;
  }
  Pose8 cur;
  for (int i = 0; i < 8; ++i) cur.v[i] = cur_pose_host[i];
  retrieve_kernel<<<1, kRetrieveThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      poses_dev, valid_dev, n_slots, cur, k, max_k, scratch_of_device[dev], slots_out_dev, dist_out_dev, nullptr);
  return cudaGetLastError() == cudaSuccess ? WK_OK : WK_ERR_CUDA;
}
