// World Compression (Section 4.3, Eq. 5): score every non-anchor key by its mean cosine similarity to the
// anchor-frame keys, keep the n_keep lowest pooled scores.
//
// The mean over anchors is pulled inside the dot product: s_j = (k_j . m) / |k_j| with
// m = (1/T) sum_i a_i / |a_i|, so a chunk is read exactly once (3T*D bf16) instead of T^2 times.
//
//   anchor_norms, anchor_accumulate
//                 read the T anchor rows (the second time from L2): fp64 row norms, then m in fp64 with thread-owned
//                 columns; the per-CTA slices are added in a fixed order -> m64, m32 = fp32(m64), |m|
//   score_pass    reads the (F-1)T non-anchor rows once, fp32 dot with the shared-memory-staged m32 and fp32
//                 norm, warp-shuffle reductions -> s32
//   select_pass   per problem: the n_keep-th smallest s32 (radix select) is the threshold; tokens further than
//                 a proved fp32 error band from it are decided at once, the few inside the band are re-scored
//                 in fp64 against m64 and ranked exactly by (score, index); emits the ascending index list
//
// The selection is therefore decided in fp64 wherever fp32 could not decide it, and is reproducible
// run to run (no floating-point atomics anywhere).
#include "wk_internal.cuh"

namespace wk {
namespace {

constexpr int kAnchorThreads = 256;
constexpr int kColSplit = 2;          // column halves per row slice in the fp64 accumulation
constexpr int kMaxNormParts = 32;     // |m|^2 arrives in up to this many per-CTA shares per problem (D <= 16384)
constexpr int kMaxAnchorParts = 16;   // slices per problem in the fp64 accumulation (matches the scratch layout)
constexpr int kScoreThreads = 256;
constexpr int kScoreRowsPerCta = 64;
constexpr int kSelectThreads = 1024;
constexpr int kSelectThreadsHead = 256;   // per-head problems (128 columns)

__device__ __forceinline__ double bf16_to_f64(uint32_t bits16) {
  return static_cast<double>(__uint_as_float(bits16 << 16));
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// The five kernels of one call depend on each other in a chain and are launched with launch_chained (wk_internal.cuh):
// nothing is read or written before dep_wait(), so only launch latency and block scheduling overlap.

// Where the rows of problem b live.  A chunk is [F*T][rs] bf16; with whole-token keys (one keep-set per chunk) a
// problem is a chunk and D = rs; with per-head keys a chunk holds hs = n_heads problems, problem (chunk, h) owning
// columns [h*D, (h+1)*D) of every row, D = head_dim.
// The kernels are instantiated for both cases, so that the whole-key case keeps its plain arithmetic (row pitch = D).
struct RowMap {
  int64_t stride;   // elements between chunks
  int rs;           // elements between token rows
  int hs;           // problems per chunk
  template <bool kPerHead>
  __device__ __forceinline__ const __nv_bfloat16* base(const __nv_bfloat16* K, int b, int D) const {
    if (kPerHead) return K + static_cast<int64_t>(b / hs) * stride + static_cast<int64_t>(b % hs) * D;
    return K + static_cast<int64_t>(b) * stride;
  }
  template <bool kPerHead>
  __device__ __forceinline__ int pitch(int D) const { return kPerHead ? rs : D; }
};

// ------------------------------------------------------------------------------------------------
// anchor pass, two streaming kernels with no block barrier in their loops.
//   anchor_norms:      one warp per anchor row, fp64 squared norm -> 1/|a_i| (0 for a zero key)
//   anchor_accumulate: grid = (parts * kColSplit, batch), block = D/(8 kColSplit) threads; a thread owns 8 columns and adds
//                      a_i[8t..] / |a_i| over the rows of its slice in fp64; the anchor rows come from L2 the second
//                      time.  The last CTA of a problem adds the slices in a fixed order -> m64, m32 = fp32(m64), |m|.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kAnchorThreads)
anchor_norms(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int D, double* __restrict__ inv_norm) {
  dep_release();
  const int b = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * (kAnchorThreads / 32) + warp;
  if (r >= T) return;
  const int vecs = D >> 3;
  const uint4* row = reinterpret_cast<const uint4*>(K + static_cast<int64_t>(b) * stride + static_cast<int64_t>(r) * D);
  double n2a = 0.0, n2b = 0.0;
  for (int v0 = lane; v0 < vecs; v0 += 128) {
    uint4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) q[u] = v0 + 32 * u < vecs ? __ldg(row + v0 + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double x0 = bf16_to_f64(w[e] & 0xFFFFu), x1 = bf16_to_f64(w[e] >> 16);
        n2a = fma(x0, x0, n2a);
        n2b = fma(x1, x1, n2b);
      }
    }
  }
  const double n2 = warp_sum(n2a + n2b);
  if (lane == 0) inv_norm[static_cast<int64_t>(b) * T + r] = n2 > 0.0 ? 1.0 / sqrt(n2) : 0.0;   // zero key: cosine 0
}

// Per-head keys: the same pass over whole rows (all heads of a token are one contiguous row), with the sums taken per
// 128-column block.  A warp covers 256 columns = two heads per step; lanes 0-15 reduce one head, lanes 16-31 the other.
// Problem index of (chunk, head) = chunk * n_heads + head, as everywhere in the per-head path.
__device__ __forceinline__ double half_warp_sum(double v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float half_warp_sum(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(kAnchorThreads)
head_norms(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int D, int H, double* __restrict__ inv_norm) {
  dep_release();
  const int chunk = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * (kAnchorThreads / 32) + warp;
  if (r >= T) return;
  const int vecs = D >> 3;
  const uint4* row = reinterpret_cast<const uint4*>(K + static_cast<int64_t>(chunk) * stride + static_cast<int64_t>(r) * D);
  for (int v0 = lane; v0 - lane < vecs; v0 += 128) {
    uint4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) q[u] = v0 + 32 * u < vecs ? __ldg(row + v0 + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
      double n2a = 0.0, n2b = 0.0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double x0 = bf16_to_f64(w[e] & 0xFFFFu), x1 = bf16_to_f64(w[e] >> 16);
        n2a = fma(x0, x0, n2a);
        n2b = fma(x1, x1, n2b);
      }
      const double n2 = half_warp_sum(n2a + n2b);
      const int head = (v0 + 32 * u) >> 4;
      if ((lane & 15) == 0 && head < H)
        inv_norm[(static_cast<int64_t>(chunk) * H + head) * T + r] = n2 > 0.0 ? 1.0 / sqrt(n2) : 0.0;   // zero key: cosine 0
    }
  }
}

template <bool kPerHead>
__global__ void __launch_bounds__(512)
anchor_accumulate(const __nv_bfloat16* __restrict__ K, RowMap rm, int T, int D, int parts,
                  const double* __restrict__ inv_norm, double* __restrict__ partial) {
  dep_wait();
  dep_release();
  const int b = blockIdx.y, part = blockIdx.x / kColSplit, csplit = blockIdx.x % kColSplit;
  const int tid = threadIdx.x, nthreads = blockDim.x;
  const int vecs = D >> 3;
  const int vec = csplit * nthreads + tid;   // the 16-byte column group this thread owns
  // per-head keys: b is the chunk, the row is the whole token (D = all heads) and the norm is the one of this thread's head
  const uint4* Kb = reinterpret_cast<const uint4*>(K + static_cast<int64_t>(b) * rm.stride);
  const int rsv = D >> 3;   // row pitch in 16-byte vectors
  const double* inv = inv_norm + (kPerHead ? (static_cast<int64_t>(b) * rm.hs + (vec >> 4)) : static_cast<int64_t>(b)) * T;
  if (vec < vecs) {
    double acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0;
    constexpr int U = 8;   // rows in flight per thread
    for (int r0 = part; r0 < T; r0 += U * parts) {
      uint4 q[U];
      double sc[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int r = r0 + u * parts;
        q[u] = r < T ? __ldg(Kb + static_cast<int64_t>(r) * rsv + vec) : make_uint4(0, 0, 0, 0);
        sc[u] = r < T ? __ldg(inv + r) : 0.0;
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          acc[2 * e] = fma(bf16_to_f64(w[e] & 0xFFFFu), sc[u], acc[2 * e]);
          acc[2 * e + 1] = fma(bf16_to_f64(w[e] >> 16), sc[u], acc[2 * e + 1]);
        }
      }
    }
    double* my = partial + (static_cast<int64_t>(b) * parts + part) * D + 8 * vec;
#pragma unroll
    for (int e = 0; e < 8; ++e) my[e] = acc[e];
  }
}

// Adds the row slices of every problem in a fixed order: m64, m32 = fp32(m64) and this CTA's share of |m|^2.
// grid = (ceil(D / 512), batch), 256 threads, two columns per thread; all loads are issued before the first addition.
template <bool kPerHead>
__global__ void __launch_bounds__(256)
anchor_reduce(const double* __restrict__ partial, int T, int D, int parts, int H, double* __restrict__ m64,
              float* __restrict__ m32, double* __restrict__ mnorm2_part) {
  __shared__ double red2[8];
  dep_wait();
  dep_release();
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = 2 * (blockIdx.x * 256 + tid);
  const double* pb = partial + static_cast<int64_t>(b) * parts * D;
  double nn = 0.0;
  if (c < D) {
    double2 v[kMaxAnchorParts];
#pragma unroll
    for (int p = 0; p < kMaxAnchorParts; ++p)
      v[p] = p < parts ? __ldcg(reinterpret_cast<const double2*>(pb + static_cast<int64_t>(p) * D + c)) : make_double2(0.0, 0.0);
    double t0 = 0.0, t1 = 0.0;
#pragma unroll
    for (int p = 0; p < kMaxAnchorParts; ++p) {
      t0 += v[p].x;
      t1 += v[p].y;
    }
    t0 /= static_cast<double>(T);
    t1 /= static_cast<double>(T);
    *reinterpret_cast<double2*>(m64 + static_cast<int64_t>(b) * D + c) = make_double2(t0, t1);
    *reinterpret_cast<float2*>(m32 + static_cast<int64_t>(b) * D + c) = make_float2(static_cast<float>(t0), static_cast<float>(t1));
    nn = fma(t0, t0, fma(t1, t1, 0.0));
  }
  nn = warp_sum(nn);
  if (lane == 0) red2[warp] = nn;
  __syncthreads();
  if (kPerHead) {
    // a warp covers 64 columns: two warps per head, four heads per block; |m_h|^2 is one share per (chunk, head)
    const int head = blockIdx.x * 4 + tid;
    if (tid < 4 && head < H)
      mnorm2_part[(static_cast<int64_t>(b) * H + head) * kMaxNormParts] = red2[2 * tid] + red2[2 * tid + 1];
  } else if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += red2[w];
    mnorm2_part[static_cast<int64_t>(b) * kMaxNormParts + blockIdx.x] = t;
  }
}

// Fallback for very wide rows (D > 8192): same arithmetic, accumulators in shared memory.
__global__ void __launch_bounds__(kAnchorThreads)
anchor_pass_wide(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int D, int parts,
                 double* __restrict__ partial, uint32_t* __restrict__ counters, double* __restrict__ m64,
                 float* __restrict__ m32, double* __restrict__ mnorm) {
  extern __shared__ __align__(16) uint8_t smem[];
  double* acc = reinterpret_cast<double*>(smem);   // [D]
  __shared__ double red[kAnchorThreads / 32];
  __shared__ double inv_s;
  __shared__ uint32_t is_last;
  const int b = blockIdx.y, part = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(b) * stride;
  for (int c = tid; c < D; c += kAnchorThreads) acc[c] = 0.0;
  __syncthreads();
  for (int r = part; r < T; r += parts) {
    const uint16_t* row = reinterpret_cast<const uint16_t*>(Kb + static_cast<int64_t>(r) * D);
    double n2 = 0.0;
    for (int c = tid; c < D; c += kAnchorThreads) {
      double x = bf16_to_f64(row[c]);
      n2 = fma(x, x, n2);
    }
    n2 = warp_sum(n2);
    if (lane == 0) red[warp] = n2;
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      for (int w = 0; w < kAnchorThreads / 32; ++w) t += red[w];
      inv_s = t > 0.0 ? 1.0 / sqrt(t) : 0.0;
    }
    __syncthreads();
    const double s = inv_s;
    for (int c = tid; c < D; c += kAnchorThreads) acc[c] = fma(bf16_to_f64(row[c]), s, acc[c]);
    __syncthreads();
  }
  double* my = partial + (static_cast<int64_t>(b) * parts + part) * D;
  for (int c = tid; c < D; c += kAnchorThreads) my[c] = acc[c];
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&counters[b], 1u) == static_cast<uint32_t>(parts - 1));
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const double* pb = partial + static_cast<int64_t>(b) * parts * D;
  double nn = 0.0;
  for (int c = tid; c < D; c += kAnchorThreads) {
    double s = 0.0;
    for (int p = 0; p < parts; ++p) s += __ldcg(pb + static_cast<int64_t>(p) * D + c);
    s /= static_cast<double>(T);
    m64[static_cast<int64_t>(b) * D + c] = s;
    m32[static_cast<int64_t>(b) * D + c] = static_cast<float>(s);
    nn = fma(s, s, nn);
  }
  nn = warp_sum(nn);
  __syncthreads();
  if (lane == 0) red[warp] = nn;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < kAnchorThreads / 32; ++w) t += red[w];
    mnorm[static_cast<int64_t>(b) * kMaxNormParts] = t;   // |m|^2, a single share
    counters[b] = 0;
  }
}

// ------------------------------------------------------------------------------------------------
// score pass.  grid = (ceil(NA / kScoreRowsPerCta), batch); one warp per row; m32 staged in shared memory.
// Per lane the fp32 accumulation is a chain of 8 * ceil(D/256) fused multiply-adds followed by five
// shuffle additions; select_pass derives its error band from exactly this order.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kScoreThreads)
score_pass(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int NA, int D,
           const float* __restrict__ m32, float* __restrict__ s32, float* __restrict__ scores_out,
           uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  dep_wait();
  dep_release();
  float4* m = reinterpret_cast<float4*>(smem);   // [D/4]
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float4* msrc = reinterpret_cast<const float4*>(m32 + static_cast<int64_t>(b) * D);
  for (int i = tid; i < (D >> 2); i += kScoreThreads) m[i] = __ldcg(msrc + i);
  __syncthreads();
  const int vecs = D >> 3;
  const int j0 = blockIdx.x * kScoreRowsPerCta;
  const int j1 = min(NA, j0 + kScoreRowsPerCta);
  const int pitch = D;
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(b) * stride + static_cast<int64_t>(T) * pitch;
  // two rows per warp at a time, so that twice as many 16-byte loads are in flight
  constexpr int W = kScoreThreads / 32;
  for (int j = j0 + warp; j < j1; j += 2 * W) {
    const int jb = j + W;
    const bool has_b = jb < j1;
    const uint4* row_a = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(j) * pitch);
    const uint4* row_b = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(has_b ? jb : j) * pitch);
    float dot_a = 0.f, n2_a = 0.f, dot_b = 0.f, n2_b = 0.f;
    for (int v0 = lane; v0 < vecs; v0 += 128) {
      uint4 qa[4], qb[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        qa[u] = v < vecs ? __ldg(row_a + v) : make_uint4(0, 0, 0, 0);
        qb[u] = v < vecs ? __ldg(row_b + v) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        if (v < vecs) {
          const float4 ma = m[2 * v], mb = m[2 * v + 1];
          const float mm[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
          const uint32_t wa[4] = {qa[u].x, qa[u].y, qa[u].z, qa[u].w}, wb[4] = {qb[u].x, qb[u].y, qb[u].z, qb[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float x;
            x = bf16lo(wa[e]); dot_a = fmaf(x, mm[2 * e], dot_a); n2_a = fmaf(x, x, n2_a);
            x = bf16hi(wa[e]); dot_a = fmaf(x, mm[2 * e + 1], dot_a); n2_a = fmaf(x, x, n2_a);
            x = bf16lo(wb[e]); dot_b = fmaf(x, mm[2 * e], dot_b); n2_b = fmaf(x, x, n2_b);
            x = bf16hi(wb[e]); dot_b = fmaf(x, mm[2 * e + 1], dot_b); n2_b = fmaf(x, x, n2_b);
          }
        }
      }
    }
    dot_a = warp_sum(dot_a);
    n2_a = warp_sum(n2_a);
    dot_b = warp_sum(dot_b);
    n2_b = warp_sum(n2_b);
    if (lane < 2 && (lane == 0 || has_b)) {
      const float dot = lane ? dot_b : dot_a, n2 = lane ? n2_b : n2_a;
      const int jj = lane ? jb : j;
      const float sc = n2 == 0.f ? 0.f : __fdiv_rn(dot, __fsqrt_rn(n2));   // a NaN norm stays NaN and is reported
      if (!isfinite(sc)) atomicOr(status, WK_DEV_NONFINITE);
      s32[static_cast<int64_t>(b) * NA + jj] = sc;
      if (scores_out) scores_out[static_cast<int64_t>(b) * NA + jj] = sc;
    }
  }
}

// Per-head keys: whole rows again, the dot product and the squared norm taken per 128-column block (lanes 0-15 / 16-31
// of a 256-column step).  Per lane and head: 8 fused multiply-adds, then 4 shuffle additions -- inside the error band
// select_pass derives for D = 128.
__global__ void __launch_bounds__(kScoreThreads)
head_score(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int NA, int D, int H, const float* __restrict__ m32,
           float* __restrict__ s32, float* __restrict__ scores_out, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  dep_wait();
  dep_release();
  float4* m = reinterpret_cast<float4*>(smem);   // [D/4]: the heads' mean unit anchors, side by side
  const int chunk = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float4* msrc = reinterpret_cast<const float4*>(m32 + static_cast<int64_t>(chunk) * D);
  for (int i = tid; i < (D >> 2); i += kScoreThreads) m[i] = __ldcg(msrc + i);
  __syncthreads();
  const int vecs = D >> 3;
  const int j0 = blockIdx.x * kScoreRowsPerCta;
  const int j1 = min(NA, j0 + kScoreRowsPerCta);
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(chunk) * stride + static_cast<int64_t>(T) * D;
  constexpr int W = kScoreThreads / 32;
  for (int j = j0 + warp; j < j1; j += W) {
    const uint4* row = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(j) * D);
    for (int v0 = lane; v0 - lane < vecs; v0 += 128) {
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) q[u] = v0 + 32 * u < vecs ? __ldg(row + v0 + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        float dot = 0.f, n2 = 0.f;
        if (v < vecs) {
          const float4 ma = m[2 * v], mb = m[2 * v + 1];
          const float mm[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
          const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float x;
            x = bf16lo(w[e]); dot = fmaf(x, mm[2 * e], dot); n2 = fmaf(x, x, n2);
            x = bf16hi(w[e]); dot = fmaf(x, mm[2 * e + 1], dot); n2 = fmaf(x, x, n2);
          }
        }
        dot = half_warp_sum(dot);
        n2 = half_warp_sum(n2);
        const int head = v >> 4;
        if ((lane & 15) == 0 && head < H) {
          const float sc = n2 == 0.f ? 0.f : __fdiv_rn(dot, __fsqrt_rn(n2));   // a NaN norm stays NaN and is reported
          if (!isfinite(sc)) atomicOr(status, WK_DEV_NONFINITE);
          const int64_t at = (static_cast<int64_t>(chunk) * H + head) * NA + j;
          s32[at] = sc;
          if (scores_out) scores_out[at] = sc;
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// select pass.  One CTA per problem.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t f32_key(float f) {   // order-preserving map float -> uint32
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_f32(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

template <bool kPerHead>
__global__ void __launch_bounds__(kPerHead ? kSelectThreadsHead : kSelectThreads)
select_pass(const __nv_bfloat16* __restrict__ K, RowMap rm, int T, int NA, int D, int n_keep,
            const float* __restrict__ s32, const double* __restrict__ m64, const double* __restrict__ mnorm,
            int n_norm_parts, int32_t* __restrict__ keep_idx, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  // a problem of 128 columns has little to do in the refinement: a quarter of the threads, four problems per SM at once
  constexpr int kThr = kPerHead ? kSelectThreadsHead : kSelectThreads;
  dep_wait();
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem);                       // [NA]
  int32_t* band_idx = reinterpret_cast<int32_t*>(keys + NA);                // [NA]
  double* band_s = reinterpret_cast<double*>(band_idx + NA);                // [NA] (8-byte aligned: 8*NA)
  uint8_t* flag = reinterpret_cast<uint8_t*>(band_s + NA);                  // [NA]
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sel_prefix, sel_rank, n_band, n_below;
  __shared__ uint32_t warp_tot[32];
  __shared__ double band_red[8][kThr / 32];
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = T + n_keep;
  int32_t* out = keep_idx + static_cast<int64_t>(b) * C;
  for (int i = tid; i < T; i += kThr) out[i] = i;                 // the anchor frame is kept whole
  if (n_keep == 0) return;
  if (n_keep == NA) {
    for (int j = tid; j < NA; j += kThr) out[T + j] = T + j;
    return;
  }
  const float* sb = s32 + static_cast<int64_t>(b) * NA;
  for (int j = tid; j < NA; j += kThr) keys[j] = f32_key(sb[j]);
  if (tid == 0) { sel_prefix = 0; sel_rank = static_cast<uint32_t>(n_keep - 1); n_band = 0; n_below = 0; }
  __syncthreads();
  // radix select: the key of 0-based rank n_keep-1
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = sel_prefix;
    const uint32_t mask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
    for (int j = tid; j < NA; j += kThr) {
      const uint32_t k = keys[j];
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 0xFFu], 1u);
    }
    __syncthreads();
    if (warp == 0) {
      // find the bin in which the cumulative count passes the wanted rank: 8 bins per lane, then a warp scan
      uint32_t h[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { h[i] = hist[lane * 8 + i]; tot += h[i]; }
      uint32_t incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const uint32_t r = sel_rank;
      uint32_t c = incl - tot;                 // count in the bins of lower lanes
      if (c <= r && r < incl) {                 // exactly one lane holds the crossing
        int bin = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (c + h[i] <= r) { c += h[i]; bin = i + 1; }
          else break;
        }
        sel_prefix = prefix | (static_cast<uint32_t>(lane * 8 + bin) << shift);
        sel_rank = r - c;
      }
    }
    __syncthreads();
  }
  const float theta = key_f32(sel_prefix);
  // fp32 error band.  Per lane: n_l = 8*ceil(D/256) products in a fused chain, then 5 shuffle adds, the rounding of
  // m to fp32, the norm (same chain), one sqrt and one division: |s32 - s| <= (2 n_l + 32) 2^-24 |m|.
  const int n_l = 8 * ((D + 255) / 256);
  double mn2 = 0.0;
  for (int i = 0; i < n_norm_parts; ++i) mn2 += mnorm[static_cast<int64_t>(b) * kMaxNormParts + i];
  const double eps = (2.0 * n_l + 32.0) * 5.9604644775390625e-08 * sqrt(mn2) * 1.000001;
  const double lo = static_cast<double>(theta) - 2.0 * eps;
  const double hi = static_cast<double>(theta) + 2.0 * eps;
  uint32_t my_below = 0;
  for (int j = tid; j < NA; j += kThr) {
    const double s = static_cast<double>(key_f32(keys[j]));
    uint8_t f = 0;
    if (s < lo) { f = 1; ++my_below; }
    else if (s <= hi) { const uint32_t p = atomicAdd(&n_band, 1u); band_idx[p] = j; }
    flag[j] = f;
  }
  my_below = __reduce_add_sync(0xffffffffu, my_below);
  if (lane == 0 && my_below) atomicAdd(&n_below, my_below);
  __syncthreads();
  const int nb = static_cast<int>(n_band);
  const int need = n_keep - static_cast<int>(n_below);   // >= 1: the threshold token itself is in the band
  // exact fp64 scores of the band tokens: the whole CTA works on four tokens at a time (thread = one 16-byte vector
  // of the row), partial sums meet in shared memory and are added in a fixed order
  const int pitch = rm.pitch<kPerHead>(D);
  const __nv_bfloat16* Nb = rm.base<kPerHead>(K, b, D) + static_cast<int64_t>(T) * pitch;
  const double* mb = m64 + static_cast<int64_t>(b) * D;
  const int vecs = D >> 3;
  for (int t0 = 0; t0 < nb; t0 += 4) {
    double dot[4] = {0.0, 0.0, 0.0, 0.0}, n2[4] = {0.0, 0.0, 0.0, 0.0};
    for (int v = tid; v < vecs; v += kThr) {
      double mv[8];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double2 d2 = __ldcg(reinterpret_cast<const double2*>(mb + 8 * v) + e);
        mv[2 * e] = d2.x;
        mv[2 * e + 1] = d2.y;
      }
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        q[u] = t0 + u < nb ? __ldg(reinterpret_cast<const uint4*>(Nb + static_cast<int64_t>(band_idx[t0 + u]) * pitch) + v)
                           : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const double x0 = bf16_to_f64(w[e] & 0xFFFFu), x1 = bf16_to_f64(w[e] >> 16);
          dot[u] = fma(x0, mv[2 * e], dot[u]);
          dot[u] = fma(x1, mv[2 * e + 1], dot[u]);
          n2[u] = fma(x0, x0, n2[u]);
          n2[u] = fma(x1, x1, n2[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      dot[u] = warp_sum(dot[u]);
      n2[u] = warp_sum(n2[u]);
      if (lane == 0) {
        band_red[2 * u][warp] = dot[u];
        band_red[2 * u + 1][warp] = n2[u];
      }
    }
    __syncthreads();
    if (tid < 4 && t0 + tid < nb) {
      double d = 0.0, n = 0.0;
      for (int w = 0; w < kThr / 32; ++w) {
        d += band_red[2 * tid][w];
        n += band_red[2 * tid + 1][w];
      }
      const double sc = n == 0.0 ? 0.0 : d / sqrt(n);
      if (!isfinite(sc)) atomicOr(status, WK_DEV_NONFINITE);
      band_s[t0 + tid] = sc;
    }
    __syncthreads();
  }
  // rank the band tokens by (score, index); the `need` lowest are kept
  for (int t = tid; t < nb; t += kThr) {
    const double s = band_s[t];
    const int idx = band_idx[t];
    int rank = 0;
    for (int u = 0; u < nb; ++u) {
      const double su = band_s[u];
      rank += (su < s) || (su == s && band_idx[u] < idx);
    }
    if (rank < need) flag[idx] = 1;
  }
  __syncthreads();
  // ordered compaction of the kept indices
  const int per = (NA + kThr - 1) / kThr;
  const int a0 = min(NA, tid * per), a1 = min(NA, a0 + per);
  uint32_t cnt = 0;
  for (int j = a0; j < a1; ++j) cnt += flag[j];
  uint32_t incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    uint32_t v = lane < kThr / 32 ? warp_tot[lane] : 0u;
    uint32_t inc2 = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t w = __shfl_up_sync(0xffffffffu, inc2, o);
      if (lane >= o) inc2 += w;
    }
    warp_tot[lane] = inc2 - v;   // exclusive
  }
  __syncthreads();
  uint32_t pos = warp_tot[warp] + incl - cnt;
  for (int j = a0; j < a1; ++j) {
    if (flag[j]) out[T + pos++] = T + j;
  }
}

}  // namespace

wk_status launch_compress(wk_ctx* ctx, const __nv_bfloat16* K, int64_t stride, int chunks, int32_t* keep_idx,
                          float* scores_out, cudaStream_t s) {
  const int T = ctx->cfg.tokens_per_frame, NA = ctx->NA, n_keep = ctx->cfg.n_keep;
  // whole-token keys: one problem per chunk, D columns; per-head keys: n_heads problems per chunk, 128 columns each.
  // The streaming kernels walk whole rows either way (DF columns); only the selection sees (chunk, head) problems.
  const bool per_head = ctx->cfg.score_mode == WK_SCORE_PER_HEAD;
  const int H = ctx->cfg.n_heads, DF = ctx->D;
  const int D = per_head ? kHeadDim : DF;
  const int batch = per_head ? chunks * H : chunks;
  const RowMap rm{stride, DF, per_head ? H : 1};
  uint8_t* sc = ctx->scratch_base;
  float* m32 = reinterpret_cast<float*>(sc + ctx->sl.m32_off);
  double* m64 = reinterpret_cast<double*>(sc + ctx->sl.m64_off);
  float* s32 = reinterpret_cast<float*>(sc + ctx->sl.s32_off);
  double* mnorm = reinterpret_cast<double*>(sc + ctx->sl.mnorm_off);
  double* partial = reinterpret_cast<double*>(sc + ctx->sl.part_off);
  uint32_t* counters = reinterpret_cast<uint32_t*>(sc + ctx->sl.cnt_off);
  const int parts = ctx->sl.anchor_parts;
  const bool need_scores = (n_keep > 0 && n_keep < NA) || scores_out != nullptr;
  wk_status st = WK_OK;
  int n_norm_parts = 1;
  if (need_scores) {
    if (DF <= 8192) {
      n_norm_parts = per_head ? 1 : (DF + 511) / 512;
      double* inv_norm = reinterpret_cast<double*>(sc + ctx->sl.inv_off);
      const dim3 grid_n((T + kAnchorThreads / 32 - 1) / (kAnchorThreads / 32), chunks);
      if (per_head) head_norms<<<grid_n, kAnchorThreads, 0, s>>>(K, stride, T, DF, H, inv_norm);
      else anchor_norms<<<grid_n, kAnchorThreads, 0, s>>>(K, stride, T, DF, inv_norm);
      if ((st = after_launch(ctx)) != WK_OK) return st;
      const int threads = ((DF / 8 + kColSplit * 32 - 1) / (kColSplit * 32)) * 32;
      const dim3 grid_acc(parts * kColSplit, chunks);
      if (per_head) launch_chained(anchor_accumulate<true>, grid_acc, dim3(threads), 0, s, K, rm, T, DF, parts, inv_norm, partial);
      else launch_chained(anchor_accumulate<false>, grid_acc, dim3(threads), 0, s, K, rm, T, DF, parts, inv_norm, partial);
      if ((st = after_launch(ctx)) != WK_OK) return st;
      const dim3 grid_r((DF + 511) / 512, chunks);
      if (per_head) launch_chained(anchor_reduce<true>, grid_r, dim3(256), 0, s, partial, T, DF, parts, H, m64, m32, mnorm);
      else launch_chained(anchor_reduce<false>, grid_r, dim3(256), 0, s, partial, T, DF, parts, H, m64, m32, mnorm);
    } else {
      if (per_head) return WK_ERR_SHAPE;   // rows wider than 8,192 columns take the whole-key fallback only
      const dim3 grid_a(parts, chunks);
      const size_t smem_acc = static_cast<size_t>(DF) * sizeof(double);
      if (smem_acc > 200 * 1024) return WK_ERR_SHAPE;
      WK_CUDA_TRY(ctx, cudaFuncSetAttribute(anchor_pass_wide, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(smem_acc)));
      anchor_pass_wide<<<grid_a, kAnchorThreads, smem_acc, s>>>(K, stride, T, DF, parts, partial, counters, m64, m32,
                                                                mnorm);
    }
    if ((st = after_launch(ctx)) != WK_OK) return st;
    const dim3 grid_s((NA + kScoreRowsPerCta - 1) / kScoreRowsPerCta, chunks);
    const size_t smem_m = static_cast<size_t>(DF) * sizeof(float);
    if (per_head)
      launch_chained(head_score, grid_s, dim3(kScoreThreads), smem_m, s, K, stride, T, NA, DF, H, m32, s32, scores_out,
                     ctx->status_dev);
    else
      launch_chained(score_pass, grid_s, dim3(kScoreThreads), smem_m, s, K, stride, T, NA, DF, m32, s32, scores_out,
                     ctx->status_dev);
    if ((st = after_launch(ctx)) != WK_OK) return st;
  }
  const size_t smem_sel = static_cast<size_t>(NA) * (4 + 4 + 8 + 1) + 16;
  if (smem_sel > 200 * 1024) return WK_ERR_SHAPE;
  if (smem_sel > 48 * 1024) {
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(select_pass<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem_sel)));
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(select_pass<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem_sel)));
  }
  if (per_head)
    launch_chained(select_pass<true>, dim3(batch), dim3(kSelectThreadsHead), smem_sel, s, K, rm, T, NA, D, n_keep, s32, m64, mnorm,
                   n_norm_parts, keep_idx, ctx->status_dev);
  else
    launch_chained(select_pass<false>, dim3(batch), dim3(kSelectThreads), smem_sel, s, K, rm, T, NA, D, n_keep, s32, m64, mnorm,
                   n_norm_parts, keep_idx, ctx->status_dev);
  return after_launch(ctx);
}

}  // namespace wk
