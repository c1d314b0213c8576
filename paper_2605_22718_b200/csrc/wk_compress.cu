// World Compression (Section 4.3, Eq. 5): score every non-anchor key by its mean cosine similarity to the
// anchor-frame keys, keep the n_keep lowest pooled scores.
//
// The mean over anchors is pulled inside the dot product: s_j = (k_j . m) / |k_j| with
// m = (1/T) sum_i a_i / |a_i|, so a chunk is read exactly once (3T*D bf16) instead of T^2 times.
//
//   anchor_pass   reads the T anchor rows, accumulates m in fp64 (thread-owned columns, rows staged in
//                 shared memory), reduces the per-CTA partials in a fixed order -> m64, m32 = fp32(m64), |m|
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
constexpr int kAnchorRows = 8;      // rows staged per iteration (one per warp)
constexpr int kScoreThreads = 256;
constexpr int kScoreRowsPerCta = 64;
constexpr int kSelectThreads = 1024;

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

// ------------------------------------------------------------------------------------------------
// anchor pass.  grid = (parts, batch).  NP = column pairs owned by each thread = ceil(D / 512).
// ------------------------------------------------------------------------------------------------
template <int NP>
__global__ void __launch_bounds__(kAnchorThreads)
anchor_pass(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int D, int parts,
            double* __restrict__ partial, uint32_t* __restrict__ counters, double* __restrict__ m64,
            float* __restrict__ m32, double* __restrict__ mnorm) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* rows = reinterpret_cast<uint32_t*>(smem);                 // [kAnchorRows][D/2] bf16 pairs
  __shared__ double inv[kAnchorRows];
  __shared__ double red[kAnchorThreads / 32];
  __shared__ uint32_t is_last;
  const int b = blockIdx.y, part = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(b) * stride;
  const int halfD = D >> 1, vecs_per_row = D >> 3;

  double acc0[NP], acc1[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) acc0[i] = acc1[i] = 0.0;

  const int n_blocks = (T + kAnchorRows - 1) / kAnchorRows;
  for (int blk = part; blk < n_blocks; blk += parts) {
    const int r0 = blk * kAnchorRows;
    const int nr = min(kAnchorRows, T - r0);
    // stage nr rows (contiguous in global memory)
    const uint4* src = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(r0) * D);
    uint4* dst = reinterpret_cast<uint4*>(rows);
    for (int v = tid; v < nr * vecs_per_row; v += kAnchorThreads) dst[v] = __ldg(src + v);
    __syncthreads();
    // one warp per row: squared norm in fp64
    if (warp < nr) {
      const uint4* rv = reinterpret_cast<const uint4*>(rows + warp * halfD);
      double n2 = 0.0;
      for (int v = lane; v < vecs_per_row; v += 32) {
        uint4 q = rv[v];
        uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          double x0 = bf16_to_f64(w[e] & 0xFFFFu), x1 = bf16_to_f64(w[e] >> 16);
          n2 = fma(x0, x0, n2);
          n2 = fma(x1, x1, n2);
        }
      }
      n2 = warp_sum(n2);
      if (lane == 0) inv[warp] = n2 > 0.0 ? 1.0 / sqrt(n2) : 0.0;   // a zero key has cosine 0 with everything
    }
    __syncthreads();
    // thread-owned column pairs: acc += row * (1/|row|)
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      const int q = tid + i * kAnchorThreads;
      if (q < halfD) {
        for (int r = 0; r < nr; ++r) {
          const uint32_t w = rows[r * halfD + q];
          const double s = inv[r];
          acc0[i] = fma(bf16_to_f64(w & 0xFFFFu), s, acc0[i]);
          acc1[i] = fma(bf16_to_f64(w >> 16), s, acc1[i]);
        }
      }
    }
    __syncthreads();
  }
  double* my = partial + (static_cast<int64_t>(b) * parts + part) * D;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int q = tid + i * kAnchorThreads;
    if (q < halfD) {
      my[2 * q] = acc0[i];
      my[2 * q + 1] = acc1[i];
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&counters[b], 1u) == static_cast<uint32_t>(parts - 1));
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // the last CTA of this problem adds the partials in a fixed order
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
  if (lane == 0) red[warp] = nn;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < kAnchorThreads / 32; ++w) t += red[w];
    mnorm[b] = sqrt(t);
    counters[b] = 0;   // ready for the next call
  }
}

// Fallback for very wide rows (D > 5120): same arithmetic, accumulators in shared memory.
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
    mnorm[b] = sqrt(t);
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
  float4* m = reinterpret_cast<float4*>(smem);   // [D/4]
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float4* msrc = reinterpret_cast<const float4*>(m32 + static_cast<int64_t>(b) * D);
  for (int i = tid; i < (D >> 2); i += kScoreThreads) m[i] = __ldcg(msrc + i);
  __syncthreads();
  const int vecs = D >> 3;
  const int j0 = blockIdx.x * kScoreRowsPerCta;
  const int j1 = min(NA, j0 + kScoreRowsPerCta);
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(b) * stride + static_cast<int64_t>(T) * D;
  for (int j = j0 + warp; j < j1; j += kScoreThreads / 32) {
    const uint4* row = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(j) * D);
    float dot = 0.f, n2 = 0.f;
    for (int v0 = lane; v0 < vecs; v0 += 128) {
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        q[u] = v < vecs ? __ldg(row + v) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        if (v < vecs) {
          const float4 ma = m[2 * v], mb = m[2 * v + 1];
          float x;
          x = bf16lo(q[u].x); dot = fmaf(x, ma.x, dot); n2 = fmaf(x, x, n2);
          x = bf16hi(q[u].x); dot = fmaf(x, ma.y, dot); n2 = fmaf(x, x, n2);
          x = bf16lo(q[u].y); dot = fmaf(x, ma.z, dot); n2 = fmaf(x, x, n2);
          x = bf16hi(q[u].y); dot = fmaf(x, ma.w, dot); n2 = fmaf(x, x, n2);
          x = bf16lo(q[u].z); dot = fmaf(x, mb.x, dot); n2 = fmaf(x, x, n2);
          x = bf16hi(q[u].z); dot = fmaf(x, mb.y, dot); n2 = fmaf(x, x, n2);
          x = bf16lo(q[u].w); dot = fmaf(x, mb.z, dot); n2 = fmaf(x, x, n2);
          x = bf16hi(q[u].w); dot = fmaf(x, mb.w, dot); n2 = fmaf(x, x, n2);
        }
      }
    }
    dot = warp_sum(dot);
    n2 = warp_sum(n2);
    if (lane == 0) {
      const float s = n2 > 0.f ? __fdiv_rn(dot, __fsqrt_rn(n2)) : 0.f;
      if (!isfinite(s)) atomicOr(status, WK_DEV_NONFINITE);
      s32[static_cast<int64_t>(b) * NA + j] = s;
      if (scores_out) scores_out[static_cast<int64_t>(b) * NA + j] = s;
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

__global__ void __launch_bounds__(kSelectThreads)
select_pass(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int NA, int D, int n_keep,
            const float* __restrict__ s32, const double* __restrict__ m64, const double* __restrict__ mnorm,
            int32_t* __restrict__ keep_idx, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem);                       // [NA]
  int32_t* band_idx = reinterpret_cast<int32_t*>(keys + NA);                // [NA]
  double* band_s = reinterpret_cast<double*>(band_idx + NA);                // [NA] (8-byte aligned: 8*NA)
  uint8_t* flag = reinterpret_cast<uint8_t*>(band_s + NA);                  // [NA]
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sel_prefix, sel_rank, n_band, n_below;
  __shared__ uint32_t warp_tot[kSelectThreads / 32];
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = T + n_keep;
  int32_t* out = keep_idx + static_cast<int64_t>(b) * C;
  for (int i = tid; i < T; i += kSelectThreads) out[i] = i;                 // the anchor frame is kept whole
  if (n_keep == 0) return;
  if (n_keep == NA) {
    for (int j = tid; j < NA; j += kSelectThreads) out[T + j] = T + j;
    return;
  }
  const float* sb = s32 + static_cast<int64_t>(b) * NA;
  for (int j = tid; j < NA; j += kSelectThreads) keys[j] = f32_key(sb[j]);
  if (tid == 0) { sel_prefix = 0; sel_rank = static_cast<uint32_t>(n_keep - 1); n_band = 0; n_below = 0; }
  __syncthreads();
  // radix select: the key of 0-based rank n_keep-1
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = sel_prefix;
    const uint32_t mask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
    for (int j = tid; j < NA; j += kSelectThreads) {
      const uint32_t k = keys[j];
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 0xFFu], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t r = sel_rank, c = 0;
      int bin = 0;
      for (; bin < 256; ++bin) {
        if (c + hist[bin] > r) break;
        c += hist[bin];
      }
      sel_prefix = prefix | (static_cast<uint32_t>(bin) << shift);
      sel_rank = r - c;
    }
    __syncthreads();
  }
  const float theta = key_f32(sel_prefix);
  // fp32 error band.  Per lane: n_l = 8*ceil(D/256) products in a fused chain, then 5 shuffle adds, the rounding of
  // m to fp32, the norm (same chain), one sqrt and one division: |s32 - s| <= (2 n_l + 32) 2^-24 |m|.
  const int n_l = 8 * ((D + 255) / 256);
  const double eps = (2.0 * n_l + 32.0) * 5.9604644775390625e-08 * mnorm[b] * 1.000001;
  const double lo = static_cast<double>(theta) - 2.0 * eps;
  const double hi = static_cast<double>(theta) + 2.0 * eps;
  uint32_t my_below = 0;
  for (int j = tid; j < NA; j += kSelectThreads) {
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
  // exact fp64 scores of the band tokens, one warp per token
  const __nv_bfloat16* Nb = K + static_cast<int64_t>(b) * stride + static_cast<int64_t>(T) * D;
  const double* mb = m64 + static_cast<int64_t>(b) * D;
  for (int t = warp; t < nb; t += kSelectThreads / 32) {
    const uint16_t* row = reinterpret_cast<const uint16_t*>(Nb + static_cast<int64_t>(band_idx[t]) * D);
    double dot = 0.0, n2 = 0.0;
    for (int c = lane; c < D; c += 32) {
      const double x = bf16_to_f64(row[c]);
      dot = fma(x, mb[c], dot);
      n2 = fma(x, x, n2);
    }
    dot = warp_sum(dot);
    n2 = warp_sum(n2);
    if (lane == 0) {
      const double s = n2 > 0.0 ? dot / sqrt(n2) : 0.0;
      if (!isfinite(s)) atomicOr(status, WK_DEV_NONFINITE);
      band_s[t] = s;
    }
  }
  __syncthreads();
  // rank the band tokens by (score, index); the `need` lowest are kept
  for (int t = tid; t < nb; t += kSelectThreads) {
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
  const int per = (NA + kSelectThreads - 1) / kSelectThreads;
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
    uint32_t v = warp_tot[lane];
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

wk_status launch_compress(wk_ctx* ctx, const __nv_bfloat16* K, int64_t stride, int batch, int32_t* keep_idx,
                          float* scores_out, cudaStream_t s) {
  const int T = ctx->cfg.tokens_per_frame, D = ctx->D, NA = ctx->NA, n_keep = ctx->cfg.n_keep;
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
  if (need_scores) {
    const dim3 grid_a(parts, batch);
    const size_t smem_rows = static_cast<size_t>(kAnchorRows) * D * 2;
    const int np = (D + 511) / 512;
#define WK_LAUNCH_ANCHOR(NP)                                                                                         \
  do {                                                                                                               \
    if (smem_rows > 48 * 1024)                                                                                       \
      WK_CUDA_TRY(ctx, cudaFuncSetAttribute(anchor_pass<NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,            \
                                            static_cast<int>(smem_rows)));                                          \
    anchor_pass<NP><<<grid_a, kAnchorThreads, smem_rows, s>>>(K, stride, T, D, parts, partial, counters, m64, m32,   \
                                                              mnorm);                                                \
  } while (0)
    if (np <= 1) WK_LAUNCH_ANCHOR(1);
    else if (np <= 2) WK_LAUNCH_ANCHOR(2);
    else if (np <= 3) WK_LAUNCH_ANCHOR(3);
    else if (np <= 4) WK_LAUNCH_ANCHOR(4);
    else if (np <= 6) WK_LAUNCH_ANCHOR(6);
    else if (np <= 8) WK_LAUNCH_ANCHOR(8);
    else if (np <= 10) WK_LAUNCH_ANCHOR(10);
    else {
      const size_t smem_acc = static_cast<size_t>(D) * sizeof(double);
      if (smem_acc > 200 * 1024) return WK_ERR_SHAPE;
      WK_CUDA_TRY(ctx, cudaFuncSetAttribute(anchor_pass_wide, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(smem_acc)));
      anchor_pass_wide<<<grid_a, kAnchorThreads, smem_acc, s>>>(K, stride, T, D, parts, partial, counters, m64, m32,
                                                                mnorm);
    }
#undef WK_LAUNCH_ANCHOR
    if ((st = after_launch(ctx)) != WK_OK) return st;
    const dim3 grid_s((NA + kScoreRowsPerCta - 1) / kScoreRowsPerCta, batch);
    score_pass<<<grid_s, kScoreThreads, static_cast<size_t>(D) * sizeof(float), s>>>(K, stride, T, NA, D, m32, s32,
                                                                                    scores_out, ctx->status_dev);
    if ((st = after_launch(ctx)) != WK_OK) return st;
  }
  const size_t smem_sel = static_cast<size_t>(NA) * (4 + 4 + 8 + 1) + 16;
  if (smem_sel > 200 * 1024) return WK_ERR_SHAPE;
  if (smem_sel > 48 * 1024)
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(select_pass, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem_sel)));
  select_pass<<<batch, kSelectThreads, smem_sel, s>>>(K, stride, T, NA, D, n_keep, s32, m64, mnorm, keep_idx,
                                                     ctx->status_dev);
  return after_launch(ctx);
}

}  // namespace wk
