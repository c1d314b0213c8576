// World Compression (Section 4.3, Eq. 5): score every non-anchor key by its mean cosine similarity to the
// anchor-frame keys, keep the n_keep lowest pooled scores.
//
// The mean over anchors is pulled inside the dot product: s_j = (k_j . m) / |k_j| with
// m = (1/T) sum_i a_i / |a_i|, so a chunk is read exactly once (3T*D bf16) instead of T^2 times.
//
//   anchor_rows   reads the T anchor rows once.  A row is shared by a set of warps; each lane converts its share to fp64
//                 once and keeps it in registers: fp64 squared norm (warp sum, plus an exchange between the set's warps),
//                 then a_i / |a_i| is added to the lane's own fp64 column sums.  Every CTA takes an equal run of the
//                 rows of all chunks and hands in one slice of column sums per chunk it touches; the last CTA of a
//                 chunk (atomic ticket, nobody waits) adds the slices in a fixed order -> m64, m32 = fp32(m64), |m|^2
//   score_select  reads the (F-1)T non-anchor rows once: fp32 dot with the shared-memory-staged m32 and fp32 norm,
//                 warp-shuffle reductions -> s32.  The CTA that finishes a problem's last rows (ticket again) runs that
//                 problem's selection while the other CTAs are still streaming later problems:
//   selection     the n_keep-th smallest s32 (radix select) is the threshold; tokens further than a proved fp32 error
//                 band from it are decided at once, the few inside the band are re-scored in fp64 against m64 and
//                 ranked exactly by (score, index); emits the ascending index list
//   compress_fused  wide whole-token rows (more than 2,048 columns): both passes in one persistent launch, anchor CTAs
//                 (rows staged in shared memory, anchor_role) and score CTAs side by side on every SM
// Per-head keys (one keep-set per head) use anchor_rows with per-head norms, then head_score and a selection launch of
// its own (n_heads problems per chunk).
//
// The selection is therefore decided in fp64 wherever fp32 could not decide it, and is reproducible
// run to run (no floating-point atomics anywhere).
#include "ptx_sm100.cuh"
#include "wk_internal.cuh"

namespace wk {
namespace {

constexpr int kMaxNormParts = 32;     // pitch of the per-problem |m|^2 record in scratch (one share is used)
constexpr int kScoreThreads = 256;

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

// The kernels of one call depend on each other in a chain and are launched with launch_chained (wk_internal.cuh):
// nothing is read or written before dep_wait(), so only launch latency and block scheduling overlap.

// Where the rows of problem b live.  A chunk is [F*T][rs] bf16; with whole-token keys (one keep-set per chunk) a
// problem is a chunk and D = rs; with per-head keys a chunk holds hs = n_heads problems, problem (chunk, h) owning
// columns [h*D, (h+1)*D) of every row, D = head_dim.
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

// bf16 -> fp64 on the integer pipe, for NORMAL numbers: the double has the same sign, the exponent re-biased by
// 1023 - 127 = 896 and the seven mantissa bits at the top of the fraction -- two or three integer operations where the
// conversion instruction runs at a quarter of the fp64 multiply-add rate.  w holds two bf16 values (low and high half).
// An exponent field of 0 (zero, subnormal) comes out as a number below 2^-126 and a field of 255 (Inf, NaN) as one of at
// least 2^128: anchor_role looks at every row's squared norm, and a group of rows with a norm outside [2^-80, 2^250] is
// redone with the exact conversions below.  Inside that range a mis-read zero or subnormal moves a column sum by less
// than 2^-126 * 2^40 = 2^-86 per row, far below the rounding of the fp64 sums themselves.  (anchor_rows converts every
// element with the conversion instruction and needs none of this.)
// One widening multiply-add builds the whole double: the 15 magnitude bits, moved to the top of a 32-bit word, times
// 2^28 land on bits 59..45 of the 64-bit product (low word zero), and the addend carries the re-biased exponent.
__device__ __forceinline__ double mad_wide_f64(uint32_t a, uint32_t b) {
  uint64_t r;
  asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(r) : "r"(a), "r"(b), "l"(0x3800000000000000ull));
  return __longlong_as_double(static_cast<long long>(r));
}
__device__ __forceinline__ double bf16_lo_abs_fast(uint32_t w) { return mad_wide_f64(w << 17, 1u << 28); }
__device__ __forceinline__ double bf16_hi_abs_fast(uint32_t w) { return mad_wide_f64(w & 0x7FFF0000u, 1u << 29); }
__device__ __forceinline__ double bf16_lo_fast(uint32_t w) {
  const double d = bf16_lo_abs_fast(w);
  return __hiloint2double(__double2hiint(d) | static_cast<int>((w << 16) & 0x80000000u), __double2loint(d));
}
__device__ __forceinline__ double bf16_hi_fast(uint32_t w) {
  const double d = bf16_hi_abs_fast(w);
  return __hiloint2double(__double2hiint(d) | static_cast<int>(w & 0x80000000u), __double2loint(d));
}
template <bool kExact> __device__ __forceinline__ double bf16_lo(uint32_t w) {
  return kExact ? static_cast<double>(__uint_as_float(w << 16)) : bf16_lo_fast(w);
}
template <bool kExact> __device__ __forceinline__ double bf16_hi(uint32_t w) {
  return kExact ? static_cast<double>(__uint_as_float(w & 0xFFFF0000u)) : bf16_hi_fast(w);
}
template <bool kExact> __device__ __forceinline__ double bf16_lo_abs(uint32_t w) {
  return kExact ? static_cast<double>(__uint_as_float(w << 16)) : bf16_lo_abs_fast(w);
}
template <bool kExact> __device__ __forceinline__ double bf16_hi_abs(uint32_t w) {
  return kExact ? static_cast<double>(__uint_as_float(w & 0xFFFF0000u)) : bf16_hi_abs_fast(w);
}

// ------------------------------------------------------------------------------------------------
// Staged anchor role of the one-launch kernel (whole-token keys).  Work item (part, chunk) owns rows
// [part * rpp, (part + 1) * rpp) of the chunk's anchor frame and walks them in groups of G rows:
//   thread 0 keeps one bulk copy (the next group's G contiguous rows) in flight into the other half of the row buffer;
//   phase 1: the 8 warps share the group's rows (8 / G column segments per row): fp64 squared norms from shared memory
//            -> 1/|a| (0 for a zero key);
//   phase 2: thread t owns the 16-byte column groups t, t + 256, ...: a_i[c] / |a_i| is added over the rows of the group.
// The CTA writes its column sums as one slice; the last CTA of the chunk adds the slices in slice order and writes
// m64, m32 = fp32(m64) and |m|^2.  VPT = 16-byte column groups per thread = ceil(D / 2048).
// ------------------------------------------------------------------------------------------------
constexpr int kAnchorThreads = 256;
constexpr int kAnchorWarps = kAnchorThreads / 32;
constexpr double kNorm2Lo = 8.2718061255302767e-25;    // 2^-80: squared norm below which a row is redone exactly
constexpr double kNorm2Hi = 1.8092513943330656e+75;    // 2^250: likewise above

// squared norms of the group's rows: warp -> (row, column segment); n2_s[row][seg]
template <bool kExact>
__device__ __forceinline__ void group_norms(const uint8_t* buf, size_t row_bytes, int rows, int nseg, int seg_vecs, int vecs,
                                            double* n2_s) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = warp / nseg, seg = warp - r * nseg;
  if (r >= rows) return;
  const uint4* row = reinterpret_cast<const uint4*>(buf + r * row_bytes);
  const int v_begin = seg * seg_vecs, v_end = min(vecs, v_begin + seg_vecs);
  double n2a = 0.0, n2b = 0.0;
  for (int v = v_begin + lane; v < v_end; v += 32) {
    const uint4 q = row[v];
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    // three of the eight conversions go to the conversion unit, five to the integer pipe: both stay busy
    const double x0 = bf16_lo_abs<true>(w[0]), x1 = bf16_hi_abs<kExact>(w[0]);
    const double x2 = bf16_lo_abs<kExact>(w[1]), x3 = bf16_hi_abs<true>(w[1]);
    const double x4 = bf16_lo_abs<kExact>(w[2]), x5 = bf16_hi_abs<kExact>(w[2]);
    const double x6 = bf16_lo_abs<true>(w[3]), x7 = bf16_hi_abs<kExact>(w[3]);
    n2a = fma(x0, x0, n2a); n2b = fma(x1, x1, n2b);
    n2a = fma(x2, x2, n2a); n2b = fma(x3, x3, n2b);
    n2a = fma(x4, x4, n2a); n2b = fma(x5, x5, n2b);
    n2a = fma(x6, x6, n2a); n2b = fma(x7, x7, n2b);
  }
  const double n2 = warp_sum(n2a + n2b);
  if (lane == 0) n2_s[r * nseg + seg] = n2;
}

// column sums of a / |a| over the rows of the group, for the 16-byte column groups this thread owns (t, t + 256, ...)
template <int VPT, bool kExact>
__device__ __forceinline__ void group_accumulate(const uint8_t* buf, size_t row_bytes, int rows, int vecs,
                                                 const double* inv_s, double (&acc)[8 * VPT]) {
  const int tid = threadIdx.x;
  for (int r = 0; r < rows; ++r) {
    const uint4* row = reinterpret_cast<const uint4*>(buf + r * row_bytes);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vec = tid + i * kAnchorThreads;
      if (vec < vecs) {
        const uint4 q = row[vec];
        const double sc = inv_s[r];
        double* a = acc + 8 * i;
        a[0] = fma(bf16_lo<true>(q.x), sc, a[0]);
        a[1] = fma(bf16_hi<kExact>(q.x), sc, a[1]);
        a[2] = fma(bf16_lo<kExact>(q.y), sc, a[2]);
        a[3] = fma(bf16_hi<true>(q.y), sc, a[3]);
        a[4] = fma(bf16_lo<kExact>(q.z), sc, a[4]);
        a[5] = fma(bf16_hi<kExact>(q.z), sc, a[5]);
        a[6] = fma(bf16_lo<true>(q.w), sc, a[6]);
        a[7] = fma(bf16_hi<kExact>(q.w), sc, a[7]);
      }
    }
  }
}

// After a CTA has written its slice of chunk b: the last CTA of the chunk (an atomic ticket decides) adds the slices in
// slice order and writes m64, m32 = fp32(m64) and |m|^2 (per head with per-head keys).  Called by every thread of the CTA.
__device__ __forceinline__ void anchor_finish(int b, int parts, int T, int D, int hs, const double* __restrict__ partial,
                                              int max_parts, uint32_t* __restrict__ tickets, double* __restrict__ m64,
                                              float* __restrict__ m32, double* __restrict__ mnorm2, uint32_t* ready,
                                              uint32_t epoch) {
  __shared__ uint32_t s_flag;
  __shared__ double red[32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nthr = blockDim.x, nwarps = nthr >> 5;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_flag = (atomicAdd(&tickets[b], 1u) == static_cast<uint32_t>(parts - 1)) ? 1u : 0u;
  __syncthreads();
  if (!s_flag) return;
  // ---- last CTA of the chunk: add the slices in slice order.  Thread t owns column pairs t, t + 256, ...; eight
  // slices' worth of loads are in flight before the first addition.
  __threadfence();
  const double* pb = partial + static_cast<int64_t>(b) * max_parts * D;
  const double inv_T = 1.0 / static_cast<double>(T);
  const int pairs = D >> 1;
  double nn_all = 0.0;
  for (int c0 = 0; c0 < pairs; c0 += nthr) {   // uniform trip count: the per-head sums use block barriers
    const int c = c0 + tid;
    double t0 = 0.0, t1 = 0.0;
    if (c < pairs) {
      for (int p0 = 0; p0 < parts; p0 += 8) {
        double2 v[8];
#pragma unroll
        for (int pp = 0; pp < 8; ++pp)
          v[pp] = p0 + pp < parts ? __ldcg(reinterpret_cast<const double2*>(pb + static_cast<int64_t>(p0 + pp) * D) + c)
                                  : make_double2(0.0, 0.0);
#pragma unroll
        for (int pp = 0; pp < 8; ++pp) {
          t0 += v[pp].x;
          t1 += v[pp].y;
        }
      }
      t0 *= inv_T;
      t1 *= inv_T;
      reinterpret_cast<double2*>(m64 + static_cast<int64_t>(b) * D)[c] = make_double2(t0, t1);
      reinterpret_cast<float2*>(m32 + static_cast<int64_t>(b) * D)[c] =
          make_float2(static_cast<float>(t0), static_cast<float>(t1));
    }
    const double nn = fma(t0, t0, t1 * t1);
    if (hs == 1) {
      nn_all += nn;
    } else {
      // 64 column pairs per head: warps 2j and 2j + 1 of this step hold head c0 / 64 + j
      const double wsum = warp_sum(nn);
      __syncthreads();
      if (lane == 0) red[warp] = wsum;
      __syncthreads();
      const int head = (c0 >> 6) + tid;
      if (tid < nwarps / 2 && head < hs)
        mnorm2[(static_cast<int64_t>(b) * hs + head) * kMaxNormParts] = red[2 * tid] + red[2 * tid + 1];
    }
  }
  if (hs == 1) {
    const double wsum = warp_sum(nn_all);
    if (lane == 0) red[warp] = wsum;
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      for (int w = 0; w < nwarps; ++w) t += red[w];
      mnorm2[static_cast<int64_t>(b) * kMaxNormParts] = t;
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    tickets[b] = 0;   // ready for the next call
    if (ready) {
      __threadfence();                                   // m64 / m32 / |m|^2 of every thread are out before the flag
      *reinterpret_cast<volatile uint32_t*>(ready + b) = epoch;
    }
  }
}

// The work of one anchor CTA (slice `part` of `parts` of chunk b).  `ready` (may be null): a word per chunk that the last
// CTA of the chunk sets to `epoch` once m64 / m32 / |m|^2 are written, for score CTAs of the same launch to poll.
template <int VPT>
__device__ __forceinline__ void anchor_role(uint8_t* smem, int b, int part, int parts, const __nv_bfloat16* __restrict__ K,
                                            int64_t stride, int T, int D, int G, int rpp,
                                            double* __restrict__ partial, int max_parts, uint32_t* __restrict__ tickets,
                                            double* __restrict__ m64, float* __restrict__ m32, double* __restrict__ mnorm2,
                                            uint32_t* __restrict__ status, uint32_t* ready, uint32_t epoch,
                                            uint64_t* bar, uint32_t& gbase) {
  // bar[2]: the caller's two mbarriers (initialised once per CTA, count 1); gbase: bulk copies this CTA has waited for so
  // far -- copy number n lands in buffer n & 1 and completes phase n >> 1 of barrier n & 1
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t row_bytes = static_cast<size_t>(D) * 2;
  const int nseg = kAnchorWarps / G;                                        // column segments per row in phase 1
  uint8_t* rows_s = smem;                                                   // [2][G][D] bf16
  double* inv_s = reinterpret_cast<double*>(smem + 2 * G * row_bytes);      // [G]
  double* n2_s = inv_s + G;                                                 // [G][nseg]
  const int r0 = min(T, part * rpp), r1 = min(T, r0 + rpp);
  const int n_groups = (r1 - r0 + G - 1) / G;
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(b) * stride;
  auto issue = [&](int g) {   // thread 0: one bulk copy of the group's rows (contiguous in memory)
    const int ra = r0 + g * G;
    const uint32_t bytes = static_cast<uint32_t>(min(G, r1 - ra) * row_bytes);
    const uint32_t n = gbase + g;
    ptx::mbar_expect_tx(&bar[n & 1], bytes);
    ptx::bulk_load_1d(rows_s + (n & 1) * G * row_bytes, Kb + static_cast<int64_t>(ra) * D, bytes, &bar[n & 1]);
  };
  if (tid == 0 && n_groups > 0) {
    ptx::fence_proxy_async_smem();   // the buffers may have been written with ordinary stores by the work item before
    issue(0);
  }
  double acc[8 * VPT];
#pragma unroll
  for (int i = 0; i < 8 * VPT; ++i) acc[i] = 0.0;
  const int vecs = D >> 3;
  const int seg_vecs = (((vecs >> 4) + nseg - 1) / nseg) << 4;   // whole 128-column blocks per segment
  int armed = n_groups > 0 ? 1 : 0;   // groups whose copy has been issued
  int g = 0;
  for (; g < n_groups; ++g) {
    if (g + 1 < n_groups) {
      if (tid == 0) issue(g + 1);     // its buffer was released by the barrier that ended group g - 1
      armed = g + 2;
    }
    const uint32_t n_cur = gbase + g;
    const bool landed = ptx::mbar_wait(&bar[n_cur & 1], (n_cur >> 1) & 1);
    if (__syncthreads_or(!landed)) {  // a copy that never lands: report, stop reading, still hand in the slice
      if (tid == 0) atomicOr(status, WK_DEV_TIMEOUT);
      break;
    }
    const int rows = min(G, r1 - (r0 + g * G));
    const uint8_t* buf = rows_s + (n_cur & 1) * G * row_bytes;
    // ---- phase 1: norms (integer-pipe conversions; redone exactly when a norm falls outside the safe range)
    group_norms<false>(buf, row_bytes, rows, nseg, seg_vecs, vecs, n2_s);
    bool redo = false;
    if (nseg == 1) {
      // one warp holds a whole row's squared norm: its first lane finishes the row on the spot, so that the eight
      // reciprocal square roots run side by side and one barrier (the vote below) ends the phase
      if (warp < rows && lane == 0) {
        const double n2 = n2_s[warp];
        inv_s[warp] = n2 == 0.0 ? 0.0 : 1.0 / sqrt(n2);
        redo = !(n2 >= kNorm2Lo && n2 <= kNorm2Hi);
      }
    } else {
      __syncthreads();
    }
    auto finish_norms = [&](bool check) {
      for (int r = tid; r < rows; r += kAnchorThreads) {
        double n2 = 0.0;
        for (int sg = 0; sg < nseg; ++sg) n2 += n2_s[r * nseg + sg];
        inv_s[r] = n2 == 0.0 ? 0.0 : 1.0 / sqrt(n2);   // zero key: cosine 0; a NaN norm stays NaN
        if (check) redo = redo || !(n2 >= kNorm2Lo && n2 <= kNorm2Hi);
      }
    };
    if (nseg != 1) finish_norms(true);
    const bool exact = __syncthreads_or(redo) != 0;
    if (exact) {
      group_norms<true>(buf, row_bytes, rows, nseg, seg_vecs, vecs, n2_s);
      __syncthreads();
      finish_norms(false);
      __syncthreads();
      group_accumulate<VPT, true>(buf, row_bytes, rows, vecs, inv_s, acc);
    } else {
      // ---- phase 2
      group_accumulate<VPT, false>(buf, row_bytes, rows, vecs, inv_s, acc);
    }
    __syncthreads();   // the group's buffer, inv_s and n2_s may be overwritten from here on
  }
  // a copy still in flight when the loop was left early must land before the CTA gives up its shared memory
  if (tid == 0) {
    for (int gg = g; gg < armed; ++gg)   // empty unless the loop was left at group g < n_groups
      for (uint32_t i = 0; i < (1u << 16); ++i)
        if (ptx::mbar_try_wait(&bar[(gbase + gg) & 1], ((gbase + gg) >> 1) & 1)) break;
  }
  gbase += static_cast<uint32_t>(armed);   // every issued copy has been waited for (or given up on) by now
  __syncthreads();
  // ---- this CTA's slice
  double* my = partial + (static_cast<int64_t>(b) * max_parts + part) * D;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vec = tid + i * kAnchorThreads;
    if (vec < vecs) {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        __stcg(reinterpret_cast<double2*>(my + 8 * vec) + e, make_double2(acc[8 * i + 2 * e], acc[8 * i + 2 * e + 1]));
    }
  }
  anchor_finish(b, parts, T, D, 1, partial, max_parts, tickets, m64, m32, mnorm2, ready, epoch);
}

// ------------------------------------------------------------------------------------------------
// anchor pass, rows held in registers.  grid = one CTA per SM, NW warps.  The anchor rows of all chunks,
// numbered chunk by chunk, are cut into equal runs, one per CTA.  A row is read by a SET of wpr consecutive warps
// (the fewest that leave a lane at most 6, with per-head keys 3, 16-byte column groups); lane l of warp w of the set owns the column
// groups (w * 32 + l) + 32 * wpr * i, i < VPL.  The CTA's NW / wpr sets take the rows of the run round robin;
// every lane
//   converts its share of the row to fp64 once (the conversion unit's rate, a quarter of the fp64 multiply-add rate, is
//   what bounds this kernel: one conversion per element, not one per phase) and issues the loads of its share of the
//   set's next row into the registers just freed;
//   phase 1: squares its share; the row's squared norm is a warp sum (plus an exchange between the set's warps through
//            shared memory when wpr > 1); with per-head keys a sum over the 16 lanes that hold one head's 128 columns;
//            1/|a| from the fp32 reciprocal square root and two Newton steps in fp64 (within a few units of the last
//            place, the order of the rounding of the fp64 column sums themselves);
//   phase 2: adds a / |a| to its own column sums, which stay in registers for the whole run.
// Nothing is staged in shared memory and the sets never wait for one another inside the row loop.  At a chunk boundary
// and at the end the sets' column sums are added in set order in shared memory, the CTA writes them as its slice of
// that chunk and anchor_finish does the rest.
// ------------------------------------------------------------------------------------------------
// NW warps per CTA and at most kRowMaxVpl column groups per lane: 8 warps x 6 groups for whole-token keys (255 registers
// per thread), 16 warps x 3 groups for per-head keys (128 registers; measured faster there: 109 against 124 us per cfg2
// call, 624 against 690 us at the LingBot shape -- and 2 us slower for whole-token keys).
constexpr int kRowWarpsWhole = 8, kRowMaxVplWhole = 6;
constexpr int kRowWarpsHead = 16, kRowMaxVplHead = 3;
constexpr int kFusedScoreRows = 64;   // rows of a score item of the one-launch kernel (measured: 64-80 best at 5,120 columns)
constexpr int kFusedMinCols = 2048;   // whole-token rows wider than this take the one-launch path (measured faster there)
constexpr double kRowNorm2Hi = 1.2676506002282294e+30;    // 2^100: above it (or below 2^-80) 1/|a| is a true division

__device__ __forceinline__ double rsqrt_newton(double x) {   // x in [2^-80, 2^100]: inside fp32's normal range
  double y = static_cast<double>(rsqrtf(static_cast<float>(x)));
  const double h = 0.5 * x;
  y = fma(y, fma(-h * y, y, 0.5), y);
  y = fma(y, fma(-h * y, y, 0.5), y);
  return y;
}
__device__ __forceinline__ double inverse_norm(double n2) {
  if (n2 >= kNorm2Lo && n2 <= kRowNorm2Hi) return rsqrt_newton(n2);
  return n2 == 0.0 ? 0.0 : 1.0 / sqrt(n2);   // zero key: cosine 0; a NaN norm stays NaN
}

__device__ __forceinline__ void set_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// The lane's share of one row, converted to fp64 ONCE (x, kept in registers for phase 2), with the sum of squares of
// each of its column groups.  One conversion instruction per element: the conversion unit's rate (a quarter of the
// fp64 multiply-add rate) is what bounds the kernel, and converting once instead of once per phase is what the
// registers are spent on.
template <int VPL>
__device__ __forceinline__ void row_convert(const uint4 (&q)[VPL], uint32_t active, double (&x)[8 * VPL], double (&p)[VPL]) {
#pragma unroll
  for (int i = 0; i < VPL; ++i) {
    const uint32_t w[4] = {q[i].x, q[i].y, q[i].z, q[i].w};
    double* xi = x + 8 * i;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      xi[2 * e] = static_cast<double>(__uint_as_float(w[e] << 16));
      xi[2 * e + 1] = static_cast<double>(__uint_as_float(w[e] & 0xFFFF0000u));
    }
    double a = xi[0] * xi[0], c = xi[1] * xi[1];
    a = fma(xi[2], xi[2], a); c = fma(xi[3], xi[3], c);
    a = fma(xi[4], xi[4], a); c = fma(xi[5], xi[5], c);
    a = fma(xi[6], xi[6], a); c = fma(xi[7], xi[7], c);
    p[i] = (active >> i) & 1u ? a + c : 0.0;   // a column group past the end of the row repeats column 0: masked out
  }
}

// 1/|a| for each of the lane's column groups from their sums of squares (all equal with whole-token keys).
template <int VPL, int NW>
__device__ __forceinline__ void row_inverse_norms(const double (&p)[VPL], int hs, int wpr, int set, int wr, double* n2x,
                                                  int& xc, double (&inv)[VPL]) {
  const int lane = threadIdx.x & 31;
  if (hs == 1) {
    double n2 = p[0];
#pragma unroll
    for (int i = 1; i < VPL; ++i) n2 += p[i];
    n2 = warp_sum(n2);
    if (wpr > 1) {
      // the set's warps leave their shares in one of two rows of n2x (alternating, so that one barrier per exchange
      // is enough: a warp can only be one exchange ahead of the slowest warp of its set)
      double* xs = n2x + (xc & 1) * NW + set * wpr;
      ++xc;
      if (lane == 0) xs[wr] = n2;
      set_barrier(1 + set, wpr * 32);
      if (wpr == 2) {
        const double2 t = *reinterpret_cast<const double2*>(xs);
        n2 = t.x + t.y;
      } else if (wpr == 4) {
        const double2 t = *reinterpret_cast<const double2*>(xs), u = *reinterpret_cast<const double2*>(xs + 2);
        n2 = (t.x + t.y) + (u.x + u.y);
      } else {
        n2 = xs[0];
        for (int w2 = 1; w2 < wpr; ++w2) n2 += xs[w2];
      }
    }
    const double r = inverse_norm(n2);
#pragma unroll
    for (int i = 0; i < VPL; ++i) inv[i] = r;
  } else {
#pragma unroll
    for (int i = 0; i < VPL; ++i) inv[i] = inverse_norm(half_warp_sum(p[i]));   // 16 lanes = 128 columns = one head
  }
}

template <int VPL, int NW>
__global__ void __launch_bounds__(NW * 32, 1)
anchor_rows(const __nv_bfloat16* __restrict__ K, int64_t stride, int chunks, int T, int D, int hs, int wpr, int R,
            double* __restrict__ partial, int max_parts, uint32_t* __restrict__ tickets, double* __restrict__ m64,
            float* __restrict__ m32, double* __restrict__ mnorm2) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(16) double n2x[2 * NW];
  double* sacc = reinterpret_cast<double*>(smem);   // [n_sets][D]
  dep_release();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_sets = NW / wpr, set = warp / wpr, wr = warp - set * wpr;
  const int vecs = D >> 3, vstep = 32 * wpr, v0 = wr * 32 + lane;
  uint32_t active = 0;
  int voff[VPL];
#pragma unroll
  for (int i = 0; i < VPL; ++i) {
    const bool on = v0 + i * vstep < vecs;
    active |= (on ? 1u : 0u) << i;
    voff[i] = on ? v0 + i * vstep : 0;
  }
  // the anchor rows of all chunks, numbered chunk by chunk, are cut into runs of R rows, one per CTA: every SM gets the
  // same number of rows and a CTA hands in one slice per chunk its run touches (one or two at the benchmark shapes)
  const int64_t total = static_cast<int64_t>(chunks) * T;
  const int64_t g_end = min(total, static_cast<int64_t>(blockIdx.x + 1) * R);
  int xc = 0;
  for (int64_t g = static_cast<int64_t>(blockIdx.x) * R; g < g_end;) {
    const int b = static_cast<int>(g / T);
    const int r0 = static_cast<int>(g - static_cast<int64_t>(b) * T);
    const int r1 = static_cast<int>(min(static_cast<int64_t>(T), r0 + (g_end - g)));
    g += r1 - r0;
    const uint4* Kb = reinterpret_cast<const uint4*>(K + static_cast<int64_t>(b) * stride);
    // loads carry no predicate: a row past the end of the run is read from the chunk's last row and never used, and a
    // column group past the end of the row is read from column 0 and masked out of the norm (its sums are not stored)
    auto load_row = [&](int r, uint4 (&q)[VPL]) {
      const uint4* row = Kb + static_cast<int64_t>(min(r, T - 1)) * vecs;
#pragma unroll
      for (int i = 0; i < VPL; ++i) q[i] = __ldcs(row + voff[i]);
    };
    double acc[8 * VPL];
#pragma unroll
    for (int i = 0; i < 8 * VPL; ++i) acc[i] = 0.0;
    uint4 q[VPL];
    int r = r0 + set;
    load_row(r, q);
    for (; r < r1; r += n_sets) {
      double x[8 * VPL], p[VPL], inv[VPL];
      row_convert<VPL>(q, active, x, p);
      load_row(r + n_sets, q);   // the next row's loads fly while this one is finished
      row_inverse_norms<VPL, NW>(p, hs, wpr, set, wr, n2x, xc, inv);
#pragma unroll
      for (int i = 0; i < VPL; ++i)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[8 * i + e] = fma(x[8 * i + e], inv[i], acc[8 * i + e]);
    }
    // ---- every set leaves its column sums in its own row of sacc; the slice is their sum in set order
    double* mine = sacc + static_cast<size_t>(set) * D;
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      if ((active >> i) & 1u) {
        double2* dst = reinterpret_cast<double2*>(mine + 8 * voff[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) dst[e] = make_double2(acc[8 * i + 2 * e], acc[8 * i + 2 * e + 1]);
      }
    }
    __syncthreads();
    // the CTAs whose runs touch chunk b, in order: first .. last; this one's slice number is its place among them
    const int first = static_cast<int>((static_cast<int64_t>(b) * T) / R);
    const int last = static_cast<int>((static_cast<int64_t>(b + 1) * T - 1) / R);
    const int part = static_cast<int>(blockIdx.x) - first;
    double2* my = reinterpret_cast<double2*>(partial + (static_cast<int64_t>(b) * max_parts + part) * D);
    const int pairs = D >> 1;
    for (int c = tid; c < pairs; c += NW * 32) {
      double2 t = reinterpret_cast<const double2*>(sacc)[c];
      for (int s2 = 1; s2 < n_sets; ++s2) {
        const double2 o = reinterpret_cast<const double2*>(sacc + static_cast<size_t>(s2) * D)[c];
        t.x += o.x;
        t.y += o.y;
      }
      __stcg(my + c, t);
    }
    anchor_finish(b, last - first + 1, T, D, hs, partial, max_parts, tickets, m64, m32, mnorm2, nullptr, 0u);
    __syncthreads();   // sacc and anchor_finish's shared words are free for the next chunk
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
// selection of one problem by one CTA of kThr threads (a device function: the score kernel's last CTA of a problem calls
// it in place; per-head keys and the trivial cases n_keep = 0 / all have a kernel of their own around it).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t f32_key(float f) {   // order-preserving map float -> uint32
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_f32(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

template <int kThr, bool kPerHead>
__device__ __forceinline__ void select_problem(uint8_t* smem, int b, const __nv_bfloat16* __restrict__ K, RowMap rm, int T,
                                               int NA, int D, int n_keep, const float* __restrict__ s32,
                                               const double* __restrict__ m64, const double* __restrict__ mnorm,
                                               int32_t* __restrict__ keep_idx, uint32_t* __restrict__ status) {
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem);                       // [NA]
  int32_t* band_idx = reinterpret_cast<int32_t*>(keys + NA);                // [NA]
  double* band_s = reinterpret_cast<double*>(band_idx + NA);                // [NA] (8-byte aligned: 8*NA)
  uint8_t* flag = reinterpret_cast<uint8_t*>(band_s + NA);                  // [NA]
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sel_prefix, sel_rank, n_band, n_below;
  __shared__ uint32_t warp_tot[32];
  __shared__ double band_red[8][kThr / 32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = T + n_keep;
  int32_t* out = keep_idx + static_cast<int64_t>(b) * C;
  for (int i = tid; i < T; i += kThr) out[i] = i;                 // the anchor frame is kept whole
  if (n_keep == 0) return;
  if (n_keep == NA) {
    for (int j = tid; j < NA; j += kThr) out[T + j] = T + j;
    return;
  }
  const float* sb = s32 + static_cast<int64_t>(b) * NA;
  for (int j = tid; j < NA; j += kThr) keys[j] = f32_key(__ldcg(sb + j));   // written by other CTAs: read through L2
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
  const double mn2 = __ldcg(mnorm + static_cast<int64_t>(b) * kMaxNormParts);
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

// One CTA per problem: per-head keys (n_heads problems per chunk) and the cases that need no scores.
constexpr int kSelectThreads = 256;
template <bool kPerHead>
__global__ void __launch_bounds__(kSelectThreads)
select_pass(const __nv_bfloat16* __restrict__ K, RowMap rm, int T, int NA, int D, int n_keep,
            const float* __restrict__ s32, const double* __restrict__ m64, const double* __restrict__ mnorm,
            int32_t* __restrict__ keep_idx, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  dep_wait();
  select_problem<kSelectThreads, kPerHead>(smem, blockIdx.x, K, rm, T, NA, D, n_keep, s32, m64, mnorm, keep_idx, status);
}

// ------------------------------------------------------------------------------------------------
// score pass + selection.  grid = blocks of rows (nblk equal blocks per chunk, sized at launch), problem-major (blockIdx.x = b * nblk + block), so that
// the problems finish in order; one warp per row; m32 staged in shared memory.  The CTA that hands in the last rows of
// a problem (atomic ticket; nobody waits) runs that problem's selection on the spot, under the streaming of the
// problems behind it.
// Per lane the fp32 accumulation is two chains of 4 * ceil(D/256) fused multiply-adds (the low and the high halves of
// the packed pairs), one addition of the two, then five shuffle additions: no deeper than the single chain of
// 8 * ceil(D/256) + 5 operations the selection's error band is derived for.
// ------------------------------------------------------------------------------------------------
// The work of one score CTA: block `blk` (one of nblk equal blocks of rows) of chunk b, and the chunk's selection if this CTA hands in
// the chunk's last block.
__device__ __forceinline__ bool score_role(uint8_t* smem, int b, int blk, const __nv_bfloat16* __restrict__ K, int64_t stride,
                                           int T, int NA, int D, int n_keep, int nblk, const float* __restrict__ m32,
                                           const double* __restrict__ m64, const double* __restrict__ mnorm,
                                           float* __restrict__ s32, float* __restrict__ scores_out,
                                           uint32_t* __restrict__ tickets, int32_t* __restrict__ keep_idx,
                                           uint32_t* __restrict__ status, bool m_staged = false) {
  // m_staged: the chunk's m32 is in shared memory already (the CTA's previous item was a block of the same chunk).
  // Returns true if shared memory still holds it on return, false if the selection has used the space.
  __shared__ uint32_t s_last;
  float4* m = reinterpret_cast<float4*>(smem);   // [D/4]; the selection reuses the space afterwards
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (!m_staged) {
    const float4* msrc = reinterpret_cast<const float4*>(m32 + static_cast<int64_t>(b) * D);
    for (int i = tid; i < (D >> 2); i += kScoreThreads) m[i] = __ldcg(msrc + i);
    __syncthreads();
  }
  const int vecs = D >> 3;
  const int rows = (NA + nblk - 1) / nblk;   // the chunk's non-anchor rows in nblk equal blocks
  const int j0 = min(NA, blk * rows);
  const int j1 = min(NA, j0 + rows);
  const int pitch = D;
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(b) * stride + static_cast<int64_t>(T) * pitch;
  // two rows per warp at a time, so that twice as many 16-byte loads are in flight
  constexpr int W = kScoreThreads / 32;
  for (int j = j0 + warp; j < j1; j += 2 * W) {
    const int jb = j + W;
    const bool has_b = jb < j1;
    const uint4* row_a = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(j) * pitch);
    const uint4* row_b = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(has_b ? jb : j) * pitch);
    // packed fp32 pairs: one instruction multiplies-and-adds the two bf16 values of a 32-bit word; the low and the high
    // halves keep separate sums (half as long as a single chain would be), added once at the end
    uint64_t dot2_a = 0, n22_a = 0, dot2_b = 0, n22_b = 0;
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
          const uint64_t mm[4] = {ptx::pack_f32x2(ma.x, ma.y), ptx::pack_f32x2(ma.z, ma.w), ptx::pack_f32x2(mb.x, mb.y),
                                  ptx::pack_f32x2(mb.z, mb.w)};
          const uint32_t wa[4] = {qa[u].x, qa[u].y, qa[u].z, qa[u].w}, wb[4] = {qb[u].x, qb[u].y, qb[u].z, qb[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint64_t xa = ptx::pack_f32x2(bf16lo(wa[e]), bf16hi(wa[e]));
            const uint64_t xb = ptx::pack_f32x2(bf16lo(wb[e]), bf16hi(wb[e]));
            dot2_a = ptx::fma_f32x2(xa, mm[e], dot2_a);
            n22_a = ptx::fma_f32x2(xa, xa, n22_a);
            dot2_b = ptx::fma_f32x2(xb, mm[e], dot2_b);
            n22_b = ptx::fma_f32x2(xb, xb, n22_b);
          }
        }
      }
    }
    float lo_, hi_;
    ptx::unpack_f32x2(dot2_a, lo_, hi_); float dot_a = lo_ + hi_;
    ptx::unpack_f32x2(n22_a, lo_, hi_);  float n2_a = lo_ + hi_;
    ptx::unpack_f32x2(dot2_b, lo_, hi_); float dot_b = lo_ + hi_;
    ptx::unpack_f32x2(n22_b, lo_, hi_);  float n2_b = lo_ + hi_;
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
  if (keep_idx == nullptr) return true;   // scores only
  // hand in this block of rows; the CTA that completes the problem selects
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&tickets[b], 1u) == static_cast<uint32_t>(nblk - 1)) ? 1u : 0u;
  __syncthreads();
  if (!s_last) return true;
  __threadfence();
  if (tid == 0) tickets[b] = 0;   // ready for the next call
  const RowMap rm{stride, D, 1};
  select_problem<kScoreThreads, false>(smem, b, K, rm, T, NA, D, n_keep, s32, m64, mnorm, keep_idx, status);
  return false;
}

__global__ void __launch_bounds__(kScoreThreads)
score_select(const __nv_bfloat16* __restrict__ K, int64_t stride, int T, int NA, int D, int n_keep, int nblk,
             const float* __restrict__ m32, const double* __restrict__ m64, const double* __restrict__ mnorm,
             float* __restrict__ s32, float* __restrict__ scores_out, uint32_t* __restrict__ tickets,
             int32_t* __restrict__ keep_idx, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  dep_wait();
  dep_release();
  score_role(smem, blockIdx.x / nblk, blockIdx.x % nblk, K, stride, T, NA, D, n_keep, nblk, m32, m64, mnorm, s32, scores_out,
             tickets, keep_idx, status);
}

// ------------------------------------------------------------------------------------------------
// Both passes in one launch.  The anchor pass is bound by instruction issue (fp64), the score pass by memory; run side
// by side on the same SMs they overlap instead of adding up.  The grid is persistent (as many CTAs as fit the machine);
// every CTA takes work items from two queues until both are empty:
//   anchor items (chunk, slice), chunk-major, always available;
//   score items (chunk, block of rows), chunk-major; the head of that queue is available once its chunk's `ready` word
//   carries this call's epoch, i.e. once the chunk's last anchor CTA has written the mean anchor.
// Half of the CTAs prefer score items and half anchor items (each falls back to the other kind), so that both kinds
// run on every SM; nobody waits while there is work of either kind.  The only wait left: a CTA that has taken a score item
// of a chunk that is not ready yet (the head moved on between its look and its take) -- bounded, status WK_DEV_TIMEOUT.
// ------------------------------------------------------------------------------------------------
struct FusedQueue {
  uint32_t a_next, s_next, exited, pad;
};

template <int VPT>
__global__ void __launch_bounds__(kAnchorThreads, VPT == 1 ? 4 : (VPT == 2 ? 3 : 2))
compress_fused(const __nv_bfloat16* __restrict__ K, int64_t stride, int chunks, int T, int NA, int D, int n_keep, int G,
               int rpp, int parts, int nblk, int layer_ctas, double* __restrict__ partial, int max_parts,
               uint32_t* __restrict__ tickets_a, uint32_t* __restrict__ tickets_s, uint32_t* ready, FusedQueue* q,
               uint32_t epoch, double* __restrict__ m64, float* __restrict__ m32, double* __restrict__ mnorm,
               float* __restrict__ s32, float* __restrict__ scores_out, int32_t* __restrict__ keep_idx,
               uint32_t* __restrict__ status) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bar[2];
  __shared__ int s_kind, s_item;
  dep_release();
  const int tid = threadIdx.x;
  if (tid == 0) {
    ptx::mbar_init(&bar[0], 1);
    ptx::mbar_init(&bar[1], 1);
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const uint32_t a_total = static_cast<uint32_t>(chunks) * parts, s_total = static_cast<uint32_t>(chunks) * nblk;
  // CTAs that share an SM have block indices layer_ctas apart (one per SM and "layer"): alternate the preference by layer
  const bool prefer_score = ((blockIdx.x / layer_ctas) & 1) != 0;
  uint32_t gbase = 0;
  int staged_chunk = -1;   // chunk whose m32 this CTA's shared memory holds, if any
  volatile uint32_t* vq_a = &q->a_next;
  volatile uint32_t* vq_s = &q->s_next;
  for (uint32_t idle = 0; idle < (1u << 20);) {
    if (tid == 0) {
      int kind = -1, item = 0;      // kind: 0 anchor, 1 score, -1 nothing available now, -2 all work handed out
      for (int attempt = 0; attempt < 2 && kind < 0; ++attempt) {
        const bool want_score = (attempt == 0) == prefer_score;
        if (want_score) {
          const uint32_t cur = *vq_s;
          if (cur < s_total && *reinterpret_cast<volatile uint32_t*>(ready + cur / nblk) == epoch) {
            const uint32_t i = atomicAdd(&q->s_next, 1u);
            if (i < s_total) { kind = 1; item = static_cast<int>(i); }
          }
        } else if (*vq_a < a_total) {
          const uint32_t i = atomicAdd(&q->a_next, 1u);
          if (i < a_total) { kind = 0; item = static_cast<int>(i); }
        }
      }
      if (kind < 0 && *vq_a >= a_total && *vq_s >= s_total) kind = -2;
      if (kind == 1) {
        // the take may have run ahead of the look into the next chunk: wait for that chunk (rare, short, bounded)
        const int c = item / nblk;
        bool ok = false;
        for (uint32_t i = 0; i < (1u << 22); ++i) {
          if (*reinterpret_cast<volatile uint32_t*>(ready + c) == epoch) { ok = true; break; }
          __nanosleep(100);
        }
        if (!ok) { atomicOr(status, WK_DEV_TIMEOUT); kind = -3; }
        __threadfence();            // the chunk's m32 / m64 are read after the flag
      }
      s_kind = kind;
      s_item = item;
    }
    __syncthreads();
    const int kind = s_kind, item = s_item;
    __syncthreads();
    if (kind == -2) break;
    if (kind == -1) { ++idle; __nanosleep(200); continue; }
    if (kind == 0) {
      staged_chunk = -1;
      anchor_role<VPT>(smem, item / parts, item % parts, parts, K, stride, T, D, G, rpp, partial, max_parts, tickets_a,
                       m64, m32, mnorm, status, ready, epoch, bar, gbase);
    } else if (kind == 1) {
      const int c = item / nblk;
      const bool kept = score_role(smem, c, item % nblk, K, stride, T, NA, D, n_keep, nblk, m32, m64, mnorm, s32,
                                   scores_out, tickets_s, keep_idx, status, staged_chunk == c);
      staged_chunk = kept ? c : -1;
    }
    __syncthreads();
  }
  // the CTA that leaves last puts the queue back for the next call
  if (tid == 0) {
    if (s_kind != -2) atomicOr(status, WK_DEV_TIMEOUT);   // left because nothing became available for far too long
    if (atomicAdd(&q->exited, 1u) == gridDim.x - 1) {
      q->a_next = 0u;
      q->s_next = 0u;
      q->exited = 0u;
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
  const int rows = (NA + gridDim.x - 1) / gridDim.x;   // the chunk's non-anchor rows in gridDim.x equal blocks
  const int j0 = min(NA, static_cast<int>(blockIdx.x) * rows);
  const int j1 = min(NA, j0 + rows);
  const __nv_bfloat16* Kb = K + static_cast<int64_t>(chunk) * stride + static_cast<int64_t>(T) * D;
  constexpr int W = kScoreThreads / 32;
  // two rows per warp at a time, so that twice as many 16-byte loads are in flight
  for (int j = j0 + warp; j < j1; j += 2 * W) {
    const int jb = j + W;
    const bool has_b = jb < j1;
    const uint4* row_a = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(j) * D);
    const uint4* row_b = reinterpret_cast<const uint4*>(Kb + static_cast<int64_t>(has_b ? jb : j) * D);
    for (int v0 = lane; v0 - lane < vecs; v0 += 128) {
      uint4 qa[4], qb[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool in = v0 + 32 * u < vecs;
        qa[u] = in ? __ldg(row_a + v0 + 32 * u) : make_uint4(0, 0, 0, 0);
        qb[u] = in ? __ldg(row_b + v0 + 32 * u) : make_uint4(0, 0, 0, 0);
      }
      // 16 partial sums per lane: for each of the four column groups u the pair (dot, |k|^2) of row j and of row jb
      float val[16];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u;
        float dot_a = 0.f, n2_a = 0.f, dot_b = 0.f, n2_b = 0.f;
        if (v < vecs) {
          // packed fp32 pairs, as in score_role: the low and the high halves of the words keep separate sums of four
          // terms each, added once at the end (no deeper than the single chain of eight the error band was derived for)
          const float4 ma = m[2 * v], mb = m[2 * v + 1];
          const uint64_t mm[4] = {ptx::pack_f32x2(ma.x, ma.y), ptx::pack_f32x2(ma.z, ma.w), ptx::pack_f32x2(mb.x, mb.y),
                                  ptx::pack_f32x2(mb.z, mb.w)};
          const uint32_t wa[4] = {qa[u].x, qa[u].y, qa[u].z, qa[u].w}, wb[4] = {qb[u].x, qb[u].y, qb[u].z, qb[u].w};
          uint64_t d2a = 0, s2a = 0, d2b = 0, s2b = 0;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint64_t xa = ptx::pack_f32x2(bf16lo(wa[e]), bf16hi(wa[e]));
            const uint64_t xb = ptx::pack_f32x2(bf16lo(wb[e]), bf16hi(wb[e]));
            d2a = ptx::fma_f32x2(xa, mm[e], d2a);
            s2a = ptx::fma_f32x2(xa, xa, s2a);
            d2b = ptx::fma_f32x2(xb, mm[e], d2b);
            s2b = ptx::fma_f32x2(xb, xb, s2b);
          }
          float lo_, hi_;
          ptx::unpack_f32x2(d2a, lo_, hi_); dot_a = lo_ + hi_;
          ptx::unpack_f32x2(s2a, lo_, hi_); n2_a = lo_ + hi_;
          ptx::unpack_f32x2(d2b, lo_, hi_); dot_b = lo_ + hi_;
          ptx::unpack_f32x2(s2b, lo_, hi_); n2_b = lo_ + hi_;
        }
        val[4 * u + 0] = dot_a;
        val[4 * u + 1] = n2_a;
        val[4 * u + 2] = dot_b;
        val[4 * u + 3] = n2_b;
      }
      // Sum over the 16 lanes that hold a head's 128 columns, all 16 sums at once: at every step a lane keeps the half of
      // its sums that its lane bit selects and hands the other half to its partner (8 + 4 + 2 + 1 shuffles instead of
      // 16 x 4); lane l of the half-warp ends with sum number l, added in the same butterfly order as half_warp_sum.
#pragma unroll
      for (int step = 0; step < 4; ++step) {
        const int o = 8 >> step, n_keep_vals = 8 >> step;
        const bool upper = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < n_keep_vals; ++i) {
          const float keep = upper ? val[i + n_keep_vals] : val[i];
          const float send = upper ? val[i] : val[i + n_keep_vals];
          val[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
      }
      // sum number l = 4 u + k: k = 0 / 2 are the dots of rows j / jb, their squared norms sit one lane up
      const float n2 = __shfl_down_sync(0xffffffffu, val[0], 1);
      const int l16 = lane & 15, u_of = l16 >> 2, k_of = l16 & 3;
      const int v_of = v0 - lane + 32 * u_of + (lane & 16);   // a column group of this lane's half-warp and group u_of
      const int head = v_of >> 4;
      if ((k_of & 1) == 0 && v_of < vecs && head < H && (k_of == 0 || has_b)) {
        const float dot = val[0];
        const float sc = n2 == 0.f ? 0.f : __fdiv_rn(dot, __fsqrt_rn(n2));   // a NaN norm stays NaN and is reported
        if (!isfinite(sc)) atomicOr(status, WK_DEV_NONFINITE);
        const int64_t at = (static_cast<int64_t>(chunk) * H + head) * NA + (k_of ? jb : j);
        s32[at] = sc;
        if (scores_out) scores_out[at] = sc;
      }
    }
  }
}

}  // namespace

namespace {

template <int VPL, int NW>
void launch_rows(dim3 grid, size_t smem, cudaStream_t s, const __nv_bfloat16* K, int64_t stride, int chunks, int T, int D,
                 int hs, int wpr, int R, double* partial, int max_parts, uint32_t* tickets, double* m64, float* m32,
                 double* mnorm) {
  if (smem > 40 * 1024)   // the kernel's static shared memory comes on top
    cudaFuncSetAttribute(anchor_rows<VPL, NW>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  anchor_rows<VPL, NW><<<grid, NW * 32, smem, s>>>(K, stride, chunks, T, D, hs, wpr, R, partial, max_parts, tickets, m64, m32,
                                                   mnorm);
}

template <int VPT>
void launch_fused(unsigned grid, size_t smem, cudaStream_t s, const __nv_bfloat16* K, int64_t stride, int chunks, int T, int NA,
                  int D, int n_keep, int G, int rpp, int parts, int nblk, int layer_ctas, double* partial, int max_parts,
                  uint32_t* tickets_a, uint32_t* tickets_s, uint32_t* ready, FusedQueue* q, uint32_t epoch, double* m64,
                  float* m32, double* mnorm, float* s32, float* scores_out, int32_t* keep_idx, uint32_t* status) {
  if (smem > 48 * 1024)
    cudaFuncSetAttribute(compress_fused<VPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  compress_fused<VPT><<<grid, kAnchorThreads, smem, s>>>(K, stride, chunks, T, NA, D, n_keep, G, rpp, parts, nblk, layer_ctas,
                                                         partial, max_parts, tickets_a, tickets_s, ready, q, epoch, m64, m32,
                                                         mnorm, s32, scores_out, keep_idx, status);
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
  uint32_t* tickets = reinterpret_cast<uint32_t*>(sc + ctx->sl.cnt_off);   // [2][max_batch]: anchor pass, score pass
  const int max_parts = ctx->sl.anchor_parts;
  const bool need_scores = (n_keep > 0 && n_keep < NA) || scores_out != nullptr;
  const size_t smem_sel = static_cast<size_t>(NA) * (4 + 4 + 8 + 1) + 16;
  const size_t smem_m = static_cast<size_t>(DF) * sizeof(float);
  if (smem_sel > 200 * 1024 || smem_m > 200 * 1024) return WK_ERR_SHAPE;
  wk_status st = WK_OK;
  if (need_scores) {
    const bool select_here_f = !per_head && n_keep > 0 && n_keep < NA;
    if (DF <= 8192 && select_here_f && DF > kFusedMinCols) {
      // wide whole-token keys with a real selection: both passes in one launch (anchor CTAs and score CTAs side by side)
      // rows per group: two groups of G rows of DF bf16 in shared memory, at most one row per warp
      int G = kAnchorWarps;
      while (G > 1 && 2 * static_cast<size_t>(G) * DF * 2 > 100 * 1024) G >>= 1;
      const int nseg = kAnchorWarps / G;
      const size_t smem_a = 2 * static_cast<size_t>(G) * DF * 2 + static_cast<size_t>(G) * (1 + nseg) * sizeof(double);
      const int vpt = (DF / 8 + kAnchorThreads - 1) / kAnchorThreads;   // 2 .. 4 here
      const int nblk = (NA + kFusedScoreRows - 1) / kFusedScoreRows;
      const size_t smem_s = smem_sel > smem_m ? smem_sel : smem_m;
      const size_t smem_f = smem_a > smem_s ? smem_a : smem_s;
      // persistent grid: what fits the machine at this shared-memory size
      int per_sm = static_cast<int>((220 * 1024) / (smem_f + 2048));
      const int by_regs = vpt == 1 ? 4 : (vpt == 2 ? 3 : 2);
      if (per_sm > by_regs) per_sm = by_regs;
      if (per_sm < 1) per_sm = 1;
      // slices per chunk: about a third more than CTA slots (measured: shorter items even out the end of the launch;
      // flat between 1.2 and 1.6 slots' worth)
      int parts = (ctx->sm_count * per_sm * 27 / 20 + chunks - 1) / chunks;
      if (parts < 1) parts = 1;
      if (parts > max_parts) parts = max_parts;
      if (parts > (T + G - 1) / G) parts = (T + G - 1) / G;
      int rpp = (T + parts - 1) / parts;
      rpp = (rpp + G - 1) / G * G;            // whole groups, so that only a chunk's last slice has a short group
      parts = (T + rpp - 1) / rpp;
      unsigned grid_f = static_cast<unsigned>(ctx->sm_count * per_sm);
      const unsigned items = static_cast<unsigned>(chunks) * static_cast<unsigned>(parts + nblk);
      if (grid_f > items) grid_f = items;
      uint32_t* ready = tickets + 2 * ctx->max_batch;
      FusedQueue* q = reinterpret_cast<FusedQueue*>(tickets + 3 * ctx->max_batch);
      const uint32_t epoch = ++ctx->compress_epoch;
#define WK_FUSED(V) launch_fused<V>(grid_f, smem_f, s, K, stride, chunks, T, NA, DF, n_keep, G, rpp, parts, nblk, ctx->sm_count, partial, max_parts, tickets, tickets + ctx->max_batch, ready, q, epoch, m64, m32, mnorm, s32, scores_out, keep_idx, ctx->status_dev)
      if (vpt <= 1) WK_FUSED(1);
      else if (vpt == 2) WK_FUSED(2);
      else if (vpt == 3) WK_FUSED(3);
      else WK_FUSED(4);
#undef WK_FUSED
      return after_launch(ctx);
    } else if (DF <= 8192) {
      // warps per row: the fewest that leave a lane at most the mode's number of 16-byte column groups
      const int vecs = DF / 8;
      const int nw = per_head ? kRowWarpsHead : kRowWarpsWhole;
      const int max_vpl = per_head ? kRowMaxVplHead : kRowMaxVplWhole;
      int wpr = 1;
      while (wpr < nw && (vecs + 32 * wpr - 1) / (32 * wpr) > max_vpl) wpr <<= 1;
      const int vpl = (vecs + 32 * wpr - 1) / (32 * wpr);
      const int n_sets = nw / wpr;
      const int hs = per_head ? H : 1;
      const size_t smem_r = static_cast<size_t>(n_sets) * DF * sizeof(double);
      // rows per CTA: an even share of all chunks' anchor rows, and never so few that a chunk is cut into more slices
      // than the scratch holds
      const int64_t total = static_cast<int64_t>(chunks) * T;
      int64_t R = (total + ctx->sm_count - 1) / ctx->sm_count;
      const int64_t r_min = (T + max_parts - 2) / (max_parts - 1);
      if (R < r_min) R = r_min;
      const dim3 grid(static_cast<unsigned>((total + R - 1) / R));
#define WK_ROWS(V, W) launch_rows<V, W>(grid, smem_r, s, K, stride, chunks, T, DF, hs, wpr, static_cast<int>(R), partial, max_parts, tickets, m64, m32, mnorm)
      if (per_head) {
        switch (vpl) {
          case 1: WK_ROWS(1, kRowWarpsHead); break;
          case 2: WK_ROWS(2, kRowWarpsHead); break;
          default: WK_ROWS(3, kRowWarpsHead); break;
        }
      } else {
        switch (vpl) {
          case 1: WK_ROWS(1, kRowWarpsWhole); break;
          case 2: WK_ROWS(2, kRowWarpsWhole); break;
          case 3: WK_ROWS(3, kRowWarpsWhole); break;
          case 4: WK_ROWS(4, kRowWarpsWhole); break;
          case 5: WK_ROWS(5, kRowWarpsWhole); break;
          default: WK_ROWS(6, kRowWarpsWhole); break;
        }
      }
#undef WK_ROWS
    } else {
      if (per_head) return WK_ERR_SHAPE;   // rows wider than 8,192 columns take the whole-key fallback only
      const dim3 grid_a(max_parts, chunks);
      const size_t smem_acc = static_cast<size_t>(DF) * sizeof(double);
      if (smem_acc > 200 * 1024) return WK_ERR_SHAPE;
      WK_CUDA_TRY(ctx, cudaFuncSetAttribute(anchor_pass_wide, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(smem_acc)));
      anchor_pass_wide<<<grid_a, kAnchorThreads, smem_acc, s>>>(K, stride, T, DF, max_parts, partial, tickets, m64, m32,
                                                                mnorm);
    }
    if ((st = after_launch(ctx)) != WK_OK) return st;
    // blocks of rows of score_select / head_score: whole rounds of its 8 warps x 2 rows, and as few full waves of CTAs (four resident
    // per SM) as blocks of at most 128 rows allow -- a last wave that is nearly empty costs as much as a full one
    int srows = 128;
    for (int waves = 1; waves <= 64; ++waves) {
      const int64_t per = (static_cast<int64_t>(NA) * chunks + static_cast<int64_t>(ctx->sm_count) * 4 * waves - 1) /
                          (static_cast<int64_t>(ctx->sm_count) * 4 * waves);
      const int r16 = static_cast<int>((per + 15) / 16 * 16);
      if (r16 <= 128) { srows = r16 < 16 ? 16 : r16; break; }
    }
    const int nblk = (NA + srows - 1) / srows;
    if (per_head) {
      if (smem_m > 48 * 1024)
        WK_CUDA_TRY(ctx, cudaFuncSetAttribute(head_score, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_m)));
      launch_chained(head_score, dim3(nblk, chunks), dim3(kScoreThreads), smem_m, s, K, stride, T, NA, DF, H, m32, s32,
                     scores_out, ctx->status_dev);
      if ((st = after_launch(ctx)) != WK_OK) return st;
    } else {
      const bool select_here = n_keep > 0 && n_keep < NA;
      const size_t smem_s = select_here && smem_sel > smem_m ? smem_sel : smem_m;
      if (smem_s > 48 * 1024)
        WK_CUDA_TRY(ctx, cudaFuncSetAttribute(score_select, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_s)));
      launch_chained(score_select, dim3(static_cast<unsigned>(nblk) * chunks), dim3(kScoreThreads), smem_s, s, K, stride, T, NA,
                     DF, n_keep, nblk, m32, m64, mnorm, s32, scores_out, tickets + ctx->max_batch,
                     select_here ? keep_idx : static_cast<int32_t*>(nullptr), ctx->status_dev);
      if ((st = after_launch(ctx)) != WK_OK) return st;
      if (select_here) return WK_OK;
    }
  }
  // per-head keys, and the cases that need no scores (n_keep = 0 or everything kept): a selection launch of its own
  if (smem_sel > 48 * 1024) {
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(select_pass<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem_sel)));
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(select_pass<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem_sel)));
  }
  if (per_head)
    launch_chained(select_pass<true>, dim3(batch), dim3(kSelectThreads), smem_sel, s, K, rm, T, NA, D, n_keep, s32, m64, mnorm,
                   keep_idx, ctx->status_dev);
  else
    launch_chained(select_pass<false>, dim3(batch), dim3(kSelectThreads), smem_sel, s, K, rm, T, NA, D, n_keep, s32, m64, mnorm,
                   keep_idx, ctx->status_dev);
  return after_launch(ctx);
}

}  // namespace wk
