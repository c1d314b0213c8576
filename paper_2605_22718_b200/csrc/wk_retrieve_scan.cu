// World Retrieval (Eq. 4, distance of Section 5.1) over a pose array of any length: the same fp64 arithmetic and the
// same tie rule as retrieve_kernel, organised so that millions of candidates are read from memory ONCE.
//
// The distance d_i = t_i / max t + r_i / max r needs both maxima, which are only known after every pose has been seen.
// What can be decided earlier: if k real candidates ("pivots") are certain to be closer than candidate j whatever the
// two maxima turn out to be, j is not among the k best.  With T* / R* the largest translation / rotation term of the
// pivots, mt_lo any lower bound of max t, and max r <= pi (an angle), that holds when
//       r_j > R* + (pi / mt_lo) * max(0, T* - t_j)
// (a pivot with the larger translation term loses at most (T* - t_j) / mt_lo there and gains at least (r_j - R*) / pi).
//
//   scan_sample  a strided sample of the candidates (one in 128, 2^15 .. 2^18 of them): per block the largest t,
//                and for each of k disjoint sample classes the candidate with the smallest r + pi t / (roughly max t),
//                in fp32 -- pivots only have to be real candidates, not the best ones
//   scan_filter  the single pass over all poses: every block first merges the sample blocks' records and takes the
//                pivots' exact fp64 terms (T*, R*, mt_lo); then per candidate a dozen fp32 operations: the test above
//                with every quantity rounded to the safe side, and running fp32 maxima -- the exact fp64 terms are
//                only formed for a candidate whose fp32 value comes within rounding of the thread's record, so the true
//                maxima are never missed.  Survivors (typically 1-2 %) go to an index list
//   scan_select  the exact distances of the listed candidates with the final maxima: every block keeps its k best by
//                rank counting under (distance, index).  If the list overflowed (poses that cannot be pruned, e.g. all
//                rotations equal) it walks all poses instead: the two-read path, slower but always right.  The block
//                that hands in its list last (atomic ticket) merges the lists and writes the result in rank order
//
// Nothing here depends on the order in which threads or blocks run: the k best under (distance, index) are unique, and
// a non-finite pose is never a candidate (it sets WK_DEV_NONFINITE).
#include "wk_internal.cuh"

namespace wk {
namespace {

constexpr int kScanMaxK = 64;
constexpr int kScanThreads = 256;
constexpr int kScanUnroll = 4;       // candidates per thread and round after the first
constexpr int kScanLow = 256;        // a list longer than this is cut back to k at the end of the round
constexpr int kSelThreads = 512;     // scan_select: two blocks per SM, so that one loads while the other is at a barrier
constexpr int kScanWarm = 256;       // candidates of the first, list-seeding round
constexpr int kPendLow = 256;        // survivors of the cheap bound are decided once this many have gathered
constexpr int kScanCap = kScanLow + kSelThreads + 64;   // between two checks at most one entry per thread is added
constexpr int kScanMaxBlocks = 1024;

constexpr int kSampleBlocks = 128;          // scan_sample's grid
constexpr int kSampleThreads = 256;
constexpr int kSampleBatch = 4;             // samples a thread has in flight
constexpr uint32_t kSurvivorCap = 1u << 20;  // entries of the survivor list

struct ScanHeader {
  unsigned long long t_max_bits;     // max squared translation distance, as the bits of a non-negative double
  unsigned long long dot_min_bits;   // min |<q_cur, q_i>|, likewise
  uint32_t n_surv;                   // survivors appended so far (may exceed the capacity: then `overflow` is set)
  uint32_t overflow;
  uint32_t ticket;                   // blocks of the exact pass that have handed in their list
  uint32_t pad;
};
// one record per scan_sample block
struct SampleRecord {
  double t_max;                              // largest squared translation distance among the block's samples (fp32 value)
  double dot_min;                            // smallest |quaternion dot| among them (fp32 value; 2 = none)
  unsigned long long best[kScanMaxK];        // per class: (fp32 key bits << 32) | candidate index; ~0 = none
};
struct ScanEntry {
  double d;
  int32_t i;      // -1: empty
  int32_t pad;
};

struct Cand {
  double t;       // squared translation distance
  double adot;    // |quaternion dot|
};
// Same operations in the same order as retrieve_kernel, so that both entry points give the same distances.
__device__ __forceinline__ Cand candidate(const float4 a, const float4 b, const float* cur) {
  Cand c;
  const double dx = static_cast<double>(a.x) - static_cast<double>(cur[0]);
  const double dy = static_cast<double>(a.y) - static_cast<double>(cur[1]);
  const double dz = static_cast<double>(a.z) - static_cast<double>(cur[2]);
  c.t = dx * dx + dy * dy + dz * dz;
  const double dot = static_cast<double>(b.x) * cur[4] + static_cast<double>(b.y) * cur[5] +
                     static_cast<double>(b.z) * cur[6] + static_cast<double>(b.w) * cur[7];
  c.adot = fabs(dot);
  return c;
}

struct Cur8 { float v[8]; };

// fp32 surrogates of a candidate's two terms, from the fp32 inputs: t32 = squared translation distance (relative error
// below 1e-6), adot32 = |quaternion dot| (absolute error below 4e-7 for unit quaternions).
__device__ __forceinline__ void cheap_terms(const float4 a, const float4 b, const float* cur, float& t32, float& adot32) {
  const float dx = a.x - cur[0], dy = a.y - cur[1], dz = a.z - cur[2];
  t32 = dx * dx + dy * dy + dz * dz;
  adot32 = fabsf(b.x * cur[4] + b.y * cur[5] + b.z * cur[6] + b.w * cur[7]);
}
// lower bound of the rotation term 2 acos(|dot|): acos(x) >= sqrt(2 (1 - x)) on [0, 1]; 4e-7 covers the fp32 dot
__device__ __forceinline__ float rot_lower_bound(float adot32) {
  const float om = fmaxf(0.f, 1.f - adot32 - 4e-7f);
  return 2.f * sqrtf(om + om) * (1.f - 3e-6f);
}

__global__ void __launch_bounds__(kSampleThreads)
scan_sample(const float4* __restrict__ poses, const int32_t* __restrict__ valid, int64_t n, int64_t n_samples, Cur8 cur,
            int k, ScanHeader* __restrict__ h, SampleRecord* __restrict__ rec) {
  __shared__ float s_tmax[kSampleThreads / 32], s_dmin[kSampleThreads / 32];
  __shared__ unsigned long long s_best[kScanMaxK];
  dep_release();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (blockIdx.x == 0 && tid == 0) {   // the header fields scan_filter accumulates into
    h->t_max_bits = 0ull;
    h->dot_min_bits = static_cast<unsigned long long>(__double_as_longlong(2.0));
    h->n_surv = 0u;
    h->overflow = 0u;
    h->ticket = 0u;
  }
  for (int g = tid; g < kScanMaxK; g += kSampleThreads) s_best[g] = ~0ull;
  // sample s is candidate floor(s * n / n_samples) (integer arithmetic); block b takes samples b, b + gridDim.x, ...; class of a sample =
  // its position in the block's sequence modulo k, so that classes are disjoint sets of candidates
  const int64_t per_block = (n_samples + gridDim.x - 1) / gridDim.x;
  // A thread takes positions tid, tid + 256, ... of the block's sequence, kSampleBatch at a time: the loads of a batch
  // are all issued before the first is used, so that a batch is one trip to memory instead of four in a row.  (What is
  // left is the rate at which DRAM opens rows: every sample is a 32-byte read from a row of its own.)
  // The weight pi / (largest t) of the key comes from the block's first 256 samples (any positive weight gives valid
  // pivots, a rough one just picks slightly different ones); the record's t_max covers all of the block's samples.
  float tmax = 0.f, dmin = 2.f, wt = 0.f;
  for (int64_t q0 = 0; q0 < per_block; q0 += kSampleBatch * kSampleThreads) {   // the same trips for every thread
    float4 a[kSampleBatch], b[kSampleBatch];
    int64_t ci[kSampleBatch];
    int vflag[kSampleBatch];
    bool ok[kSampleBatch];
#pragma unroll
    for (int u = 0; u < kSampleBatch; ++u) {
      const int64_t q = q0 + u * kSampleThreads + tid;
      const int64_t smp = q * gridDim.x + blockIdx.x;
      ok[u] = q < per_block && smp < n_samples;
      ci[u] = ok[u] ? smp * n / n_samples : 0;   // n_samples <= n: strictly increasing in smp, so samples are distinct
      vflag[u] = 1;
      a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      b[u] = a[u];
      if (ok[u]) {
        if (valid) vflag[u] = __ldg(valid + ci[u]);
        a[u] = __ldg(poses + 2 * ci[u]);
        b[u] = __ldg(poses + 2 * ci[u] + 1);
      }
    }
    float t32[kSampleBatch], ad32[kSampleBatch];
#pragma unroll
    for (int u = 0; u < kSampleBatch; ++u) {
      cheap_terms(a[u], b[u], cur.v, t32[u], ad32[u]);
      ok[u] = ok[u] && vflag[u] != 0 && t32[u] < 3.0e38f && ad32[u] < 3.0e38f;   // false for NaN and Inf: not a candidate
    }
    if (q0 == 0) {
      float est = ok[0] ? t32[0] : 0.f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) est = fmaxf(est, __shfl_xor_sync(0xffffffffu, est, o));
      if (lane == 0) s_tmax[warp] = est;
      __syncthreads();
      est = s_tmax[0];
      for (int w = 1; w < kSampleThreads / 32; ++w) est = fmaxf(est, s_tmax[w]);
      __syncthreads();
      wt = est > 0.f ? 3.14159274f / est : 0.f;
    }
#pragma unroll
    for (int u = 0; u < kSampleBatch; ++u) {
      if (!ok[u]) continue;
      tmax = fmaxf(tmax, t32[u]);
      dmin = fminf(dmin, ad32[u]);
      if (k > 0) {
        const float om = fmaxf(0.f, 1.f - ad32[u]);
        const float key = 2.f * sqrtf(om + om) + wt * t32[u];   // ~ r + pi t / max t, non-negative
        atomicMin(&s_best[static_cast<int>((q0 + u * kSampleThreads + tid) % k)],
                  (static_cast<unsigned long long>(__float_as_uint(key)) << 32) | static_cast<unsigned long long>(ci[u]));
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    dmin = fminf(dmin, __shfl_xor_sync(0xffffffffu, dmin, o));
  }
  if (lane == 0) { s_tmax[warp] = tmax; s_dmin[warp] = dmin; }
  __syncthreads();
  tmax = s_tmax[0];
  dmin = s_dmin[0];
  for (int w = 1; w < kSampleThreads / 32; ++w) { tmax = fmaxf(tmax, s_tmax[w]); dmin = fminf(dmin, s_dmin[w]); }
  __syncthreads();
  SampleRecord* my = rec + blockIdx.x;
  if (tid == 0) { my->t_max = static_cast<double>(tmax); my->dot_min = static_cast<double>(dmin); }
  for (int g = tid; g < kScanMaxK; g += kSampleThreads) my->best[g] = s_best[g];
}

// The single pass over all poses.
__global__ void __launch_bounds__(kScanThreads, 4)
scan_filter(const float4* __restrict__ poses, const int32_t* __restrict__ valid, int64_t n, Cur8 cur, int k,
            const SampleRecord* __restrict__ rec, int n_rec, ScanHeader* __restrict__ h, uint32_t* __restrict__ surv,
            uint32_t* __restrict__ status) {
  __shared__ double s_t[kScanMaxK], s_r[kScanMaxK];
  __shared__ float s_Tstar, s_Rstar, s_slope, s_rec_t, s_rec_d;
  __shared__ double s_mt[kScanThreads / 32], s_md[kScanThreads / 32];
  dep_wait();
  dep_release();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // ---- pivots: per class the best record over the sample blocks (four threads per class, a quarter of the records
  // each), then the exact terms of those k candidates
  __shared__ unsigned long long s_best[kScanMaxK];
  if (tid < kScanMaxK) s_best[tid] = ~0ull;
  __syncthreads();
  {
    const int g = tid & (kScanMaxK - 1), part = tid >> 6;   // 256 threads = 64 classes x 4 parts
    if (g < k) {
      unsigned long long best = ~0ull;
      for (int b = part; b < n_rec; b += kScanThreads / kScanMaxK) {
        const unsigned long long v = __ldcg(&rec[b].best[g]);
        best = v < best ? v : best;
      }
      if (best != ~0ull) atomicMin(&s_best[g], best);
    }
    double tm = tid < n_rec ? __ldcg(&rec[tid].t_max) : 0.0;   // n_rec <= 128 < 256 threads
    double dm = tid < n_rec ? __ldcg(&rec[tid].dot_min) : 2.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      tm = fmax(tm, __shfl_xor_sync(0xffffffffu, tm, o));
      dm = fmin(dm, __shfl_xor_sync(0xffffffffu, dm, o));
    }
    if (lane == 0) { s_mt[warp] = tm; s_md[warp] = dm; }
  }
  __syncthreads();
  if (tid < kScanMaxK) {
    double t = -1.0, r = -1.0;   // negative: no pivot in this class
    if (tid < k && s_best[tid] != ~0ull) {
      const int64_t i = static_cast<int64_t>(s_best[tid] & 0xFFFFFFFFull);
      const Cand c = candidate(__ldg(poses + 2 * i), __ldg(poses + 2 * i + 1), cur.v);
      if (isfinite(c.t) && isfinite(c.adot)) {
        t = c.t;
        r = 2.0 * acos(fmin(1.0, c.adot));
      }
    }
    s_t[tid] = t;
    s_r[tid] = r;
  }
  __syncthreads();
  if (tid == 0) {
    double mt_lo = 0.0, md_hi = 2.0;
    for (int w = 0; w < kScanThreads / 32; ++w) { mt_lo = fmax(mt_lo, s_mt[w]); md_hi = fmin(md_hi, s_md[w]); }
    // the sample's records seed every thread's: a candidate below them (by more than fp32 rounding) cannot hold a maximum
    s_rec_t = static_cast<float>(mt_lo);
    s_rec_d = static_cast<float>(md_hi);
    mt_lo *= 1.0 - 2e-6;   // the records hold fp32 values: below the true maximum after this
    double Ts = 0.0, Rs = 0.0;
    bool all = k > 0;
    for (int g = 0; g < k; ++g) {
      all = all && s_t[g] >= 0.0;
      Ts = fmax(Ts, s_t[g]);
      Rs = fmax(Rs, s_r[g]);
    }
    if (!all) {             // fewer than k pivots: nothing can be ruled out
      s_Tstar = INFINITY;
      s_Rstar = INFINITY;
      s_slope = 0.f;
    } else {                // every quantity rounded to the side that keeps more candidates
      s_Tstar = Ts < 3.0e38 ? __double2float_ru(Ts * (1.0 + 1e-6)) : INFINITY;
      s_Rstar = __double2float_ru(Rs * (1.0 + 1e-6));
      s_slope = (Ts > 0.0 && mt_lo > 0.0) ? __double2float_ru(3.1415927 / mt_lo * (1.0 + 1e-6)) : (Ts > 0.0 ? INFINITY : 0.f);
    }
  }
  __syncthreads();
  const float Tstar = s_Tstar, Rstar = s_Rstar, slope = s_slope;
  // ---- the stream
  __shared__ uint32_t s_wbuf[kScanThreads / 32][64];
  uint32_t* wbuf = s_wbuf[warp];
  int wcnt = 0;                          // entries in the warp's buffer (the same value in all 32 lanes)
  auto flush = [&]() {
    uint32_t base = 0;
    if (lane == 0) base = atomicAdd(&h->n_surv, static_cast<uint32_t>(wcnt));
    base = __shfl_sync(0xffffffffu, base, 0);
    for (int j = lane; j < wcnt; j += 32) {
      if (base + j < kSurvivorCap) surv[base + j] = wbuf[j];
      else h->overflow = 1u;
    }
    __syncwarp();
  };
  float rec_t = s_rec_t, rec_d = s_rec_d;   // this thread's fp32 records, seeded with the sample's
  double mt = 0.0, mdot = 2.0;           // exact maxima over the candidates whose fp32 value came near the record
  bool bad = false;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kScanThreads;
  // the loop bound is the warp's first index, so that all 32 lanes make the same number of trips (the survivor
  // bookkeeping below uses warp-wide votes); lanes past the end just have nothing live
  for (int64_t i0 = static_cast<int64_t>(blockIdx.x) * kScanThreads + tid; i0 - lane < n; i0 += kScanUnroll * stride) {
    float4 a[kScanUnroll], b[kScanUnroll];
    bool live[kScanUnroll];
#pragma unroll
    for (int u = 0; u < kScanUnroll; ++u) {
      const int64_t i = i0 + u * stride;
      live[u] = i < n && !(valid && !__ldg(valid + i));
      if (live[u]) {
        a[u] = __ldg(poses + 2 * i);
        b[u] = __ldg(poses + 2 * i + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < kScanUnroll; ++u) {
      bool keep = false;
      if (live[u]) {
        float t32, adot32;
        cheap_terms(a[u], b[u], cur.v, t32, adot32);
        // exact terms only near a record (also for NaN / overflow, which fail both comparisons' negations)
        if (!(t32 * (1.f + 4e-6f) < rec_t) || !(adot32 * (1.f - 4e-6f) - 2e-6f > rec_d)) {
          const Cand c = candidate(a[u], b[u], cur.v);
          if (isfinite(c.t) && isfinite(c.adot)) {
            mt = fmax(mt, c.t);
            mdot = fmin(mdot, c.adot);
            rec_t = fmaxf(rec_t, t32);
            rec_d = fminf(rec_d, adot32);
          } else {
            bad = true;
            live[u] = false;
          }
        }
        if (live[u]) {
          const float gap = fmaxf(0.f, Tstar - t32 * (1.f - 3e-6f));
          keep = !(rot_lower_bound(adot32) > Rstar + slope * gap);   // NaN on either side keeps the candidate
        }
      }
      // survivors gather in a buffer of the warp's own (no block barrier anywhere in the stream); a full buffer takes
      // consecutive places in the list with one atomic for the lot
      const unsigned m = __ballot_sync(0xffffffffu, keep);
      if (m) {
        if (keep) wbuf[wcnt + __popc(m & ((1u << lane) - 1u))] = static_cast<uint32_t>(i0 + u * stride);
        wcnt += __popc(m);
        __syncwarp();
        if (wcnt >= 32) {
          flush();
          wcnt = 0;
        }
      }
    }
  }
  {
    // what is left in the warps' buffers at the end: one atomic for the whole block (every warp of every block arrives
    // here at about the same time, and thousands of atomics on one word would queue up)
    __shared__ int s_wcnt[kScanThreads / 32];
    __shared__ uint32_t s_base;
    if (lane == 0) s_wcnt[warp] = wcnt;
    __syncthreads();
    if (tid == 0) {
      int total = 0;
      for (int w = 0; w < kScanThreads / 32; ++w) total += s_wcnt[w];
      s_base = total > 0 ? atomicAdd(&h->n_surv, static_cast<uint32_t>(total)) : 0u;
    }
    __syncthreads();
    uint32_t base = s_base;
    for (int w = 0; w < warp; ++w) base += static_cast<uint32_t>(s_wcnt[w]);
    for (int j = lane; j < wcnt; j += 32) {
      if (base + j < kSurvivorCap) surv[base + j] = wbuf[j];
      else h->overflow = 1u;
    }
  }
  if (bad) atomicOr(status, WK_DEV_NONFINITE);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mt = fmax(mt, __shfl_xor_sync(0xffffffffu, mt, o));
    mdot = fmin(mdot, __shfl_xor_sync(0xffffffffu, mdot, o));
  }
  if (lane == 0) { s_mt[warp] = mt; s_md[warp] = mdot; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kScanThreads / 32; ++w) { mt = fmax(mt, s_mt[w]); mdot = fmin(mdot, s_md[w]); }
    atomicMax(&h->t_max_bits, static_cast<unsigned long long>(__double_as_longlong(mt)));
    atomicMin(&h->dot_min_bits, static_cast<unsigned long long>(__double_as_longlong(mdot)));
  }
}

// Rank of each of n entries under (key, index), by counting, with all of the block's threads: P threads share an entry
// (each counts over every P-th other entry), P the largest power of two with n * P <= blockDim.x.  rank[] is shared
// memory of at least n words.  Ends with a block barrier.
__device__ __forceinline__ void block_rank(const unsigned long long* key, const int32_t* idx, int n, int* rank) {
  for (int e = threadIdx.x; e < n; e += blockDim.x) rank[e] = 0;
  __syncthreads();
  int shift = 0;
  while (shift < 5 && (n << (shift + 1)) <= static_cast<int>(blockDim.x)) ++shift;
  const int P = 1 << shift;
  for (int slot = threadIdx.x; slot < (n << shift); slot += blockDim.x) {
    const int e = slot >> shift, p = slot & (P - 1);
    const unsigned long long ke = key[e];
    const int32_t ie = idx[e];
    int r = 0;
#pragma unroll 4
    for (int u = p; u < n; u += P) {
      const unsigned long long ku = key[u];
      r += (ku < ke) || (ku == ke && idx[u] < ie);
    }
    if (r) atomicAdd(&rank[e], r);
  }
  __syncthreads();
}

// The k best (distance, index) pairs seen so far by one block, in shared memory.  Distances are non-negative, so their
// bit patterns order like the values and every comparison is an integer one.
struct TopK {
  unsigned long long* key;   // [2][kScanCap] distance bits
  int32_t* idx;              // [2][kScanCap]
  int* rank_s;               // [kScanCap] scratch of compact()
  int* cnt;                  // entries in the list
  double* tau;               // current k-th best distance (+inf until k entries are known)
  int k;

  __device__ __forceinline__ void init(unsigned long long* k_, int32_t* i_, int* r_, int* c_, double* t_, int kk) {
    key = k_; idx = i_; rank_s = r_; cnt = c_; tau = t_; k = kk;
    if (threadIdx.x == 0) { *cnt = 0; *tau = INFINITY; }
    __syncthreads();
  }
  __device__ __forceinline__ void push(double dist, int32_t i) {   // caller has checked dist <= *tau
    const int pos = atomicAdd(cnt, 1);
    key[pos] = static_cast<unsigned long long>(__double_as_longlong(dist));
    idx[pos] = i;
  }
  // Barrier at the end of a round of pushes; true (for every thread alike) when the list has grown past kScanLow and
  // is to be cut back.  The thread whose push came last reads the final count, so the OR over the block cannot miss it.
  __device__ __forceinline__ bool round_end() {
    return __syncthreads_or(*reinterpret_cast<volatile int*>(cnt) > kScanLow) != 0;
  }
  // Cuts the list back to its k best, sorted, by exact rank counting (quadratic in the list length, which is why the
  // list is kept short); all threads of the block call it together.
  __device__ __forceinline__ void compact() {
    __shared__ unsigned long long s_gmin[kScanMaxK];
    __shared__ unsigned long long s_cut;
    __shared__ int s_m;
    __syncthreads();
    const int n = *cnt;
    unsigned long long* key2 = key + kScanCap;
    int32_t* i2 = idx + kScanCap;
    // Counting ranks costs n^2 comparisons, so a long list is thinned first: deal the entries into k groups; the
    // largest of the groups' minima has k entries at or below it, so nothing above it is among the k best.
    const bool thin = k > 0 && n > 4 * k;
    if (threadIdx.x < kScanMaxK) s_gmin[threadIdx.x] = ~0ull;
    if (threadIdx.x == 0) { s_m = 0; s_cut = ~0ull; }
    __syncthreads();
    if (thin) {
      for (int e = threadIdx.x; e < n; e += blockDim.x) atomicMin(&s_gmin[e % k], key[e]);
      __syncthreads();
      if (threadIdx.x < 32) {
        unsigned long long v = 0ull;
        for (int g = threadIdx.x; g < k; g += 32) v = s_gmin[g] > v ? s_gmin[g] : v;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
          v = w > v ? w : v;
        }
        if (threadIdx.x == 0) s_cut = v;
      }
      __syncthreads();
    }
    const unsigned long long cut = s_cut;
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
      const unsigned long long ke = key[e];
      if (ke <= cut) {
        const int pos = atomicAdd(&s_m, 1);
        key2[pos] = ke;
        i2[pos] = idx[e];
      }
    }
    __syncthreads();
    const int n2 = s_m;
    block_rank(key2, i2, n2, rank_s);
    for (int e = threadIdx.x; e < n2; e += blockDim.x) {
      const int rank = rank_s[e];
      if (rank < k) { key[rank] = key2[e]; idx[rank] = i2[e]; }
    }
    const int m = n2 < k ? n2 : k;
    __syncthreads();
    if (threadIdx.x == 0) {
      *cnt = m;
      *tau = (m == k && k > 0) ? __longlong_as_double(static_cast<long long>(key[k - 1])) : INFINITY;
    }
    __syncthreads();
  }
  __device__ __forceinline__ double dist_at(int e) const { return __longlong_as_double(static_cast<long long>(key[e])); }
};

__global__ void __launch_bounds__(kSelThreads, 2)
scan_select(const float4* __restrict__ poses, const int32_t* __restrict__ valid_all, int64_t n_all, Cur8 cur,
            ScanHeader* __restrict__ h, const uint32_t* __restrict__ surv, int k,
            ScanEntry* __restrict__ block_out /*[gridDim.x][k]*/, int out_capacity, int32_t* __restrict__ ids_out,
            double* __restrict__ dist_out) {
  __shared__ unsigned long long s_key[2 * kScanCap];
  __shared__ int32_t s_i[2 * kScanCap];
  __shared__ int s_rank[2 * kScanCap];
  __shared__ __align__(8) int32_t s_pend[kPendLow + kScanUnroll * kSelThreads];   // candidates that passed the cheap bound
  __shared__ int s_cnt, s_npend[2];
  __shared__ uint32_t s_last;
  __shared__ unsigned long long s_min;
  __shared__ double s_tau;
  __shared__ float s_tau_hi;
  dep_wait();
  dep_release();
  TopK top;
  top.init(s_key, s_i, s_rank, &s_cnt, &s_tau, k);
  // what is walked: the survivor list, or -- if it overflowed -- every pose (entry e is then candidate e)
  const bool listed = h->overflow == 0u;
  const int64_t n = listed ? static_cast<int64_t>(h->n_surv) : n_all;
  const int32_t* valid = listed ? nullptr : valid_all;      // listed candidates have been checked already
  auto cand_of = [&](int64_t e) -> int32_t { return listed ? static_cast<int32_t>(__ldg(surv + e)) : static_cast<int32_t>(e); };
  const double mt = __longlong_as_double(static_cast<long long>(h->t_max_bits));
  const double mr = 2.0 * acos(fmin(1.0, __longlong_as_double(static_cast<long long>(h->dot_min_bits))));
  // Cheap lower bound of the distance, in fp32 from the fp32 inputs: acos(x) >= sqrt(2 (1 - x)) on [0, 1], so
  //   d >= t / mt + 2 sqrt(2 (1 - |dot|)) / mr.
  // Its rounding error is below 1e-6 relative once 4e-7 is taken off 1 - |dot| (the absolute error of the fp32 dot);
  // a candidate is dropped only when the bound exceeds tau by more than 2e-6 relative, so no candidate that belongs to
  // the k best is ever dropped.  Everything that passes is decided by the exact fp64 distance.
  const float inv_mt = mt > 0.0 ? static_cast<float>(1.0 / mt) : 0.f;
  const float inv_mr = mr > 0.0 ? static_cast<float>(2.0 / mr) : 0.f;
  auto refresh = [&]() {
    if (threadIdx.x == 0) {
      const double t = s_tau * (1.0 + 2e-6);
      s_tau_hi = t < 3.0e38 ? __double2float_ru(t) : INFINITY;
    }
    __syncthreads();
  };
  auto passes = [&](const float4 a, const float4 b) -> bool {
    const float dx = a.x - cur.v[0], dy = a.y - cur.v[1], dz = a.z - cur.v[2];
    const float t = dx * dx + dy * dy + dz * dz;
    const float dot = fabsf(b.x * cur.v[4] + b.y * cur.v[5] + b.z * cur.v[6] + b.w * cur.v[7]);
    const float om = fmaxf(0.f, 1.f - dot - 4e-7f);
    const float lb = t * inv_mt + sqrtf(om + om) * inv_mr;
    return !(lb > s_tau_hi) || t > 3.0e38f;   // an fp32 overflow of t says nothing about t / mt
  };
  // exact distance of one candidate, the arithmetic of retrieve_kernel
  auto exact_of = [&](const float4 pa, const float4 pb, int32_t i, double tau) {
    const Cand c = candidate(pa, pb, cur.v);
    if (!isfinite(c.t) || !isfinite(c.adot)) return;         // not a candidate (reported by the pass that read it first)
    const double rot = 2.0 * acos(fmin(1.0, c.adot));
    const double ta = mt > 0.0 ? c.t / mt : 0.0;
    const double rb = mr > 0.0 ? rot / mr : 0.0;
    const double dist = ta + rb;
    if (dist <= tau) top.push(dist, i);
  };
  auto exact = [&](int32_t i, double tau) {
    exact_of(__ldg(poses + 2 * static_cast<int64_t>(i)), __ldg(poses + 2 * static_cast<int64_t>(i) + 1), i, tau);
  };
  if (threadIdx.x == 0) s_npend[0] = s_npend[1] = 0;
  refresh();
  // The first pass over kScanWarm candidates cuts the list at once: that gives a first k-th best, after which few of
  // the later candidates pass the bound.  Later rounds take kScanUnroll candidates per thread.
  // (a survivor list needs no seeding: nearly all of it is wanted anyway, and the extra round trip to memory would
  // only lengthen a short kernel)
  const int64_t warm0 = static_cast<int64_t>(blockIdx.x) * kScanWarm;
  const int64_t warm_all = listed ? 0 : static_cast<int64_t>(gridDim.x) * kScanWarm;
  if (!listed) {
    if (k > 0 && threadIdx.x < kScanWarm) {
      const int64_t e = warm0 + threadIdx.x;
      if (e < n) {
        const int32_t i = cand_of(e);
        if (!(valid && !__ldg(valid + i))) exact(i, INFINITY);
      }
    }
    top.compact();
    refresh();
  }
  const int64_t step = static_cast<int64_t>(gridDim.x) * kSelThreads;
  const int64_t lane_off = warm_all + static_cast<int64_t>(blockIdx.x) * kSelThreads + threadIdx.x;
  const int64_t rest = n > warm_all ? n - warm_all : 0;
  const int64_t rounds = (rest + step * kScanUnroll - 1) / (step * kScanUnroll);
  // The survivors of the bound wait in s_pend until kPendLow of them have gathered (or the scan ends) and are then
  // decided one per thread with no idle lanes in between: the divisions and the acos are fp64, a warp pays for them in
  // full even when a single lane needs them, and their latency would otherwise sit in every round.
  auto drain = [&]() {
    const int np = s_npend[0];
    for (int e0 = 0; e0 < np; e0 += kSelThreads) {
      const double tau = s_tau;
      if (e0 + threadIdx.x < np) exact(s_pend[e0 + threadIdx.x], tau);
      if (top.round_end()) top.compact();
    }
    __syncthreads();
    if (threadIdx.x == 0) s_npend[0] = 0;
    refresh();
  };
  for (int64_t r = 0; r < rounds && k > 0; ++r) {
    float4 a[kScanUnroll], b[kScanUnroll];
    int32_t ci[kScanUnroll];
    bool live[kScanUnroll];
#pragma unroll
    for (int u = 0; u < kScanUnroll; ++u) {
      // a survivor list is dealt out entry by entry (block b takes entries b, b + gridDim.x, ...), so that a short list
      // is shared by all blocks; a full scan takes whole 512-pose runs per block, for coalesced loads
      const int64_t e = listed ? ((r * kScanUnroll + u) * kSelThreads + threadIdx.x) * gridDim.x + blockIdx.x
                               : (r * kScanUnroll + u) * step + lane_off;
      live[u] = e < n;
      if (live[u]) {
        ci[u] = cand_of(e);
        live[u] = !(valid && !__ldg(valid + ci[u]));
      }
      if (live[u]) {
        a[u] = __ldg(poses + 2 * static_cast<int64_t>(ci[u]));
        b[u] = __ldg(poses + 2 * static_cast<int64_t>(ci[u]) + 1);
      }
    }
    if (listed) {
      // listed candidates have passed a sharper test already: straight to the exact distance, one entry per thread
      // and list check (the list has room for one push per thread between checks)
#pragma unroll
      for (int u = 0; u < kScanUnroll; ++u) {
        if ((r * kScanUnroll + u) * kSelThreads * gridDim.x + blockIdx.x >= n) break;   // same for the whole block
        if (live[u]) exact_of(a[u], b[u], ci[u], s_tau);
        if (top.round_end()) top.compact();
      }
      continue;
    }
#pragma unroll
    for (int u = 0; u < kScanUnroll; ++u)
      if (live[u] && passes(a[u], b[u])) s_pend[atomicAdd(&s_npend[0], 1)] = ci[u];
    // the thread whose push came last reads the final count, so the OR over the block cannot miss a full list
    if (__syncthreads_or(*reinterpret_cast<volatile int*>(&s_npend[0]) > kPendLow)) drain();
  }
  __syncthreads();
  if (!listed) drain();
  top.compact();
  for (int e = threadIdx.x; e < k; e += blockDim.x) {
    ScanEntry o;
    o.d = e < s_cnt ? top.dist_at(e) : INFINITY;
    o.i = e < s_cnt ? s_i[e] : -1;
    o.pad = 0;
    __stcg(reinterpret_cast<double2*>(block_out + static_cast<int64_t>(blockIdx.x) * k + e),
           make_double2(o.d, __longlong_as_double((static_cast<long long>(static_cast<uint32_t>(o.pad)) << 32) |
                                                  static_cast<uint32_t>(o.i))));
  }
  // ---- hand in the list; the block that hands in last merges them all (nobody waits for anybody)
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&h->ticket, 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int n_lists = static_cast<int>(gridDim.x);
  const int tid = threadIdx.x;
  const unsigned long long kInf = static_cast<unsigned long long>(__double_as_longlong(INFINITY));
  auto entry = [&](int list, int e) -> ScanEntry {
    const double2 v = __ldcg(reinterpret_cast<const double2*>(block_out + static_cast<int64_t>(list) * k + e));
    ScanEntry x;
    x.d = v.x;
    x.i = static_cast<int32_t>(static_cast<uint32_t>(__double_as_longlong(v.y) & 0xFFFFFFFFll));
    x.pad = 0;
    return x;
  };
  for (int e = tid; e < out_capacity; e += blockDim.x) {
    ids_out[e] = -1;
    if (dist_out) dist_out[e] = 0.0;
  }
  if (tid == 0) { s_min = kInf; s_cnt = 0; h->ticket = 0u; }
  __syncthreads();
  if (k == 0) return;
  // A list that holds k entries proves that k candidates lie within its last distance: nothing beyond the smallest such
  // distance can be among the k best.  Every list is sorted, so what remains of it is a prefix.
  // Likewise the k-th smallest of the lists' first entries: k candidates lie within it.  With candidates dealt to the
  // blocks at random this is the sharper cut by far (it leaves little more than k entries).
  unsigned long long* heads = reinterpret_cast<unsigned long long*>(s_pend);   // [n_lists] <= 1024 (s_pend is free by now)
  for (int l = tid; l < n_lists; l += blockDim.x) {
    const ScanEntry x = entry(l, k - 1);
    if (x.i >= 0) atomicMin(&s_min, static_cast<unsigned long long>(__double_as_longlong(x.d)));
    const ScanEntry f = entry(l, 0);
    heads[l] = f.i >= 0 ? static_cast<unsigned long long>(__double_as_longlong(f.d)) : kInf;
  }
  __syncthreads();
  // (any k lists give a valid cut; the first 128 keep the counting short and still leave only a few k entries)
  const int n_heads = n_lists < 128 ? n_lists : 128;
  if (n_heads >= k) {
    for (int l = tid; l < n_heads; l += blockDim.x) {
      const unsigned long long hl = heads[l];
      int rank = 0;
      for (int u = 0; u < n_heads; ++u) {
        const unsigned long long hu = heads[u];
        rank += (hu < hl) || (hu == hl && u < l);
      }
      if (rank == k - 1 && hl != kInf) atomicMin(&s_min, hl);
    }
  }
  __syncthreads();
  const unsigned long long cut = s_min;
  __syncthreads();   // heads (in s_pend) is dead from here on
  constexpr int kGather = 2 * kScanCap;      // the two halves of the key / index arrays, free by now
  for (int l = tid; l < n_lists; l += blockDim.x) {
    for (int e = 0; e < k; ++e) {
      const ScanEntry x = entry(l, e);
      const unsigned long long key = static_cast<unsigned long long>(__double_as_longlong(x.d));
      if (x.i < 0 || key > cut) break;
      const int pos = atomicAdd(&s_cnt, 1);
      if (pos < kGather) { s_key[pos] = key; s_i[pos] = x.i; }
    }
  }
  __syncthreads();
  const int n_g = s_cnt;
  if (n_g <= kGather) {
    // exact rank under (distance, index) among the gathered entries
    block_rank(s_key, s_i, n_g, s_rank);
    for (int e = tid; e < n_g; e += blockDim.x) {
      const int rank = s_rank[e];
      if (rank < k && rank < out_capacity) {
        ids_out[rank] = s_i[e];
        if (dist_out) dist_out[rank] = __longlong_as_double(static_cast<long long>(s_key[e]));
      }
    }
    return;
  }
  // Too many entries at or below the cut (many equal distances): take the smallest head of the lists k times.  Thread
  // t walks lists t, t + blockDim.x, ...; s_pend holds each list's head position.
  __shared__ int s_win_idx;
  for (int l = tid; l < n_lists; l += blockDim.x) s_pend[l] = 0;
  for (int out = 0; out < k && out < out_capacity; ++out) {
    if (tid == 0) { s_min = kInf; s_win_idx = 0x7fffffff; }
    __syncthreads();
    for (int l = tid; l < n_lists; l += blockDim.x) {
      if (s_pend[l] < k) {
        const ScanEntry x = entry(l, s_pend[l]);
        if (x.i >= 0) atomicMin(&s_min, static_cast<unsigned long long>(__double_as_longlong(x.d)));
      }
    }
    __syncthreads();
    const unsigned long long best = s_min;
    if (best == kInf) break;
    for (int l = tid; l < n_lists; l += blockDim.x) {
      if (s_pend[l] < k) {
        const ScanEntry x = entry(l, s_pend[l]);
        if (x.i >= 0 && static_cast<unsigned long long>(__double_as_longlong(x.d)) == best) atomicMin(&s_win_idx, x.i);
      }
    }
    __syncthreads();
    const int win = s_win_idx;
    for (int l = tid; l < n_lists; l += blockDim.x) {
      if (s_pend[l] < k) {
        const ScanEntry x = entry(l, s_pend[l]);
        if (x.i == win) ++s_pend[l];
      }
    }
    if (tid == 0) {
      ids_out[out] = win;
      if (dist_out) dist_out[out] = __longlong_as_double(static_cast<long long>(best));
    }
    __syncthreads();
  }
}

}  // namespace

namespace {
struct ScanScratch {
  ScanHeader* h;
  SampleRecord* rec;
  uint32_t* surv;
  ScanEntry* block_out;
  size_t total;
};
ScanScratch carve(void* base) {
  ScanScratch sc;
  uint8_t* p = static_cast<uint8_t*>(base);
  size_t off = 0;
  sc.h = reinterpret_cast<ScanHeader*>(p + off);        off += align_up(sizeof(ScanHeader), 256);
  sc.rec = reinterpret_cast<SampleRecord*>(p + off);    off += align_up(sizeof(SampleRecord) * kSampleBlocks, 256);
  sc.surv = reinterpret_cast<uint32_t*>(p + off);       off += align_up(sizeof(uint32_t) * kSurvivorCap, 256);
  sc.block_out = reinterpret_cast<ScanEntry*>(p + off); off += static_cast<size_t>(kScanMaxBlocks) * kScanMaxK * sizeof(ScanEntry);
  sc.total = off;
  return sc;
}
}  // namespace

size_t retrieve_scan_scratch_bytes() { return carve(nullptr).total; }

wk_status launch_retrieve_scan(wk_ctx* ctx, const float* poses, const int32_t* valid, int64_t n, const float* cur_pose,
                               int k, int32_t* ids_out, double* dist_out, int out_capacity, void* scratch, cudaStream_t s) {
  const ScanScratch sc = carve(scratch);
  Cur8 cur;
  for (int i = 0; i < 8; ++i) cur.v[i] = cur_pose[i];
  // the sample: one candidate in 128, at least 2^15 (all of them below that), at most 2^18
  int64_t n_samples = n / 128;
  if (n_samples < (1 << 15)) n_samples = (1 << 15);
  if (n_samples > (1 << 18)) n_samples = (1 << 18);
  if (n_samples > n) n_samples = n;
  int sample_blocks = static_cast<int>((n_samples + kSampleThreads - 1) / kSampleThreads);
  if (sample_blocks > kSampleBlocks) sample_blocks = kSampleBlocks;
  if (sample_blocks < 1) sample_blocks = 1;
  // the stream: four resident 256-thread blocks per SM; the exact pass: two resident 512-thread blocks per SM
  int64_t blocks = static_cast<int64_t>(ctx->sm_count) * 4;
  const int64_t needed = (n + kScanThreads - 1) / kScanThreads;
  if (blocks > needed) blocks = needed;
  if (blocks < 1) blocks = 1;
  int64_t sel_blocks = static_cast<int64_t>(ctx->sm_count) * 2;
  const int64_t sel_needed = (n + kSelThreads - 1) / kSelThreads;
  if (sel_blocks > sel_needed) sel_blocks = sel_needed;
  if (sel_blocks > kScanMaxBlocks) sel_blocks = kScanMaxBlocks;
  if (sel_blocks < 1) sel_blocks = 1;
  wk_status st;
  const float4* p4 = reinterpret_cast<const float4*>(poses);
  scan_sample<<<sample_blocks, kSampleThreads, 0, s>>>(p4, valid, n, n_samples, cur, k, sc.h, sc.rec);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  launch_chained(scan_filter, dim3(static_cast<unsigned>(blocks)), dim3(kScanThreads), 0, s, p4, valid, n, cur, k, sc.rec,
                 sample_blocks, sc.h, sc.surv, ctx->status_dev);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  launch_chained(scan_select, dim3(static_cast<unsigned>(sel_blocks)), dim3(kSelThreads), 0, s, p4, valid, n, cur, sc.h,
                 sc.surv, k, sc.block_out, out_capacity, ids_out, dist_out);
  return after_launch(ctx);
}

}  // namespace wk
