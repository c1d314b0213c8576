// World Retrieval (Eq. 4, distance of Section 5.1) over a pose array of any length: the same fp64 arithmetic and the
// same tie rule as retrieve_kernel, organised as a streaming scan so that millions of candidates run at memory speed.
//
//   scan_init    resets the header (maxima, candidate count)
//   scan_max     pass 1: max squared translation distance and min |quaternion dot| over the valid candidates
//                (order-independent: integer atomics on the bit patterns of non-negative doubles)
//   scan_select  pass 2: every block keeps the k best (distance, index) pairs of its share.  A candidate is dropped
//                as soon as a lower bound of its distance exceeds the block's current k-th best, which spares most of
//                them the divisions and the acos; survivors go to a shared-memory list that is cut back to k by exact
//                rank counting whenever it fills
//   scan_merge   one block repeats that selection over the blocks' lists and writes the result in rank order
//
// Nothing here depends on the order in which threads or blocks run: the k best under (distance, index) are unique.
#include "wk_internal.cuh"

namespace wk {
namespace {

constexpr int kScanThreads = 256;
constexpr int kScanUnroll = 4;       // candidates per thread and round after the first
constexpr int kScanLow = 256;        // a list longer than this is cut back to k at the end of the round
constexpr int kSelThreads = 512;     // scan_select: two blocks per SM, so that one loads while the other is at a barrier
constexpr int kScanWarm = 256;       // candidates of the first, list-seeding round
constexpr int kPendLow = 256;        // survivors of the cheap bound are decided once this many have gathered
constexpr int kScanCap = kScanLow + kSelThreads + 64;   // between two checks at most one entry per thread is added
constexpr int kScanMaxK = 64;
constexpr int kScanMaxBlocks = 1024;
constexpr int kMergeThreads = 1024;

struct ScanHeader {
  unsigned long long t_max_bits;     // max squared translation distance, as the bits of a non-negative double
  unsigned long long dot_min_bits;   // min |<q_cur, q_i>|, likewise
  unsigned long long n_valid;
  unsigned long long reserved;
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

__global__ void scan_init(ScanHeader* h) {
  dep_release();
  h->t_max_bits = 0ull;
  h->dot_min_bits = static_cast<unsigned long long>(__double_as_longlong(2.0));
  h->n_valid = 0ull;
  h->reserved = 0ull;
}

__global__ void __launch_bounds__(kScanThreads)
scan_max(const float4* __restrict__ poses, const int32_t* __restrict__ valid, int64_t n, Cur8 cur, ScanHeader* h) {
  dep_wait();
  dep_release();
  double mt = 0.0, mdot = 2.0;
  unsigned int cnt = 0;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kScanThreads + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * kScanThreads) {
    if (valid && !__ldg(valid + i)) continue;
    const Cand c = candidate(__ldg(poses + 2 * i), __ldg(poses + 2 * i + 1), cur.v);
    mt = fmax(mt, c.t);
    mdot = fmin(mdot, c.adot);
    ++cnt;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mt = fmax(mt, __shfl_xor_sync(0xffffffffu, mt, o));
    mdot = fmin(mdot, __shfl_xor_sync(0xffffffffu, mdot, o));
    cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  }
  if ((threadIdx.x & 31) == 0 && cnt > 0) {
    atomicMax(&h->t_max_bits, static_cast<unsigned long long>(__double_as_longlong(mt)));
    atomicMin(&h->dot_min_bits, static_cast<unsigned long long>(__double_as_longlong(mdot)));
    atomicAdd(&h->n_valid, static_cast<unsigned long long>(cnt));
  }
}

// The k best (distance, index) pairs seen so far by one block, in shared memory.  Distances are non-negative, so their
// bit patterns order like the values and every comparison is an integer one.
struct TopK {
  unsigned long long* key;   // [2][kScanCap] distance bits
  int32_t* idx;              // [2][kScanCap]
  int* cnt;                  // entries in the list
  double* tau;               // current k-th best distance (+inf until k entries are known)
  int k;

  __device__ __forceinline__ void init(unsigned long long* k_, int32_t* i_, int* c_, double* t_, int kk) {
    key = k_; idx = i_; cnt = c_; tau = t_; k = kk;
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
    __syncthreads();
    const int n = *cnt;
    unsigned long long* key2 = key + kScanCap;
    int32_t* i2 = idx + kScanCap;
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
      const unsigned long long ke = key[e];
      const int32_t ie = idx[e];
      int rank = 0;
#pragma unroll 4
      for (int u = 0; u < n; ++u) {
        const unsigned long long ku = key[u];
        rank += (ku < ke) || (ku == ke && idx[u] < ie);
      }
      if (rank < k) { key2[rank] = ke; i2[rank] = ie; }
    }
    __syncthreads();
    const int m = n < k ? n : k;
    for (int e = threadIdx.x; e < m; e += blockDim.x) { key[e] = key2[e]; idx[e] = i2[e]; }
    if (threadIdx.x == 0) {
      *cnt = m;
      *tau = (m == k && k > 0) ? __longlong_as_double(static_cast<long long>(key2[k - 1])) : INFINITY;
    }
    __syncthreads();
  }
  __device__ __forceinline__ double dist_at(int e) const { return __longlong_as_double(static_cast<long long>(key[e])); }
};

__global__ void __launch_bounds__(kSelThreads, 2)
scan_select(const float4* __restrict__ poses, const int32_t* __restrict__ valid, int64_t n, Cur8 cur,
            const ScanHeader* __restrict__ h, int k, ScanEntry* __restrict__ block_out /*[gridDim.x][k]*/) {
  __shared__ unsigned long long s_key[2 * kScanCap];
  __shared__ int32_t s_i[2 * kScanCap];
  __shared__ int32_t s_pend[kPendLow + kScanUnroll * kSelThreads];   // candidates that passed the cheap bound
  __shared__ int s_cnt, s_npend[2];
  __shared__ double s_tau;
  __shared__ float s_tau_hi;
  dep_wait();
  dep_release();
  TopK top;
  top.init(s_key, s_i, &s_cnt, &s_tau, k);
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
  auto exact = [&](int32_t i, double tau) {
    const Cand c = candidate(__ldg(poses + 2 * static_cast<int64_t>(i)), __ldg(poses + 2 * static_cast<int64_t>(i) + 1), cur.v);
    const double rot = 2.0 * acos(fmin(1.0, c.adot));
    const double ta = mt > 0.0 ? c.t / mt : 0.0;
    const double rb = mr > 0.0 ? rot / mr : 0.0;
    const double dist = ta + rb;
    if (dist <= tau) top.push(dist, i);
  };
  if (threadIdx.x == 0) s_npend[0] = s_npend[1] = 0;
  refresh();
  // The first pass over kScanWarm candidates cuts the list at once: that gives a first k-th best, after which few of
  // the later candidates pass the bound.  Later rounds take kScanUnroll candidates per thread.
  const int64_t warm0 = static_cast<int64_t>(blockIdx.x) * kScanWarm;
  const int64_t warm_all = static_cast<int64_t>(gridDim.x) * kScanWarm;
  if (k > 0 && threadIdx.x < kScanWarm) {
    const int64_t i = warm0 + threadIdx.x;
    if (i < n && !(valid && !__ldg(valid + i))) exact(static_cast<int32_t>(i), INFINITY);
  }
  top.compact();
  refresh();
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
    bool live[kScanUnroll];
#pragma unroll
    for (int u = 0; u < kScanUnroll; ++u) {
      const int64_t i = (r * kScanUnroll + u) * step + lane_off;
      live[u] = i < n && !(valid && !__ldg(valid + i));
      if (live[u]) {
        a[u] = __ldg(poses + 2 * i);
        b[u] = __ldg(poses + 2 * i + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < kScanUnroll; ++u)
      if (live[u] && passes(a[u], b[u]))
        s_pend[atomicAdd(&s_npend[0], 1)] = static_cast<int32_t>((r * kScanUnroll + u) * step + lane_off);
    // the thread whose push came last reads the final count, so the OR over the block cannot miss a full list
    if (__syncthreads_or(*reinterpret_cast<volatile int*>(&s_npend[0]) > kPendLow)) drain();
  }
  __syncthreads();
  drain();
  top.compact();
  for (int e = threadIdx.x; e < k; e += blockDim.x) {
    ScanEntry o;
    o.d = e < s_cnt ? top.dist_at(e) : INFINITY;
    o.i = e < s_cnt ? s_i[e] : -1;
    o.pad = 0;
    block_out[static_cast<int64_t>(blockIdx.x) * k + e] = o;
  }
}

// Merges the blocks' sorted lists: one thread per list holds its head; the block takes the smallest head k times.
__global__ void __launch_bounds__(kMergeThreads)
scan_merge(const ScanEntry* __restrict__ block_out, int n_lists, int k, int out_capacity, int32_t* __restrict__ ids_out,
           double* __restrict__ dist_out) {
  __shared__ unsigned long long s_wkey[kMergeThreads / 32];
  __shared__ int32_t s_widx[kMergeThreads / 32];
  __shared__ int s_wlist[kMergeThreads / 32];
  __shared__ int s_winner;
  dep_wait();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned long long kInf = static_cast<unsigned long long>(__double_as_longlong(INFINITY));
  int pos = 0;   // head of this thread's list; the entry after it is fetched ahead, off the critical path
  unsigned long long key, nkey;
  int32_t idx, nidx;
  auto load = [&](int at, unsigned long long& kk, int32_t& ii) {
    kk = kInf;
    ii = 0x7fffffff;
    if (tid < n_lists && at < k) {
      const ScanEntry x = block_out[static_cast<int64_t>(tid) * k + at];
      if (x.i >= 0) { kk = static_cast<unsigned long long>(__double_as_longlong(x.d)); ii = x.i; }
    }
  };
  load(0, key, idx);
  load(1, nkey, nidx);
  for (int e = tid; e < out_capacity; e += kMergeThreads) {
    ids_out[e] = -1;
    if (dist_out) dist_out[e] = 0.0;
  }
  for (int out = 0; out < k; ++out) {
    // smallest (distance, index) over the heads: warp shuffles, then the warps' winners
    unsigned long long bk = key;
    int32_t bi = idx;
    int bl = tid;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, o);
      const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
      if (ok < bk || (ok == bk && oi < bi)) { bk = ok; bi = oi; bl = ol; }
    }
    if (lane == 0) { s_wkey[warp] = bk; s_widx[warp] = bi; s_wlist[warp] = bl; }
    __syncthreads();
    if (warp == 0) {
      bk = s_wkey[lane]; bi = s_widx[lane]; bl = s_wlist[lane];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, o);
        const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
        if (ok < bk || (ok == bk && oi < bi)) { bk = ok; bi = oi; bl = ol; }
      }
      if (lane == 0) {
        s_winner = (bi != 0x7fffffff) ? bl : -1;
        if (bi != 0x7fffffff) {
          ids_out[out] = bi;
          if (dist_out) dist_out[out] = __longlong_as_double(static_cast<long long>(bk));
        }
      }
    }
    __syncthreads();
    const int w = s_winner;
    if (w < 0) break;          // every list is exhausted
    if (tid == w) {
      ++pos;
      key = nkey;
      idx = nidx;
      load(pos + 1, nkey, nidx);
    }
  }
}

}  // namespace

size_t retrieve_scan_scratch_bytes() {
  return sizeof(ScanHeader) + static_cast<size_t>(kScanMaxBlocks) * kScanMaxK * sizeof(ScanEntry);
}

wk_status launch_retrieve_scan(wk_ctx* ctx, const float* poses, const int32_t* valid, int64_t n, const float* cur_pose,
                               int k, int32_t* ids_out, double* dist_out, int out_capacity, void* scratch, cudaStream_t s) {
  ScanHeader* h = static_cast<ScanHeader*>(scratch);
  ScanEntry* block_out = reinterpret_cast<ScanEntry*>(h + 1);
  Cur8 cur;
  for (int i = 0; i < 8; ++i) cur.v[i] = cur_pose[i];
  // pass 1: four resident 256-thread blocks per SM; pass 2: two resident 512-thread blocks per SM (fewer, longer lists
  // to merge).  Fewer blocks when there is less than a round of work.
  int64_t blocks = static_cast<int64_t>(ctx->sm_count) * 4;
  const int64_t needed = (n + kScanThreads - 1) / kScanThreads;
  if (blocks > needed) blocks = needed;
  if (blocks > kScanMaxBlocks) blocks = kScanMaxBlocks;
  if (blocks < 1) blocks = 1;
  int64_t sel_blocks = static_cast<int64_t>(ctx->sm_count) * 2;
  const int64_t sel_needed = (n + kSelThreads - 1) / kSelThreads;
  if (sel_blocks > sel_needed) sel_blocks = sel_needed;
  if (sel_blocks > kScanMaxBlocks) sel_blocks = kScanMaxBlocks;
  if (sel_blocks < 1) sel_blocks = 1;
  wk_status st;
  scan_init<<<1, 1, 0, s>>>(h);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  const float4* p4 = reinterpret_cast<const float4*>(poses);
  launch_chained(scan_max, dim3(static_cast<unsigned>(blocks)), dim3(kScanThreads), 0, s, p4, valid, n, cur, h);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  launch_chained(scan_select, dim3(static_cast<unsigned>(sel_blocks)), dim3(kSelThreads), 0, s, p4, valid, n, cur, h, k,
                 block_out);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  launch_chained(scan_merge, dim3(1), dim3(kMergeThreads), 0, s, block_out, static_cast<int>(sel_blocks), k, out_capacity,
                 ids_out, dist_out);
  return after_launch(ctx);
}

}  // namespace wk
