// Memory attention (Section 4.2): the denoising chunk's queries attend, unmasked, over
// [dense segments ..., retrieved pool slots ...] of one layer.  O = softmax(scale Q K^T) V per head.
//
// Flash-style kernel on the 5th-generation tensor cores:
//   * a work unit is (head, 256 query rows = two 128-row Q tiles); the flat space unit x KV tile is cut into equal
//     contiguous ranges, one per CTA (one CTA per SM by default), so every SM gets the same amount of work.  A range
//     that covers a whole unit writes bf16 output directly; otherwise it writes a normalised fp32 partial plus its
//     log-sum-exp and combine_kernel merges the (at most three) pieces of that unit;
//   * K/V tiles (128 rows x 128 columns of one head, bf16) are fetched by TMA straight from where they lie:
//     a dense segment (2-D tensor map per segment) or a pool slot (3-D tensor map [layer*slot][row][col]; the
//     slot id is read from device memory, so the retrieval result never visits the host).  Rows past the end
//     of a segment/slot are zero-filled by TMA and masked to -inf before the row maximum;
//   * S = Q K^T and O += P V are tcgen05.mma (M = 128, N = 128, K = 16 steps) with fp32 accumulators in tensor
//     memory: S0, S1, O0, O1 fill all 512 columns; P (bf16) overwrites S in place and is the A operand of
//     the P V product directly from tensor memory;
//   * warp roles: warps 0-3 / 4-7 = softmax of Q tile 0 / 1 (one thread per row, online softmax in fp32 in
//     the exp2 domain, running maximum updated lazily), warp 8 = MMA issue, warp 9 = TMA producer.
// Every wait is bounded; a wait that runs out sets WK_DEV_TIMEOUT, the CTA drains and frees its tensor memory.
#include "ptx_sm100.cuh"
#include "wk_internal.cuh"

namespace wk {
namespace {

using namespace ptx;

constexpr int kThreads = 320;
constexpr int kMmaWarp = 8, kTmaWarp = 9;
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;   // one TMA box: 128 rows x 64 bf16 = 16 KB
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes; // 128 x 128 bf16
constexpr int kStagesK = 3, kStagesV = 2;           // K is wanted one MMA group earlier than V: it gets the spare 32 KB
constexpr size_t kSmemBytes = 1024 + 2 * kTileBytes + (kStagesK + kStagesV) * kTileBytes;   // align slack + Q0,Q1 + K,V stages
constexpr float kRescaleThreshold = 8.0f;           // log2 units: P stays <= 2^8 between maximum updates
constexpr int kPairRows = 2 * kTileQ;
constexpr int kMaxPieces = 32;                      // most ranges one unit may be cut into

struct AttnParams {
  CUtensorMap tm_q;
  CUtensorMap tm_kpool, tm_vpool;
  CUtensorMap tm_kd[kMaxDenseSegs], tm_vd[kMaxDenseSegs];
  int seg_tile_prefix[kMaxDenseSegs + 1];
  int seg_rows[kMaxDenseSegs];
  int n_segs, n_dense_tiles;
  const int32_t* slots;
  const int32_t* valid;
  int n_slots, pool_slots, layer, C, tiles_per_slot;
  int n_tiles, n_qpairs, n_units;
  int lq, H;
  int lse_only;     // 1: only the log-sum-exp is wanted (query-based retrieval): no V loads, no P V product, no O
  int slot_units;   // 1: every listed slot is a problem of its own: unit = (slot ordinal, head, q-pair), n_tiles =
                    //    tiles_per_slot, lse laid out [slot ordinal][H][lq]; stale slots give -inf and are not reported
  float scale_log2;
  __nv_bfloat16* O;
  float* lse;
  float* opart;     // [2 * gridDim.x][256][128] fp32
  float* lsepart;   // [2 * gridDim.x][256]
  uint32_t* status;
};

__device__ __forceinline__ int64_t range_start(const AttnParams& p, int c, int G) {
  return static_cast<int64_t>(c) * p.n_units * p.n_tiles / G;
}

struct TileInfo {
  int seg;    // >= 0: dense segment index; -1: pool
  int row0;
  int z;
  int nv;     // valid rows (> 0)
};

// Walks the effective KV tiles of [tb, te): dense segments first, then pool slots; stale or -1 slots are skipped.
// Two levels, so that stepping to the next tile of the same segment touches no memory: (segment, tile in segment).
struct TileIter {
  int t, te;       // flat tile position, end of the range
  int seg;         // dense segment index, or n_segs + index into the slot list
  int r, n_r;      // tile inside the current segment / slot, and how many it has
  int tail;        // valid rows of its last tile
  int z;           // pool matrix index (layer * pool_slots + slot)
  bool ok;         // false for a stale or -1 slot
  __device__ __forceinline__ void enter(const AttnParams& p, bool report) {
    if (seg < p.n_segs) {
      n_r = p.seg_tile_prefix[seg + 1] - p.seg_tile_prefix[seg];
      tail = p.seg_rows[seg] - (n_r - 1) * kTileKV;
      z = 0;
      ok = true;
    } else {
      n_r = p.tiles_per_slot;
      tail = p.C - (n_r - 1) * kTileKV;
      const int si = seg - p.n_segs;
      ok = false;
      z = 0;
      if (si < p.n_slots) {
        const int slot = __ldg(p.slots + si);
        ok = slot >= 0 && slot < p.pool_slots;
        if (ok) ok = __ldg(p.valid + slot) != 0;
        if (!ok && report && slot != -1) atomicOr(p.status, WK_DEV_BAD_SLOT);   // never dereferenced
        if (ok) z = p.layer * p.pool_slots + slot;
      }
    }
  }
  __device__ __forceinline__ void init(const AttnParams& p, int tb, int te_, bool report) {
    t = tb;
    te = te_;
    if (tb < p.n_dense_tiles) {
      seg = 0;
      while (seg + 1 < p.n_segs && tb >= p.seg_tile_prefix[seg + 1]) ++seg;
      r = tb - p.seg_tile_prefix[seg];
    } else {
      const int u = tb - p.n_dense_tiles;
      const int si = u / p.tiles_per_slot;
      seg = p.n_segs + si;
      r = u - si * p.tiles_per_slot;
    }
    n_r = 0;
    tail = 0;
    z = 0;
    ok = false;
    if (t < te) enter(p, report);
  }
  __device__ __forceinline__ bool next(const AttnParams& p, TileInfo& ti, bool report) {
    while (t < te) {
      if (r == n_r) {   // first tile of the next segment / slot
        ++seg;
        r = 0;
        enter(p, report);
        continue;
      }
      ti.seg = seg < p.n_segs ? seg : -1;
      ti.row0 = r * kTileKV;
      ti.z = z;
      ti.nv = (r == n_r - 1) ? tail : kTileKV;
      ++r;
      ++t;
      if (ok) return true;
    }
    return false;
  }
};

#ifdef WK_ATTN_PROFILE
// Stage timers for one designated thread per role of CTA 0: clock deltas are accumulated in registers and added into the
// words after the status word when the role finishes.  Built only for profiling runs; the product build has none of this.
#define WK_PROF_DECL uint32_t prof_t = clock(); uint32_t prof_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#define WK_PROF(slot, cond)                              \
  do {                                                   \
    const uint32_t now__ = clock();                      \
    prof_acc[(slot) & 7] += now__ - prof_t;              \
    prof_t = now__;                                      \
  } while (0)
#define WK_PROF_FLUSH(base, cond)                                                          \
  do {                                                                                     \
    if (cond)                                                                              \
      for (int i__ = 0; i__ < 8; ++i__) atomicAdd(p.status + 8 + (base) + i__, prof_acc[i__] >> 4); \
  } while (0)
#else
#define WK_PROF_DECL
#define WK_PROF(slot, cond)
#define WK_PROF_FLUSH(base, cond)
#endif

struct __align__(8) Barriers {
  uint64_t q_full, q_empty;
  uint64_t k_full[kStagesK], k_empty[kStagesK], v_full[kStagesV], v_empty[kStagesV];
  uint64_t s_full[2], p_full[2], o_done[2], o_free[2];
};

// Bounded wait that also gives up when another role has already aborted.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                              uint32_t* status) {
  for (uint32_t i = 0; i < WK_WAIT_CAP; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicOr(status, WK_DEV_TIMEOUT);
  return false;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// P = 2^(s * scale - m) for one row of a tile: rounds to bf16, stores into tensor memory over S (64 columns), returns
// the fp32 row sum.  The exponentials are the kernel's second bound (16 per clock and SM on the special-function unit,
// as many clocks per tile as its tensor-core work), so kPoly of every 8 column pairs take 2^x from the FMA pipe instead:
// x = n + f with n = round(x) by the add-a-large-constant trick, 2^f on [-1/2, 1/2] by a cubic (relative error 7.7e-5,
// far inside the bf16 rounding P gets anyway: 2e-3), 2^n by adding n to the exponent field; all in packed fp32 pairs.
// That path needs x >= -126 (it clamps at -120; such a weight is 1e-36 of the row's largest) and finite x, so tiles with
// masked columns (-inf) take kPoly = 0.
// kStore = false (LSE-only launches): only the row sum is wanted, nothing is written.
#ifndef WK_ATTN_POLY
#define WK_ATTN_POLY 2
#endif
template <bool kStore, int kPoly>
__device__ __forceinline__ float exp_store_tile(const float (&s)[128], uint64_t scale2, uint64_t neg_m2, uint32_t tS) {
  uint64_t acc0 = 0, acc1 = 0, acc2 = 0, acc3 = 0;   // four independent (lo, hi) sums
  const uint64_t magic2 = pack_f32x2(12582912.f, 12582912.f), nmagic2 = pack_f32x2(-12582912.f, -12582912.f);
  const uint64_t mone2 = pack_f32x2(-1.f, -1.f);
  const uint64_t c0 = pack_f32x2(0.9999289512634277f, 0.9999289512634277f);
  const uint64_t c1 = pack_f32x2(0.6932762265205383f, 0.6932762265205383f);
  const uint64_t c2 = pack_f32x2(0.242604061961174f, 0.242604061961174f);
  const uint64_t c3 = pack_f32x2(0.055088773369789124f, 0.055088773369789124f);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint64_t e = fma_f32x2(pack_f32x2(s[c * 32 + 2 * i], s[c * 32 + 2 * i + 1]), scale2, neg_m2);
      float e0, e1, p0, p1;
      unpack_f32x2(e, e0, e1);
      if ((i & 7) < kPoly) {
        const uint64_t x = pack_f32x2(fmaxf(e0, -120.f), fmaxf(e1, -120.f));
        const uint64_t t = add_f32x2(x, magic2);                  // low mantissa bits = round(x)
        const uint64_t f = fma_f32x2(add_f32x2(t, nmagic2), mone2, x);   // x - round(x), in [-1/2, 1/2]
        uint64_t y = fma_f32x2(c3, f, c2);
        y = fma_f32x2(y, f, c1);
        y = fma_f32x2(y, f, c0);
        float t0, t1, y0, y1;
        unpack_f32x2(t, t0, t1);
        unpack_f32x2(y, y0, y1);
        p0 = __uint_as_float(__float_as_uint(y0) + (__float_as_uint(t0) << 23));
        p1 = __uint_as_float(__float_as_uint(y1) + (__float_as_uint(t1) << 23));
      } else {
        p0 = ex2_approx(e0);
        p1 = ex2_approx(e1);
      }
      const uint64_t pp = pack_f32x2(p0, p1);
      if ((i & 3) == 0) acc0 = add_f32x2(acc0, pp);
      else if ((i & 3) == 1) acc1 = add_f32x2(acc1, pp);
      else if ((i & 3) == 2) acc2 = add_f32x2(acc2, pp);
      else acc3 = add_f32x2(acc3, pp);
      if (kStore) pk[i] = pack_bf16x2(p0, p1);
    }
    if (kStore) tmem_st_x16(tS + c * 16, pk);
  }
  float a, b;
  unpack_f32x2(add_f32x2(add_f32x2(acc0, acc1), add_f32x2(acc2, acc3)), a, b);
  return a + b;
}

// One piece of work: unit u, KV tiles [tb, te), and where its result goes.
struct Piece {
  int h, q0, tb, te, slot;   // slot < 0: the piece covers the whole unit -> direct output
  int ord;                   // slot ordinal the unit belongs to (0 unless every slot is its own problem)
  bool has_q1;
};
struct PieceWalker {
  int64_t pos, end, start;
  int cta;
  __device__ __forceinline__ void init(const AttnParams& p) {
    cta = blockIdx.x;
    start = range_start(p, cta, gridDim.x);
    end = range_start(p, cta + 1, gridDim.x);
    pos = start;
  }
  __device__ __forceinline__ bool next(const AttnParams& p, Piece& pc) {
    if (pos >= end) return false;
    int u = static_cast<int>(pos / p.n_tiles);
    pc.tb = static_cast<int>(pos - static_cast<int64_t>(u) * p.n_tiles);
    const int64_t room = end - pos;
    pc.te = static_cast<int>(min(static_cast<int64_t>(p.n_tiles), pc.tb + room));
    const bool full = pc.tb == 0 && pc.te == p.n_tiles;
    pc.slot = full ? -1 : 2 * cta + (pos == start ? 0 : 1);
    pos += pc.te - pc.tb;
    pc.ord = 0;
    if (p.slot_units) {   // the unit's tiles are those of one slot: shift the range into that slot's part of the tile space
      const int base = p.H * p.n_qpairs;
      pc.ord = u / base;
      u -= pc.ord * base;
      pc.tb += pc.ord * p.tiles_per_slot;
      pc.te += pc.ord * p.tiles_per_slot;
    }
    pc.h = u / p.n_qpairs;
    pc.q0 = (u - pc.h * p.n_qpairs) * kPairRows;
    pc.has_q1 = pc.q0 + kTileQ < p.lq;
    return true;
  }
};

// kLse = true is the LSE-only instantiation (query-based retrieval): no V, no P, no O; a softmax thread hands its S
// buffer back as soon as the row is in registers, so the next Q K^T runs under the exponentials.
template <bool kLse>
__global__ void __launch_bounds__(kThreads, 1)
memory_attention_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                                   // [2 q tiles][2 halves][128 rows][128 B]
  uint8_t* sK = sQ + 2 * kTileBytes;                    // [stages][2 halves][128][128 B]
  uint8_t* sV = sK + kStagesK * kTileBytes;
  __shared__ Barriers bars;
  __shared__ uint32_t s_tmem;
  __shared__ volatile uint32_t s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(&bars.q_full, 1);
    mbar_init(&bars.q_empty, 1);
    for (int s = 0; s < kStagesK; ++s) { mbar_init(&bars.k_full[s], 1); mbar_init(&bars.k_empty[s], 1); }
    for (int s = 0; s < kStagesV; ++s) { mbar_init(&bars.v_full[s], 1); mbar_init(&bars.v_empty[s], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.s_full[i], 1); mbar_init(&bars.p_full[i], 4); mbar_init(&bars.o_done[i], 1);
      mbar_init(&bars.o_free[i], 4);
    }
    s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s_tmem, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      PieceWalker walk;
      walk.init(p);
      Piece pc;
      uint32_t jk = 0, n = 0;
      uint32_t armed_q = 0, armed_k = 0, armed_v = 0;   // loads armed so far (a barrier's u-th use completes its phase u)
      bool ok = true;
      while (ok && walk.next(p, pc)) {
        if (!(ok = wait_or_abort(&bars.q_empty, (n & 1) ^ 1, &s_abort, p.status))) break;
        mbar_expect_tx(&bars.q_full, 2 * kTileBytes);
        armed_q = n + 1;
        for (int i = 0; i < 2; ++i)
          for (int half = 0; half < 2; ++half)
            tma_load_2d(sQ + i * kTileBytes + half * kHalfTileBytes, &p.tm_q, &bars.q_full, pc.h * kHeadDim + half * 64,
                        pc.q0 + i * kTileQ);
        TileIter it;
        const bool report = !p.slot_units;
        it.init(p, pc.tb, pc.te, report);
        TileInfo ti;
        const int x = pc.h * kHeadDim;
        while (it.next(p, ti, report)) {
          const int sk = jk % kStagesK, st = jk % kStagesV;
          const uint32_t phk = (jk / kStagesK) & 1, ph = (jk / kStagesV) & 1;
          if (!(ok = wait_or_abort(&bars.k_empty[sk], phk ^ 1, &s_abort, p.status))) break;
          mbar_expect_tx(&bars.k_full[sk], kTileBytes);
          armed_k = jk + 1;
          uint8_t* dk = sK + sk * kTileBytes;
          if (ti.seg >= 0) {
            tma_load_2d(dk, &p.tm_kd[ti.seg], &bars.k_full[sk], x, ti.row0);
            tma_load_2d(dk + kHalfTileBytes, &p.tm_kd[ti.seg], &bars.k_full[sk], x + 64, ti.row0);
          } else {
            tma_load_3d(dk, &p.tm_kpool, &bars.k_full[sk], x, ti.row0, ti.z);
            tma_load_3d(dk + kHalfTileBytes, &p.tm_kpool, &bars.k_full[sk], x + 64, ti.row0, ti.z);
          }
          if (kLse) { ++jk; continue; }   // no P V product: V is not fetched
          if (!(ok = wait_or_abort(&bars.v_empty[st], ph ^ 1, &s_abort, p.status))) break;
          mbar_expect_tx(&bars.v_full[st], kTileBytes);
          armed_v = jk + 1;
          uint8_t* dv = sV + st * kTileBytes;
          if (ti.seg >= 0) {
            tma_load_2d(dv, &p.tm_vd[ti.seg], &bars.v_full[st], x, ti.row0);
            tma_load_2d(dv + kHalfTileBytes, &p.tm_vd[ti.seg], &bars.v_full[st], x + 64, ti.row0);
          } else {
            tma_load_3d(dv, &p.tm_vpool, &bars.v_full[st], x, ti.row0, ti.z);
            tma_load_3d(dv + kHalfTileBytes, &p.tm_vpool, &bars.v_full[st], x + 64, ti.row0, ti.z);
          }
          ++jk;
        }
        ++n;
      }
      // After an abort the consumers no longer wait for the tiles in flight, so this thread does: a CTA must not free
      // its shared memory under copies that are still landing.  Per stage, the load armed last is use u = (count - 1 -
      // stage) / stages of that stage's barrier, whose phase u has parity u & 1; a stage that was never armed is skipped.
      if (s_abort) {
        auto drain = [](uint64_t* bar, uint32_t use) {
          for (uint32_t i = 0; i < (1u << 16); ++i)
            if (mbar_try_wait(bar, use & 1)) break;
        };
        if (armed_q > 0) drain(&bars.q_full, armed_q - 1);
        for (uint32_t s = 0; s < kStagesK; ++s)
          if (armed_k > s) drain(&bars.k_full[s], (armed_k - 1 - s) / kStagesK);
        for (uint32_t s = 0; s < kStagesV; ++s)
          if (armed_v > s) drain(&bars.v_full[s], (armed_v - 1 - s) / kStagesV);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issue
    // The whole warp runs the control flow (waits, counters, descriptor arithmetic) so that everything stays
    // warp-uniform; one elected lane issues the tensor-core instructions and the commits.
    {
      const uint32_t idesc_qk = idesc_bf16_f32(128, 128, 0, 0);
      const uint32_t idesc_pv = idesc_bf16_f32(128, 128, 0, 1);
      const uint32_t aQ = smem_u32(sQ), aK = smem_u32(sK), aV = smem_u32(sV);
      // descriptor low words of the tile bases; a K = 16 step advances them by a constant
      const uint32_t hi = smem_desc_hi_sw128(1024);
      const uint32_t q_lo0 = smem_desc_lo(aQ, 16), q_lo1 = smem_desc_lo(aQ + kTileBytes, 16);
      const uint32_t k_lo0 = smem_desc_lo(aK, 16), v_lo0 = smem_desc_lo(aV, kHalfTileBytes);
      auto issue_s = [&](int i, uint32_t st) {
        const uint32_t d = tmem + i * 128;
        const uint32_t a_lo = i ? q_lo1 : q_lo0, b_lo = k_lo0 + st * (kTileBytes >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t off = (k >> 2) * (kHalfTileBytes >> 4) + (k & 3) * 2;   // 32 bytes per step inside a 128-byte row
            mma_ss_lohi(d, a_lo + off, b_lo + off, hi, idesc_qk, k > 0);
          }
        }
        __syncwarp();
      };
      auto issue_pv = [&](int i, uint32_t st, bool accumulate) {
        const uint32_t d = tmem + 256 + i * 128;
        const uint32_t b_lo = v_lo0 + st * (kTileBytes >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            // A = P from tensor memory (bf16 pairs, 8 columns per K = 16 step); B = V, rows = K dimension, MN-major:
            // 16 rows of 128 bytes = 2048 bytes per step
            mma_ts_lohi(d, tmem + i * 128 + k * 8, b_lo + k * 128, hi, idesc_pv, (accumulate || k > 0) ? 1u : 0u);
          }
        }
        __syncwarp();
      };
      auto commit = [&](uint64_t* bar) {
        if (elect_one()) mma_commit(bar);
        __syncwarp();
      };
      PieceWalker walk;
      walk.init(p);
      Piece pc;
      // stage and phase of the K tile whose Q K^T is issued next / of the V tile whose P V is issued next: counters
      // instead of divisions on the issuing path
      uint32_t ks = 0, kph = 0, vs = 0, vph = 0;
      uint32_t g0 = 0, g1 = 0, n = 0;   // running tile counts of the two Q tiles, running piece count
      uint32_t e0 = 0, e1 = 0;          // pieces in which Q tile 0 / 1 produced output so far
      WK_PROF_DECL
      bool ok = true;
      while (ok && walk.next(p, pc)) {
        int n_eff = 0;
        {
          TileIter it;
          it.init(p, pc.tb, pc.te, false);
          TileInfo ti;
          while (it.next(p, ti, false)) ++n_eff;
        }
        const bool q1 = pc.has_q1;
        if (!(ok = wait_or_abort(&bars.q_full, n & 1, &s_abort, p.status))) break;
        ++n;
        if (n_eff == 0) {
          if (lane == 0) mbar_arrive(&bars.q_empty);
          continue;
        }
        // O0 / O1 are about to be overwritten: the epilogue of the last piece that used them must have read them.
        // o_free[i] completes once per piece in which warpgroup i ran an epilogue, so neither side can run two
        // phases ahead of the other (a parity wait cannot tell phase n from phase n + 2).
        if (e0 > 0 && !(ok = wait_or_abort(&bars.o_free[0], (e0 - 1) & 1, &s_abort, p.status))) break;
        ++e0;
        if (q1) {
          if (e1 > 0 && !(ok = wait_or_abort(&bars.o_free[1], (e1 - 1) & 1, &s_abort, p.status))) break;
          ++e1;
        }
        auto next_k = [&]() { if (++ks == kStagesK) { ks = 0; kph ^= 1; } };
        auto next_v = [&]() { if (++vs == kStagesV) { vs = 0; vph ^= 1; } };
        {
          if (!(ok = wait_or_abort(&bars.k_full[ks], kph, &s_abort, p.status))) break;
          tc_fence_after();
          issue_s(0, ks);
          commit(&bars.s_full[0]);
          if (q1) { issue_s(1, ks); commit(&bars.s_full[1]); }
          commit(&bars.k_empty[ks]);
          if (n_eff == 1) commit(&bars.q_empty);
          next_k();
        }
        for (int j = 0; j < n_eff; ++j) {
          const bool more = j + 1 < n_eff;
          WK_PROF(10, blockIdx.x == 0);
          if (!kLse && !(ok = wait_or_abort(&bars.v_full[vs], vph, &s_abort, p.status))) break;
          WK_PROF(11, blockIdx.x == 0);
          if (!(ok = wait_or_abort(&bars.p_full[0], (g0 + j) & 1, &s_abort, p.status))) break;
          WK_PROF(12, blockIdx.x == 0);
          tc_fence_after();
          if (!kLse) issue_pv(0, vs, j > 0);
          commit(&bars.o_done[0]);
          if (more) {
            WK_PROF(13, blockIdx.x == 0);
            if (!(ok = wait_or_abort(&bars.k_full[ks], kph, &s_abort, p.status))) break;
            WK_PROF(14, blockIdx.x == 0);
            tc_fence_after();
            issue_s(0, ks);
            commit(&bars.s_full[0]);
          }
          if (q1) {
            WK_PROF(15, blockIdx.x == 0);
            if (!(ok = wait_or_abort(&bars.p_full[1], (g1 + j) & 1, &s_abort, p.status))) break;
            WK_PROF(16, blockIdx.x == 0);
            tc_fence_after();
            if (!kLse) issue_pv(1, vs, j > 0);
            commit(&bars.o_done[1]);
          }
          if (!kLse) commit(&bars.v_empty[vs]);
          next_v();
          if (more) {
            if (q1) { issue_s(1, ks); commit(&bars.s_full[1]); }
            commit(&bars.k_empty[ks]);
            if (j + 2 == n_eff) commit(&bars.q_empty);   // the last Q K^T of this piece has been issued
            next_k();
          }
        }
        g0 += n_eff;
        if (q1) g1 += n_eff;
      }
      WK_PROF_FLUSH(8, blockIdx.x == 0);
    }
  } else {
    // ------------------------------------------------------------------ softmax warpgroups (one thread per query row)
    const int wg = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + wg * 128;
    const uint32_t tO = tmem + lane_base + 256 + wg * 128;
    PieceWalker walk;
    walk.init(p);
    Piece pc;
    uint32_t g = 0;   // running tile count of this warpgroup
    bool ok = true;
    WK_PROF_DECL
    const uint64_t scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
    while (ok && walk.next(p, pc)) {
      const bool active = (wg == 0) || pc.has_q1;
      float m_used = -INFINITY, l = 0.f;
      int j = 0;
      if (active) {
        TileIter it;
        it.init(p, pc.tb, pc.te, false);
        TileInfo ti;
        while (it.next(p, ti, false)) {
          const int nv = ti.nv;
          WK_PROF(0, blockIdx.x == 0 && tid == 0);
          if (!(ok = wait_or_abort(&bars.s_full[wg], g & 1, &s_abort, p.status))) break;
          WK_PROF(1, blockIdx.x == 0 && tid == 0);
          tc_fence_after();
          // the whole S row (128 fp32) is held in registers: one pass for the row maximum, one for the exponentials
          float s[128];
          float c0 = -INFINITY, c1 = -INFINITY, c2 = -INFINITY, c3 = -INFINITY;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            // the second 64 columns are in flight while the maximum of the first 64 is taken
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              uint32_t r[32];
              tmem_ld_x32(tS + hf * 64 + c * 32, r);
#pragma unroll
              for (int i = 0; i < 32; ++i) s[hf * 64 + c * 32 + i] = __uint_as_float(r[i]);
            }
            if (hf == 1) {
#pragma unroll
              for (int i = 0; i < 64; i += 8) {
                c0 = fmax3(c0, s[i], s[i + 1]);
                c1 = fmax3(c1, s[i + 2], s[i + 3]);
                c2 = fmax3(c2, s[i + 4], s[i + 5]);
                c3 = fmax3(c3, s[i + 6], s[i + 7]);
              }
            }
            tc_wait_ld();
          }
          WK_PROF(2, blockIdx.x == 0 && tid == 0);
          if (kLse) {   // S is in registers and nothing goes back into the buffer: release it now
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.p_full[wg]);
          }
          const bool full_tile = nv == kTileKV;
          if (!full_tile) {   // rows past the end of the segment were zero-filled by TMA: mask them out
            c0 = c1 = c2 = c3 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 128; ++i) s[i] = i < nv ? s[i] : -INFINITY;
#pragma unroll
            for (int i = 0; i < 64; i += 8) {
              c0 = fmax3(c0, s[i], s[i + 1]);
              c1 = fmax3(c1, s[i + 2], s[i + 3]);
              c2 = fmax3(c2, s[i + 4], s[i + 5]);
              c3 = fmax3(c3, s[i + 6], s[i + 7]);
            }
          }
#pragma unroll
          for (int i = 64; i < 128; i += 8) {
            c0 = fmax3(c0, s[i], s[i + 1]);
            c1 = fmax3(c1, s[i + 2], s[i + 3]);
            c2 = fmax3(c2, s[i + 4], s[i + 5]);
            c3 = fmax3(c3, s[i + 6], s[i + 7]);
          }
          const float mx = fmaxf(fmax3(c0, c1, c2), c3);
          const float m_new = fmaxf(m_used, mx * p.scale_log2);
          float alpha = 1.f;
          bool rescale = false;
          if (m_new > m_used + kRescaleThreshold) {    // also true on the first tile (m_used = -inf)
            alpha = ex2_approx(m_used - m_new);
            m_used = m_new;
            rescale = j > 0;
          }
          l *= alpha;
          const uint64_t neg_m2 = pack_f32x2(-m_used, -m_used);
          WK_PROF(3, blockIdx.x == 0 && tid == 0);
          // masked columns hold -inf and come out as 0 (special-function path only)
          l += full_tile ? exp_store_tile<!kLse, WK_ATTN_POLY>(s, scale2, neg_m2, tS)
                         : exp_store_tile<!kLse, 0>(s, scale2, neg_m2, tS);
          if (!kLse && __any_sync(0xffffffffu, rescale)) {
            // the previous P V product must have landed before O is touched
            if (!(ok = wait_or_abort(&bars.o_done[wg], (g - 1) & 1, &s_abort, p.status))) break;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t r[32];
              tmem_ld_x32(tO + c * 32, r);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
              tmem_st_x32(tO + c * 32, r);
            }
          }
          WK_PROF(4, blockIdx.x == 0 && tid == 0);
          if (!kLse) {
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.p_full[wg]);   // one arrival per warp: the wait above covered all 32 lanes' stores
          }
          WK_PROF(5, blockIdx.x == 0 && tid == 0);
          ++j;
          ++g;
        }
        // ---------------------------------------------------------------- epilogue of this piece
        const int prow = wg * kTileQ + row;
        const int qrow = pc.q0 + prow;
        if (ok && j > 0) ok = wait_or_abort(&bars.o_done[wg], (g - 1) & 1, &s_abort, p.status);
        if (ok) {
          tc_fence_after();
          const float inv_l = (j > 0 && l > 0.f) ? 1.f / l : 0.f;
          const float lse = (j > 0 && l > 0.f) ? (m_used + log2f(l)) * 0.6931471805599453f : -INFINITY;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            if (!kLse && j > 0) {
              tmem_ld_x32(tO + c * 32, r);
              tc_wait_ld();
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = 0u;
            }
            if (!kLse && qrow < p.lq) {
              if (pc.slot < 0) {
                uint4* dst = reinterpret_cast<uint4*>(p.O + (static_cast<int64_t>(qrow) * p.H + pc.h) * kHeadDim + c * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                  uint4 o;
                  o.x = pack_bf16x2(__uint_as_float(r[8 * v + 0]) * inv_l, __uint_as_float(r[8 * v + 1]) * inv_l);
                  o.y = pack_bf16x2(__uint_as_float(r[8 * v + 2]) * inv_l, __uint_as_float(r[8 * v + 3]) * inv_l);
                  o.z = pack_bf16x2(__uint_as_float(r[8 * v + 4]) * inv_l, __uint_as_float(r[8 * v + 5]) * inv_l);
                  o.w = pack_bf16x2(__uint_as_float(r[8 * v + 6]) * inv_l, __uint_as_float(r[8 * v + 7]) * inv_l);
                  dst[v] = o;
                }
              } else {
                float4* dst = reinterpret_cast<float4*>(
                    p.opart + (static_cast<int64_t>(pc.slot) * kPairRows + prow) * kHeadDim + c * 32);
#pragma unroll
                for (int v = 0; v < 8; ++v)
                  dst[v] = make_float4(__uint_as_float(r[4 * v]) * inv_l, __uint_as_float(r[4 * v + 1]) * inv_l,
                                       __uint_as_float(r[4 * v + 2]) * inv_l, __uint_as_float(r[4 * v + 3]) * inv_l);
              }
            }
          }
          if (qrow < p.lq) {
            if (pc.slot < 0) {
              if (p.lse) p.lse[(static_cast<int64_t>(pc.ord) * p.H + pc.h) * p.lq + qrow] = lse;
            } else {
              p.lsepart[static_cast<int64_t>(pc.slot) * kPairRows + prow] = lse;
            }
          }
        }
      }
      // O of this piece has been read: the next piece that uses this accumulator may overwrite it
      if (active && j > 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.o_free[wg]);
      }
    }
    WK_PROF_FLUSH(0, blockIdx.x == 0 && tid == 0);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// Merge the pieces of every unit that was cut: O = sum_s w_s O_s / sum_s w_s with w_s = exp(lse_s - max lse).
// One warp per (unit, row of the 256-row pair); units written directly by a single CTA are left alone.
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ opart, const float* __restrict__ lsepart, int G, int n_units, int n_tiles,
               int n_qpairs, int H, int lq, __nv_bfloat16* __restrict__ O, float* __restrict__ lse_out) {
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp_global >= n_units * kPairRows) return;
  const int u = warp_global / kPairRows, prow = warp_global - u * kPairRows;
  const int h = u / n_qpairs, qrow = (u - h * n_qpairs) * kPairRows + prow;
  if (qrow >= lq) return;
  const int64_t W = static_cast<int64_t>(n_units) * n_tiles;
  const int64_t ustart = static_cast<int64_t>(u) * n_tiles, uend = ustart + n_tiles;
  auto start_of = [&](int c) { return static_cast<int64_t>(c) * W / G; };
  int c = static_cast<int>(ustart * G / W);
  if (c >= G) c = G - 1;
  while (c > 0 && start_of(c) > ustart) --c;
  while (c + 1 < G && start_of(c + 1) <= ustart) ++c;
  if (start_of(c) <= ustart && start_of(c + 1) >= uend) return;   // one CTA covered the whole unit
  int slot[kMaxPieces];
  int np = 0;
  for (int cc = c; cc < G && start_of(cc) < uend && np < kMaxPieces; ++cc) {
    const int64_t sc = start_of(cc), ec = start_of(cc + 1);
    if (ec <= ustart || ec == sc) continue;
    const int64_t ps = sc > ustart ? sc : ustart;
    slot[np++] = 2 * cc + (ps == sc ? 0 : 1);
  }
  float mx = -INFINITY;
  for (int s = 0; s < np; ++s) mx = fmaxf(mx, lsepart[static_cast<int64_t>(slot[s]) * kPairRows + prow]);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float wsum = 0.f;
  for (int s = 0; s < np; ++s) {
    const int64_t idx = static_cast<int64_t>(slot[s]) * kPairRows + prow;
    const float ls = lsepart[idx];
    const float w = (ls == -INFINITY) ? 0.f : expf(ls - mx);
    const float4 o = reinterpret_cast<const float4*>(opart + idx * kHeadDim)[lane];
    acc.x = fmaf(w, o.x, acc.x); acc.y = fmaf(w, o.y, acc.y); acc.z = fmaf(w, o.z, acc.z); acc.w = fmaf(w, o.w, acc.w);
    wsum += w;
  }
  const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
  uint2 out;
  out.x = ptx::pack_bf16x2(acc.x * inv, acc.y * inv);
  out.y = ptx::pack_bf16x2(acc.z * inv, acc.w * inv);
  reinterpret_cast<uint2*>(O + (static_cast<int64_t>(qrow) * H + h) * kHeadDim)[lane] = out;
  if (lse_out && lane == 0) lse_out[static_cast<int64_t>(h) * lq + qrow] = wsum > 0.f ? mx + logf(wsum) : -INFINITY;
}

}  // namespace

int attention_partial_slots(int n_heads, int max_lq, int max_splits) {
  const int units = n_heads * ((max_lq + kPairRows - 1) / kPairRows);
  const int by_split = units * (max_splits > 1 ? max_splits : 1);
  return 2 * (by_split > 256 ? by_split : 256);
}

wk_status launch_attention(wk_ctx* ctx, int layer, const __nv_bfloat16* Q, int lq, const wk_dense_seg* segs, int n_segs,
                           const int32_t* slots_dev, int n_slots, __nv_bfloat16* O, float* lse, int kv_splits,
                           cudaStream_t s, bool lse_only) {
  if (!ctx->attn_attr_set) {   // the attribute belongs to the device the context lives on
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(memory_attention_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBytes)));
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(memory_attention_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBytes)));
    ctx->attn_attr_set = true;
  }
  AttnParams p;
  wk_status st = encode_rows_map(ctx, Q, lq, kTileQ, &p.tm_q);
  if (st != WK_OK) return st;
  p.tm_kpool = ctx->tm_kpool;
  p.tm_vpool = ctx->tm_vpool;
  int tiles = 0;
  for (int i = 0; i < n_segs; ++i) {
    const CUtensorMap* mk = cached_rows_map(ctx, segs[i].K, segs[i].n_tokens, &st);
    if (st != WK_OK) return st;
    p.tm_kd[i] = *mk;
    const CUtensorMap* mv = cached_rows_map(ctx, segs[i].V, segs[i].n_tokens, &st);
    if (st != WK_OK) return st;
    p.tm_vd[i] = *mv;
    p.seg_tile_prefix[i] = tiles;
    p.seg_rows[i] = segs[i].n_tokens;
    tiles += (segs[i].n_tokens + kTileKV - 1) / kTileKV;
  }
  for (int i = n_segs; i < kMaxDenseSegs; ++i) {
    p.tm_kd[i] = p.tm_q;
    p.tm_vd[i] = p.tm_q;
    p.seg_rows[i] = 0;
  }
  for (int i = n_segs; i <= kMaxDenseSegs; ++i) p.seg_tile_prefix[i] = tiles;
  p.n_segs = n_segs;
  p.n_dense_tiles = tiles;
  p.slots = slots_dev;
  p.valid = ctx->valid_dev;
  p.n_slots = n_slots;
  p.pool_slots = ctx->cfg.pool_slots;
  p.layer = layer;
  p.C = ctx->C;
  p.tiles_per_slot = (ctx->C + kTileKV - 1) / kTileKV;
  p.n_tiles = tiles + n_slots * p.tiles_per_slot;
  p.lq = lq;
  p.lse_only = lse_only ? 1 : 0;
  p.slot_units = p.lse_only;
  p.H = ctx->cfg.n_heads;
  p.n_qpairs = (lq + kPairRows - 1) / kPairRows;
  p.n_units = p.n_qpairs * p.H;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.O = O;
  p.lse = lse;
  p.opart = reinterpret_cast<float*>(ctx->scratch_base + ctx->sl.opart_off);
  p.lsepart = reinterpret_cast<float*>(ctx->scratch_base + ctx->sl.lsepart_off);
  p.status = ctx->status_dev;
  if (lse_only) {
    // every listed slot is scored on its own: one unit per (slot, head, q-pair), each over that slot's tiles only
    if (n_segs != 0 || n_slots < 1) return WK_ERR_ARG;
    p.n_tiles = p.tiles_per_slot;
    p.n_units *= n_slots;
  }
  const int64_t W = static_cast<int64_t>(p.n_units) * p.n_tiles;
  int64_t G;
  if (lse_only) {
    // whole units per CTA (nothing to merge): the largest divisor of the unit count that fits the SMs, unless that
    // would leave more than a quarter of them idle -- then one CTA per unit
    G = 1;
    for (int g = ctx->sm_count < p.n_units ? ctx->sm_count : p.n_units; g >= 1; --g)
      if (p.n_units % g == 0) { G = g; break; }
    if (G * 4 < static_cast<int64_t>(ctx->sm_count) * 3 && p.n_units > G) G = p.n_units;
  } else if (kv_splits == 0) {
    // One CTA per (head, q-pair) whenever that keeps most SMs busy: under the board's power cap the extra fp32
    // partials and the combine pass of a finer cut cost more than the idle SMs (measured at the Matrix-Game shape:
    // 132 CTAs beat 148 equal ranges by 12 %).  Small problems are cut into one equal range per SM instead.
    if (p.n_units * 4 >= ctx->sm_count * 3) {
      G = p.n_units;
    } else {
      G = ctx->sm_count;
      if (G > static_cast<int64_t>(p.n_units) * (kMaxPieces - 2)) G = static_cast<int64_t>(p.n_units) * (kMaxPieces - 2);
    }
  } else if (kv_splits > 0) {
    int sp = kv_splits < p.n_tiles ? kv_splits : p.n_tiles;
    if (sp > kMaxPieces) sp = kMaxPieces;
    G = static_cast<int64_t>(p.n_units) * sp;  // every unit cut into exactly sp ranges
  } else {
    G = -static_cast<int64_t>(kv_splits);      // caller-chosen number of equal ranges
    if (G * p.n_tiles > W * (kMaxPieces - 2)) return WK_ERR_SHAPE;   // a unit would be cut into too many pieces
  }
  if (G > W) G = W;
  const int max_slots = attention_partial_slots(p.H, ctx->max_lq, ctx->max_splits);
  if (!lse_only && 2 * G > max_slots) return WK_ERR_SHAPE;
  if (lse_only) memory_attention_kernel<true><<<static_cast<unsigned>(G), kThreads, kSmemBytes, s>>>(p);
  else memory_attention_kernel<false><<<static_cast<unsigned>(G), kThreads, kSmemBytes, s>>>(p);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  if (!lse_only && G != p.n_units) {   // some unit was cut
    const int64_t warps = static_cast<int64_t>(p.n_units) * kPairRows;
    combine_kernel<<<static_cast<unsigned>((warps * 32 + 255) / 256), 256, 0, s>>>(
        p.opart, p.lsepart, static_cast<int>(G), p.n_units, p.n_tiles, p.n_qpairs, p.H, lq, O, lse);
    if ((st = after_launch(ctx)) != WK_OK) return st;
  }
  return WK_OK;
}

}  // namespace wk
