// Memory attention (Section 4.2): the denoising chunk's queries attend, unmasked, over
// [dense segments ..., retrieved pool slots ...] of one layer.  O = softmax(scale Q K^T) V per head.
//
// Flash-style kernel on the 5th-generation tensor cores:
//   * one CTA owns two 128-row Q tiles of one head (256 query rows) and a contiguous range of KV tiles;
//   * K/V tiles (128 rows x 128 columns of one head, bf16) are fetched by TMA straight from where they lie:
//     a dense segment (2-D tensor map per segment) or a pool slot (3-D tensor map [layer*slot][row][col]; the
//     slot id is read from device memory, so the retrieval result never visits the host).  Rows past the end
//     of a segment/slot are zero-filled by TMA and masked to -inf before the row maximum;
//   * S = Q K^T and O += P V are tcgen05.mma (M = 128, N = 128, K = 16 steps) with fp32 accumulators in tensor
//     memory: S0, S1, O0, O1 fill all 512 columns; P (bf16) overwrites S in place and is the A operand of
//     the P V product directly from tensor memory;
//   * warp roles: warps 0-3 / 4-7 = softmax of Q tile 0 / 1 (one thread per row, online softmax in fp32 in
//     the exp2 domain, running maximum updated lazily), warp 8 = MMA issue, warp 9 = TMA producer;
//   * with kv splits, each CTA writes normalised fp32 partials + log-sum-exp and a combine kernel merges them.
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
constexpr int kStages = 2;
constexpr size_t kSmemBytes = 1024 + 2 * kTileBytes + 2 * kStages * kTileBytes;   // align slack + Q0,Q1 + K,V stages
constexpr float kRescaleThreshold = 8.0f;           // log2 units: P stays <= 2^8 between maximum updates

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
  int n_tiles, splits;
  int lq, lq_pad, H;
  float scale_log2;
  __nv_bfloat16* O;
  float* lse;
  float* opart;
  float* lsepart;
  uint32_t* status;
};

struct TileInfo {
  int seg;    // >= 0: dense segment index; -1: pool
  int row0;
  int z;
  int nv;     // valid rows, 0 = skip
};

__device__ __forceinline__ TileInfo kv_tile(const AttnParams& p, int t, bool report) {
  TileInfo ti;
  if (t < p.n_dense_tiles) {
    int i = 0;
    while (i + 1 < p.n_segs && t >= p.seg_tile_prefix[i + 1]) ++i;
    ti.seg = i;
    ti.row0 = (t - p.seg_tile_prefix[i]) * kTileKV;
    ti.z = 0;
    ti.nv = min(kTileKV, p.seg_rows[i] - ti.row0);
  } else {
    const int u = t - p.n_dense_tiles;
    const int si = u / p.tiles_per_slot, r = u - si * p.tiles_per_slot;
    const int slot = __ldg(p.slots + si);
    ti.seg = -1;
    ti.row0 = r * kTileKV;
    bool ok = slot >= 0 && slot < p.pool_slots;
    if (ok) ok = __ldg(p.valid + slot) != 0;
    if (!ok) {
      if (report && slot != -1) atomicOr(p.status, WK_DEV_BAD_SLOT);   // never dereferenced
      ti.nv = 0;
      ti.z = 0;
    } else {
      ti.z = p.layer * p.pool_slots + slot;
      ti.nv = min(kTileKV, p.C - ti.row0);
    }
  }
  return ti;
}

struct __align__(8) Barriers {
  uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2], p_full[2], o_done[2];
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

__global__ void __launch_bounds__(kThreads, 1)
memory_attention_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                                   // [2 q tiles][2 halves][128 rows][128 B]
  uint8_t* sK = sQ + 2 * kTileBytes;                    // [stages][2 halves][128][128 B]
  uint8_t* sV = sK + kStages * kTileBytes;
  __shared__ Barriers bars;
  __shared__ uint32_t s_tmem;
  __shared__ volatile uint32_t s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int qpair = blockIdx.x, h = blockIdx.y, split = blockIdx.z;
  const int q0 = qpair * 2 * kTileQ;
  const bool has_q1 = q0 + kTileQ < p.lq;
  const int t0 = static_cast<int>(static_cast<int64_t>(p.n_tiles) * split / p.splits);
  const int t1 = static_cast<int>(static_cast<int64_t>(p.n_tiles) * (split + 1) / p.splits);

  if (tid == 0) {
    mbar_init(&bars.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars.k_full[s], 1); mbar_init(&bars.k_empty[s], 1);
      mbar_init(&bars.v_full[s], 1); mbar_init(&bars.v_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.s_full[i], 1); mbar_init(&bars.p_full[i], 128); mbar_init(&bars.o_done[i], 1);
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
      mbar_expect_tx(&bars.q_full, 2 * kTileBytes);
      for (int i = 0; i < 2; ++i)
        for (int half = 0; half < 2; ++half)
          tma_load_2d(sQ + i * kTileBytes + half * kHalfTileBytes, &p.tm_q, &bars.q_full, h * kHeadDim + half * 64,
                      q0 + i * kTileQ);
      int j = 0;
      const bool report = (blockIdx.x == 0 && blockIdx.y == 0);
      for (int t = t0; t < t1; ++t) {
        const TileInfo ti = kv_tile(p, t, report);
        if (ti.nv == 0) continue;
        const int st = j % kStages;
        const uint32_t ph = (j / kStages) & 1;
        const int x = h * kHeadDim;
        if (!wait_or_abort(&bars.k_empty[st], ph ^ 1, &s_abort, p.status)) break;
        mbar_expect_tx(&bars.k_full[st], kTileBytes);
        uint8_t* dk = sK + st * kTileBytes;
        if (ti.seg >= 0) {
          tma_load_2d(dk, &p.tm_kd[ti.seg], &bars.k_full[st], x, ti.row0);
          tma_load_2d(dk + kHalfTileBytes, &p.tm_kd[ti.seg], &bars.k_full[st], x + 64, ti.row0);
        } else {
          tma_load_3d(dk, &p.tm_kpool, &bars.k_full[st], x, ti.row0, ti.z);
          tma_load_3d(dk + kHalfTileBytes, &p.tm_kpool, &bars.k_full[st], x + 64, ti.row0, ti.z);
        }
        if (!wait_or_abort(&bars.v_empty[st], ph ^ 1, &s_abort, p.status)) break;
        mbar_expect_tx(&bars.v_full[st], kTileBytes);
        uint8_t* dv = sV + st * kTileBytes;
        if (ti.seg >= 0) {
          tma_load_2d(dv, &p.tm_vd[ti.seg], &bars.v_full[st], x, ti.row0);
          tma_load_2d(dv + kHalfTileBytes, &p.tm_vd[ti.seg], &bars.v_full[st], x + 64, ti.row0);
        } else {
          tma_load_3d(dv, &p.tm_vpool, &bars.v_full[st], x, ti.row0, ti.z);
          tma_load_3d(dv + kHalfTileBytes, &p.tm_vpool, &bars.v_full[st], x + 64, ti.row0, ti.z);
        }
        ++j;
      }
      // Do not leave while copies may still be landing in shared memory: wait (bounded) for the loads issued last.
      if (s_abort) {
        for (int s = 0; s < kStages; ++s) {
          for (uint32_t i = 0; i < (1u << 16); ++i)
            if (mbar_try_wait(&bars.k_full[s], 0) || mbar_try_wait(&bars.k_full[s], 1)) break;
          for (uint32_t i = 0; i < (1u << 16); ++i)
            if (mbar_try_wait(&bars.v_full[s], 0) || mbar_try_wait(&bars.v_full[s], 1)) break;
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issue (one thread)
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16_f32(128, 128, 0, 0);
      const uint32_t idesc_pv = idesc_bf16_f32(128, 128, 0, 1);
      const uint32_t aQ = smem_u32(sQ), aK = smem_u32(sK), aV = smem_u32(sV);
      // number of tiles this CTA really processes
      int n_eff = 0;
      for (int t = t0; t < t1; ++t) n_eff += (kv_tile(p, t, false).nv != 0);
      auto issue_s = [&](int i, int st) {
        const uint32_t d = tmem + i * 128;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * kHalfTileBytes + (k & 3) * 32;
          mma_ss(d, smem_desc_sw128(aQ + i * kTileBytes + off, 16, 1024), smem_desc_sw128(aK + st * kTileBytes + off, 16, 1024),
                 idesc_qk, k > 0);
        }
      };
      auto issue_pv = [&](int i, int st, bool accumulate) {
        const uint32_t d = tmem + 256 + i * 128;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          // A = P from tensor memory (bf16 pairs, 8 columns per K = 16 step); B = V, rows = K dimension, MN-major
          mma_ts(d, tmem + i * 128 + k * 8, smem_desc_sw128(aV + st * kTileBytes + k * 2048, kHalfTileBytes, 1024), idesc_pv,
                 accumulate || k > 0);
        }
      };
      bool ok = n_eff > 0 && wait_or_abort(&bars.q_full, 0, &s_abort, p.status);
      if (ok) ok = wait_or_abort(&bars.k_full[0], 0, &s_abort, p.status);
      if (ok) {
        tc_fence_after();
        issue_s(0, 0);
        mma_commit(&bars.s_full[0]);
        if (has_q1) { issue_s(1, 0); mma_commit(&bars.s_full[1]); }
        mma_commit(&bars.k_empty[0]);
      }
      for (int j = 0; ok && j < n_eff; ++j) {
        const int st = j % kStages, stn = (j + 1) % kStages;
        const uint32_t ph = (j / kStages) & 1, phn = ((j + 1) / kStages) & 1;
        const bool more = j + 1 < n_eff;
        if (!(ok = wait_or_abort(&bars.v_full[st], ph, &s_abort, p.status))) break;
        if (!(ok = wait_or_abort(&bars.p_full[0], j & 1, &s_abort, p.status))) break;
        tc_fence_after();
        issue_pv(0, st, j > 0);
        mma_commit(&bars.o_done[0]);
        if (more) {
          if (!(ok = wait_or_abort(&bars.k_full[stn], phn, &s_abort, p.status))) break;
          tc_fence_after();
          issue_s(0, stn);
          mma_commit(&bars.s_full[0]);
        }
        if (has_q1) {
          if (!(ok = wait_or_abort(&bars.p_full[1], j & 1, &s_abort, p.status))) break;
          tc_fence_after();
          issue_pv(1, st, j > 0);
          mma_commit(&bars.o_done[1]);
        }
        mma_commit(&bars.v_empty[st]);
        if (more) {
          if (has_q1) { issue_s(1, stn); mma_commit(&bars.s_full[1]); }
          mma_commit(&bars.k_empty[stn]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warpgroups (one thread per query row)
    const int wg = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + wg * 128;
    const uint32_t tO = tmem + lane_base + 256 + wg * 128;
    const bool active = (wg == 0) || has_q1;
    float m_used = -INFINITY, l = 0.f;
    int j = 0;
    bool ok = true;
    if (active) {
      for (int t = t0; t < t1 && ok; ++t) {
        const int nv = kv_tile(p, t, false).nv;
        if (nv == 0) continue;
        if (!(ok = wait_or_abort(&bars.s_full[wg], j & 1, &s_abort, p.status))) break;
        tc_fence_after();
        float s[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld_x32(tS + c * 32, r);
#pragma unroll
          for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
        }
        tc_wait_ld();
        float mx = -INFINITY;
        if (nv == kTileKV) {
#pragma unroll
          for (int i = 0; i < 128; ++i) mx = fmaxf(mx, s[i]);
        } else {
#pragma unroll
          for (int i = 0; i < 128; ++i) {
            s[i] = i < nv ? s[i] : -INFINITY;       // rows past the end of the segment were zero-filled by TMA
            mx = fmaxf(mx, s[i]);
          }
        }
        const float m_new = fmaxf(m_used, mx * p.scale_log2);
        float alpha = 1.f;
        bool rescale = false;
        if (m_new > m_used + kRescaleThreshold) {    // also true on the first tile (m_used = -inf)
          alpha = ex2_approx(m_used - m_new);
          m_used = m_new;
          rescale = j > 0;
        }
        l *= alpha;
        const float neg_m = -m_used;
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2_approx(fmaf(s[c * 32 + 2 * i], p.scale_log2, neg_m));
            const float p1 = ex2_approx(fmaf(s[c * 32 + 2 * i + 1], p.scale_log2, neg_m));
            sum += p0 + p1;
            pk[i] = pack_bf16x2(p0, p1);
          }
          tmem_st_x16(tS + c * 16, pk);
        }
        l += sum;
        if (__any_sync(0xffffffffu, rescale)) {
          // the previous P V product must have landed before O is touched
          if (!(ok = wait_or_abort(&bars.o_done[wg], (j - 1) & 1, &s_abort, p.status))) break;
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
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&bars.p_full[wg]);
        ++j;
      }
      // ---------------------------------------------------------------- epilogue
      const int qrow = q0 + wg * kTileQ + row;
      if (ok && j > 0) ok = wait_or_abort(&bars.o_done[wg], (j - 1) & 1, &s_abort, p.status);
      if (ok) {
        tc_fence_after();
        const float inv_l = (j > 0 && l > 0.f) ? 1.f / l : 0.f;
        const float lse = (j > 0 && l > 0.f) ? (m_used + log2f(l)) * 0.6931471805599453f : -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          if (j > 0) {
            tmem_ld_x32(tO + c * 32, r);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = 0u;
          }
          if (qrow < p.lq) {
            if (p.splits == 1) {
              uint4* dst = reinterpret_cast<uint4*>(p.O + (static_cast<int64_t>(qrow) * p.H + h) * kHeadDim + c * 32);
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
                  p.opart + ((static_cast<int64_t>(split) * p.H + h) * p.lq_pad + qrow) * kHeadDim + c * 32);
#pragma unroll
              for (int v = 0; v < 8; ++v)
                dst[v] = make_float4(__uint_as_float(r[4 * v]) * inv_l, __uint_as_float(r[4 * v + 1]) * inv_l,
                                     __uint_as_float(r[4 * v + 2]) * inv_l, __uint_as_float(r[4 * v + 3]) * inv_l);
            }
          }
        }
        if (qrow < p.lq) {
          if (p.splits == 1) {
            if (p.lse) p.lse[static_cast<int64_t>(h) * p.lq + qrow] = lse;
          } else {
            p.lsepart[(static_cast<int64_t>(split) * p.H + h) * p.lq_pad + qrow] = lse;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// Merge split-KV partials: O = sum_s w_s O_s / sum_s w_s with w_s = exp(lse_s - max lse).  One warp per (row, head).
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ opart, const float* __restrict__ lsepart, int splits, int H, int lq, int lq_pad,
               __nv_bfloat16* __restrict__ O, float* __restrict__ lse_out) {
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp_global >= lq * H) return;
  const int qrow = warp_global / H, h = warp_global - qrow * H;
  float mx = -INFINITY;
  for (int s = 0; s < splits; ++s) mx = fmaxf(mx, lsepart[(static_cast<int64_t>(s) * H + h) * lq_pad + qrow]);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float wsum = 0.f;
  for (int s = 0; s < splits; ++s) {
    const int64_t idx = (static_cast<int64_t>(s) * H + h) * lq_pad + qrow;
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

wk_status launch_attention(wk_ctx* ctx, int layer, const __nv_bfloat16* Q, int lq, const wk_dense_seg* segs, int n_segs,
                           const int32_t* slots_dev, int n_slots, __nv_bfloat16* O, float* lse, int kv_splits,
                           cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    WK_CUDA_TRY(ctx, cudaFuncSetAttribute(memory_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBytes)));
    attr_set = true;
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
  p.H = ctx->cfg.n_heads;
  p.lq_pad = static_cast<int>(align_up(static_cast<size_t>(ctx->max_lq), 2 * kTileQ));
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.O = O;
  p.lse = lse;
  p.opart = reinterpret_cast<float*>(ctx->scratch_base + ctx->sl.opart_off);
  p.lsepart = reinterpret_cast<float*>(ctx->scratch_base + ctx->sl.lsepart_off);
  p.status = ctx->status_dev;
  const int n_qpairs = (lq + 2 * kTileQ - 1) / (2 * kTileQ);
  const int units = n_qpairs * p.H;
  int splits = kv_splits;
  const int max_splits = ctx->max_splits > 1 ? ctx->max_splits : 1;
  if (splits == 0) {
    // fill the SMs when there are few (head, q-pair) units, but keep at least 8 KV tiles per split
    splits = ctx->sm_count / units;
    const int by_tiles = p.n_tiles / 8;
    if (splits > by_tiles) splits = by_tiles;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
  }
  if (splits > p.n_tiles) splits = p.n_tiles;
  p.splits = splits;
  const dim3 grid(n_qpairs, p.H, splits);
  memory_attention_kernel<<<grid, kThreads, kSmemBytes, s>>>(p);
  if ((st = after_launch(ctx)) != WK_OK) return st;
  if (splits > 1) {
    const int warps = lq * p.H;
    combine_kernel<<<(warps * 32 + 255) / 256, 256, 0, s>>>(p.opart, p.lsepart, splits, p.H, lq, p.lq_pad, O, lse);
    if ((st = after_launch(ctx)) != WK_OK) return st;
  }
  return WK_OK;
}

}  // namespace wk
