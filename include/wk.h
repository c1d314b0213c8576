/*
 * worldkv-b200: C ABI of the WorldKV hot path on one B200 (sm_100a).
 *
 * The calls follow the paper's statement of the method:
 *   - World Compression (Section 4.3, Eq. 5): wk_compress_chunk
 *   - the chunk pool of evicted KV chunks (Section 4.2):  wk_pool_append / wk_pool_evict
 *   - World Retrieval (Section 4.2 Eq. 4, distance of Section 5.1): wk_retrieve
 *   - attention of the denoising chunk over [window + retrieved chunks] (Section 4.2): wk_memory_attention
 *
 * Conventions
 *   - All tensor arguments are DEVICE pointers unless the name ends in _host.  bf16 tensors are
 *     token-major: one row per token holding all heads, [tokens][n_heads][head_dim], row stride
 *     D = n_heads * head_dim elements, base address 16-byte aligned.
 *   - Every call returns a wk_status: 0 on success, negative on error.  Errors that can be told from
 *     the arguments are returned before anything is launched and leave all state untouched.
 *   - Every call that touches the device makes the context's device current (cudaSetDevice) first.
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL = legacy default
 *     stream) and is asynchronous.  Anomalies only the device can see (a stale slot id, a bounded
 *     wait that ran out, a non-finite score) set bits in a status word read with wk_poll_status.
 *   - Ownership: the caller owns every device buffer, including pool storage and scratch (sizes come
 *     from wk_pool_bytes / wk_scratch_bytes; the context only keeps host-side bookkeeping and tensor
 *     maps).  No call allocates device memory.  One context may be used by one host thread at a time.
 *   - The calls of one context share its scratch buffer: enqueue them on one stream, or order the streams yourself.
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x, wk_create fails.
 */
#ifndef WK_H_
#define WK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t wk_status;
enum {
  WK_OK = 0,
  WK_ERR_ARG = -1,        /* NULL pointer, misaligned pointer, negative count, bad config field */
  WK_ERR_SHAPE = -2,      /* a size outside what the context was created for */
  WK_ERR_POOL_FULL = -3,  /* wk_pool_append with no free slot */
  WK_ERR_BAD_SLOT = -4,   /* host-visible slot id out of range or not valid */
  WK_ERR_CUDA = -5,       /* a CUDA runtime/driver call failed (wk_last_cuda_error has the code) */
  WK_ERR_TIMEOUT = -6,    /* reported by wk_poll_status: a bounded device wait ran out */
  WK_ERR_NONFINITE = -7,  /* reported by wk_poll_status: a score was NaN/Inf */
  WK_ERR_UNBOUND = -8,    /* wk_bind has not been called */
  WK_ERR_NO_DEVICE = -9   /* no sm_100-class device */
};

/* bits of the device status word (wk_poll_status) */
enum { WK_DEV_BAD_SLOT = 1u, WK_DEV_TIMEOUT = 2u, WK_DEV_NONFINITE = 4u };

typedef struct wk_ctx wk_ctx;

typedef struct {
  int32_t n_layers;
  int32_t n_heads;
  int32_t head_dim;          /* must be 128 */
  int32_t tokens_per_frame;  /* T */
  int32_t frames_per_chunk;  /* F (the paper uses 3); frame 0 of a chunk is the anchor */
  int32_t n_keep;            /* kept non-anchor tokens per chunk, 0 .. (F-1)*T; the paper's P = 25 % is (F-1)*T/4 */
  int32_t pool_slots;        /* capacity of the chunk pool, in chunks */
  int32_t max_k;             /* largest retrieval budget / slot list length */
  int32_t max_dense_segments;/* 1..8 */
  int32_t device;            /* CUDA device ordinal */
  float softmax_scale;       /* 0 selects 1/sqrt(head_dim) */
  int32_t score_mode;        /* WK_SCORE_WHOLE_KEY or WK_SCORE_PER_HEAD: what Eq. 5 takes as a token's key */
} wk_config;

/* Eq. 5 scores "keys"; the paper does not say whether that is the whole per-layer key of a token or one attention
 * head's key.  Both readings are built:
 *   WK_SCORE_WHOLE_KEY  all heads concatenated (d = n_heads * 128): one keep-set per (layer, chunk), shared by the heads
 *   WK_SCORE_PER_HEAD   one head's key (d = 128): one keep-set per (layer, chunk, head); stored row c of head h is then
 *                       token keep_idx[h][c] of that head, so the pool layout and the attention call do not change */
enum { WK_SCORE_WHOLE_KEY = 0, WK_SCORE_PER_HEAD = 2 };

/* ---- context ------------------------------------------------------------------------------- */

/* Validates the config, selects the device and creates host-side state.  No device memory is taken. */
wk_status wk_create(const wk_config* cfg, wk_ctx** out);
void wk_destroy(wk_ctx* ctx);

/* Bytes of pool storage for this config: K and V rows of every slot of every layer
 * ([n_layers][pool_slots][T + n_keep][D] bf16, twice), slot poses and validity flags. */
size_t wk_pool_bytes(const wk_config* cfg);
/* Bytes of scratch: per-problem mean anchor vectors and scores for up to max_batch compression
 * problems per call, and fp32 split-KV partials for queries of up to max_lq tokens with up to
 * max_splits KV splits. */
size_t wk_scratch_bytes(const wk_config* cfg, int32_t max_batch, int32_t max_lq, int32_t max_splits);
/* Hands the context its two caller-owned device buffers (256-byte aligned).  The pool buffer must be
 * zero-filled by the caller the first time (all slots invalid).  Clears a few hundred bytes of the
 * scratch buffer with a synchronous cudaMemset; enqueues nothing else. */
wk_status wk_bind(wk_ctx* ctx, void* pool_dev, size_t pool_bytes, void* scratch_dev, size_t scratch_bytes,
                  int32_t max_batch, int32_t max_lq, int32_t max_splits);

/* ---- World Compression (Section 4.3, Eq. 5) ----------------------------------------------- */

/* For each of `batch` independent (layer, chunk) problems: the score of every non-anchor key is its
 * mean cosine similarity to the T anchor-frame keys (whole-token keys, all heads concatenated); the
 * n_keep lowest pooled scores are kept, ties to the lowest index.
 *   K_chunks     [batch] problems, problem b at K_chunks + b * batch_stride_elems, each [F*T][D] bf16
 *   keep_idx_out [batch][T + n_keep] int32: chunk-local token indices, ascending (anchors 0..T-1 first);
 *                with WK_SCORE_PER_HEAD [batch][n_heads][T + n_keep], the score of a token then being taken on the
 *                128 columns of that head alone
 *   scores_out   [batch][(F-1)*T] fp32 ([batch][n_heads][(F-1)*T] per head) or NULL: the fp32 first-pass scores, for
 *                inspection only; the selection itself is decided on fp64 values near the threshold
 * Errors: WK_ERR_ARG, WK_ERR_SHAPE (batch > max_batch), WK_ERR_UNBOUND. */
wk_status wk_compress_chunk(wk_ctx* ctx, const void* K_chunks, int64_t batch_stride_elems, int32_t batch,
                            int32_t* keep_idx_out, float* scores_out, void* stream);

/* ---- chunk pool (Section 4.2) -------------------------------------------------------------- */

/* Stores one chunk: for layers layer0 .. layer0+n-1 gathers rows keep_idx[l][0 .. T+n_keep) of that
 * layer's K and V chunk into the lowest free slot, and records the chunk's pose
 * [tx, ty, tz, 0, qw, qx, qy, qz].  A chunk may be appended in several calls covering different layer
 * ranges: the first call (slot_io_host = -1 on entry) picks the slot and returns it; later calls pass it
 * back.  The slot becomes visible to wk_retrieve / wk_memory_attention once every layer is stored.
 *   K_chunks, V_chunks  layer l at + (l - layer0) * batch_stride_elems, each [F*T][D] bf16
 *   keep_idx_dev        [n][T + n_keep] int32, or [n][n_heads][T + n_keep] with WK_SCORE_PER_HEAD (the output of
 *                       wk_compress_chunk)
 * Errors: WK_ERR_POOL_FULL, WK_ERR_BAD_SLOT (slot_io_host not an open append), WK_ERR_SHAPE, WK_ERR_ARG. */
wk_status wk_pool_append(wk_ctx* ctx, int32_t layer0, int32_t n, const void* K_chunks, const void* V_chunks,
                         int64_t batch_stride_elems, const int32_t* keep_idx_dev, const float* pose_host,
                         int64_t chunk_tag, int32_t* slot_io_host, void* stream);
/* World Compression "applied once per chunk at storage time" (Section 4.3) as one call: for layers layer0 .. layer0+n-1
 * scores the chunk's non-anchor keys (Eq. 5), selects the keep-sets and stores the kept rows of K and V in the pool --
 * the same pool bytes, slot choice and bookkeeping as wk_compress_chunk followed by wk_pool_append, in one host call
 * and one chain of launches: the gather is queued behind the selection on the device and walks the layers last to
 * first, so that the keys the scoring pass touched last are gathered while L2 still holds them.
 *   keep_idx_dev  [n][T + n_keep] int32 ([n][n_heads][T + n_keep] with WK_SCORE_PER_HEAD), caller-owned: receives the
 *                 keep-sets (the gather reads them from there)
 *   evict_oldest_if_full  non-zero: if this call has to pick a slot and none is free, the oldest stored chunk
 *                 (wk_pool_oldest) is evicted first; *evicted_slot_host (may be NULL) receives its slot, else -1
 *   slot_io_host, pose_host, chunk_tag  as in wk_pool_append (n <= max_batch; a chunk may be stored in several calls)
 * Errors (all before anything is launched): WK_ERR_POOL_FULL, WK_ERR_BAD_SLOT, WK_ERR_SHAPE, WK_ERR_ARG, WK_ERR_UNBOUND. */
wk_status wk_pool_compress_append(wk_ctx* ctx, int32_t layer0, int32_t n, const void* K_chunks, const void* V_chunks,
                                  int64_t batch_stride_elems, int32_t* keep_idx_dev, const float* pose_host,
                                  int64_t chunk_tag, int32_t evict_oldest_if_full, int32_t* slot_io_host,
                                  int32_t* evicted_slot_host, void* stream);
/* Frees a slot (stream-ordered: kernels already enqueued still see it).  WK_ERR_BAD_SLOT if not valid. */
wk_status wk_pool_evict(wk_ctx* ctx, int32_t slot, void* stream);
int32_t wk_pool_oldest(const wk_ctx* ctx);   /* valid slot with the earliest append, -1 if empty */
int32_t wk_pool_count(const wk_ctx* ctx);    /* number of valid slots */
int64_t wk_pool_tag(const wk_ctx* ctx, int32_t slot); /* chunk_tag given at append, -1 if not valid */

/* ---- host-memory tier (Section 7: every stored chunk in CPU memory, only the chunks the current attention needs on
 *      the GPU; the paper leaves hiding the transfer to future work) ---------------------------------------------- */

/* Bytes of one stored chunk in host memory: K then V, each [n_layers][T + n_keep][D] bf16. */
size_t wk_host_chunk_bytes(const wk_ctx* ctx);

/* Copies the chunk held by a visible slot to host memory in the layout above: two strided device-to-host copies on
 * `stream`, asynchronous when host_dst is page-locked.  The slot stays as it is (evict it afterwards to free it).
 * Errors: WK_ERR_BAD_SLOT (slot not visible), WK_ERR_ARG, WK_ERR_UNBOUND, WK_ERR_CUDA. */
wk_status wk_pool_store_host(wk_ctx* ctx, int32_t slot, void* host_dst, void* stream);

/* Brings layers layer0 .. layer0+n-1 of a chunk written by wk_pool_store_host back into the pool: into the lowest free
 * slot on the first call (slot_io_host = -1 on entry, the slot is returned), into that slot on later calls, exactly as
 * wk_pool_append does; the slot becomes visible, with the given pose, once every layer has been loaded.  Loading layer
 * by layer lets the copy of layer l + 1 run under the attention of layer l.  host_src points at the start of the chunk's
 * host image (not at the layer); copies run on `stream`.
 * Errors: WK_ERR_POOL_FULL, WK_ERR_BAD_SLOT, WK_ERR_SHAPE, WK_ERR_ARG, WK_ERR_UNBOUND, WK_ERR_CUDA. */
wk_status wk_pool_load_host(wk_ctx* ctx, int32_t layer0, int32_t n, const void* host_src, const float* pose_host,
                            int64_t chunk_tag, int32_t* slot_io_host, void* stream);

/* ---- World Retrieval (Section 4.2 Eq. 4; Section 5.1) -------------------------------------- */

/* Distance of every stored chunk's pose to cur_pose: squared-L2 translation distance and geodesic
 * rotation angle, each divided by its maximum over the stored chunks, summed.  Writes the min(k, M)
 * slots with the smallest distance, ties to the lowest slot, in rank order.
 *   slots_out_dev [max_k] int32 (entries past the count are set to -1); dist_out_dev [max_k] fp64 or NULL
 *   n_out_host    the count min(k, M), known on the host (M counts the valid slots)
 * A stored or current pose with a NaN/Inf component is not a candidate: WK_DEV_NONFINITE is set and the places it would
 * have taken stay -1.
 * Errors: WK_ERR_SHAPE (k > max_k or k < 0), WK_ERR_ARG, WK_ERR_UNBOUND. */
wk_status wk_retrieve(wk_ctx* ctx, const float* cur_pose_host, int32_t k, int32_t* slots_out_dev,
                      double* dist_out_dev, int32_t* n_out_host, void* stream);

/* Query-based retrieval (Appendix C ranks the stored chunks by how much attention the current denoising query pays
 * them and gives no formula).  Score of a stored chunk = the softmax mass the queries Q put on that
 * chunk's stored keys of `layer` when they attend over all stored chunks, averaged over heads and query rows (scores
 * are >= 0 and sum to 1); the min(k, M) largest win, ties to the lowest slot, written in rank order.
 *   Q [lq][H][128] bf16; slots_out_dev [max_k] int32 (-1 past the count); score_out_dev [max_k] fp32 or NULL.
 * Cost: one Q K^T pass over every stored chunk of the layer (the P V half of attention is skipped).
 * Errors: WK_ERR_SHAPE (lq > max_lq, k > max_k, layer out of range, pool_slots > 1024), WK_ERR_ARG, WK_ERR_UNBOUND. */
wk_status wk_retrieve_query(wk_ctx* ctx, int32_t layer, const void* Q, int32_t lq, int32_t k, int32_t* slots_out_dev,
                            float* score_out_dev, int32_t* n_out_host, void* stream);

/* World Retrieval over a plain pose array of any length (Eq. 4 with the distance of Section 5.1, same semantics as
 * wk_retrieve: squared-L2 translation distance and geodesic rotation angle, each divided by its maximum over the valid
 * candidates, summed, in fp64; the min(k, valid candidates) smallest win, ties to the lowest index, rank order).  For
 * candidate sets far beyond a pool's slot table (the paper's pools hold 10^2..10^3 chunks; this call is what makes
 * "GB/s of retrieval" measurable at 2^16..2^24 poses).  The poses are read once: a sampled set of k real candidates
 * rules most others out before the two maxima are known (a candidate that k others beat for every possible pair of
 * maxima is not among the k best); the few that remain are ranked exactly afterwards.  Pose sets where nothing can be
 * ruled out (e.g. all rotations equal) are read a second time instead; the result is the same either way.  A pose with
 * a NaN/Inf component is never a candidate and sets WK_DEV_NONFINITE.
 *   poses_dev [n][8] fp32 (tx ty tz _ qw qx qy qz), 16-byte aligned; valid_dev [n] int32 or NULL (all valid);
 *   cur_pose_host [8]; ids_out_dev [out_capacity] int32 (-1 past the count); dist_out_dev [out_capacity] fp64 or NULL;
 *   scratch_dev: wk_retrieve_scan_scratch_bytes() bytes, 16-byte aligned, caller-owned, contents irrelevant on entry.
 * ctx supplies the device, the SM count and the status word; its pool is not touched (an unbound context is fine).
 * Errors: WK_ERR_SHAPE (k < 0, k > 64, k > out_capacity, n < 0 or n >= 2^31, scratch too small), WK_ERR_ARG. */
size_t wk_retrieve_scan_scratch_bytes(void);
wk_status wk_retrieve_scan(wk_ctx* ctx, const float* poses_dev, const int32_t* valid_dev, int64_t n,
                           const float* cur_pose_host, int32_t k, int32_t* ids_out_dev, double* dist_out_dev,
                           int32_t out_capacity, void* scratch_dev, size_t scratch_bytes, void* stream);

/* The paper has no counterpart to this call: it exists for callers that may not allocate device memory.
 * Same computation and same results as wk_retrieve, but with no context and no caller-provided scratch: the two
 * doubles per slot the kernel needs live in a fixed array compiled into the library (64 KB, held by every GPU that
 * loads the library until the process exits).  Use it where cudaMalloc is off the table, for example from code that
 * runs while a CUDA graph is being captured, from a service whose memory pool is sized once at start-up and then
 * frozen, or from a plug-in that must not touch the host application's allocator.
 *   poses_dev [n_slots][8] fp32 and valid_dev [n_slots] int32 are the pool's slot table (a slot with valid = 0 is not
 *   a candidate); cur_pose_host [8]; slots_out_dev [max_k] int32 and dist_out_dev [max_k] fp64 (or NULL) as in
 *   wk_retrieve (entries past min(k, M) are -1 / 0).
 * Limits and caveats: n_slots <= 4096, else WK_ERR_SHAPE and nothing is launched.  The first call on each device looks
 * up the array's device address (cudaGetSymbolAddress, with that device current); make that first call outside any
 * stream capture.  All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 * (different streams) race on it; calls on one stream are safe.  Nothing in the array has to start at zero: every
 * entry a call reads it has written first.  Calls no cudaMalloc/cudaFree and no allocating library routine.
 * A pose with a NaN/Inf component is not a candidate (there is no status word to report it through here).
 * Errors: WK_ERR_ARG, WK_ERR_SHAPE, WK_ERR_NO_DEVICE, WK_ERR_CUDA. */
wk_status wk_retrieve_noalloc(const float* poses_dev, const int32_t* valid_dev, int32_t n_slots,
                              const float* cur_pose_host, int32_t k, int32_t max_k, int32_t* slots_out_dev,
                              double* dist_out_dev, void* stream);

/* ---- memory attention (Section 4.2) -------------------------------------------------------- */

typedef struct {
  const void* K;      /* [n_tokens][H][128] bf16 */
  const void* V;      /* [n_tokens][H][128] bf16 */
  int32_t n_tokens;   /* > 0 */
  int32_t reserved;   /* 0 */
} wk_dense_seg;

/* O = softmax(scale * Q K^T) V per head, unmasked, over the dense segments (denoising chunk, window,
 * sink ...) followed by the stored rows of each listed pool slot of `layer`.  Nothing is concatenated
 * in memory: K/V tiles are fetched where they lie.
 *   Q [lq][H][128] bf16, O same shape; lse_out [H][lq] fp32 (natural log) or NULL
 *   slots_dev [n_slots] int32 in device memory (e.g. wk_retrieve's output); an entry that is -1 is
 *             skipped silently, any other out-of-range or invalid entry is skipped and sets
 *             WK_DEV_BAD_SLOT; a slot listed twice is attended twice
 *   kv_splits 0 = default: one CTA per (head, 256-row query block) when those fill at least three quarters of the SMs
 *             (nothing is merged afterwards), else the (block x KV-tile) space cut into one equal range per SM;
 *             s in 1 .. max_splits = cut every block's KV range into s parts; -g = cut the whole space into g
 *             equal ranges (g CTAs; needs 2 g partial slots, see wk_scratch_bytes)
 * Errors: WK_ERR_SHAPE (lq > max_lq, n_slots > max_k, n_segs > max_dense_segments, kv_splits > max_splits),
 * WK_ERR_ARG (no KV at all: n_segs = 0 and n_slots = 0), WK_ERR_UNBOUND, WK_ERR_CUDA. */
wk_status wk_memory_attention(wk_ctx* ctx, int32_t layer, const void* Q, int32_t lq, const wk_dense_seg* segs_host,
                              int32_t n_segs, const int32_t* slots_dev, int32_t n_slots, void* O, float* lse_out,
                              int32_t kv_splits, void* stream);

/* ---- status -------------------------------------------------------------------------------- */

/* Synchronises the stream, reads and clears the device status word.  Returns WK_OK when no bit is set,
 * else the error of the most severe bit; *device_flags (may be NULL) receives the raw bits. */
wk_status wk_poll_status(wk_ctx* ctx, uint32_t* device_flags, void* stream);
const char* wk_status_string(wk_status s);
int32_t wk_last_cuda_error(const wk_ctx* ctx);
/* Number of kernels this context has launched since creation (for benchmark bookkeeping). */
int64_t wk_launch_count(const wk_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* WK_H_ */
