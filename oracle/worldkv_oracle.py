"""CPU oracle for the WorldKV hot path -- TEST INFRASTRUCTURE, not the product.

Plain numpy, fp64 throughout (bf16 inputs are widened exactly), written from the paper's
definitions with no blocking, fusion or reordering beyond what those definitions state.
It shares no code with the CUDA path and must never be imported by it; only the tests,
the smoke check and the benchmark's CPU-baseline legs call it.

What each function follows
--------------------------
* ``compression_scores_definitional`` -- Eq. 5 (Section 4.3) literally: for each non-anchor
  key, the mean over the T anchor keys of the cosine similarity.
* ``compression_scores_factorised``   -- the same quantity after pulling the sum over anchors
  inside the dot product: s_j = (k_j / |k_j|) . m with m = (1/T) sum_i a_i / |a_i|.  An exact
  algebraic identity; both forms are kept and compared.
* ``keep_set`` -- Section 4.3: the scores of all non-anchor frames go into one pool and the
  lowest-scoring share of it is retained: the n_keep lowest pooled scores; the compressed chunk
  is every anchor token plus those.
* ``compress_chunk_per_head`` -- the same, with one attention head's key as the vector of Eq. 5
  (the other reading of R1): one keep-set per head.
* ``retrieval_distances`` / ``retrieve`` -- Eq. 4 (Section 4.2) with the distance of Section 5.1:
  squared-L2 translation distance and geodesic rotation distance, each normalised across
  the candidate set, summed; the smallest k win.
* ``attention`` -- the attention of Section 4.2's assembled window: every query attends,
  unmasked, to [dense segments ..., retrieved pool chunks ...]; softmax(scale q K^T) V.
* ``PoolModel`` -- the chunk pool of Section 4.2 (evicted chunks are kept, each filed under its
  camera pose) as a slot table.
* ``query_scores`` / ``retrieve_query`` -- the query-based retrieval of Appendix C: a stored chunk's
  score is the softmax mass the current queries put on its keys (reading R12 below).

Readings taken where the paper is silent (each is one line of code below)
-------------------------------------------------------------------------
R1  d in Eq. 5 is the whole per-layer key of a token (all heads concatenated); one keep-set
    per (layer, chunk).  The per-head reading (d = head_dim, one keep-set per head) is kept beside it.
R2  the retained share of the pool is passed as the integer n_keep; ties are broken by the lowest pooled index.
R3  a zero key has cosine 0 with everything (and still counts in the 1/T).
R4  normalising a distance term over the candidates = dividing it by its maximum over them; a
    term whose maximum is 0 contributes 0.
R5  geodesic rotation distance = 2 acos(min(1, |<q_cur, q_i>|)), in [0, pi].
R6  retrieval ties are broken by the lowest slot index; k > M returns all M.
R7  softmax scale = 1 / sqrt(head_dim); no mask, no positional re-encoding of stored keys.
R8  a retrieved slot listed twice is attended twice (multiset semantics).
R12 query-based retrieval: one layer's queries, logits scaled by 1/sqrt(head_dim), softmax over all
    stored keys of that layer per head and query row, a chunk's mass = the sum over its keys,
    score = the mean over heads and rows; ties to the lowest slot.

Pins: see tests/test_oracle_*.py (closed forms, brute force on tiny inputs, invariants, and
independent textbook/library restatements).  No function here is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------------------
# bf16 widening (exact)
# --------------------------------------------------------------------------------------


def widen_bf16(bits) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64, exactly."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _as_f64(x) -> np.ndarray:
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return widen_bf16(x)
    return x.astype(np.float64)


# --------------------------------------------------------------------------------------
# World Compression (Section 4.3, Eq. 5)
# --------------------------------------------------------------------------------------


def _unit_rows(X: np.ndarray) -> np.ndarray:
    """Rows divided by their Euclidean norm; a zero row stays zero (reading R3)."""
    n = np.sqrt(np.sum(X * X, axis=1))
    out = np.zeros_like(X)
    nz = n > 0
    out[nz] = X[nz] / n[nz, None]
    return out


def compression_scores_definitional(K_chunk, T: int) -> np.ndarray:
    """Eq. 5 as printed.  K_chunk: [F*T, d] keys of one chunk at one layer, frame-major,
    anchor frame first.  Returns s[(F-1)*T]: pooled index j is chunk-local token T + j."""
    K = _as_f64(K_chunk)
    A = K[:T]            # anchor-frame keys  k_i^(a)
    N = K[T:]            # non-anchor keys    k_j^(f), frames 1..F-1 in order
    cos = _unit_rows(N) @ _unit_rows(A).T        # cos[j, i]
    return cos.sum(axis=1) / T                   # (1/T) sum_i


def compression_scores_factorised(K_chunk, T: int) -> np.ndarray:
    """Same scores through the mean unit anchor m = (1/T) sum_i a_i/|a_i|."""
    K = _as_f64(K_chunk)
    m = _unit_rows(K[:T]).sum(axis=0) / T
    return _unit_rows(K[T:]) @ m


def keep_set(scores: np.ndarray, T: int, n_keep: int) -> Tuple[np.ndarray, float]:
    """Indices (chunk-local, ascending) of the compressed chunk: all T anchor tokens plus the
    n_keep non-anchor tokens with the lowest pooled score, ties to the lowest index (R2).
    Also returns the margin between the last kept and the first dropped score (inf when
    nothing is dropped or nothing is kept)."""
    scores = np.asarray(scores, dtype=np.float64)
    n = scores.shape[0]
    if not (0 <= n_keep <= n):
        raise ValueError("n_keep out of range")
    order = np.lexsort((np.arange(n), scores))   # by score, then by index
    kept = np.sort(order[:n_keep])
    margin = float("inf")
    if 0 < n_keep < n:
        margin = float(scores[order[n_keep]] - scores[order[n_keep - 1]])
    idx = np.concatenate([np.arange(T, dtype=np.int64), T + kept]).astype(np.int32)
    return idx, margin


def compress_chunk(K_chunk, T: int, n_keep: int, form: str = "factorised"):
    """Scores + keep-set of one (layer, chunk).  Returns (keep_idx int32[T+n_keep], scores, margin)."""
    if form == "definitional":
        s = compression_scores_definitional(K_chunk, T)
    elif form == "factorised":
        s = compression_scores_factorised(K_chunk, T)
    else:
        raise ValueError(form)
    idx, margin = keep_set(s, T, n_keep)
    return idx, s, margin


def compress_chunk_per_head(K_chunk, T: int, n_keep: int, n_heads: int, form: str = "factorised"):
    """The other reading of Eq. 5's key vector: one attention head's key (d = head_dim) instead of the whole
    per-layer key, hence one keep-set per (layer, chunk, head).  K_chunk: [F*T, n_heads*head_dim]; head h owns
    columns [h*head_dim, (h+1)*head_dim).  Returns (keep_idx int32[n_heads][T+n_keep], scores [n_heads][(F-1)*T],
    smallest margin over the heads)."""
    Kf = np.asarray(K_chunk)
    d = Kf.shape[1] // n_heads
    idx, sc, margin = [], [], float("inf")
    for h in range(n_heads):
        i, s, m = compress_chunk(Kf[:, h * d:(h + 1) * d], T, n_keep, form)
        idx.append(i)
        sc.append(s)
        margin = min(margin, m)
    return np.stack(idx), np.stack(sc), margin


# --------------------------------------------------------------------------------------
# World Retrieval (Section 4.2 Eq. 4, Section 5.1 distance)
# --------------------------------------------------------------------------------------


def retrieval_distances(cur_pose, poses) -> np.ndarray:
    """Combined distance of every candidate pose to the current pose.
    Pose = [tx, ty, tz, _, qw, qx, qy, qz]; poses: [M, 8]."""
    cur = np.asarray(cur_pose, dtype=np.float64)
    P = np.asarray(poses, dtype=np.float64).reshape(-1, 8)
    if P.shape[0] == 0:
        return np.zeros(0)
    dt = np.sum((P[:, 0:3] - cur[0:3]) ** 2, axis=1)            # squared L2 in translation
    dots = np.abs(P[:, 4:8] @ cur[4:8])
    dr = 2.0 * np.arccos(np.minimum(1.0, dots))                 # geodesic angle (R5)
    dt_max, dr_max = dt.max(), dr.max()
    dt_n = dt / dt_max if dt_max > 0 else np.zeros_like(dt)     # normalised over candidates (R4)
    dr_n = dr / dr_max if dr_max > 0 else np.zeros_like(dr)
    return dt_n + dr_n


def retrieve(cur_pose, poses, slots: Sequence[int], k: int):
    """Top-k of Eq. 4 with sim = -distance.  ``poses[i]`` belongs to slot ``slots[i]`` (ascending).
    Returns (slot ids int32[min(k, M)] in rank order, their distances, margin to rank k+1)."""
    slots = np.asarray(slots, dtype=np.int64)
    d = retrieval_distances(cur_pose, poses)
    order = np.lexsort((slots, d))               # by distance, then by slot (R6)
    kk = min(k, len(slots))
    chosen = order[:kk]
    margin = float("inf")
    if 0 < kk < len(slots):
        margin = float(d[order[kk]] - d[order[kk - 1]])
    return slots[chosen].astype(np.int32), d[chosen], margin


# --------------------------------------------------------------------------------------
# Memory attention (Section 4.2: denoising + window + retrieved chunks, unmasked)
# --------------------------------------------------------------------------------------


def attention(Q, K, V, scale: Optional[float] = None, rows: Optional[np.ndarray] = None):
    """softmax(scale * Q K^T) V per head.  Q: [Lq, H, d]; K, V: [Lkv, H, d] (bf16 bits or floats).
    ``rows`` restricts the computation to some query rows (rows are independent).
    Returns (O [n_rows, H, d] fp64, LSE [H, n_rows] fp64, natural log)."""
    Qf, Kf, Vf = _as_f64(Q), _as_f64(K), _as_f64(V)
    if rows is not None:
        Qf = Qf[np.asarray(rows)]
    Lq, H, d = Qf.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)                                   # R7
    O = np.empty((Lq, H, d))
    LSE = np.empty((H, Lq))
    for h in range(H):
        S = scale * (Qf[:, h, :] @ Kf[:, h, :].T)                  # [Lq, Lkv]
        mx = S.max(axis=1, keepdims=True)
        E = np.exp(S - mx)
        Z = E.sum(axis=1, keepdims=True)
        O[:, h, :] = (E / Z) @ Vf[:, h, :]
        LSE[h] = (mx + np.log(Z))[:, 0]
    return O, LSE


def merge_partials(O_parts: Sequence[np.ndarray], LSE_parts: Sequence[np.ndarray]):
    """Combine attention results over disjoint KV subsets: O = sum_s w_s O_s with
    w_s = exp(LSE_s - LSE), LSE = log sum_s exp(LSE_s).  O_s: [Lq, H, d]; LSE_s: [H, Lq]."""
    L = np.stack(LSE_parts)                                        # [S, H, Lq]
    mx = L.max(axis=0)
    lse = mx + np.log(np.exp(L - mx).sum(axis=0))
    O = np.zeros_like(O_parts[0])
    for Os, Ls in zip(O_parts, LSE_parts):
        O += np.exp(Ls - lse).T[:, :, None] * Os
    return O, lse


# --------------------------------------------------------------------------------------
# Chunk pool (Section 4.2) as a slot table, and KV-set assembly
# --------------------------------------------------------------------------------------


@dataclass
class PoolModel:
    """Fixed number of slots; each valid slot holds, per layer, the C = T + n_keep kept rows of
    K and V of one chunk, plus the chunk's pose.  Append takes the lowest free slot; eviction
    is explicit and by slot; ``oldest`` is the valid slot with the smallest append sequence
    number."""
    n_slots: int
    n_layers: int
    K: dict = field(default_factory=dict)      # (layer, slot) -> [C, H, d]
    V: dict = field(default_factory=dict)
    pose: dict = field(default_factory=dict)   # slot -> [8]
    seq: dict = field(default_factory=dict)    # slot -> append sequence number
    tag: dict = field(default_factory=dict)    # slot -> caller's chunk tag
    _next_seq: int = 0

    def valid_slots(self) -> List[int]:
        return sorted(self.pose.keys())

    def count(self) -> int:
        return len(self.pose)

    def oldest(self) -> int:
        return min(self.seq, key=lambda s: self.seq[s]) if self.seq else -1

    def append(self, K_layers, V_layers, keep_idx_layers, pose, tag: int = 0) -> int:
        """Store one chunk: for every layer, the rows ``keep_idx`` of that layer's K and V."""
        free = [s for s in range(self.n_slots) if s not in self.pose]
        if not free:
            raise RuntimeError("pool full")
        s = free[0]
        for l in range(self.n_layers):
            idx = np.asarray(keep_idx_layers[l])
            Kl, Vl = np.asarray(K_layers[l]), np.asarray(V_layers[l])
            if idx.ndim == 1:
                self.K[(l, s)] = Kl[idx]
                self.V[(l, s)] = Vl[idx]
            else:   # one keep-set per head: stored row c of head h is token idx[h][c] of that head
                self.K[(l, s)] = np.stack([Kl[idx[h], h] for h in range(idx.shape[0])], axis=1)
                self.V[(l, s)] = np.stack([Vl[idx[h], h] for h in range(idx.shape[0])], axis=1)
        self.pose[s] = np.asarray(pose, dtype=np.float32).copy()
        self.seq[s] = self._next_seq
        self.tag[s] = tag
        self._next_seq += 1
        return s

    def evict(self, slot: int) -> None:
        if slot not in self.pose:
            raise KeyError("bad slot")
        for l in range(self.n_layers):
            del self.K[(l, slot)], self.V[(l, slot)]
        del self.pose[slot], self.seq[slot], self.tag[slot]

    def retrieve(self, cur_pose, k: int):
        slots = self.valid_slots()
        poses = np.stack([self.pose[s] for s in slots]) if slots else np.zeros((0, 8))
        return retrieve(cur_pose, poses, slots, k)


def assemble_kv(dense_segments, pool: Optional[PoolModel], layer: int, slots: Sequence[int]):
    """The KV set one layer's queries see: dense segments in the given order, then the stored
    rows of each listed pool slot in the given order (R8: repeats are kept).  Slots that are
    not valid are skipped.  Segments are (K, V) pairs of [n, H, d]."""
    Ks = [np.asarray(k) for k, _ in dense_segments]
    Vs = [np.asarray(v) for _, v in dense_segments]
    for s in slots:
        s = int(s)
        if pool is not None and (layer, s) in pool.K:
            Ks.append(pool.K[(layer, s)])
            Vs.append(pool.V[(layer, s)])
    return np.concatenate(Ks, axis=0), np.concatenate(Vs, axis=0)


def memory_attention(Q, dense_segments, pool: Optional[PoolModel], layer: int, slots: Sequence[int],
                     scale: Optional[float] = None, rows: Optional[np.ndarray] = None):
    """Attention of one layer's query chunk over the assembled KV set."""
    K, V = assemble_kv(dense_segments, pool, layer, slots)
    return attention(Q, K, V, scale=scale, rows=rows)


# --------------------------------------------------------------------------------------
# Query-based retrieval (Appendix C: rank stored chunks by their attention score with
# respect to the current denoising query)
# --------------------------------------------------------------------------------------
# Reading taken (the paper gives no formula): the score of a stored chunk is the attention mass the
# current queries put on that chunk's stored keys when they attend over ALL stored chunks of the
# layer, averaged over heads and query rows; the k largest scores win, ties to the lowest slot.


def query_scores(Q, pool: PoolModel, layer: int, scale: Optional[float] = None):
    """Returns (slots ascending, score per slot).  Scores are non-negative and sum to 1.

    Reading R12 written out: per head and query row ONE softmax over all stored keys of the layer; a chunk's mass is
    the sum of the weights of its own keys; its score is the mean of that mass over heads and rows."""
    slots = pool.valid_slots()
    Qf = _as_f64(Q)
    Lq, H, d = Qf.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    if not slots:
        return slots, np.zeros(0)
    Kall = np.concatenate([_as_f64(pool.K[(layer, s)]) for s in slots], axis=0)       # [sum of C, H, d]
    owner = np.concatenate([np.full(pool.K[(layer, s)].shape[0], n) for n, s in enumerate(slots)])
    score = np.zeros(len(slots))
    for h in range(H):
        S = scale * (Qf[:, h, :] @ Kall[:, h, :].T)                  # [Lq, all stored keys]
        W = np.exp(S - S.max(axis=1, keepdims=True))
        W /= W.sum(axis=1, keepdims=True)                            # softmax over every stored key
        for n in range(len(slots)):
            score[n] += W[:, owner == n].sum()                       # the chunk's share, summed over the rows
    return slots, score / (H * Lq)


def retrieve_query(Q, pool: PoolModel, layer: int, k: int, scale: Optional[float] = None):
    """Top-k chunks by query_scores.  Returns (slot ids in rank order, their scores, margin to rank k+1)."""
    slots, score = query_scores(Q, pool, layer, scale)
    slots = np.asarray(slots, dtype=np.int64)
    order = np.lexsort((slots, -score))
    kk = min(k, len(slots))
    chosen = order[:kk]
    margin = float("inf")
    if 0 < kk < len(slots):
        margin = float(score[order[kk - 1]] - score[order[kk]])
    return slots[chosen].astype(np.int32), score[chosen], margin
