"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o
from wk_testlib import Scenario, assert_attention_close, attention_errors, bf16_to_f64

pytestmark = pytest.mark.gpu


def make_kv(**kw):
    from paper_2605_22718_b200 import WorldKV
    return WorldKV(**kw)


# ----------------------------------------------------------------------------- generators
def test_device_generators_match_numpy():
    T, D = 96, 256
    k = torch.empty((3 * T, D), dtype=torch.bfloat16, device="cuda")
    for layer, chunk in [(0, 0), (2, 5)]:
        wd.key_chunk(k, 7, layer, chunk, T, D, 0.1)
        np.testing.assert_array_equal(wd.to_host_bits(k), wi.key_chunk_bf16(7, layer, chunk, T, D, 0.1))
    v = torch.empty((3 * T, D), dtype=torch.bfloat16, device="cuda")
    wd.value_chunk(v, 7, 1, 4, T, D)
    np.testing.assert_array_equal(wd.to_host_bits(v), wi.value_chunk_bf16(7, 1, 4, T, D))
    q = torch.empty((50, D), dtype=torch.bfloat16, device="cuda")
    wd.query(q, 7, 1, 2, 3)
    np.testing.assert_array_equal(wd.to_host_bits(q), wi.query_bf16(7, 1, 2, 3, 50, D))


# ----------------------------------------------------------------------------- compression
@pytest.mark.parametrize("T,H,n_keep,batch,sigma", [
    (880, 2, 440, 6, 0.1),        # cfg0 shape, several problems in one call
    (37, 1, 18, 3, 0.1),          # ragged everything
    (100, 3, 50, 2, 0.05),
    (256, 12, 128, 2, 0.1),       # Matrix-Game row width
    (64, 40, 32, 1, 0.05),        # LingBot row width
    (200, 16, 100, 3, 0.1),       # 2,048 columns: two warps share a row of the anchor pass
    (96, 13, 48, 2, 0.1),         # 1,664 columns: two warps per row, some lanes without a column group
    (45, 20, 30, 5, 0.1),         # wide rows, several short chunks
    (4, 2, 4, 400, 0.1),          # hundreds of tiny chunks: a CTA's run of anchor rows crosses three or four of them
])
def test_compress_matches_oracle(T, H, n_keep, batch, sigma):
    D = H * 128
    kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=2, max_k=1, max_batch=batch)
    K = np.stack([wi.key_chunk_bf16(11, b, b + 1, T, D, sigma) for b in range(batch)])
    Kd = wd.to_device_bf16(K)
    scores = torch.empty((batch, 2 * T), dtype=torch.float32, device="cuda")
    keep = kv.compress_chunk(Kd, scores_out=scores).cpu().numpy()
    st, flags = kv.poll_status()
    assert st == 0 and flags == 0
    for b in range(batch):
        idx, s, margin = o.compress_chunk(K[b], T, n_keep)
        assert margin > 1e-11
        np.testing.assert_array_equal(keep[b], idx)
        np.testing.assert_allclose(scores[b].cpu().numpy(), s, atol=2e-6)
    keep2 = kv.compress_chunk(Kd).cpu().numpy()                          # run-to-run reproducible
    np.testing.assert_array_equal(keep, keep2)


def test_compress_retention_ladder_and_degenerate_inputs():
    T, H = 48, 2
    D = H * 128
    K = wi.key_chunk_bf16(3, 0, 2, T, D, 0.1)
    for n_keep in (0, T // 4, T // 2, T, 3 * T // 2, 2 * T, 1, 2 * T - 1):
        kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=1, max_k=1)
        keep = kv.compress_chunk(wd.to_device_bf16(K)[None]).cpu().numpy()[0]
        np.testing.assert_array_equal(keep, o.compress_chunk(K, T, n_keep)[0])
    # all keys identical: every score ties, the lowest indices are kept
    kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=T // 2, pool_slots=1, max_k=1)
    same = np.tile(K[:1], (3 * T, 1))
    keep = kv.compress_chunk(wd.to_device_bf16(same)[None]).cpu().numpy()[0]
    np.testing.assert_array_equal(keep, np.arange(T + T // 2))
    # zero keys score 0 (no NaN), among negative and positive scores
    Kz = K.copy()
    Kz[T + 5] = 0
    Kz[2] = 0
    keep = kv.compress_chunk(wd.to_device_bf16(Kz)[None]).cpu().numpy()[0]
    np.testing.assert_array_equal(keep, o.compress_chunk(Kz, T, T // 2)[0])
    assert kv.poll_status() == (0, 0)


@pytest.mark.parametrize("H", [2, 12, 40])
def test_compress_scores_only_and_extreme_row_norms(H):
    """Keep everything but ask for the scores (the anchor pass and the score pass run, no selection), on keys whose
    anchor rows span 2^-70 .. 2^70 in scale: cosine scores do not depend on a row's scale, and 1/|a| leaves the range of
    the fast reciprocal square root for the true division."""
    T = 40
    D = H * 128
    bits = wi.key_chunk_bf16(5, 1, 3, T, D, 0.1)
    scale = np.ones(3 * T, dtype=np.float32)
    scale[0], scale[1], scale[2], scale[3] = 2.0 ** 70, 2.0 ** -70, 2.0 ** 55, 2.0 ** -45
    scale[T + 1], scale[T + 2] = 2.0 ** 40, 2.0 ** -40
    f32 = (bits.astype(np.uint32) << 16).view(np.float32) * scale[:, None]   # a power of two keeps the 8-bit mantissa
    Kb = (f32.view(np.uint32) >> 16).astype(np.uint16)
    assert np.array_equal((Kb.astype(np.uint32) << 16).view(np.float32), f32)
    kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=2 * T, pool_slots=1, max_k=1)
    scores = torch.empty((1, 2 * T), dtype=torch.float32, device="cuda")
    keep = kv.compress_chunk(wd.to_device_bf16(Kb)[None], scores_out=scores).cpu().numpy()[0]
    np.testing.assert_array_equal(keep, np.arange(3 * T))
    assert kv.poll_status() == (0, 0)
    np.testing.assert_allclose(scores[0].cpu().numpy(), o.compression_scores_definitional(Kb, T), atol=2e-6)
    # the same keys unscaled give the same scores: the scale of a row cancels in a cosine
    np.testing.assert_allclose(o.compression_scores_definitional(Kb, T), o.compression_scores_definitional(bits, T),
                               atol=1e-12)


# ----------------------------------------------------------------------------- pool + retrieval
def test_pool_and_retrieval_cfg0():
    w = wi.WORKLOADS["cfg0"]
    kv = make_kv(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=8, max_batch=1)
    sc = Scenario(kv, w.seed, w.sigma, 1, w.T, w.n_heads, w.n_keep, w.pool_chunks)
    poses = wi.random_poses(w.seed, w.pool_chunks + 1)
    for c in range(w.pool_chunks):
        assert sc.append_chunk(c, poses[c]) == c
    assert min(sc.margins) > 1e-11
    assert kv.pool_count() == 8 and kv.pool_oldest() == 0
    from paper_2605_22718_b200 import WkError, WK_ERR_POOL_FULL, WK_ERR_BAD_SLOT
    with pytest.raises(WkError) as e:
        sc.append_chunk(9, poses[8], check=False)
    assert e.value.status == WK_ERR_POOL_FULL
    # stored rows are the kept rows
    C, D = w.C, w.D
    Kpool = kv.pool[:8 * C * D * 2].view(torch.bfloat16).view(8, C, w.n_heads, 128)
    for s in (0, 5):
        np.testing.assert_array_equal(wd.to_host_bits(Kpool[s]), sc.pool.K[(0, s)])
    dist = torch.empty(8, dtype=torch.float64, device="cuda")
    cur = poses[8]
    for k in (1, 3, 8):
        ids, n = kv.retrieve(cur, k, dist_out=dist)
        ref_ids, ref_d, margin = sc.pool.retrieve(cur, k)
        assert n == len(ref_ids) and margin > 1e-9
        np.testing.assert_array_equal(ids.cpu().numpy()[:n], ref_ids)
        assert (ids.cpu().numpy()[n:] == -1).all()
        np.testing.assert_allclose(dist.cpu().numpy()[:n], ref_d, rtol=1e-12, atol=1e-14)
    # evict two slots, append one (lowest free slot), retrieve again
    kv.pool_evict(3); sc.pool.evict(3)
    kv.pool_evict(0); sc.pool.evict(0)
    with pytest.raises(WkError) as e:
        kv.pool_evict(3)
    assert e.value.status == WK_ERR_BAD_SLOT
    assert kv.pool_oldest() == sc.pool.oldest() == 1
    assert sc.append_chunk(10, poses[3]) == 0
    ids, n = kv.retrieve(cur, 8)
    ref_ids, _, _ = sc.pool.retrieve(cur, 8)
    assert n == 7
    np.testing.assert_array_equal(ids.cpu().numpy()[:n], ref_ids)
    assert kv.pool_tag(0) == 10 and kv.pool_tag(3) == -1
    assert kv.poll_status() == (0, 0)


def test_retrieval_empty_pool_and_loop_workload():
    kv = make_kv(n_layers=1, n_heads=1, tokens_per_frame=8, n_keep=4, pool_slots=130, max_k=16)
    ids, n = kv.retrieve(wi.random_poses(0, 1)[0], 4)
    assert n == 0 and (ids.cpu().numpy() == -1).all()
    sc = Scenario(kv, 1, 0.1, 1, 8, 1, 4, 130)
    poses = wi.loop_poses(1, 128)
    for c in range(125):
        sc.append_chunk(c, poses[c], check=(c < 3))
    for k in (4, 16):
        ids, n = kv.retrieve(poses[127], k)
        ref_ids, _, margin = sc.pool.retrieve(poses[127], k)
        assert margin > 1e-9
        np.testing.assert_array_equal(ids.cpu().numpy()[:n], ref_ids)


# ----------------------------------------------------------------------------- memory attention
def _cfg0_scene():
    w = wi.WORKLOADS["cfg0"]
    kv = make_kv(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=8, max_batch=1, max_lq=w.Lq, max_splits=8)
    sc = Scenario(kv, w.seed, w.sigma, 1, w.T, w.n_heads, w.n_keep, w.pool_chunks)
    poses = wi.random_poses(w.seed, w.pool_chunks + 1)
    for c in range(w.pool_chunks):
        sc.append_chunk(c, poses[c])
    return w, kv, sc, poses


def test_memory_attention_cfg0_all_rows():
    """cfg0 in full: 880 queries over current frame (880) + window (1,760) + the retrieved chunk (1,320)."""
    w, kv, sc, poses = _cfg0_scene()
    Qb = wi.query_bf16(w.seed, 0, 0, 20, w.Lq, w.D)
    Q = wd.to_device_bf16(Qb).view(w.Lq, w.n_heads, 128)
    cur_d, cur_h = sc.dense_segment(0, 20, w.T)
    win_d, win_h = sc.dense_segment(0, 19, 2 * w.T)
    slots, n = kv.retrieve(poses[8], w.k)
    ref_slots, _, _ = sc.pool.retrieve(poses[8], w.k)
    np.testing.assert_array_equal(slots.cpu().numpy()[:n], ref_slots)
    O_ref, L_ref = o.memory_attention(Qb.reshape(w.Lq, w.n_heads, 128), [cur_h, win_h], sc.pool, 0, ref_slots)
    assert o.assemble_kv([cur_h, win_h], sc.pool, 0, ref_slots)[0].shape[0] == 3960
    for splits in (1, 2, 5, 0):
        lse = torch.empty((w.n_heads, w.Lq), dtype=torch.float32, device="cuda")
        O = kv.memory_attention(0, Q, [cur_d, win_d], slots, n, lse_out=lse, kv_splits=splits)
        assert kv.poll_status() == (0, 0)
        err, rel = assert_attention_close(O, O_ref, f"splits={splits}")
        np.testing.assert_allclose(lse.cpu().numpy(), L_ref, atol=2e-3)
    # segment / slot order does not matter; duplicates and invalid slots follow the stated semantics
    many = torch.tensor([5, 2, -1, 7, 2], dtype=torch.int32, device="cuda")
    O = kv.memory_attention(0, Q, [win_d, cur_d], many, 5)
    O_ref2, _ = o.memory_attention(Qb.reshape(w.Lq, w.n_heads, 128), [win_h, cur_h], sc.pool, 0, [5, 2, 7, 2])
    assert_attention_close(O, O_ref2, "multiset slots")
    assert kv.poll_status() == (0, 0)
    bad = torch.tensor([5, 99, 3], dtype=torch.int32, device="cuda")
    kv.pool_evict(3)
    O = kv.memory_attention(0, Q, [cur_d], bad, 3)
    from paper_2605_22718_b200 import WK_ERR_BAD_SLOT, WK_DEV_BAD_SLOT
    assert kv.poll_status() == (WK_ERR_BAD_SLOT, WK_DEV_BAD_SLOT)
    sc.pool.evict(3)
    O_ref3, _ = o.memory_attention(Qb.reshape(w.Lq, w.n_heads, 128), [cur_h], sc.pool, 0, [5])
    assert_attention_close(O, O_ref3, "stale slots skipped")


@pytest.mark.parametrize("lq,seg_rows,n_slots,H", [
    (1, [1], 0, 1),                # smallest possible problem
    (129, [127, 300], 2, 2),       # ragged q tiles and ragged segments
    (300, [], 3, 3),               # pool only
    (257, [40, 128, 129, 5], 1, 1),
    (600, [2000, 77], 3, 2),       # three q-pairs per head, the last without a second Q tile; 20 KV tiles
])
def test_memory_attention_ragged_shapes(lq, seg_rows, n_slots, H):
    T, n_keep = 40, 23                       # C = 63: less than one KV tile per slot
    kv = make_kv(n_layers=2, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=4, max_k=4, max_batch=2,
                 max_lq=lq, max_splits=4, max_dense_segments=4)
    sc = Scenario(kv, 5, 0.1, 2, T, H, n_keep, 4)
    poses = wi.random_poses(5, 4)
    for c in range(3):
        sc.append_chunk(c, poses[c])
    layer = 1
    Qb = wi.query_bf16(5, layer, 0, 0, lq, H * 128)
    Q = wd.to_device_bf16(Qb).view(lq, H, 128)
    segs_d, segs_h = [], []
    for i, n in enumerate(seg_rows):
        reps = (n + 3 * T - 1) // (3 * T)
        Kb = np.concatenate([wi.key_chunk_bf16(5, layer, 30 + 4 * i + r, T, H * 128, 0.1) for r in range(reps)])[:n]
        Vb = np.concatenate([wi.value_chunk_bf16(5, layer, 30 + 4 * i + r, T, H * 128) for r in range(reps)])[:n]
        segs_d.append((wd.to_device_bf16(Kb).view(n, H, 128), wd.to_device_bf16(Vb).view(n, H, 128)))
        segs_h.append((Kb.reshape(n, H, 128), Vb.reshape(n, H, 128)))
    slot_list = [2, 0, 1][:n_slots]
    slots = torch.tensor(slot_list + [-1], dtype=torch.int32, device="cuda")
    O_ref, L_ref = o.memory_attention(Qb.reshape(lq, H, 128), segs_h, sc.pool, layer, slot_list)
    # 0: one range per SM; s > 0: s ranges per (head, q-pair); -g: g equal ranges over the whole space, so that one
    # CTA runs on from a q-pair without a second Q tile into one with it, and the other way round
    for splits in (1, 0, 3, -2, -4, -5, -7):
        lse = torch.empty((H, lq), dtype=torch.float32, device="cuda")
        O = kv.memory_attention(layer, Q, segs_d, slots, n_slots, lse_out=lse, kv_splits=splits)
        assert kv.poll_status() == (0, 0)
        assert_attention_close(O, O_ref, f"splits={splits}")
        np.testing.assert_allclose(lse.cpu().numpy(), L_ref, atol=2e-3)


def test_argument_errors_are_reported_before_launch():
    from paper_2605_22718_b200 import WkError, WK_ERR_SHAPE, WK_ERR_ARG
    kv = make_kv(n_layers=1, n_heads=1, tokens_per_frame=16, n_keep=8, pool_slots=2, max_k=2, max_batch=1, max_lq=64)
    n0 = kv.launch_count()
    Q = torch.zeros((65, 1, 128), dtype=torch.bfloat16, device="cuda")
    seg = (torch.zeros((16, 1, 128), dtype=torch.bfloat16, device="cuda"),) * 2
    with pytest.raises(WkError) as e:
        kv.memory_attention(0, Q, [seg], None, 0)
    assert e.value.status == WK_ERR_SHAPE
    with pytest.raises(WkError) as e:
        kv.memory_attention(0, Q[:8], [], None, 0)
    assert e.value.status == WK_ERR_ARG
    with pytest.raises(WkError) as e:
        kv.memory_attention(3, Q[:8], [seg], None, 0)
    assert e.value.status == WK_ERR_SHAPE
    with pytest.raises(WkError) as e:
        kv.retrieve([0] * 8, 5)
    assert e.value.status == WK_ERR_SHAPE
    with pytest.raises(WkError) as e:
        kv.compress_chunk(torch.zeros((2, 48, 128), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == WK_ERR_SHAPE
    assert kv.launch_count() == n0


@pytest.mark.parametrize("per_head", [False, True])
def test_compress_append_in_one_call_stores_the_same_pool_bytes(per_head):
    """wk_pool_compress_append against wk_compress_chunk + wk_pool_append (same slots, same stored rows, same keep-sets)
    and against the oracle's pool model, including the evict-oldest-when-full path and a chunk stored in two calls."""
    from paper_2605_22718_b200 import WkError, WK_ERR_POOL_FULL, SCORE_PER_HEAD
    T, H, n_keep, L, slots = 40, 3, 21, 4, 3
    D, C_rows = H * 128, T + n_keep
    mode = SCORE_PER_HEAD if per_head else 0
    kw = dict(n_layers=L, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=slots, max_k=slots, max_batch=L,
              score_mode=mode)
    kv_a, kv_b = make_kv(**kw), make_kv(**kw)
    ref = Scenario(kv_b, 13, 0.1, L, T, H, n_keep, slots, per_head=per_head)
    poses = wi.random_poses(13, 6)
    pool_words = 2 * L * slots * C_rows * D            # K then V, bf16 elements

    def store_fused(chunk, **extra):
        K, V = ref.chunk_bits(chunk)
        Kd, Vd = wd.to_device_bf16(np.stack(K)), wd.to_device_bf16(np.stack(V))
        return kv_a.pool_compress_append(0, L, Kd, Vd, poses[chunk], chunk_tag=chunk, **extra)

    for c in range(3):
        slot, evicted, keep = store_fused(c)
        assert ref.append_chunk(c, poses[c]) == slot and evicted == -1     # Scenario checks kv_b's keep-sets vs the oracle
        ref_keep = [o.compress_chunk_per_head(k, T, n_keep, H)[0] if per_head else o.compress_chunk(k, T, n_keep)[0]
                    for k in ref.chunk_bits(c)[0]]
        np.testing.assert_array_equal(keep.cpu().numpy(), np.stack(ref_keep))
    a = kv_a.pool[:pool_words * 2].view(torch.int16)
    b = kv_b.pool[:pool_words * 2].view(torch.int16)
    assert torch.equal(a, b)
    # full pool: refused without the flag (and nothing launched), oldest evicted with it
    n0 = kv_a.launch_count()
    with pytest.raises(WkError) as e:
        store_fused(3)
    assert e.value.status == WK_ERR_POOL_FULL and kv_a.launch_count() == n0
    slot, evicted, _ = store_fused(3, evict_oldest_if_full=True)
    assert (slot, evicted) == (0, 0) and kv_a.pool_tag(0) == 3 and kv_a.pool_count() == 3
    kv_b.pool_evict(0); ref.pool.evict(0)
    assert ref.append_chunk(3, poses[3]) == 0
    assert torch.equal(kv_a.pool[:pool_words * 2].view(torch.int16), kv_b.pool[:pool_words * 2].view(torch.int16))
    # a chunk stored in two calls (layers 0-1, then 2-3) becomes visible after the second
    kv_a.pool_evict(1)
    K, V = ref.chunk_bits(4)
    Kd, Vd = wd.to_device_bf16(np.stack(K)), wd.to_device_bf16(np.stack(V))
    slot, _, _ = kv_a.pool_compress_append(0, 2, Kd[:2], Vd[:2], poses[4], chunk_tag=4)
    assert slot == 1 and kv_a.pool_count() == 2
    slot2, _, _ = kv_a.pool_compress_append(2, 2, Kd[2:], Vd[2:], poses[4], chunk_tag=4, slot=slot)
    assert slot2 == 1 and kv_a.pool_count() == 3 and kv_a.pool_tag(1) == 4
    kv_b.pool_evict(1); ref.pool.evict(1)
    assert ref.append_chunk(4, poses[4]) == 1
    assert torch.equal(kv_a.pool[:pool_words * 2].view(torch.int16), kv_b.pool[:pool_words * 2].view(torch.int16))
    assert kv_a.poll_status() == (0, 0) and kv_b.poll_status() == (0, 0)
