"""GPU parity at the benchmark's full sizes, on sampled outputs the oracle can compute one by one.

Pools are filled on the device through the product path (generate -> wk_compress_chunk -> wk_pool_append); the oracle
regenerates, with the numpy generators, exactly the chunks and columns it needs (the retrieved chunks in full width for
the keep-set, the sampled heads' columns of every KV row for attention) and compares:
  * retrieved slot ids: bit-exact;  * keep-sets of the retrieved chunks: bit-exact;
  * attention rows (first/last rows of Q tiles, the ragged last tile) for a few heads: max-abs 2e-2, rel-L2 1e-2.
"""
import os
import sys

import numpy as np
import pytest
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o
from wk_testlib import ATOL_MAX_ABS, RTOL_L2

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def head_cols(h):
    return np.arange(h * 128, (h + 1) * 128)


def fill_pool_on_device(kv, w, poses, layer_count=1):
    """Every chunk 0 .. pool_chunks-1 of every layer, through compress + append; returns the device keep-sets."""
    L, T, D = layer_count, w.T, w.D
    K = torch.empty((L, w.F * T, D), dtype=torch.bfloat16, device="cuda")
    V = torch.empty_like(K)
    keeps = torch.empty((w.pool_chunks, L, w.C), dtype=torch.int32, device="cuda")
    for c in range(w.pool_chunks):
        for l in range(L):
            wd.key_chunk(K[l], w.seed, l, c, T, D, w.sigma, w.F)
            wd.value_chunk(V[l], w.seed, l, c, T, D, w.F)
        kv.compress_chunk(K, keep_idx_out=keeps[c])
        assert kv.pool_append(0, L, K, V, keeps[c], poses[c], chunk_tag=c) == c
    return keeps


def dense_rows_device(w, layer, chunks, n_rows):
    """[n_rows, H, 128] K and V made of the leading rows of consecutive generated chunks."""
    K = torch.empty((n_rows, w.D), dtype=torch.bfloat16, device="cuda")
    V = torch.empty_like(K)
    tmp = torch.empty((w.F * w.T, w.D), dtype=torch.bfloat16, device="cuda")
    r0 = 0
    for c in chunks:
        r1 = min(n_rows, r0 + w.F * w.T)
        wd.key_chunk(tmp, w.seed, layer, c, w.T, w.D, w.sigma, w.F)
        K[r0:r1] = tmp[:r1 - r0]
        wd.value_chunk(tmp, w.seed, layer, c, w.T, w.D, w.F)
        V[r0:r1] = tmp[:r1 - r0]
        r0 = r1
    return K.view(n_rows, w.n_heads, 128), V.view(n_rows, w.n_heads, 128)


def dense_rows_host(w, layer, chunks, n_rows, cols):
    K = np.concatenate([wi.key_chunk_bf16(w.seed, layer, c, w.T, w.D, w.sigma, w.F, cols=cols) for c in chunks])[:n_rows]
    V = np.concatenate([wi.value_chunk_bf16(w.seed, layer, c, w.T, w.D, w.F, cols=cols) for c in chunks])[:n_rows]
    return K, V


def check_sampled_attention(w, layer, O, lse, q_stream, dense_specs, slot_chunks, keep_of_chunk, heads, rows):
    """O: device [Lq, H, 128].  q_stream = (step, chunk) of the query generator; dense_specs = [(chunks, n_rows)];
    slot_chunks = chunk index of every attended slot, in order; keep_of_chunk[c] = oracle keep-set (or None = all)."""
    errs = []
    for h in heads:
        cols = head_cols(h)
        Q = wi.query_bf16(w.seed, layer, q_stream[0], q_stream[1], w.Lq, w.D, cols=cols)[rows]
        Ks, Vs = [], []
        for chunks, n_rows in dense_specs:
            Kd, Vd = dense_rows_host(w, layer, chunks, n_rows, cols)
            Ks.append(Kd); Vs.append(Vd)
        for c in slot_chunks:
            Kc = wi.key_chunk_bf16(w.seed, layer, c, w.T, w.D, w.sigma, w.F, cols=cols)
            Vc = wi.value_chunk_bf16(w.seed, layer, c, w.T, w.D, w.F, cols=cols)
            idx = keep_of_chunk[c]
            Ks.append(Kc if idx is None else Kc[idx]); Vs.append(Vc if idx is None else Vc[idx])
        Kall, Vall = np.concatenate(Ks)[:, None, :], np.concatenate(Vs)[:, None, :]
        O_ref, L_ref = o.attention(Q[:, None, :], Kall, Vall)
        got = O[rows, h, :].float().cpu().numpy().astype(np.float64)
        errs.append((np.abs(got - O_ref[:, 0]).max(), np.linalg.norm(got - O_ref[:, 0]) / np.linalg.norm(O_ref[:, 0])))
        if lse is not None:
            np.testing.assert_allclose(lse[h, rows].cpu().numpy(), L_ref[0], atol=2e-3)
    worst_abs, worst_rel = max(e[0] for e in errs), max(e[1] for e in errs)
    assert worst_abs <= ATOL_MAX_ABS and worst_rel <= RTOL_L2, f"max-abs {worst_abs:.3e} rel-L2 {worst_rel:.3e}"
    return worst_abs, worst_rel


def oracle_keep_set(w, layer, chunk, cache=None):
    """The oracle's keep-set of one generated chunk.  Its full-width keys are drawn by the device side of the seeded
    input generator (bit-identical to the numpy side, see test_device_generators_match_numpy), which at D = 5,120 is far
    quicker than numpy; the scores, the selection and the margin are the oracle's."""
    if cache is not None and chunk in cache:
        return cache[chunk]
    tmp = torch.empty((w.F * w.T, w.D), dtype=torch.bfloat16, device="cuda")
    wd.key_chunk(tmp, w.seed, layer, chunk, w.T, w.D, w.sigma, w.F)
    idx, _, m = o.compress_chunk(wd.to_host_bits(tmp), w.T, w.n_keep)
    assert m > 1e-11
    if cache is not None:
        cache[chunk] = idx
    return idx


SAMPLE_ROWS = {2640: [0, 1, 127, 128, 255, 256, 1333, 2559, 2560, 2639],
               4680: [0, 127, 128, 2300, 4607, 4608, 4679]}


def test_cfg1_matrix_game_single_layer():
    from paper_2605_22718_b200 import WorldKV
    w = wi.WORKLOADS["cfg1"]
    kv = WorldKV(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=w.k, max_batch=1, max_lq=w.Lq, max_splits=8)
    poses = wi.loop_poses(w.seed, w.pool_chunks + 3)
    keeps = fill_pool_on_device(kv, w, poses)
    cur_chunk = w.pool_chunks + 2
    slots, n = kv.retrieve(poses[cur_chunk], w.k)
    ref_slots, _, margin = o.retrieve(poses[cur_chunk], poses[:w.pool_chunks], list(range(w.pool_chunks)), w.k)
    assert margin > 1e-9 and n == w.k
    np.testing.assert_array_equal(slots.cpu().numpy()[:n], ref_slots)
    assert {0, 1} <= set(ref_slots.tolist())          # the loop closes: the chunks around the start come back
    keep_of = {}
    for c in ref_slots.tolist():
        idx, _, m = o.compress_chunk(wi.key_chunk_bf16(w.seed, 0, c, w.T, w.D, w.sigma), w.T, w.n_keep)
        assert m > 1e-11
        np.testing.assert_array_equal(keeps[c, 0].cpu().numpy(), idx)
        keep_of[c] = idx
    Q = torch.empty((w.Lq, w.n_heads, 128), dtype=torch.bfloat16, device="cuda")
    wd.query(Q, w.seed, 0, 0, cur_chunk)
    cur = dense_rows_device(w, 0, [cur_chunk], w.Lq)
    win = dense_rows_device(w, 0, [w.pool_chunks, w.pool_chunks + 1], w.window_frames * w.T)
    lse = torch.empty((w.n_heads, w.Lq), dtype=torch.float32, device="cuda")
    O = kv.memory_attention(0, Q, [cur, win], slots, n, lse_out=lse)
    assert kv.poll_status() == (0, 0)
    rows = SAMPLE_ROWS[w.Lq]
    check_sampled_attention(w, 0, O, lse, (0, cur_chunk), [([cur_chunk], w.Lq), ([w.pool_chunks, w.pool_chunks + 1], w.window_frames * w.T)],
                            ref_slots.tolist(), keep_of, heads=[0, 7, 11], rows=rows)
    O2 = kv.memory_attention(0, Q, [cur, win], slots, n, kv_splits=3)      # a cut KV range gives the same answer
    assert float((O2.float() - O.float()).abs().max()) <= 2e-3


@pytest.mark.parametrize("name,heads", [("paper_mg", [2, 9]), ("paper_lb", [0, 23, 39])])
def test_paper_default_window_both_model_shapes(name, heads):
    """Section 5.1's window: sink 3 + retrieved 9 (six compressed chunks) + recent 3 + denoising 3 = 18 latent frames,
    passed as three dense segments plus six pool slots, at 880 (12 heads) and 1,560 (40 heads) tokens per frame."""
    from paper_2605_22718_b200 import WorldKV
    w = wi.WORKLOADS[name]
    assert w.Lkv == 18 * w.T
    kv = WorldKV(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=w.k, max_batch=1, max_lq=w.Lq, max_splits=2, max_dense_segments=3)
    poses = wi.loop_poses(w.seed, w.pool_chunks + 3)
    keeps = fill_pool_on_device(kv, w, poses)
    cur_chunk = w.pool_chunks + 2
    slots, n = kv.retrieve(poses[cur_chunk], w.k)
    ref_slots, _, margin = o.retrieve(poses[cur_chunk], poses[:w.pool_chunks], list(range(w.pool_chunks)), w.k)
    assert margin > 1e-9 and n == 6
    np.testing.assert_array_equal(slots.cpu().numpy()[:n], ref_slots)
    keep_of = {}
    for c in ref_slots.tolist():
        keep_of[c] = oracle_keep_set(w, 0, c)
        np.testing.assert_array_equal(keeps[c, 0].cpu().numpy(), keep_of[c])
    Q = torch.empty((w.Lq, w.n_heads, 128), dtype=torch.bfloat16, device="cuda")
    wd.query(Q, w.seed, 0, 0, cur_chunk)
    cur = dense_rows_device(w, 0, [cur_chunk], w.Lq)
    sink = dense_rows_device(w, 0, [w.pool_chunks + 4], 3 * w.T)       # any chunk that is not in the pool
    recent = dense_rows_device(w, 0, [w.pool_chunks + 1], 3 * w.T)
    lse = torch.empty((w.n_heads, w.Lq), dtype=torch.float32, device="cuda")
    O = kv.memory_attention(0, Q, [sink, recent, cur], slots, n, lse_out=lse)
    assert kv.poll_status() == (0, 0)
    check_sampled_attention(w, 0, O, lse, (0, cur_chunk),
                            [([w.pool_chunks + 4], 3 * w.T), ([w.pool_chunks + 1], 3 * w.T), ([cur_chunk], w.Lq)],
                            ref_slots.tolist(), keep_of, heads=heads, rows=SAMPLE_ROWS[w.Lq])


def test_cfg3_lingbot_single_layer_and_k_sweep():
    from paper_2605_22718_b200 import WorldKV
    w = wi.WORKLOADS["cfg3"]
    kv = WorldKV(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=16, max_batch=1, max_lq=w.Lq, max_splits=4)
    poses = wi.loop_poses(w.seed, w.pool_chunks + 3)
    keeps = fill_pool_on_device(kv, w, poses)
    cur_chunk = w.pool_chunks + 2
    Q = torch.empty((w.Lq, w.n_heads, 128), dtype=torch.bfloat16, device="cuda")
    wd.query(Q, w.seed, 0, 0, cur_chunk)
    cur = dense_rows_device(w, 0, [cur_chunk], w.Lq)
    win = dense_rows_device(w, 0, [w.pool_chunks, w.pool_chunks + 1], w.window_frames * w.T)
    lses, keep_cache = {}, {}
    for k in w.k_sweep:
        slots, n = kv.retrieve(poses[cur_chunk], k)
        ref_slots, _, margin = o.retrieve(poses[cur_chunk], poses[:w.pool_chunks], list(range(w.pool_chunks)), k)
        assert margin > 1e-9
        np.testing.assert_array_equal(slots.cpu().numpy()[:n], ref_slots)
        lse = torch.empty((w.n_heads, w.Lq), dtype=torch.float32, device="cuda")
        O = kv.memory_attention(0, Q, [cur, win], slots, n, lse_out=lse)
        assert kv.poll_status() == (0, 0)
        assert torch.isfinite(O.float()).all()
        lses[k] = lse.clone()
        # the oracle leg at every budget: the retrieved chunks' keep-sets (full width) bit-exact, then sampled rows --
        # two heads and seven rows at k = 2, one head and four rows at the larger budgets
        for c in ref_slots.tolist():
            idx = oracle_keep_set(w, 0, c, keep_cache)
            np.testing.assert_array_equal(keeps[c, 0].cpu().numpy(), idx)
        heads, rows = ([0, 39], SAMPLE_ROWS[w.Lq]) if k == 2 else ([(7 * k) % w.n_heads], [0, 128, 2300, 4679])
        check_sampled_attention(w, 0, O, lse, (0, cur_chunk),
                                [([cur_chunk], w.Lq), ([w.pool_chunks, w.pool_chunks + 1], w.window_frames * w.T)],
                                ref_slots.tolist(), keep_cache, heads=heads, rows=rows)
        if k == 8:      # properties that hold at any size: slot order does not matter
            rev = torch.flip(slots[:n], dims=[0]).contiguous()
            O_rev = kv.memory_attention(0, Q, [win, cur], rev, n)
            assert float((O_rev.float() - O.float()).abs().max()) <= 4e-3
    ks = sorted(lses)
    for a, b in zip(ks[:-1], ks[1:]):   # attending to more keys can only raise the log-sum-exp
        assert bool((lses[b] >= lses[a] - 1e-4).all())


def test_cfg4_full_uncompressed_history_and_kv_splits():
    from paper_2605_22718_b200 import WorldKV
    w = wi.WORKLOADS["cfg4"]
    kv = WorldKV(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=w.pool_chunks, max_batch=1, max_lq=w.Lq, max_splits=16)
    assert w.C == 3 * w.T                                           # n_keep = 2T: chunks are stored whole
    poses = wi.loop_poses(w.seed, w.pool_chunks + 3)
    keeps = fill_pool_on_device(kv, w, poses)
    np.testing.assert_array_equal(keeps[17, 0].cpu().numpy(), np.arange(3 * w.T))
    cur_chunk = w.pool_chunks + 2
    slots, n = kv.retrieve(poses[cur_chunk], w.pool_chunks)
    ref_slots, _, _ = o.retrieve(poses[cur_chunk], poses[:w.pool_chunks], list(range(w.pool_chunks)), w.pool_chunks)
    assert n == w.pool_chunks
    np.testing.assert_array_equal(slots.cpu().numpy(), ref_slots)
    Q = torch.empty((w.Lq, w.n_heads, 128), dtype=torch.bfloat16, device="cuda")
    wd.query(Q, w.seed, 0, 0, cur_chunk)
    cur = dense_rows_device(w, 0, [cur_chunk], w.Lq)
    outs = {}
    for splits in (0, 1, 4, 16):
        lse = torch.empty((w.n_heads, w.Lq), dtype=torch.float32, device="cuda")
        outs[splits] = (kv.memory_attention(0, Q, [cur], slots, n, lse_out=lse, kv_splits=splits), lse)
        assert kv.poll_status() == (0, 0)
    O, lse = outs[0]
    assert 330000 + w.Lq == w.Lq + w.pool_chunks * w.C
    check_sampled_attention(w, 0, O, lse, (0, cur_chunk), [([cur_chunk], w.Lq)], ref_slots.tolist(),
                            {c: None for c in range(w.pool_chunks)}, heads=[5], rows=[0, 1300, 2639])
    for splits in (1, 4, 16):
        assert float((outs[splits][0].float() - O.float()).abs().max()) <= 2e-3
        assert float((outs[splits][1] - lse).abs().max()) <= 2e-3


def test_cfg4c_compressed_history_and_kv_splits():
    """The one-minute history with every chunk compressed to 50 %: 125 x 1,320 = 165,000 stored tokens, all attended
    (plus the 2,640 of the denoising chunk).  All 125 keep-sets are compared with the oracle's; sampled rows at every
    KV split against the oracle."""
    from paper_2605_22718_b200 import WorldKV
    w = wi.WORKLOADS["cfg4c"]
    kv = WorldKV(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                 max_k=w.pool_chunks, max_batch=1, max_lq=w.Lq, max_splits=16)
    assert w.pool_chunks * w.C == 165000 and 2 * w.C == 3 * w.T
    poses = wi.loop_poses(w.seed, w.pool_chunks + 3)
    keeps = fill_pool_on_device(kv, w, poses)
    keep_of = {}
    for c in range(w.pool_chunks):
        keep_of[c] = oracle_keep_set(w, 0, c)
        np.testing.assert_array_equal(keeps[c, 0].cpu().numpy(), keep_of[c])
    cur_chunk = w.pool_chunks + 2
    slots, n = kv.retrieve(poses[cur_chunk], w.pool_chunks)
    ref_slots, _, _ = o.retrieve(poses[cur_chunk], poses[:w.pool_chunks], list(range(w.pool_chunks)), w.pool_chunks)
    assert n == w.pool_chunks
    np.testing.assert_array_equal(slots.cpu().numpy(), ref_slots)
    Q = torch.empty((w.Lq, w.n_heads, 128), dtype=torch.bfloat16, device="cuda")
    wd.query(Q, w.seed, 0, 0, cur_chunk)
    cur = dense_rows_device(w, 0, [cur_chunk], w.Lq)
    for splits, head in ((0, 5), (1, 0), (4, 11), (16, 7)):
        lse = torch.empty((w.n_heads, w.Lq), dtype=torch.float32, device="cuda")
        O = kv.memory_attention(0, Q, [cur], slots, n, lse_out=lse, kv_splits=splits)
        assert kv.poll_status() == (0, 0)
        check_sampled_attention(w, 0, O, lse, (0, cur_chunk), [([cur_chunk], w.Lq)], ref_slots.tolist(), keep_of,
                                heads=[head], rows=[0, 129, 1300, 2639])


def test_cfg2_chunk_step_in_the_bench_configuration():
    """The benchmark's own object and launch configuration (30 layers, 250-chunk pool): one chunk step, then one
    (layer, denoising step) output and the step's retrieval and compression are checked against the oracle."""
    sys.path.insert(0, ROOT)
    import bench
    w = wi.WORKLOADS["cfg2"]
    b = bench.ChunkStepBench(w, 0, e2e=False)
    kv = b.kv
    tags = [kv.pool_tag(s) for s in range(w.pool_chunks)]
    assert tags == list(range(w.pool_chunks))
    b.step()
    torch.cuda.synchronize()
    assert kv.poll_status() == (0, 0)
    pose = b.poses[w.pool_chunks]
    ref_slots, _, margin = o.retrieve(pose, b.poses[:w.pool_chunks], list(range(w.pool_chunks)), w.k)
    assert margin > 1e-9
    np.testing.assert_array_equal(b.slots.cpu().numpy()[:w.k], ref_slots)
    layer, step = 17, 2
    keep_of = {}
    for c in ref_slots.tolist():
        idx, _, m = o.compress_chunk(wi.key_chunk_bf16(w.seed, layer, c, w.T, w.D, w.sigma), w.T, w.n_keep)
        assert m > 1e-11
        keep_of[c] = idx
    base = w.pool_chunks + 4
    check_sampled_attention(w, layer, b.O[layer, step], None, (step, 0),
                            [([base + 3], w.Lq), ([base + 1, base + 2], w.window_frames * w.T)],
                            ref_slots.tolist(), keep_of, heads=[3, 10], rows=SAMPLE_ROWS[w.Lq])
    # the chunk that left the window in this step: its keep-set for two layers, and the slot it went to
    for l in (0, 29):
        idx, _, m = o.compress_chunk(wi.key_chunk_bf16(w.seed, l, w.pool_chunks, w.T, w.D, w.sigma), w.T, w.n_keep)
        assert m > 1e-11
        np.testing.assert_array_equal(b.keep[l].cpu().numpy(), idx)
    assert kv.pool_count() == w.pool_chunks and kv.pool_tag(0) == w.pool_chunks    # oldest evicted, slot 0 reused
