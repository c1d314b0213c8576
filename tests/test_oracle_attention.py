"""Pins for the attention oracle (Section 4.2's assembled window, softmax attention)."""
import math

import numpy as np
import pytest
import torch

import wkinputs as wi
from oracle import worldkv_oracle as o


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_two_key_closed_form_and_default_scale():
    """d = 4, q = (2,0,0,0), keys (1,0,0,0) and 0: logits are 2/sqrt(4) = 1 and 0, so the weights are
    e/(1+e) and 1/(1+e).  Pins the scale, the softmax direction and the P V contraction."""
    Q = np.zeros((1, 1, 4)); Q[0, 0, 0] = 2.0
    K = np.zeros((2, 1, 4)); K[0, 0, 0] = 1.0
    V = np.array([[[1.0, 10.0, 0.0, -1.0]], [[3.0, 20.0, 0.0, 1.0]]])
    O, LSE = o.attention(Q, K, V)
    w = math.e / (1 + math.e)
    np.testing.assert_allclose(O[0, 0], w * V[0, 0] + (1 - w) * V[1, 0], atol=1e-15)
    assert LSE[0, 0] == pytest.approx(math.log(1 + math.e), abs=1e-15)
    O2, _ = o.attention(Q, K, V, scale=0.0)
    np.testing.assert_allclose(O2[0, 0], V.mean(axis=0)[0], atol=1e-15)


def test_degenerate_cases():
    Q, K, V = rnd((5, 3, 8), 0), rnd((7, 3, 8), 1), rnd((7, 3, 8), 2)
    O, _ = o.attention(Q, K[:1], V[:1])                                  # one key: O = v0
    np.testing.assert_allclose(O, np.broadcast_to(V[0], O.shape), atol=1e-15)
    Vc = np.broadcast_to(V[3], V.shape)
    np.testing.assert_allclose(o.attention(Q, K, Vc)[0], np.broadcast_to(V[3], Q.shape), atol=1e-14)
    O0, L0 = o.attention(Q, np.zeros_like(K), V)                         # K = 0: uniform weights
    np.testing.assert_allclose(O0, np.broadcast_to(V.mean(0), Q.shape), atol=1e-15)
    np.testing.assert_allclose(L0, math.log(7), atol=1e-15)
    ones = np.ones_like(V)                                               # weights sum to one
    np.testing.assert_allclose(o.attention(Q, K, ones)[0], 1.0, atol=1e-14)


def test_heads_are_independent_and_not_mixed():
    Q, K, V = rnd((4, 2, 8), 3), rnd((9, 2, 8), 4), rnd((9, 2, 8), 5)
    O, L = o.attention(Q, K, V)
    for h in range(2):
        Oh, Lh = o.attention(Q[:, h:h + 1], K[:, h:h + 1], V[:, h:h + 1])
        np.testing.assert_allclose(O[:, h], Oh[:, 0], atol=1e-15)
        np.testing.assert_allclose(L[h], Lh[0], atol=1e-15)


def test_matches_torch_sdpa_fp64():
    Q, K, V = rnd((33, 3, 16), 6), rnd((70, 3, 16), 7), rnd((70, 3, 16), 8)
    t = lambda x: torch.from_numpy(x).permute(1, 0, 2)[None]            # [1, H, L, d]
    ref = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V))[0].permute(1, 0, 2).numpy()
    O, LSE = o.attention(Q, K, V)
    np.testing.assert_allclose(O, ref, atol=1e-13)
    ref_lse = torch.logsumexp(torch.einsum("qhd,khd->hqk", torch.from_numpy(Q), torch.from_numpy(K)) / 4.0, -1)
    np.testing.assert_allclose(LSE, ref_lse.numpy(), atol=1e-13)
    rows = np.array([0, 5, 32])
    np.testing.assert_allclose(o.attention(Q, K, V, rows=rows)[0], ref[rows], atol=1e-13)


def test_split_anywhere_and_merge():
    Q, K, V = rnd((6, 2, 8), 9), rnd((50, 2, 8), 10) * 3, rnd((50, 2, 8), 11)
    O, L = o.attention(Q, K, V)
    for cuts in ([1], [17, 18], [10, 25, 49]):
        b = [0] + cuts + [50]
        parts = [o.attention(Q, K[a:c], V[a:c]) for a, c in zip(b[:-1], b[1:])]
        Om, Lm = o.merge_partials([p[0] for p in parts], [p[1] for p in parts])
        np.testing.assert_allclose(Om, O, atol=1e-14)
        np.testing.assert_allclose(Lm, L, atol=1e-14)


def _tiny_pool(T=6, H=2, d=8, n_chunks=4, n_keep=None, seed=0):
    D = H * d
    n_keep = 2 * T if n_keep is None else n_keep
    pool = o.PoolModel(n_slots=n_chunks + 1, n_layers=1)
    Ks, Vs = [], []
    for c in range(n_chunks):
        K = wi.key_chunk_bf16(seed, 0, c, T, D, 0.1).reshape(3 * T, H, d)
        V = wi.value_chunk_bf16(seed, 0, c, T, D).reshape(3 * T, H, d)
        idx, _, _ = o.compress_chunk(K.reshape(3 * T, D), T, n_keep)
        pool.append([K], [V], [idx], wi.random_poses(seed, n_chunks)[c], tag=c)
        Ks.append(K); Vs.append(V)
    return pool, Ks, Vs


def test_identity_pool_equals_full_history_attention():
    """n_keep = 2T and k = M: the memory attention is attention over the concatenated history."""
    T, H, d = 6, 2, 8
    pool, Ks, Vs = _tiny_pool(T, H, d)
    Q = wi.query_bf16(0, 0, 0, 0, T, H * d).reshape(T, H, d)
    cur = (wi.key_chunk_bf16(0, 0, 9, T, H * d, 0.1).reshape(-1, H, d), wi.value_chunk_bf16(0, 0, 9, T, H * d).reshape(-1, H, d))
    O, L = o.memory_attention(Q, [cur], pool, 0, pool.valid_slots())
    Kfull = np.concatenate([cur[0]] + Ks); Vfull = np.concatenate([cur[1]] + Vs)
    Of, Lf = o.attention(Q, Kfull, Vfull)
    np.testing.assert_array_equal(O, Of)
    np.testing.assert_array_equal(L, Lf)


def test_permuting_segments_and_slots_leaves_output_unchanged():
    T, H, d = 6, 2, 8
    pool, Ks, Vs = _tiny_pool(T, H, d, n_keep=T // 2)
    assert pool.K[(0, 0)].shape == (T + T // 2, H, d)
    Q = wi.query_bf16(0, 0, 0, 0, 2 * T, H * d).reshape(2 * T, H, d)
    segs = [(Ks[0][:T], Vs[0][:T]), (Ks[1][:5], Vs[1][:5])]
    O, L = o.memory_attention(Q, segs, pool, 0, [0, 1, 2, 3])
    O2, L2 = o.memory_attention(Q, segs[::-1], pool, 0, [3, 1, 0, 2])
    np.testing.assert_allclose(O2, O, atol=1e-12)
    np.testing.assert_allclose(L2, L, atol=1e-12)
    O3, _ = o.memory_attention(Q, segs, pool, 0, [0, 1, 2, 3, 7, -1])     # invalid slots are skipped
    np.testing.assert_array_equal(O3, O)
    O4, _ = o.memory_attention(Q, segs, pool, 0, [0, 0])                  # multiset semantics (R8)
    K2, V2 = o.assemble_kv(segs, pool, 0, [0])
    O5, _ = o.attention(Q, np.concatenate([K2, pool.K[(0, 0)]]), np.concatenate([V2, pool.V[(0, 0)]]))
    np.testing.assert_array_equal(O4, O5)


def test_compressed_rows_are_the_kept_rows():
    T, H, d = 8, 1, 8
    pool, Ks, Vs = _tiny_pool(T, H, d, n_chunks=2, n_keep=T // 2)
    idx, _, _ = o.compress_chunk(Ks[1].reshape(3 * T, -1), T, T // 2)
    np.testing.assert_array_equal(pool.K[(0, 1)], Ks[1][idx])
    np.testing.assert_array_equal(pool.V[(0, 1)], Vs[1][idx])
    assert len(idx) == T + T // 2


def test_bf16_inputs_are_widened_exactly():
    bits = np.array([0x3F80, 0xBF80, 0x4049, 0x0000, 0x3DCD], dtype=np.uint16)       # 1, -1, 3.140625, 0, 0.10009765625
    np.testing.assert_array_equal(o.widen_bf16(bits), [1.0, -1.0, 3.140625, 0.0, 0.10009765625])


def test_cfg0_kv_length():
    w = wi.WORKLOADS["cfg0"]
    assert w.Lkv == 3960 and w.Lq == 880
    assert wi.WORKLOADS["cfg1"].Lkv == 13200 and wi.WORKLOADS["cfg2"].Lkv == 18480
