"""Pins for the compression oracle (Eq. 5 and the keep-set of Section 4.3)."""
import math
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import wkinputs as wi
from oracle import worldkv_oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_sizes.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def _chunk(anchor, others):
    return np.concatenate([np.asarray(anchor, float), np.asarray(others, float)], axis=0)


@pytest.mark.parametrize("form", [o.compression_scores_definitional, o.compression_scores_factorised])
def test_planar_closed_form(form):
    """In the plane the cosine of two vectors is cos(angle difference): a key at angle phi scores
    mean_i cos(phi - theta_i), whatever the vectors' lengths.  Catches a missing normalisation,
    a wrong denominator, a transposed operand and a wrong anchor frame."""
    T = 5
    theta = np.array([0.1, 0.7, 1.9, 3.0, 4.4])
    ra = np.array([0.5, 1.0, 2.0, 3.0, 0.25])
    phi = np.linspace(-3, 3, 2 * T)
    rn = np.linspace(0.3, 4.0, 2 * T)
    A = np.stack([ra * np.cos(theta), ra * np.sin(theta)], 1)
    N = np.stack([rn * np.cos(phi), rn * np.sin(phi)], 1)
    expect = np.array([np.mean(np.cos(p - theta)) for p in phi])
    got = form(_chunk(A, N), T)
    np.testing.assert_allclose(got, expect, atol=1e-14)
    assert got.shape == (2 * T,)


@pytest.mark.parametrize("form", [o.compression_scores_definitional, o.compression_scores_factorised])
def test_basis_anchor_closed_forms(form):
    T, D = 6, 9
    A = np.eye(D)[:T] * np.arange(1, T + 1)[:, None]       # anchors: scaled distinct basis vectors
    N = np.zeros((2 * T, D))
    N[0, 2] = 7.0                 # parallel to one anchor  ->  1/T
    N[1, 2] = -0.5                # antiparallel            -> -1/T
    N[2, 7] = 3.0                 # orthogonal to all       ->  0
    N[3, :T] = 1.0                # equal mix of all anchors -> T * (1/sqrt(T)) / T = 1/sqrt(T)
    N[4, :] = 0.0                 # zero key                ->  0 (reading R3)
    N[5, 0], N[5, 1] = 3.0, 4.0   # 3-4-5 triangle          -> (0.6 + 0.8) / T
    N[6:] = N[0]
    s = form(_chunk(A, N), T)
    np.testing.assert_allclose(s[:6], [1 / T, -1 / T, 0, 1 / math.sqrt(T), 0, 1.4 / T], atol=1e-15)


def test_zero_anchor_still_counts_in_mean():
    """A zero anchor key contributes cosine 0 but the mean stays over all T anchors (R3)."""
    A = np.array([[1.0, 0.0], [0.0, 0.0]])
    N = np.array([[2.0, 0.0], [0.0, 1.0], [1.0, 0.0], [1.0, 1.0]])
    for form in (o.compression_scores_definitional, o.compression_scores_factorised):
        np.testing.assert_allclose(form(_chunk(A, N), 2), [0.5, 0.0, 0.5, 0.5 / math.sqrt(2)], atol=1e-15)


def test_scale_invariance_and_row_permutations():
    rng = np.random.default_rng(3)
    T, D = 7, 12
    K = rng.standard_normal((3 * T, D))
    s = o.compression_scores_definitional(K, T)
    K2 = K * rng.uniform(0.1, 9.0, size=(3 * T, 1))                      # positive row scaling
    np.testing.assert_allclose(o.compression_scores_definitional(K2, T), s, atol=1e-14)
    perm_a = rng.permutation(T)
    K3 = np.concatenate([K[:T][perm_a], K[T:]])                         # anchors in another order
    np.testing.assert_allclose(o.compression_scores_definitional(K3, T), s, atol=1e-14)
    perm_n = rng.permutation(2 * T)
    K4 = np.concatenate([K[:T], K[T:][perm_n]])                         # non-anchors permuted
    np.testing.assert_allclose(o.compression_scores_definitional(K4, T), s[perm_n], atol=1e-14)
    Rot, _ = np.linalg.qr(rng.standard_normal((D, D)))                  # cosine is rotation invariant
    np.testing.assert_allclose(o.compression_scores_definitional(K @ Rot, T), s, atol=1e-13)


def test_brute_force_loops_tiny():
    """Eq. 5 with explicit Python loops and math.sqrt on a tiny case."""
    rng = np.random.default_rng(11)
    T, D, F = 4, 5, 3
    K = rng.standard_normal((F * T, D))
    expect = []
    for j in range(T, F * T):
        acc = 0.0
        for i in range(T):
            dot = sum(K[j][c] * K[i][c] for c in range(D))
            nj = math.sqrt(sum(v * v for v in K[j]))
            ni = math.sqrt(sum(v * v for v in K[i]))
            acc += dot / (nj * ni)
        expect.append(acc / T)
    np.testing.assert_allclose(o.compression_scores_definitional(K, T), expect, atol=1e-14)
    np.testing.assert_allclose(o.compression_scores_factorised(K, T), expect, atol=1e-14)


def test_forms_agree_on_generated_chunks():
    for seed, chunk in [(0, 0), (0, 3), (5, 1)]:
        K = wi.key_chunk_bf16(seed, 0, chunk, 880, 256, 0.1)
        i1, s1, m1 = o.compress_chunk(K, 880, 440, "definitional")
        i2, s2, m2 = o.compress_chunk(K, 880, 440, "factorised")
        assert np.abs(s1 - s2).max() < 1e-12
        assert m1 > 1e-11, "generated chunk is tie-ambiguous"
        np.testing.assert_array_equal(i1, i2)


def test_keep_set_planar_order():
    """Keys at known angles from a single anchor direction: the kept ones are those at the
    largest angles (lowest cosine), returned as ascending chunk-local indices after the anchors."""
    T = 4
    A = np.tile([[1.0, 0.0]], (T, 1))
    ang = np.array([0.1, 2.0, 0.3, 3.0, 1.0, 2.5, 0.2, 1.5])
    N = np.stack([np.cos(ang), np.sin(ang)], 1)
    idx, s, margin = o.compress_chunk(_chunk(A, N), T, 3)
    np.testing.assert_allclose(s, np.cos(ang), atol=1e-15)
    np.testing.assert_array_equal(idx, [0, 1, 2, 3, T + 1, T + 3, T + 5])     # angles 2.0, 3.0, 2.5
    assert margin == pytest.approx(math.cos(1.5) - math.cos(2.0))


def test_tie_break_lowest_index():
    T, D = 5, 3
    K = np.ones((3 * T, D))                     # every score is exactly 1
    idx, s, margin = o.compress_chunk(K, T, 4)
    np.testing.assert_allclose(s, 1.0, atol=1e-15)
    idx2, _ = o.keep_set(np.ones(2 * T), T, 4)
    np.testing.assert_array_equal(idx2, list(range(T)) + [T, T + 1, T + 2, T + 3])
    idx3, m3 = o.keep_set(np.array([0.5, 0.1, 0.5, 0.1, 0.5, 0.9]), 3, 3)
    np.testing.assert_array_equal(idx3, [0, 1, 2, 3 + 0, 3 + 1, 3 + 3])       # 0.1, 0.1, then the first 0.5
    assert m3 == 0.0


def test_counts_match_paper_sizes():
    g = _golden()
    F = int(g["frames_per_chunk"])
    assert g["window_frames_total"] == (g["window_frames_sink"] + g["window_frames_retrieval"]
                                        + g["window_frames_recent"] + g["window_frames_denoising"])
    for T in (int(g["tokens_per_frame_matrix_game"]), int(g["tokens_per_frame_lingbot"])):
        n_keep = int(g["retain_fraction_non_anchor"] * (F - 1) * T)
        rng = np.random.default_rng(T)
        idx, _ = o.keep_set(rng.standard_normal((F - 1) * T), T, n_keep)
        assert len(idx) == g["compressed_chunk_in_frames"] * T == 0.5 * F * T   # exactly 50 %
        assert len(np.unique(idx)) == len(idx) and (np.diff(idx) > 0).all()
        np.testing.assert_array_equal(idx[:T], np.arange(T))                    # anchor kept whole
    assert wi.WORKLOADS["cfg0"].C == 1320 and wi.WORKLOADS["cfg3"].C == 2340
    # storage model behind "approximately 3.4 GB per chunk": K and V, 16-bit, 40 layers x 5120 wide
    gb = 3 * 1560 * 2 * 2 * 5120 * 40 / 1e9
    assert abs(gb - g["lingbot_chunk_gigabytes_all_layers"]) / gb < 0.15


def test_retention_ladder_is_nested():
    """Table 2's ladder 3 -> {1.0, 1.25, 1.5, 2.0, 2.5, 3.0}: keep-sets are nested, the ends are
    anchor-only and identity."""
    T = 16
    K = wi.key_chunk_bf16(2, 0, 0, T, 32, 0.1)
    prev = None
    for n_keep in (0, T // 4, T // 2, T, 3 * T // 2, 2 * T):
        idx, _, _ = o.compress_chunk(K, T, n_keep)
        assert len(idx) == T + n_keep
        if prev is not None:
            assert set(prev) <= set(idx)
        prev = idx
    np.testing.assert_array_equal(o.compress_chunk(K, T, 0)[0], np.arange(T))
    np.testing.assert_array_equal(o.compress_chunk(K, T, 2 * T)[0], np.arange(3 * T))


@settings(max_examples=40, deadline=None)
@given(st.integers(1, 6), st.integers(1, 7), st.integers(0, 2 ** 31 - 1), st.data())
def test_keep_set_is_the_sorted_prefix(T, D, seed, data):
    rng = np.random.default_rng(seed)
    K = rng.integers(-2, 3, size=(3 * T, D)).astype(float)      # small integers: many exact ties
    n_keep = data.draw(st.integers(0, 2 * T))
    idx, s, _ = o.compress_chunk(K, T, n_keep, "definitional")
    kept = idx[T:] - T
    ranked = sorted(range(2 * T), key=lambda j: (s[j], j))[:n_keep]
    assert sorted(ranked) == list(kept)
    dropped = sorted(set(range(2 * T)) - set(kept))
    if len(kept) and dropped:
        assert max(s[kept]) <= min(s[dropped])


def test_redrawn_positions_are_enriched_in_the_keep_set():
    """Soft sanity check of generator + oracle together: positions redrawn after the anchor frame
    have keys unrelated to the anchor at the same position and are kept more often."""
    T = 880
    K = wi.key_chunk_bf16(0, 0, 4, T, 256, 0.1)
    idx, _, _ = o.compress_chunk(K, T, 440)
    r1 = wi.redraw_mask(0, 0, [13], T)[0]
    r2 = wi.redraw_mask(0, 0, [14], T)[0] | r1
    redrawn = np.concatenate([r1, r2])
    kept = idx[T:] - T
    assert redrawn[kept].mean() > redrawn.mean() + 0.05


# ----------------------------------------------------------------------------- per-head keep-sets
def _head_chunk(T=12, H=3, d=8, seed=0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((3 * T, H * d)), T, H, d


def test_per_head_with_one_head_is_the_whole_key_reading():
    K, T, H, d = _head_chunk(H=1)
    idx, sc, m = o.compress_chunk_per_head(K, T, T // 2, 1)
    idx0, sc0, m0 = o.compress_chunk(K, T, T // 2)
    np.testing.assert_array_equal(idx[0], idx0)
    np.testing.assert_array_equal(sc[0], sc0)
    assert m == m0


def test_per_head_scores_are_blind_to_the_other_heads():
    """Brute force per head from the definition (mean cosine to every anchor key of that head), and: changing head 1's
    columns leaves head 0's and head 2's keep-sets alone; permuting the heads permutes the keep-sets."""
    K, T, H, d = _head_chunk()
    idx, sc, _ = o.compress_chunk_per_head(K, T, 7, H)
    for h in range(H):
        Kh = K[:, h * d:(h + 1) * d]
        A, N = Kh[:T], Kh[T:]
        cos = (N / np.linalg.norm(N, axis=1, keepdims=True)) @ (A / np.linalg.norm(A, axis=1, keepdims=True)).T
        np.testing.assert_allclose(sc[h], cos.mean(axis=1), atol=1e-14)
        keep = np.sort(np.argsort(cos.mean(axis=1), kind="stable")[:7]) + T
        np.testing.assert_array_equal(idx[h], np.concatenate([np.arange(T), keep]))
    K2 = K.copy()
    K2[:, d:2 * d] = np.random.default_rng(9).standard_normal((3 * T, d))
    idx2, _, _ = o.compress_chunk_per_head(K2, T, 7, H)
    np.testing.assert_array_equal(idx2[0], idx[0])
    np.testing.assert_array_equal(idx2[2], idx[2])
    assert not np.array_equal(idx2[1], idx[1])
    perm = [2, 0, 1]
    Kp = np.concatenate([K[:, p * d:(p + 1) * d] for p in perm], axis=1)
    idxp, _, _ = o.compress_chunk_per_head(Kp, T, 7, H)
    np.testing.assert_array_equal(idxp, idx[perm])


def test_per_head_redundancy_is_found_head_by_head():
    """Head 0 of the second frame repeats the anchor frame's head 0 (most similar to the anchors -> dropped first),
    head 1 of the third frame does; each head drops its own redundant frame."""
    rng = np.random.default_rng(4)
    T, d = 10, 16
    base = rng.standard_normal((T, d))
    K = rng.standard_normal((3 * T, 2 * d))
    K[:T, :d] = base + 5.0                      # a common offset makes anchor keys of head 0 alike
    K[T:2 * T, :d] = base + 5.0                 # frame 1, head 0: copies of the anchors
    K[:T, d:] = base - 5.0
    K[2 * T:, d:] = base - 5.0                  # frame 2, head 1: copies of the anchors
    idx, _, _ = o.compress_chunk_per_head(K, T, T, 2)
    np.testing.assert_array_equal(idx[0][T:], np.arange(2 * T, 3 * T))   # head 0 keeps frame 2
    np.testing.assert_array_equal(idx[1][T:], np.arange(T, 2 * T))       # head 1 keeps frame 1


def test_pool_model_stores_per_head_rows():
    K, T, H, d = _head_chunk()
    V = np.random.default_rng(2).standard_normal(K.shape)
    idx, _, _ = o.compress_chunk_per_head(K, T, 5, H)
    pool = o.PoolModel(n_slots=2, n_layers=1)
    s = pool.append([K.reshape(-1, H, d)], [V.reshape(-1, H, d)], [idx], wi.random_poses(0, 1)[0])
    Ks = pool.K[(0, s)]
    assert Ks.shape == (T + 5, H, d)
    for h in range(H):
        np.testing.assert_array_equal(Ks[:, h], K.reshape(-1, H, d)[idx[h], h])
        np.testing.assert_array_equal(pool.V[(0, s)][:, h], V.reshape(-1, H, d)[idx[h], h])
