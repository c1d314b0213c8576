"""Pins for the query-based retrieval oracle (Appendix C)."""
import numpy as np

import wkinputs as wi
from oracle import worldkv_oracle as o


def _pool(keys_per_chunk, H=2, d=8):
    pool = o.PoolModel(n_slots=len(keys_per_chunk) + 2, n_layers=1)
    for c, K in enumerate(keys_per_chunk):
        K = np.asarray(K, float).reshape(-1, H, d)
        pool.append([K], [np.zeros_like(K)], [np.arange(K.shape[0])], wi.random_poses(0, 8)[c % 8], tag=c)
    return pool


def test_mass_through_per_chunk_log_sum_exp():
    """Independent route to the same numbers: a log-sum-exp per stored chunk, then a softmax over the chunks' values
    (exp(lse_c) is the chunk's un-normalised mass, so normalising over chunks gives its share)."""
    rng = np.random.default_rng(0)
    H, d, Lq = 2, 8, 5
    chunks = [rng.standard_normal((n, H, d)) * 2 for n in (3, 7, 4, 6)]
    pool = _pool(chunks, H, d)
    Q = rng.standard_normal((Lq, H, d))
    slots, score = o.query_scores(Q, pool, 0)
    lse = np.empty((4, H, Lq))
    for c, K in enumerate(chunks):
        for h in range(H):
            S = (Q[:, h] @ K[:, h].T) / np.sqrt(d)
            mx = S.max(axis=1)
            lse[c, h] = mx + np.log(np.exp(S - mx[:, None]).sum(axis=1))
    w = np.exp(lse - lse.max(axis=0))
    expect = (w / w.sum(axis=0)).mean(axis=(1, 2))
    np.testing.assert_allclose(score, expect, atol=1e-14)
    assert abs(score.sum() - 1) < 1e-14 and slots == [0, 1, 2, 3]


def test_mass_brute_force_loops():
    """The definition with explicit loops on a tiny case: every (head, row) normalises over all stored keys."""
    rng = np.random.default_rng(5)
    H, d, Lq = 1, 4, 2
    chunks = [rng.standard_normal((n, H, d)) for n in (2, 3)]
    pool = _pool(chunks, H, d)
    Q = rng.standard_normal((Lq, H, d))
    expect = np.zeros(2)
    for r in range(Lq):
        logits = [[float(Q[r, 0] @ k[0]) / np.sqrt(d) for k in K] for K in chunks]
        Z = sum(np.exp(x) for row in logits for x in row)
        for c in range(2):
            expect[c] += sum(np.exp(x) for x in logits[c]) / Z
    np.testing.assert_allclose(o.query_scores(Q, pool, 0)[1], expect / Lq, atol=1e-14)


def test_closed_forms():
    H, d = 1, 4
    Q = np.ones((3, H, d))
    zero = np.zeros((5, H, d))
    one = _pool([zero], H, d)
    np.testing.assert_allclose(o.query_scores(Q, one, 0)[1], [1.0])                    # a single chunk takes all the mass
    same = _pool([zero, zero, zero], H, d)
    np.testing.assert_allclose(o.query_scores(Q, same, 0)[1], [1 / 3] * 3, atol=1e-15)  # K = 0: mass follows key counts
    uneven = _pool([np.zeros((2, H, d)), np.zeros((6, H, d))], H, d)
    np.testing.assert_allclose(o.query_scores(Q, uneven, 0)[1], [0.25, 0.75], atol=1e-15)
    # one chunk holds a key aligned with every query: logit 2*4/sqrt(4) = 4 against 0 -> mass e^4 / (e^4 + 5 + 4)
    hot = np.zeros((5, H, d)); hot[2] = 2.0
    pool = _pool([zero, hot], H, d)
    e4 = np.exp(4.0)
    np.testing.assert_allclose(o.query_scores(Q, pool, 0)[1], [5 / (e4 + 9), (e4 + 4) / (e4 + 9)], atol=1e-14)
    ids, sc, margin = o.retrieve_query(Q, pool, 0, 1)
    assert ids.tolist() == [1] and margin > 0.5
    ids, _, margin = o.retrieve_query(Q, same, 0, 2)                                   # exact ties: lowest slots win
    assert ids.tolist() == [0, 1] and margin == 0.0
    ids, _, _ = o.retrieve_query(Q, same, 0, 9)
    assert ids.tolist() == [0, 1, 2]


def test_ranking_follows_the_chunk_a_query_was_drawn_from():
    """Queries equal to (scaled) keys of chunk 2 put most of their mass on chunk 2."""
    rng = np.random.default_rng(3)
    H, d = 2, 16
    chunks = [rng.standard_normal((12, H, d)) for _ in range(5)]
    pool = _pool(chunks, H, d)
    Q = 6.0 * chunks[2][:8]
    ids, sc, _ = o.retrieve_query(Q, pool, 0, 2)
    assert ids[0] == 2 and sc[0] > 0.9
    pool.evict(2)
    assert 2 not in o.retrieve_query(Q, pool, 0, 5)[0]
