"""Pins for the pool model (Section 4.2: evicted chunks are stored, indexed by their pose)."""
import numpy as np
import pytest

import wkinputs as wi
from oracle import worldkv_oracle as o


def _chunk(T, D, c):
    return (wi.key_chunk_bf16(0, 0, c, T, D, 0.1), wi.value_chunk_bf16(0, 0, c, T, D))


def test_lowest_free_slot_fifo_oldest_and_full():
    T, D = 4, 8
    pool = o.PoolModel(n_slots=3, n_layers=2)
    poses = wi.random_poses(0, 6)
    idx = np.arange(T + 2, dtype=np.int32)
    slots = []
    for c in range(3):
        K, V = _chunk(T, D, c)
        slots.append(pool.append([K, K], [V, V], [idx, idx], poses[c], tag=c))
    assert slots == [0, 1, 2] and pool.count() == 3 and pool.oldest() == 0
    with pytest.raises(RuntimeError):
        K, V = _chunk(T, D, 3)
        pool.append([K, K], [V, V], [idx, idx], poses[3])
    pool.evict(1)
    assert pool.valid_slots() == [0, 2] and pool.oldest() == 0
    K, V = _chunk(T, D, 4)
    assert pool.append([K, K], [V, V], [idx, idx], poses[4], tag=4) == 1     # lowest free slot is reused
    pool.evict(0)
    assert pool.oldest() == 2                                               # append order, not slot order
    with pytest.raises(KeyError):
        pool.evict(0)
    assert pool.K[(1, 1)].shape == (T + 2, D)
    np.testing.assert_array_equal(pool.K[(1, 1)], K[idx])


def test_pool_retrieve_uses_only_valid_slots():
    pool = o.PoolModel(n_slots=8, n_layers=1)
    poses = wi.random_poses(3, 8)
    T, D = 4, 8
    idx = np.arange(T, dtype=np.int32)
    for c in range(8):
        K, V = _chunk(T, D, c)
        pool.append([K], [V], [idx], poses[c])
    ids_all, _, _ = pool.retrieve(poses[5], 3)
    assert ids_all[0] == 5
    pool.evict(5)
    ids, dist, _ = pool.retrieve(poses[5], 8)
    assert 5 not in ids and len(ids) == 7
    ref_ids, ref_d, _ = o.retrieve(poses[5], np.delete(poses, 5, axis=0), [0, 1, 2, 3, 4, 6, 7], 8)
    np.testing.assert_array_equal(ids, ref_ids)
    np.testing.assert_array_equal(dist, ref_d)
