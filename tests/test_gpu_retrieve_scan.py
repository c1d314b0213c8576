"""GPU parity of the streaming retrieval scan (Eq. 4, distance of Section 5.1) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import wkinputs as wi
from oracle import worldkv_oracle as o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kv():
    from paper_2605_22718_b200 import WorldKV
    return WorldKV(n_layers=1, n_heads=1, tokens_per_frame=40, n_keep=23, pool_slots=2, max_k=2, max_batch=1, max_lq=64,
                   max_splits=2, max_dense_segments=1)


def _check(kv, poses, cur, k, valid=None, need_margin=True):
    n = poses.shape[0]
    P = torch.from_numpy(poses).cuda()
    V = None if valid is None else torch.from_numpy(valid.astype(np.int32)).cuda()
    ids = torch.full((max(k, 1) + 3,), 77, dtype=torch.int32, device="cuda")
    dist = torch.full((max(k, 1) + 3,), -5.0, dtype=torch.float64, device="cuda")
    kv.retrieve_scan(P, cur, k, valid=V, ids_out=ids, dist_out=dist)
    cand = np.arange(n) if valid is None else np.nonzero(valid)[0]
    ref_ids, ref_d, margin = o.retrieve(cur, poses[cand], cand, k)
    got = ids.cpu().numpy()
    cnt = len(ref_ids)
    if need_margin:
        assert margin > 1e-9, margin       # the k-th and (k+1)-th are far enough apart for ids to be unique in fp64
    np.testing.assert_array_equal(got[:cnt], ref_ids)
    assert (got[cnt:] == -1).all()
    np.testing.assert_allclose(dist.cpu().numpy()[:cnt], ref_d, rtol=0, atol=1e-12)
    return got[:cnt]


@pytest.mark.parametrize("n,k", [(1, 1), (5, 8), (300, 8), (300, 64), (4096, 16), (65539, 8), (100003, 1)])
def test_scan_matches_oracle_small_and_ragged(kv, n, k):
    poses = wi.random_poses(21, n + 1)
    _check(kv, poses[1:], poses[0], k)
    valid = (wi.hash64(5, wi.STREAM_MISC, np.arange(n)) % np.uint64(3) != 0) if n > 1 else np.ones(1, bool)
    _check(kv, poses[1:], poses[0], k, valid=valid)


def test_scan_agrees_with_the_pool_sized_entry_point(kv):
    from paper_2605_22718_b200 import retrieve_noalloc
    poses = wi.loop_poses(4, 2000)
    P = torch.from_numpy(poses[:-1].copy()).cuda()
    valid = torch.ones(P.shape[0], dtype=torch.int32, device="cuda")
    valid[::7] = 0
    a = torch.empty(8, dtype=torch.int32, device="cuda")
    da = torch.empty(8, dtype=torch.float64, device="cuda")
    retrieve_noalloc(P, valid, poses[-1], 8, 8, a, da)
    b = torch.empty(8, dtype=torch.int32, device="cuda")
    db = torch.empty(8, dtype=torch.float64, device="cuda")
    kv.retrieve_scan(P, poses[-1], 8, valid=valid, ids_out=b, dist_out=db)
    assert torch.equal(a, b) and torch.equal(da, db)     # same arithmetic, same bits


def test_scan_ties_and_degenerate_sets(kv):
    poses = wi.random_poses(9, 50)
    cur = poses[0]
    dup = np.concatenate([poses[1:], poses[1:], poses[1:]])          # every pose three times: ties -> lowest index
    got = _check(kv, dup, cur, 6, need_margin=False)
    assert got[1] == got[0] + 49 and got[2] == got[0] + 98 and got[4] == got[3] + 49      # copies in index order
    same_t = poses[1:].copy(); same_t[:, 0:3] = cur[0:3]             # zero translation maximum: term dropped
    _check(kv, same_t, cur, 4)
    same_q = poses[1:].copy(); same_q[:, 4:8] = cur[4:8]             # zero rotation maximum
    _check(kv, same_q, cur, 4)
    all_same = np.repeat(cur[None], 40, axis=0)                      # both maxima zero: every distance 0
    got = _check(kv, all_same, cur, 5, need_margin=False)
    assert got.tolist() == [0, 1, 2, 3, 4]
    none_valid = np.zeros(49, bool)
    assert len(_check(kv, poses[1:], cur, 3, valid=none_valid, need_margin=False)) == 0
    P = torch.empty((0, 8), dtype=torch.float32, device="cuda")
    assert (kv.retrieve_scan(P, cur, 2).cpu().numpy() == -1).all()   # empty candidate set
    assert (kv.retrieve_scan(torch.from_numpy(poses).cuda(), cur, 0).cpu().numpy() == -1).all()


def test_scan_adversarial_order(kv):
    """Candidates sorted from far to near: every one of them beats the running k-th best, so the list is cut back
    again and again."""
    poses = wi.random_poses(33, 20001)
    cur, P = poses[0], poses[1:]
    d = o.retrieval_distances(cur, P)
    _check(kv, P[np.argsort(-d)].copy(), cur, 16)


@pytest.mark.parametrize("log2n,k", [(20, 16), (20, 64), (24, 16)])
def test_scan_full_size(kv, log2n, k):
    n = 1 << log2n
    poses = wi.random_poses(100 + log2n, n + 1)
    _check(kv, poses[1:], poses[0], k)


def test_scan_when_nothing_can_be_ruled_out(kv):
    """Pure translation (every stored rotation equals the current one): no candidate can be ruled out before the
    maxima are known, the survivor list overflows (more than 2^20 entries) and the call falls back to walking every pose
    a second time.  The answer must not change."""
    n = (1 << 20) + 300001
    poses = wi.random_poses(55, n + 1)
    poses[:, 4:8] = poses[0, 4:8]
    _check(kv, poses[1:], poses[0], 16)
    assert kv.poll_status() == (0, 0)


def test_scan_on_a_camera_loop(kv):
    """Poses along a jittered loop (neighbouring candidates are near-duplicates of each other), 300,000 of them."""
    poses = wi.loop_poses(8, 300001)
    _check(kv, poses[:-1].copy(), poses[-1], 8)
    valid = wi.hash64(6, wi.STREAM_MISC, np.arange(300000)) % np.uint64(4) != 0
    _check(kv, poses[:-1].copy(), poses[-1], 8, valid=valid)


def test_scan_skips_non_finite_poses_and_reports_them(kv):
    from paper_2605_22718_b200 import WK_DEV_NONFINITE, WK_ERR_NONFINITE
    n = 70000
    poses = wi.random_poses(77, n + 1)
    P = poses[1:].copy()
    bad = [5, 40000, 69999]
    P[5, 0] = np.nan
    P[40000, 6] = np.inf
    P[69999, 2] = -np.inf
    ok = np.ones(n, bool)
    ok[bad] = False
    Pd = torch.from_numpy(P).cuda()
    ids = torch.empty(8, dtype=torch.int32, device="cuda")
    dist = torch.empty(8, dtype=torch.float64, device="cuda")
    kv.retrieve_scan(Pd, poses[0], 8, ids_out=ids, dist_out=dist)
    st, flags = kv.poll_status()
    assert st == WK_ERR_NONFINITE and flags & WK_DEV_NONFINITE
    cand = np.nonzero(ok)[0]
    ref_ids, ref_d, margin = o.retrieve(poses[0], P[cand], cand, 8)
    assert margin > 1e-9
    np.testing.assert_array_equal(ids.cpu().numpy(), ref_ids)
    np.testing.assert_allclose(dist.cpu().numpy(), ref_d, rtol=0, atol=1e-12)


def test_scan_many_equal_distances(kv):
    """200,000 copies of one pose (all distances 0) and 200,000 copies of another: every block's list is full of ties,
    far more entries tie at the cut than the merging block gathers at once, and the answer is still the lowest indices."""
    poses = wi.random_poses(12, 3)
    P = np.concatenate([np.repeat(poses[1][None], 200000, axis=0), np.repeat(poses[2][None], 200000, axis=0)])
    got = _check(kv, P, poses[0], 16, need_margin=False)
    d = o.retrieval_distances(poses[0], poses[1:3])
    first = 0 if d[0] <= d[1] else 200000
    assert got.tolist() == list(range(first, first + 16))
    same = np.repeat(poses[0][None], 300000, axis=0)
    assert _check(kv, same, poses[0], 64, need_margin=False).tolist() == list(range(64))
