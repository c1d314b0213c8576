"""Pins for the retrieval oracle (Eq. 4 with the pose distance of Section 5.1)."""
import math

import numpy as np
import pytest
from scipy.spatial.transform import Rotation

import wkinputs as wi
from oracle import worldkv_oracle as o


def pose(t=(0, 0, 0), q=(1, 0, 0, 0)):
    q = np.asarray(q, float)
    q = q / np.linalg.norm(q)
    return np.array([t[0], t[1], t[2], 0, q[0], q[1], q[2], q[3]], float)


def quat_axis(axis, phi):
    axis = np.asarray(axis, float) / np.linalg.norm(axis)
    return np.concatenate([[math.cos(phi / 2)], math.sin(phi / 2) * axis])


def test_identical_pose_is_distance_zero_and_rank_one():
    poses = wi.random_poses(1, 9).astype(float)
    d = o.retrieval_distances(poses[4], poses)
    assert d[4] == 0.0 and (np.delete(d, 4) > 0).all()
    ids, dist, _ = o.retrieve(poses[4], poses, list(range(9)), 3)
    assert ids[0] == 4 and dist[0] == 0.0


def test_translation_term_is_squared_l2_over_max():
    cur = pose()
    cand = np.stack([pose((1, 0, 0)), pose((0, 2, 0)), pose((0, 0, -3)), pose((0, 0, 0))])
    np.testing.assert_allclose(o.retrieval_distances(cur, cand), [1 / 9, 4 / 9, 1.0, 0.0], atol=1e-15)


def test_rotation_term_is_geodesic_angle_over_max():
    cur = pose()
    phis = [0.3, 1.2, math.pi, 4.0, 6.0]                     # beyond pi the short way round is 2 pi - phi
    cand = np.stack([pose(q=quat_axis((1, 2, -1), p)) for p in phis])
    ang = np.array([0.3, 1.2, math.pi, 2 * math.pi - 4.0, 2 * math.pi - 6.0])
    np.testing.assert_allclose(o.retrieval_distances(cur, cand), ang / math.pi, atol=1e-12)


def test_q_and_minus_q_are_the_same_rotation():
    cur = pose(q=quat_axis((0, 0, 1), 0.4))
    a = pose((1, 1, 1), quat_axis((0, 1, 0), 1.0))
    b = a.copy()
    b[4:8] *= -1
    far = pose((5, 5, 5), quat_axis((1, 0, 0), 2.0))
    d = o.retrieval_distances(cur, np.stack([a, b, far]))
    assert d[0] == pytest.approx(d[1], abs=1e-15)


def test_sum_of_the_two_normalised_terms():
    cur = pose()
    cand = np.stack([pose((2, 0, 0), quat_axis((0, 0, 1), 0.5)),
                     pose((1, 0, 0), quat_axis((0, 0, 1), 1.0)),
                     pose((0, 0, 0), quat_axis((0, 0, 1), 0.25))])
    np.testing.assert_allclose(o.retrieval_distances(cur, cand), [1 + 0.5, 0.25 + 1, 0 + 0.25], atol=1e-12)
    ids, dist, margin = o.retrieve(cur, cand, [3, 5, 9], 2)
    np.testing.assert_array_equal(ids, [9, 5])
    assert margin == pytest.approx(0.25)


def test_matches_scipy_relative_rotation_magnitude():
    """The geodesic term against an independent library: |log(R_cur^-1 R_i)| from scipy."""
    poses = wi.random_poses(7, 40).astype(float)
    cur = wi.random_poses(8, 1)[0].astype(float)
    to_scipy = lambda q: Rotation.from_quat(np.roll(q, -1, axis=-1))       # (w,x,y,z) -> (x,y,z,w)
    ang = (to_scipy(cur[4:8]).inv() * to_scipy(poses[:, 4:8])).magnitude()
    dt = ((poses[:, :3] - cur[:3]) ** 2).sum(1)
    np.testing.assert_allclose(o.retrieval_distances(cur, poses), dt / dt.max() + ang / ang.max(), atol=1e-7)


def test_ranking_invariant_to_rigid_motion_and_uniform_scale():
    poses = wi.random_poses(3, 30).astype(float)
    cur = wi.random_poses(4, 1)[0].astype(float)
    base, _, margin = o.retrieve(cur, poses, list(range(30)), 30)
    assert margin == float("inf")
    g = Rotation.from_rotvec([0.3, -1.0, 0.7])
    shift = np.array([3.0, -2.0, 5.0])

    def move(p):
        p = np.atleast_2d(p).copy()
        p[:, :3] = 2.5 * g.apply(p[:, :3]) + shift                          # rotate, scale, translate positions
        r = g * Rotation.from_quat(np.roll(p[:, 4:8], -1, axis=1))         # left-multiply orientations
        p[:, 4:8] = np.roll(r.as_quat(), 1, axis=1)
        return p

    moved, _, _ = o.retrieve(move(cur)[0], move(poses), list(range(30)), 30)
    np.testing.assert_array_equal(base, moved)


def test_exact_circle_neighbours_and_tie_break():
    """Jitter-free loop: the pose at angle 0 has neighbours at +-1 step, exactly tied; the lower
    slot wins the tie (R6)."""
    n = 16
    poses = wi.loop_poses(0, n, jitter=0.0).astype(np.float64)
    # build the exact circle in fp64 so that the two neighbours tie exactly
    phi = 2 * np.pi * np.arange(n) / n
    exact = np.zeros((n, 8))
    exact[:, 0], exact[:, 1] = np.cos(phi), np.sin(phi)
    exact[:, 4], exact[:, 7] = np.cos(phi / 2), np.sin(phi / 2)
    exact[n - 1, :] = exact[1, :] * [1, -1, 1, 1, 1, 1, 1, -1]           # mirror image of pose 1: same distances
    ids, dist, _ = o.retrieve(exact[0], exact, list(range(n)), 3)
    assert ids[0] == 0
    assert dist[1] == dist[2]
    np.testing.assert_array_equal(ids[1:], [1, n - 1])
    assert poses.shape == (n, 8)


def test_brute_force_sort_and_edge_cases():
    poses = wi.random_poses(11, 50).astype(float)
    slots = sorted(np.random.default_rng(0).choice(200, 50, replace=False).tolist())
    cur = wi.random_poses(12, 1)[0].astype(float)
    d = o.retrieval_distances(cur, poses)
    expect = [s for _, s in sorted(zip(d.tolist(), slots))]
    for k in (1, 4, 50, 80):                                              # k > M returns all M
        ids, dist, _ = o.retrieve(cur, poses, slots, k)
        np.testing.assert_array_equal(ids, expect[:min(k, 50)])
        assert (np.diff(dist) >= 0).all()
    ids, dist, margin = o.retrieve(cur, np.zeros((0, 8)), [], 4)          # empty pool
    assert len(ids) == 0 and margin == float("inf")
    ident = pose((1, 2, 3))                                               # exactly unit quaternion
    one = o.retrieval_distances(ident, ident[None])                       # single identical candidate: both maxima are 0 (R4)
    np.testing.assert_array_equal(one, [0.0])


def test_loop_workload_revisits_its_start():
    """cfg1-style camera loop: the current pose (last of 128) retrieves the chunks around the start."""
    poses = wi.loop_poses(1, 128).astype(float)
    ids, _, margin = o.retrieve(poses[127], poses[:125], list(range(125)), 4)
    assert set(ids.tolist()) == {0, 1, 124, 123} or set(ids.tolist()) == {0, 1, 124, 2}
    assert margin > 1e-9
