"""Seeded camera trajectories (host only; a few KB of fp32).

A pose record is 8 fp32 numbers ``[tx, ty, tz, 0, qw, qx, qy, qz]`` with a unit quaternion.
Three recipes, matching the benchmark workloads:

* ``random_poses``: t ~ N(0, I3), q = a normalised N(0, I4) draw (the tiny case).
* ``loop_poses``: a camera walking once around a circle with its heading along the
  tangent, plus seeded jitter, so that the last poses revisit the first ones (the paper's
  loop-closure setting).  The jitter removes the exact ties a perfect circle has.
* ``action_rollout_poses``: keyboard-style actions (W/A/S/D steps rotated by the current
  yaw, yaw/pitch increments, stop) accumulated into a pseudo-pose (Section 5.1), with a
  scripted return to an earlier pose every ``revisit_every`` chunks.
"""
from __future__ import annotations

import numpy as np


def _quat_yaw_pitch(yaw: np.ndarray, pitch: np.ndarray) -> np.ndarray:
    """Unit quaternion (w, x, y, z) of a rotation by ``yaw`` about z followed by ``pitch`` about y."""
    cy, sy = np.cos(yaw / 2), np.sin(yaw / 2)
    cp, sp = np.cos(pitch / 2), np.sin(pitch / 2)
    # q = q_z(yaw) * q_y(pitch)
    return np.stack([cy * cp, -sy * sp, cy * sp, sy * cp], axis=-1)


def _pack(t: np.ndarray, q: np.ndarray) -> np.ndarray:
    q = q / np.linalg.norm(q, axis=-1, keepdims=True)
    out = np.zeros((t.shape[0], 8), dtype=np.float32)
    out[:, 0:3] = t
    out[:, 4:8] = q
    # re-normalise after the fp32 rounding so stored quaternions are as close to unit as fp32 allows
    qq = out[:, 4:8].astype(np.float64)
    out[:, 4:8] = (qq / np.linalg.norm(qq, axis=-1, keepdims=True)).astype(np.float32)
    return out


def random_poses(seed: int, n: int) -> np.ndarray:
    rng = np.random.default_rng([seed, 101])
    return _pack(rng.standard_normal((n, 3)), rng.standard_normal((n, 4)))


def loop_poses(seed: int, n: int, radius: float = 10.0, jitter: float = 1e-2) -> np.ndarray:
    """n poses on a jittered circle; pose n-1 is one step short of pose 0 again."""
    rng = np.random.default_rng([seed, 202])
    phi = 2 * np.pi * np.arange(n) / n
    t = np.stack([radius * np.cos(phi), radius * np.sin(phi), np.zeros(n)], axis=-1)
    t = t + jitter * rng.standard_normal((n, 3))
    yaw = phi + np.pi / 2 + jitter * rng.standard_normal(n)
    pitch = jitter * rng.standard_normal(n)
    return _pack(t, _quat_yaw_pitch(yaw, pitch))


def action_rollout_poses(seed: int, n: int, revisit_every: int = 20, step: float = 0.5,
                         turn: float = 0.2, jitter: float = 1e-2) -> np.ndarray:
    """Pseudo-poses of an n-chunk keyboard rollout with periodic scripted revisits."""
    rng = np.random.default_rng([seed, 303])
    pos = np.zeros(3)
    yaw = 0.0
    pitch = 0.0
    ts, yaws, pitches = [], [], []
    for i in range(n):
        if i > 0 and i % revisit_every == 0:
            j = int(rng.integers(0, max(1, i - revisit_every // 2)))  # jump back to an earlier pose
            pos = ts[j] + jitter * rng.standard_normal(3)
            yaw = yaws[j] + jitter * rng.standard_normal()
            pitch = pitches[j] + jitter * rng.standard_normal()
        else:
            a = int(rng.integers(0, 9))  # W A S D yaw+ yaw- pitch+ pitch- stop
            fwd = np.array([np.cos(yaw), np.sin(yaw), 0.0])
            left = np.array([-np.sin(yaw), np.cos(yaw), 0.0])
            if a == 0:
                pos = pos + step * fwd
            elif a == 1:
                pos = pos + step * left
            elif a == 2:
                pos = pos - step * fwd
            elif a == 3:
                pos = pos - step * left
            elif a == 4:
                yaw += turn
            elif a == 5:
                yaw -= turn
            elif a == 6:
                pitch = min(pitch + turn, 1.2)
            elif a == 7:
                pitch = max(pitch - turn, -1.2)
            pos = pos + 1e-3 * jitter * rng.standard_normal(3)  # no two chunks share a pose exactly
        ts.append(pos.copy())
        yaws.append(yaw)
        pitches.append(pitch)
    return _pack(np.array(ts), _quat_yaw_pitch(np.array(yaws), np.array(pitches)))
