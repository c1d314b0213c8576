"""Seeded synthetic inputs for the WorldKV hot path.

This package only *draws inputs*: counter-based random numbers, the key-redundancy
stream, camera trajectories and the five benchmark workload descriptions.  It holds
none of the method's arithmetic (no cosine scores, no pose distances, no softmax) and
is the one module that both the CPU oracle's tests and the CUDA path's tests consume.
"""
from .gen import (  # noqa: F401
    STREAM_K_BASE, STREAM_K_NOISE, STREAM_K_REDRAW, STREAM_Q, STREAM_V, STREAM_MISC,
    hash64, normal_f32, f32_to_bf16_bits, bf16_bits_to_f32, bf16_bits_to_f64,
    normal_bf16, key_frames_bf16, key_chunk_bf16, value_chunk_bf16, query_bf16,
    redraw_mask,
)
from .poses import random_poses, loop_poses, action_rollout_poses  # noqa: F401
from .workloads import WORKLOADS, Workload  # noqa: F401
