"""The seeded generators: determinism, random access, distribution, bf16 rounding."""
import numpy as np
import torch

import wkinputs as wi


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(0).standard_normal(200000).astype(np.float32) * 3
    x[:6] = [1.00390625, 1.01171875, 0.0, -0.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8]   # exact ties among them
    ours = wi.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(ours, ref)
    np.testing.assert_array_equal(wi.bf16_bits_to_f32(ours), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_normals_are_standard_and_random_access():
    z = wi.normal_f32(3, wi.STREAM_MISC, np.arange(400000))
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1) < 5e-3
    assert abs((z ** 3).mean()) < 2e-2 and abs((z ** 4).mean() - 2.85) < 5e-2     # Irwin-Hall n=8 kurtosis
    np.testing.assert_array_equal(z[1000:1010], wi.normal_f32(3, wi.STREAM_MISC, np.arange(1000, 1010)))
    assert not np.array_equal(z[:100], wi.normal_f32(4, wi.STREAM_MISC, np.arange(100)))
    assert abs(np.corrcoef(z[:-1], z[1:])[0, 1]) < 5e-3


def test_key_stream_structure():
    T, D, sigma = 64, 32, 0.1
    a = wi.key_chunk_bf16(5, 2, 3, T, D, sigma)
    b = wi.key_frames_bf16(5, 2, 9, 3, T, D, sigma)                 # chunk 3 = frames 9..11
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(a[T:2 * T], wi.key_frames_bf16(5, 2, 10, 1, T, D, sigma))
    prev = wi.bf16_bits_to_f64(wi.key_frames_bf16(5, 2, 8, 1, T, D, sigma))
    cur = wi.bf16_bits_to_f64(a[:T])
    redrawn = wi.redraw_mask(5, 2, [9], T)[0]
    diff = np.sqrt(((cur - prev) ** 2).mean(axis=1))
    assert (diff[~redrawn] < 0.25).all()                          # inherited positions differ by noise only
    assert (diff[redrawn] > 0.8).all()                            # redrawn positions are fresh draws
    assert 0.05 < redrawn.mean() < 0.55
    frac = wi.redraw_mask(5, 2, np.arange(1, 200), T).mean()
    assert abs(frac - 0.3) < 0.02
    assert wi.redraw_mask(5, 2, [0], T).all()
    other_layer = wi.key_chunk_bf16(5, 3, 3, T, D, sigma)
    assert not np.array_equal(a, other_layer)


def test_queries_values_poses():
    v = wi.value_chunk_bf16(1, 0, 2, 16, 8)
    assert v.shape == (48, 8) and v.dtype == np.uint16
    q = wi.query_bf16(1, 0, 1, 2, 48, 8)
    assert q.shape == (48, 8) and not np.array_equal(q, v)
    for poses in (wi.random_poses(0, 8), wi.loop_poses(1, 128), wi.action_rollout_poses(2, 370)):
        assert poses.dtype == np.float32 and poses.shape[1] == 8
        np.testing.assert_allclose(np.linalg.norm(poses[:, 4:8].astype(float), axis=1), 1.0, atol=1e-6)
        assert len(np.unique(poses, axis=0)) == len(poses)
    np.testing.assert_array_equal(wi.loop_poses(1, 128), wi.loop_poses(1, 128))
