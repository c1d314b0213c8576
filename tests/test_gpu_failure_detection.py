"""Failure detection on the GPU, in forms that fault, trap or hang nothing.

Every anomaly here is made on the host (a NaN written into an input, an index out of range, a barrier that nothing
completes inside a test-only kernel); the device reports it through a status word and returns normally, and the
context keeps working afterwards.
"""
import ctypes as C
import os

import numpy as np
import pytest
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def make_kv(**kw):
    from paper_2605_22718_b200 import WorldKV
    return WorldKV(**kw)


def test_bounded_wait_gives_up_and_reports_timeout():
    """The product's mbarrier wait (ptx_sm100.cuh), built with a cap of 4,096 tries, on a barrier nobody completes:
    the kernel comes back within milliseconds with WK_DEV_TIMEOUT set; on a barrier that is completed it sets nothing.
    The status word used is a context's own, so wk_poll_status maps the bit to WK_ERR_TIMEOUT and clears it."""
    from paper_2605_22718_b200 import WK_DEV_TIMEOUT, WK_ERR_TIMEOUT
    from paper_2605_22718_b200.build import LIB_WAIT_PROBE, build_all
    if not os.path.exists(LIB_WAIT_PROBE):
        build_all()
    lib = C.CDLL(LIB_WAIT_PROBE)
    lib.wk_test_wait_probe.restype = C.c_int
    lib.wk_test_wait_probe.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
    kv = make_kv(n_layers=1, n_heads=1, tokens_per_frame=8, n_keep=4, pool_slots=2, max_k=2)
    # the status word is the first word of the pool buffer's last 256 bytes
    status_ptr = kv.pool.data_ptr() + kv.pool.numel() - 256
    tries = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    assert lib.wk_test_wait_probe(status_ptr, 1, tries.data_ptr(), stream) == 0
    assert kv.poll_status() == (0, 0) and int(tries.item()) == 0
    t0.record()
    assert lib.wk_test_wait_probe(status_ptr, 0, tries.data_ptr(), stream) == 0
    t1.record()
    assert kv.poll_status() == (WK_ERR_TIMEOUT, WK_DEV_TIMEOUT)
    assert int(tries.item()) == 4096
    assert t0.elapsed_time(t1) < 2000.0            # the wait ran out by itself, in well under two seconds
    assert kv.poll_status() == (0, 0)              # the bit was cleared and the context is still usable
    ids, n = kv.retrieve([0, 0, 0, 0, 1, 0, 0, 0], 1)
    assert n == 0 and kv.poll_status() == (0, 0)


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), float("-inf")])
def test_non_finite_key_sets_the_status_bit(bad):
    from paper_2605_22718_b200 import WK_DEV_NONFINITE, WK_ERR_NONFINITE
    T, H = 48, 2
    D = H * 128
    kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=T // 2, pool_slots=1, max_k=1)
    K = wi.key_chunk_bf16(3, 0, 2, T, D, 0.1)
    Kd = wd.to_device_bf16(K)[None].clone()
    Kd[0, T + 7, 5] = bad                           # one non-anchor key is poisoned, on the host side of the call
    keep = kv.compress_chunk(Kd)                    # the call itself still returns a full-size index list
    st, flags = kv.poll_status()
    assert st == WK_ERR_NONFINITE and flags & WK_DEV_NONFINITE
    k = keep.cpu().numpy()[0]
    assert k.shape == (T + T // 2,) and (k[:T] == np.arange(T)).all()
    # the context is not poisoned: the clean chunk gives the oracle's keep-set afterwards
    keep = kv.compress_chunk(wd.to_device_bf16(K)[None]).cpu().numpy()[0]
    np.testing.assert_array_equal(keep, o.compress_chunk(K, T, T // 2)[0])
    assert kv.poll_status() == (0, 0)


def test_non_finite_anchor_key_sets_the_status_bit():
    from paper_2605_22718_b200 import WK_DEV_NONFINITE, WK_ERR_NONFINITE
    T, H = 48, 1
    kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=T // 2, pool_slots=1, max_k=1)
    Kd = wd.to_device_bf16(wi.key_chunk_bf16(3, 0, 2, T, H * 128, 0.1))[None].clone()
    Kd[0, 3, 100] = float("nan")                    # an anchor key: the mean unit anchor and with it every score is NaN
    kv.compress_chunk(Kd)
    st, flags = kv.poll_status()
    assert st == WK_ERR_NONFINITE and flags & WK_DEV_NONFINITE


def test_out_of_range_keep_index_is_not_dereferenced():
    from paper_2605_22718_b200 import WK_DEV_BAD_SLOT, WK_ERR_BAD_SLOT
    T, H = 16, 1
    C_rows = T + 8
    kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=8, pool_slots=2, max_k=2)
    K = wd.to_device_bf16(wi.key_chunk_bf16(4, 0, 0, T, 128, 0.1))[None]
    V = wd.to_device_bf16(wi.value_chunk_bf16(4, 0, 0, T, 128))[None]
    keep = kv.compress_chunk(K).clone()
    keep[0, 5] = 3 * T                              # one past the chunk
    keep[0, 9] = -4
    slot = kv.pool_append(0, 1, K, V, keep, [0, 0, 0, 0, 1, 0, 0, 0], chunk_tag=1)
    assert kv.poll_status() == (WK_ERR_BAD_SLOT, WK_DEV_BAD_SLOT)
    Kpool = kv.pool[:2 * C_rows * 128 * 2].view(torch.bfloat16).view(2, C_rows, 128)
    rows = wd.to_host_bits(Kpool[slot])
    src = wd.to_host_bits(K[0])
    good = [r for r in range(C_rows) if r not in (5, 9)]
    np.testing.assert_array_equal(rows[good], src[keep.cpu().numpy()[0][good]])
    assert (rows[[5, 9]] == 0).all()                # nothing was written for the bad entries (the pool started zeroed)


def test_non_finite_pose_is_not_a_candidate():
    from paper_2605_22718_b200 import WK_DEV_NONFINITE, WK_ERR_NONFINITE
    T = 8
    kv = make_kv(n_layers=1, n_heads=1, tokens_per_frame=T, n_keep=4, pool_slots=12, max_k=12)
    poses = wi.random_poses(9, 13).astype(np.float32)
    poses[4, 1] = np.nan
    poses[7, 5] = np.inf
    K = wd.to_device_bf16(wi.key_chunk_bf16(4, 0, 0, T, 128, 0.1))[None]
    V = wd.to_device_bf16(wi.value_chunk_bf16(4, 0, 0, T, 128))[None]
    keep = kv.compress_chunk(K)
    for c in range(12):
        assert kv.pool_append(0, 1, K, V, keep, poses[c], chunk_tag=c) == c
    dist = torch.empty(12, dtype=torch.float64, device="cuda")
    ids, n = kv.retrieve(poses[12], 12, dist_out=dist)
    st, flags = kv.poll_status()
    assert st == WK_ERR_NONFINITE and flags & WK_DEV_NONFINITE
    finite = [s for s in range(12) if s not in (4, 7)]
    ref_ids, ref_d, _ = o.retrieve(poses[12], poses[finite], finite, 12)
    got = ids.cpu().numpy()
    np.testing.assert_array_equal(got[:10], ref_ids)
    assert (got[10:] == -1).all()                   # the host-side count (12) includes the two; their places stay empty
    np.testing.assert_allclose(dist.cpu().numpy()[:10], ref_d, rtol=1e-12, atol=1e-14)
