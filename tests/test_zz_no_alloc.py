"""wk_retrieve_noalloc -- the entry point for callers that cannot call cudaMalloc (code running under stream capture,
services with a frozen memory pool, plug-ins that must stay out of the host's allocator).  It keeps its scratch in an
array compiled into the library, so this file checks that it returns exactly what wk_retrieve returns, twice in a row
(the shared scratch keeps the previous call's contents), through the C ABI.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import wkinputs as wi

pytestmark = pytest.mark.gpu


def test_noalloc_retrieval_matches_wk_retrieve_twice_in_a_row():
    from paper_2605_22718_b200 import WorldKV, WkError, retrieve_noalloc, WK_ERR_SHAPE
    n_slots, max_k, T, n_keep = 40, 8, 8, 4
    kv = WorldKV(n_layers=1, n_heads=1, tokens_per_frame=T, n_keep=n_keep, pool_slots=n_slots, max_k=max_k)
    poses = wi.random_poses(21, n_slots + 2)
    K = torch.zeros((1, 3 * T, 128), dtype=torch.bfloat16, device="cuda")
    keep = torch.arange(T + n_keep, dtype=torch.int32, device="cuda")[None].contiguous()
    for c in range(n_slots - 5):                                 # leave some slots empty
        kv.pool_append(0, 1, K, K, keep, poses[c], chunk_tag=c)
    kv.pool_evict(3)
    kv.pool_evict(17)
    # the same slot table, as plain caller-owned tensors
    valid_host = np.zeros(n_slots, dtype=np.int32)
    valid_host[:n_slots - 5] = 1
    valid_host[[3, 17]] = 0
    poses_dev = torch.from_numpy(poses[:n_slots].copy()).cuda()
    valid_dev = torch.from_numpy(valid_host).cuda()
    slots_a = torch.empty(max_k, dtype=torch.int32, device="cuda")
    dist_a = torch.empty(max_k, dtype=torch.float64, device="cuda")
    slots_b = torch.empty(max_k, dtype=torch.int32, device="cuda")
    dist_b = torch.empty(max_k, dtype=torch.float64, device="cuda")
    for cur, k in ((poses[n_slots], 8), (poses[n_slots + 1], 3)):     # two calls in a row on the shared scratch
        _, n = kv.retrieve(cur, k, slots_out=slots_a, dist_out=dist_a)
        retrieve_noalloc(poses_dev, valid_dev, cur, k, max_k, slots_b, dist_b)
        torch.cuda.synchronize()
        assert n == k
        np.testing.assert_array_equal(slots_b.cpu().numpy(), slots_a.cpu().numpy())
        np.testing.assert_allclose(dist_b.cpu().numpy(), dist_a.cpu().numpy(), rtol=0, atol=1e-12)
        assert (valid_host[slots_b.cpu().numpy()[:k]] == 1).all()
    # beyond the built-in scratch: rejected before any launch
    big = torch.zeros((4097, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(WkError) as e:
        retrieve_noalloc(big, torch.zeros(4097, dtype=torch.int32, device="cuda"), poses[0], 1, max_k, slots_b)
    assert e.value.status == WK_ERR_SHAPE


def test_noalloc_retrieval_at_the_largest_slot_table_against_the_oracle():
    """n_slots = 4096 is the last size the built-in array holds (its final element is in use).  A third of the slots are
    marked empty; ids and distances are compared with the oracle, a second warmed call must leave the device's free
    memory where it was (nothing was allocated on the way), and bad arguments are turned away before any launch."""
    from paper_2605_22718_b200 import WkError, retrieve_noalloc, WK_ERR_ARG
    from oracle import worldkv_oracle as o
    n_slots, max_k = 4096, 16
    poses = wi.random_poses(33, n_slots + 1)
    valid_host = np.ones(n_slots, dtype=np.int32)
    valid_host[::3] = 0
    valid_host[n_slots - 1] = 1                                     # the last slot is a candidate
    poses_dev = torch.from_numpy(poses[:n_slots].astype(np.float32)).cuda()
    valid_dev = torch.from_numpy(valid_host).cuda()
    slots = torch.empty(max_k, dtype=torch.int32, device="cuda")
    dist = torch.empty(max_k, dtype=torch.float64, device="cuda")
    cur = poses[n_slots]
    cand = np.nonzero(valid_host)[0]
    ref_ids, ref_d, margin = o.retrieve(cur, poses[cand], cand.tolist(), max_k)
    assert margin > 1e-9
    retrieve_noalloc(poses_dev, valid_dev, cur, max_k, max_k, slots, dist)      # warms the symbol-address set-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    retrieve_noalloc(poses_dev, valid_dev, cur, max_k, max_k, slots, dist)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    np.testing.assert_array_equal(slots.cpu().numpy(), ref_ids)
    np.testing.assert_allclose(dist.cpu().numpy(), ref_d, rtol=1e-12, atol=1e-14)
    # the current pose equals the last slot's: the last element of the built-in array takes part in the ranking
    far = poses[n_slots - 1].copy()
    retrieve_noalloc(poses_dev, valid_dev, far, 1, max_k, slots, dist)
    torch.cuda.synchronize()
    assert int(slots[0]) == n_slots - 1 and float(dist[0]) == 0.0 and (slots.cpu().numpy()[1:] == -1).all()
    for args in ((poses_dev, valid_dev, cur, max_k + 1, max_k, slots),      # k > max_k
                 (poses_dev, valid_dev, cur, 1, 0, slots),                  # max_k < 1
                 (poses_dev, valid_dev, cur, -1, max_k, slots)):            # k < 0
        with pytest.raises(WkError) as e:
            retrieve_noalloc(*args)
        assert e.value.status == WK_ERR_ARG
    from paper_2605_22718_b200 import binding
    lib = binding.load_library()
    import ctypes as C
    pose_arr = (C.c_float * 8)(*[float(x) for x in cur])
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.wk_retrieve_noalloc(None, valid_dev.data_ptr(), 4, pose_arr, 1, max_k, slots.data_ptr(), None, stream) == WK_ERR_ARG
    assert lib.wk_retrieve_noalloc(poses_dev.data_ptr(), valid_dev.data_ptr(), 4, pose_arr, 1, max_k, None, None, stream) == WK_ERR_ARG
