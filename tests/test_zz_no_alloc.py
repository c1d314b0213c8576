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
