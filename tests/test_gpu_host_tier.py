"""Host-memory tier (Section 7): a stored chunk copied to host memory and brought back attends exactly as before."""
import numpy as np
import pytest
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o
from wk_testlib import Scenario, assert_attention_close

pytestmark = pytest.mark.gpu


def test_store_evict_load_roundtrip():
    from paper_2605_22718_b200 import WorldKV, WkError, WK_ERR_BAD_SLOT, WK_ERR_POOL_FULL
    L, T, H, n_keep, S = 3, 40, 2, 23, 5
    C = T + n_keep
    kv = WorldKV(n_layers=L, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=S, max_k=4, max_batch=L, max_lq=200,
                 max_splits=4, max_dense_segments=2)
    sc = Scenario(kv, 17, 0.1, L, T, H, n_keep, S)
    poses = wi.random_poses(17, 8)
    for c in range(4):
        sc.append_chunk(c, poses[c])
    nbytes = kv.host_chunk_bytes()
    assert nbytes == 2 * L * C * H * 128 * 2
    img = [torch.empty(nbytes // 2, dtype=torch.int16).pin_memory() for _ in range(2)]
    kv.pool_store_host(1, img[0])
    kv.pool_store_host(2, img[1])
    torch.cuda.synchronize()
    # the host image is K then V, each [L][C][D], holding exactly the kept rows the oracle's pool model holds
    for i, slot in enumerate((1, 2)):
        bits = img[i].numpy().view(np.uint16).reshape(2, L, C, H, 128)
        for l in range(L):
            np.testing.assert_array_equal(bits[0, l], sc.pool.K[(l, slot)])
            np.testing.assert_array_equal(bits[1, l], sc.pool.V[(l, slot)])
    layer, lq = 1, 150
    Qb = wi.query_bf16(17, layer, 0, 0, lq, H * 128)
    Q = wd.to_device_bf16(Qb).view(lq, H, 128)
    seg_d, seg_h = sc.dense_segment(layer, 6, 90)
    before = torch.tensor([2, 1], dtype=torch.int32, device="cuda")
    O_before = kv.memory_attention(layer, Q, [seg_d], before, 2).clone()
    O_ref, _ = o.memory_attention(Qb.reshape(lq, H, 128), [seg_h], sc.pool, layer, [2, 1])
    assert_attention_close(O_before, O_ref, "before the round trip")
    with pytest.raises(WkError) as e:
        kv.pool_store_host(4, img[0])            # slot 4 holds nothing
    assert e.value.status == WK_ERR_BAD_SLOT
    # free slots 0, 1, 2; chunk 2 comes back first (layers out of order, in two calls), so it lands in slot 0
    for s in (0, 1, 2):
        kv.pool_evict(s)
    s2 = kv.pool_load_host(2, 1, img[1], poses[2], chunk_tag=2)
    assert s2 == 0 and kv.pool_count() == 1                      # not visible before every layer is there
    with pytest.raises(WkError) as e:
        kv.pool_load_host(2, 1, img[1], poses[2], slot=s2)       # the same layer twice
    assert e.value.status == WK_ERR_BAD_SLOT
    assert kv.pool_load_host(0, 2, img[1], poses[2], slot=s2) == 0
    s1 = kv.pool_load_host(0, L, img[0], poses[1], chunk_tag=1)
    assert s1 == 1 and kv.pool_count() == 3 and kv.pool_tag(0) == 2 and kv.pool_tag(1) == 1
    after = torch.tensor([s2, s1], dtype=torch.int32, device="cuda")
    O_after = kv.memory_attention(layer, Q, [seg_d], after, 2)
    assert kv.poll_status() == (0, 0)
    assert torch.equal(O_before, O_after)                        # same bytes in, same kernel: same bits out
    # the reloaded chunks are found by their poses
    slots, n = kv.retrieve(poses[2], 1)
    assert n == 1 and int(slots[0]) == s2
    # a full pool refuses the load
    assert kv.pool_load_host(0, L, img[0], poses[5]) == 2
    assert kv.pool_load_host(0, L, img[0], poses[6]) == 4
    with pytest.raises(WkError) as e:
        kv.pool_load_host(0, L, img[0], poses[7])
    assert e.value.status == WK_ERR_POOL_FULL
