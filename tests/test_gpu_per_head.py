"""Per-head keep-sets (Eq. 5 read with one head's key): compression, append and attention against the oracle."""
import numpy as np
import pytest
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o
from wk_testlib import Scenario, assert_attention_close

pytestmark = pytest.mark.gpu


def _kv(**kw):
    from paper_2605_22718_b200 import WorldKV, SCORE_PER_HEAD
    return WorldKV(score_mode=SCORE_PER_HEAD, **kw)


@pytest.mark.parametrize("T,H,n_keep,batch,sigma", [
    (37, 3, 18, 3, 0.1),          # ragged everything
    (880, 2, 440, 4, 0.1),        # cfg0 shape
    (256, 12, 128, 2, 0.1),       # Matrix-Game head count
    (880, 12, 440, 3, 0.1),       # the benchmark's chunk shape
    (1560, 40, 780, 1, 0.05),     # LingBot shape: 40 heads
    (100, 5, 0, 2, 0.1),          # keep nothing
    (100, 5, 200, 2, 0.1),        # keep everything
    (64, 2, 1, 2, 0.05),
])
def test_per_head_compress_matches_oracle(T, H, n_keep, batch, sigma):
    D = H * 128
    kv = _kv(n_layers=batch, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=2, max_k=1, max_batch=batch)
    Kb = [wi.key_chunk_bf16(31, l, 7, T, D, sigma) for l in range(batch)]
    Kd = wd.to_device_bf16(np.stack(Kb))
    scores = torch.empty((batch, H, 2 * T), dtype=torch.float32, device="cuda")
    keep = kv.compress_chunk(Kd, scores_out=scores if 0 < n_keep < 2 * T else None)
    assert keep.shape == (batch, H, T + n_keep)
    assert kv.poll_status() == (0, 0)
    for l in range(batch):
        idx, sc, margin = o.compress_chunk_per_head(Kb[l], T, n_keep, H)
        if 0 < n_keep < 2 * T:
            assert margin > 1e-11, margin
            np.testing.assert_allclose(scores[l].cpu().numpy(), sc, atol=2e-6)
        np.testing.assert_array_equal(keep[l].cpu().numpy(), idx)
    # heads do differ: the keep-sets of two heads of the same chunk are not the same list
    if H > 1 and 0 < n_keep < 2 * T and T >= 64:
        k0 = keep[0].cpu().numpy()
        assert any(not np.array_equal(k0[0], k0[h]) for h in range(1, H))


def test_per_head_pool_and_attention():
    """Stored row c of head h is that head's own c-th kept token; attention over such slots against the oracle."""
    L, T, H, n_keep, S = 2, 96, 3, 40, 4
    kv = _kv(n_layers=L, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=S, max_k=4, max_batch=L, max_lq=200,
             max_splits=4, max_dense_segments=2)
    sc = Scenario(kv, 23, 0.1, L, T, H, n_keep, S, per_head=True)
    poses = wi.random_poses(23, 4)
    for c in range(3):
        sc.append_chunk(c, poses[c])          # checks the keep-sets and the slot
    assert min(sc.margins) > 1e-11
    # the pool holds exactly the oracle's rows
    img = torch.empty(kv.host_chunk_bytes() // 2, dtype=torch.int16).pin_memory()
    kv.pool_store_host(1, img)
    torch.cuda.synchronize()
    bits = img.numpy().view(np.uint16).reshape(2, L, T + n_keep, H, 128)
    for l in range(L):
        np.testing.assert_array_equal(bits[0, l], sc.pool.K[(l, 1)])
        np.testing.assert_array_equal(bits[1, l], sc.pool.V[(l, 1)])
    layer, lq = 1, 170
    Qb = wi.query_bf16(23, layer, 0, 0, lq, H * 128)
    Q = wd.to_device_bf16(Qb).view(lq, H, 128)
    seg_d, seg_h = sc.dense_segment(layer, 9, 100)
    slots = torch.tensor([2, 0, 1], dtype=torch.int32, device="cuda")
    O = kv.memory_attention(layer, Q, [seg_d], slots, 3)
    assert kv.poll_status() == (0, 0)
    O_ref, _ = o.memory_attention(Qb.reshape(lq, H, 128), [seg_h], sc.pool, layer, [2, 0, 1])
    assert_attention_close(O, O_ref, "per-head slots")
