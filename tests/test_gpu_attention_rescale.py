"""GPU parity of the memory attention (Section 4.2) on inputs whose running row maximum keeps rising.

The kernel keeps O un-normalised in tensor memory and rescales it only when a row's running maximum has risen by more
than 8 (log2 units) since the last rescale.  Unit-variance Q and K never raise the maximum that far after the first KV
tile, so these cases build the logits on purpose: queries scaled up, keys whose logits climb from tile to tile, one
dominating key planted deep in the last pool slot, a whole prefix of the KV set that underflows against a later tile,
and non-default softmax scales.  Every case asserts first -- on the oracle's own fp64 logits -- that the rise it plants
really exceeds the kernel's threshold, so the path cannot silently go unreached; then O and the log-sum-exp are compared
element-wise with the oracle, directly and through split KV ranges (partials + combine).
"""
import numpy as np
import pytest
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o
from wk_testlib import assert_attention_close

pytestmark = pytest.mark.gpu

LOG2E = 1.4426950408889634
RISE = 8.0            # the kernel's lazy-rescale threshold, log2 units
TILE = 128


def make_kv(**kw):
    from paper_2605_22718_b200 import WorldKV
    return WorldKV(**kw)


def bf16(x):
    return wi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def normals(seed, stream, shape):
    n = int(np.prod(shape))
    return wi.normal_f32(seed, wi.STREAM_MISC + stream, np.arange(n, dtype=np.uint64)).reshape(shape)


def late_rises(Q, parts, scale, rows, h):
    """For the sampled rows of head h: how many KV tiles after the first lift the running maximum (as a lazily updated
    maximum would track it) by more than RISE log2 units.  parts = K bit arrays [n, H, 128] in attended order; KV tiles
    restart at every part, as the kernel's do."""
    q = wi.bf16_bits_to_f64(Q[rows, h])
    counts = np.zeros(len(rows), dtype=np.int64)
    m_used = np.full(len(rows), -np.inf)
    first = True
    for K in parts:
        k = wi.bf16_bits_to_f64(K[:, h])
        for r0 in range(0, k.shape[0], TILE):
            mx = (scale * LOG2E * (q @ k[r0:r0 + TILE].T)).max(axis=1)
            up = mx > m_used + RISE
            if not first:
                counts += up
            m_used = np.where(up, mx, m_used)
            first = False
    return counts


class Scene:
    """A small context whose pool slots hold hand-built chunks: appended through wk_compress_chunk + wk_pool_append
    and mirrored in the oracle's pool model with the oracle's own keep-sets."""

    def __init__(self, H, T, n_keep, slots, lq, softmax_scale=0.0, max_splits=8):
        self.H, self.T, self.n_keep = H, T, n_keep
        self.kv = make_kv(n_layers=1, n_heads=H, tokens_per_frame=T, n_keep=n_keep, pool_slots=slots, max_k=slots,
                          max_batch=1, max_lq=lq, max_splits=max_splits, max_dense_segments=4,
                          softmax_scale=softmax_scale)
        self.pool = o.PoolModel(n_slots=slots, n_layers=1)
        self.scale = softmax_scale if softmax_scale > 0 else 1.0 / np.sqrt(128.0)

    def append(self, Kb, Vb, tag):
        """Kb, Vb: bf16 bits [3T, H*128]."""
        Kd, Vd = wd.to_device_bf16(Kb[None]), wd.to_device_bf16(Vb[None])
        keep = self.kv.compress_chunk(Kd)
        idx, _, margin = o.compress_chunk(Kb, self.T, self.n_keep)
        assert margin > 1e-11
        np.testing.assert_array_equal(keep.cpu().numpy()[0], idx)
        pose = [float(tag), 0, 0, 0, 1, 0, 0, 0]
        slot = self.kv.pool_append(0, 1, Kd, Vd, keep, pose, chunk_tag=tag)
        assert slot == self.pool.append([Kb.reshape(-1, self.H, 128)], [Vb.reshape(-1, self.H, 128)], [idx], pose, tag)
        return slot

    def check(self, Qb, segs, slot_list, splits_list, what, min_rises=1, min_share=0.5):
        """Qb [lq, H*128] bits; segs = [(K bits [n, H*128], V bits)].  Asserts the planted rise, then parity."""
        H, lq = self.H, Qb.shape[0]
        Q3 = Qb.reshape(lq, H, 128)
        segs_h = [(k.reshape(-1, H, 128), v.reshape(-1, H, 128)) for k, v in segs]
        parts = [k for k, _ in segs_h] + [self.pool.K[(0, s)] for s in slot_list]
        rows = np.arange(lq)
        for h in range(H):
            rises = late_rises(Q3, parts, self.scale, rows, h)
            assert (rises >= min_rises).mean() >= min_share, f"{what}: head {h} reaches the rescale on too few rows"
        O_ref, L_ref = o.memory_attention(Q3, segs_h, self.pool, 0, slot_list, scale=self.scale)
        Q = wd.to_device_bf16(Qb).view(lq, H, 128)
        segs_d = [(wd.to_device_bf16(k).view(-1, H, 128), wd.to_device_bf16(v).view(-1, H, 128)) for k, v in segs]
        slots = torch.tensor(list(slot_list) + [-1], dtype=torch.int32, device="cuda")
        for splits in splits_list:
            lse = torch.empty((H, lq), dtype=torch.float32, device="cuda")
            O = self.kv.memory_attention(0, Q, segs_d, slots, len(slot_list), lse_out=lse, kv_splits=splits)
            assert self.kv.poll_status() == (0, 0)
            assert_attention_close(O, O_ref, f"{what}, splits={splits}")
            np.testing.assert_allclose(lse.cpu().numpy(), L_ref, rtol=2e-6, atol=2e-3)


SPLITS = (1, 0, 3, -5)


def unit_chunk(seed, stream, T, H):
    D = H * 128
    return bf16(normals(seed, stream, (3 * T, D))), bf16(normals(seed, stream + 1, (3 * T, D)))


@pytest.mark.parametrize("factor", [4.0, 6.0, 8.0])
def test_scaled_queries(factor):
    """Unit-variance keys, queries `factor` times larger: the logits' spread grows with it, so later tiles overtake the
    first tile's maximum by more than the threshold on most rows."""
    H, T, lq = 2, 64, 300
    sc = Scene(H, T, 32, 3, lq)
    for c in range(3):
        sc.append(*unit_chunk(21, 10 * c, T, H), tag=c)
    Qb = bf16(factor * normals(21, 100, (lq, H * 128)))
    segs = [(bf16(normals(21, 200, (1500, H * 128))), bf16(normals(21, 201, (1500, H * 128))))]
    sc.check(Qb, segs, [2, 0, 1], SPLITS, f"Q x {factor}", min_share={4.0: 0.05, 6.0: 0.3, 8.0: 0.5}[factor])


def test_per_row_query_factor():
    """Every query row has its own scale in [1, 8]: rows of one tile rescale at different tiles (alpha = 1 for the rows
    that do not, in the same warp-wide pass)."""
    H, T, lq = 1, 64, 257
    sc = Scene(H, T, 32, 2, lq)
    sc.append(*unit_chunk(22, 0, T, H), tag=0)
    f = 1.0 + 7.0 * (np.arange(lq) % 16) / 15.0
    Qb = bf16(f[:, None] * normals(22, 100, (lq, 128)))
    segs = [(bf16(normals(22, 200, (2100, 128))), bf16(normals(22, 201, (2100, 128))))]
    sc.check(Qb, segs, [0], SPLITS, "per-row factor", min_share=0.2)


def climbing_keys(seed, stream, n, D, step, start=0.0):
    """Keys with a common direction u (all ones) whose weight grows by `step` per 128-row tile: against a query with a
    positive component along u the logits climb tile by tile."""
    a = start + step * (np.arange(n) // TILE)
    return bf16(normals(seed, stream, (n, D)) + a[:, None] * np.ones((1, D), dtype=np.float32)), a


def test_logits_climb_tile_by_tile():
    """Every KV tile beats the one before by about 16 log2 units: the rescale fires on every tile of every row, in the
    dense segments and on through the pool slots."""
    H, T, lq = 2, 64, 200
    D = H * 128
    sc = Scene(H, T, 2 * T, 2, lq)            # n_keep = 2T: chunks are stored whole, so the planted order survives
    Qb = bf16(normals(23, 100, (lq, D)) + 1.0)                      # component 1 along u in every head
    K1, a1 = climbing_keys(23, 1, 900, D, 1.0)
    K2, a2 = climbing_keys(23, 2, 300, D, 1.0, start=a1[-1] + 1.0)
    V1, V2 = bf16(normals(23, 3, (900, D))), bf16(normals(23, 4, (300, D)))
    top = a2[-1] + 1.0
    for c in range(2):
        Kc, ac = climbing_keys(23, 10 + c, 3 * T, D, 1.0, start=top)
        top = ac[-1] + 1.0
        sc.append(Kc, bf16(normals(23, 20 + c, (3 * T, D))), tag=c)
    n_tiles = 8 + 3 + 2 * 2
    sc.check(Qb, [(K1, V1), (K2, V2)], [0, 1], SPLITS, "climbing logits", min_rises=n_tiles - 3, min_share=0.95)


def test_one_late_key_dominates():
    """Thousands of ordinary keys, then one key in the last tile of the last pool slot whose logit exceeds everything
    before it by far more than the threshold: O collapses onto that key's value."""
    H, T, lq = 2, 64, 384
    D = H * 128
    sc = Scene(H, T, 2 * T, 3, lq)
    Qb = bf16(normals(24, 100, (lq, D)) + 1.0)
    segs = [(bf16(normals(24, 1, (4000, D))), bf16(normals(24, 2, (4000, D))))]
    for c in range(3):
        Kc = normals(24, 10 + c, (3 * T, D))
        if c == 2:
            Kc[3 * T - 7] += 4.0                                     # ~ +45 nats along u for every row
        sc.append(bf16(Kc), bf16(normals(24, 20 + c, (3 * T, D))), tag=c)
    sc.check(Qb, segs, [0, 1, 2], SPLITS + (4,), "planted late key", min_share=0.99)
    # the planted key carries (almost) all of the mass: the reference output is that key's value row
    O_ref, _ = o.memory_attention(Qb.reshape(lq, H, 128), [], sc.pool, 0, [2])
    v = wi.bf16_bits_to_f64(sc.pool.V[(0, 2)][3 * T - 7])
    assert np.abs(O_ref - v[None]).max() < 1e-6


def test_prefix_underflows_against_a_later_tile():
    """The first tiles sit more than 100 log2 units below a later one: the factor applied to O and to the running sum
    underflows to zero, and what was accumulated before must vanish without leaving NaN or Inf behind."""
    H, T, lq = 1, 64, 130
    D = 128
    sc = Scene(H, T, 2 * T, 1, lq)
    Qb = bf16(normals(25, 100, (lq, D)) + 1.0)
    low = bf16(normals(25, 1, (700, D)) - 6.0)                       # ~ -68 nats
    high = bf16(normals(25, 2, (300, D)) + 6.0)                      # ~ +68 nats: 195 log2 units above
    Vl, Vh = bf16(normals(25, 3, (700, D))), bf16(normals(25, 4, (300, D)))
    sc.append(bf16(normals(25, 10, (3 * T, D)) + 6.0), bf16(normals(25, 11, (3 * T, D))), tag=0)
    q = wi.bf16_bits_to_f64(Qb)
    gap = (sc.scale * LOG2E * (q @ wi.bf16_bits_to_f64(high).T)).max(axis=1) - \
          (sc.scale * LOG2E * (q @ wi.bf16_bits_to_f64(low).T)).max(axis=1)
    assert gap.min() > 100 * LOG2E
    sc.check(Qb, [(low, Vl), (high, Vh)], [0], SPLITS, "underflowing prefix", min_share=0.99)


@pytest.mark.parametrize("scale", [0.02, 0.25])
def test_softmax_scale_from_the_config(scale):
    """wk_config.softmax_scale other than the 1/sqrt(128) default: 0.02 flattens the softmax, 0.25 sharpens it (and
    reaches the rescale on its own with climbing keys)."""
    H, T, lq = 2, 64, 260
    D = H * 128
    sc = Scene(H, T, 32, 2, lq, softmax_scale=scale)
    assert abs(sc.scale - scale) < 1e-12
    for c in range(2):
        sc.append(*unit_chunk(26, 10 * c, T, H), tag=c)
    Qb = bf16(normals(26, 100, (lq, D)) + 1.0)
    step = 0.02 / scale                                               # ~ +15 log2 units per tile at either scale...
    K1, _ = climbing_keys(26, 1, 1300, D, 4.0 * step)
    segs = [(K1, bf16(normals(26, 2, (1300, D))))]
    sc.check(Qb, segs, [1, 0], SPLITS, f"softmax_scale={scale}", min_rises=3, min_share=0.9)
