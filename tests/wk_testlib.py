"""Shared helpers for the GPU parity tests: build the same scenario on the device (through the C ABI)
and in the oracle's pool model, from the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

import wkinputs as wi
from wkinputs import device as wd
from oracle import worldkv_oracle as o

ATOL_MAX_ABS = 2e-2     # attention tolerance for bf16 inputs: max-abs
RTOL_L2 = 1e-2          # and relative L2


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def attention_errors(O_gpu: torch.Tensor, O_ref: np.ndarray):
    g = bf16_to_f64(O_gpu).reshape(O_ref.shape)
    err = np.abs(g - O_ref).max()
    rel = np.linalg.norm(g - O_ref) / max(np.linalg.norm(O_ref), 1e-300)
    return err, rel


def assert_attention_close(O_gpu: torch.Tensor, O_ref: np.ndarray, what=""):
    err, rel = attention_errors(O_gpu, O_ref)
    assert err <= ATOL_MAX_ABS and rel <= RTOL_L2, f"{what}: max-abs {err:.3e}, rel-L2 {rel:.3e}"
    return err, rel


class Scenario:
    """A pool filled through wk_compress_chunk + wk_pool_append, mirrored in the oracle's PoolModel."""

    def __init__(self, kv, seed: int, sigma: float, n_layers: int, T: int, H: int, n_keep: int, pool_slots: int,
                 F: int = 3, per_head: bool = False):
        self.kv, self.seed, self.sigma, self.per_head = kv, seed, sigma, per_head
        self.L, self.T, self.H, self.D, self.F, self.n_keep = n_layers, T, H, H * 128, F, n_keep
        self.pool = o.PoolModel(n_slots=pool_slots, n_layers=n_layers)
        self.margins = []

    def chunk_bits(self, chunk: int):
        K = [wi.key_chunk_bf16(self.seed, l, chunk, self.T, self.D, self.sigma, self.F) for l in range(self.L)]
        V = [wi.value_chunk_bf16(self.seed, l, chunk, self.T, self.D, self.F) for l in range(self.L)]
        return K, V

    def append_chunk(self, chunk: int, pose, check=True) -> int:
        K, V = self.chunk_bits(chunk)
        Kd = wd.to_device_bf16(np.stack(K))
        Vd = wd.to_device_bf16(np.stack(V))
        keep = self.kv.compress_chunk(Kd)
        ref = []
        for l in range(self.L):
            if self.per_head:
                idx, _, margin = o.compress_chunk_per_head(K[l], self.T, self.n_keep, self.H)
            else:
                idx, _, margin = o.compress_chunk(K[l], self.T, self.n_keep)
            ref.append(idx)
            self.margins.append(margin)
        if check:
            np.testing.assert_array_equal(keep.cpu().numpy(), np.stack(ref))
        slot = self.kv.pool_append(0, self.L, Kd, Vd, keep, pose, chunk_tag=chunk)
        Kh = [k.reshape(-1, self.H, 128) for k in K]
        Vh = [v.reshape(-1, self.H, 128) for v in V]
        slot_ref = self.pool.append(Kh, Vh, ref, pose, tag=chunk)
        assert slot == slot_ref
        return slot

    def dense_segment(self, layer: int, chunk: int, n_rows: int):
        """First n_rows rows of a generated chunk as a dense (K, V) segment: (device pair, host pair)."""
        K = wi.key_chunk_bf16(self.seed, layer, chunk, self.T, self.D, self.sigma, self.F)[:n_rows]
        V = wi.value_chunk_bf16(self.seed, layer, chunk, self.T, self.D, self.F)[:n_rows]
        dev = (wd.to_device_bf16(K).view(n_rows, self.H, 128), wd.to_device_bf16(V).view(n_rows, self.H, 128))
        host = (K.reshape(n_rows, self.H, 128), V.reshape(n_rows, self.H, 128))
        return dev, host
