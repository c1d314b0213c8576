"""ctypes binding of libworldkv.so: the same calls as include/wk.h, argument marshalling only.

PyTorch supplies device memory and streams; every step of the path runs in the library's kernels.
There is no fallback: if the shared library is missing or no sm_100 device is present, loading or
``wk_create`` fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libworldkv.so")

WK_OK = 0
WK_ERR_ARG, WK_ERR_SHAPE, WK_ERR_POOL_FULL, WK_ERR_BAD_SLOT = -1, -2, -3, -4
WK_ERR_CUDA, WK_ERR_TIMEOUT, WK_ERR_NONFINITE, WK_ERR_UNBOUND, WK_ERR_NO_DEVICE = -5, -6, -7, -8, -9
WK_DEV_BAD_SLOT, WK_DEV_TIMEOUT, WK_DEV_NONFINITE = 1, 2, 4


class wk_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("tokens_per_frame", C.c_int32), ("frames_per_chunk", C.c_int32), ("n_keep", C.c_int32),
                ("pool_slots", C.c_int32), ("max_k", C.c_int32), ("max_dense_segments", C.c_int32),
                ("device", C.c_int32), ("softmax_scale", C.c_float), ("score_mode", C.c_int32)]


class wk_dense_seg(C.Structure):
    _fields_ = [("K", C.c_void_p), ("V", C.c_void_p), ("n_tokens", C.c_int32), ("reserved", C.c_int32)]


SCORE_WHOLE_KEY, SCORE_PER_HEAD = 0, 2     # wk_config.score_mode


class WkError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_string(status)} ({status})")
        self.status = status


_lib = None


def load_library() -> C.CDLL:
    """Loads libworldkv.so (built in-tree by paper_2605_22718_b200.build) and declares its symbols."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2605_22718_b200.build` (needs nvcc); "
                           "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    cfgp = C.POINTER(wk_config)
    sigs = {
        "wk_create": (i32, [cfgp, C.POINTER(vp)]),
        "wk_destroy": (None, [vp]),
        "wk_pool_bytes": (sz, [cfgp]),
        "wk_scratch_bytes": (sz, [cfgp, i32, i32, i32]),
        "wk_bind": (i32, [vp, vp, sz, vp, sz, i32, i32, i32]),
        "wk_compress_chunk": (i32, [vp, vp, i64, i32, vp, vp, vp]),
        "wk_pool_append": (i32, [vp, i32, i32, vp, vp, i64, vp, C.POINTER(C.c_float), i64, C.POINTER(i32), vp]),
        "wk_pool_compress_append": (i32, [vp, i32, i32, vp, vp, i64, vp, C.POINTER(C.c_float), i64, i32, C.POINTER(i32),
                                          C.POINTER(i32), vp]),
        "wk_pool_evict": (i32, [vp, i32, vp]),
        "wk_pool_oldest": (i32, [vp]),
        "wk_pool_count": (i32, [vp]),
        "wk_pool_tag": (i64, [vp, i32]),
        "wk_retrieve": (i32, [vp, C.POINTER(C.c_float), i32, vp, vp, C.POINTER(i32), vp]),
        "wk_retrieve_query": (i32, [vp, i32, vp, i32, i32, vp, vp, C.POINTER(i32), vp]),
        "wk_host_chunk_bytes": (C.c_size_t, [vp]),
        "wk_pool_store_host": (i32, [vp, i32, vp, vp]),
        "wk_pool_load_host": (i32, [vp, i32, i32, vp, C.POINTER(C.c_float), C.c_int64, C.POINTER(i32), vp]),
        "wk_retrieve_scan_scratch_bytes": (C.c_size_t, []),
        "wk_retrieve_scan": (i32, [vp, vp, vp, C.c_int64, C.POINTER(C.c_float), i32, vp, vp, i32, vp, C.c_size_t, vp]),
        "wk_retrieve_noalloc": (i32, [vp, vp, i32, C.POINTER(C.c_float), i32, i32, vp, vp, vp]),
        "wk_memory_attention": (i32, [vp, i32, vp, i32, C.POINTER(wk_dense_seg), i32, vp, i32, vp, vp, i32, vp]),
        "wk_poll_status": (i32, [vp, C.POINTER(C.c_uint32), vp]),
        "wk_status_string": (C.c_char_p, [i32]),
        "wk_last_cuda_error": (i32, [vp]),
        "wk_launch_count": (i64, [vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


EXPORTED_SYMBOLS = ("wk_create", "wk_destroy", "wk_pool_bytes", "wk_scratch_bytes", "wk_bind", "wk_compress_chunk",
                    "wk_pool_append", "wk_pool_compress_append", "wk_pool_evict", "wk_pool_oldest", "wk_pool_count", "wk_pool_tag", "wk_retrieve",
                    "wk_retrieve_noalloc", "wk_retrieve_query", "wk_retrieve_scan", "wk_retrieve_scan_scratch_bytes",
                    "wk_host_chunk_bytes", "wk_pool_store_host", "wk_pool_load_host",
                    "wk_memory_attention", "wk_poll_status", "wk_status_string", "wk_last_cuda_error",
                    "wk_launch_count")


def status_string(status: int) -> str:
    return load_library().wk_status_string(status).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def retrieve_noalloc(poses: torch.Tensor, valid: torch.Tensor, cur_pose: Sequence[float], k: int, max_k: int,
                     slots_out: torch.Tensor, dist_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """wk_retrieve_noalloc: pose retrieval for callers that may not allocate device memory (no context, scratch built
    into the library).  poses [n_slots, 8] fp32, valid [n_slots] int32, slots_out [max_k] int32, dist_out [max_k] fp64 -- all
    preallocated by the caller; this wrapper allocates nothing either."""
    pose_arr = (C.c_float * 8)(*[float(x) for x in cur_pose])
    st = load_library().wk_retrieve_noalloc(poses.data_ptr(), valid.data_ptr(), poses.shape[0], pose_arr, k, max_k,
                                            slots_out.data_ptr(), _ptr(dist_out), _stream(stream))
    if st != WK_OK:
        raise WkError(st, "wk_retrieve_noalloc")


class WorldKV:
    """One library context plus the two device buffers it needs (allocated through torch).

    Method names and arguments mirror include/wk.h.  Tensors are CUDA tensors: bf16 [tokens, H, 128]
    (or [tokens, D]) contiguous; index tensors int32.
    """

    def __init__(self, n_layers: int, n_heads: int, tokens_per_frame: int, n_keep: int, pool_slots: int, max_k: int,
                 frames_per_chunk: int = 3, max_dense_segments: int = 4, device: int = 0, softmax_scale: float = 0.0,
                 max_batch: int = 1, max_lq: int = 0, max_splits: int = 1, score_mode: int = 0):
        self.lib = load_library()
        self.cfg = wk_config(n_layers, n_heads, 128, tokens_per_frame, frames_per_chunk, n_keep, pool_slots, max_k,
                             max_dense_segments, device, softmax_scale, score_mode)
        self.score_mode, self.n_heads = score_mode, n_heads
        self.T, self.F, self.H, self.D = tokens_per_frame, frames_per_chunk, n_heads, n_heads * 128
        self.C = tokens_per_frame + n_keep
        self.NA = (frames_per_chunk - 1) * tokens_per_frame
        self.n_layers, self.pool_slots, self.max_k = n_layers, pool_slots, max_k
        self.max_lq = max_lq if max_lq > 0 else frames_per_chunk * tokens_per_frame
        handle = C.c_void_p()
        st = self.lib.wk_create(C.byref(self.cfg), C.byref(handle))
        if st != WK_OK:
            raise WkError(st, "wk_create")
        self.ctx = handle
        self.device = torch.device("cuda", device)
        pool_bytes = self.lib.wk_pool_bytes(C.byref(self.cfg))
        scratch_bytes = self.lib.wk_scratch_bytes(C.byref(self.cfg), max_batch, self.max_lq, max_splits)
        self.pool = torch.zeros(pool_bytes, dtype=torch.uint8, device=self.device)
        self.scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=self.device)
        torch.cuda.synchronize(self.device)
        st = self.lib.wk_bind(self.ctx, self.pool.data_ptr(), pool_bytes, self.scratch.data_ptr(), scratch_bytes,
                              max_batch, self.max_lq, max_splits)
        if st != WK_OK:
            raise WkError(st, "wk_bind")

    def close(self) -> None:
        if getattr(self, "ctx", None):
            self.lib.wk_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        self.close()

    # ---- World Compression --------------------------------------------------------------------
    def compress_chunk(self, K_chunks: torch.Tensor, keep_idx_out: Optional[torch.Tensor] = None,
                       scores_out: Optional[torch.Tensor] = None, batch: Optional[int] = None,
                       batch_stride_elems: Optional[int] = None, stream=None) -> torch.Tensor:
        """K_chunks: [batch, F*T, D] bf16.  Returns keep_idx [batch, T + n_keep] int32 ([batch, H, T + n_keep] with
        per-head keep-sets)."""
        if batch is None:
            batch = K_chunks.shape[0] if K_chunks.dim() == 3 else 1
        if batch_stride_elems is None:
            batch_stride_elems = K_chunks.stride(0) if K_chunks.dim() == 3 else self.F * self.T * self.D
        if keep_idx_out is None:
            shape = (batch, self.n_heads, self.C) if self.score_mode == SCORE_PER_HEAD else (batch, self.C)
            keep_idx_out = torch.empty(shape, dtype=torch.int32, device=self.device)
        st = self.lib.wk_compress_chunk(self.ctx, K_chunks.data_ptr(), batch_stride_elems, batch,
                                        keep_idx_out.data_ptr(), _ptr(scores_out), _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_compress_chunk")
        return keep_idx_out

    # ---- chunk pool ---------------------------------------------------------------------------
    def pool_append(self, layer0: int, n: int, K_chunks: torch.Tensor, V_chunks: torch.Tensor, keep_idx: torch.Tensor,
                    pose: Sequence[float], chunk_tag: int = 0, slot: int = -1,
                    batch_stride_elems: Optional[int] = None, stream=None) -> int:
        if batch_stride_elems is None:
            batch_stride_elems = K_chunks.stride(0) if K_chunks.dim() == 3 else self.F * self.T * self.D
        pose_arr = (C.c_float * 8)(*[float(x) for x in pose])
        slot_io = C.c_int32(slot)
        st = self.lib.wk_pool_append(self.ctx, layer0, n, K_chunks.data_ptr(), V_chunks.data_ptr(), batch_stride_elems,
                                     keep_idx.data_ptr(), pose_arr, chunk_tag, C.byref(slot_io), _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_pool_append")
        return slot_io.value

    def pool_compress_append(self, layer0: int, n: int, K_chunks: torch.Tensor, V_chunks: torch.Tensor,
                             pose: Sequence[float], chunk_tag: int = 0, slot: int = -1, evict_oldest_if_full: bool = False,
                             keep_idx: Optional[torch.Tensor] = None, batch_stride_elems: Optional[int] = None,
                             stream=None) -> Tuple[int, int, torch.Tensor]:
        """wk_pool_compress_append: returns (slot, evicted slot or -1, keep_idx)."""
        if batch_stride_elems is None:
            batch_stride_elems = K_chunks.stride(0) if K_chunks.dim() == 3 else self.F * self.T * self.D
        if keep_idx is None:
            shape = (n, self.n_heads, self.C) if self.score_mode == SCORE_PER_HEAD else (n, self.C)
            keep_idx = torch.empty(shape, dtype=torch.int32, device=self.device)
        pose_arr = (C.c_float * 8)(*[float(x) for x in pose])
        slot_io, evicted = C.c_int32(slot), C.c_int32(-1)
        st = self.lib.wk_pool_compress_append(self.ctx, layer0, n, K_chunks.data_ptr(), V_chunks.data_ptr(),
                                              batch_stride_elems, keep_idx.data_ptr(), pose_arr, chunk_tag,
                                              1 if evict_oldest_if_full else 0, C.byref(slot_io), C.byref(evicted),
                                              _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_pool_compress_append")
        return slot_io.value, evicted.value, keep_idx

    def pool_evict(self, slot: int, stream=None) -> None:
        st = self.lib.wk_pool_evict(self.ctx, slot, _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_pool_evict")

    def pool_oldest(self) -> int:
        return self.lib.wk_pool_oldest(self.ctx)

    def pool_count(self) -> int:
        return self.lib.wk_pool_count(self.ctx)

    def pool_tag(self, slot: int) -> int:
        return self.lib.wk_pool_tag(self.ctx, slot)

    # ---- World Retrieval ----------------------------------------------------------------------
    def retrieve(self, cur_pose: Sequence[float], k: int, slots_out: Optional[torch.Tensor] = None,
                 dist_out: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, int]:
        """Returns (slots_out int32[max_k] on the device, count = min(k, M))."""
        if slots_out is None:
            slots_out = torch.empty(max(1, self.max_k), dtype=torch.int32, device=self.device)
        pose_arr = (C.c_float * 8)(*[float(x) for x in cur_pose])
        n_out = C.c_int32(0)
        st = self.lib.wk_retrieve(self.ctx, pose_arr, k, slots_out.data_ptr(), _ptr(dist_out), C.byref(n_out),
                                  _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_retrieve")
        return slots_out, n_out.value

    # ---- host-memory tier ----------------------------------------------------------------------
    def host_chunk_bytes(self) -> int:
        return self.lib.wk_host_chunk_bytes(self.ctx)

    def pool_store_host(self, slot: int, host_dst: torch.Tensor, stream=None) -> None:
        """Copies the chunk in `slot` into a (page-locked) host tensor of host_chunk_bytes() bytes."""
        assert not host_dst.is_cuda and host_dst.numel() * host_dst.element_size() >= self.host_chunk_bytes()
        st = self.lib.wk_pool_store_host(self.ctx, slot, host_dst.data_ptr(), _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_pool_store_host")

    def pool_load_host(self, layer0: int, n: int, host_src: torch.Tensor, pose: Sequence[float], chunk_tag: int = -1,
                       slot: int = -1, stream=None) -> int:
        """Loads layers [layer0, layer0 + n) of a host chunk image into the pool; returns the slot."""
        assert not host_src.is_cuda and host_src.numel() * host_src.element_size() >= self.host_chunk_bytes()
        pose_arr = (C.c_float * 8)(*[float(x) for x in pose])
        slot_io = C.c_int32(slot)
        st = self.lib.wk_pool_load_host(self.ctx, layer0, n, host_src.data_ptr(), pose_arr, chunk_tag, C.byref(slot_io),
                                        _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_pool_load_host")
        return slot_io.value

    def retrieve_scan(self, poses: torch.Tensor, cur_pose: Sequence[float], k: int, valid: Optional[torch.Tensor] = None,
                      ids_out: Optional[torch.Tensor] = None, dist_out: Optional[torch.Tensor] = None,
                      scratch: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """Retrieval over a plain pose array [n, 8] fp32 of any length; returns ids_out int32 (-1 past the count)."""
        if ids_out is None:
            ids_out = torch.empty(max(1, k), dtype=torch.int32, device=self.device)
        if scratch is None:
            scratch = torch.empty(self.lib.wk_retrieve_scan_scratch_bytes(), dtype=torch.uint8, device=self.device)
        pose_arr = (C.c_float * 8)(*[float(x) for x in cur_pose])
        st = self.lib.wk_retrieve_scan(self.ctx, poses.data_ptr(), _ptr(valid), poses.shape[0], pose_arr, k,
                                       ids_out.data_ptr(), _ptr(dist_out), ids_out.numel(), scratch.data_ptr(),
                                       scratch.numel(), _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_retrieve_scan")
        return ids_out

    def retrieve_query(self, layer: int, Q: torch.Tensor, k: int, slots_out: Optional[torch.Tensor] = None,
                       score_out: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, int]:
        """Query-based retrieval: returns (slots_out int32[max_k] on the device, count = min(k, M))."""
        if slots_out is None:
            slots_out = torch.empty(max(1, self.max_k), dtype=torch.int32, device=self.device)
        n_out = C.c_int32(0)
        st = self.lib.wk_retrieve_query(self.ctx, layer, Q.data_ptr(), Q.shape[0], k, slots_out.data_ptr(), _ptr(score_out),
                                        C.byref(n_out), _stream(stream))
        if st != WK_OK:
            raise WkError(st, "wk_retrieve_query")
        return slots_out, n_out.value

    # ---- memory attention ---------------------------------------------------------------------
    def memory_attention(self, layer: int, Q: torch.Tensor, segs: Sequence[Tuple[torch.Tensor, torch.Tensor]],
                         slots: Optional[torch.Tensor], n_slots: int, O: Optional[torch.Tensor] = None,
                         lse_out: Optional[torch.Tensor] = None, kv_splits: int = 0, stream=None) -> torch.Tensor:
        lq = Q.shape[0]
        if O is None:
            O = torch.empty_like(Q)
        arr = (wk_dense_seg * max(1, len(segs)))()
        for i, (k, v) in enumerate(segs):
            arr[i] = wk_dense_seg(k.data_ptr(), v.data_ptr(), k.shape[0], 0)
        st = self.lib.wk_memory_attention(self.ctx, layer, Q.data_ptr(), lq, arr, len(segs), _ptr(slots), n_slots,
                                          O.data_ptr(), _ptr(lse_out), kv_splits, _stream(stream))
        if st != WK_OK:
            raise WkError(st, f"wk_memory_attention (last CUDA error {self.last_cuda_error()})")
        return O

    # ---- status -------------------------------------------------------------------------------
    def poll_status(self, stream=None) -> Tuple[int, int]:
        flags = C.c_uint32(0)
        st = self.lib.wk_poll_status(self.ctx, C.byref(flags), _stream(stream))
        return st, flags.value

    def launch_count(self) -> int:
        return self.lib.wk_launch_count(self.ctx)

    def last_cuda_error(self) -> int:
        return self.lib.wk_last_cuda_error(self.ctx)
