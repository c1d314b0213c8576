#!/usr/bin/env python
"""Benchmark of the WorldKV hot path on B200: one "step" = one chunk step of the full denoising pass
(workload cfg2: 30 layers x 4 denoising steps of memory attention over window + top-8 retrieved chunks from a
250-chunk compressed pool, plus retrieval, and compression + pool append of the chunk leaving the window).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2|cfg1|cfg3|cfg0]

Prints ONE JSON line.  `value` = attention FLOPs of a chunk step / chunk-step time (whole hot path in the
denominator), inputs resident in HBM; `e2e` = the same with the step's inputs copied from pinned host memory and
its outputs copied back inside the timed region.  `--impl reference` times the CPU oracle on a bounded sample.
With N > 1 (torchrun) every rank runs an independent replica of the workload (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import wkinputs as wi  # noqa: E402

METRIC = "memory-attn TFLOP/s over the whole chunk step (attention + retrieval + compression + pool append)"
UNIT = "TFLOP/s"



def ncu_traffic_bytes_per_launch(workload_name: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per memory_attention_kernel launch, from the figures file written
    beside the ncu summary (profiles/memory_attention_cfg2_shape.json).  The capture ran on the cfg2 per-call shape with
    a small pool; the traffic of a launch does not depend on the pool size, so it stands for every cfg2* workload.
    Other workloads (and a missing file) report null."""
    path = os.path.join(ROOT, "profiles", "memory_attention_cfg2_shape.json")
    if not workload_name.startswith("cfg2") or not os.path.exists(path):
        return None
    with open(path) as f:
        d = json.load(f)
    return d["dram_bytes_read_per_launch"] + d["dram_bytes_write_per_launch"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            res.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return res


# ------------------------------------------------------------------------------------------ distributed helpers
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value_ms: float, device) -> float:
    """Largest of the ranks' timings (every rank gets it)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return value_ms
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


# ------------------------------------------------------------------------------------------ workload on the device
class ChunkStepBench:
    """Holds the pool, the per-layer window buffers and rotating inputs of one workload, and runs chunk steps."""

    def __init__(self, w: wi.Workload, device_index: int, evict_sets: int = 4, e2e: bool = True, kv_splits: int = 0,
                 prefill: bool = True, max_splits: int = 8, max_k: int = 0):
        import torch
        from paper_2605_22718_b200 import WorldKV
        from wkinputs import device as wd
        self.torch, self.wd, self.w = torch, wd, w
        self.kv_splits = kv_splits
        self.dev = torch.device("cuda", device_index)
        torch.cuda.set_device(self.dev)
        L, H, T, D = w.n_layers, w.n_heads, w.T, w.D
        self.kv = WorldKV(n_layers=L, n_heads=H, tokens_per_frame=T, n_keep=w.n_keep, pool_slots=w.pool_chunks,
                          max_k=max(w.k, max_k, 1), max_dense_segments=1 + w.window_segments, device=device_index,
                          max_batch=L, max_lq=w.Lq, max_splits=max_splits)
        bf = torch.bfloat16
        n_poses = w.pool_chunks + 4096
        if w.trajectory == "actions":
            self.poses = wi.action_rollout_poses(w.seed, n_poses)
        elif w.trajectory == "loop":
            self.poses = wi.loop_poses(w.seed, w.pool_chunks + 3)
        else:
            self.poses = wi.random_poses(w.seed, n_poses)
        # pool pre-fill through the product path: generate -> compress -> append, all layers of a chunk per call
        Kc = torch.empty((L, w.F * T, D), dtype=bf, device=self.dev)
        Vc = torch.empty((L, w.F * T, D), dtype=bf, device=self.dev)
        self.keep = torch.empty((L, w.C), dtype=torch.int32, device=self.dev)
        for c in range(w.pool_chunks if prefill else 0):
            for l in range(L):
                wd.key_chunk(Kc[l], w.seed, l, c, T, D, w.sigma, w.F)
                wd.value_chunk(Vc[l], w.seed, l, c, T, D, w.F)
            self.kv.compress_chunk(Kc, keep_idx_out=self.keep)
            self.kv.pool_append(0, L, Kc, Vc, self.keep, self.poses[c % len(self.poses)], chunk_tag=c)
        # chunks leaving the window: a few distinct input sets, rotated
        self.evK = [torch.empty((L, w.F * T, D), dtype=bf, device=self.dev) for _ in range(evict_sets)]
        self.evV = [torch.empty((L, w.F * T, D), dtype=bf, device=self.dev) for _ in range(evict_sets)]
        for i in range(evict_sets):
            for l in range(L):
                wd.key_chunk(self.evK[i][l], w.seed, l, w.pool_chunks + i, T, D, w.sigma, w.F)
                wd.value_chunk(self.evV[i][l], w.seed, l, w.pool_chunks + i, T, D, w.F)
        # per-layer dense segments: the denoising chunk and the native window
        nwin = w.window_frames * T
        self.curK = torch.empty((L, w.Lq, H, 128), dtype=bf, device=self.dev)
        self.curV = torch.empty((L, w.Lq, H, 128), dtype=bf, device=self.dev)
        self.winK = torch.empty((L, max(nwin, 1), H, 128), dtype=bf, device=self.dev)
        self.winV = torch.empty((L, max(nwin, 1), H, 128), dtype=bf, device=self.dev)
        base = w.pool_chunks + evict_sets
        for l in range(L):
            wd.fill_normal_bf16(self.curV[l], w.seed, wi.STREAM_V + l, (base + 3) * w.F * T * D)
            tmp = torch.empty((w.F * T, D), dtype=bf, device=self.dev)
            wd.key_chunk(tmp, w.seed, l, base + 3, T, D, w.sigma, w.F)
            self.curK[l].view(-1, D)[:] = tmp[:w.Lq]
            for j in range((nwin + w.F * T - 1) // (w.F * T)):
                r0, r1 = j * w.F * T, min(nwin, (j + 1) * w.F * T)
                wd.key_chunk(tmp, w.seed, l, base + 1 + j, T, D, w.sigma, w.F)
                self.winK[l].view(-1, D)[r0:r1] = tmp[:r1 - r0]
                wd.value_chunk(tmp, w.seed, l, base + 1 + j, T, D, w.F)
                self.winV[l].view(-1, D)[r0:r1] = tmp[:r1 - r0]
        # one Q and one O per (layer, denoising step): rotating buffers far larger than L2
        S = w.denoise_steps
        self.Q = torch.empty((L, S, w.Lq, H, 128), dtype=bf, device=self.dev)
        for l in range(L):
            for s in range(S):
                wd.query(self.Q[l, s], w.seed, l, s, 0)
        self.O = torch.empty_like(self.Q)
        self.slots = torch.full((max(w.k, max_k, 1),), -1, dtype=torch.int32, device=self.dev)
        self.step_no = 0
        self.attn_events = []
        self.e2e = e2e
        # buffer sets: set 0 is the resident one; the end-to-end leg double-buffers Q, the denoising chunk's K/V and O
        # so that host copies of neighbouring steps overlap with compute
        self.sets = [(self.Q, self.curK, self.curV, self.O)]
        if e2e:
            self.hQ = torch.empty(self.Q.shape, dtype=bf, pin_memory=True)
            self.hQ.copy_(self.Q)
            self.hcurK = torch.empty(self.curK.shape, dtype=bf, pin_memory=True)
            self.hcurK.copy_(self.curK)
            self.hcurV = torch.empty(self.curV.shape, dtype=bf, pin_memory=True)
            self.hcurV.copy_(self.curV)
            self.hO = torch.empty(self.O.shape, dtype=bf, pin_memory=True)
            self.sets.append((torch.empty_like(self.Q), torch.empty_like(self.curK), torch.empty_like(self.curV),
                              torch.empty_like(self.O)))
            self.h2d_stream = torch.cuda.Stream(device=self.dev)
            self.d2h_stream = torch.cuda.Stream(device=self.dev)
        torch.cuda.synchronize(self.dev)
        st, flags = self.kv.poll_status()
        if st != 0:
            raise RuntimeError(f"device status after setup: {st} flags {flags}")

    def attention_flops_per_call(self) -> float:
        return self.w.attention_flops()

    def attention_calls_per_step(self) -> int:
        return self.w.n_layers * self.w.denoise_steps

    def step(self, record_attention_events: bool = False, buffer_set: int = 0):
        torch, w, kv = self.torch, self.w, self.kv
        Q, curK, curV, O = self.sets[buffer_set]
        i = self.step_no
        self.step_no += 1
        pose = self.poses[(w.pool_chunks + i) % len(self.poses)]
        _, n = kv.retrieve(pose, w.k, slots_out=self.slots)
        if record_attention_events:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        for s in range(w.denoise_steps):
            for l in range(w.n_layers):
                segs = [(curK[l], curV[l])]
                if w.window_frames > 0:
                    rows = self.winK.shape[1] // w.window_segments
                    for q in range(w.window_segments):
                        segs.append((self.winK[l, q * rows:(q + 1) * rows], self.winV[l, q * rows:(q + 1) * rows]))
                kv.memory_attention(l, Q[l, s], segs, self.slots, n, O=O[l, s], kv_splits=self.kv_splits)
        if record_attention_events:
            e1.record()
            self.attn_events.append((e0, e1))
        # the chunk leaving the window: one call scores, selects, evicts the oldest stored chunk and stores the kept rows
        j = i % len(self.evK)
        kv.pool_compress_append(0, w.n_layers, self.evK[j], self.evV[j], pose, chunk_tag=w.pool_chunks + i,
                                evict_oldest_if_full=True, keep_idx=self.keep)

    def time_steps(self, steps: int):
        """K chunk steps with every input already resident in HBM."""
        torch = self.torch
        barrier()
        torch.cuda.synchronize(self.dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            self.step(record_attention_events=True)
        e1.record()
        torch.cuda.synchronize(self.dev)
        barrier()
        return e0.elapsed_time(e1)

    def isolated_attention(self, k: int | None = None, kv_splits: int | None = None):
        """The attention call timed on its own, before the sustained steps heat the board into its power cap (the burst
        peak it is set beside was measured the same way).  k / kv_splits override the workload's retrieval budget and
        the split setting (the sweeps of the LingBot-shaped and the full-history workloads)."""
        torch, w, kv = self.torch, self.w, self.kv
        k = w.k if k is None else k
        splits = self.kv_splits if kv_splits is None else kv_splits
        out = {}
        # the attention call timed on its own: 5 warm-up calls, then 24 timed ones whose Q / O / window rotate over the
        # layers' buffers (each call reads other memory than the one before it); median of per-call event times
        pose = self.poses[w.pool_chunks % len(self.poses)]
        _, n_sl = kv.retrieve(pose, k, slots_out=self.slots)

        def attn_call(i):
            l, s_ = i % w.n_layers, (i // w.n_layers) % w.denoise_steps
            segs = [(self.curK[l], self.curV[l])]
            if w.window_frames > 0:
                rows = self.winK.shape[1] // w.window_segments
                for q in range(w.window_segments):
                    segs.append((self.winK[l, q * rows:(q + 1) * rows], self.winV[l, q * rows:(q + 1) * rows]))
            kv.memory_attention(l, self.Q[l, s_], segs, self.slots, n_sl, O=self.O[l, s_], kv_splits=splits)

        for i in range(5):
            attn_call(i)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(24)]
        for i, (a, b) in enumerate(evs):
            a.record()
            attn_call(5 + i)
            b.record()
        torch.cuda.synchronize(self.dev)
        us = statistics.median(a.elapsed_time(b) for a, b in evs) * 1e3
        out["attention_isolated"] = {"us_per_call": us, "tflops": w.attention_flops(k=min(k, n_sl)) / us / 1e6, "calls": 24,
                                     "k": min(k, n_sl), "lkv": w.Lq + w.window_frames * w.T + min(k, n_sl) * w.C}
        return out["attention_isolated"]

    def side_metrics(self, iters: int = 20):
        """The bandwidth-bound calls timed on their own (CUDA events, rotating input sets larger than L2):
        wk_compress_chunk over all layers of a chunk, and wk_retrieve."""
        torch, w, kv = self.torch, self.w, self.kv
        out = {}
        for i in range(4):
            kv.compress_chunk(self.evK[i % len(self.evK)], keep_idx_out=self.keep)
        torch.cuda.synchronize(self.dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            kv.compress_chunk(self.evK[i % len(self.evK)], keep_idx_out=self.keep)
        e1.record()
        torch.cuda.synchronize(self.dev)
        us = e0.elapsed_time(e1) / iters * 1e3
        nbytes = w.n_layers * w.F * w.T * w.D * 2
        out["compress"] = {"us_per_call": us, "bytes_per_call": nbytes, "gbs": nbytes / us / 1e3, "problems": w.n_layers}
        # the same call with one keep-set per head (n_heads problems of 128 columns per chunk instead of one of D columns)
        from paper_2605_22718_b200 import WorldKV, SCORE_PER_HEAD
        kvh = WorldKV(n_layers=w.n_layers, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=1, max_k=1,
                      device=self.dev.index, max_batch=w.n_layers, score_mode=SCORE_PER_HEAD)
        keep_h = torch.empty((w.n_layers, w.n_heads, w.C), dtype=torch.int32, device=self.dev)
        for i in range(4):
            kvh.compress_chunk(self.evK[i % len(self.evK)], keep_idx_out=keep_h)
        torch.cuda.synchronize(self.dev)
        e0.record()
        for i in range(iters):
            kvh.compress_chunk(self.evK[i % len(self.evK)], keep_idx_out=keep_h)
        e1.record()
        torch.cuda.synchronize(self.dev)
        us = e0.elapsed_time(e1) / iters * 1e3
        out["compress_per_head"] = {"us_per_call": us, "bytes_per_call": nbytes, "gbs": nbytes / us / 1e3,
                                    "problems": w.n_layers * w.n_heads}
        del kvh
        pose = self.poses[w.pool_chunks % len(self.poses)]
        e0.record()
        for i in range(iters):
            kv.retrieve(pose, w.k, slots_out=self.slots)
        e1.record()
        torch.cuda.synchronize(self.dev)
        out["retrieve"] = {"us_per_call": e0.elapsed_time(e1) / iters * 1e3, "candidates": kv.pool_count()}
        # query-based retrieval (the appendix variant): the denoising chunk's queries scored against every stored chunk
        # of one layer; the layer rotates so that successive calls read different pool memory
        n = max(2, iters // 4)
        kv.retrieve_query(0, self.Q[0, 0], w.k, slots_out=self.slots)
        torch.cuda.synchronize(self.dev)
        e0.record()
        for i in range(n):
            kv.retrieve_query((i + 1) % w.n_layers, self.Q[(i + 1) % w.n_layers, 0], w.k, slots_out=self.slots)
        e1.record()
        torch.cuda.synchronize(self.dev)
        us = e0.elapsed_time(e1) / n * 1e3
        flops = 2.0 * w.Lq * kv.pool_count() * (w.T + w.n_keep) * w.D
        out["retrieve_query"] = {"us_per_call": us, "candidates": kv.pool_count(), "tflops": flops / us / 1e6}
        # pose retrieval as a streaming scan over far more candidates than a pool holds (32 bytes per candidate): the
        # sizes at which "GB/s of retrieval" means something.  Seeded device-side draws: t ~ N(0, I), q = normalised N(0, I4).
        scan = {}
        gen = torch.Generator(device=self.dev)
        gen.manual_seed(1000 + w.seed)
        ids = torch.empty(16, dtype=torch.int32, device=self.dev)
        for log2n in (16, 20, 24):
            n_c = 1 << log2n
            P = torch.randn((n_c, 8), generator=gen, device=self.dev, dtype=torch.float32)
            P[:, 4:8] /= P[:, 4:8].norm(dim=1, keepdim=True)
            P[:, 3] = 0
            for i in range(3):
                kv.retrieve_scan(P, pose, 16, ids_out=ids)
            torch.cuda.synchronize(self.dev)
            e0.record()
            for i in range(10):
                kv.retrieve_scan(P, pose, 16, ids_out=ids)
            e1.record()
            torch.cuda.synchronize(self.dev)
            us = e0.elapsed_time(e1) / 10 * 1e3
            scan[f"2^{log2n}"] = {"us_per_call": us, "gbs": 32.0 * n_c / us / 1e3}
            del P
        out["retrieve_scan"] = scan
        return out

    def time_steps_e2e(self, steps: int):
        """K chunk steps through the public calls with HOST buffers: every step's Q and denoising-chunk K/V are copied
        from pinned host memory and its O is copied back, inside the timed region.  Copies run on two copy streams and
        are double-buffered, so step i+1's inputs and step i-1's outputs move while step i computes."""
        torch = self.torch
        cs = torch.cuda.current_stream(self.dev)
        ev_h2d, ev_comp, ev_d2h = [None] * steps, [None] * steps, [None] * steps

        def issue_h2d(i):
            Q, curK, curV, _ = self.sets[i % 2]
            with torch.cuda.stream(self.h2d_stream):
                if i >= 2:
                    self.h2d_stream.wait_event(ev_comp[i - 2])      # the buffers' previous user has finished
                Q.copy_(self.hQ, non_blocking=True)
                curK.copy_(self.hcurK, non_blocking=True)
                curV.copy_(self.hcurV, non_blocking=True)
                ev_h2d[i] = torch.cuda.Event()
                ev_h2d[i].record(self.h2d_stream)

        barrier()
        torch.cuda.synchronize(self.dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        self.h2d_stream.wait_event(e0)
        issue_h2d(0)
        for i in range(steps):
            if i + 1 < steps:
                issue_h2d(i + 1)
            cs.wait_event(ev_h2d[i])
            if i >= 2:
                cs.wait_event(ev_d2h[i - 2])                         # O of this buffer set has been read back
            self.step(buffer_set=i % 2)
            ev_comp[i] = torch.cuda.Event()
            ev_comp[i].record(cs)
            with torch.cuda.stream(self.d2h_stream):
                self.d2h_stream.wait_event(ev_comp[i])
                self.hO.copy_(self.sets[i % 2][3], non_blocking=True)
                ev_d2h[i] = torch.cuda.Event()
                ev_d2h[i].record(self.d2h_stream)
        cs.wait_event(ev_d2h[steps - 1])
        if steps >= 2:
            cs.wait_event(ev_d2h[steps - 2])
        e1.record()
        torch.cuda.synchronize(self.dev)
        barrier()
        return e0.elapsed_time(e1)


# ------------------------------------------------------------------------------------------ CPU oracle legs
class OracleSample:
    """The oracle, as it stands, on a bounded sample of the workload: some query rows of one attention call over the
    full KV set of one layer, one compression problem, one retrieval.  Inputs are generated once (untimed)."""

    def __init__(self, w: wi.Workload):
        from oracle import worldkv_oracle as o
        self.o, self.w = o, w
        try:
            from threadpoolctl import threadpool_info
            self.threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            self.threads = os.cpu_count() or 1
        T, D, H = w.T, w.D, w.n_heads
        self.k = min(w.k, 8)
        self.pool = o.PoolModel(n_slots=self.k, n_layers=1)
        self.poses = wi.random_poses(w.seed, self.k + 1)
        self.K0 = None
        for c in range(self.k):
            K = wi.key_chunk_bf16(w.seed, 0, c, T, D, w.sigma, w.F)
            V = wi.value_chunk_bf16(w.seed, 0, c, T, D, w.F)
            if self.K0 is None:
                self.K0 = K
            idx, _, _ = o.compress_chunk(K, T, w.n_keep)
            self.pool.append([K.reshape(-1, H, 128)], [V.reshape(-1, H, 128)], [idx], self.poses[c])
        n_dense = w.Lq + w.window_frames * T
        reps = (n_dense + w.F * T - 1) // (w.F * T)
        Kd = np.concatenate([wi.key_chunk_bf16(w.seed, 0, 100 + r, T, D, w.sigma, w.F) for r in range(reps)])[:n_dense]
        Vd = np.concatenate([wi.value_chunk_bf16(w.seed, 0, 100 + r, T, D, w.F) for r in range(reps)])[:n_dense]
        self.dense = [(Kd.reshape(-1, H, 128), Vd.reshape(-1, H, 128))]
        self.Q = wi.query_bf16(w.seed, 0, 0, 0, w.Lq, D).reshape(w.Lq, H, 128)
        self.many_poses = wi.random_poses(w.seed + 1, w.pool_chunks)
        self.lkv = n_dense + self.k * w.C

    def run(self, attn_rows: int):
        o, w = self.o, self.w
        attn_rows = min(attn_rows, w.Lq)
        rows = np.linspace(0, w.Lq - 1, attn_rows).astype(np.int64)
        t0 = time.perf_counter()
        o.compress_chunk(self.K0, w.T, w.n_keep)
        t_compress = time.perf_counter() - t0
        t0 = time.perf_counter()
        o.retrieve(self.poses[self.k], self.many_poses, list(range(w.pool_chunks)), w.k)
        t_retrieve = time.perf_counter() - t0
        t0 = time.perf_counter()
        o.memory_attention(self.Q, self.dense, self.pool, 0, list(range(self.k)), rows=rows)
        t_attn = time.perf_counter() - t0
        calls = w.n_layers * w.denoise_steps
        est_step_s = t_attn * (w.Lq / attn_rows) * calls + t_compress * w.n_layers + t_retrieve
        flops_step = 4.0 * w.Lq * self.lkv * 128 * w.n_heads * calls
        return {"value": flops_step / est_step_s / 1e12, "unit": UNIT, "cores": self.threads, "kind": "oracle",
                "sample": (f"{attn_rows} of {w.Lq} query rows of one attention call over {self.lkv} KV tokens "
                           f"({t_attn:.2f} s), one compression problem ({t_compress:.2f} s), one retrieval over "
                           f"{w.pool_chunks} poses ({t_retrieve * 1e3:.2f} ms); scaled to {calls} calls + "
                           f"{w.n_layers} problems per step"),
                "est_step_ms": est_step_s * 1e3, "sample_seconds": t_attn + t_compress + t_retrieve}


def oracle_attention_sample(w: wi.Workload, k: int, rows: int = 32):
    """The oracle's attention on `rows` query rows of ONE head over the workload's KV length, inputs drawn for that
    head's 128 columns only (seconds even at the LingBot width); scaled to all rows and heads.  Pool rows are the
    leading C rows of generated chunks (the timing does not depend on which rows are kept)."""
    from oracle import worldkv_oracle as o
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    cols = np.arange(128)
    n_dense = w.Lq + w.window_frames * w.T
    reps = (n_dense + w.F * w.T - 1) // (w.F * w.T)
    Ks = [np.concatenate([wi.key_chunk_bf16(w.seed, 0, 100 + r, w.T, w.D, w.sigma, w.F, cols=cols) for r in range(reps)])[:n_dense]]
    Vs = [np.concatenate([wi.value_chunk_bf16(w.seed, 0, 100 + r, w.T, w.D, w.F, cols=cols) for r in range(reps)])[:n_dense]]
    for c in range(k):
        Ks.append(wi.key_chunk_bf16(w.seed, 0, c, w.T, w.D, w.sigma, w.F, cols=cols)[:w.C])
        Vs.append(wi.value_chunk_bf16(w.seed, 0, c, w.T, w.D, w.F, cols=cols)[:w.C])
    K, V = np.concatenate(Ks)[:, None, :], np.concatenate(Vs)[:, None, :]
    rows = min(rows, w.Lq)
    Q = wi.query_bf16(w.seed, 0, 0, 0, w.Lq, w.D, cols=cols)[np.linspace(0, w.Lq - 1, rows).astype(np.int64)][:, None, :]
    t0 = time.perf_counter()
    o.attention(Q, K, V)
    dt = time.perf_counter() - t0
    est_call_s = dt * (w.Lq / rows) * w.n_heads
    return {"value": 4.0 * w.Lq * K.shape[0] * 128 * w.n_heads / est_call_s / 1e12, "unit": UNIT, "cores": threads,
            "kind": "oracle", "sample": f"{rows} of {w.Lq} query rows of one head over {K.shape[0]} KV tokens ({dt:.2f} s), "
                                        f"scaled to all rows and {w.n_heads} heads"}


def run_config_sweep(args):
    """One JSON line per (workload, retrieval budget, KV split): the attention call timed on its own (median of 24
    calls), for the single-layer benchmark workloads -- the Matrix-Game shape (cfg1), the LingBot shape at
    k = 2, 4, 8, 16 (cfg3), the full one-minute history uncompressed and compressed at every split setting
    (cfg4, cfg4c), and the paper's own window on both shapes."""
    import torch
    rank, local, world = dist_env()
    if rank != 0:
        return
    peaks = load_peaks()
    plan = [("cfg1", [None], [0]), ("cfg3", [2, 4, 8, 16], [0]), ("paper_mg", [None], [0]), ("paper_lb", [None], [0]),
            ("cfg4", [None], [1, 2, 4, 8, 16, 0]), ("cfg4c", [None], [1, 2, 4, 8, 16, 0])]
    only = set(args.sweep_only.split(",")) if args.sweep_only else None
    for name, ks, splits_list in plan:
        if only and name not in only:
            continue
        w = wi.WORKLOADS[name]
        b = ChunkStepBench(w, local, e2e=False, max_splits=16, max_k=max([k or 0 for k in ks] + [w.k]))
        sampler = ClockSampler(local)
        for k in ks:
            cpu = None if args.no_cpu_baseline else oracle_attention_sample(w, w.k if k is None else k)
            for sp in splits_list:
                sampler.start()
                iso = b.isolated_attention(k=k, kv_splits=sp)
                clocks = sampler.stop()
                st, flags = b.kv.poll_status()
                if st != 0:
                    raise RuntimeError(f"device status {st} flags {flags}")
                line = {"workload": name, "heads": w.n_heads, "tokens_per_frame": w.T, "lq": w.Lq, "k": iso["k"],
                        "lkv": iso["lkv"], "kv_splits": sp, "us_per_call": iso["us_per_call"], "tflops": iso["tflops"],
                        "frac_of_burst_peak": iso["tflops"] / peaks["bf16_tflops"],
                        "frac_of_sustained_peak": iso["tflops"] / peaks["bf16_tflops_sustained"],
                        "clocks": clocks, "cpu_baseline": cpu, "data": "synthetic"}
                print(json.dumps(line), flush=True)
        del b
        torch.cuda.empty_cache()


def run_reference(args, w: wi.Workload):
    rank, _, world = dist_env()
    if rank != 0:
        return
    sample = OracleSample(w)
    rows = max(1, args.oracle_rows // 4)
    times, last = [], None
    for i in range(args.warmup + args.steps):
        last = sample.run(rows)
        if i >= args.warmup:
            times.append(last)
    value = statistics.mean(t["value"] for t in times)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": statistics.mean(t["est_step_ms"] for t in times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "layers": w.n_layers, "denoise_steps": w.denoise_steps, "heads": w.n_heads,
                       "tokens_per_frame": w.T, "lq": w.Lq, "lkv": w.Lkv, "pool_chunks": w.pool_chunks, "k": w.k,
                       "l2": "inputs_larger_than_l2", "parallelism": "replicas" if world > 1 else "1gpu",
                       "note": "CPU oracle on a bounded sample per step, scaled to one chunk step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "sample_seconds": statistics.mean(t["sample_seconds"] for t in times)}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ main
def run_ours(args, w: wi.Workload):
    import torch
    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("NCCL_DEBUG", "INFO")   # the communicator log (stderr) shows the ranks that joined
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2605_22718_b200.build import build_all
    if rank == 0:
        build_all()
    barrier()
    peaks = load_peaks()
    bench = ChunkStepBench(w, local_rank, e2e=not args.no_e2e, kv_splits=args.kv_splits)
    dev = bench.dev
    isolated = bench.isolated_attention()
    # the bandwidth-bound calls are timed on their own as well, before the sustained steps heat the board (right after
    # them the SM clock is still at its power-capped level and these short kernels would be timed at it)
    side = bench.side_metrics()
    lingbot = None
    if w.name == "cfg2" and rank == 0 and not args.no_lingbot:
        # the other model shape (1,560 tokens per frame, 40 heads): its attention call and its compression batch, timed
        # on their own (a 3.8 GB pool beside the 61 GB one)
        lingbot = lingbot_figures(local_rank, peaks)
    for _ in range(args.warmup):
        bench.step()
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(local_rank)
    launches0 = bench.kv.launch_count()
    if rank == 0:
        sampler.start()
    if args.profiler_range:   # lets `ncu --profile-from-start off` see the timed steps only
        torch.cuda.cudart().cudaProfilerStart()
    ms = bench.time_steps(args.steps)
    if args.profiler_range:
        torch.cuda.cudart().cudaProfilerStop()
    clocks = sampler.stop() if rank == 0 else None
    launches = bench.kv.launch_count() - launches0
    ms = max_over_ranks(ms, dev)
    attn_ms = [a.elapsed_time(b) for a, b in bench.attn_events]
    st, flags = bench.kv.poll_status()
    if st != 0:
        raise RuntimeError(f"device status after the timed region: {st} flags {flags}")
    e2e = None
    if not args.no_e2e:
        bench.time_steps_e2e(2)   # warm the copy path
        ms_e2e = max_over_ranks(bench.time_steps_e2e(args.steps), dev)
    side["compress"]["frac_of_hbm_peak"] = side["compress"]["gbs"] / peaks["hbm_gbs"]
    side["compress"]["peak_gbs"] = peaks["hbm_gbs"]
    for key in ("2^16", "2^20", "2^24"):
        side["retrieve_scan"][key]["frac_of_hbm_peak"] = side["retrieve_scan"][key]["gbs"] / peaks["hbm_gbs"]
    calls = bench.attention_calls_per_step()
    flops_call = bench.attention_flops_per_call()
    flops_step = flops_call * calls
    ms_per_step = ms / args.steps
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12
    if not args.no_e2e:
        h2d = bench.hQ.numel() * 2 + bench.hcurK.numel() * 2 + bench.hcurV.numel() * 2
        d2h = bench.hO.numel() * 2
        e2e = {"value": world * flops_step / (ms_e2e / args.steps * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps,
               "note": "copied per step: Q and the denoising chunk's K/V in, O out; the window's K/V and the chunk "
                       "leaving the window stay on the device, where a model produces them"}
    if rank != 0:
        return
    attn_launch_ms = statistics.mean(attn_ms) / calls
    achieved = flops_call / (attn_launch_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    comp_bytes = 7.5 * w.T * w.D * 2 * w.n_layers
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": w.name, "layers": w.n_layers, "denoise_steps": w.denoise_steps, "heads": w.n_heads,
                   "tokens_per_frame": w.T, "lq": w.Lq, "lkv": w.Lkv, "pool_chunks": w.pool_chunks, "k": w.k,
                   "l2": "inputs_larger_than_l2", "parallelism": "replicas" if world > 1 else "1gpu"},
        "chunk_step_ms": ms_per_step,
        "attention": {"calls_per_step": calls, "flops_per_call": flops_call, "ms_per_call": attn_launch_ms,
                      "tflops": achieved, "share_of_step": statistics.mean(attn_ms) / ms_per_step},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "peak_source": peaks["source"] + " sustained",
                     "traffic": ncu_traffic_bytes_per_launch(w.name),
                     "kernel": "memory_attention_kernel"},
        "attention_isolated": dict(isolated, frac_of_burst_peak=isolated["tflops"] / peaks["bf16_tflops"]),
        "compress": side["compress"], "compress_per_head": side["compress_per_head"], "retrieve": side["retrieve"], "retrieve_query": side["retrieve_query"],
        "retrieve_scan": side["retrieve_scan"],
        "attention_lingbot": None if lingbot is None else lingbot["attention"],
        "compress_lingbot": None if lingbot is None else lingbot["compress"],
        "compress_append_bytes_per_step": comp_bytes,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
    }
    if not args.no_cpu_baseline:
        cb = OracleSample(w).run(args.oracle_rows)
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line), flush=True)


def lingbot_figures(device_index: int, peaks):
    """cfg3 (LingBot-World-Fast shape, k = 8): the attention call timed on its own, and wk_compress_chunk over 40 layers'
    worth of chunks (1.9 GB of keys per call)."""
    import torch
    from paper_2605_22718_b200 import WorldKV
    from wkinputs import device as wd
    w = wi.WORKLOADS["cfg3"]
    b = ChunkStepBench(w, device_index, e2e=False)
    iso = b.isolated_attention()
    st, flags = b.kv.poll_status()
    if st != 0:
        raise RuntimeError(f"device status {st} flags {flags}")
    out = {"attention": dict(iso, workload="cfg3", heads=w.n_heads, tokens_per_frame=w.T,
                             frac_of_burst_peak=iso["tflops"] / peaks["bf16_tflops"])}
    del b
    torch.cuda.empty_cache()
    batch = 40
    kv = WorldKV(n_layers=1, n_heads=w.n_heads, tokens_per_frame=w.T, n_keep=w.n_keep, pool_slots=1, max_k=1,
                 device=device_index, max_batch=batch)
    sets = []
    for i in range(3):
        K = torch.empty((batch, w.F * w.T, w.D), dtype=torch.bfloat16, device=f"cuda:{device_index}")
        for l in range(batch):
            wd.key_chunk(K[l], w.seed, l, i, w.T, w.D, w.sigma, w.F)
        sets.append(K)
    keep = torch.empty((batch, w.C), dtype=torch.int32, device=f"cuda:{device_index}")
    for i in range(3):
        kv.compress_chunk(sets[i], keep_idx_out=keep)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(24):
        kv.compress_chunk(sets[i % 3], keep_idx_out=keep)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / 24 * 1e3
    nbytes = batch * w.F * w.T * w.D * 2
    out["compress"] = {"us_per_call": us, "bytes_per_call": nbytes, "gbs": nbytes / us / 1e3, "problems": batch,
                       "frac_of_hbm_peak": nbytes / us / 1e3 / peaks["hbm_gbs"], "workload": "cfg3 shape, 40 problems"}
    return out


def run_host_tier(args, w):
    """The chunk step with every stored chunk in page-locked host memory (the paper's CPU-offloading direction, Section 7):
    the device pool holds only two sets of k slots.  While step i computes, the k chunks step i + 1 will attend to are
    picked by pose over the host tier's pose table (wk_retrieve_scan) and loaded on a copy stream; the chunk leaving the
    window is compressed, appended, copied out to the host tier and evicted.  The poses of the rollout are scripted, so
    the next pose is known one step ahead; in a live rollout it is the pending action's pose.  One JSON line."""
    import dataclasses
    import torch
    rank, local, world = dist_env()
    if rank != 0:
        return
    k = max(w.k, 1)
    n_host = 4 * k
    w2 = dataclasses.replace(w, pool_chunks=2 * k + 2, name=f"{w.name}_host_tier")
    b = ChunkStepBench(w2, local, e2e=False, kv_splits=args.kv_splits, prefill=False)
    kv, dev = b.kv, b.dev
    L, T, D = w.n_layers, w.T, w.D
    nbytes = kv.host_chunk_bytes()
    host = [torch.empty(nbytes // 2, dtype=torch.int16).pin_memory() for _ in range(n_host + 1)]
    host_pose = torch.zeros((n_host, 8), dtype=torch.float32)
    comp, copy, out = torch.cuda.current_stream(dev), torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    # fill the host tier through the product path: generate -> compress -> append -> copy out -> evict
    Kc, Vc = b.evK[0], b.evV[0]
    for c in range(n_host):
        for l in range(L):
            b.wd.key_chunk(Kc[l], w.seed, l, c, T, D, w.sigma, w.F)
            b.wd.value_chunk(Vc[l], w.seed, l, c, T, D, w.F)
        kv.compress_chunk(Kc, keep_idx_out=b.keep)
        slot = kv.pool_append(0, L, Kc, Vc, b.keep, b.poses[c], chunk_tag=c)
        kv.pool_store_host(slot, host[c])
        kv.pool_evict(slot)
        host_pose[c] = torch.from_numpy(np.asarray(b.poses[c], dtype=np.float32))
    torch.cuda.synchronize(dev)
    pose_dev = host_pose.to(dev)
    # transfer rates of one chunk image, each direction on its own
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(4):
        s = kv.pool_load_host(0, L, host[i], b.poses[i])
        kv.pool_evict(s)
    e1.record()
    torch.cuda.synchronize(dev)
    h2d_gbs = 4 * nbytes / e0.elapsed_time(e1) / 1e6
    s = kv.pool_load_host(0, L, host[0], b.poses[0])
    e0.record()
    for i in range(4):
        kv.pool_store_host(s, host[n_host])
    e1.record()
    torch.cuda.synchronize(dev)
    kv.pool_evict(s)
    d2h_gbs = 4 * nbytes / e0.elapsed_time(e1) / 1e6
    ids_dev = torch.empty(k, dtype=torch.int32, device=dev)
    scratch = torch.empty(kv.lib.wk_retrieve_scan_scratch_bytes(), dtype=torch.uint8, device=dev)
    sets = [[], []]                      # device slots of the two chunk sets
    slot_lists = [torch.full((k,), -1, dtype=torch.int32, device=dev) for _ in range(2)]
    loaded = [None, None]                # event: set i is on the device
    done = [None, None]                  # event: the step that used set i has finished
    stored = [None, -1]                  # event: the last copy-out has left its slot; that slot (kept until then)

    def fetch(step: int):
        """Pick and load the chunks of `step` into set step % 2 (copy stream)."""
        j = step % 2
        with torch.cuda.stream(copy):
            if done[j] is not None:
                copy.wait_event(done[j])
            for sl in sets[j]:
                kv.pool_evict(sl, stream=copy)
            pose = b.poses[(n_host + step) % len(b.poses)]
            kv.retrieve_scan(pose_dev, pose, k, ids_out=ids_dev, scratch=scratch, stream=copy)
            ids = ids_dev.cpu().tolist()                     # waits for the copy stream only
            sets[j] = [kv.pool_load_host(0, L, host[c], host_pose[c].tolist(), chunk_tag=c, stream=copy) for c in ids if c >= 0]
            slot_lists[j][:len(sets[j])] = torch.tensor(sets[j], dtype=torch.int32)
            loaded[j] = torch.cuda.Event()
            loaded[j].record(copy)

    def step(i: int):
        j = i % 2
        comp.wait_event(loaded[j])
        for st in range(w.denoise_steps):
            for l in range(L):
                segs = [(b.curK[l], b.curV[l])]
                if w.window_frames > 0:
                    segs.append((b.winK[l], b.winV[l]))
                kv.memory_attention(l, b.Q[l, st], segs, slot_lists[j], len(sets[j]), O=b.O[l, st], kv_splits=args.kv_splits)
        done[j] = torch.cuda.Event()
        done[j].record(comp)
        # the chunk leaving the window goes to the host tier, replacing its oldest chunk
        e = i % len(b.evK)
        if stored[0] is not None:        # the previous copy-out has finished: only now is its slot given back
            comp.wait_event(stored[0])
            kv.pool_evict(stored[1])
        kv.compress_chunk(b.evK[e], keep_idx_out=b.keep)
        slot = kv.pool_append(0, L, b.evK[e], b.evV[e], b.keep, b.poses[(n_host + i) % len(b.poses)], chunk_tag=n_host + i)
        ev = torch.cuda.Event()
        ev.record(comp)
        with torch.cuda.stream(out):
            out.wait_event(ev)
            kv.pool_store_host(slot, host[n_host], stream=out)
            stored[0] = torch.cuda.Event()
            stored[0].record(out)
            stored[1] = slot

    fetch(0)
    total = max(3, args.warmup) + args.steps
    for i in range(total):
        if i == max(3, args.warmup):
            t0 = torch.cuda.Event(enable_timing=True)
            t0.record(comp)
        step(i)
        fetch(i + 1)
    t1 = torch.cuda.Event(enable_timing=True)
    t1.record(comp)
    torch.cuda.synchronize(dev)
    st, flags = kv.poll_status()
    if st != 0:
        raise RuntimeError(f"device status {st} flags {flags}")
    ms = t0.elapsed_time(t1) / args.steps
    flops = w.attention_flops() * b.attention_calls_per_step()
    print(json.dumps({"metric": "chunk step with the stored chunks in host memory", "unit": "ms", "workload": w.name,
                      "steps": args.steps, "chunk_step_ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                      "host_chunks": n_host, "chunk_bytes": nbytes, "fetch_bytes_per_step": k * nbytes,
                      "store_bytes_per_step": nbytes, "h2d_gbs": h2d_gbs, "d2h_gbs": d2h_gbs, "data": "synthetic"}))


def run_retention_sweep(args, w):
    """Throughput against retention (the intra-chunk compression ratios of the ablation in Section 5.4, as a cost curve): the same chunk step
    with n_keep in {0, T/4, T/2, T, 3T/2, 2T} kept non-anchor tokens per stored chunk, i.e. stored chunks of
    T + n_keep rows.  One JSON line with one point per rung; the pool holds 2k chunks (the step's traffic does not
    depend on how many more are stored)."""
    import dataclasses
    import torch
    rank, local, world = dist_env()
    if rank != 0:
        return
    T = w.T
    points = []
    for nk in (0, T // 4, T // 2, T, 3 * T // 2, 2 * T):
        w2 = dataclasses.replace(w, n_keep=nk, pool_chunks=2 * max(w.k, 1), name=f"{w.name}_keep{nk}")
        b = ChunkStepBench(w2, local, e2e=False, kv_splits=args.kv_splits)
        for _ in range(max(3, args.warmup)):
            b.step()
        b.attn_events = []
        ms = b.time_steps(args.steps)
        attn_ms = statistics.mean(e0.elapsed_time(e1) for e0, e1 in b.attn_events) / b.attention_calls_per_step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(10):
            b.kv.compress_chunk(b.evK[i % len(b.evK)], keep_idx_out=b.keep)
        e1.record()
        torch.cuda.synchronize(b.dev)
        st, flags = b.kv.poll_status()
        if st != 0:
            raise RuntimeError(f"device status {st} flags {flags}")
        points.append({"n_keep": nk, "retention": (T + nk) / (w.F * T), "stored_rows_per_chunk": T + nk, "lkv": w2.Lkv,
                       "chunk_step_ms": ms / args.steps, "attention_us_per_call": attn_ms * 1e3,
                       "attention_tflops": w2.attention_flops() / (attn_ms * 1e-3) / 1e12,
                       "compress_us_per_call": e0.elapsed_time(e1) / 10 * 1e3,
                       "pool_bytes_per_chunk": 2 * w.n_layers * (T + nk) * w.D * 2})
        del b
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "chunk-step cost against retention", "unit": "ms", "workload": w.name, "steps": args.steps,
                      "k": w.k, "data": "synthetic", "points": points}))


def spawn_replicas(n: int) -> int:
    """`bench.py --gpus N` started as a plain process: re-runs itself as N ranks (one per GPU) under torch.distributed.run
    with the same arguments, so that N replicas are measured whichever way the script is started.  Returns the exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(wi.WORKLOADS))
    ap.add_argument("--oracle-rows", type=int, default=1024)
    ap.add_argument("--kv-splits", type=int, default=0, help="wk_memory_attention's kv_splits argument (0 = default)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--profiler-range", action="store_true", help="bracket the timed steps with cudaProfilerStart/Stop")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--host-tier", action="store_true",
                    help="instead of the bench line: the chunk step with the stored chunks fetched from host memory")
    ap.add_argument("--config-sweep", action="store_true",
                    help="instead of the bench line: the attention call of cfg1, cfg3 (k sweep), cfg4 / cfg4c (split sweep) "
                         "and the paper's window on both shapes, one JSON line each")
    ap.add_argument("--sweep-only", default="", help="comma-separated workload names to restrict --config-sweep to")
    ap.add_argument("--no-lingbot", action="store_true", help="skip the LingBot-shape figures of the default line")
    ap.add_argument("--retention-sweep", action="store_true",
                    help="instead of the bench line: chunk-step cost for n_keep in {0, T/4, T/2, T, 3T/2, 2T}")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus))
    w = wi.WORKLOADS[args.workload]
    if args.config_sweep:
        run_config_sweep(args)
    elif args.host_tier:
        run_host_tier(args, w)
    elif args.retention_sweep:
        run_retention_sweep(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
