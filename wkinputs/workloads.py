"""The five benchmark workloads as data (shapes only; tensors come from ``gen``/``poses``).

Shapes follow the paper's two backbones: 880 (Matrix-Game-2.0) and 1,560 (LingBot-World-Fast)
tokens per latent frame (Section 1), 3-frame chunks (Section 3), the anchor kept whole plus
25 % of the 2T non-anchor tokens (Section 4.3).  Head counts, head_dim, layer count,
denoising steps and pool sizes are the benchmark's.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Tuple


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    n_layers: int
    n_heads: int
    head_dim: int
    T: int                 # tokens per latent frame
    F: int                 # latent frames per chunk
    q_frames: int          # frames in the query (denoising) chunk
    window_frames: int     # native sliding-window frames besides the denoising chunk
    n_keep: int            # kept non-anchor tokens per stored chunk
    pool_chunks: int       # M: stored chunks when the measurement starts
    k: int                 # retrieval budget
    sigma: float           # key noise of the redundancy generator
    denoise_steps: int = 1
    trajectory: str = "loop"           # "random" | "loop" | "actions"
    k_sweep: Tuple[int, ...] = field(default_factory=tuple)
    rollout_chunks: int = 0
    window_segments: int = 1           # the dense window is passed as this many equal segments (e.g. sink + recent)

    @property
    def D(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def Lq(self) -> int:
        return self.q_frames * self.T

    @property
    def C(self) -> int:
        """Rows of one stored (compressed) chunk."""
        return self.T + self.n_keep

    @property
    def Lkv(self) -> int:
        return self.Lq + self.window_frames * self.T + min(self.k, self.pool_chunks) * self.C

    def attention_flops(self, k: int | None = None) -> float:
        lkv = self.Lq + self.window_frames * self.T + (self.k if k is None else k) * self.C
        return 4.0 * self.Lq * lkv * self.head_dim * self.n_heads


WORKLOADS = {
    # tiny correctness case: 880 + 1,760 + 1 x 1,320 = 3,960 KV tokens
    "cfg0": Workload("cfg0", seed=0, n_layers=1, n_heads=2, head_dim=128, T=880, F=3, q_frames=1,
                     window_frames=2, n_keep=440, pool_chunks=8, k=1, sigma=0.1, trajectory="random"),
    # Matrix-Game-2.0-shaped single layer: 2,640 + 5,280 + 4 x 1,320 = 13,200 KV tokens
    "cfg1": Workload("cfg1", seed=1, n_layers=1, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                     window_frames=6, n_keep=440, pool_chunks=125, k=4, sigma=0.1, trajectory="loop"),
    # full denoising pass: 30 layers x 4 steps, top-8, pool of 250 chunks, 120-chunk rollout
    "cfg2": Workload("cfg2", seed=2, n_layers=30, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                     window_frames=6, n_keep=440, pool_chunks=250, k=8, sigma=0.1, denoise_steps=4,
                     trajectory="actions", rollout_chunks=120),
    # profiling case: cfg2's per-call shapes (18,480 KV tokens, 30-problem compression batch is cut to 2 layers)
    # with a pool small enough (260 MB) for multi-pass profiler captures
    "cfg2_small": Workload("cfg2_small", seed=2, n_layers=2, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                           window_frames=6, n_keep=440, pool_chunks=16, k=8, sigma=0.1, denoise_steps=4,
                           trajectory="actions", rollout_chunks=8),
    # profiling case: all 30 layers (so compression runs at its real batch of 30 problems) with a 4-chunk pool (1 GB)
    "cfg2_pool4": Workload("cfg2_pool4", seed=2, n_layers=30, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                           window_frames=6, n_keep=440, pool_chunks=4, k=4, sigma=0.1, denoise_steps=4,
                           trajectory="actions", rollout_chunks=8),
    # LingBot-World-Fast-shaped single layer, k swept over {2, 4, 8, 16}
    "cfg3": Workload("cfg3", seed=3, n_layers=1, n_heads=40, head_dim=128, T=1560, F=3, q_frames=3,
                     window_frames=6, n_keep=780, pool_chunks=80, k=8, sigma=0.05, trajectory="loop",
                     k_sweep=(2, 4, 8, 16)),
    # the paper's own window (Section 5.1): 18 latent frames = sink 3 + retrieved 9 (six chunks compressed to 1.5
    # frames each) + recent 3 + denoising 3, on both model shapes; sink and recent are separate dense segments
    "paper_mg": Workload("paper_mg", seed=5, n_layers=1, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                         window_frames=6, n_keep=440, pool_chunks=125, k=6, sigma=0.1, trajectory="loop",
                         window_segments=2),
    "paper_lb": Workload("paper_lb", seed=6, n_layers=1, n_heads=40, head_dim=128, T=1560, F=3, q_frames=3,
                         window_frames=6, n_keep=780, pool_chunks=80, k=6, sigma=0.05, trajectory="loop",
                         window_segments=2),
    # full-KV stress: the whole uncompressed one-minute history (125 x 2,640 = 330,000 tokens)
    "cfg4": Workload("cfg4", seed=4, n_layers=1, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                     window_frames=0, n_keep=1760, pool_chunks=125, k=125, sigma=0.1, trajectory="loop"),
    # the same one-minute history with every chunk compressed to 50 % (125 x 1,320 = 165,000 tokens), all of it attended
    "cfg4c": Workload("cfg4c", seed=4, n_layers=1, n_heads=12, head_dim=128, T=880, F=3, q_frames=3,
                      window_frames=0, n_keep=440, pool_chunks=125, k=125, sigma=0.1, trajectory="loop"),
}
