"""Seeded synthetic workloads for the FAST-AR attention step.

This module only draws random inputs.  It contains none of the method's
arithmetic (no similarity search, no merging, no hashing decisions, no
attention) and is the single piece of code that both the CPU oracle's tests
and the CUDA path's tests/bench feed from.

The data model follows the two observations the paper motivates its method
with (Section 4, Fig. 3 and Fig. 4): queries/keys cluster semantically and keys
repeat from frame to frame, and only a few prompt tokens matter per frame.

  * centroids  c[h][z] ~ N(0, I_d),  z < C   (per head)
  * cluster map M0(y, x): index of the nearest of C seed points thrown uniformly
    on the toroidal token grid (shared by all heads); frame t uses
    M_t(y, x) = M0(y, (x - floor(shift * t)) mod W)
  * key   k = c[M_t] + sigma * eps,  query q = c[M_t] + sigma * eps'
  * a fraction `resample` of the tokens of every frame (per head independently)
    is replaced by a fresh N(0, I_d) key, its query being that key + sigma*eps'
  * values ~ N(0, I_d)
  * prompt K_p, V_p ~ N(0, I_d); per frame `relevant` tokens at distinct random
    positions are overwritten by 0.8*c_z + 0.6*|c_z|*u  (u a unit vector
    orthogonal to c_z) for the `relevant` most populous clusters z of the frame
  * the LSH projection matrix R[T*b][d] ~ N(0, 1)

Every tensor is rounded once to bf16 (round-to-nearest-even) and returned both
as float32 (bf16-exact values) and as the uint16 bit pattern.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np


# --------------------------------------------------------------------------- #
# bf16 helpers (storage format only)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 -> bf16 bit pattern (uint16), round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounding = ((u >> 16) & 1) + 0x7FFF
    return ((u + rounding) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# --------------------------------------------------------------------------- #
# configuration
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    num_heads: int
    head_dim: int
    grid_h: int
    grid_w: int
    frames_per_chunk: int
    clusters: int
    sigma: float
    resample: float
    shift: float
    prompt_tokens: int
    relevant: int
    capacity: int            # TempCache capacity in tokens
    block: int               # Bq = Bk = page size
    keep_blocks: int         # AnnSA key blocks kept per query block
    keep_prompt: int         # AnnCA prompt tokens kept per frame
    prior_chunks: int        # chunks already in the cache before the timed step
    lsh_tables: int = 4
    lsh_bits: int = 8
    tau: float = 0.9
    seed: int = 20260201

    @property
    def frame_len(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def chunk_tokens(self) -> int:
        return self.frames_per_chunk * self.frame_len


CONFIGS: Dict[str, WorkloadConfig] = {
    # tiny single-head step; 4 past frames (1024 keys) + 1 new frame; 20 blocks of 64
    "c0": WorkloadConfig("c0", 1, 64, 16, 16, 1, 32, 0.1, 0.10, 1.0, 32, 4,
                         capacity=1280, block=64, keep_blocks=4, keep_prompt=8,
                         prior_chunks=4),
    # one DiT layer shaped like a Wan2.1-1.3B autoregressive backbone
    "c1": WorkloadConfig("c1", 12, 128, 30, 52, 3, 256, 0.1, 0.10, 1.0, 512, 16,
                         capacity=32768, block=128, keep_blocks=32, keep_prompt=64,
                         prior_chunks=6),
    # long rollout on the c1 layer (120 chunks, slower drift)
    "c2": WorkloadConfig("c2", 12, 128, 30, 52, 3, 256, 0.05, 0.05, 0.5, 512, 16,
                         capacity=32768, block=128, keep_blocks=32, keep_prompt=64,
                         prior_chunks=0),
    # world-model-scale layer
    "c3": WorkloadConfig("c3", 40, 128, 45, 80, 3, 512, 0.1, 0.10, 1.0, 512, 16,
                         capacity=65536, block=128, keep_blocks=32, keep_prompt=32,
                         prior_chunks=6),
}


def sweep_config(cache_len: int, head_dim: int, keep_den: int) -> WorkloadConfig:
    """One point of the roofline sweep: 8 heads, 4096 queries (one 64x64 frame),
    cache of `cache_len` keys, keep 1/keep_den of the key blocks."""
    block = 128
    cap = cache_len + 4096
    nkb = cache_len // block
    return WorkloadConfig(f"c4_L{cache_len}_d{head_dim}_f{keep_den}", 8, head_dim, 64, 64, 1,
                          256, 0.1, 0.10, 1.0, 512, 16, capacity=cap, block=block,
                          keep_blocks=max(1, nkb // keep_den), keep_prompt=64,
                          prior_chunks=cache_len // 4096)


def small_config(**kw) -> WorkloadConfig:
    """A scaled-down multi-head case for tests: spans several 128-tiles and has
    ragged tails, yet the oracle finishes in seconds."""
    base = WorkloadConfig("small", 2, 128, 12, 25, 2, 24, 0.1, 0.10, 1.0, 80, 6,
                          capacity=2048, block=128, keep_blocks=4, keep_prompt=24,
                          prior_chunks=2)
    return replace(base, **kw)


# --------------------------------------------------------------------------- #
# generator
# --------------------------------------------------------------------------- #
def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=np.random.SeedSequence([seed, *stream]).generate_state(2, np.uint64)))


@dataclass
class Workload:
    cfg: WorkloadConfig
    centroids: np.ndarray = field(init=False)      # [H][C][d] float32
    map0: np.ndarray = field(init=False)           # [gh][gw] int32

    def __post_init__(self):
        c = self.cfg
        self.centroids = _rng(c.seed, 1).standard_normal((c.num_heads, c.clusters, c.head_dim)).astype(np.float32)
        r = _rng(c.seed, 2)
        pts = np.stack([r.uniform(0, c.grid_h, c.clusters), r.uniform(0, c.grid_w, c.clusters)], axis=1)
        yy, xx = np.meshgrid(np.arange(c.grid_h) + 0.5, np.arange(c.grid_w) + 0.5, indexing="ij")
        dy = np.abs(yy[..., None] - pts[:, 0])
        dx = np.abs(xx[..., None] - pts[:, 1])
        dy = np.minimum(dy, c.grid_h - dy)
        dx = np.minimum(dx, c.grid_w - dx)
        self.map0 = np.argmin(dy * dy + dx * dx, axis=-1).astype(np.int32)

    # -- per-frame pieces ---------------------------------------------------- #
    def cluster_map(self, t: int) -> np.ndarray:
        """Cluster index of every token of frame t, flattened row-major."""
        c = self.cfg
        s = int(np.floor(c.shift * t))
        x = (np.arange(c.grid_w) - s) % c.grid_w
        return self.map0[:, x].reshape(-1)

    def frame(self, t: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(Q, K, V) of frame t, each [H][frame_len][d] float32 holding bf16-exact values."""
        c = self.cfg
        n, H, d = c.frame_len, c.num_heads, c.head_dim
        m = self.cluster_map(t)
        r = _rng(c.seed, 3, t)
        base = self.centroids[:, m, :]                                   # [H][n][d]
        k = base + c.sigma * r.standard_normal((H, n, d)).astype(np.float32)
        q = base + c.sigma * r.standard_normal((H, n, d)).astype(np.float32)
        v = r.standard_normal((H, n, d)).astype(np.float32)
        n_res = int(round(c.resample * n))
        if n_res > 0:
            for h in range(H):
                idx = r.choice(n, size=n_res, replace=False)
                fresh = r.standard_normal((n_res, d)).astype(np.float32)
                k[h, idx] = fresh
                q[h, idx] = fresh + c.sigma * r.standard_normal((n_res, d)).astype(np.float32)
        return round_bf16(q), round_bf16(k), round_bf16(v)

    def chunk(self, ci: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(Q, K, V) of chunk ci = frames [ci*F, (ci+1)*F), each [H][F*frame_len][d]."""
        F = self.cfg.frames_per_chunk
        parts = [self.frame(ci * F + f) for f in range(F)]
        return tuple(np.concatenate([p[i] for p in parts], axis=1) for i in range(3))

    def prompt(self, ci: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(K_p, V_p, planted) for chunk ci.  K_p, V_p: [H][np][d]; planted:
        [F][relevant] prompt positions made relevant to frame f of the chunk.
        The random part of the prompt is the same for every chunk."""
        c = self.cfg
        H, d, P, F = c.num_heads, c.head_dim, c.prompt_tokens, c.frames_per_chunk
        r0 = _rng(c.seed, 4)
        kp = r0.standard_normal((H, P, d)).astype(np.float32)
        vp = r0.standard_normal((H, P, d)).astype(np.float32)
        r = _rng(c.seed, 5, ci)
        pos = r.choice(P, size=F * c.relevant, replace=False).reshape(F, c.relevant)
        for f in range(F):
            m = self.cluster_map(ci * F + f)
            top = np.argsort(-np.bincount(m, minlength=c.clusters), kind="stable")[: c.relevant]
            for s, z in enumerate(top):
                cz = self.centroids[:, z, :]                              # [H][d]
                u = r.standard_normal((H, d)).astype(np.float32)
                u -= (np.sum(u * cz, axis=1, keepdims=True) / np.sum(cz * cz, axis=1, keepdims=True)) * cz
                u /= np.linalg.norm(u, axis=1, keepdims=True)
                kp[:, pos[f, s], :] = 0.8 * cz + 0.6 * np.linalg.norm(cz, axis=1, keepdims=True) * u
        return round_bf16(kp), round_bf16(vp), pos

    def lsh_projection(self) -> np.ndarray:
        """R[T*b][d] float32 (bf16-exact): row t*b+u is the u-th direction of table t."""
        c = self.cfg
        r = _rng(c.seed, 6)
        return round_bf16(r.standard_normal((c.lsh_tables * c.lsh_bits, c.head_dim)).astype(np.float32))

    def counts(self, n_slots: int, max_count: int, stream: int = 0) -> np.ndarray:
        """Multiplicities in {1..max_count} for an imported cache ([H][n_slots] int32)."""
        r = _rng(self.cfg.seed, 7, stream)
        return r.integers(1, max_count + 1, size=(self.cfg.num_heads, n_slots)).astype(np.int32)
