"""Seeded synthetic inputs for the sink+window attention path.

This module only draws random numbers and rounds them to bfloat16 storage.  It
holds none of the method's arithmetic (no RoPE, no slot rule, no softmax), so
both the CUDA path's tests and the CPU oracle's tests may read inputs from it
and see identical bytes.

All tensors are bfloat16 *bit patterns* held in ``numpy.uint16`` arrays with the
token-major layout ``[tokens, heads, head_dim]`` that a QKV projection emits.
They stand in for the Q/K/V activations of a Wan2.1-1.3B-shaped DiT layer; the
real activations need trained weights and prompt suites that are not available
offline.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    """Shape of one stream: the seven cache integers plus grid and schedule."""

    name: str
    layers: int
    heads: int
    head_dim: int
    grid_h: int
    grid_w: int
    chunk_frames: int
    sink_frames: int
    window_frames: int
    n_chunks: int
    seed: int
    steps_per_chunk: int = 1      # denoising passes before the commit pass
    outlier_frac: float = 0.0     # fraction of entries multiplied by outlier_scale
    outlier_scale: float = 20.0
    rope_theta: float = 10000.0

    @property
    def tokens_per_frame(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def chunk_tokens(self) -> int:
        return self.chunk_frames * self.tokens_per_frame

    @property
    def cache_args(self):
        return (self.layers, self.heads, self.head_dim, self.tokens_per_frame,
                self.chunk_frames, self.sink_frames, self.window_frames)


# The five workloads of the benchmark definition (index = config number).
CONFIGS = [
    Workload("tiny", 1, 2, 64, 4, 4, 1, 1, 2, n_chunks=8, seed=0),
    Workload("wan1.3b_layer", 1, 12, 128, 30, 52, 3, 3, 9, n_chunks=24, seed=1),
    Workload("full_stack_decode", 30, 12, 128, 30, 52, 3, 3, 9, n_chunks=7, seed=2,
             steps_per_chunk=4),
    Workload("long_stream", 30, 12, 128, 30, 52, 3, 3, 9, n_chunks=320, seed=3,
             steps_per_chunk=4),
    Workload("batched_sweep", 1, 12, 128, 30, 52, 3, 3, 9, n_chunks=51, seed=4,
             outlier_frac=0.01),
]
# Config 2's equivalence reference: sink 3 + window 18 covers all 21 frames.
FULL_CAUSAL = replace(CONFIGS[2], name="full_stack_full_causal", window_frames=18)
# Config 3: a prompt switch (recache) before every 40th chunk.
LONG_STREAM_SWITCH_EVERY = 40
# Config 4: stream positions (chunks already generated) and the window sweep.
SWEEP_POSITIONS = (0, 1, 2, 3, 6, 13, 29, 50)
SWEEP_WINDOWS = (3, 6, 9, 18)
RECACHE_PASS = 7  # pass id used to seed recache tensors


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float64."""
    return bf16_bits_to_f32(b).astype(np.float64)


def normal_bf16(rng: np.random.Generator, shape, outlier_frac: float = 0.0,
                outlier_scale: float = 20.0) -> np.ndarray:
    """N(0,1) in float32, optional sparse outliers, rounded to bf16 bits."""
    x = rng.standard_normal(shape, dtype=np.float32)
    if outlier_frac > 0.0:
        mask = rng.random(shape, dtype=np.float32) < outlier_frac
        x = np.where(mask, x * np.float32(outlier_scale), x)
    return f32_to_bf16_bits(x)


def call_rng(seed: int, chunk: int, layer: int = 0, pass_id: int = 0,
             stream: int = 0) -> np.random.Generator:
    """One generator per (seed, stream, chunk, layer, pass) so calls are random-access."""
    return np.random.default_rng([seed, stream, chunk, layer, pass_id])


def chunk_qkv(wl: Workload, chunk: int, layer: int = 0, pass_id: int = 0,
              stream: int = 0, n_frames: int | None = None):
    """Q, K, V (bf16 bits, [tokens, H, D]) for one call.

    ``n_frames`` defaults to the chunk size; recache calls pass the number of
    ring-resident frames instead.
    """
    nf = wl.chunk_frames if n_frames is None else n_frames
    shape = (nf * wl.tokens_per_frame, wl.heads, wl.head_dim)
    rng = call_rng(wl.seed, chunk, layer, pass_id, stream)
    q = normal_bf16(rng, shape, wl.outlier_frac, wl.outlier_scale)
    k = normal_bf16(rng, shape, wl.outlier_frac, wl.outlier_scale)
    v = normal_bf16(rng, shape, wl.outlier_frac, wl.outlier_scale)
    return q, k, v


def sample_rows(n_rows: int, n_samples: int, tile: int = 128, seed: int = 0, edges: bool = True) -> np.ndarray:
    """Query rows to check at sizes where the oracle cannot do every row.

    With ``edges`` (the default) the result always holds the first and the last
    row of every ``tile``-row tile, the ragged last tile's ends included, however
    small ``n_samples`` is; random rows then fill it up to ``n_samples``.  With
    ``edges=False`` it is ``n_samples`` random rows plus the first and last one
    (for timing samples, where the count matters and the placement does not).
    """
    must = {0, n_rows - 1}
    if edges:
        for t0 in range(0, n_rows, tile):
            must.update((t0, min(t0 + tile, n_rows) - 1))
    rng = np.random.default_rng([seed, n_rows, n_samples])
    rest = n_samples - len(must)
    while rest > 0:
        must.update(int(r) for r in rng.integers(0, n_rows, size=rest))
        rest = min(n_samples, n_rows) - len(must)
    return np.asarray(sorted(must), dtype=np.int64)


class InputPool:
    """A few pre-drawn (q, k, v) chunk sets that long schedules index into.

    The full-stack and long-stream workloads make tens of thousands of calls;
    drawing fresh tensors for each would take hours on the host.  Call
    (chunk, layer, pass, stream) uses set ``index(...)`` of the pool, so any call's
    inputs can be regenerated on their own (the oracle replays only sampled calls).
    """

    def __init__(self, wl: Workload, n_sets: int = 6, n_frames: int | None = None,
                 pass_id: int = 0):
        self.wl = wl
        self.n_sets = n_sets
        self.sets = [chunk_qkv(wl, 1000 + i, pass_id=pass_id, n_frames=n_frames) for i in range(n_sets)]

    def index(self, chunk: int, layer: int = 0, pass_id: int = 0, stream: int = 0) -> int:
        return (chunk * 7 + layer * 3 + pass_id * 5 + stream * 11) % self.n_sets

    def get(self, chunk: int, layer: int = 0, pass_id: int = 0, stream: int = 0):
        return self.sets[self.index(chunk, layer, pass_id, stream)]
