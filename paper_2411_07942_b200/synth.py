"""Seeded synthetic activations shaped like the paper's workloads.

The paper calibrates on WikiText sequences and evaluates real LLM activations
(Section 3, Section 4); neither is available offline, so BF16 partial sums with
the structure the paper describes -- a few feature columns whose range is
consistently enormous (Section 1, Figure 1) -- stand in for them.

This module holds input generation ONLY: no step of the codec is computed here.
The same BF16 bit patterns are handed to the CUDA library and to the CPU oracle
(generated once, then uploaded or downloaded), never regenerated per side.

Recipe, for every config:
    sigma_j = exp(sd * n_j),  n_j ~ N(0, 1) per feature, shared by all shards
    O       = outlier columns, c_j their multiplier (1 elsewhere)
    Y^(i)[t, j] = bf16_rne(sigma_j * c_j * z),  z ~ N(0, 1) i.i.d.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    n_shards: int          # N tensor-parallel devices (simulated as N buffers)
    tokens: int            # T rows of one synchronisation
    features: int          # E
    sd: float              # sd of log sigma_j
    n_outliers: int        # |O|
    outlier_lo: float      # c_j drawn log-uniformly in [lo, hi] (lo == hi: constant)
    outlier_hi: float
    calib_seqs: int        # sequences per shard in the calibration set
    calib_tokens: int      # S tokens per calibration sequence
    seed: int
    fixed_outliers: tuple = field(default=())   # explicit outlier columns, if fixed

    @property
    def k(self) -> int:
        return self.features // 64


WORKLOADS = {
    # BASELINE config 1: "Tiny", seed 0, 4 fixed outlier columns scaled x50, 64 calibration tokens
    "tiny": Workload("tiny", 2, 16, 256, 0.5, 4, 50.0, 50.0, 4, 16, 0,
                     fixed_outliers=(17, 64, 131, 250)),
    # config 2: Llama-2-13B-shaped prefill
    "llama13b_prefill": Workload("llama13b_prefill", 4, 2048, 5120, 0.7, 51, 20.0, 200.0, 128, 2048, 2000),
    # config 3: Gemma-2-27B-shaped decode
    "gemma27b_decode": Workload("gemma27b_decode", 8, 64, 4608, 0.7, 46, 20.0, 200.0, 32, 512, 3000),
    # config 4: calibration pass (N = the paper's TP degree)
    "calibration": Workload("calibration", 8, 2048, 4608, 0.7, 46, 20.0, 200.0, 512, 2048, 4000),
    # config 5: large sweep
    "large": Workload("large", 16, 8192, 8192, 0.7, 41, 100.0, 1000.0, 16, 1024, 5000),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> BF16 bit patterns (round to nearest even); input generation only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def column_scales(w: Workload) -> np.ndarray:
    """sigma_j * c_j for every feature (float32), and nothing else."""
    rng = np.random.Generator(np.random.Philox(w.seed))
    sigma = np.exp(w.sd * rng.standard_normal(w.features)).astype(np.float32)
    if w.fixed_outliers:
        cols = np.array(w.fixed_outliers, dtype=np.int64)
    else:
        cols = rng.permutation(w.features)[: w.n_outliers]
    if w.outlier_lo == w.outlier_hi:
        mult = np.full(len(cols), w.outlier_lo, dtype=np.float32)
    else:
        lo, hi = np.log(w.outlier_lo), np.log(w.outlier_hi)
        mult = np.exp(rng.uniform(lo, hi, size=len(cols))).astype(np.float32)
    scale = sigma.copy()
    scale[cols] *= mult
    return scale


def outlier_columns(w: Workload) -> np.ndarray:
    if w.fixed_outliers:
        return np.array(sorted(w.fixed_outliers), dtype=np.int64)
    rng = np.random.Generator(np.random.Philox(w.seed))
    rng.standard_normal(w.features)
    return np.sort(rng.permutation(w.features)[: w.n_outliers])


def activations_np(w: Workload, shard: int, rows: int, stream: int = 0, scale=None) -> np.ndarray:
    """[rows, E] BF16 bit patterns (uint16) for one shard, generated on the host.

    ``stream`` separates independent draws (0 = the inference batch, 1 + q =
    calibration sequence q)."""
    scale = column_scales(w) if scale is None else scale
    rng = np.random.Generator(np.random.Philox(key=w.seed + 1 + shard + 1000 * (stream + 1)))
    z = rng.standard_normal((rows, w.features), dtype=np.float32)
    return f32_to_bf16_bits(z * scale[None, :])


def calibration_np(w: Workload, shard: int, n_seq: int | None = None, tokens: int | None = None,
                   scale=None) -> np.ndarray:
    """[n_seq, S, E] BF16 bit patterns of one shard's calibration sequences."""
    n_seq = w.calib_seqs if n_seq is None else n_seq
    tokens = w.calib_tokens if tokens is None else tokens
    scale = column_scales(w) if scale is None else scale
    return np.stack([activations_np(w, shard, tokens, stream=1 + q, scale=scale) for q in range(n_seq)])


def activations_torch(w: Workload, shard: int, rows: int, device, stream: int = 0, scale=None):
    """[rows, E] torch.bfloat16 on ``device`` from a seeded device generator.

    Used where the host generator would be too slow (full-size benchmark
    buffers); the oracle then receives a download of exactly these bits."""
    import torch

    scale = column_scales(w) if scale is None else scale
    g = torch.Generator(device=device)
    g.manual_seed(w.seed + 1 + shard + 1000 * (stream + 1))
    sc = torch.from_numpy(scale).to(device)
    out = torch.empty((rows, w.features), dtype=torch.bfloat16, device=device)
    step = max(1, (1 << 26) // w.features)        # bound the float32 temporary
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        z = torch.randn((r1 - r0, w.features), generator=g, device=device, dtype=torch.float32)
        out[r0:r1] = (z * sc).to(torch.bfloat16)
    return out
