"""Seeded synthetic inputs for ARMOR's per-layer optimisation.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic.  Both the CUDA path's tests/benchmark and the CPU oracle's
tests take their inputs from here, so the two sides see identical data.

Recipe (one layer):
  * weight      W[i][j] = sigma * g,           g ~ N(0,1)
  * activations X[t][c] = s_c * g_tc,          g ~ N(0,1) or Laplace(0,1)
  * channel scale s_c = exp(N(0,1)) is the per-channel standard deviation;
    the first ``n_outlier`` channels of a seeded permutation are multiplied by
    ``outlier_scale`` (heavy "outlier channels" as seen in LLM activations).
X is produced in token chunks whose random stream depends only on
(seed, chunk index, chunk_rows), so a large calibration set never has to exist
in one piece and any chunk can be regenerated on its own.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Iterator

import numpy as np
import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    d_out: int
    d_in: int
    d_block: int
    n_tokens: int
    n_iters: int
    seed: int
    sigma: float = 0.02
    n_outlier: int = 4
    outlier_scale: float = 50.0
    laplace: bool = False
    n_keep: int = 2
    m_group: int = 4
    chunk_rows: int = 8192

    def with_(self, **kw) -> "LayerConfig":
        return replace(self, **kw)


def _k_out(d_in: int) -> int:
    return max(1, round(0.001 * d_in))


# The benchmark's workloads.  Index 0 is the small case the CPU oracle finishes
# in seconds; index 1 is the one the headline metric is quoted on.
CONFIGS = {
    "tiny": LayerConfig("tiny", 256, 256, 32, 4096, 20, seed=0, n_outlier=4,
                        outlier_scale=20.0, chunk_rows=1024),
    "llama7b_attn": LayerConfig("llama7b_attn", 4096, 4096, 128, 262144, 50, seed=2,
                                n_outlier=_k_out(4096)),
    "llama8b_up": LayerConfig("llama8b_up", 14336, 4096, 128, 262144, 50, seed=3,
                              n_outlier=_k_out(4096)),
    "llama8b_down": LayerConfig("llama8b_down", 4096, 14336, 128, 262144, 50, seed=3,
                                n_outlier=_k_out(14336), laplace=True),
    "qwen_q": LayerConfig("qwen_q", 5120, 5120, 128, 262144, 50, seed=4,
                          n_outlier=_k_out(5120)),
    "qwen_kv": LayerConfig("qwen_kv", 1024, 5120, 128, 262144, 50, seed=4,
                           n_outlier=_k_out(5120)),
    "mlp70b_up": LayerConfig("mlp70b_up", 28672, 8192, 256, 131072, 30, seed=5,
                             sigma=0.015, n_outlier=_k_out(8192)),
    "mlp70b_down": LayerConfig("mlp70b_down", 8192, 28672, 256, 131072, 30, seed=5,
                               sigma=0.015, n_outlier=_k_out(28672), laplace=True),
}


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 1_000_003 + int(stream) * 7919 + 12345) % (2**63 - 1))
    return g


def make_weight(cfg: LayerConfig) -> np.ndarray:
    """W [d_out, d_in] fp32, iid N(0, sigma^2)."""
    w = torch.randn(cfg.d_out, cfg.d_in, generator=_gen(cfg.seed, 1), dtype=torch.float32)
    return (w * cfg.sigma).numpy()


def channel_scales(cfg: LayerConfig) -> np.ndarray:
    """Per-channel standard deviation s_c [d_in] fp32 (log-normal, with outlier channels)."""
    g = _gen(cfg.seed, 2)
    s = torch.exp(torch.randn(cfg.d_in, generator=g, dtype=torch.float32))
    perm = torch.randperm(cfg.d_in, generator=g)
    s[perm[: cfg.n_outlier]] *= cfg.outlier_scale
    return s.numpy()


def n_chunks(cfg: LayerConfig) -> int:
    return (cfg.n_tokens + cfg.chunk_rows - 1) // cfg.chunk_rows


def activation_chunk(cfg: LayerConfig, index: int, scales: torch.Tensor | None = None,
                     out: torch.Tensor | None = None) -> torch.Tensor:
    """Chunk ``index`` of X: rows [index*chunk_rows, ...) as a CPU fp32 tensor."""
    lo = index * cfg.chunk_rows
    rows = min(cfg.chunk_rows, cfg.n_tokens - lo)
    if rows <= 0:
        raise IndexError("chunk index past the end of the calibration set")
    if scales is None:
        scales = torch.from_numpy(channel_scales(cfg))
    g = _gen(cfg.seed, 1000 + index)
    if out is None:
        out = torch.empty(rows, cfg.d_in, dtype=torch.float32)
    else:
        out = out[:rows]
    if cfg.laplace:
        u = torch.rand(rows, cfg.d_in, generator=g, dtype=torch.float32) - 0.5
        # inverse-CDF draw of Laplace(0, 1); clamp keeps log() finite at u = -0.5
        out.copy_(-torch.sign(u) * torch.log1p((-2.0 * u.abs()).clamp_(min=-1.0 + 1e-7)))
    else:
        torch.randn(rows, cfg.d_in, generator=g, dtype=torch.float32, out=out)
    out.mul_(scales)
    return out


def activation_chunks(cfg: LayerConfig) -> Iterator[torch.Tensor]:
    scales = torch.from_numpy(channel_scales(cfg))
    for i in range(n_chunks(cfg)):
        yield activation_chunk(cfg, i, scales)


def make_activations(cfg: LayerConfig) -> np.ndarray:
    """Whole X [n_tokens, d_in] fp32 (use only where it fits in host memory)."""
    out = torch.empty(cfg.n_tokens, cfg.d_in, dtype=torch.float32)
    scales = torch.from_numpy(channel_scales(cfg))
    for i in range(n_chunks(cfg)):
        lo = i * cfg.chunk_rows
        activation_chunk(cfg, i, scales, out=out[lo: lo + cfg.chunk_rows])
    return out.numpy()


def make_tokens(cfg: LayerConfig, n: int, stream: int = 77) -> np.ndarray:
    """A batch x [n, d_in] fp32 of inference-time activations (same distribution as X)."""
    scales = torch.from_numpy(channel_scales(cfg))
    x = torch.randn(n, cfg.d_in, generator=_gen(cfg.seed, stream), dtype=torch.float32)
    return (x * scales).numpy()


def coupled_blocks(nb: int, d_block: int, strength: float) -> np.ndarray:
    """Wrapper blocks [nb, d_block, d_block] fp64 whose columns are nearly parallel: the identity plus
    ``strength / sqrt(d_block)`` in every entry.  Test input for states in which the updates of different
    groups of one row-block overlap strongly."""
    eye = np.eye(d_block, dtype=np.float64)
    return np.broadcast_to(eye + strength / np.sqrt(d_block), (nb, d_block, d_block)).copy()
