"""Seeded synthetic inputs for the AGZO hot path: shapes and value recipes only.

This module holds none of the method's arithmetic.  It produces the tensors that both the
CUDA library and the CPU checker are fed with (host generators, numpy, bit-reproducible
from the seed) and the full-size resident layer sets the benchmark times (device
generators, torch, same distributions).

The paper fine-tunes Qwen3 / Pangu checkpoints on SuperGLUE-style tasks; neither the
checkpoints nor the datasets are used here.  The stand-ins keep what the hot path is
sensitive to: the layer shapes of a Qwen3 block, the weight scale, the token count, and
an activation matrix whose spectrum has a dominant low-rank part (Section 3.2 reports
rapidly decaying activation spectra).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np
import torch

# (name, d_in, d_out) of the seven linear layers of one Qwen3 block
def _block(hidden, q_out, kv_out, inter):
    return [("q", hidden, q_out), ("k", hidden, kv_out), ("v", hidden, kv_out),
            ("o", q_out, hidden), ("gate", hidden, inter), ("up", hidden, inter),
            ("down", inter, hidden)]


@dataclass(frozen=True)
class LayerSetConfig:
    name: str
    n_blocks: int
    block: Tuple[Tuple[str, int, int], ...]
    m: int                 # tokens per activation matrix
    planted_rank: int      # rank of the dominant activation component
    ranks: Tuple[int, ...]
    w_std: float = 0.02

    def layers(self) -> List[Tuple[str, int, int]]:
        out = []
        for b in range(self.n_blocks):
            for (nm, di, do) in self.block:
                out.append((f"{b}.{nm}", di, do))
        return out

    def n_params(self) -> int:
        return self.n_blocks * sum(di * do for (_, di, do) in self.block)

    def x_elems(self) -> int:
        return self.n_blocks * sum(self.m * di for (_, di, _) in self.block)


QWEN3_0P6B = LayerSetConfig("qwen3-0.6b-shapes", 28, tuple(_block(1024, 2048, 1024, 3072)),
                            m=16 * 512, planted_rank=32, ranks=(8,))
QWEN3_1P7B = LayerSetConfig("qwen3-1.7b-shapes", 28, tuple(_block(2048, 2048, 1024, 6144)),
                            m=16 * 1024, planted_rank=64, ranks=(4, 8, 16))
QWEN3_8B = LayerSetConfig("qwen3-8b-shapes", 36, tuple(_block(4096, 4096, 1024, 12288)),
                          m=8 * 2048, planted_rank=64, ranks=(1, 4, 16, 64))
LAYER_SETS = {c.name: c for c in (QWEN3_0P6B, QWEN3_1P7B, QWEN3_8B)}


# ------------------------------------------------------------------ host generators (numpy)
def to_bf16_values(x: np.ndarray) -> np.ndarray:
    """float32 array rounded onto the bf16 grid (torch's cast), kept as float32."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def gaussian_weights(d_out: int, d_in: int, std: float, seed: int, bf16: bool) -> np.ndarray:
    rng = np.random.default_rng([seed, 0x57])
    w = (rng.standard_normal((d_out, d_in)) * std).astype(np.float32)
    return to_bf16_values(w) if bf16 else w


def planted_activations(m: int, d_in: int, p: int, seed: int, bf16: bool) -> np.ndarray:
    """x_t = n_t + sqrt(10) B c_t with n_t ~ N(0, I), c_t ~ N(0, I_p), B d_in x p orthonormal:
    covariance I + 10 B B^T ("a planted rank-p component of 10x variance")."""
    rng = np.random.default_rng([seed, 0x58])
    x = rng.standard_normal((m, d_in))
    if p > 0:
        B, _ = np.linalg.qr(rng.standard_normal((d_in, p)))
        x += np.sqrt(10.0) * (rng.standard_normal((m, p)) @ B.T)
    x = x.astype(np.float32)
    return to_bf16_values(x) if bf16 else x


def graded_activations(m: int, d_in: int, n_dirs: int, seed: int, bf16: bool, ratio: float = 2.0 ** -0.5,
                       floor: float = 0.0) -> np.ndarray:
    """Activations with a geometric spectrum: singular values sigma_k = sigma_0 * ratio^k over the first
    n_dirs directions (random orthonormal singular vectors on both sides), entries of order one, plus
    an optional isotropic noise floor of standard deviation `floor` per entry.  Stands in for the
    rapidly decaying activation spectra of Section 3.2."""
    rng = np.random.default_rng([seed, 0x5C])
    U, _ = np.linalg.qr(rng.standard_normal((m, n_dirs)))
    W, _ = np.linalg.qr(rng.standard_normal((d_in, n_dirs)))
    s = ratio ** np.arange(n_dirs)
    s = s * np.sqrt(m * d_in / np.sum(s * s))          # rms entry = 1
    x = (U * s) @ W.T
    if floor > 0.0:
        x = x + floor * rng.standard_normal((m, d_in))
    x = x.astype(np.float32)
    return to_bf16_values(x) if bf16 else x


def massive_activations(m: int, d_in: int, seed: int, bf16: bool, factor: float = 100.0,
                        channel: int = 7, token: int = 11) -> np.ndarray:
    """N(0,1) activations in which one channel (column) and one token (row) are `factor` times
    larger than the rest: the outlier features and sink tokens of language models."""
    rng = np.random.default_rng([seed, 0x5D])
    x = rng.standard_normal((m, d_in))
    x[:, channel % d_in] *= factor
    x[token % m, :] *= factor
    x = x.astype(np.float32)
    return to_bf16_values(x) if bf16 else x


def plain_activations(m: int, d_in: int, seed: int, bf16: bool = False) -> np.ndarray:
    rng = np.random.default_rng([seed, 0x59])
    x = rng.standard_normal((m, d_in)).astype(np.float32)
    return to_bf16_values(x) if bf16 else x


def least_squares_problem(seed: int = 0, d_in: int = 256, d_out: int = 256, m: int = 512):
    """Single fp32 linear layer: X ~ N(0,1), Y = X W*^T + 0.01 N(0,1), W* ~ N(0, 1/d_in),
    start W0 ~ N(0, 1/d_in) from an independent stream."""
    rng = np.random.default_rng([seed, 0x5A])
    X = rng.standard_normal((m, d_in)).astype(np.float32)
    Wstar = (rng.standard_normal((d_out, d_in)) / np.sqrt(d_in)).astype(np.float32)
    Y = (X.astype(np.float64) @ Wstar.astype(np.float64).T
         + 0.01 * rng.standard_normal((m, d_out))).astype(np.float32)
    W0 = (rng.standard_normal((d_out, d_in)) / np.sqrt(d_in)).astype(np.float32)
    return X, Y, W0


def mlp_problem(seed: int = 0, n_layers: int = 8, width: int = 1024, m: int = 16 * 256):
    """8-layer MLP stack: weights ~ N(0, 1/width), inputs N(0,1), fixed random target."""
    rng = np.random.default_rng([seed, 0x5B])
    Ws = [(rng.standard_normal((width, width)) / np.sqrt(width)).astype(np.float32)
          for _ in range(n_layers)]
    x0 = rng.standard_normal((m, width)).astype(np.float32)
    target = rng.standard_normal((m, width)).astype(np.float32)
    return Ws, x0, target


# ------------------------------------------------------------------ device generators (torch)
def device_weights(d_out: int, d_in: int, std: float, gen: torch.Generator, device) -> torch.Tensor:
    w = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=device)
    w.normal_(0.0, std, generator=gen)
    return w


def device_planted_activations(m: int, d_in: int, p: int, gen: torch.Generator, device,
                               chunk: int = 4096) -> torch.Tensor:
    """Same recipe as planted_activations, sampled by torch on the device in token chunks."""
    x = torch.empty((m, d_in), dtype=torch.bfloat16, device=device)
    B = torch.linalg.qr(torch.randn((d_in, p), generator=gen, device=device,
                                    dtype=torch.float32)).Q if p > 0 else None
    for t0 in range(0, m, chunk):
        t1 = min(m, t0 + chunk)
        blk = torch.randn((t1 - t0, d_in), generator=gen, device=device, dtype=torch.float32)
        if B is not None:
            c = torch.randn((t1 - t0, p), generator=gen, device=device, dtype=torch.float32)
            blk.addmm_(c, B.t(), alpha=float(np.sqrt(10.0)))
        x[t0:t1] = blk.to(torch.bfloat16)
    return x
