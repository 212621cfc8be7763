"""Shared pieces of the GPU parity tests: upload seeded host data, run the library through
its C ABI, bring results back, compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B

DEV = "cuda:0"


def to_dev(x: np.ndarray, bf16: bool, pitch: int | None = None, fill: float = 7.0):
    """Uploads a 2-D float32 array; with `pitch` the rows sit in a wider buffer whose padding
    holds a sentinel (returns (view, whole buffer))."""
    dt = torch.bfloat16 if bf16 else torch.float32
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    if pitch is None:
        d = t.to(DEV).to(dt).contiguous()
        return d, d
    buf = torch.full((x.shape[0] + 2, pitch), fill, dtype=dt, device=DEV)
    view = buf[1:1 + x.shape[0], : x.shape[1]]
    view.copy_(t.to(DEV).to(dt))
    return view, buf


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def bf16_ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Distance in bf16 steps between two arrays of bf16-representable float32 values."""
    def key(x):
        u = O.f32_to_bf16_bits(x).astype(np.int32)
        return np.where(u & 0x8000, 0x8000 - u, u)   # monotone integer order
    return np.abs(key(a) - key(b))


def f32_ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    def key(x):
        u = np.ascontiguousarray(x, dtype=np.float32).view(np.int32).astype(np.int64)
        return np.where(u < 0, -(u & 0x7FFFFFFF), u)
    return np.abs(key(a) - key(b))


def projector_distance(Va: np.ndarray, Vb: np.ndarray) -> float:
    """|| Va^T Va - Vb^T Vb ||_F for V stored as r rows of length d_in, without forming the
    d_in x d_in projectors: ||Pa - Pb||^2 = ||Va Va^T||^2 + ||Vb Vb^T||^2 - 2 ||Va Vb^T||^2."""
    Va = Va.astype(np.float64)
    Vb = Vb.astype(np.float64)
    a = np.linalg.norm(Va @ Va.T) ** 2
    b = np.linalg.norm(Vb @ Vb.T) ** 2
    c = np.linalg.norm(Va @ Vb.T) ** 2
    return float(np.sqrt(max(a + b - 2 * c, 0.0)))


def cancellation_floor(w_in: np.ndarray, coef: float, seed: int, layer_id: int, V: np.ndarray,
                       rel: float = 2.0 ** -20):
    """Rounding noise of the operands of w + c*(G V^T): rel * max(|w|, |c| |G||V|).
    Where the sum cancels, the result's own ulp is smaller than this noise, so no finite
    precision evaluation can match an exact one to an ulp of the result there.
    rel = 2^-20 for the CUDA-core kernels (fp32 FMA chain over r terms); 2^-16 for the
    tensor-core kernel, whose factors are hi + lo bf16 pairs (each carries 2^-18 of its value
    as residual, two factors per product, one binade of slack)."""
    G = np.abs(O.gen_G(seed, layer_id, w_in.shape[0], V.shape[0]).astype(np.float64))
    A = abs(float(coef)) * (G @ np.abs(V.astype(np.float64)))
    return rel * np.maximum(np.abs(w_in.astype(np.float64)), A)


def tc_mismatch_bound(want: np.ndarray, coef: float, seed: int, layer_id: int, V: np.ndarray) -> float:
    """Share of bf16 results that may land on the neighbouring grid point under the tensor-core
    kernel.  Its factors are hi + lo bf16 pairs, so c*z carries an absolute error up to
    e_ij = 2^-17 |c| (|G||V|)_ij (2^-18 of each factor, two factors); a result within e_ij of a
    rounding boundary can round the other way, which has probability 2 e_ij / ulp(w'_ij).
    The bound is the mean of that over the matrix (never below the 1e-3 of the other kernels)."""
    G = np.abs(O.gen_G(seed, layer_id, want.shape[0], V.shape[0]).astype(np.float64))
    e = 2.0 ** -17 * abs(float(coef)) * (G @ np.abs(V.astype(np.float64)))
    mag = np.maximum(np.abs(want.astype(np.float64)), 2.0 ** -126)
    ulp = 2.0 ** (np.floor(np.log2(mag)) - 7)
    return max(1e-3, float(np.minimum(1.0, 2.0 * e / ulp).mean()))


def assert_weights_match(got: np.ndarray, want: np.ndarray, storage: str, frac: float = 1e-3,
                         floor=None):
    """<= 1 bf16 ulp everywhere with at most `frac` of the elements differing (fp32 storage:
    <= 4 fp32 ulp, no bound on how many differ in the last bits); an element
    whose absolute difference is within `floor` (see cancellation_floor) counts as equal."""
    d = bf16_ulp_distance(got, want) if storage == "bf16" else f32_ulp_distance(got, want)
    if floor is not None:
        d = np.where(np.abs(got.astype(np.float64) - want) <= floor, np.minimum(d, 1), d)
    lim = 1 if storage == "bf16" else 4
    assert d.max() <= lim, f"max ulp distance {d.max()} ({storage})"
    if storage == "bf16":   # an fp32 result legitimately differs in its last bit often
        assert (d > 0).mean() <= frac, f"mismatching fraction {(d > 0).mean()}"


class Ctx:
    """Context sized for a layer list, destroyed on exit."""

    def __init__(self, layers, extra=0):
        self.ctx = B.agzo_create(layers, 0, extra)

    def __enter__(self):
        return self.ctx

    def __exit__(self, *a):
        torch.cuda.synchronize()
        B.agzo_destroy(self.ctx)
