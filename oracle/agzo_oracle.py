"""CPU oracle for the AGZO per-step hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library must compute.  It is
imported by the tests, by the smoke check and by the benchmark's CPU-baseline leg and by
nothing else; the product path never calls it and it shares no code with the CUDA
sources.  Everything is numpy in float64 unless the method itself fixes a precision
(uint32 Philox words, float32 Gaussians, bf16/fp32 weight storage).

Notation follows the paper with the library's letters in brackets:
  H  (d_in x m)  activations, stored here as X = H^T (m x d_in, one token per row)
  A  (d_in x r)  orthonormal basis               [V, stored as r rows of length d_in]
  R  (d_out x r) Gaussian left factor            [G]
  Delta = R A^T  low-rank direction              [Z = G V^T]
  mu, eta, g     smoothing, step size, scalar    [eps, lr, ghat]

Parity status: every function below is pinned by a test that does not go through the
function itself (published Philox known-answer vectors, distribution tests, numpy's QR /
SVD, closed forms for quadratic losses, brute-force gradients, Monte-Carlo against the
closed form of Theorem 4.4).  Nothing in this file is "parity unpinned".
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

# --------------------------------------------------------------------------------------
# Counter-based generator: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
# The paper only says "generate R from seed s_l" (Algorithm 2, step 2); the concrete
# generator and the counter layout are a reading of this build:
#   key     = (seed & 0xffffffff, seed >> 32)            the step seed
#   counter = (b & 0xffffffff, b >> 32, layer_id, tag)   b = e >> 2
# where e is the row-major linear index of the element inside the matrix being drawn
# (R is d_out x r, Omega is m x r) and element e takes output word  e & 3  of block b.
# --------------------------------------------------------------------------------------
PHILOX_M0 = np.uint64(0xD2511F53)
PHILOX_M1 = np.uint64(0xCD9E8D57)
PHILOX_W0 = 0x9E3779B9
PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)

TAG_G = 0        # left factor R_l of Eq. (agzo-perturb)
TAG_OMEGA = 1    # test matrix Omega of Algorithm 1
TAG_DENSE = 2    # dense Gaussian direction for non-matrix parameters (Eq. agzo-perturb, case 2)
TAG_BASIS = 3    # Gaussian right factor V_l of LOZO (Eq. lozo-layer-perturb), for comparison runs


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of Philox-4x32 on arrays of counters; returns four uint32 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK32
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK32
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK32
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK32
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = PHILOX_M0 * c0          # 32x32 -> 64 bit products, exact in uint64
        p1 = PHILOX_M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK32
        hi1, lo1 = p1 >> _SH32, p1 & _MASK32
        n0 = hi1 ^ c1 ^ np.uint64(k0)
        n1 = lo1
        n2 = hi0 ^ c3 ^ np.uint64(k1)
        n3 = lo0
        c0, c1, c2, c3 = n0, n1, n2, n3
        k0 = (k0 + PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + PHILOX_W1) & 0xFFFFFFFF
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def philox_words(seed: int, layer_id: int, tag: int, n: int, first: int = 0) -> np.ndarray:
    """uint32 word of elements first .. first+n-1 of stream (seed, layer_id, tag)."""
    e = np.arange(first, first + n, dtype=np.uint64)
    b = e >> np.uint64(2)
    blocks, inv = np.unique(b, return_inverse=True)
    w = philox4x32_10(blocks & _MASK32, blocks >> _SH32, layer_id, tag,
                      seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    w = np.stack(w, axis=1)                       # (n_blocks, 4)
    return w[inv, (e & np.uint64(3)).astype(np.int64)]


def gaussian_stream(seed: int, layer_id: int, tag: int, n: int) -> np.ndarray:
    """Standard normals, float32, elements 0..n-1 of stream (seed, layer_id, tag).

    Box-Muller on word pairs of one Philox block (x0,x1) and (x2,x3):
      u1 = ((x >> 8) + 1) * 2^-24  in (0, 1],   u2 = (x' >> 8) * 2^-24  in [0, 1)
      s  = sqrt(-2 ln u1);  lane 0 / 2 = s cos(2 pi u2),  lane 1 / 3 = s sin(2 pi u2)
    evaluated in float64 and rounded once to float32.
    """
    nb = (n + 3) // 4
    blocks = np.arange(nb, dtype=np.uint64)
    x0, x1, x2, x3 = philox4x32_10(blocks & _MASK32, blocks >> _SH32, layer_id, tag,
                                   seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    out = np.empty((nb, 4), dtype=np.float64)
    for lane, (xa, xb) in ((0, (x0, x1)), (2, (x2, x3))):
        u1 = ((xa >> np.uint32(8)).astype(np.float64) + 1.0) * 2.0 ** -24
        u2 = (xb >> np.uint32(8)).astype(np.float64) * 2.0 ** -24
        s = np.sqrt(-2.0 * np.log(u1))
        out[:, lane] = s * np.cos(2.0 * np.pi * u2)
        out[:, lane + 1] = s * np.sin(2.0 * np.pi * u2)
    return out.reshape(-1)[:n].astype(np.float32)


def gen_G(seed: int, layer_id: int, d_out: int, r: int) -> np.ndarray:
    """R_l of Eq. (agzo-perturb): d_out x r i.i.d. N(0,1), float32, row-major stream."""
    return gaussian_stream(seed, layer_id, TAG_G, d_out * r).reshape(d_out, r)


def gen_omega(seed: int, layer_id: int, m: int, r: int) -> np.ndarray:
    """Gaussian test matrix Omega of Algorithm 1, m x r, float32."""
    return gaussian_stream(seed, layer_id, TAG_OMEGA, m * r).reshape(m, r)


def gen_gaussian_basis(seed: int, layer_id: int, r: int, d_in: int) -> np.ndarray:
    """V_l^T of Eq. (lozo-layer-perturb): r x d_in i.i.d. N(0,1), float32, row-major stream."""
    return gaussian_stream(seed, layer_id, TAG_BASIS, r * d_in).reshape(r, d_in)


def gen_dense(seed: int, layer_id: int, n: int) -> np.ndarray:
    """Dense direction u_l for a non-matrix parameter (Eq. agzo-perturb, second case)."""
    return gaussian_stream(seed, layer_id, TAG_DENSE, n)


# --------------------------------------------------------------------------------------
# Storage precisions
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    r = np.where(nan, (u >> np.uint32(16)) | np.uint32(0x0040), r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float32 values rounded (RNE) onto the bfloat16 grid, kept as float32."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# --------------------------------------------------------------------------------------
# Algorithm 1: SubspaceExtract(H, r, K)
# --------------------------------------------------------------------------------------
RANK_TOL = 1e-4


def qr_positive(Y: np.ndarray):
    """Thin QR of a d x r panel with R_kk > 0, by modified Gram-Schmidt applied twice.

    The paper writes [Q, ~] = qr(Y) without fixing signs; the low-rank direction R A^T
    depends on the basis and not only on its span, so the unique factorisation with a
    positive diagonal is taken.

    Rank deficiency (Algorithm 1 only assumes r << min(d_out, d_in, m) and says nothing
    about it): column k is dependent on the columns before it when what is left of it after
    they are projected out, R_kk, is at most RANK_TOL times the column's own length
    ||y_k||.  Such a column is returned as zero and reported.  The test is relative to the
    column itself, not to R_11: the columns of Y = H (H^T Q) carry the squared singular
    values of H, and Section 3.2 reports rapidly decaying activation spectra, so a small
    column is the normal case and says nothing about dependence.
    Returns (Q, R, deficient) with Q d x r float64.
    """
    Y = np.asarray(Y, dtype=np.float64)
    d, r = Y.shape
    Q = np.zeros((d, r))
    R = np.zeros((r, r))
    deficient = False
    for j in range(r):
        v = Y[:, j].copy()
        own = np.sqrt(v @ v)
        for _ in range(2):
            for i in range(j):
                c = Q[:, i] @ v
                R[i, j] += c
                v -= c * Q[:, i]
        nrm = np.sqrt(v @ v)
        R[j, j] = nrm
        if nrm <= RANK_TOL * own or nrm == 0.0:
            deficient = True
            continue
        Q[:, j] = v / nrm
    return Q, R, deficient


def extract_subspace(X: np.ndarray, r: int, K: int, seed: int, layer_id: int,
                     return_info: bool = False):
    """Algorithm 1 on H = X^T.  X is m x d_in (float32 values; bf16 inputs arrive already
    widened).  Returns V as r rows of length d_in, float32 (the paper's A, transposed)."""
    Xd = np.asarray(X, dtype=np.float64)
    m, d_in = Xd.shape
    Omega = gen_omega(seed, layer_id, m, r).astype(np.float64)
    Y = Xd.T @ Omega                       # Y <- H Omega
    deficient = False
    for _ in range(K):
        Q, _, bad = qr_positive(Y)         # [Q,~] <- qr(Y)
        deficient |= bad
        Y = Xd.T @ (Xd @ Q)                # Y <- H (H^T Q)
    Q, _, bad = qr_positive(Y)
    deficient |= bad
    V = np.ascontiguousarray(Q.T).astype(np.float32)
    if return_info:
        return V, {"deficient": bool(deficient), "V64": np.ascontiguousarray(Q.T)}
    return V


# --------------------------------------------------------------------------------------
# Eq. (agzo-perturb) and the in-place passes of Algorithm 2
# --------------------------------------------------------------------------------------
def lowrank_direction(G: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Delta = R A^T  (d_out x d_in) in float64 from float32 factors. V is r x d_in."""
    return np.asarray(G, dtype=np.float64) @ np.asarray(V, dtype=np.float64)


def apply_direction(W: np.ndarray, V: np.ndarray, seed: int, layer_id: int, coef,
                    storage: str = "bf16") -> np.ndarray:
    """W <- W + coef * R A^T with R regenerated from (seed, layer_id).

    W holds float32 values (bf16-representable when storage == "bf16").  The sum is
    formed in float64, rounded once to float32 and, for bf16 storage, once more (RNE) to
    bf16: "the fp32 result rounded to bf16".  coef is a float32 number."""
    d_out, d_in = W.shape
    r = V.shape[0]
    Z = lowrank_direction(gen_G(seed, layer_id, d_out, r), V)
    c = float(np.float32(coef))
    out32 = (np.asarray(W, dtype=np.float64) + c * Z).astype(np.float32)
    if storage == "bf16":
        return round_bf16(out32)
    if storage == "f32":
        return out32
    raise ValueError(storage)


def apply_dense(w: np.ndarray, seed: int, layer_id: int, coef, storage: str = "bf16"):
    """Second case of Eq. (agzo-perturb): w <- w + coef * u, u ~ N(0, I) from the seed."""
    u = gen_dense(seed, layer_id, w.size).astype(np.float64).reshape(w.shape)
    out32 = (np.asarray(w, dtype=np.float64) + float(np.float32(coef)) * u).astype(np.float32)
    return round_bf16(out32) if storage == "bf16" else out32


def ghat_two_point(f_plus, f_minus, eps) -> np.float32:
    """Central two-point scalar (f+ - f-) / (2 eps), float64 then rounded to float32."""
    e = float(np.float32(eps))
    return np.float32((float(f_plus) - float(f_minus)) / (2.0 * e))


def ghat_one_sided(f_plus, f_zero, mu) -> np.float32:
    """Algorithm 2, step 3: g <- (f+ - f0) / mu."""
    e = float(np.float32(mu))
    return np.float32((float(f_plus) - float(f_zero)) / e)


def update_coefficient(eps, lr, ghat, mode: int) -> np.float32:
    """Coefficient of Delta in the fused restore-and-update pass.

    mode 0 (two-point): weights sit at W - eps*Delta, so W <- W + (eps - lr*g) Delta.
    mode 1 (Algorithm 2 as printed): weights sit at W + mu*Delta, W <- W - (mu + lr*g) Delta.
    """
    e, l, g = float(np.float32(eps)), float(np.float32(lr)), float(np.float32(ghat))
    return np.float32(e - l * g) if mode == 0 else np.float32(-(e + l * g))


def agzo_step(layers, loss_fn, seed: int, eps, lr, K: int, mode: int = 0):
    """One AGZO iteration (Algorithm 2) over a list of layer dicts.

    Each layer dict holds: W (float32 values), X (m x d_in), r, layer_id, storage
    ("bf16" | "f32") and optionally W16 (bf16 compute copy of an fp32 master).  loss_fn
    takes the list of *compute* weights and returns a float.  Weights are replaced in the
    dicts.  Returns dict(f_plus, f_other, ghat, V=[...]).

    With a master/compute pair the master is never perturbed: the compute copy is
    rewritten as bf16(master +- eps*Delta) and the update is applied to the master.
    """
    def compute_weights():
        return [L["W16"] if L.get("W16") is not None else L["W"] for L in layers]

    Vs = []
    f_zero = loss_fn(compute_weights())                       # step 1: forward + extraction
    for L in layers:
        L["V"] = extract_subspace(L["X"], L["r"], K, seed, L["layer_id"])
        Vs.append(L["V"])

    def shift(coef, master_coef_for_pair):
        for L in layers:
            if L.get("W16") is not None:
                L["W16"] = apply_direction(L["W"], L["V"], seed, L["layer_id"],
                                           master_coef_for_pair, "bf16")
            else:
                L["W"] = apply_direction(L["W"], L["V"], seed, L["layer_id"], coef,
                                         L["storage"])

    shift(np.float32(eps), np.float32(eps))                   # step 2: W + eps*Delta
    f_plus = loss_fn(compute_weights())
    if mode == 0:
        shift(np.float32(-2.0) * np.float32(eps), -np.float32(eps))   # W - eps*Delta
        f_other = loss_fn(compute_weights())
        g = ghat_two_point(f_plus, f_other, eps)
    else:
        f_other = f_zero
        g = ghat_one_sided(f_plus, f_zero, eps)
    c = update_coefficient(eps, lr, g, mode)
    c_master = np.float32(-float(np.float32(lr)) * float(g))
    for L in layers:                                          # step 3: restore & update
        if L.get("W16") is not None:
            L["W"] = apply_direction(L["W"], L["V"], seed, L["layer_id"], c_master, "f32")
            L["W16"] = round_bf16(L["W"])
        else:
            L["W"] = apply_direction(L["W"], L["V"], seed, L["layer_id"], c, L["storage"])
    return {"f_plus": float(f_plus), "f_other": float(f_other), "ghat": g, "V": Vs}


# --------------------------------------------------------------------------------------
# Losses of the two small workloads (the "user's model"; only the harness needs these)
# --------------------------------------------------------------------------------------
def least_squares_loss(W, X, Yt) -> float:
    """f(W) = 1/(2m) || X W^T - Y ||_F^2 for one linear layer."""
    E = np.asarray(X, np.float64) @ np.asarray(W, np.float64).T - np.asarray(Yt, np.float64)
    return float((E * E).sum() / (2.0 * X.shape[0]))


def least_squares_grad(W, X, Yt) -> np.ndarray:
    """Gradient of least_squares_loss: (1/m) E^T X  (the Q H^T of Eq. grad-matrix-form)."""
    Xd = np.asarray(X, np.float64)
    E = Xd @ np.asarray(W, np.float64).T - np.asarray(Yt, np.float64)
    return E.T @ Xd / X.shape[0]


def gelu(x: np.ndarray) -> np.ndarray:
    return 0.5 * x * (1.0 + _erf(x / np.sqrt(2.0)))


def mlp_forward(weights, x0, bf16_compute: bool, collect_inputs: bool = False):
    """h <- GELU(h W_l^T) for all but the last layer, linear last layer.

    With bf16_compute the weights passed in are bf16 values and every layer's input is
    rounded to bf16 (products exact, accumulation float64)."""
    h = np.asarray(x0, np.float64)
    inputs = []
    n = len(weights)
    for i, W in enumerate(weights):
        if bf16_compute:
            h = round_bf16(h.astype(np.float32)).astype(np.float64)
        if collect_inputs:
            inputs.append(h.astype(np.float32))
        h = h @ np.asarray(W, np.float64).T
        if i + 1 < n:
            h = gelu(h)
    return (h, inputs) if collect_inputs else h


def mse_loss(out, target) -> float:
    d = np.asarray(out, np.float64) - np.asarray(target, np.float64)
    return float((d * d).mean())


# --------------------------------------------------------------------------------------
# Closed forms used by the tests (Theorem 4.4)
# --------------------------------------------------------------------------------------
def beta(D: int) -> float:
    """beta_D = Gamma(D/2) / (sqrt(pi) Gamma((D+1)/2)), Theorem 4.4."""
    from scipy.special import gammaln
    return float(np.exp(gammaln(D / 2.0) - gammaln((D + 1) / 2.0)) / np.sqrt(np.pi))
