"""Pins for the CPU oracle: each checks it against something fixed by the paper or by
mathematics that does not pass through the oracle's own formula."""
import os

import numpy as np
import pytest
import scipy.stats
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import workloads as WL

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- generator
def _read_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_philox_known_answer_vectors():
    for row in _read_rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in row]
        out = O.philox4x32_10(*[np.array([c]) for c in v[:4]], v[4], v[5])
        assert [int(o[0]) for o in out] == v[6:]


def test_philox_stream_indexing_is_block_then_lane():
    # element e of a stream is word (e & 3) of the block with counter (e >> 2, layer, tag)
    seed, layer, tag = 0x123456789ABCDEF, 7, 1
    w = O.philox_words(seed, layer, tag, 37)
    for e in (0, 1, 5, 18, 36):
        blk = O.philox4x32_10(np.array([e >> 2]), np.array([0]), layer, tag,
                              seed & 0xFFFFFFFF, seed >> 32)
        assert int(w[e]) == int(blk[e & 3][0])
    # a window of the stream equals the same elements of the whole stream
    assert np.array_equal(O.philox_words(seed, layer, tag, 9, first=14), w[14:23])


def test_philox_streams_are_distinct():
    n = 1 << 16
    a = O.philox_words(1, 0, 0, n)
    b = O.philox_words(1, 1, 0, n)
    c = O.philox_words(1, 0, 1, n)
    d = O.philox_words(2, 0, 0, n)
    for x, y in ((a, b), (a, c), (a, d), (b, c)):
        assert (x == y).mean() < 1e-3
    # a bijection on counters cannot repeat 128-bit blocks
    blocks = a.reshape(-1, 4)
    assert len({tuple(r) for r in blocks.tolist()}) == blocks.shape[0]


def test_gaussians_are_standard_normal():
    g = O.gaussian_stream(5, 3, O.TAG_G, 1 << 20).astype(np.float64)
    n = g.size
    assert abs(g.mean()) < 4.0 / np.sqrt(n)
    assert abs(g.var() - 1.0) < 4.0 * np.sqrt(2.0 / n)
    assert abs((g ** 4).mean() - 3.0) < 4.0 * np.sqrt(96.0 / n)
    assert abs((g ** 3).mean()) < 4.0 * np.sqrt(15.0 / n)
    assert scipy.stats.kstest(g[: 1 << 17], "norm").pvalue > 1e-3
    # the four lanes of a block are uncorrelated, and so are neighbouring elements
    q = g.reshape(-1, 4)
    c = np.corrcoef(q.T)
    assert np.abs(c - np.eye(4)).max() < 5.0 / np.sqrt(q.shape[0])
    assert abs(np.corrcoef(g[:-1], g[1:])[0, 1]) < 5.0 / np.sqrt(n)
    # tails exist and are finite (u1 is never 0)
    assert np.isfinite(g).all() and np.abs(g).max() > 4.0


def test_G_and_omega_layouts():
    G = O.gen_G(9, 2, 10, 3)
    flat = O.gaussian_stream(9, 2, O.TAG_G, 30)
    assert G.shape == (10, 3) and np.array_equal(G.reshape(-1), flat)
    Om = O.gen_omega(9, 2, 6, 5)
    assert np.array_equal(Om.reshape(-1), O.gaussian_stream(9, 2, O.TAG_OMEGA, 30))
    assert not np.array_equal(Om.reshape(-1), flat)


# ----------------------------------------------------------------------------- bf16 rounding
def test_bf16_rounding_matches_torch_everywhere():
    hi = np.arange(1 << 16, dtype=np.uint32) << 16
    cases = [hi, hi | 0x7FFF, hi | 0x8000, hi | 0x8001, hi | 0xFFFF, hi | 0x0001]
    u = np.concatenate(cases).astype(np.uint32)
    x = u.view(np.float32)
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = O.f32_to_bf16_bits(x)
    nan = np.isnan(x)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.isnan(O.bf16_bits_to_f32(got[nan])).all()
    assert np.array_equal(O.bf16_bits_to_f32(got[~nan]),
                          torch.from_numpy(x.copy()).to(torch.bfloat16).float().numpy()[~nan])


# ----------------------------------------------------------------------------- Algorithm 1
def _posqr(M):
    Q, R = np.linalg.qr(M)
    s = np.sign(np.diag(R))
    return Q * s, (R.T * s).T


def test_qr_positive_matches_lapack_up_to_signs():
    rng = np.random.default_rng(0)
    Y = rng.standard_normal((50, 6)) @ np.diag([1, 10, 0.1, 5, 2, 1e-3])
    Q, R, bad = O.qr_positive(Y)
    Qn, Rn = _posqr(Y)
    assert not bad
    assert np.all(np.diag(R) > 0)
    assert np.abs(Q - Qn).max() < 1e-10 and np.abs(R - Rn).max() < 1e-9
    assert np.abs(Q @ R - Y).max() < 1e-12


def test_extract_is_orthonormal():
    X = WL.planted_activations(300, 96, 12, seed=1, bf16=False)
    for r in (1, 4, 8):
        V = O.extract_subspace(X, r, 3, seed=4, layer_id=2, return_info=True)[1]["V64"]
        assert np.abs(V @ V.T - np.eye(r)).max() < 1e-12


@pytest.mark.parametrize("K", [0, 1, 3])
def test_extract_equals_q_factor_of_power_matrix(K):
    # In exact arithmetic the intermediate QRs only rescale by upper-triangular factors
    # with positive diagonals, so A is the positive-diagonal Q of (H H^T)^K H Omega.
    m, d_in, r = 40, 12, 3
    X = WL.plain_activations(m, d_in, seed=3).astype(np.float64)
    Om = O.gen_omega(11, 5, m, r).astype(np.float64)
    M = X.T @ Om
    C = X.T @ X
    for _ in range(K):
        M = C @ M
    Qn, _ = _posqr(M)
    V = O.extract_subspace(X, r, K, seed=11, layer_id=5, return_info=True)[1]["V64"]
    assert np.abs(V.T - Qn).max() < 1e-8


def test_extract_lies_in_the_row_space_of_X():
    m, d_in, r = 6, 32, 4            # m < d_in so the statement is not vacuous
    X = WL.plain_activations(m, d_in, seed=8).astype(np.float64)
    V = O.extract_subspace(X, r, 3, seed=1, layer_id=0, return_info=True)[1]["V64"]
    P = np.linalg.pinv(X) @ X        # projector onto row(X) = col(H)
    assert np.abs(V - V @ P).max() < 1e-10


def test_extract_quality_follows_the_power_iteration_ablation():
    # K = 3 is close to the exact top-r singular subspace, K = 1 visibly worse, and more
    # steps never hurt (the power-iteration ablation table, qualitatively).  A decaying
    # spectrum is used so that the top-r subspace is well defined.
    rng = np.random.default_rng(5)
    m, d_in, r = 400, 64, 4
    U, _ = np.linalg.qr(rng.standard_normal((m, d_in)))
    Vt, _ = np.linalg.qr(rng.standard_normal((d_in, d_in)))
    s = 1.0 / (1.0 + np.arange(d_in)) ** 0.5
    X = (U * s) @ Vt.T
    _, _, vt = np.linalg.svd(X, full_matrices=False)
    best = np.linalg.norm(X @ vt[:r].T) ** 2

    def energy(K):
        V = O.extract_subspace(X, r, K, seed=2, layer_id=1, return_info=True)[1]["V64"]
        return np.linalg.norm(X @ V.T) ** 2 / best

    e0, e1, e3, e5 = energy(0), energy(1), energy(3), energy(5)
    assert e0 < e1 < e3 <= e5 + 1e-12 <= 1.0 + 1e-9
    assert e3 > 0.93 and e1 < e3 - 0.03


def test_extract_finds_a_planted_subspace():
    m, d_in, p, r = 512, 128, 8, 8
    rng = np.random.default_rng([21, 0x58])      # same stream as the generator: recover B
    rng.standard_normal((m, d_in))
    B, _ = np.linalg.qr(rng.standard_normal((d_in, p)))
    X = WL.planted_activations(m, d_in, p, seed=21, bf16=False)
    V = O.extract_subspace(X, r, 3, seed=0, layer_id=0, return_info=True)[1]["V64"]
    resid = np.linalg.norm(V - (V @ B) @ B.T)     # part of V outside the planted space
    assert resid < 0.35 * np.sqrt(r)


def test_rank_deficient_panel_yields_zero_columns():
    m, d_in, r = 20, 16, 4
    rng = np.random.default_rng(0)
    X = np.outer(rng.standard_normal(m), rng.standard_normal(d_in))   # rank one
    X += np.outer(rng.standard_normal(m), rng.standard_normal(d_in))  # rank two
    V, info = O.extract_subspace(X, r, 2, seed=3, layer_id=0, return_info=True)
    assert info["deficient"]
    norms = np.linalg.norm(info["V64"], axis=1)
    assert np.allclose(norms[:2], 1.0) and np.all(norms[2:] == 0.0)
    assert abs(info["V64"][0] @ info["V64"][1]) < 1e-10


def test_rank_test_is_relative_to_the_column_itself():
    # qr(Y) must not depend on the scale of a column: an independent column is kept however
    # small it is next to the first one, a dependent column is dropped however large it is.
    # (A test against R_11 fails both halves.)
    rng = np.random.default_rng(7)
    Y = rng.standard_normal((40, 4))
    Qn, _ = _posqr(Y)
    for scale in (1e-9, 1e-3, 1.0, 1e6):
        Q, R, bad = O.qr_positive(Y * np.array([1.0, scale, 1.0, scale]))
        assert not bad and np.abs(Q - Qn).max() < 1e-9
    Yd = Y.copy()
    Yd[:, 2] = 3.0 * Y[:, 0] - 2.0 * Y[:, 1]            # exactly dependent
    for scale in (1e-6, 1.0, 1e13):
        Q, R, bad = O.qr_positive(Yd * np.array([1.0, 1.0, scale, 1.0]))
        assert bad and np.all(Q[:, 2] == 0.0)
        assert np.abs(np.linalg.norm(Q[:, [0, 1, 3]], axis=0) - 1.0).max() < 1e-12


def test_a_dominant_direction_does_not_cost_the_others():
    # sigma_1 / sigma_2 = 1000 (an outlier feature): the columns of Y = H (H^T Q) then differ by
    # 1e6 in length, yet Algorithm 1 returns r orthonormal columns spanning the top-r singular
    # subspace.  (With the pivot compared to R_11 the second column would be zeroed.)
    rng = np.random.default_rng(9)
    m, d_in, r = 120, 48, 4
    U, _ = np.linalg.qr(rng.standard_normal((m, d_in)))
    Wt, _ = np.linalg.qr(rng.standard_normal((d_in, d_in)))
    s = np.concatenate([[1000.0, 1.0, 0.5, 0.25], 0.01 * np.ones(d_in - 4)])
    X = (U * s) @ Wt.T
    V, info = O.extract_subspace(X, r, 3, seed=6, layer_id=1, return_info=True)
    assert not info["deficient"]
    V64 = info["V64"]
    assert np.abs(V64 @ V64.T - np.eye(r)).max() < 1e-10
    top = Wt[:, :r].T                                  # exact top-r right singular vectors
    assert np.linalg.norm(V64.T @ V64 - top.T @ top) < 1e-6


def test_graded_and_outlier_activations_keep_all_columns():
    # decaying spectrum (sigma_k = 2^(-k/2)) and "massive activation" inputs: no column is
    # dropped, the basis is orthonormal and captures nearly the energy of the exact top-r
    Xg = WL.graded_activations(600, 160, 64, seed=3, bf16=True)
    Xm = WL.massive_activations(600, 160, seed=4, bf16=True)
    for X in (Xg, Xm):
        _, _, vt = np.linalg.svd(X.astype(np.float64), full_matrices=False)
        for r in (4, 16):
            V, info = O.extract_subspace(X, r, 3, seed=2, layer_id=5, return_info=True)
            assert not info["deficient"]
            V64 = info["V64"]
            assert np.abs(V64 @ V64.T - np.eye(r)).max() < 1e-10
            best = np.linalg.norm(X.astype(np.float64) @ vt[:r].T) ** 2
            assert np.linalg.norm(X.astype(np.float64) @ V64.T) ** 2 >= (1.0 - 1e-3) * best


# ----------------------------------------------------------------------------- perturbation
def test_direction_is_confined_to_the_subspace():
    d_out, d_in, r = 24, 40, 5
    X = WL.plain_activations(64, d_in, seed=2)
    V = O.extract_subspace(X, r, 3, seed=6, layer_id=9).astype(np.float64)
    G = O.gen_G(6, 9, d_out, r)
    Z = O.lowrank_direction(G, V)
    P = V.T @ V
    assert np.abs(Z - Z @ P).max() < 1e-6                 # Delta (I - A A^T) = 0
    assert abs(np.linalg.norm(Z) - np.linalg.norm(G.astype(np.float64))) < 1e-5  # ||R A^T|| = ||R||
    assert np.linalg.matrix_rank(Z, tol=1e-6) == r
    # Z_ij = sum_k G_ik V_kj, element by element
    i, j = 7, 13
    assert abs(Z[i, j] - sum(float(G[i, k]) * V[k, j] for k in range(r))) < 1e-12


def test_apply_direction_storage_and_sign():
    d_out, d_in, r = 16, 24, 3
    W = WL.gaussian_weights(d_out, d_in, 0.02, seed=1, bf16=True)
    V = O.extract_subspace(WL.plain_activations(48, d_in, seed=4), r, 2, 8, 1)
    Z = O.lowrank_direction(O.gen_G(8, 1, d_out, r), V)
    c = np.float32(3e-3)
    Wp = O.apply_direction(W, V, 8, 1, c, "bf16")
    exact = W.astype(np.float64) + float(c) * Z
    ulp = np.spacing(np.abs(Wp).astype(np.float32)) * 2 ** 16      # bf16 ulp at |Wp|
    assert np.all(np.abs(Wp - exact) <= 0.5 * ulp * (1 + 1e-6) + 1e-12)
    assert np.array_equal(Wp, WL.to_bf16_values(Wp))              # on the bf16 grid
    Wf = O.apply_direction(W, V, 8, 1, c, "f32")
    assert np.abs(Wf - exact).max() < 1e-8
    Wm = O.apply_direction(W, V, 8, 1, -c, "f32")
    assert np.abs((Wf.astype(np.float64) + Wm) / 2 - W).max() < 1e-8  # symmetric about W


def test_dense_direction_for_non_matrix_parameters():
    w = np.zeros(1000, dtype=np.float32)
    out = O.apply_dense(w, 4, 17, np.float32(0.5), "f32")
    u = O.gaussian_stream(4, 17, O.TAG_DENSE, 1000)
    assert np.allclose(out, 0.5 * u, atol=1e-7)


# ----------------------------------------------------------------------------- gradient facts
def _brute_force_grad(f, W, h=1e-3):
    g = np.zeros_like(W, dtype=np.float64)
    for i in range(W.shape[0]):
        for j in range(W.shape[1]):
            Wp, Wm = W.copy(), W.copy()
            Wp[i, j] += h
            Wm[i, j] -= h
            g[i, j] = (f(Wp) - f(Wm)) / (2 * h)    # exact for a quadratic
    return g


def test_gradient_row_space_is_inside_the_activation_space():
    m, d_in, d_out = 8, 32, 16
    rng = np.random.default_rng(1)
    X = rng.standard_normal((m, d_in))
    Yt = rng.standard_normal((m, d_out))
    W = rng.standard_normal((d_out, d_in))
    g = _brute_force_grad(lambda w: O.least_squares_loss(w, X, Yt), W)
    assert np.abs(g - O.least_squares_grad(W, X, Yt)).max() < 1e-8      # = Q H^T
    P = np.linalg.pinv(X) @ X
    assert np.abs(g - g @ P).max() < 1e-8                               # row(grad) in col(H)
    assert np.linalg.matrix_rank(g, tol=1e-8) <= m


def test_two_point_scalar_is_the_directional_derivative_on_a_quadratic():
    m, d_in, d_out, r = 40, 24, 12, 3
    rng = np.random.default_rng(2)
    X = rng.standard_normal((m, d_in))
    Yt = rng.standard_normal((m, d_out))
    W = rng.standard_normal((d_out, d_in))
    V = O.extract_subspace(X, r, 3, 5, 0).astype(np.float64)
    Z = O.lowrank_direction(O.gen_G(5, 0, d_out, r), V)
    eps = 1e-3
    fp = O.least_squares_loss(W + eps * Z, X, Yt)
    fm = O.least_squares_loss(W - eps * Z, X, Yt)
    want = (O.least_squares_grad(W, X, Yt) * Z).sum()
    assert abs((fp - fm) / (2 * eps) - want) < 1e-9 * max(1.0, abs(want))
    # and the float32 scalar the library reports
    assert abs(float(O.ghat_two_point(fp, fm, eps)) - want) < 2e-6 * max(1.0, abs(want))
    # one-sided (Algorithm 2 as printed) carries the O(mu) curvature term exactly
    f0 = O.least_squares_loss(W, X, Yt)
    curv = (Z @ (X.T @ X / m) * Z).sum()
    assert abs((fp - f0) / eps - (want + 0.5 * eps * curv)) < 1e-8 * max(1.0, abs(want))


def test_update_decreases_a_quadratic_by_the_closed_form():
    m, d_in, d_out, r = 40, 24, 12, 3
    rng = np.random.default_rng(3)
    X = rng.standard_normal((m, d_in))
    Yt = rng.standard_normal((m, d_out))
    W = rng.standard_normal((d_out, d_in))
    V = O.extract_subspace(X, r, 3, 6, 0).astype(np.float64)
    Z = O.lowrank_direction(O.gen_G(6, 0, d_out, r), V)
    g = (O.least_squares_grad(W, X, Yt) * Z).sum()
    eta = 1e-2
    lhs = O.least_squares_loss(W - eta * g * Z, X, Yt) - O.least_squares_loss(W, X, Yt)
    rhs = -eta * g * g + 0.5 * eta ** 2 * g ** 2 * (Z @ (X.T @ X / m) * Z).sum()
    assert abs(lhs - rhs) < 1e-10 * max(1.0, abs(rhs))


def test_update_coefficient_modes():
    eps, lr, g = np.float32(1e-3), np.float32(5e-4), np.float32(1.75)
    assert abs(float(O.update_coefficient(eps, lr, g, 0)) - (1e-3 - 5e-4 * 1.75)) < 1e-9
    assert abs(float(O.update_coefficient(eps, lr, g, 1)) + (1e-3 + 5e-4 * 1.75)) < 1e-9


def test_step_on_a_quadratic_matches_the_closed_forms():
    # A whole Algorithm-2 iteration in fp32 storage on least squares: ghat equals
    # <grad, Z>, W moves by -lr*ghat*Z, both to float32 rounding.
    X, Yt, W0 = WL.least_squares_problem(seed=0, d_in=32, d_out=16, m=64)
    L = {"W": W0.copy(), "X": X, "r": 4, "layer_id": 0, "storage": "f32"}
    eps, lr = 1e-3, 5e-3
    res = O.agzo_step([L], lambda ws: O.least_squares_loss(ws[0], X, Yt), seed=0,
                      eps=eps, lr=lr, K=3, mode=0)
    V = res["V"][0].astype(np.float64)
    Z = O.lowrank_direction(O.gen_G(0, 0, 16, 4), V)
    want = (O.least_squares_grad(W0, X, Yt) * Z).sum()
    assert abs(float(res["ghat"]) - want) < 2e-3 * abs(want)    # fp32 weight storage noise
    assert np.abs(L["W"] - (W0 - lr * float(res["ghat"]) * Z)).max() < 5e-7
    # one-sided mode: two forwards, same update direction
    L1 = {"W": W0.copy(), "X": X, "r": 4, "layer_id": 0, "storage": "f32"}
    res1 = O.agzo_step([L1], lambda ws: O.least_squares_loss(ws[0], X, Yt), seed=0,
                       eps=eps, lr=lr, K=3, mode=1)
    curv = (Z @ (X.astype(np.float64).T @ X.astype(np.float64) / X.shape[0]) * Z).sum()
    want1 = want + 0.5 * eps * curv                     # one-sided difference, exact on a quadratic
    assert abs(float(res1["ghat"]) - want1) < 2e-3 * abs(want1)
    assert np.abs(L1["W"] - (W0 - lr * float(res1["ghat"]) * Z)).max() < 5e-7


def test_master_compute_pair_never_perturbs_the_master():
    X, Yt, W0 = WL.least_squares_problem(seed=1, d_in=32, d_out=16, m=64)
    seen = []

    def loss(ws):
        seen.append(ws[0].copy())
        return O.least_squares_loss(ws[0], X, Yt)

    L = {"W": W0.copy(), "W16": O.round_bf16(W0), "X": X, "r": 2, "layer_id": 3,
         "storage": "f32"}
    res = O.agzo_step([L], loss, seed=7, eps=1e-2, lr=1e-3, K=2, mode=0)
    V = res["V"][0].astype(np.float64)
    Z = O.lowrank_direction(O.gen_G(7, 3, 16, 2), V)
    assert np.array_equal(seen[0], O.round_bf16(W0))
    assert np.array_equal(seen[1], O.round_bf16((W0 + 1e-2 * Z).astype(np.float32)))
    assert np.array_equal(seen[2], O.round_bf16((W0 - 1e-2 * Z).astype(np.float32)))
    assert np.abs(L["W"] - (W0 - 1e-3 * float(res["ghat"]) * Z)).max() < 5e-7
    assert np.array_equal(L["W16"], O.round_bf16(L["W"]))


# ----------------------------------------------------------------------------- Theorem 4.4 / Lemma A.1
def test_beta_closed_form_and_bounds():
    for D, b in [(int(r[0]), float(r[1])) for r in _read_rows("beta_bounds.txt")]:
        assert abs(O.beta(D) - b) < 1e-12
    for D in (2, 3, 16, 100, 4096):
        assert np.sqrt(2 / (np.pi * D)) <= O.beta(D) <= np.sqrt(2 / (np.pi * (D - 1)))


def test_expected_cosine_matches_theorem_4_4():
    # Monte-Carlo over seeds with the oracle's own G: mean cos(ghat0, Gtrue) equals
    # beta_{d_out r} ||Gtrue A|| / ||Gtrue||.
    d_out, d_in, r, n = 4, 10, 2, 20000
    rng = np.random.default_rng(4)
    Gt = rng.standard_normal((d_out, d_in))
    A, _ = np.linalg.qr(rng.standard_normal((d_in, r)))
    V = A.T
    cos = np.empty(n)
    for s in range(n):
        Z = O.lowrank_direction(O.gen_G(s, 1, d_out, r), V)
        est = (Gt * Z).sum() * Z
        cos[s] = (est * Gt).sum() / (np.linalg.norm(est) * np.linalg.norm(Gt))
    want = O.beta(d_out * r) * np.linalg.norm(Gt @ A) / np.linalg.norm(Gt)
    assert abs(cos.mean() - want) < 4 * cos.std() / np.sqrt(n)


def test_gaussian_moment_identity():
    # Lemma A.1: E[<M, R> R] = M
    d_out, r, n = 3, 2, 40000
    M = np.array([[1.0, -2.0], [0.5, 0.0], [3.0, 1.0]])
    acc = np.zeros_like(M)
    for s in range(n):
        R = O.gen_G(s, 2, d_out, r).astype(np.float64)
        acc += (M * R).sum() * R
    # Var of each entry of <M,R>R is at most 3||M||^2
    assert np.abs(acc / n - M).max() < 5 * np.sqrt(3 * (M * M).sum() / n)


# ----------------------------------------------------------------------------- harness forwards
def test_gelu_and_mlp_forward_against_torch():
    Ws, x0, tgt = WL.mlp_problem(seed=0, n_layers=3, width=32, m=16)
    out = O.mlp_forward(Ws, x0, bf16_compute=False)
    h = torch.from_numpy(x0).double()
    for i, W in enumerate(Ws):
        h = h @ torch.from_numpy(W).double().t()
        if i + 1 < len(Ws):
            h = torch.nn.functional.gelu(h)
    assert np.abs(out - h.numpy()).max() < 1e-12
    assert abs(O.mse_loss(out, tgt)
               - torch.nn.functional.mse_loss(h, torch.from_numpy(tgt).double()).item()) < 1e-12
    out16, ins = O.mlp_forward([O.round_bf16(W) for W in Ws], x0, True, collect_inputs=True)
    assert len(ins) == 3 and np.array_equal(ins[0], WL.to_bf16_values(x0))
    assert np.abs(out16 - out).max() < 0.2


def test_gaussian_right_factor_of_the_lozo_comparison():
    """Eq. (lozo-layer-perturb): both factors Gaussian.  The right factor is its own stream (tag 3), laid
    out as r rows of d_in, independent of the left factor's stream, and U V^T has E||Delta||_F^2 = d_out d_in r."""
    r, d_in, d_out = 4, 96, 64
    V = O.gen_gaussian_basis(9, 5, r, d_in)
    flat = O.gaussian_stream(9, 5, O.TAG_BASIS, r * d_in)
    assert V.shape == (r, d_in) and np.array_equal(V.reshape(-1), flat)
    assert not np.array_equal(flat[: d_out * r], O.gen_G(9, 5, d_out, r).reshape(-1)[: r * d_in][: d_out * r])
    big = O.gen_gaussian_basis(1, 0, 8, 50000)
    assert abs(big.mean()) < 5e-3 and abs(big.var() - 1.0) < 1e-2
    tot = 0.0
    for s in range(200):
        D = O.lowrank_direction(O.gen_G(s, 0, d_out, r), O.gen_gaussian_basis(s, 0, r, d_in))
        tot += (D * D).sum()
    assert abs(tot / 200 / (d_out * d_in * r) - 1.0) < 0.05
