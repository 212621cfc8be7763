"""Power-iteration ablation on synthetic inputs (the paper's appendix "Power-Iteration Ablation"
compares K = 1, 3, 5 with an exact SVD on a trained model; here the same question is put to a
least-squares layer with planted activations, where everything has a closed form).

For V from Algorithm 1 with K power steps, two deterministic quality figures:
  energy(V) = ||X V^T||_F^2 / (sum of the r largest squared singular values of X), and
  rho(V)    = ||grad V^T||_F / ||grad||_F, the factor of Theorem 4.4's bound that depends on V
              (grad = the layer's true gradient, which lies in the row space of X).
The GPU's figures must equal the oracle's, grow with K, and K = 3 must recover most of what the
exact SVD gets while K = 0 (the sketch alone) does not.
"""
import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import DEV, Ctx, to_dev

pytestmark = pytest.mark.gpu


def test_more_power_steps_capture_more_of_the_activation_energy_and_of_the_gradient():
    m, d_in, d_out, p, seed = 2048, 512, 128, 32, 7
    ranks = (1, 8, 16)
    X = WL.planted_activations(m, d_in, p, seed=5, bf16=True)
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((d_out, d_in)) / np.sqrt(d_in)).astype(np.float32)
    Yt = rng.standard_normal((m, d_out)).astype(np.float32)
    grad = O.least_squares_grad(W, X, Yt)
    X64 = X.astype(np.float64)
    _, S, Vt = np.linalg.svd(X64, full_matrices=False)

    def figures(V, r):
        V = V.astype(np.float64)
        return (np.linalg.norm(X64 @ V.T) ** 2 / (S[:r] ** 2).sum(),
                np.linalg.norm(grad @ V.T) / np.linalg.norm(grad))

    Xd, _ = to_dev(X, True)
    Vds = [torch.zeros(r, d_in, device=DEV) for r in ranks]
    layers = [B.make_layer(X=Xd, V=Vd, r=r, layer_id=i) for i, (r, Vd) in enumerate(zip(ranks, Vds))]
    table = {r: [] for r in ranks}
    with Ctx(layers) as ctx:
        for K in (0, 1, 3, 5):
            B.agzo_extract_subspace(ctx, layers, seed, K)
            torch.cuda.synchronize()
            assert B.agzo_poll(ctx) == B.AGZO_OK
            for i, r in enumerate(ranks):
                got = figures(Vds[i].cpu().numpy(), r)
                want = figures(O.extract_subspace(X, r, K, seed, i), r)
                assert abs(got[0] - want[0]) <= 2e-3 and abs(got[1] - want[1]) <= 2e-3, (K, r, got, want)
                table[r].append(got)
    for r in ranks:
        energy = [e for e, _ in table[r]]
        rho = [g for _, g in table[r]]
        exact_rho = np.linalg.norm(grad @ Vt[:r].T) / np.linalg.norm(grad)
        assert all(b >= a - 1e-3 for a, b in zip(energy, energy[1:])), energy
        assert all(b >= a - 1e-3 for a, b in zip(rho, rho[1:])), rho
        assert energy[0] < 0.6 and energy[2] > 0.85 and energy[3] <= 1.0 + 1e-6     # K = 0, 3, 5
        assert rho[2] >= 0.88 * exact_rho and rho[0] <= 0.7 * exact_rho
