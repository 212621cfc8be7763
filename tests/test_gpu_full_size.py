"""Parity at the full layer sizes of the Qwen3-8B-shaped configuration, in the launch
configuration the benchmark times (default options: tensor-core extraction in waves, tensor-core
in-place pass).  One transformer block's distinct shapes are enough: the 36 blocks repeat them.

The oracle is fast enough for whole layers here (its products are a few GFLOP), so every element
is compared, with the tolerances of test_gpu_parity.py.
"""
import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import (DEV, Ctx, assert_weights_match, cancellation_floor, projector_distance,
                         tc_mismatch_bound, to_dev, to_host)

pytestmark = pytest.mark.gpu

M_TOKENS = 8 * 2048


@pytest.mark.parametrize("d_in,r", [(4096, 16), (12288, 16), (4096, 64), (4096, 1)])
def test_extraction_of_a_full_size_layer(d_in, r):
    X = WL.planted_activations(M_TOKENS, d_in, 64, seed=d_in + r, bf16=True)
    Xd, _ = to_dev(X, True)
    Vd = torch.zeros(r, d_in, device=DEV)
    layers = [B.make_layer(X=Xd, V=Vd, r=r, layer_id=7)]
    with Ctx(layers) as ctx:
        B.agzo_extract_subspace(ctx, layers, 3, 3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    Vg = to_host(Vd)
    Vo = O.extract_subspace(X, r, 3, 3, 7)
    assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
    assert projector_distance(Vg, Vo) <= 1e-3
    assert np.abs(Vg - Vo).max() <= 1e-3


@pytest.mark.parametrize("d_out,d_in,r", [(12288, 4096, 16), (4096, 12288, 16), (1024, 4096, 8), (4096, 4096, 4),
                                           (4096, 4096, 64)])
def test_in_place_passes_on_a_full_size_layer(d_out, d_in, r):
    seed, layer_id, eps = 5, 3, 1e-3
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=d_out + r, bf16=True)
    Vh = O.extract_subspace(WL.plain_activations(256, d_in, seed=r), r, 1, 3, layer_id)
    Wd, _ = to_dev(W0, True)
    Vd, _ = to_dev(Vh, False)
    layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=layer_id)]
    ghat = torch.tensor([0.41], device=DEV)
    tc = r >= 8                      # the default options send these layers to the tensor-core kernel
    rel = 2.0 ** -16 if tc else 2.0 ** -20
    with Ctx(layers) as ctx:
        B.agzo_perturb(ctx, layers, seed, eps)
        want = O.apply_direction(W0, Vh, seed, layer_id, np.float32(eps), "bf16")
        assert_weights_match(to_host(Wd), want, "bf16", floor=cancellation_floor(W0, eps, seed, layer_id, Vh, rel))
        cur = to_host(Wd)
        B.agzo_perturb(ctx, layers, seed, -2 * eps)
        want = O.apply_direction(cur, Vh, seed, layer_id, np.float32(-2 * eps), "bf16")
        assert_weights_match(to_host(Wd), want, "bf16", floor=cancellation_floor(cur, 2 * eps, seed, layer_id, Vh, rel))
        cur = to_host(Wd)
        B.agzo_restore_update(ctx, layers, seed, eps, 1e-3, 0, ghat)
        c = O.update_coefficient(eps, 1e-3, np.float32(0.41), 0)
        want = O.apply_direction(cur, Vh, seed, layer_id, c, "bf16")
        frac = tc_mismatch_bound(want, c, seed, layer_id, Vh) if tc else 1e-3
        assert_weights_match(to_host(Wd), want, "bf16", frac=frac,
                             floor=cancellation_floor(cur, c, seed, layer_id, Vh, rel))
        assert B.agzo_poll(ctx) == B.AGZO_OK
