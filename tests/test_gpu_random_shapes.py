"""Seeded random shapes: ragged rows and columns, every rank class, padded pitches, staged and
regenerated R, one or two column panels, shared inputs, several waves, all extraction paths.
Every case is compared with the oracle like the hand-picked cases of test_gpu_parity.py."""
import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import (DEV, Ctx, assert_weights_match, cancellation_floor, projector_distance, tc_mismatch_bound,
                         to_dev, to_host)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed0", [1, 2])
def test_tensor_core_pass_on_random_shapes(seed0):
    rng = np.random.default_rng(seed0)
    for case in range(30):
        r = int(rng.choice([3, 4, 5, 7, 8, 9, 15, 16, 17, 23, 24, 31, 32, 33, 40, 47, 48, 49, 63, 64]))
        d_out = int(rng.integers(1, 700))
        d_in = int(rng.integers(max(r, 8) // 8 + 1, 160)) * 8
        extra = int(rng.choice([0, 8, 24]))
        stage, panels = int(rng.choice([0, 1, 2])), int(rng.choice([0, 1, 2]))
        seed, lid = int(rng.integers(0, 1 << 30)), int(rng.integers(0, 1000))
        c = float(rng.choice([1e-3, -2e-3, 3e-2]))
        what = dict(r=r, d_out=d_out, d_in=d_in, extra=extra, stage=stage, panels=panels, c=c)
        W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=case, bf16=True)
        Vh = O.extract_subspace(WL.plain_activations(max(2 * r, 32), d_in, seed=case), r, 1, 3, lid)
        Wd, _ = to_dev(W0, True, pitch=d_in + extra if extra else None)
        Vd, _ = to_dev(Vh, False)
        layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=lid)]
        with Ctx(layers, extra=1 << 22) as ctx:
            B.agzo_set_option(ctx, "rmw_path", 2)
            B.agzo_set_option(ctx, "rmw_stage_r", stage)
            B.agzo_set_option(ctx, "rmw_tc_panels", panels)
            cur = W0
            for coef in (c, -c):          # the second pass finds staged images of the same seed in place
                B.agzo_perturb(ctx, layers, seed, coef)
                torch.cuda.synchronize()
                assert B.agzo_poll(ctx) == B.AGZO_OK, what
                want = O.apply_direction(cur, Vh, seed, lid, np.float32(coef), "bf16")
                # share of results that may land on the neighbouring bf16 value: derived from the split-bf16
                # operands of the product (2^-17 |c| (|G||V|)_ij against the result's own step), as in the
                # hand-picked cases
                assert_weights_match(to_host(Wd), want, "bf16", frac=tc_mismatch_bound(want, coef, seed, lid, Vh),
                                     floor=cancellation_floor(cur, coef, seed, lid, Vh, rel=2.0 ** -16))
                cur = to_host(Wd)


@pytest.mark.parametrize("seed0", [3, 4])
def test_extraction_on_random_shapes(seed0):
    rng = np.random.default_rng(seed0)
    for case in range(20):
        nl = int(rng.integers(1, 5))
        K = int(rng.choice([0, 1, 2, 3]))
        path = int(rng.choice([0, 1, 2, 3]))
        seed = int(rng.integers(0, 1 << 30))
        share = int(rng.integers(0, 2))
        specs, Xs, devs, layers = [], [], [], []
        for i in range(nl):
            if i > 0 and share and rng.random() < 0.5:      # read the previous layer's buffer
                m, d_in, X, Xd = specs[-1][0], specs[-1][1], Xs[-1], devs[-1][0]
            else:
                m = int(rng.integers(256, 3000))
                d_in = int(rng.integers(16, 140)) * 8
                X = WL.planted_activations(m, d_in, 16, seed=1000 * case + i, bf16=True)
                Xd, _ = to_dev(X, True)
            r = min(int(rng.choice([1, 2, 3, 4, 7, 8, 9, 16, 24, 31, 32, 48, 64])), d_in, m)
            Vd = torch.zeros(r, d_in, device=DEV)
            specs.append((m, d_in, r)); Xs.append(X); devs.append((Xd, Vd))
            layers.append(B.make_layer(X=Xd, V=Vd, r=r, layer_id=7 * case + i))
        what = dict(specs=specs, K=K, path=path, share=share)
        with Ctx(layers) as ctx:
            B.agzo_set_option(ctx, "extract_path", path)
            B.agzo_set_option(ctx, "extract_fused", 2 if path == 2 else 0)   # path 2: fused power steps where shapes allow
            B.agzo_set_option(ctx, "share_inputs", share)
            if rng.random() < 0.3:
                B.agzo_set_option(ctx, "wave_bytes", int(rng.integers(1, 8)) << 20)
            B.agzo_extract_subspace(ctx, layers, seed, K)
            torch.cuda.synchronize()
            assert B.agzo_poll(ctx) == B.AGZO_OK, what
        for i, ((m, d_in, r), X) in enumerate(zip(specs, Xs)):
            Vg = to_host(devs[i][1])
            Vo = O.extract_subspace(X, r, K, seed, 7 * case + i)
            assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5, (what, i)
            assert projector_distance(Vg, Vo) <= 1e-3, (what, i)
