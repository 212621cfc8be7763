"""Whole AGZO iterations (Algorithm 2) through agzo_step on the two small workloads:
the single fp32 least-squares layer and the 8-layer GELU MLP with fp32 masters and bf16
compute copies.  The forward passes are the caller's model: torch on the device here,
numpy in the oracle.

Tolerances: ghat within 1e-3 relative (relative to the larger of |ghat| and the RMS of
ghat over the run); V projector distance <= 1e-3; weights as in test_gpu_parity when both
sides are fed the same V and ghat, and 1e-6 absolute for the free-running fp32 masters."""
import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import (DEV, Ctx, assert_weights_match, cancellation_floor, projector_distance,
                         to_dev, to_host)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [0, 1])
def test_single_fp32_layer_least_squares_step(mode):
    X, Yt, W0 = WL.least_squares_problem(seed=0)          # 256 -> 256, 512 tokens
    r, eps, lr, K, seed = 4, 1e-3, 5e-4, 3, 0
    Xd, _ = to_dev(X, False)
    Yd = torch.from_numpy(Yt).to(DEV).double()
    Wd, _ = to_dev(W0, False)
    Vd = torch.zeros(r, 256, device=DEV)
    layers = [B.make_layer(W=Wd, X=Xd, V=Vd, r=r, layer_id=0)]
    losses = torch.zeros(2, device=DEV, dtype=torch.float64)
    ghat = torch.zeros(1, device=DEV)
    seen = []

    def loss_fn(phase, slot, stream):
        seen.append(phase)
        E = Xd.double() @ Wd.double().t() - Yd
        losses[slot] = (E * E).sum() / (2 * X.shape[0])

    with Ctx(layers) as ctx:
        B.agzo_step(ctx, layers, seed=seed, eps=eps, lr=lr, K=K, mode=mode, loss_fn=loss_fn,
                    d_losses2=losses, d_ghat=ghat)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    assert seen == ([0, 1, 2] if mode == 0 else [0, 1])

    L = {"W": W0.copy(), "X": X, "r": r, "layer_id": 0, "storage": "f32"}
    res = O.agzo_step([L], lambda ws: O.least_squares_loss(ws[0], X, Yt), seed, eps, lr, K, mode)
    f_plus, f_other = [float(v) for v in losses.cpu()]
    g = float(ghat)
    assert abs(f_plus - res["f_plus"]) <= 1e-6 * abs(res["f_plus"])
    assert abs(f_other - res["f_other"]) <= 1e-6 * abs(res["f_other"])
    assert abs(g - float(res["ghat"])) <= 1e-3 * abs(float(res["ghat"]))
    Vg = to_host(Vd)
    assert projector_distance(Vg, res["V"][0]) <= 1e-3
    # each side with its own V and ghat: within 1e-3 of the size of the update
    assert np.abs(to_host(Wd) - L["W"]).max() <= 1e-3 * np.abs(L["W"] - W0).max()
    # same V and ghat on both sides: the update itself to fp32 rounding
    c = np.float32(-float(np.float32(lr)) * float(np.float32(g)))
    Z = O.lowrank_direction(O.gen_G(seed, 0, 256, r), Vg)
    assert np.abs(to_host(Wd) - (W0 + float(c) * Z)).max() <= 2e-7


def test_callback_failure_restores_the_weights():
    X, Yt, W0 = WL.least_squares_problem(seed=1, d_in=64, d_out=32, m=128)
    Xd, _ = to_dev(X, False)
    Wd, _ = to_dev(W0, False)
    Vd = torch.zeros(2, 64, device=DEV)
    layers = [B.make_layer(W=Wd, X=Xd, V=Vd, r=2, layer_id=0)]
    losses = torch.zeros(2, device=DEV, dtype=torch.float64)
    ghat = torch.zeros(1, device=DEV)

    def loss_fn(phase, slot, stream):
        if phase == 2:
            raise RuntimeError("forward failed")

    with Ctx(layers) as ctx:
        with pytest.raises(B.AgzoError) as e:
            B.agzo_step(ctx, layers, seed=3, eps=1e-2, lr=1e-3, K=2, mode=0, loss_fn=loss_fn,
                        d_losses2=losses, d_ghat=ghat)
        assert e.value.status == B.AGZO_ERR_CALLBACK
    assert np.abs(to_host(Wd) - W0).max() <= 1e-7       # back at W within fp32 rounding


@pytest.mark.parametrize("mode,fail_at", [(0, 3), (0, 4), (0, 5), (1, 3), (1, 4)])
def test_a_failing_library_call_inside_a_step_restores_the_weights(mode, fail_at):
    # The failure is made on the host: the option lets the n-th internal call of agzo_step
    # (1 extract, 2 perturb, 3 flip [mode 0] / ghat [mode 1], then ghat, restore+update) return an
    # error before it launches anything.  No GPU fault is involved.  Whatever fails after the
    # first pass, the step must leave W where it started.
    X, Yt, W0 = WL.least_squares_problem(seed=2, d_in=64, d_out=32, m=128)
    Xd, _ = to_dev(X, False)
    Wd, _ = to_dev(W0, False)
    Vd = torch.zeros(2, 64, device=DEV)
    layers = [B.make_layer(W=Wd, X=Xd, V=Vd, r=2, layer_id=0)]
    losses = torch.zeros(2, device=DEV, dtype=torch.float64)
    ghat = torch.zeros(1, device=DEV)
    seen = []
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "debug_fail_step_call", fail_at)
        with pytest.raises(B.AgzoError) as e:
            B.agzo_step(ctx, layers, seed=3, eps=1e-2, lr=1e-3, K=2, mode=mode,
                        loss_fn=lambda phase, slot, stream: seen.append(phase),
                        d_losses2=losses, d_ghat=ghat)
        assert e.value.status == B.AGZO_ERR_CUDA
        torch.cuda.synchronize()
        moved = np.abs(to_host(Wd) - W0).max()
        assert moved <= 1e-7, moved                      # back at W within fp32 rounding
        # the context keeps working, and a step without the injected failure does move W
        B.agzo_set_option(ctx, "debug_fail_step_call", 0)

        def loss_fn(phase, slot, stream):
            losses[slot] = 1.0 + 0.25 * slot

        B.agzo_step(ctx, layers, seed=3, eps=1e-2, lr=1e-3, K=2, mode=mode, loss_fn=loss_fn,
                    d_losses2=losses, d_ghat=ghat)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    assert np.abs(to_host(Wd) - W0).max() > 1e-6


def test_mlp_master_compute_pair_ten_steps():
    """Ten AGZO steps on the 8-layer MLP, seeds 0..9, checked in lock step.

    With eps = 1e-3 the shift eps*Delta is below one bf16 ulp of most weights, so f+ - f- is
    a few 1e-7 of f and a handful of compute-copy elements that round to the other neighbour
    move ghat by percents: two free-running implementations cannot agree on ghat to 1e-3
    here.  Each stage is therefore compared on the same inputs: Algorithm 1 on the device's
    X, the passes on the device's V and ghat, and ghat itself through the oracle's forward
    on the device's perturbed compute copies."""
    n_layers, width, m = 8, 1024, 16 * 256
    r, eps, lr, K = 8, 1e-3, 1e-4, 3
    Ws, x0, target = WL.mlp_problem(seed=0, n_layers=n_layers, width=width, m=m)

    W32 = [torch.from_numpy(w).to(DEV) for w in Ws]
    W16 = [w.to(torch.bfloat16) for w in W32]
    Xb = [torch.zeros(m, width, device=DEV, dtype=torch.bfloat16) for _ in range(n_layers)]
    Vd = [torch.zeros(r, width, device=DEV) for _ in range(n_layers)]
    x0d = torch.from_numpy(x0).to(DEV)
    tgt = torch.from_numpy(target).to(DEV).double()
    layers = [B.make_layer(W=W32[i], W16=W16[i], X=Xb[i], V=Vd[i], r=r, layer_id=i)
              for i in range(n_layers)]
    losses = torch.zeros(2, device=DEV, dtype=torch.float64)
    ghat = torch.zeros(1, device=DEV)
    snap = {}

    def gpu_loss(phase, slot, stream):      # the caller's model: bf16 storage, exact products
        snap[phase] = [to_host(w) for w in W16]
        h = x0d.double()
        for i in range(n_layers):
            hb = h.to(torch.float32).to(torch.bfloat16)
            if phase == 0:
                Xb[i].copy_(hb)
            h = hb.double() @ W16[i].double().t()
            if i + 1 < n_layers:
                h = torch.nn.functional.gelu(h)
        losses[slot] = ((h - tgt) ** 2).mean()

    def cpu_loss(ws):
        return O.mse_loss(O.mlp_forward(ws, x0, bf16_compute=True), target)

    worst = {"proj": 0.0, "ghat": 0.0, "loss": 0.0}
    with Ctx(layers) as ctx:
        arr = B.layer_array(layers)
        for seed in range(10):
            before32 = [to_host(w) for w in W32]
            B.agzo_step(ctx, layers, seed=seed, eps=eps, lr=lr, K=K, mode=0, loss_fn=gpu_loss,
                        d_losses2=losses, d_ghat=ghat, arr=arr)
            fp, fm = [float(v) for v in losses.cpu()]
            g = np.float32(float(ghat))
            check = range(n_layers) if seed in (0, 9) else (seed % n_layers,)
            for i in check:
                Vg = to_host(Vd[i])
                Vo = O.extract_subspace(to_host(Xb[i]), r, K, seed, i)
                worst["proj"] = max(worst["proj"], projector_distance(Vg, Vo))
                assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
                assert np.array_equal(snap[0][i], O.round_bf16(before32[i]))
                fl = cancellation_floor(before32[i], eps, seed, i, Vg)
                assert_weights_match(snap[1][i], O.apply_direction(before32[i], Vg, seed, i, np.float32(eps), "bf16"), "bf16", floor=fl)
                assert_weights_match(snap[2][i], O.apply_direction(before32[i], Vg, seed, i, np.float32(-eps), "bf16"), "bf16", floor=fl)
                c = np.float32(-float(np.float32(lr)) * float(g))
                want32 = O.apply_direction(before32[i], Vg, seed, i, c, "f32")
                assert_weights_match(to_host(W32[i]), want32, "f32",
                                     floor=cancellation_floor(before32[i], c, seed, i, Vg))
                assert np.array_equal(to_host(W16[i]), O.round_bf16(to_host(W32[i])))
            # ghat through the oracle's forward on the device's perturbed compute copies
            fp_o, fm_o = cpu_loss(snap[1]), cpu_loss(snap[2])
            worst["loss"] = max(worst["loss"], abs(fp - fp_o) / fp_o, abs(fm - fm_o) / fm_o)
            g_o = float(O.ghat_two_point(fp_o, fm_o, eps))
            worst["ghat"] = max(worst["ghat"], abs(float(g) - g_o) / abs(g_o))
        assert B.agzo_poll(ctx) == B.AGZO_OK
    assert worst["proj"] <= 1e-3, worst
    assert worst["ghat"] <= 1e-3, worst


def test_pair_passes_match_oracle_in_lock_step():
    # the three pair-mode passes against the oracle with the same V and ghat on both sides
    d_out, d_in, r, seed = 384, 1024, 8, 4
    W0 = (WL.gaussian_weights(d_out, d_in, 1 / 32.0, seed=2, bf16=False))
    Vh = O.extract_subspace(WL.plain_activations(64, d_in, seed=2), r, 1, 3, 6)
    Wd, _ = to_dev(W0, False)
    W16d = Wd.to(torch.bfloat16)
    Vd, _ = to_dev(Vh, False)
    layers = [B.make_layer(W=Wd, W16=W16d, V=Vd, r=r, layer_id=6)]
    ghat = torch.tensor([2.5], device=DEV)
    with Ctx(layers) as ctx:
        B.agzo_perturb(ctx, layers, seed, 1e-3)
        assert np.array_equal(to_host(Wd), W0)                       # master untouched
        fl = cancellation_floor(W0, 1e-3, seed, 6, Vh)
        assert_weights_match(to_host(W16d), O.apply_direction(W0, Vh, seed, 6, np.float32(1e-3), "bf16"), "bf16", floor=fl)
        B.agzo_perturb(ctx, layers, seed, -1e-3)
        assert_weights_match(to_host(W16d), O.apply_direction(W0, Vh, seed, 6, np.float32(-1e-3), "bf16"), "bf16", floor=fl)
        B.agzo_restore(ctx, layers, seed, 1e-3)
        assert np.array_equal(to_host(W16d), O.round_bf16(W0))
        B.agzo_restore_update(ctx, layers, seed, 1e-3, 1e-2, 0, ghat)
        W1 = O.apply_direction(W0, Vh, seed, 6, np.float32(-1e-2 * np.float32(2.5)), "f32")
        assert_weights_match(to_host(Wd), W1, "f32", floor=cancellation_floor(W0, 2.5e-2, seed, 6, Vh))
        assert (to_host(W16d) != O.round_bf16(to_host(Wd))).sum() == 0
