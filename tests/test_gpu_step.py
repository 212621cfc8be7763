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

from gpu_helpers import DEV, Ctx, assert_weights_match, projector_distance, to_dev, to_host

pytestmark = pytest.mark.gpu


def _slot_writer(d_out3):
    base = d_out3.data_ptr()

    def write(d_loss_ptr, value):
        d_out3[(d_loss_ptr - base) // 4] = value.to(torch.float32)
    return write


@pytest.mark.parametrize("mode", [0, 1])
def test_single_fp32_layer_least_squares_step(mode):
    X, Yt, W0 = WL.least_squares_problem(seed=0)          # 256 -> 256, 512 tokens
    r, eps, lr, K, seed = 4, 1e-3, 5e-4, 3, 0
    Xd, _ = to_dev(X, False)
    Yd = torch.from_numpy(Yt).to(DEV).double()
    Wd, _ = to_dev(W0, False)
    Vd = torch.zeros(r, 256, device=DEV)
    layers = [B.make_layer(W=Wd, X=Xd, V=Vd, r=r, layer_id=0)]
    out3 = torch.zeros(3, device=DEV)
    write = _slot_writer(out3)
    seen = []

    def loss_fn(phase, d_loss, stream):
        seen.append(phase)
        E = Xd.double() @ Wd.double().t() - Yd
        write(d_loss, (E * E).sum() / (2 * X.shape[0]))

    with Ctx(layers) as ctx:
        B.agzo_step(ctx, layers, seed=seed, eps=eps, lr=lr, K=K, mode=mode, loss_fn=loss_fn,
                    d_out3=out3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    assert seen == ([0, 1, 2] if mode == 0 else [0, 1])

    L = {"W": W0.copy(), "X": X, "r": r, "layer_id": 0, "storage": "f32"}
    res = O.agzo_step([L], lambda ws: O.least_squares_loss(ws[0], X, Yt), seed, eps, lr, K, mode)
    f_plus, f_other, g = [float(v) for v in out3.cpu()]
    assert abs(f_plus - res["f_plus"]) <= 1e-6 * abs(res["f_plus"])
    assert abs(f_other - res["f_other"]) <= 1e-6 * abs(res["f_other"])
    assert abs(g - float(res["ghat"])) <= 1e-3 * abs(float(res["ghat"]))
    Vg = to_host(Vd)
    assert projector_distance(Vg, res["V"][0]) <= 1e-3
    assert np.abs(to_host(Wd) - L["W"]).max() <= 1e-6
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
    out3 = torch.zeros(3, device=DEV)

    def loss_fn(phase, d_loss, stream):
        if phase == 2:
            raise RuntimeError("forward failed")

    with Ctx(layers) as ctx:
        with pytest.raises(B.AgzoError) as e:
            B.agzo_step(ctx, layers, seed=3, eps=1e-2, lr=1e-3, K=2, mode=0, loss_fn=loss_fn,
                        d_out3=out3)
        assert e.value.status == B.AGZO_ERR_CALLBACK
    assert np.abs(to_host(Wd) - W0).max() <= 1e-7       # back at W within fp32 rounding


def test_mlp_master_compute_pair_ten_steps():
    n_layers, width, m = 8, 1024, 16 * 256
    r, eps, lr, K = 8, 1e-3, 1e-4, 3
    Ws, x0, target = WL.mlp_problem(seed=0, n_layers=n_layers, width=width, m=m)

    # ---- device side: the caller's model in torch (bf16 storage, exact products)
    W32 = [torch.from_numpy(w).to(DEV) for w in Ws]
    W16 = [w.to(torch.bfloat16) for w in W32]
    Xb = [torch.zeros(m, width, device=DEV, dtype=torch.bfloat16) for _ in range(n_layers)]
    Vd = [torch.zeros(r, width, device=DEV) for _ in range(n_layers)]
    x0d = torch.from_numpy(x0).to(DEV)
    tgt = torch.from_numpy(target).to(DEV).double()
    layers = [B.make_layer(W=W32[i], W16=W16[i], X=Xb[i], V=Vd[i], r=r, layer_id=i)
              for i in range(n_layers)]
    out3 = torch.zeros(3, device=DEV)
    write = _slot_writer(out3)

    def gpu_loss(phase, d_loss, stream):
        h = x0d.double()
        for i in range(n_layers):
            hb = h.to(torch.float32).to(torch.bfloat16)
            if phase == 0:
                Xb[i].copy_(hb)
            h = hb.double() @ W16[i].double().t()
            if i + 1 < n_layers:
                h = torch.nn.functional.gelu(h)
        write(d_loss, ((h - tgt) ** 2).mean())

    # ---- oracle side
    OL = [{"W": Ws[i].copy(), "W16": O.round_bf16(Ws[i]), "X": None, "r": r, "layer_id": i,
           "storage": "f32"} for i in range(n_layers)]

    def cpu_loss(ws):
        out, ins = O.mlp_forward(ws, x0, bf16_compute=True, collect_inputs=True)
        for i in range(n_layers):
            OL[i]["X"] = ins[i]
        return O.mse_loss(out, target)

    g_gpu, g_cpu = [], []
    with Ctx(layers) as ctx:
        arr = B.layer_array(layers)
        for seed in range(10):
            B.agzo_step(ctx, layers, seed=seed, eps=eps, lr=lr, K=K, mode=0, loss_fn=gpu_loss,
                        d_out3=out3, arr=arr)
            res = O.agzo_step(OL, cpu_loss, seed, eps, lr, K, 0)
            fp, fm, g = [float(v) for v in out3.cpu()]
            g_gpu.append(g)
            g_cpu.append(float(res["ghat"]))
            if seed in (0, 9):
                for i in (0, 3, 7):
                    assert projector_distance(to_host(Vd[i]), res["V"][i]) <= 1e-3
                    assert np.array_equal(to_host(Xb[i]), OL[i]["X"]) or \
                        (to_host(Xb[i]) != OL[i]["X"]).mean() < 1e-4
            assert abs(fp - res["f_plus"]) <= 1e-5 * abs(res["f_plus"])
        assert B.agzo_poll(ctx) == B.AGZO_OK
    g_gpu, g_cpu = np.array(g_gpu), np.array(g_cpu)
    scale = np.sqrt((g_cpu ** 2).mean())
    assert np.all(np.abs(g_gpu - g_cpu) <= 1e-3 * np.maximum(np.abs(g_cpu), scale)), (g_gpu, g_cpu)
    for i in range(n_layers):
        assert np.abs(to_host(W32[i]) - OL[i]["W"]).max() <= 1e-6
        d = to_host(W16[i]) != OL[i]["W16"]
        assert d.mean() <= 1e-3


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
        assert_weights_match(to_host(W16d), O.apply_direction(W0, Vh, seed, 6, np.float32(1e-3), "bf16"), "bf16")
        B.agzo_perturb(ctx, layers, seed, -1e-3)
        assert_weights_match(to_host(W16d), O.apply_direction(W0, Vh, seed, 6, np.float32(-1e-3), "bf16"), "bf16")
        B.agzo_restore(ctx, layers, seed, 1e-3)
        assert np.array_equal(to_host(W16d), O.round_bf16(W0))
        B.agzo_restore_update(ctx, layers, seed, 1e-3, 1e-2, 0, ghat)
        W1 = O.apply_direction(W0, Vh, seed, 6, np.float32(-1e-2 * np.float32(2.5)), "f32")
        assert_weights_match(to_host(Wd), W1, "f32")
        assert (to_host(W16d) != O.round_bf16(to_host(Wd))).sum() == 0
