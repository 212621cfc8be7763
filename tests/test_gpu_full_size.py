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
    tc = r >= 3                      # the default options send these layers to the tensor-core kernel
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


# ---- the Qwen3-1.7B-shaped configuration at its own shapes: d_in 2048 / 6144, d_out up to 6144,
# m = 16 x 1024 tokens, planted rank 64, r in {4, 8, 16}
@pytest.mark.parametrize("d_in,r", [(2048, 4), (2048, 16), (6144, 8), (6144, 16)])
def test_extraction_of_a_1p7b_shaped_layer(d_in, r):
    cfg = WL.QWEN3_1P7B
    X = WL.planted_activations(cfg.m, d_in, cfg.planted_rank, seed=d_in + r, bf16=True)
    Xd, _ = to_dev(X, True)
    Vd = torch.zeros(r, d_in, device=DEV)
    layers = [B.make_layer(X=Xd, V=Vd, r=r, layer_id=11)]
    with Ctx(layers) as ctx:
        B.agzo_extract_subspace(ctx, layers, 3, 3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    Vg = to_host(Vd)
    Vo = O.extract_subspace(X, r, 3, 3, 11)
    assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
    assert projector_distance(Vg, Vo) <= 1e-3
    assert np.abs(Vg - Vo).max() <= 1e-3


@pytest.mark.parametrize("d_out,d_in,r", [(6144, 2048, 4), (6144, 2048, 8), (6144, 2048, 16),
                                           (2048, 6144, 4), (2048, 6144, 8), (2048, 6144, 16), (1024, 2048, 8)])
def test_in_place_passes_on_a_1p7b_shaped_layer(d_out, d_in, r):
    seed, layer_id, eps = 6, 4, 1e-3
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=d_out + r, bf16=True)
    Vh = O.extract_subspace(WL.plain_activations(256, d_in, seed=r), r, 1, 3, layer_id)
    Wd, _ = to_dev(W0, True)
    Vd, _ = to_dev(Vh, False)
    layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=layer_id)]
    ghat = torch.tensor([-0.27], device=DEV)
    rel = 2.0 ** -16                 # tensor-core pass (r >= 3)
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
        c = O.update_coefficient(eps, 1e-3, np.float32(-0.27), 0)
        want = O.apply_direction(cur, Vh, seed, layer_id, c, "bf16")
        assert_weights_match(to_host(Wd), want, "bf16", frac=tc_mismatch_bound(want, c, seed, layer_id, Vh),
                             floor=cancellation_floor(cur, c, seed, layer_id, Vh, rel))
        assert B.agzo_poll(ctx) == B.AGZO_OK


def test_every_layer_of_the_0p6b_shaped_set_in_one_grouped_launch():
    """All 196 layers of the Qwen3-0.6B-shaped set (0.44 G bf16 weights) perturbed by one call, every
    weight compared with the oracle; the layer shapes repeat per block, so the directions are
    computed per distinct (layer_id, shape) as the library sees them."""
    cfg = WL.QWEN3_0P6B
    r, seed, eps = 8, 11, 1e-3
    specs = cfg.layers()
    host_W, dev_W, dev_V, host_V, layers = [], [], [], [], []
    Vcache = {}
    for i, (name, d_in, d_out) in enumerate(specs):
        W0 = WL.gaussian_weights(d_out, d_in, cfg.w_std, seed=1000 + i, bf16=True)
        if d_in not in Vcache:      # any orthonormal basis will do for the pass; one per input width
            Vcache[d_in] = O.extract_subspace(WL.plain_activations(64, d_in, seed=d_in), r, 1, 3, 0)
        Vh = Vcache[d_in]
        Wd, _ = to_dev(W0, True)
        Vd, _ = to_dev(Vh, False)
        host_W.append(W0); host_V.append(Vh); dev_W.append(Wd); dev_V.append(Vd)
        layers.append(B.make_layer(W=Wd, V=Vd, r=r, layer_id=i))
    with Ctx(layers) as ctx:
        B.agzo_perturb(ctx, layers, seed, eps)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    for i in range(len(specs)):
        want = O.apply_direction(host_W[i], host_V[i], seed, i, np.float32(eps), "bf16")
        assert_weights_match(to_host(dev_W[i]), want, "bf16",
                             floor=cancellation_floor(host_W[i], eps, seed, i, host_V[i], 2.0 ** -16))


def test_extraction_of_two_blocks_of_the_0p6b_shaped_set_with_shared_inputs():
    """Blocks 0 and 27 of the Qwen3-0.6B-shaped set in one call, q/k/v and gate/up reading one
    activation buffer each as in a transformer block."""
    cfg = WL.QWEN3_0P6B
    r, K, seed = 8, 3, 4
    layers, keep, checks = [], [], []
    for blk in (0, 27):
        Xq = WL.planted_activations(cfg.m, 1024, cfg.planted_rank, seed=100 + blk, bf16=True)
        Xo = WL.planted_activations(cfg.m, 2048, cfg.planted_rank, seed=200 + blk, bf16=True)
        Xg = WL.planted_activations(cfg.m, 1024, cfg.planted_rank, seed=300 + blk, bf16=True)
        Xd = WL.planted_activations(cfg.m, 3072, cfg.planted_rank, seed=400 + blk, bf16=True)
        dq, do_, dg, dd = (to_dev(x, True)[0] for x in (Xq, Xo, Xg, Xd))
        for j, (Xh, Xdev) in enumerate([(Xq, dq), (Xq, dq), (Xq, dq), (Xo, do_), (Xg, dg), (Xg, dg), (Xd, dd)]):
            lid = 7 * blk + j
            V = torch.zeros(r, Xh.shape[1], device=DEV)
            keep.append((Xdev, V))
            layers.append(B.make_layer(X=Xdev, V=V, r=r, layer_id=lid))
            checks.append((Xh, V, lid))
    with Ctx(layers) as ctx:
        B.agzo_extract_subspace(ctx, layers, seed, K)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    for Xh, V, lid in checks:
        Vg = to_host(V)
        Vo = O.extract_subspace(Xh, r, K, seed, lid)
        assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
        assert projector_distance(Vg, Vo) <= 1e-3
        assert np.abs(Vg - Vo).max() <= 1e-3


def test_whole_batch_token_slabs_with_a_ragged_second_slab():
    # 32 layers of d_in = 4096 have 1024 column blocks between them: the X^T T product then takes token
    # slabs of up to 16384 tokens, here one full slab and a ragged one of 520.  The layers read one
    # buffer but are not grouped (share_inputs off), so each sweeps it alone with its own Omega.
    m, d_in, r, K, seed, n = 16384 + 520, 4096, 4, 1, 9, 32
    X = WL.planted_activations(m, d_in, 16, seed=77, bf16=True)
    Xd, _ = to_dev(X, True)
    Vds = [torch.zeros(r, d_in, device=DEV) for _ in range(n)]
    layers = [B.make_layer(X=Xd, V=Vds[i], r=r, layer_id=100 + i) for i in range(n)]
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "share_inputs", 0)
        B.agzo_extract_subspace(ctx, layers, seed, K)
        torch.cuda.synchronize()
        assert B.agzo_poll(ctx) == B.AGZO_OK
    for i in (0, 17, 31):
        Vg = to_host(Vds[i])
        Vo = O.extract_subspace(X, r, K, seed, 100 + i)
        assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
        assert projector_distance(Vg, Vo) <= 1e-3


@pytest.mark.parametrize("r", [16, 64])
def test_whole_8b_shaped_set_as_the_benchmark_runs_it_sampled_layers(r):
    """The benchmark's own workload and launch configuration: all 252 layers of the Qwen3-8B-shaped
    set resident (13.9 GB of weights, 43.5 GB of activations, generated on the device as bench.py
    does), r = 16 (the timed case) and r = 64 (staged R operands, three-stage products), K = 3,
    default options, one extraction and one pass over the whole set.  The
    oracle recomputes sampled layers from the same bytes: the first and the last layer, a
    down-projection (d_in = 12288) and layers from the middle (other waves, other streams)."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    torch.cuda.empty_cache()          # blocks cached by earlier tests count as used
    free, _ = torch.cuda.mem_get_info()
    if free < 75 * 2 ** 30:
        pytest.skip("needs 75 GB of free device memory")
    cfg = WL.QWEN3_8B
    K, seed, eps = 3, 123, 1e-3
    dev = torch.device(DEV)
    Ws, Xs, Vs, layers = bench.build_layer_set(cfg, r, dev)
    sample = [0, 6, 101, 125, 251]
    W_before = {i: to_host(Ws[i]) for i in sample}
    arr = B.layer_array(layers)
    with Ctx(layers) as ctx:
        B.agzo_extract_subspace(ctx, layers, seed, K, arr=arr)
        B.agzo_perturb(ctx, layers, seed, eps, arr=arr)
        torch.cuda.synchronize()
        assert B.agzo_poll(ctx) == B.AGZO_OK
    for i in sample:
        X = Xs[i].float().cpu().numpy()
        Vg = to_host(Vs[i])
        Vo = O.extract_subspace(X, r, K, seed, i)
        assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5, i
        assert projector_distance(Vg, Vo) <= 1e-3, i
        want = O.apply_direction(W_before[i], Vg, seed, i, np.float32(eps), "bf16")
        assert_weights_match(to_host(Ws[i]), want, "bf16",
                             floor=cancellation_floor(W_before[i], eps, seed, i, Vg, 2.0 ** -16))
    del Ws, Xs, Vs
    torch.cuda.empty_cache()
