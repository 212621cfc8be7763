"""GPU-vs-oracle parity through the C ABI, on seeded inputs.

Tolerances (stated as numbers):
  Philox words and the element -> (block, lane) map ........ bit-exact
  normals ................................................... |d| <= 2e-6 * max(1, |g|)
  V (projector) ............................................. ||VtV_gpu - VtV_cpu||_F <= 1e-3
  V orthonormality .......................................... max |V V^T - I| <= 1e-5
  bf16 weights after a pass (same V on both sides) .......... <= 1 bf16 ulp, <= 1e-3 of them differ
  fp32 weights .............................................. <= 4 fp32 ulp
    (where w + c*z cancels, the ulp of the result is below the rounding noise of the
     operands; there the bound is 2^-20 * max(|w|, |c| |G||V|) for the CUDA-core kernels and
     2^-16 * the same for the tensor-core kernel with its hi+lo bf16 factors, see gpu_helpers)
  ghat ...................................................... 1e-3 relative
"""
import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import (DEV, Ctx, assert_weights_match, bf16_ulp_distance, cancellation_floor,
                         projector_distance, tc_mismatch_bound, to_dev, to_host)

pytestmark = pytest.mark.gpu


# ----------------------------------------------------------------------------- generator
def test_philox_words_bit_exact():
    V = torch.zeros(1, 8, device=DEV)
    with Ctx([B.make_layer(V=V, r=1, layer_id=0, d_in=8)]) as ctx:
        for seed, layer, tag, first, n in [(0, 0, 0, 0, 4099), (0xDEADBEEFCAFEF00D, 251, 1, 0, 1000),
                                           (7, 3, 2, (1 << 34) + 5, 257), (1, 0xFFFFFFFF, 0, 3, 64)]:
            got = B.agzo_debug_philox(ctx, seed, layer, tag, first, n).cpu().numpy().view(np.uint32)
            want = O.philox_words(seed, layer, tag, n, first=first)
            assert np.array_equal(got, want)
        assert B.agzo_debug_philox(ctx, 1, 1, 1, 0, 0).numel() == 0


def test_gaussians_match_the_oracle():
    V = torch.zeros(1, 8, device=DEV)
    with Ctx([B.make_layer(V=V, r=1, layer_id=0, d_in=8)]) as ctx:
        n = 1 << 20
        for seed, layer, tag in [(0, 0, 0), (12345678901234, 17, 1), (3, 9, 2)]:
            got = B.agzo_debug_gaussian(ctx, seed, layer, tag, 0, n).cpu().numpy()
            want = O.gaussian_stream(seed, layer, tag, n)
            err = np.abs(got.astype(np.float64) - want) / np.maximum(1.0, np.abs(want))
            assert err.max() <= 2e-6


# ----------------------------------------------------------------------------- in-place passes
RMW_CASES = [
    # d_out, d_in, r, storage, pitch_extra, label
    (300, 1024, 8, "bf16", 0, "two column tiles, ragged rows"),
    (257, 520, 4, "bf16", 8, "ragged tile edge, padded pitch"),
    (64, 256, 1, "bf16", 0, "r=1"),
    (130, 512, 2, "bf16", 0, "r=2"),
    (96, 768, 3, "bf16", 0, "r=3 (padded rank chunk)"),
    (520, 1536, 16, "bf16", 0, "r=16"),
    (300, 640, 24, "bf16", 0, "r=24 shared-memory kernel"),
    (260, 512, 64, "bf16", 0, "r=64"),
    (256, 256, 4, "f32", 0, "fp32 storage"),
    (100, 136, 8, "f32", 4, "fp32 padded pitch"),
    (37, 50, 5, "bf16", 1, "unaligned: scalar kernel"),
    (19, 27, 3, "f32", 0, "unaligned fp32"),
]
# the tensor-core kernel (bf16 weights, 16-byte aligned rows): every rank class, ragged tiles,
# several row chunks and column panels per layer
RMW_TC_CASES = [c + (2,) for c in RMW_CASES if c[3] == "bf16" and c[4] != 1] + [
    (1300, 1096, 16, "bf16", 8, "two row chunks, five panels, ragged box", 2),
    (2200, 520, 8, "bf16", 0, "three row chunks", 2),
    (300, 384, 40, "bf16", 0, "three K atoms", 2),
    (200, 192, 33, "bf16", 0, "odd rank above 32", 2),
    (130, 72, 7, "bf16", 0, "odd rank, Philox blocks straddle rows", 2),
]


@pytest.mark.parametrize("d_out,d_in,r,storage,extra,label,path",
                         [c + (1,) for c in RMW_CASES] + RMW_TC_CASES)
def test_perturb_restore_update_match_oracle(d_out, d_in, r, storage, extra, label, path):
    seed, layer_id = 11, 5
    bf = storage == "bf16"
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=d_out + d_in, bf16=bf)
    Vh = O.extract_subspace(WL.plain_activations(max(2 * r, 32), d_in, seed=r), r, 1, 3, layer_id)
    Wd, Wbuf = to_dev(W0, bf, pitch=d_in + extra if extra else None)
    Vd, Vbuf = to_dev(Vh, False, pitch=d_in + (4 if extra else 0) if extra else None)
    layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=layer_id)]
    ghat = torch.tensor([0.73], device=DEV)
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "rmw_path", path)
        eps = 1e-3
        def floor(w_in, c):
            return cancellation_floor(w_in, c, seed, layer_id, Vh, rel=2.0 ** -16 if path == 2 else 2.0 ** -20)

        B.agzo_perturb(ctx, layers, seed, eps)
        want = O.apply_direction(W0, Vh, seed, layer_id, np.float32(eps), storage)
        assert_weights_match(to_host(Wd), want, storage, floor=floor(W0, eps))
        # the oracle is fed the GPU's weights from here on so that mismatches do not compound
        cur = to_host(Wd)
        B.agzo_perturb(ctx, layers, seed, -2 * eps)
        want = O.apply_direction(cur, Vh, seed, layer_id, np.float32(-2 * eps), storage)
        assert_weights_match(to_host(Wd), want, storage, floor=floor(cur, 2 * eps))
        cur = to_host(Wd)
        B.agzo_restore(ctx, layers, seed, -eps)
        want = O.apply_direction(cur, Vh, seed, layer_id, np.float32(eps), storage)
        assert_weights_match(to_host(Wd), want, storage, floor=floor(cur, eps))
        cur = to_host(Wd)
        B.agzo_update(ctx, layers, seed, 5e-2, ghat)
        c = np.float32(-5e-2 * np.float32(0.73))
        want = O.apply_direction(cur, Vh, seed, layer_id, c, storage)
        # a step this large (c*Delta as big as W itself) shows the tensor-core kernel's split
        # factors: the share of results on the other grid point has its own derived bound
        frac = tc_mismatch_bound(want, c, seed, layer_id, Vh) if path == 2 else 1e-3
        assert_weights_match(to_host(Wd), want, storage, frac=frac, floor=floor(cur, c))
        assert B.agzo_poll(ctx) == B.AGZO_OK
    if extra:  # the padding around W and V is untouched
        w = Wbuf.float()
        assert bool((w[0] == 7).all() and (w[-1] == 7).all() and (w[:, d_in:] == 7).all())
        assert bool((Vbuf[0] == 7).all() and (Vbuf[:, d_in:] == 7).all())


def test_staged_R_is_rewritten_when_the_seed_changes_or_extraction_used_the_scratch():
    d_out, d_in, r, layer_id = 300, 640, 24, 2
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=8, bf16=True)
    X = WL.planted_activations(512, d_in, 16, seed=4, bf16=True)
    Wd, _ = to_dev(W0, True)
    Xd, _ = to_dev(X, True)
    Vd = torch.zeros(r, d_in, device=DEV)
    layers = [B.make_layer(W=Wd, X=Xd, V=Vd, r=r, layer_id=layer_id)]
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "rmw_path", 2)
        B.agzo_extract_subspace(ctx, layers, 1, 2)
        torch.cuda.synchronize()
        Vh = Vd.cpu().numpy()

        def one_pass(seed, c):
            before = to_host(Wd)
            B.agzo_perturb(ctx, layers, seed, c)
            want = O.apply_direction(before, Vh, seed, layer_id, np.float32(c), "bf16")
            assert_weights_match(to_host(Wd), want, "bf16",
                                 floor=cancellation_floor(before, c, seed, layer_id, Vh, rel=2.0 ** -16))

        one_pass(5, 1e-3)          # writes the images of seed 5
        one_pass(5, -2e-3)         # finds them
        one_pass(6, 1e-3)          # another seed: rewritten
        one_pass(5, 1e-3)          # and back
        B.agzo_extract_subspace(ctx, layers, 1, 2)     # the scratch now holds extraction's panels
        torch.cuda.synchronize()
        assert np.array_equal(Vd.cpu().numpy(), Vh)
        one_pass(5, -1e-3)         # same seed as the last pass, yet rewritten
        assert B.agzo_poll(ctx) == B.AGZO_OK


@pytest.mark.parametrize("stage", [1, 2])
def test_tensor_core_pass_with_and_without_staged_R(stage):
    # stage 2: R tiles written to scratch by a fill kernel even at r = 8; stage 1: regenerated in the pass at r = 40
    d_out, d_in, r = (300, 640, 8) if stage == 2 else (300, 384, 40)
    seed, layer_id = 4, 2
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=8, bf16=True)
    Vh = O.extract_subspace(WL.plain_activations(2 * r + 16, d_in, seed=r), r, 1, 3, layer_id)
    Wd, _ = to_dev(W0, True)
    Vd, _ = to_dev(Vh, False)
    layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=layer_id)]
    with Ctx(layers, extra=1 << 20) as ctx:
        B.agzo_set_option(ctx, "rmw_path", 2)
        B.agzo_set_option(ctx, "rmw_stage_r", stage)
        for c in (1e-3, -2e-3):
            before = to_host(Wd)
            B.agzo_perturb(ctx, layers, seed, c)
            want = O.apply_direction(before, Vh, seed, layer_id, np.float32(c), "bf16")
            assert_weights_match(to_host(Wd), want, "bf16",
                                 floor=cancellation_floor(before, c, seed, layer_id, Vh, rel=2.0 ** -16))
        assert B.agzo_poll(ctx) == B.AGZO_OK


def test_restore_update_fused_modes():
    d_out, d_in, r, seed = 200, 512, 8, 21
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=1, bf16=True)
    Vh = O.extract_subspace(WL.plain_activations(64, d_in, seed=2), r, 1, 3, 0)
    Vd, _ = to_dev(Vh, False)
    g = np.float32(-1.37)
    ghat = torch.tensor([float(g)], device=DEV)
    for mode in (0, 1):
        Wd, _ = to_dev(W0, True)
        layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=0)]
        with Ctx(layers) as ctx:
            B.agzo_restore_update(ctx, layers, seed, 1e-3, 2e-3, mode, ghat)
            c = O.update_coefficient(1e-3, 2e-3, g, mode)
            want = O.apply_direction(W0, Vh, seed, 0, c, "bf16")
            assert_weights_match(to_host(Wd), want, "bf16",
                                 floor=cancellation_floor(W0, c, seed, 0, Vh, rel=2.0 ** -16))


def test_many_layers_one_launch_mixed_shapes_and_ranks():
    rng = np.random.default_rng(0)
    shapes = [(128, 256, 2), (300, 512, 8), (64, 1024, 8), (257, 264, 5), (33, 40, 3), (512, 512, 1)]
    host, layers, devW = [], [], []
    for i, (do, di, r) in enumerate(shapes):
        W0 = WL.gaussian_weights(do, di, 0.02, seed=i, bf16=True)
        Vh = O.extract_subspace(WL.plain_activations(32, di, seed=i), r, 1, 9, 100 + i)
        Wd, _ = to_dev(W0, True)
        Vd, _ = to_dev(Vh, False)
        host.append((W0, Vh, r))
        devW.append((Wd, Vd))
        layers.append(B.make_layer(W=Wd, V=Vd, r=r, layer_id=100 + i))
    with Ctx(layers) as ctx:
        B.agzo_perturb(ctx, layers, 77, 2e-3)
        for i, (W0, Vh, r) in enumerate(host):
            want = O.apply_direction(W0, Vh, 77, 100 + i, np.float32(2e-3), "bf16")
            assert_weights_match(to_host(devW[i][0]), want, "bf16",
                                 floor=cancellation_floor(W0, 2e-3, 77, 100 + i, Vh,
                                                          rel=2.0 ** -16 if r >= 3 else 2.0 ** -20))


def test_perturb_is_deterministic_and_regenerates_the_same_direction():
    d_out, d_in, r = 512, 1024, 8
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=3, bf16=False)
    Vh = O.extract_subspace(WL.plain_activations(64, d_in, seed=2), r, 1, 3, 0)
    Vd, _ = to_dev(Vh, False)
    outs = []
    for _ in range(2):
        Wd, _ = to_dev(W0, False)
        layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=1)]
        with Ctx(layers) as ctx:
            B.agzo_perturb(ctx, layers, 5, 1e-2)
            outs.append(to_host(Wd))
            B.agzo_restore(ctx, layers, 5, 1e-2)
            back = to_host(Wd)
    assert np.array_equal(outs[0], outs[1])
    assert np.abs(back - W0).max() < 1e-8     # fp32: W + cZ - cZ returns to W within rounding


def test_dense_direction():
    w0 = WL.gaussian_weights(1, 100003, 0.5, seed=9, bf16=True).reshape(-1)
    wd = torch.from_numpy(w0).to(DEV).to(torch.bfloat16)
    V = torch.zeros(1, 8, device=DEV)
    scale = torch.tensor([-2.0], device=DEV)
    with Ctx([B.make_layer(V=V, r=1, layer_id=0, d_in=8)]) as ctx:
        B.agzo_perturb_dense(ctx, wd, 4, 33, 1e-2)
        want = O.apply_dense(w0, 4, 33, np.float32(1e-2), "bf16")
        d = bf16_ulp_distance(to_host(wd), want)
        assert d.max() <= 1 and (d > 0).mean() < 1e-3
        w1 = to_host(wd)
        B.agzo_perturb_dense(ctx, wd, 4, 33, 1e-2, d_scale=scale)
        want = O.apply_dense(w1, 4, 33, np.float32(-2e-2), "bf16")
        d = bf16_ulp_distance(to_host(wd), want)
        assert d.max() <= 1 and (d > 0).mean() < 1e-3


@pytest.mark.parametrize("n,bf16,offset", [(100003, False, 0), (4099, True, 1), (4099, False, 3), (5, True, 0), (8, True, 0),
                                             (1 << 20, True, 0)])
def test_dense_direction_sizes_dtypes_and_alignments(n, bf16, offset):
    # vector path (16-byte aligned, eight elements per thread) with its scalar tail, the scalar path for a
    # vector that does not start on a 16-byte boundary, fp32 storage, tiny vectors; sentinels on both sides
    w0 = WL.gaussian_weights(1, n, 0.5, seed=n + offset, bf16=bf16).reshape(-1)
    dt = torch.bfloat16 if bf16 else torch.float32
    buf = torch.full((n + offset + 16,), 7.0, dtype=dt, device=DEV)
    wd = buf[offset:offset + n]
    wd.copy_(torch.from_numpy(w0).to(DEV).to(dt))
    V = torch.zeros(1, 8, device=DEV)
    with Ctx([B.make_layer(V=V, r=1, layer_id=0, d_in=8)]) as ctx:
        B.agzo_perturb_dense(ctx, wd, 6, 35, 3e-2)
        torch.cuda.synchronize()
    want = O.apply_dense(w0, 6, 35, np.float32(3e-2), "bf16" if bf16 else "f32")
    got = to_host(wd)
    if bf16:
        d = bf16_ulp_distance(got, want)
        assert d.max() <= 1 and (d > 0).mean() < 1e-3 + 2.0 / n
    else:
        # 4 fp32 ulp of the operands: where w + c u cancels, the result's own ulp is below the rounding of the
        # normals (a few 1e-7 relative), which no fp32 evaluation can beat
        u = np.abs(O.gen_dense(6, 35, n).astype(np.float64))
        scale = np.maximum(np.abs(w0.astype(np.float64)), 3e-2 * u)
        assert np.all(np.abs(got.astype(np.float64) - want) <= 4 * 2.0 ** -23 * scale)
    assert bool((buf[:offset] == 7).all() and (buf[offset + n:] == 7).all())


def test_gaussian_right_factor_matches_the_oracle_and_feeds_the_passes():
    specs = [(300, 640, 8), (64, 100, 3)]
    devs, layers = [], []
    for i, (do, di, r) in enumerate(specs):
        W0 = WL.gaussian_weights(do, di, 0.02, seed=30 + i, bf16=True)
        Wd, _ = to_dev(W0, True)
        Vbuf = torch.full((r + 2, di + 4), 7.0, device=DEV)
        devs.append((W0, Wd, Vbuf))
        layers.append(B.make_layer(W=Wd, V=Vbuf[1:1 + r, :di], r=r, layer_id=50 + i))
    with Ctx(layers) as ctx:
        B.agzo_fill_gaussian_basis(ctx, layers, 77)
        B.agzo_perturb(ctx, layers, 77, 1e-3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    for i, (do, di, r) in enumerate(specs):
        W0, Wd, Vbuf = devs[i]
        Vg = to_host(Vbuf[1:1 + r, :di])
        Vo = O.gen_gaussian_basis(77, 50 + i, r, di)
        assert (np.abs(Vg.astype(np.float64) - Vo) / np.maximum(1.0, np.abs(Vo))).max() <= 2e-6
        assert bool((Vbuf[0] == 7).all() and (Vbuf[-1] == 7).all() and (Vbuf[:, di:] == 7).all())
        want = O.apply_direction(W0, Vg, 77, 50 + i, np.float32(1e-3), "bf16")     # U V^T with the device's V
        assert_weights_match(to_host(Wd), want, "bf16",
                             floor=cancellation_floor(W0, 1e-3, 77, 50 + i, Vg, rel=2.0 ** -16))


def test_ghat_scalar():
    V = torch.zeros(1, 8, device=DEV)
    fp = torch.tensor([0.731234], device=DEV, dtype=torch.float64)
    fo = torch.tensor([0.729876], device=DEV, dtype=torch.float64)
    g = torch.zeros(1, device=DEV)
    with Ctx([B.make_layer(V=V, r=1, layer_id=0, d_in=8)]) as ctx:
        B.agzo_ghat(ctx, fp, fo, 1e-3, 0, g)
        want = O.ghat_two_point(0.731234, 0.729876, 1e-3)
        assert abs(g.item() - float(want)) <= 1e-6 * abs(float(want))
        B.agzo_ghat(ctx, fp, fo, 1e-3, 1, g)
        want = O.ghat_one_sided(0.731234, 0.729876, 1e-3)
        assert abs(g.item() - float(want)) <= 1e-6 * abs(float(want))


# ----------------------------------------------------------------------------- Algorithm 1
EXTRACT_CASES = [
    # m, d_in, r, K, planted, x_bf16, path
    (512, 256, 4, 3, 0, False, 1),       # the single-layer fp32 problem's shape
    (700, 520, 8, 3, 16, True, 1),       # ragged everything
    (1000, 384, 1, 3, 8, True, 1),
    (333, 200, 16, 2, 32, True, 1),
    (2048, 1024, 8, 3, 32, True, 1),
    (640, 256, 24, 1, 32, True, 1),
    (300, 128, 64, 1, 0, False, 1),
    (400, 96, 5, 0, 0, False, 1),        # K = 0: just qr(H Omega)
    # the tensor-core kernels (bf16 X, 16-byte aligned rows)
    (2048, 1024, 8, 0, 32, True, 2),     # K = 0: Omega fill + X^T T + panel QR
    (2048, 1024, 8, 1, 32, True, 2),     # K = 1 adds X Q
    (2048, 1024, 8, 3, 32, True, 2),
    (700, 520, 8, 3, 16, True, 2),       # ragged tiles, padded pitch
    (1000, 384, 1, 3, 8, True, 2),
    (333, 200, 16, 2, 32, True, 2),
    (640, 256, 24, 1, 32, True, 2),
    (512, 256, 64, 1, 0, True, 2),
    (4096, 3072, 4, 3, 32, True, 2),     # several column chunks and slabs; fused power step on clusters of 6
    (1024, 4096, 16, 2, 32, True, 2),    # fused power step, clusters of 8
    (1536, 2048, 8, 3, 32, True, 2),     # clusters of 4
    (900, 136, 3, 2, 8, True, 2),        # a single CTA per cluster, ragged token tile
    (640, 5000, 8, 2, 32, True, 2),      # clusters of 10 (beyond the portable size), ragged last slice
    (400, 8192, 16, 2, 32, True, 2),     # clusters of 16, 512-column slices
    (384, 12288, 16, 2, 32, True, 2),    # clusters of 16, 768-column slices
    (520, 9000, 4, 2, 32, True, 2),      # clusters of 12 on 768-column slices, the last one partly filled
    (512, 6144, 16, 2, 32, True, 2),     # 12 slices of 512 would overflow the exchange buffer at r = 16: 8 of 768
    (512, 6144, 8, 2, 32, True, 2),      # 8 slices of 768 keep more SMs busy than 12 of 512
    # the same tensor-core products without the fused power step (two sweeps over X per step)
    (2048, 1024, 8, 3, 32, True, 3),
    (700, 520, 8, 3, 16, True, 3),
    (333, 200, 16, 2, 32, True, 3),
    (4096, 3072, 4, 3, 32, True, 3),
]


def _run_extract(X, r, K, seed, layer_id, path, x_bf16, pitch=None):
    Xd, _ = to_dev(X, x_bf16, pitch=pitch)
    Vd = torch.full((r + 2, X.shape[1] + 4), 7.0, device=DEV)
    Vv = Vd[1:1 + r, : X.shape[1]]
    layers = [B.make_layer(X=Xd, V=Vv, r=r, layer_id=layer_id)]
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "extract_path", path)
        B.agzo_set_option(ctx, "extract_fused", 2 if path == 2 else 0)
        B.agzo_extract_subspace(ctx, layers, seed, K)
        st = B.agzo_poll(ctx)
    assert bool((Vd[0] == 7).all() and (Vd[-1] == 7).all() and (Vd[:, X.shape[1]:] == 7).all())
    return to_host(Vv), st


@pytest.mark.parametrize("m,d_in,r,K,planted,x_bf16,path", EXTRACT_CASES)
def test_extract_matches_oracle(m, d_in, r, K, planted, x_bf16, path):
    X = (WL.planted_activations(m, d_in, planted, seed=m, bf16=x_bf16) if planted
         else WL.plain_activations(m, d_in, seed=m, bf16=x_bf16))
    Vg, st = _run_extract(X, r, K, seed=13, layer_id=4, path=path, x_bf16=x_bf16,
                          pitch=d_in + 8 if d_in % 16 else None)
    assert st == B.AGZO_OK
    Vo = O.extract_subspace(X, r, K, 13, 4)
    assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
    assert projector_distance(Vg, Vo) <= 1e-3
    assert np.abs(Vg - Vo).max() <= 1e-3          # the basis itself, not only its span


def test_extract_many_layers_in_waves():
    specs = [(600, 256, 4), (512, 512, 8), (900, 128, 2), (512, 256, 8), (384, 320, 6)]
    Xs = [WL.planted_activations(m, d, 16, seed=i, bf16=True) for i, (m, d, r) in enumerate(specs)]
    devs, layers = [], []
    for i, ((m, d, r), X) in enumerate(zip(specs, Xs)):
        Xd, _ = to_dev(X, True)
        Vd = torch.zeros(r, d, device=DEV)
        devs.append((Xd, Vd))
        layers.append(B.make_layer(X=Xd, V=Vd, r=r, layer_id=i))
    for wave_bytes in (1 << 30, 400 * 1024, 1):      # one wave, several, one layer per wave
        with Ctx(layers) as ctx:
            B.agzo_set_option(ctx, "extract_path", 1)
            B.agzo_set_option(ctx, "wave_bytes", wave_bytes)
            B.agzo_extract_subspace(ctx, layers, 3, 3)
            assert B.agzo_poll(ctx) == B.AGZO_OK
        for i, ((m, d, r), X) in enumerate(zip(specs, Xs)):
            Vo = O.extract_subspace(X, r, 3, 3, i)
            assert projector_distance(to_host(devs[i][1]), Vo) <= 1e-3


def test_fused_shares_cross_layers_of_different_rank():
    """Layers of one cluster size form one tile list that is cut into contiguous shares, so a cluster's share
    runs from one layer into the next: ranks 3, 16 and 8 (8- and 16-column operand panels, the launch sized
    for the largest), token counts that are no multiples of the tile, more tiles than clusters and fewer."""
    for specs in ([(900, 1024, 3), (1500, 1024, 16), (700, 1024, 8), (300, 1024, 16)],
                  [(20000, 512, 8), (9000, 512, 4)],          # one CTA per cluster: 227 tiles over up to 148 shares
                  [(640, 2048, 16), (640, 2048, 5)]):
        Xs = [WL.planted_activations(m, d, 16, seed=70 + i, bf16=True) for i, (m, d, r) in enumerate(specs)]
        devs, layers = [], []
        for i, ((m, d, r), X) in enumerate(zip(specs, Xs)):
            Xd, _ = to_dev(X, True)
            Vd = torch.zeros(r, d, device=DEV)
            devs.append((Xd, Vd))
            layers.append(B.make_layer(X=Xd, V=Vd, r=r, layer_id=i))
        with Ctx(layers) as ctx:
            B.agzo_set_option(ctx, "extract_fused", 2)
            fz = B.agzo_query_fused(ctx, layers)
            assert len(set(fz)) == 1 and fz[0] > 0, fz
            B.agzo_extract_subspace(ctx, layers, 11, 2)
            assert B.agzo_poll(ctx) == B.AGZO_OK
        for i, ((m, d, r), X) in enumerate(zip(specs, Xs)):
            Vo = O.extract_subspace(X, r, 2, 11, i)
            Vg = to_host(devs[i][1])
            assert projector_distance(Vg, Vo) <= 1e-3, (specs, i)
            assert np.abs(Vg - Vo).max() <= 1e-3, (specs, i)


def test_which_layers_take_the_fused_power_step():
    """The default: a layer whose X is larger than an L2-sized wave and whose cluster size keeps most SMs busy
    runs its power steps in the fused kernel; small waves, shared inputs and the option 0 do not."""
    big = WL.planted_activations(9000, 4096, 16, seed=3, bf16=True)      # 74 MB of bf16
    small = WL.planted_activations(512, 1024, 16, seed=4, bf16=True)
    Xb, _ = to_dev(big, True)
    Xs, _ = to_dev(small, True)
    Vb = torch.zeros(8, 4096, device=DEV)
    Vs = torch.zeros(8, 1024, device=DEV)
    Vs2 = torch.zeros(8, 1024, device=DEV)
    layers = [B.make_layer(X=Xb, V=Vb, r=8, layer_id=0), B.make_layer(X=Xs, V=Vs, r=8, layer_id=1)]
    with Ctx(layers) as ctx:
        cap = B.agzo_query_cluster_capacity(ctx)
        sms = torch.cuda.get_device_properties(DEV).multi_processor_count
        assert cap[0] == 0 and cap[1] == sms
        assert all(cap[c] * c <= sms for c in range(1, 17))
        assert all(cap[c] >= cap[c + 1] for c in range(1, 16))
        B.agzo_set_option(ctx, "wave_bytes", 1)                 # one layer per wave
        fz = B.agzo_query_fused(ctx, layers)
        assert fz[1] == 0                                       # 1 MB of activations: stays in L2
        assert fz[0] == (8 if cap[8] * 8 * 10 >= sms * 7 else 0)
        B.agzo_extract_subspace(ctx, layers, 9, 3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
        Vo = O.extract_subspace(big, 8, 3, 9, 0)
        assert projector_distance(to_host(Vb), Vo) <= 1e-3
        B.agzo_set_option(ctx, "extract_fused", 2)
        assert B.agzo_query_fused(ctx, layers) == [8, 2]
        B.agzo_set_option(ctx, "extract_fused", 0)
        assert B.agzo_query_fused(ctx, layers) == [0, 0]
    # two layers on one X: one sweep serves both, which beats one fused pass each
    shared = [B.make_layer(X=Xs, V=Vs, r=8, layer_id=1), B.make_layer(X=Xs, V=Vs2, r=8, layer_id=2)]
    with Ctx(shared) as ctx:
        B.agzo_set_option(ctx, "wave_bytes", 1 << 40)
        assert B.agzo_query_fused(ctx, shared) == [0, 0]
        B.agzo_set_option(ctx, "extract_fused", 2)
        assert B.agzo_query_fused(ctx, shared) == [2, 2]


def test_extract_wave_mixes_fused_and_unfused_layers():
    # d_in = 4608 and r = 24 are beyond the fused kernel's shapes; the others run fused on clusters of 2, 1 and 4
    specs = [(640, 1024, 8), (512, 4608, 4), (700, 264, 16), (512, 512, 24), (768, 2048, 2)]
    Xs = [WL.planted_activations(m, d, 16, seed=10 + i, bf16=True) for i, (m, d, r) in enumerate(specs)]
    devs, layers = [], []
    for i, ((m, d, r), X) in enumerate(zip(specs, Xs)):
        Xd, _ = to_dev(X, True)
        Vd = torch.zeros(r, d, device=DEV)
        devs.append((Xd, Vd))
        layers.append(B.make_layer(X=Xd, V=Vd, r=r, layer_id=i))
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "extract_path", 2)
        B.agzo_set_option(ctx, "extract_fused", 2)
        B.agzo_extract_subspace(ctx, layers, 5, 3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    for i, ((m, d, r), X) in enumerate(zip(specs, Xs)):
        Vo = O.extract_subspace(X, r, 3, 5, i)
        Vg = to_host(devs[i][1])
        assert projector_distance(Vg, Vo) <= 1e-3
        assert np.abs(Vg - Vo).max() <= 1e-3


def test_layers_that_share_their_input_are_served_by_one_sweep():
    # q/k/v-like and gate/up-like groups on shared X buffers, a layer of its own in between
    shapes = [(1024, 512), (640, 264), (900, 1024)]
    Xh = [WL.planted_activations(m, d, 16, seed=20 + i, bf16=True) for i, (m, d) in enumerate(shapes)]
    Xd = [to_dev(x, True, pitch=x.shape[1] + 8 if x.shape[1] % 16 else None)[0] for x in Xh]
    plan = [(0, 8), (0, 4), (0, 16), (1, 5), (2, 8), (2, 8)]      # (which X, r)
    results = {}
    for share in (1, 0):
        Vs, layers = [], []
        for i, (xi, r) in enumerate(plan):
            V = torch.zeros(r, Xh[xi].shape[1], device=DEV)
            Vs.append(V)
            layers.append(B.make_layer(X=Xd[xi], V=V, r=r, layer_id=40 + i))
        with Ctx(layers) as ctx:
            B.agzo_set_option(ctx, "extract_path", 3)
            B.agzo_set_option(ctx, "share_inputs", share)
            B.agzo_extract_subspace(ctx, layers, 9, 3)
            assert B.agzo_poll(ctx) == B.AGZO_OK
        results[share] = [to_host(V) for V in Vs]
    for i, (xi, r) in enumerate(plan):
        Vo = O.extract_subspace(Xh[xi], r, 3, 9, 40 + i)
        Vg = results[1][i]
        assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
        assert projector_distance(Vg, Vo) <= 1e-3
        assert np.abs(Vg - Vo).max() <= 1e-3
        # grouping changes which CTA computes a column, not what is computed
        assert np.abs(Vg - results[0][i]).max() <= 1e-6


# ---- decaying and outlier spectra (Section 3.2 reports rapidly decaying activation spectra; language
# models have channels and tokens a hundred times larger than the rest).  Every path: 1 CUDA cores,
# 3 tensor cores in two sweeps, 2 tensor cores with the fused power step (r <= 16).
def _spectrum_case(kind):
    m, d_in = 2048, 512
    if kind == "graded":          # sigma_k = 2^(-k/2) over 64 directions, nothing else but bf16 rounding
        return WL.graded_activations(m, d_in, 64, seed=3, bf16=True)
    if kind == "graded+floor":    # the same on an isotropic floor of 1e-2 per entry
        return WL.graded_activations(m, d_in, 64, seed=3, bf16=True, floor=1e-2)
    if kind == "massive100":      # one channel and one token 100 times the rest
        return WL.massive_activations(m, d_in, seed=4, bf16=True)
    return WL.massive_activations(m, d_in, seed=4, bf16=True, factor=1000.0)


@pytest.mark.parametrize("path", [1, 3, 2])
@pytest.mark.parametrize("kind,r", [("graded", 4), ("graded", 16), ("graded+floor", 4), ("graded+floor", 16),
                                     ("massive100", 4), ("massive100", 16), ("massive100", 64)])
def test_extract_on_decaying_and_outlier_spectra(kind, r, path):
    # sigma_1 / sigma_r up to about 200: no column may be dropped and the 1e-3 projector bound holds
    if path == 2 and r > 16:
        pytest.skip("the fused power step serves r <= 16")
    X = _spectrum_case(kind)
    Vg, st = _run_extract(X, r, 3, seed=5, layer_id=3, path=path, x_bf16=True)
    Vo, info = O.extract_subspace(X, r, 3, 5, 3, return_info=True)
    assert st == B.AGZO_OK and not info["deficient"]
    assert np.abs(Vg.astype(np.float64) @ Vg.T - np.eye(r)).max() <= 1e-5
    assert projector_distance(Vg, Vo) <= 1e-3


@pytest.mark.parametrize("path", [1, 3])
@pytest.mark.parametrize("kind,r,both_flag", [("graded", 64, True), ("graded+floor", 64, False),
                                               ("massive1000", 4, True), ("massive1000", 16, True),
                                               ("massive1000", 64, True)])
def test_extract_beyond_what_fp32_resolves(kind, r, both_flag, path):
    # sigma_1 / sigma_r above 1e3: the trailing columns of Y = H (H^T Q) lie at or below fp32 noise of the
    # leading ones, so a float32 device and the float64 oracle cannot agree on them to 1e-3.  What is
    # unique is compared: the same verdict on dependent columns (and equally many of them), an
    # orthonormal basis, the leading directions, and the energy of X that the basis captures.
    X = _spectrum_case(kind)
    Vg, st = _run_extract(X, r, 3, seed=5, layer_id=3, path=path, x_bf16=True)
    Vo, info = O.extract_subspace(X, r, 3, 5, 3, return_info=True)
    assert info["deficient"] == both_flag
    assert st == (B.AGZO_WARN_RANK_DEFICIENT if both_flag else B.AGZO_OK)
    live_g, live_o = np.abs(Vg).sum(1) > 0, np.abs(Vo).sum(1) > 0
    assert live_g.sum() == live_o.sum()
    Vl = Vg[live_g].astype(np.float64)
    assert np.abs(Vl @ Vl.T - np.eye(len(Vl))).max() <= 1e-5
    Xd = X.astype(np.float64)
    eg, eo = np.linalg.norm(Xd @ Vg.T.astype(np.float64)) ** 2, np.linalg.norm(Xd @ Vo.T.astype(np.float64)) ** 2
    assert abs(eg / eo - 1.0) <= 1e-6
    if kind.startswith("graded"):        # well separated leading directions: compared as a subspace
        assert projector_distance(Vg[:8], Vo[:8]) <= 1e-3


def test_extract_rank_deficient_panel_is_reported():
    rng = np.random.default_rng(0)
    m, d_in, r = 256, 128, 4
    X = (np.outer(rng.standard_normal(m), rng.standard_normal(d_in))
         + np.outer(rng.standard_normal(m), rng.standard_normal(d_in))).astype(np.float32)
    Vg, st = _run_extract(X, r, 2, seed=3, layer_id=0, path=1, x_bf16=False)
    assert st == B.AGZO_WARN_RANK_DEFICIENT
    Vo, info = O.extract_subspace(X, r, 2, 3, 0, return_info=True)
    assert info["deficient"]
    assert np.all(Vg[2:] == 0.0) and np.all(Vo[2:] == 0.0)
    assert projector_distance(Vg[:2], Vo[:2]) <= 1e-3


@pytest.mark.parametrize("r,p", [(20, 13), (40, 17), (64, 33), (64, 1), (17, 16)])
def test_extract_low_rank_input_across_the_register_tiles_of_the_factorisation(r, p):
    """X of exact rank p < r: the factorisation meets its first dependent column at index p, which for
    these sizes lies in every position of the 16 x 16 thread arrangement that owns the matrix (first,
    second and third block of rows, a block boundary).  The dependent columns come out zero and flagged on
    both sides, the others span the same space."""
    rng = np.random.default_rng(r * 100 + p)
    m, d_in = 512, 256
    X = sum(np.outer(rng.standard_normal(m), rng.standard_normal(d_in)) for _ in range(p)).astype(np.float32)
    Vg, st = _run_extract(X, r, 2, seed=3, layer_id=0, path=1, x_bf16=False)
    assert st == B.AGZO_WARN_RANK_DEFICIENT
    Vo, info = O.extract_subspace(X, r, 2, 3, 0, return_info=True)
    assert info["deficient"]
    live_g, live_o = np.abs(Vg).sum(1) > 0, np.abs(Vo).sum(1) > 0
    assert live_g.sum() == live_o.sum() == p
    assert np.array_equal(live_g, live_o)
    Vl = Vg[live_g].astype(np.float64)
    assert np.abs(Vl @ Vl.T - np.eye(p)).max() <= 1e-5
    assert projector_distance(Vg[live_g], Vo[live_o]) <= 1e-3


def test_empty_layer_list_and_argument_errors():
    V = torch.zeros(4, 64, device=DEV)
    W = torch.zeros(32, 64, device=DEV, dtype=torch.bfloat16)
    X = torch.zeros(16, 64, device=DEV, dtype=torch.bfloat16)
    good = B.make_layer(W=W, X=X, V=V, r=4, layer_id=0)
    with Ctx([good]) as ctx:
        L = B.lib()
        assert L.agzo_perturb(ctx.handle, None, 0, 0, 1e-3, None) == B.AGZO_OK
        assert L.agzo_extract_subspace(ctx.handle, None, 0, 0, 3, None) == B.AGZO_OK
        assert L.agzo_perturb(ctx.handle, None, 1, 0, 1e-3, None) == B.AGZO_ERR_INVALID_ARG

        def status(fn, layer, *args):
            return fn(ctx.handle, B.layer_array([layer]), 1, *args)

        bad_r = B.make_layer(W=W, X=X, V=V, r=4, layer_id=0); bad_r.r = 65
        assert status(L.agzo_perturb, bad_r, 0, 1e-3, None) == B.AGZO_ERR_INVALID_ARG
        r_gt_m = B.make_layer(W=W, X=X[:2], V=V, r=4, layer_id=0)
        assert status(L.agzo_extract_subspace, r_gt_m, 0, 3, None) == B.AGZO_ERR_INVALID_ARG
        no_x = B.make_layer(W=W, V=V, r=4, layer_id=0)
        assert status(L.agzo_extract_subspace, no_x, 0, 3, None) == B.AGZO_ERR_INVALID_ARG
        no_w = B.make_layer(X=X, V=V, r=4, layer_id=0)
        assert status(L.agzo_perturb, no_w, 0, 1e-3, None) == B.AGZO_ERR_INVALID_ARG
        assert status(L.agzo_extract_subspace, good, 0, 17, None) == B.AGZO_ERR_INVALID_ARG
        bad_dt = B.make_layer(W=W, X=X, V=V, r=4, layer_id=0); bad_dt.w_dtype = 5
        assert status(L.agzo_perturb, bad_dt, 0, 1e-3, None) == B.AGZO_ERR_UNSUPPORTED
        pair_bf16 = B.make_layer(W=W, W16=W, X=X, V=V, r=4, layer_id=0)
        assert status(L.agzo_perturb, pair_bf16, 0, 1e-3, None) == B.AGZO_ERR_UNSUPPORTED
        assert L.agzo_update(ctx.handle, B.layer_array([good]), 1, 0, 1e-3, None, None) == B.AGZO_ERR_INVALID_ARG
        # a workspace that is too small for the layers is refused, nothing is launched
    small = B.Context(0, 4096)
    big = B.make_layer(X=torch.zeros(4096, 64, device=DEV), V=V, r=4, layer_id=0)
    assert B.lib().agzo_extract_subspace(small.handle, B.layer_array([big]), 1, 0, 3, None) == B.AGZO_ERR_WORKSPACE
    B.agzo_destroy(small)
    assert bool((W == 0).all())


def test_a_device_side_wait_that_nothing_ends_gives_up_and_is_reported():
    """Failure detection without a fault: the library's bounded wait, on a barrier that nobody
    completes, returns after its time limit; the condition reaches the host through the status
    word, and the context keeps working."""
    import time
    d_out, d_in, r, seed = 130, 256, 8, 3
    W0 = WL.gaussian_weights(d_out, d_in, 0.02, seed=1, bf16=True)
    Vh = O.extract_subspace(WL.plain_activations(64, d_in, seed=2), r, 1, 3, 0)
    Wd, _ = to_dev(W0, True)
    Vd, _ = to_dev(Vh, False)
    layers = [B.make_layer(W=Wd, V=Vd, r=r, layer_id=0)]
    with Ctx(layers) as ctx:
        assert B.agzo_poll(ctx) == B.AGZO_OK
        t0 = time.perf_counter()
        B.agzo_debug_wait_timeout(ctx)
        assert B.agzo_poll(ctx) == B.AGZO_ERR_TIMEOUT          # poll waits for the stream
        assert 1.0 < time.perf_counter() - t0 < 20.0           # the limit is two seconds
        assert B.agzo_poll(ctx) == B.AGZO_OK                   # reported once, then cleared
        B.agzo_perturb(ctx, layers, seed, 1e-3)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    want = O.apply_direction(W0, Vh, seed, 0, np.float32(1e-3), "bf16")
    assert_weights_match(to_host(Wd), want, "bf16",
                         floor=cancellation_floor(W0, 1e-3, seed, 0, Vh, rel=2.0 ** -16))
