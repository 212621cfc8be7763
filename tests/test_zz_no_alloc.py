"""The allocation-free entry point agzo_extract_subspace_static against the regular one.

Some callers cannot allocate device memory at the moment they need a subspace (a forward hook
while another framework owns the allocator, a callback where cudaMalloc would stall the
device), so the library offers Algorithm 1 for one layer on a scratch array that is part of
the library itself.  This file is named so that pytest collects it last: if it fails, a run
that stops at the first failure has already run everything else.  Every call shares that one
array and finds the previous call's bytes in it, hence two different problems back to back.
"""
import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import DEV, Ctx, projector_distance, to_dev, to_host

pytestmark = pytest.mark.gpu


def _regular(Xd, r, K, seed, layer_id):
    V = torch.zeros(r, Xd.shape[1], device=DEV)
    layers = [B.make_layer(X=Xd, V=V, r=r, layer_id=layer_id)]
    with Ctx(layers) as ctx:
        B.agzo_set_option(ctx, "extract_path", 1)      # the kernels the static variant uses
        B.agzo_extract_subspace(ctx, layers, seed, K)
        assert B.agzo_poll(ctx) == B.AGZO_OK
    return to_host(V)


def _warm_up_the_static_entry_point():
    """The first call on a device loads the library's kernels and looks up the scratch array's
    address; the driver may set memory aside for that.  The no-allocation property is about the
    calls after it, so one small call comes first."""
    X = torch.randn(64, 32, device=DEV)
    V = torch.zeros(2, 32, device=DEV)
    B.agzo_extract_subspace_static(X, V, 2, 1, 0, 0)
    torch.cuda.synchronize()


def test_static_scratch_variant_matches_the_regular_entry_point_twice_in_a_row():
    _warm_up_the_static_entry_point()
    cases = [(1500, 520, 8, 3, 21, 4, True, 528),      # ragged sizes, padded pitch, bf16
             (700, 256, 4, 2, 22, 9, False, None)]     # a smaller fp32 problem right after
    for (m, d_in, r, K, seed, layer_id, bf16, pitch) in cases:
        X = WL.planted_activations(m, d_in, 16, seed=m, bf16=bf16)
        Xd, _ = to_dev(X, bf16, pitch=pitch)
        want = _regular(Xd, r, K, seed, layer_id)
        Vbuf = torch.full((r + 2, d_in + 4), 7.0, device=DEV)
        V = Vbuf[1:1 + r, :d_in]
        flag = torch.full((1,), -1, dtype=torch.int32, device=DEV)
        torch.cuda.synchronize()
        # Two counters, because the library calls the CUDA runtime directly and torch's caching
        # allocator would not see a cudaMalloc made there: the driver's own count of free device
        # bytes, and torch's cumulative count of allocations (frees by the garbage collector in
        # the meantime cannot move it, a new allocation would).
        free_before = torch.cuda.mem_get_info()[0]
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        B.agzo_extract_subspace_static(Xd, V, r, K, seed, layer_id, d_rank_deficient=flag)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before
        got = to_host(V)
        assert int(flag) == 0
        assert np.abs(got.astype(np.float64) @ got.T - np.eye(r)).max() <= 1e-5
        # against the existing entry point (same kernels, workspace scratch) ...
        assert projector_distance(got, want) <= 1e-3
        assert np.abs(got - want).max() <= 1e-3
        # ... and against the oracle itself
        Vo = O.extract_subspace(X, r, K, seed, layer_id)
        assert projector_distance(got, Vo) <= 1e-3
        assert np.abs(got - Vo).max() <= 1e-3
        assert bool((Vbuf[0] == 7).all() and (Vbuf[-1] == 7).all() and (Vbuf[:, d_in:] == 7).all())


def test_static_scratch_variant_refuses_what_does_not_fit():
    X = torch.zeros(16384, 4096, dtype=torch.bfloat16, device=DEV)
    V = torch.zeros(16, 4096, device=DEV)
    with pytest.raises(B.AgzoError) as e:
        B.agzo_extract_subspace_static(X, V, 16, 3, 0, 0)
    assert e.value.status == B.AGZO_ERR_WORKSPACE
    with pytest.raises(B.AgzoError) as e:
        B.agzo_extract_subspace_static(X[:8], V, 16, 3, 0, 0)      # r > m
    assert e.value.status == B.AGZO_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((V == 0).all())
