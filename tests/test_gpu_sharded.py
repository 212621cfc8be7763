"""Token-sharded extraction (agzo_set_allreduce) on one GPU: two host threads stand for two
data-parallel ranks, each with its own context, stream and shard of the tokens.  The ranks meet
only on the host, inside the all-reduce callback (a thread barrier, then a device sum), so no
kernel ever waits for another rank's kernel.  Both ranks must return the V that the oracle
computes from the whole batch (Algorithm 1 on the concatenated X), and the same V bit for bit.
"""
import threading

import numpy as np
import pytest
import torch

from oracle import agzo_oracle as O
from paper_2601_17261_b200 import binding as B
from paper_2601_17261_b200 import workloads as WL

from gpu_helpers import DEV, Ctx, projector_distance, to_dev

pytestmark = pytest.mark.gpu


class HostAllReduce:
    """Sum over `world` threads of one process: every rank adds the buffers in rank order."""

    def __init__(self, world: int):
        self.world = world
        self.barrier = threading.Barrier(world, timeout=120)
        self.bufs = [None] * world
        self.calls = [0] * world
        self.counts = [[] for _ in range(world)]

    def fn(self, rank: int):
        def allreduce(buf: torch.Tensor, stream_ptr: int) -> None:
            st = torch.cuda.ExternalStream(stream_ptr, device=buf.device)
            st.synchronize()                     # this rank's panels are complete
            self.bufs[rank] = buf
            self.calls[rank] += 1
            self.counts[rank].append(buf.numel())
            self.barrier.wait()
            with torch.cuda.stream(st):
                total = self.bufs[0].clone()
                for p in range(1, self.world):
                    total += self.bufs[p]
            st.synchronize()
            self.barrier.wait()                  # every rank has read every buffer
            with torch.cuda.stream(st):
                buf.copy_(total)
        return allreduce


def run_ranks(world, body):
    errors, results = [], [None] * world

    def target(rank):
        try:
            results[rank] = body(rank)
        except BaseException as e:  # noqa: BLE001 - reported by the main thread
            errors.append(e)

    threads = [threading.Thread(target=target, args=(p,)) for p in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    return results


@pytest.mark.parametrize("path,K,fused", [(1, 3, 0), (2, 3, 0), (2, 0, 0), (2, 3, 2)])
def test_two_token_shards_give_the_whole_batch_subspace(path, K, fused):
    # fused = 2: the power steps run in the cluster kernel, whose partial sums per layer are counted differently
    # the split points are odd, so a rank's first element of Omega falls inside a Philox block
    specs = [(1100, 256, 3, 517), (1536, 512, 8, 768), (900, 384, 6, 333)]   # m, d_in, r, tokens of rank 0
    seed = 21
    Xs = [WL.planted_activations(m, d, 16, seed=40 + i, bf16=True) for i, (m, d, r, m0) in enumerate(specs)]
    hub = HostAllReduce(2)

    def body(rank):
        torch.cuda.set_device(0)
        stream = torch.cuda.Stream()
        devs, layers = [], []
        for i, ((m, d, r, m0), X) in enumerate(zip(specs, Xs)):
            Xp = X[:m0] if rank == 0 else X[m0:]
            Xd, _ = to_dev(np.ascontiguousarray(Xp), True)
            Vd = torch.zeros(r, d, device=DEV)
            devs.append((Xd, Vd))
            layers.append(B.make_layer(X=Xd, V=Vd, r=r, layer_id=i))
        # every rank has the same token offset for all its layers: take equal split points per call
        torch.cuda.synchronize()
        out = []
        for i, (m, d, r, m0) in enumerate(specs):          # one call per layer: the offsets differ
            with Ctx([layers[i]]) as ctx:
                B.agzo_set_option(ctx, "extract_path", path)
                B.agzo_set_option(ctx, "extract_fused", fused)
                B.agzo_set_allreduce(ctx, hub.fn(rank), 0 if rank == 0 else m0)
                B.agzo_extract_subspace(ctx, [layers[i]], seed, K, stream=stream)
                stream.synchronize()
                assert B.agzo_poll(ctx) == B.AGZO_OK
            out.append(devs[i][1].cpu().numpy())
        return out

    B.lib()
    got = run_ranks(2, body)
    assert hub.calls[0] == hub.calls[1] == len(specs) * (K + 1)
    assert hub.counts[0] == hub.counts[1]
    for i, ((m, d, r, m0), X) in enumerate(zip(specs, Xs)):
        want = O.extract_subspace(X, r, K, seed, i)
        assert np.array_equal(got[0][i], got[1][i]), "the ranks hold different V"
        assert projector_distance(got[0][i], want) <= 1e-3
        assert np.abs(got[0][i] @ got[0][i].T - np.eye(r)).max() <= 1e-5


def test_many_layers_in_one_sharded_call_use_one_buffer_per_wave():
    # equal split point for all layers of the call; several layers per wave, two waves; layers 1 and 2
    # read the same buffer (as q and k of a block do) and are served by one sweep over it
    m, m0 = 1024, 512
    specs = [(256, 4), (512, 8), (512, 6), (256, 2)]
    seed = 5
    Xs = [WL.planted_activations(m, d, 16, seed=60 + i, bf16=True) for i, (d, r) in enumerate(specs)]
    Xs[2] = Xs[1]
    hub = HostAllReduce(2)

    def body(rank):
        torch.cuda.set_device(0)
        stream = torch.cuda.Stream()
        keep, layers = [], []
        for i, ((d, r), X) in enumerate(zip(specs, Xs)):
            if i == 2:
                Xd = keep[1][0]
            else:
                Xd, _ = to_dev(np.ascontiguousarray(X[:m0] if rank == 0 else X[m0:]), True)
            Vd = torch.zeros(r, d, device=DEV)
            keep.append((Xd, Vd))
            layers.append(B.make_layer(X=Xd, V=Vd, r=r, layer_id=i))
        torch.cuda.synchronize()
        with Ctx(layers) as ctx:
            B.agzo_set_option(ctx, "wave_bytes", 800 * 1024)      # layers 0 to 2 (768 KiB of X), then layer 3
            B.agzo_set_allreduce(ctx, hub.fn(rank), rank * m0)
            B.agzo_extract_subspace(ctx, layers, seed, 2, stream=stream)
            stream.synchronize()
            assert B.agzo_poll(ctx) == B.AGZO_OK
            # back to a single rank: the same context extracts from its own shard alone
            B.agzo_set_allreduce(ctx, None)
            B.agzo_extract_subspace(ctx, layers[:1], seed, 2, stream=stream)
            stream.synchronize()
            alone = keep[0][1].cpu().numpy().copy()
        return [v.cpu().numpy() for _, v in keep][1:], alone

    B.lib()
    got = run_ranks(2, body)
    waves = hub.calls[0] // 3
    assert waves >= 2 and hub.calls[0] == hub.calls[1] == 3 * waves
    for i, ((d, r), X) in enumerate(zip(specs, Xs)):
        if i == 0:
            continue
        want = O.extract_subspace(X, r, 2, seed, i)
        assert np.array_equal(got[0][0][i - 1], got[1][0][i - 1])
        assert projector_distance(got[0][0][i - 1], want) <= 1e-3
    for rank in range(2):    # the unsharded call sees only the rank's own tokens, Omega rows from 0
        Xp = Xs[0][:m0] if rank == 0 else Xs[0][m0:]
        assert projector_distance(got[rank][1], O.extract_subspace(Xp, specs[0][1], 2, seed, 0)) <= 1e-3


def test_a_failing_allreduce_ends_the_call_with_the_callback_status():
    X = WL.planted_activations(512, 256, 16, seed=3, bf16=True)
    Xd, _ = to_dev(X, True)
    Vd = torch.zeros(4, 256, device=DEV)
    layers = [B.make_layer(X=Xd, V=Vd, r=4, layer_id=0)]

    def broken(buf, stream_ptr):
        raise RuntimeError("no peers")

    with Ctx(layers) as ctx:
        B.agzo_set_allreduce(ctx, broken, 0)
        with pytest.raises(B.AgzoError) as e:
            B.agzo_extract_subspace(ctx, layers, 1, 1)
        assert e.value.status == B.AGZO_ERR_CALLBACK
        torch.cuda.synchronize()
        B.agzo_set_allreduce(ctx, None)
        B.agzo_extract_subspace(ctx, layers, 1, 1)       # the context is still usable
        torch.cuda.synchronize()
        assert B.agzo_poll(ctx) == B.AGZO_OK
    assert projector_distance(Vd.cpu().numpy(), O.extract_subspace(X, 4, 1, 1, 0)) <= 1e-3
