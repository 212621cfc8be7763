"""The N > 1 logic on CPU: two gloo ranks.

The in-place passes have no exchange step (every rank of a zeroth-order data-parallel job holds
the whole model and applies the same seeded perturbation), so the benchmark runs replicas.  What
its ranks share is the measurement protocol: a timing is the maximum over ranks, rank 0 alone
reports, and the reference arm runs on rank 0 only.  Extraction does shard, over tokens: the
ranks sum their Y panels before every qr(Y) (agzo_set_allreduce); the identity behind it and the
torch.distributed adapter are run here on the oracle's arithmetic.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
        out[rank] = ms
        # every rank regenerates the same direction from the same seed: nothing to exchange
        from oracle import agzo_oracle as O
        g = torch.from_numpy(O.gen_G(7, 3, 16, 4).copy())
        gathered = [torch.zeros_like(g) for _ in range(world)]
        dist.all_gather(gathered, g)
        out[world + rank] = all(bool((x == g).all()) for x in gathered)
    finally:
        dist.destroy_process_group()


def test_timing_is_the_maximum_over_ranks_and_directions_need_no_exchange():
    world, port = 2, 29611
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == 15.0
        assert out[2] and out[3]


def _sharded_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import agzo_oracle as O
    from paper_2601_17261_b200 import workloads as WL
    from paper_2601_17261_b200.binding import torch_allreduce
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        m, d_in, r, K, seed, layer_id, m0 = 96, 40, 5, 3, 9, 2, 37
        X = WL.planted_activations(m, d_in, 8, seed=1, bf16=True).astype(np.float64)   # same on both ranks
        rows = slice(0, m0) if rank == 0 else slice(m0, m)
        Xp = X[rows]
        allreduce = torch_allreduce()
        calls = 0

        def summed(Yp):     # the library hands the callback one flat fp32 buffer; here it is fp64
            nonlocal calls
            buf = torch.from_numpy(np.ascontiguousarray(Yp).reshape(-1))
            allreduce(buf, 0)
            calls += 1
            return buf.numpy().reshape(Yp.shape)

        # the rank's rows of the whole batch's test matrix, then Algorithm 1 with every Y summed
        Omega = O.gen_omega(seed, layer_id, m, r).astype(np.float64)[rows]
        Y = summed(Xp.T @ Omega)
        for _ in range(K):
            Q, _, _ = O.qr_positive(Y)
            Y = summed(Xp.T @ (Xp @ Q))
        Q, _, _ = O.qr_positive(Y)
        want = O.extract_subspace(X, r, K, seed, layer_id, return_info=True)[1]["V64"]
        out[rank] = (float(np.abs(Q.T - want).max()), calls)
    finally:
        dist.destroy_process_group()


def test_token_shards_summed_before_every_qr_give_the_whole_batch_subspace():
    world, port = 2, 29613
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_sharded_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            err, calls = out[rank]
            assert err <= 1e-9 and calls == 4


def test_single_rank_timing_is_passed_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, None, torch.device("cpu")) == 3.25
    assert bench.whole_job_units(2.0, 4) == 8.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0
    assert not [l for l in p.stdout.splitlines() if l.startswith("{")]


def test_bench_launcher_starts_one_process_per_rank(tmp_path):
    """`python bench.py --gpus N` run as a plain command starts N local ranks itself.  The launcher is
    exercised here with a stub worker: every process must see its own RANK / LOCAL_RANK, the common
    WORLD_SIZE and a rendezvous on 127.0.0.1, and the exit codes come back in rank order."""
    import bench
    stub = ("import os, sys; d = sys.argv[1]; r = os.environ['RANK']; "
            "open(os.path.join(d, 'rank_' + r), 'w').write(' '.join(os.environ[k] for k in "
            "('RANK', 'LOCAL_RANK', 'WORLD_SIZE', 'MASTER_ADDR', 'MASTER_PORT'))); sys.exit(3 if r == '2' else 0)")
    codes = bench.spawn_ranks(4, [str(tmp_path)], worker=[sys.executable, "-c", stub])
    assert codes == [0, 0, 3, 0]
    seen = sorted(p.name for p in tmp_path.iterdir())
    assert seen == ["rank_0", "rank_1", "rank_2", "rank_3"]
    ports = set()
    for i in range(4):
        rank, local, world, addr, port = (tmp_path / f"rank_{i}").read_text().split()
        assert (rank, local, world, addr) == (str(i), str(i), "4", "127.0.0.1")
        ports.add(port)
    assert len(ports) == 1
