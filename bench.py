"""Benchmark of the AGZO per-step hot path on synthetic Qwen3-shaped layer sets.

One "step" = Algorithm 1 for every layer (K = 3) + the three in-place passes of a two-point
AGZO iteration (perturb +eps, flip -2 eps, fused restore-and-update) + the scalar; forward
passes are the caller's model and are excluded ("step overhead").  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--rank R]
  python bench.py --impl reference ...      # the CPU oracle on the host cores

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of
the same step on its own GPU (the path has no exchange step; weights are replicated in
zeroth-order data parallelism and every rank applies the same seeded perturbation).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2601_17261_b200 import workloads as WL  # noqa: E402

K_POWER = 3
# DRAM bytes moved per algorithmic byte, from the ncu capture of each kernel on a 4-block
# slice of the 8B-shaped layer set (summaries under profiles/); traffic grows in proportion
# to the activation bytes a launch sweeps.  Reset an entry to None when its kernel changes.
TRAFFIC_PER_ALGORITHMIC_BYTE = {"tc_xt_t_kernel": (4.865880 + 0.011429) / 4.831838,
                                "fused_power_step_kernel": (3.272938 + 0.009340) / 3.221225}
# Thread-level instructions per weight of the dense-direction kernel (one Philox + Box-Muller normal per weight):
# ncu smsp__thread_inst_executed.sum / weights on a 4096 x 4096 bf16 layer (profiles/dense_vec_kernel_*.md).
DENSE_INST_PER_WEIGHT = 933126144 / (4096 * 4096)
EPS = 1e-3
LR = 1e-6
METRIC = "agzo_step_overhead_ms"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "200", "-i", str(device_index)], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(",") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for nm, v in zip(names, r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(nm)
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["sm_max_mhz"] = float(max(mx))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- workload
def build_layer_set(cfg: WL.LayerSetConfig, rank: int, device, seed: int = 1000, alias_inputs: bool = False):
    """Resident tensors of one layer set: bf16 W and X per layer (torch device generators,
    same recipe as the host generators the parity tests use), fp32 V."""
    from paper_2601_17261_b200 import binding as B
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    Ws, Xs, Vs, layers = [], [], [], []
    for i, (name, d_in, d_out) in enumerate(cfg.layers()):
        W = WL.device_weights(d_out, d_in, cfg.w_std, gen, device)
        kind = name.split(".")[-1]
        if alias_inputs and kind in ("k", "v", "up"):
            X = Xs[-1]          # k, v read q's input; up reads gate's: one buffer, as in a transformer block
        else:
            X = WL.device_planted_activations(cfg.m, d_in, cfg.planted_rank, gen, device)
        V = torch.zeros(rank, d_in, dtype=torch.float32, device=device)
        Ws.append(W); Xs.append(X); Vs.append(V)
        layers.append(B.make_layer(W=W, X=X, V=V, r=rank, layer_id=i))
    return Ws, Xs, Vs, layers


def algorithmic_work(cfg: WL.LayerSetConfig, rank: int, alias_inputs: bool = False):
    n_w = cfg.n_params()
    x_elems = cfg.x_elems()
    if alias_inputs:   # q/k/v and gate/up read one buffer each: distinct activation bytes only
        x_elems = cfg.n_blocks * sum(cfg.m * di for (nm, di, _) in cfg.block if nm not in ("k", "v", "up"))
    rmw_bytes_pass = 4 * n_w + sum(4 * rank * di for (_, di, _) in cfg.layers())
    extract_bytes = (K_POWER + 1) * 2 * x_elems          # X read once per product pair (fused)
    extract_bytes_unfused = (2 * K_POWER + 1) * 2 * x_elems
    extract_flops = sum((2 * K_POWER + 1) * 2 * cfg.m * di * rank + (K_POWER + 1) * 2 * di * rank * rank
                        for (_, di, _) in cfg.layers())
    return {"rmw_bytes_per_pass": rmw_bytes_pass, "extract_bytes_fused": extract_bytes,
            "extract_bytes_unfused": extract_bytes_unfused, "extract_flops": extract_flops,
            "x_bytes": 2 * x_elems, "w_bytes": 2 * n_w}


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_layer_seconds(cfg: WL.LayerSetConfig, rank: int, X_host, W_host, seed: int = 0):
    """The oracle, as it stands, on the given layers (Algorithm 1 + the three passes of a two-point
    step); returns the seconds each layer took."""
    from oracle import agzo_oracle as O
    out = []
    for i, (X, W) in enumerate(zip(X_host, W_host)):
        t0 = time.perf_counter()
        V = O.extract_subspace(X, rank, K_POWER, seed, i)
        W1 = O.apply_direction(W, V, seed, i, np.float32(EPS), "bf16")
        W2 = O.apply_direction(W1, V, seed, i, np.float32(-2 * EPS), "bf16")
        g = O.ghat_two_point(1.0, 0.999, EPS)
        O.apply_direction(W2, V, seed, i, O.update_coefficient(EPS, LR, g, 0), "bf16")
        out.append(time.perf_counter() - t0)
    return out


def oracle_block_seconds(cfg: WL.LayerSetConfig, rank: int, X_host, W_host, seed: int = 0):
    """Block 0 (7 layers) through the oracle: the sample both CPU legs time."""
    return float(sum(oracle_layer_seconds(cfg, rank, X_host, W_host, seed)))


def cpu_baseline_leg(cfg: WL.LayerSetConfig, rank: int, n_layers_total: int):
    """The oracle on block 0 with all host cores (every block has the same shapes, so the block's time
    is multiplied by the number of blocks), and its second layer once more on one thread."""
    Xh, Wh = host_block(cfg)
    per_layer = oracle_layer_seconds(cfg, rank, Xh, Wh)
    t = float(sum(per_layer))
    out = {"value": t * 1e3 * cfg.n_blocks, "unit": "ms", "cores": os.cpu_count(), "kind": "oracle",
           "sample": f"block 0 ({len(cfg.block)} of {n_layers_total} layers) timed ({t:.1f} s), "
                     f"time x{cfg.n_blocks} blocks"}
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            t1 = oracle_layer_seconds(cfg, rank, Xh[1:2], Wh[1:2])[0]
        out["single_thread"] = {"sample": "layer 1 of block 0 (%s)" % cfg.block[1][0], "seconds_one_thread": t1,
                                "seconds_all_cores": per_layer[1]}
    except Exception as e:  # noqa: BLE001 - the thread limit is a convenience of the report
        out["single_thread"] = {"unavailable": repr(e)}
    return out


def host_block(cfg: WL.LayerSetConfig, n_layers: int = 7, seed: int = 1000):
    """First layers of block 0 generated on the host with the numpy recipe (bf16 values as float32)."""
    Xs, Ws = [], []
    for i, (name, d_in, d_out) in enumerate(cfg.block[:n_layers]):
        Xs.append(WL.planted_activations(cfg.m, d_in, cfg.planted_rank, seed + i, bf16=True))
        Ws.append(WL.gaussian_weights(d_out, d_in, cfg.w_std, seed + i, bf16=True))
    return Xs, Ws


def workload_string(cfg: WL.LayerSetConfig, rank_r: int, mode: int) -> str:
    """The one description of the workload that both arms print."""
    return (f"{cfg.name}: {len(cfg.layers())} layers, {cfg.n_params() / 1e9:.3f} G weights, m={cfg.m} tokens, "
            f"r={rank_r}, K={K_POWER}, eps={EPS}, " + ("two-point" if mode == 0 else "one-sided"))


def run_reference(args, cfg, rank_r):
    """--impl reference: the CPU oracle on the host cores; a step = block 0 of the layer set,
    extrapolated to all blocks (every block has the same shapes)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    cores = os.cpu_count() or 1
    # A step is the sample the cpu_baseline leg of the main arm times: block 0, whole.  The first
    # step always runs it whole; if all W + K steps at that pace would take more than about four
    # minutes, the later steps time the block's first two layers and are scaled by the ratio that
    # the first step measured between the whole block and those two layers.
    Xs, Ws = host_block(cfg)
    total = args.warmup + args.steps
    first = oracle_layer_seconds(cfg, rank_r, Xs, Ws, seed=0)
    t_block, t_two = float(sum(first)), float(sum(first[:2]))
    whole = t_block * total <= 240.0
    scale = 1.0 if whole else t_block / t_two
    times = [t_block] if args.warmup == 0 else []
    for it in range(1, total):
        t = (oracle_block_seconds(cfg, rank_r, Xs, Ws, seed=it) if whole
             else float(sum(oracle_layer_seconds(cfg, rank_r, Xs[:2], Ws[:2], seed=it))) * scale)
        if it >= args.warmup:
            times.append(t)
    ms = float(np.mean(times)) * 1e3 * cfg.n_blocks
    sample = (f"block 0 ({len(cfg.block)} layers) per step, time x{cfg.n_blocks} blocks" if whole else
              f"block 0 whole in the first step ({t_block:.1f} s); later steps its first 2 layers x{scale:.2f} "
              f"(ratio measured in the first step), time x{cfg.n_blocks} blocks")
    line = {"metric": METRIC, "value": ms, "unit": "ms", "impl": "reference", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_string(cfg, rank_r, 0), "sample": sample},
            "cpu_baseline": {"value": ms, "unit": "ms", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": ms, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def spawn_ranks(n: int, argv, worker=None, env_extra=None, port: int | None = None):
    """Starts n local processes, one per GPU, as a launcher would: RANK / LOCAL_RANK / WORLD_SIZE /
    MASTER_ADDR / MASTER_PORT in the environment, the same command line.  `worker` replaces
    [python, bench.py] (the tests pass a stub).  Returns the exit codes in rank order."""
    import socket
    if port is None:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    cmd = list(worker) if worker is not None else [sys.executable, os.path.abspath(__file__)]
    procs = []
    for rk in range(n):
        env = dict(os.environ)
        env.update({"RANK": str(rk), "LOCAL_RANK": str(rk), "WORLD_SIZE": str(n), "LOCAL_WORLD_SIZE": str(n),
                    "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
        env.setdefault("NCCL_DEBUG", "INFO" if rk == 0 else "WARN")     # the communicator's own log stays on
        if env_extra:
            env.update(env_extra)
        procs.append(subprocess.Popen(cmd + list(argv), env=env))
    return [p.wait() for p in procs]


def max_over_ranks(ms: float, dist, device) -> float:
    """A timing is the slowest rank's: all-reduce MAX of the per-rank milliseconds (no-op for one rank)."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t)


def whole_job_units(per_rank_units: float, world: int) -> float:
    """Replicas (weak scaling): every rank does the same per-rank work, the job does world times it."""
    return per_rank_units * world


# ----------------------------------------------------------------------------- sweep
def sweep_entry(B, cfg, r, Ws, Xs, dev, local, peak, steps=3, wave_bytes=None, label=None, fused=-1):
    """One short run of the whole step on a resident layer set at rank r: step, extraction and one
    pass (CUDA events), the pass's bandwidth, the device status."""
    Vs = [torch.zeros(r, X.shape[1], dtype=torch.float32, device=dev) for X in Xs]
    layers = [B.make_layer(W=W, X=X, V=V, r=r, layer_id=i) for i, (W, X, V) in enumerate(zip(Ws, Xs, Vs))]
    arr = B.layer_array(layers)
    ctx = B.agzo_create(layers, local)
    if wave_bytes is not None:
        B.agzo_set_option(ctx, "wave_bytes", wave_bytes)
    if fused >= 0:
        B.agzo_set_option(ctx, "extract_fused", fused)
    n_fused = sum(1 for c in B.agzo_query_fused(ctx, layers, arr=arr) if c)
    losses = torch.tensor([1.0, 0.999], dtype=torch.float64, device=dev)
    ghat = torch.zeros(1, device=dev)
    stream = torch.cuda.current_stream()

    def step(seed):
        B.agzo_extract_subspace(ctx, layers, seed, K_POWER, arr=arr)
        B.agzo_perturb(ctx, layers, seed, EPS, arr=arr)
        B.agzo_perturb(ctx, layers, seed, -2 * EPS, arr=arr)
        B.agzo_ghat(ctx, losses[0:1], losses[1:2], EPS, 0, ghat)
        B.agzo_restore_update(ctx, layers, seed, EPS, LR, 0, ghat, arr=arr)

    def ms_of(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    step(0); step(1); step(2)          # warm-up
    ms_step = ms_of(lambda i: step(10 + i), steps)
    ms_extract = ms_of(lambda i: B.agzo_extract_subspace(ctx, layers, 200 + i, K_POWER, arr=arr), 2)
    ms_pass = ms_of(lambda i: B.agzo_perturb(ctx, layers, 300 + i, EPS if i % 2 == 0 else -EPS, arr=arr), 4)
    status = B.agzo_poll(ctx)
    B.agzo_destroy(ctx)
    work = algorithmic_work(cfg, r)
    gbps = work["rmw_bytes_per_pass"] / ms_pass / 1e6
    return {"workload": label or cfg.name, "r": r, "step_ms": ms_step, "extract_ms": ms_extract, "pass_ms": ms_pass,
            "pass_GBps": gbps, "pass_frac_of_measured_hbm": gbps / peak, "pass_frac_of_nominal_8TBps": gbps / 8000.0,
            "extract_GBps_fused_bytes": work["extract_bytes_fused"] / ms_extract / 1e6,
            "layers_with_fused_power_steps": n_fused,
            "device_status": B.status_string(status)}


def run_sweep(B, args, cfg_head, Ws, Xs, dev, local, peak):
    """The rest of the measurement grid, a few steps each: the other ranks of the headline layer set,
    then the 1.7B- and 0.6B-shaped sets (the big set is freed first).  For the 0.6B-shaped set, whose
    activation matrices (17 to 50 MB) fit L2, extraction is also timed in waves of one or two layers,
    so that the seven sweeps over a layer's X after the first find it in L2."""
    out = []
    for r in (1, 4, 64):
        if r != args.rank:
            out.append(sweep_entry(B, cfg_head, r, Ws, Xs, dev, local, peak, fused=args.extract_fused))
    Ws.clear(); Xs.clear()
    torch.cuda.empty_cache()
    for cfg, ranks in ((WL.QWEN3_1P7B, (4, 8, 16)), (WL.QWEN3_0P6B, (8,))):
        W2, X2, _, _ = build_layer_set(cfg, 1, dev)
        for r in ranks:
            out.append(sweep_entry(B, cfg, r, W2, X2, dev, local, peak, fused=args.extract_fused))
        if cfg is WL.QWEN3_0P6B:
            e = sweep_entry(B, cfg, 8, W2, X2, dev, local, peak, wave_bytes=56 << 20, fused=args.extract_fused,
                            label=cfg.name + ", extraction in waves of at most 56 MB of activations (X stays in L2 "
                                             "across the sweeps of a wave)")
            out.append(e)
        del W2, X2
        torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="agzo", choices=["agzo", "reference"])
    ap.add_argument("--workload", default=WL.QWEN3_8B.name, choices=sorted(WL.LAYER_SETS))
    ap.add_argument("--rank", type=int, default=16)
    ap.add_argument("--extract-path", type=int, default=0)
    ap.add_argument("--wave-mb", type=int, default=-1)
    ap.add_argument("--extract-streams", type=int, default=2)
    ap.add_argument("--extract-fused", type=int, default=-1,
                    help="-1: the library's default (fused power steps where a layer allows); 0/1/2: the option")
    ap.add_argument("--alias-inputs", action="store_true",
                    help="q/k/v and gate/up of a block read one activation buffer each (as in a real block)")
    ap.add_argument("--share-inputs", type=int, default=1)
    ap.add_argument("--rmw-path", type=int, default=0)
    ap.add_argument("--rmw-slots", type=int, default=0)
    ap.add_argument("--rmw-inflight", type=int, default=0)
    ap.add_argument("--rmw-panels", type=int, default=0)
    ap.add_argument("--rmw-stage-r", type=int, default=0)
    ap.add_argument("--method", default="agzo", choices=["agzo", "lozo", "mezo"],
                    help="agzo: the benchmarked path.  lozo / mezo: the same library's kernels arranged as those "
                         "estimators' step (Gaussian right factor instead of extraction; dense Gaussian direction), "
                         "for a like-for-like step-overhead comparison")
    ap.add_argument("--blocks", type=int, default=0,
                    help="keep only the first N transformer blocks of the layer set (profiling-sized runs)")
    ap.add_argument("--mode", type=int, default=0, choices=[0, 1],
                    help="0: two-point step, three in-place passes (the benchmarked form).  1: Algorithm 2 as printed, "
                         "one-sided difference, two passes (perturb, restore+update)")
    ap.add_argument("--shard-tokens", action="store_true",
                    help="every rank's activations are its own tokens of one batch of N x m tokens: extraction sums "
                         "the Y panels over the ranks (NCCL all-reduce through agzo_set_allreduce); the in-place "
                         "passes stay replicated.  Default: independent replicas")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the short sweep over the other ranks and layer sets that follows the headline region")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    cfg = WL.LAYER_SETS[args.workload]
    if args.blocks > 0:
        import dataclasses
        cfg = dataclasses.replace(cfg, n_blocks=min(args.blocks, cfg.n_blocks),
                                  name=f"{cfg.name}[first {min(args.blocks, cfg.n_blocks)} blocks]")
    r = args.rank
    if args.impl == "reference":
        return run_reference(args, cfg, r)
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        # started as a plain command: be the launcher (one process per GPU, NCCL over 127.0.0.1)
        if not torch.cuda.is_available() or torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus}: {torch.cuda.device_count() if torch.cuda.is_available() else 0} "
                             "CUDA devices visible")
        return max(spawn_ranks(args.gpus, sys.argv[1:]))

    from paper_2601_17261_b200 import binding as B
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the AGZO path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1 or args.shard_tokens:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29621")
        dist.init_process_group("nccl", device_id=dev, rank=rank, world_size=world)
    B.lib()   # fails loudly when the CUDA library is missing

    Ws, Xs, Vs, layers = build_layer_set(cfg, r, dev, alias_inputs=args.alias_inputs)
    arr = B.layer_array(layers)
    # a larger wave than the default needs more scratch than agzo_workspace_bytes reports
    ctx = B.agzo_create(layers, local, extra_bytes=(12 << 30) if args.wave_mb > 4096 else 0)
    B.agzo_set_option(ctx, "extract_path", args.extract_path)
    B.agzo_set_option(ctx, "rmw_path", args.rmw_path)
    B.agzo_set_option(ctx, "extract_streams", args.extract_streams)
    if args.extract_fused >= 0:
        B.agzo_set_option(ctx, "extract_fused", args.extract_fused)
    B.agzo_set_option(ctx, "share_inputs", args.share_inputs)
    B.agzo_set_option(ctx, "rmw_tc_slots", args.rmw_slots)
    B.agzo_set_option(ctx, "rmw_tc_inflight", args.rmw_inflight)
    B.agzo_set_option(ctx, "rmw_tc_panels", args.rmw_panels)
    B.agzo_set_option(ctx, "rmw_stage_r", args.rmw_stage_r)
    if args.wave_mb >= 0:
        B.agzo_set_option(ctx, "wave_bytes", args.wave_mb << 20)
    if args.shard_tokens:     # rank p holds tokens [p m, (p + 1) m) of the batch
        B.agzo_set_allreduce(ctx, B.torch_allreduce(), rank * cfg.m)
    work = algorithmic_work(cfg, r, args.alias_inputs)
    losses = torch.tensor([1.0, 0.999], dtype=torch.float64, device=dev)
    ghat = torch.zeros(1, device=dev)
    stream = torch.cuda.current_stream()

    def step(seed: int):
        if args.method == "mezo":      # dense N(0, I) direction on every weight, three passes
            for i, W in enumerate(Ws):
                B.agzo_perturb_dense(ctx, W.view(-1), seed, i, EPS)
            for i, W in enumerate(Ws):
                B.agzo_perturb_dense(ctx, W.view(-1), seed, i, -2 * EPS)
            B.agzo_ghat(ctx, losses[0:1], losses[1:2], EPS, 0, ghat)
            for i, W in enumerate(Ws):
                B.agzo_perturb_dense(ctx, W.view(-1), seed, i, EPS - LR, d_scale=None)
            return
        if args.method == "lozo":      # U V^T with both factors from the seed: no extraction
            B.agzo_fill_gaussian_basis(ctx, layers, seed, arr=arr)
        else:
            B.agzo_extract_subspace(ctx, layers, seed, K_POWER, arr=arr)
        B.agzo_perturb(ctx, layers, seed, EPS, arr=arr)
        if args.mode == 0:
            B.agzo_perturb(ctx, layers, seed, -2 * EPS, arr=arr)
        B.agzo_ghat(ctx, losses[0:1], losses[1:2], EPS, args.mode, ghat)
        B.agzo_restore_update(ctx, layers, seed, EPS, LR, args.mode, ghat, arr=arr)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, n, first_seed):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for i in range(n):
            fn(first_seed + i)
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / n, dist, dev)

    # ---- warm-up, then the timed region with the dominant kernel class bracketed by events
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    st_warm = B.agzo_poll(ctx)
    if st_warm != B.AGZO_OK:
        raise SystemExit("device status after warm-up: " + B.status_string(st_warm))
    tc_used = args.extract_path != 1
    # which layers run their power steps in the fused kernel (the library decides by shape and device);
    # the kernel class that moves most of the step's bytes is the one timed launch by launch
    fz = B.agzo_query_fused(ctx, layers, arr=arr) if args.method == "agzo" else [0] * len(layers)
    x_fused = sum({X.data_ptr(): X.numel() * X.element_size() for X, c in zip(Xs, fz) if c}.values())
    fused_dominant = tc_used and K_POWER * x_fused > work["x_bytes"] * (K_POWER + 1) - K_POWER * x_fused
    dom_class = B.KC_FUSED_POWER if fused_dominant else (B.KC_TC_XT_T if tc_used else B.KC_XT_T)
    B.agzo_read_counters(ctx)
    sampler = ClockSampler(local) if rank == 0 else None
    ms_step = timed(step, args.steps, 100)
    clocks = sampler.stop() if sampler else {}
    _, _, launches = B.agzo_read_counters(ctx)

    # ---- the dominant kernel's own launch duration: the same K steps once more with the
    # extraction waves on one stream (with two helper streams the kernels of two waves share
    # the GPU, and a launch's event-to-event time would include its neighbour's work)
    B.agzo_set_option(ctx, "extract_streams", 1)
    step(90)
    B.agzo_set_option(ctx, "time_kernel_class", dom_class)
    B.agzo_read_counters(ctx)
    ms_step_one_stream = timed(step, args.steps, 100)
    dom_ms, dom_n, _ = B.agzo_read_counters(ctx)
    B.agzo_set_option(ctx, "time_kernel_class", 0)
    B.agzo_set_option(ctx, "extract_streams", args.extract_streams)
    step(91)

    # ---- per-phase timings (outside the timed region), same kernels
    def phase_ms(fn, n=3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    ms_extract = phase_ms(lambda i: B.agzo_extract_subspace(ctx, layers, 200 + i, K_POWER, arr=arr), 2)
    ms_perturb = phase_ms(lambda i: B.agzo_perturb(ctx, layers, 300 + i, EPS if i % 2 == 0 else -EPS, arr=arr), 4)
    ms_update = phase_ms(lambda i: B.agzo_restore_update(ctx, layers, 400 + i, EPS, LR, 0, ghat, arr=arr), 4)

    # ---- end to end: the step's activations arrive from pinned host memory, ghat goes back
    e2e = None
    if not args.no_e2e:
        blk = len(cfg.block)
        pinned = [torch.empty_like(Xs[j], device="cpu").pin_memory() for j in range(blk)]
        for j in range(blk):
            pinned[j].copy_(Xs[j])
        g_host = torch.empty(1, dtype=torch.float32).pin_memory()
        h2d = sum(x.numel() * 2 for x in Xs)

        def e2e_step(seed):
            for i, X in enumerate(Xs):
                X.copy_(pinned[i % blk], non_blocking=True)
            step(seed)
            g_host.copy_(ghat, non_blocking=True)

        e2e_step(0)
        ms_e2e = timed(e2e_step, max(1, min(args.steps, 3)), 500)
        e2e = {"value": ms_e2e, "unit": "ms", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 4,
               "note": "X of every layer copied from pinned host memory each step (one block's "
                       "pinned buffers reused for all blocks), ghat copied back"}

    status = B.agzo_poll(ctx)
    peak, peak_kind = measured_peaks()
    if fused_dominant:     # K passes over the fused layers' X per step
        dom_bytes_per_step = K_POWER * x_fused
        dom_kernel = "fused_power_step_kernel"
        dom_name = dom_kernel + " (Y = X^T (X Q), X crossing HBM once)"
    else:                  # the sweep Y = X^T T: once over every X, K times more over the unfused layers' X
        dom_bytes_per_step = work["x_bytes"] + K_POWER * (work["x_bytes"] - x_fused)
        dom_kernel = "tc_xt_t_kernel" if tc_used else "xt_t_kernel"
        dom_name = dom_kernel + " (Y = X^T T)"
    x_bytes_per_launch = dom_bytes_per_step / max(dom_n / max(args.steps, 1), 1)
    dom_avg_ms = dom_ms / max(dom_n, 1)
    achieved = x_bytes_per_launch / (dom_avg_ms * 1e-3) / 1e9 if dom_n else None

    if rank == 0:
        line = {
            "metric": METRIC, "value": ms_step, "unit": "ms", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 storage, f32 arithmetic",
            "data": "synthetic", "method": args.method,
            "config": {"workload": workload_string(cfg, r, args.mode),
                       "l2": "inputs larger than L2 (weights %.1f GB + activations %.1f GB per step)"
                             % (work["w_bytes"] / 1e9, work["x_bytes"] / 1e9),
                       "replicas": world, "device_status": B.status_string(status),
                       "parallelism": ("token-sharded extraction (all-reduce of Y panels), replicated passes"
                                       if args.shard_tokens else "independent replicas"),
                       "inputs": ("q/k/v and gate/up share one activation buffer per block" if args.alias_inputs
                                  else "one activation buffer per layer")},
            "phases_ms": {"extract": ms_extract, "perturb": ms_perturb, "restore_update": ms_update},
            "rmw": {"GBps_perturb": work["rmw_bytes_per_pass"] / ms_perturb / 1e6,
                    "GBps_restore_update": work["rmw_bytes_per_pass"] / ms_update / 1e6,
                    "frac_of_%s_hbm" % peak_kind: work["rmw_bytes_per_pass"] / ms_perturb / 1e6 / peak,
                    "frac_of_nominal_8TBps": work["rmw_bytes_per_pass"] / ms_perturb / 1e6 / 8000.0},
            "extract": {"TFLOPs_algorithmic": work["extract_flops"] / ms_extract / 1e9,
                        "GBps_fused_bytes": work["extract_bytes_fused"] / ms_extract / 1e6,
                        "layers_with_fused_power_steps": sum(1 for c in fz if c),
                        "cluster_sizes": sorted(set(c for c in fz if c))},
            "roofline": {"kernel": dom_name, "bound": "hbm", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": (achieved / peak) if achieved else None,
                         "frac_of_nominal_8TBps": (achieved / 8000.0) if achieved else None,
                         "peak_kind": peak_kind,
                         "peak_note": "the peak is the copy rate measured on this pool (a read-and-write stream): a "
                                      "reference rate, not a ceiling -- a read-only sweep can exceed it",
                         "traffic": (TRAFFIC_PER_ALGORITHMIC_BYTE[dom_kernel] * x_bytes_per_launch
                                     if dom_kernel in TRAFFIC_PER_ALGORITHMIC_BYTE and dom_n else None),
                         "traffic_note": "dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture on the "
                                         "first 4 blocks of this workload, scaled by the X bytes a launch reads",
                         "launches": dom_n, "avg_ms": dom_avg_ms,
                         "measured_with": "extract_streams=1, %.2f ms per step" % ms_step_one_stream},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if args.method == "mezo":
            # the dense pass is bound by the arithmetic of its normals: instructions issued per second against
            # what the SMs can issue (4 schedulers x 32 lanes per SM and clock)
            sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
            mhz = clocks.get("sm_max_mhz") or 1965.0
            peak_alu = sm_count * 128 * mhz * 1e6 / 1e12
            ach = cfg.n_params() * DENSE_INST_PER_WEIGHT / (ms_step / 3 * 1e-3) / 1e12
            line["roofline"] = {"kernel": "dense_vec_kernel (w += c u, u ~ N(0, I) from the counter)", "bound": "alu",
                                "achieved": ach, "peak": peak_alu, "unit": "T thread-instructions/s",
                                "frac": ach / peak_alu, "traffic": None, "ms_per_pass": ms_step / 3,
                                "inst_per_weight": DENSE_INST_PER_WEIGHT,
                                "peak_note": "SMs x 128 lanes x the maximum SM clock; instructions per weight from ncu",
                                "GBps": 4 * cfg.n_params() / (ms_step / 3) / 1e6}
        if e2e:
            line["e2e"] = e2e
        if not args.no_cpu_baseline and world == 1:
            # one transformer block (every block has the same shapes): tens of seconds of CPU work
            line["cpu_baseline"] = cpu_baseline_leg(cfg, r, len(layers))
    B.agzo_destroy(ctx)
    ctx.workspace = None          # the sweep below sizes its own workspaces
    if rank == 0:
        if (not args.no_sweep and world == 1 and args.method == "agzo" and args.mode == 0 and args.blocks == 0
                and cfg is WL.QWEN3_8B and not args.alias_inputs):
            del layers, arr, Vs
            line["sweep"] = run_sweep(B, args, cfg, Ws, Xs, dev, local, peak)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
