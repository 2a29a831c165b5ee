#!/usr/bin/env python
"""Benchmark of the ADMM-Q layer solver on B200.

One "step" = one pass of the whole hot path over one layer's calibration set:
Hessian accumulation -> damping / scaling / factorisation -> T ADMM iterations -> local search
(with the error report).  The workload at N = 1 is the Qwen3-8B q_proj-shaped layer
(d_in = d_out = 4096, 262144 bf16 calibration rows, W3 asymmetric g128, T = 300).  With N > 1
ranks (one process per GPU; started by torchrun, or by this script itself when --gpus N > 1 is given
without a launcher around it) there are three modes:
  * default: every rank solves its own copy of the layer (independent problems, no data-path
    collective, "scaling": "weak");
  * --shard channels: ONE layer on all ranks -- token-sharded Hessian, one all-reduce of the n x n
    accumulator, replicated factorisation, channel-sharded ADMM loop and local search ("strong");
  * --stack-blocks B: the 7 B layers of config 5 dealt out to the ranks, wall time = slowest rank ("strong").

    python bench.py --gpus 1 --steps 3 --warmup 3
    python bench.py --gpus 8 --stack-blocks 36
    python bench.py --gpus 8 --workload cfg3_down --shard channels
    python bench.py --impl reference ...     # the fp64 CPU oracle on the host cores, bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

DTYPE = "f16x2-split (fp32 accumulate; one fp16 plane in the late iterations, where it resolves the products below fp32)"
METRIC = "admmq_layer_solve_time"
UNIT = "s"
# ncu counters of gemm_tc_kernel<2, EPI_STORE> per launch, keyed by (d_in, d_out); the capture and its command
# are summarised in profiles/gemm_tc_wupdate_4096x4096_ncu_full.txt
PRODUCT_DRAM_BYTES_PER_LAUNCH = {(4096, 4096): 381.0e6}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"],
                    bf16_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


# ---------------------------------------------------------------------------------------------------
# reference arm / cpu_baseline: the fp64 oracle on the host cores, bounded sample of the workload
# ---------------------------------------------------------------------------------------------------
def oracle_sample_seconds(spec, wl, device_for_inputs="cpu", iters=2, ls_cols=32):
    """Times the oracle, as it stands, on a bounded sample of one layer and scales the pieces to the
    whole layer.  Returns (estimated seconds per layer, description, threads)."""
    from oracle import admmq_oracle as O
    try:
        import threadpoolctl
        threads = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    n, p = spec.d_in, spec.d_out
    x0 = wl.gen_x_chunk(spec, 0, device_for_inputs).float().cpu().numpy()
    W = wl.gen_weight(spec, device_for_inputs).cpu().numpy().astype(np.float64)
    t = time.perf_counter()
    Hr = O.hessian_accumulate(None, x0)
    t_h = time.perf_counter() - t
    H = O.hessian_finalize(Hr, x0.shape[0])
    t = time.perf_counter()
    s, Ht, Ws = O.precondition(H, W)
    delta, z0 = O.grid_fit(W, spec.bits, spec.group_size, spec.symmetric)
    lam, U = O.eig_factor(Ht)
    HW = Ws @ Ht
    t_f = time.perf_counter() - t
    rho = spec.rho()
    D, V = Ws.copy(), np.zeros_like(Ws)
    t = time.perf_counter()
    for it in range(iters):
        Wc = O.w_update(lam, U, HW, D, V, rho[it])
        k, Dn = O.project(Wc + V / rho[it], s, delta, z0, spec.bits)
        _ = (np.linalg.norm(Wc - Dn), np.linalg.norm(Dn - D))
        V = V + rho[it] * (Wc - Dn)
        D = Dn
    t_it = (time.perf_counter() - t) / iters
    cols = min(ls_cols, p)
    t = time.perf_counter()
    O.local_search(H, W[:cols], k[:cols], delta[:cols], z0[:cols], spec.bits)
    t_ls = time.perf_counter() - t
    est = t_h * spec.n_chunks + t_f + t_it * spec.T + t_ls * (p / cols)
    desc = (f"oracle fp64 on {spec.name}: Hessian of 1 of {spec.n_chunks} chunks ({x0.shape[0]} rows) x{spec.n_chunks}, "
            f"scaling+grid+eigh in full, {iters} of {spec.T} ADMM iterations at full width x{spec.T / iters:g}, "
            f"local search on {cols} of {p} output channels x{p / cols:g}")
    return est, desc, threads


def run_reference(args, spec, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    for _ in range(args.warmup):
        oracle_sample_seconds(spec, wl)
    vals = []
    t0 = time.perf_counter()
    for _ in range(args.steps):
        est, desc, threads = oracle_sample_seconds(spec, wl)
        vals.append(est)
    wall = time.perf_counter() - t0
    v = float(np.mean(vals))
    # `value` and `ms_per_step` are the whole-layer time the sample's pieces scale to (the metric is a layer's
    # solve time, and the oracle needs minutes per layer); what one step really ran is under its own key
    desc += f"; value = the pieces scaled to the whole layer, one sampled step itself ran {wall / args.steps:.2f} s"
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * v,
        "sample_wall_ms_per_step": 1e3 * wall / args.steps,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": layer_config(spec, 1),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def layer_config(spec, world, parallelism=None):
    """The `config` object of a one-layer line (the same keys in both arms)."""
    return {"workload": spec.name, "d_in": spec.d_in, "d_out": spec.d_out, "n_tokens": spec.n_tokens, "T": spec.T,
            "bits": spec.bits, "group_size": spec.group_size, "layers_per_step": world,
            "l2": "inputs_exceed_l2", "parallelism": parallelism or f"layer-parallel x{world}"}


def spawn_ranks(n: int) -> int:
    """`--gpus N` with no launcher around this process: start N ranks of this same command line under
    torch.distributed.run (one process per GPU, rendezvous on 127.0.0.1) and wait for them."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def init_ranks(args):
    """(rank, world, local_rank, device or None).  NCCL on GPUs; gloo for --dry-run, which touches no GPU."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dev = None
    if not args.dry_run:
        torch.cuda.set_device(local_rank)
        dev = torch.device("cuda", local_rank)
    if world > 1 and not dist.is_initialized():
        if args.dry_run:
            dist.init_process_group("gloo")
        else:
            dist.init_process_group("nccl", device_id=dev)
    return rank, world, local_rank, dev


def finish_ranks():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def gather_objects(obj, world):
    import torch.distributed as dist
    if world == 1:
        return [obj]
    out = [None] * world
    dist.all_gather_object(out, obj)
    return out


# ---------------------------------------------------------------------------------------------------
def run_stack(args, wl):
    """Config 5: every linear layer of the first B decoder blocks, each quantized once from a seeded calibration
    set generated on the device (generation timed separately).  Default: every layer has its own calibration set
    and factorisation.  With --shared-h the projections that read the same activations in a decoder block
    (q/k/v; gate/up) share one calibration set, one Hessian and one factorisation, and their weights are stacked
    into one call: output channels are independent problems given H.
    With N > 1 ranks the calls are dealt out to the ranks (sharding.shard_layers: largest first, to the least
    loaded rank); every rank solves its share, and the time reported is the slowest rank's."""
    from paper_2605_11222_b200 import sharding
    rank, world, local_rank, dev = init_ranks(args)
    layers = wl.config5(n_blocks=args.stack_blocks)
    if args.tokens > 0:
        import dataclasses
        layers = [dataclasses.replace(l, n_tokens=args.tokens) for l in layers]
    T = layers[0].T
    # groups of layers solved in one call: [q, k, v], [o], [gate, up], [down] per block when H is shared
    groups = []
    if args.shared_h:
        per_block = 7
        for b in range(0, len(layers), per_block):
            blk = layers[b:b + per_block]
            groups += [blk[0:3], blk[3:4], blk[4:6], blk[6:7]]
    else:
        groups = [[l] for l in layers]
    import dataclasses
    # one cost-bearing stand-in per call (its d_out = the stacked width), dealt out like layers
    calls = [dataclasses.replace(g[0], d_out=sum(l.d_out for l in g), name="+".join(l.name for l in g)) for g in groups]
    mine = {c.name for c in sharding.shard_layers(calls, rank, world)}
    my_groups = [g for g, c in zip(groups, calls) if c.name in mine]
    config = {"workload": f"cfg5 first {args.stack_blocks} of 36 blocks", "layers": len(layers),
              "calls": len(groups), "shared_h": bool(args.shared_h), "n_tokens": layers[0].n_tokens, "T": T,
              "bits": layers[0].bits, "group_size": layers[0].group_size,
              "parallelism": f"layers dealt to {world} rank(s), no data-path collective"}
    if args.dry_run:
        names = gather_objects([l.name for g in my_groups for l in g], world)
        if rank == 0:
            print(json.dumps({"metric": "admmq_stack_solve_time", "value": None, "unit": "s", "n_gpus": world,
                              "scaling": "strong", "dry_run": True, "config": config, "layers_by_rank": names}))
        finish_ranks()
        return 0
    from paper_2605_11222_b200 import binding as B
    solvers = {}
    for n in sorted({g[0].d_in for g in my_groups}):
        solvers[n] = B.Solver(n, max(sum(l.d_out for l in g) for g in my_groups if g[0].d_in == n), T_max=T, device=dev)
    per_shape, gen_s, solve_ms, moves = {}, 0.0, 0.0, 0
    torch.cuda.synchronize(dev)
    if world > 1:
        torch.distributed.barrier()
    t_wall = time.perf_counter()
    for grp in my_groups:
        spec = grp[0]                                       # its calibration set serves the whole group
        sol = solvers[spec.d_in]
        t0 = time.perf_counter()
        W = torch.cat([wl.gen_weight(l, dev) for l in grp], dim=0) if len(grp) > 1 else wl.gen_weight(spec, dev)
        Xs = [wl.gen_x_chunk(spec, c, dev) for c in range(spec.n_chunks)]
        torch.cuda.synchronize(dev)
        gen_s += time.perf_counter() - t0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        sol.hessian_reset()
        for x in Xs:
            sol.hessian_accumulate(x)
        sol.factor(rho=spec.rho())
        codes, scale, zero, _ = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, report=False)
        rep, st = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero, report=True)
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1)
        solve_ms += ms
        moves += rep.moves
        key = f"{spec.d_in}x{W.shape[0]}"
        a = per_shape.setdefault(key, [0, 0.0])
        a[0] += 1
        a[1] += ms
        del Xs, W
    wall = time.perf_counter() - t_wall
    solve_s = sharding.max_over_ranks(solve_ms / 1e3)       # the job ends with its slowest rank
    wall_s = sharding.max_over_ranks(wall)
    per_rank = gather_objects({"solve_s": solve_ms / 1e3, "calls": len(my_groups), "generation_s": gen_s}, world)
    total_moves = int(sharding.sum_over_ranks(moves))
    if rank == 0:
        print(json.dumps({
            "metric": "admmq_stack_solve_time", "value": solve_s, "unit": "s", "n_gpus": world,
            "higher_is_better": False, "scaling": "strong", "data": "synthetic",
            "dtype": DTYPE, "config": config,
            "wall_s_with_generation": wall_s, "generation_s": gen_s, "local_search_moves": total_moves,
            "per_rank": per_rank,
            "per_shape": {k: {"calls": v[0], "s_per_call": v[1] / v[0] / 1e3} for k, v in per_shape.items()}}))
    finish_ranks()
    return 0


def run_channel_sharded(args, spec, wl):
    """ONE layer on all ranks (--shard channels): every rank accumulates the Hessian of its share of the
    calibration chunks, one all-reduce(sum) of the n x n fp32 accumulator gives every rank the whole H, the
    factorisation is replicated, and each rank runs the ADMM loop and the local search on its slice of output
    channels.  A step is the whole layer; its time is the slowest rank's."""
    from paper_2605_11222_b200 import sharding
    rank, world, local_rank, dev = init_ranks(args)
    slices = [list(sharding.channel_shard(spec.d_out, r, world)) for r in range(world)]
    chunks = [[sharding.token_shard(spec.n_chunks, r, world).start, sharding.token_shard(spec.n_chunks, r, world).stop]
              for r in range(world)]
    config = layer_config(spec, 1, f"one layer on {world} rank(s): token-sharded Hessian + all-reduce, "
                                   "replicated factorisation, channel-sharded ADMM and local search")
    if args.dry_run:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "scaling": "strong",
                              "dry_run": True, "config": config, "channel_slices": slices, "token_chunks": chunks}))
        finish_ranks()
        return 0
    from paper_2605_11222_b200 import binding as B
    j0, j1 = slices[rank]
    W = wl.gen_weight(spec, dev)
    mine = sharding.token_shard(spec.n_chunks, rank, world)
    Xs = {c: wl.gen_x_chunk(spec, c, dev) for c in mine}                  # this rank's token shard, resident
    sol = B.Solver(spec.d_in, j1 - j0, T_max=spec.T, device=dev)
    last = {}

    def step():
        out = sharding.solve_layer_sharded(sol, spec, W, lambda c: Xs[c])
        last["info"] = out[3]

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_step = sharding.max_over_ranks(e0.elapsed_time(e1) / args.steps)
    err = sharding.layer_error(last["info"])
    moves = int(sharding.sum_over_ranks(last["info"]["rep_ls"].moves))
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": ms_step / 1e3, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": False, "scaling": "strong",
            "vs_baseline": None, "dtype": DTYPE, "data": "synthetic", "config": config,
            "channel_slices": slices, "token_chunks": chunks, "allreduce_bytes_per_step": 4 * spec.d_in ** 2,
            "err_after_local_search": err, "local_search_moves": moves, "clocks": clocks}))
    finish_ranks()
    return 0


# ---------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tokens", type=int, default=0, help="calibration rows (0: the workload's own)")
    ap.add_argument("--workload", default="cfg2", help="cfg1 | cfg2 | cfg3_gate | cfg3_up | cfg3_down | "
                    "cfg4_k | cfg4_v | cfg4_o | cfg5_<q|k|v|o|gate|up|down>  (default: the metric's own, cfg2)")
    ap.add_argument("--iters", type=int, default=0, help="ADMM iterations T (0: the workload's own, 300)")
    ap.add_argument("--rho0", type=float, default=0.0,
                    help="first penalty of the geometric schedule (0: the workload's own, 0.1); a large value makes "
                         "a short run consist of late iterations, e.g. to profile their one-plane products")
    ap.add_argument("--stack-blocks", type=int, default=0,
                    help="instead of one layer: quantize the first B decoder blocks of config 5 (7 layers each, "
                         "36 = the whole stack), every layer once, and report the wall time")
    ap.add_argument("--shared-h", action="store_true",
                    help="with --stack-blocks: q/k/v and gate/up of a block share one Hessian and factorisation")
    ap.add_argument("--shard", default="layers", choices=["layers", "channels"],
                    help="with --gpus N > 1 and one layer: 'layers' = every rank its own layer (weak scaling), "
                         "'channels' = one layer on all ranks (token-sharded Hessian, channel-sharded solve)")
    ap.add_argument("--dry-run", action="store_true",
                    help="multi-rank plumbing only (gloo, no GPU, nothing solved): print what every rank would do")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    # --gpus N > 1 without a launcher around this process: start the N ranks here
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus)

    from paper_2605_11222_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    import dataclasses
    base = wl.named_workload(args.workload)
    if args.tokens > 0:
        base = dataclasses.replace(base, n_tokens=args.tokens)
    if args.iters > 0:
        base = dataclasses.replace(base, T=args.iters)
    if args.rho0 > 0:
        base = dataclasses.replace(base, rho0=args.rho0)

    if args.impl == "reference":
        return run_reference(args, base, wl)
    if args.stack_blocks > 0:
        return run_stack(args, wl)
    if args.shard == "channels":
        return run_channel_sharded(args, base, wl)
    spec = dataclasses.replace(base, seed=base.seed + rank)   # layer-parallel replicas: every rank its own layer

    from paper_2605_11222_b200 import binding as B, sharding
    import torch.distributed as dist
    rank, world, local_rank, dev = init_ranks(args)
    peaks = load_peaks()

    n, p, T = spec.d_in, spec.d_out, spec.T
    W = wl.gen_weight(spec, dev)
    Xs = [wl.gen_x_chunk(spec, c, dev) for c in range(spec.n_chunks)]     # resident in HBM (2 GiB at 262144 rows)
    sol = B.Solver(n, p, T_max=T, device=dev)
    codes = torch.empty(p, n, dtype=torch.uint8, device=dev)
    gs = spec.group_size or n
    scale = torch.empty(p, n // gs, dtype=torch.float32, device=dev)
    zero = torch.empty(p, n // gs, dtype=torch.float32, device=dev)
    resid = torch.empty(T, 2, dtype=torch.float32, device=dev)
    rho = spec.rho()
    last = {}

    def step(xs):
        sol.hessian_reset()
        for x in xs:
            sol.hessian_accumulate(x)
        sol.factor(rho=rho)
        sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                           zero=zero, resid=resid, report=False)
        rep, st = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero, report=True)
        last["rep"] = rep
        return rep

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        step(Xs)
    # ---- device-timed region, inputs resident, no per-kernel instrumentation ----
    l0 = sol.launch_count()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step(Xs)
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = e0.elapsed_time(e1)
    launches = sol.launch_count() - l0
    ms_step = sharding.max_over_ranks(ms_total / args.steps)
    rep = last["rep"]
    # ---- the same steps again with the library's per-kernel CUDA events on (breakdown, roofline) ----
    sol.set_timing(True)
    sol.reset_timing()
    barrier()
    for _ in range(args.steps):
        step(Xs)
    barrier()
    timing = sol.get_timing()
    sol.set_timing(False)

    # ---- the paper's pair-swap refinement after the timed path (a widened row: measured, not part of `value`) ----
    gen = torch.Generator(device="cpu")
    gen.manual_seed(spec.seed + 17)
    pairs = torch.randint(0, n, (5, 4096, 2), generator=gen, dtype=torch.int32).to(dev)
    ps_rep, _ = sol.pair_swap(W, spec.bits, spec.group_size, codes, scale, zero, pairs)
    pair_swap = {"rounds": 5, "pairs_per_round": 4096, "ms": ps_rep.ms, "rounds_applied": ps_rep.iters_run,
                 "moves": ps_rep.moves, "err_before": ps_rep.err_before, "err_after": ps_rep.err_after}

    # ---- a run with grid-refresh attempts at iterations 2..11 (another widened row: measured, not part of `value`) ----
    attempts = list(range(2, min(12, T)))
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    _, _, _, gr_rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                                         zero=zero, resid=resid, refresh_at=attempts)
    t1.record()
    torch.cuda.synchronize(dev)
    grid_refresh = {"attempt_iters": attempts, "accepted_at": gr_rep.refreshed_iter,
                    "quantize_layer_ms": gr_rep.ms, "err_admm": gr_rep.err_before}

    # ---- the same run with the element update inside the second product's epilogue instead of the row pass ----
    _, _, _, fu_rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                                         zero=zero, resid=resid, fused_epilogue=True)
    fused_variant = {"quantize_layer_ms": fu_rep.ms, "err_admm": fu_rep.err_before}

    # ---- the same run with two operand planes in every iteration, and the default run through the same call ----
    _, _, _, tp_rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                                         zero=zero, resid=resid, product_planes=2)
    c_two = codes.clone()
    _, _, _, df_rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                                         zero=zero, resid=resid)
    c_def = codes.clone()
    # ... and with the late iterations through the factorisation (one-plane products + solve) instead of the series
    _, _, _, ns_rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                                         zero=zero, resid=resid, wupdate_series=1)
    planes_variant = {"two_planes_always_ms": tp_rep.ms, "one_plane_without_series_ms": ns_rep.ms,
                      "default_ms": df_rep.ms,
                      "default_one_plane_iterations": df_rep.one_plane_iters,
                      "default_series_iterations": df_rep.series_iters,
                      "default_two_term_series_iterations": df_rep.series2_iters,
                      "default_no_product_iterations": df_rep.series0_iters,
                      "err_admm_two_planes": tp_rep.err_before, "err_admm_without_series": ns_rep.err_before,
                      "err_admm_default": df_rep.err_before,
                      "codes_equal_fraction": float((c_two == c_def).float().mean().item()),
                      "codes_equal_fraction_without_series": float((codes == c_def).float().mean().item())}
    n_series = int(df_rep.series_iters)
    n_series2 = int(df_rep.series2_iters)
    n_series0 = int(df_rep.series0_iters)
    n_one_plane = int(df_rep.one_plane_iters)

    # ---- a run whose grid comes from the MSE search for the clipping ratio, 100 candidates down to 0.8
    #      (another widened row: measured, not part of `value`), followed by the local search ----
    _, _, _, cl_rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                                         zero=zero, resid=resid, clip_points=100, clip_min_ratio=0.8)
    cl_ls, _ = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero)
    mse_clip = {"points": 100, "min_ratio": 0.8, "quantize_layer_ms": cl_rep.ms, "err_admm": cl_rep.err_before,
                "err_after_local_search": cl_ls.err_after}

    # ---- end to end through the public API: host (pinned) inputs, results read back ----
    e2e = None
    if not args.no_e2e:
        hostX = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for x in Xs]
        hostW = torch.empty(W.shape, dtype=W.dtype, pin_memory=True).copy_(W)
        h_codes = torch.empty(codes.shape, dtype=codes.dtype, pin_memory=True)
        h_scale = torch.empty(scale.shape, dtype=scale.dtype, pin_memory=True)
        h_zero = torch.empty(zero.shape, dtype=zero.dtype, pin_memory=True)
        stage = [torch.empty_like(Xs[0]) for _ in range(2)]
        copy_stream = torch.cuda.Stream(device=dev)
        main_stream = torch.cuda.current_stream(dev)

        def e2e_step():
            W.copy_(hostW, non_blocking=True)
            sol.hessian_reset()
            done = [None, None]
            for i, hx in enumerate(hostX):
                b = i % 2
                with torch.cuda.stream(copy_stream):
                    if done[b] is not None:
                        copy_stream.wait_event(done[b])
                    buf = stage[b][: hx.shape[0]]
                    buf.copy_(hx, non_blocking=True)
                    ready = torch.cuda.Event()
                    ready.record(copy_stream)
                main_stream.wait_event(ready)
                sol.hessian_accumulate(buf)
                done[b] = torch.cuda.Event()
                done[b].record(main_stream)
            sol.factor(rho=rho)
            sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, codes=codes, scale=scale,
                               zero=zero, resid=resid, report=False)
            r, _ = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero, report=True)
            h_codes.copy_(codes, non_blocking=True)
            h_scale.copy_(scale, non_blocking=True)
            h_zero.copy_(zero, non_blocking=True)
            torch.cuda.synchronize(dev)
            return r

        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            e2e_step()
        barrier()
        e2e_s = sharding.max_over_ranks((time.perf_counter() - t0) / args.steps)
        h2d = sum(x.numel() * x.element_size() for x in hostX) + hostW.numel() * 4
        d2h = h_codes.numel() + 4 * (h_scale.numel() + h_zero.numel()) + 64
        e2e = {"value": e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel: the two-plane fp16 tcgen05 product of the W-update ----
    # With d_out >= 1.5 d_in the library forms the n x n operator each iteration (first product: n rows) and applies
    # it in the second; otherwise both products have d_out rows.
    explicit_route = 2 * p >= 3 * n
    ms_p1, n_p1 = timing["wupdate_product1"]
    ms_p2, n_p2 = timing["wupdate_product2"]
    ms_1p, n_1p = timing["wupdate_one_plane"]
    rows_p1 = n if explicit_route else p
    flops_two_plane = 3 * 2.0 * n * n * (rows_p1 * n_p1 + p * n_p2)   # three 16-bit MMAs per K step of the 2-plane split
    flops_launch = 3 * 2.0 * p * n * n                               # of a launch with d_out rows
    avg_ms = (ms_p1 + ms_p2) / max(1, n_p1 + n_p2)
    achieved = flops_two_plane / max(1e-9, (ms_p1 + ms_p2) * 1e-3) / 1e12
    # DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of this kernel from its ncu capture;
    # known for the shape that was captured, null for every other
    traffic = PRODUCT_DRAM_BYTES_PER_LAUNCH.get((n, p))
    roofline = {"kernel": "gemm_tc_kernel<2,*> (W-update products: two-plane fp16, 3 MMAs per K step)", "bound": "tensor",
                "achieved": achieved, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_sustained"], "peak_source": peaks["source"] + ", bf16 sustained (fp16 and bf16 share the dense 16-bit peak)",
                "traffic": traffic, "launches": n_p1 + n_p2, "avg_launch_ms": avg_ms,
                "flops_per_full_launch": flops_launch,
                "product1_launch_ms": ms_p1 / max(1, n_p1), "product2_launch_ms": ms_p2 / max(1, n_p2)}
    w_update_ms = (ms_p1 + ms_p2 + ms_1p + timing["tridiag_solve"][0] + timing["row_split"][0]) / args.steps
    # one-plane launches: one product R (mu I - H~) per iteration of the truncated series, else both products of an
    # iteration, of which the first has rows_p1 rows
    # (the two-term series adds one p-row one-plane product per iteration; its two-plane product is timed as
    # a second product, p rows)
    flops_one_plane = args.steps * 2.0 * n * n * ((n_series + n_series2) * p +
                                                    (n_one_plane - n_series - n_series0) * (rows_p1 + p))
    executed_flops_per_step = (flops_two_plane + flops_one_plane) / args.steps
    breakdown = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps}
                 for k, v in timing.items()}

    # ---- the other timed kernels against their own rooflines (algorithmic bytes or executed flops per launch;
    #      times are CUDA events around each launch, so short kernels carry a few microseconds of launch gap) ----
    x_bytes = 2 if spec.x_dtype == "bf16" else 4
    chunk_rows = spec.n_tokens / max(1, spec.n_chunks)

    def _hbm(kind, bytes_per_launch):
        ms, cnt = timing[kind]
        if cnt == 0 or ms <= 0:
            return None
        gbs = bytes_per_launch * cnt / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "launches": cnt, "avg_launch_ms": ms / cnt}

    # solve: read Y fp32, write two fp16 planes, for d_out rows (the n rows of the operator on the explicit route).
    # row pass: reads z 4, w 4, V 4, codes 1; writes V 4, codes 1, two fp16 planes 4 bytes per element; on the
    # explicit route the same timer also takes the split of the n x n operator (maximum pass 4, split 4 + 4 bytes
    # per element), so a launch there is the mean of the two.
    def _row_pass_roofline():
        # all launches under the row-pass timer: T row passes (22 p n bytes), the splits of the two-term series'
        # intermediate (8 p n) and, on the explicit route, of the n x n operator (12 n^2) in the other iterations
        ms, cnt = timing["row_split"]
        if cnt == 0 or ms <= 0:
            return None
        n_fact = T - n_series - n_series2 - n_series0
        # (the last iterations, which form no product, are one pass over the state: 18 p n bytes for all of them)
        total = args.steps * (22.0 * p * n * (T - n_series0) + (18.0 * p * n if n_series0 else 0.0) +
                              8.0 * p * n * n_series2 + (12.0 * n * n * n_fact if explicit_route else 0.0))
        gbs = total / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "launches": cnt, "avg_launch_ms": ms / cnt}

    kernel_rooflines = {
        "tridiag_solve": _hbm("tridiag_solve", 8.0 * rows_p1 * n),
        "row_split": _row_pass_roofline(),
        "transpose": _hbm("transpose", 2.0 * x_bytes * chunk_rows * n),
    }
    if n_1p:
        tf1 = flops_one_plane / (ms_1p * 1e-3) / 1e12
        kernel_rooflines["wupdate_one_plane"] = {
            "kernel": "gemm_tc_pair_kernel (W-update products of the late iterations: one fp16 plane, CTA pairs, one "
                      "product per iteration of the truncated series; gemm_tc_kernel<1,STORE> where a product is "
                      "narrower than 256)",
            "bound": "tensor", "achieved": tf1, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
            "frac": tf1 / peaks["bf16_sustained"], "launches": n_1p, "avg_launch_ms": ms_1p / n_1p}
    ms_h, n_h = timing["hessian_product"]
    if n_h:
        planes = 1 if spec.x_dtype == "bf16" else 3
        tf = planes * 1.0 * chunk_rows * n * n * n_h / (ms_h * 1e-3) / 1e12   # lower-triangle tiles only
        kernel_rooflines["hessian_product"] = {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_sustained"],
                                               "unit": "TFLOP/s", "frac": tf / peaks["bf16_sustained"],
                                               "launches": n_h, "avg_launch_ms": ms_h / n_h}

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:            # the oracle is timed at N = 1 only
        est, desc, threads = oracle_sample_seconds(spec, wl)
        cpu_baseline = {"value": est, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    line = {
        "metric": METRIC, "value": ms_step / 1e3, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": layer_config(spec, world),
        "layers_per_s": world / (ms_step / 1e3),
        "w_update_useful_tflops": 4.0 * n * n * p * T / (w_update_ms * 1e-3) / 1e12,
        "w_update_executed_tflops": executed_flops_per_step / (w_update_ms * 1e-3) / 1e12,
        "one_plane_iterations": n_one_plane, "series_iterations": n_series, "two_term_series_iterations": n_series2, "no_product_iterations": n_series0, "w_update_route": "explicit operator" if explicit_route else "two products",
        "err_before_local_search": rep.err_before, "err_after_local_search": rep.err_after,
        "local_search_moves": rep.moves, "pair_swap_after_local_search": pair_swap, "admm_with_grid_refresh": grid_refresh,
        "admm_with_mse_clip_search": mse_clip, "admm_with_fused_epilogue": fused_variant,
        "admm_operand_planes": planes_variant,
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "kernel_rooflines": kernel_rooflines, "cpu_baseline": cpu_baseline,
        "breakdown": breakdown,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
