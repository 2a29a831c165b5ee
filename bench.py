#!/usr/bin/env python
"""Benchmark of the ADMM-Q layer solver on B200.

One "step" = one pass of the whole hot path over one layer's calibration set:
Hessian accumulation -> damping / scaling / factorisation -> T ADMM iterations -> local search
(with the error report).  The workload at N = 1 is the Qwen3-8B q_proj-shaped layer
(d_in = d_out = 4096, 262144 bf16 calibration rows, W3 asymmetric g128, T = 300).  With N > 1
ranks every rank solves its own layer (independent problems, no data-path collective).

    python bench.py --gpus 1 --steps 3 --warmup 3
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

METRIC = "admmq_layer_solve_time"
UNIT = "s"


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
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / args.steps,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": spec.name, "d_in": spec.d_in, "d_out": spec.d_out,
                                        "n_tokens": spec.n_tokens, "T": spec.T, "bits": spec.bits,
                                        "group_size": spec.group_size},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------------------
def run_stack(args, wl):
    """Config 5: every linear layer of the first B decoder blocks, each quantized once from a seeded calibration
    set generated on the device (generation timed separately).  Default: every layer has its own calibration set
    and factorisation.  With --shared-h the projections that read the same activations in a decoder block
    (q/k/v; gate/up) share one calibration set, one Hessian and one factorisation, and their weights are stacked
    into one call: output channels are independent problems given H."""
    from paper_2605_11222_b200 import binding as B
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
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
    solvers = {}
    for n in sorted({g[0].d_in for g in groups}):
        solvers[n] = B.Solver(n, max(sum(l.d_out for l in g) for g in groups if g[0].d_in == n), T_max=T, device=dev)
    per_shape, gen_s, solve_ms, moves = {}, 0.0, 0.0, 0
    torch.cuda.synchronize(dev)
    t_wall = time.perf_counter()
    for grp in groups:
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
    print(json.dumps({
        "metric": "admmq_stack_solve_time", "value": solve_ms / 1e3, "unit": "s", "n_gpus": 1,
        "higher_is_better": False, "data": "synthetic", "dtype": "f16x2-split (fp32 accumulate)",
        "config": {"workload": f"cfg5 first {args.stack_blocks} of 36 blocks", "layers": len(layers),
                   "calls": len(groups), "shared_h": bool(args.shared_h),
                   "n_tokens": layers[0].n_tokens, "T": T, "bits": layers[0].bits, "group_size": layers[0].group_size},
        "wall_s_with_generation": wall, "generation_s": gen_s, "local_search_moves": moves,
        "per_shape": {k: {"calls": v[0], "s_per_call": v[1] / v[0] / 1e3} for k, v in per_shape.items()}}))
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
    ap.add_argument("--stack-blocks", type=int, default=0,
                    help="instead of one layer: quantize the first B decoder blocks of config 5 (7 layers each, "
                         "36 = the whole stack), every layer once, and report the wall time")
    ap.add_argument("--shared-h", action="store_true",
                    help="with --stack-blocks: q/k/v and gate/up of a block share one Hessian and factorisation")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2605_11222_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    import dataclasses
    base = wl.named_workload(args.workload)
    if args.tokens > 0:
        base = dataclasses.replace(base, n_tokens=args.tokens)
    spec = dataclasses.replace(base, seed=base.seed + rank)
    if args.iters > 0:
        spec = dataclasses.replace(spec, T=args.iters)

    if args.impl == "reference":
        return run_reference(args, spec, wl)
    if args.stack_blocks > 0:
        return run_stack(args, wl)

    from paper_2605_11222_b200 import binding as B, sharding
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
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

    # ---- roofline of the dominant kernel: the split-bf16 tcgen05 product of the W-update ----
    ms_p1, n_p1 = timing["wupdate_product1"]
    ms_p2, n_p2 = timing["wupdate_product2"]
    flops_launch = 3 * 2.0 * p * n * n                     # three 16-bit MMAs per K step of the 2-plane split
    avg_ms = (ms_p1 + ms_p2) / max(1, n_p1 + n_p2)
    achieved = flops_launch / (avg_ms * 1e-3) / 1e12
    # DRAM bytes per launch from the committed ncu summary (both products store their result: the plain epilogue)
    traffic = None
    prof = os.path.join(ROOT, "profiles", "gemm_tc_wupdate_4096x4096_ncu_full.txt")
    if os.path.exists(prof) and (n, p) == (4096, 4096):
        vals = {}
        for ln in open(prof):
            if ln.startswith("traffic_bytes_per_launch_"):
                k, v = ln.strip().split("=")
                vals[k] = float(v)
        traffic = vals.get("traffic_bytes_per_launch_plain")
    roofline = {"kernel": "gemm_tc_kernel<2,*> (W-update products: two-plane fp16, 3 MMAs per K step)", "bound": "tensor",
                "achieved": achieved, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_sustained"], "peak_source": peaks["source"] + ", bf16 sustained (fp16 and bf16 share the dense 16-bit peak)",
                "traffic": traffic, "launches": n_p1 + n_p2, "avg_launch_ms": avg_ms,
                "product1_launch_ms": ms_p1 / max(1, n_p1), "product2_launch_ms": ms_p2 / max(1, n_p2)}
    w_update_ms = (ms_p1 + ms_p2 + timing["tridiag_solve"][0] + timing["row_split"][0]) / args.steps
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

    kernel_rooflines = {
        "tridiag_solve": _hbm("tridiag_solve", 8.0 * p * n),          # read Y fp32, write two fp16 planes
        "row_split": _hbm("row_split", 22.0 * p * n),                 # element update + plane split
        "transpose": _hbm("transpose", 2.0 * x_bytes * chunk_rows * n),
    }
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
        "vs_baseline": None, "dtype": "f16x2-split (fp32 accumulate)", "data": "synthetic",
        "config": {"workload": spec.name, "d_in": n, "d_out": p, "n_tokens": spec.n_tokens, "T": T,
                   "bits": spec.bits, "group_size": spec.group_size, "layers_per_step": world,
                   "l2": "inputs_exceed_l2", "parallelism": f"layer-parallel x{world}"},
        "layers_per_s": world / (ms_step / 1e3),
        "w_update_useful_tflops": 4.0 * n * n * p * T / (w_update_ms * 1e-3) / 1e12,
        "w_update_executed_tflops": 12.0 * n * n * p * T / (w_update_ms * 1e-3) / 1e12,
        "err_before_local_search": rep.err_before, "err_after_local_search": rep.err_after,
        "local_search_moves": rep.moves, "pair_swap_after_local_search": pair_swap, "admm_with_grid_refresh": grid_refresh,
        "admm_with_mse_clip_search": mse_clip, "admm_with_fused_epilogue": fused_variant,
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
