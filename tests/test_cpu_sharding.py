"""CPU-only checks of the multi-GPU plumbing: the within-layer sharding (token-sharded Hessian, one all-reduce,
channel-sharded solve) on two gloo ranks with a stub solver, the shard arithmetic, and bench.py's own launcher."""
import json
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_SHARD_WORKER = r'''
import dataclasses, json, sys, types
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
from paper_2605_11222_b200 import sharding, workloads as wl


class StubSolver:
    """The call surface of binding.Solver in plain torch on the CPU, with round-to-nearest as its "solve":
    enough to check what crosses ranks (token shards, the all-reduce, channel slices, the gathers)."""

    def __init__(self, n):
        self.n = n

    def hessian_reset(self):
        self.H, self.N = torch.zeros(self.n, self.n, dtype=torch.float64), 0

    def hessian_accumulate(self, x):
        self.H += x.double().T @ x.double()
        self.N += x.shape[0]

    def hessian_export(self):
        return self.H.clone(), self.N

    def hessian_import(self, H, N):
        self.H, self.N = H.clone(), N

    def factor(self, rho):
        self.Hd, self.T = self.H / self.N, len(rho)

    def _err(self, W, codes, scale, zero):
        E = (zero + scale * codes - W).double()
        return float(((E @ self.Hd) * E).sum()), E

    def quantize_layer(self, W, bits, gs, sym, resid=None, report=True):
        lo, hi = W.min(1, keepdim=True).values, W.max(1, keepdim=True).values
        delta = (hi - lo) / (2 ** bits - 1)
        codes = torch.clamp(torch.round((W - lo) / delta), 0, 2 ** bits - 1).to(torch.uint8)
        err, E = self._err(W, codes, delta, lo)
        if resid is not None:
            resid[:, 0] = E.norm()
            resid[:, 1] = (E @ self.Hd).norm()
        return codes, delta, lo, types.SimpleNamespace(err_before=err, err_after=err)

    def local_search(self, W, bits, gs, codes, scale, zero):
        err, _ = self._err(W, codes, scale, zero)
        return types.SimpleNamespace(err_before=err, err_after=err, moves=0), 0


world = int(sys.argv[4])
if world > 1:
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{sys.argv[2]}", rank=int(sys.argv[3]),
                            world_size=world)
wl.CHUNK_ROWS = 100                                   # five chunks of 100 rows: 2 + 3 over two ranks
spec = wl.small_case(64, 300, 500, group_size=0, T=3)
W = wl.gen_weight(spec)
sol = StubSolver(spec.d_in)
resid = torch.zeros(spec.T, 2, dtype=torch.float64)
codes, scale, zero, info = sharding.solve_layer_sharded(sol, spec, W, lambda c: wl.gen_x_chunk(spec, c),
                                                        resid=resid)
allc = sharding.gather_channels(codes, spec.d_out)
alls = sharding.gather_channels(scale, spec.d_out)
err = sharding.layer_error(info)
rank = dist.get_rank() if world > 1 else 0
if rank == 0:
    print(json.dumps({"codes": allc.flatten().tolist(), "scale": alls.flatten().tolist(), "err": err,
                      "H00": float(sol.Hd[0, 0]), "Hsum": float(sol.Hd.abs().sum()), "N": sol.N,
                      "resid": info["resid"].flatten().tolist(), "slice": [info["j0"], info["j1"]],
                      "chunks": list(sharding.token_shard(spec.n_chunks, rank, world))}))
if world > 1:
    dist.destroy_process_group()
'''


def _run_ranks(tmp_path, script_text, world, name):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / name
    script.write_text(script_text)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, str(port), str(r), str(world)],
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(world)]
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    return json.loads(outs[0][0].strip().splitlines()[-1])


def test_within_layer_sharding_two_ranks_gloo(tmp_path):
    """Token-sharded Hessian + one all-reduce + channel-sharded solve on two gloo ranks gives what one rank
    gives: same Hessian, same codes and grid for every channel, same layer error and residual norms."""
    one = _run_ranks(tmp_path, _SHARD_WORKER, 1, "w1.py")
    two = _run_ranks(tmp_path, _SHARD_WORKER, 2, "w2.py")
    assert one["N"] == two["N"] == 500
    assert one["chunks"] == [0, 1, 2, 3, 4] and two["chunks"] == [0, 1]
    assert two["slice"] == [0, 128] and one["slice"] == [0, 300]       # 300 channels: 128 + 172
    assert abs(one["H00"] - two["H00"]) <= 1e-12 * abs(one["H00"])
    assert abs(one["Hsum"] - two["Hsum"]) <= 1e-12 * one["Hsum"]
    assert one["codes"] == two["codes"] and len(one["codes"]) == 300 * 64
    assert one["scale"] == two["scale"]
    assert abs(one["err"] - two["err"]) <= 1e-10 * one["err"]
    assert np.allclose(one["resid"], two["resid"], rtol=1e-10)


def test_channel_and_token_shards_tile_their_ranges():
    from paper_2605_11222_b200 import sharding
    for d_out in (1, 5, 128, 300, 1024, 4096, 12288):
        for world in (1, 2, 3, 4, 8):
            parts = [sharding.channel_shard(d_out, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == d_out
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            if d_out >= 128 * world:
                assert all(j0 % 128 == 0 for j0, _ in parts) and all(j1 > j0 for j0, j1 in parts)
    for n_chunks in (1, 5, 16, 32):
        for world in (1, 2, 4, 8):
            got = [c for r in range(world) for c in sharding.token_shard(n_chunks, r, world)]
            assert got == list(range(n_chunks))


def _bench(args):
    env = dict(os.environ)
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, capture_output=True, text=True,
                       timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    return json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][-1])


def test_bench_launcher_spawns_ranks_with_disjoint_layer_sets():
    """`bench.py --gpus 2` without a launcher around it starts two ranks by itself; with --dry-run (gloo, no
    GPU, no solve) every rank reports the layers of the config-5 stack it would solve."""
    line = _bench(["--gpus", "2", "--stack-blocks", "2", "--dry-run"])
    assert line["n_gpus"] == 2 and line["scaling"] == "strong" and line["dry_run"] is True
    a, b = line["layers_by_rank"]
    assert set(a).isdisjoint(b) and len(a) + len(b) == 14 and abs(len(a) - len(b)) <= 1
    one = _bench(["--gpus", "1", "--stack-blocks", "2", "--dry-run"])
    assert one["n_gpus"] == 1 and sorted(one["layers_by_rank"][0]) == sorted(a + b)


def test_bench_dry_run_of_the_channel_sharded_layer():
    line = _bench(["--gpus", "2", "--workload", "cfg3_down", "--shard", "channels", "--dry-run"])
    assert line["n_gpus"] == 2 and line["scaling"] == "strong"
    assert line["channel_slices"] == [[0, 2048], [2048, 4096]]
    assert line["token_chunks"] == [[0, 16], [16, 32]]
