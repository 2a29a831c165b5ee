"""CPU-only checks: the C-ABI library loads and exports every declared symbol, host-side
argument validation, workload generators, and layer sharding across ranks (gloo)."""
import ctypes as C
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_11222_b200 import build, binding
    build.build()
    return binding.load_library()


def test_library_exports_every_declared_symbol(lib):
    from paper_2605_11222_b200 import binding
    inc = os.path.join(ROOT, "include")
    header = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    declared = sorted(set(re.findall(r"\b(admmq_[a-z_0-9]+)\s*\(", header)))
    assert len(declared) >= 16
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in admmq.h but not exported"
    assert sorted(binding.EXPORTS) == declared


def test_status_strings_and_workspace_sizes(lib):
    from paper_2605_11222_b200 import binding as B
    assert B.status_string(B.OK) == "ok"
    assert "order" in B.status_string(B.ERR_STATE)
    w = lib.admmq_workspace_bytes
    assert w(4096, 4096, 300) > 0
    assert w(4096, 8192, 300) > w(4096, 4096, 300) > w(2048, 4096, 300)
    assert w(4096, 4096, 500) > w(4096, 4096, 300)
    # unsupported sizes: d_in not a multiple of 8, too large, non-positive
    for bad in [(4097, 16, 10), (14344, 16, 10), (0, 16, 10), (64, 0, 10), (64, 16, 0), (64, 16, 5000)]:
        assert w(*bad) == 0
    # config 3's largest layer fits the 180 GB part many times over
    assert w(12288, 4096, 300) < 16 * 2**30


def test_create_rejects_bad_arguments_before_touching_the_device(lib):
    from paper_2605_11222_b200 import binding as B
    h = C.c_void_p()
    fake = C.c_void_p(0x10000)          # never dereferenced: every call below fails in validation
    n = lib.admmq_workspace_bytes(64, 16, 10)
    assert lib.admmq_create(None, 64, 16, 10, fake, n, None) == B.ERR_INVALID_ARG
    assert lib.admmq_create(C.byref(h), 64, 16, 10, None, n, None) == B.ERR_INVALID_ARG
    assert lib.admmq_create(C.byref(h), 60, 16, 10, fake, n, None) == B.ERR_SHAPE
    assert lib.admmq_create(C.byref(h), 64, 16, 10, C.c_void_p(0x10010), n, None) == B.ERR_INVALID_ARG
    assert lib.admmq_create(C.byref(h), 64, 16, 10, fake, n - 1, None) == B.ERR_WORKSPACE
    assert h.value is None
    for fn in (lib.admmq_destroy, lib.admmq_hessian_reset, lib.admmq_last_device_status):
        assert fn(None) == B.ERR_INVALID_ARG
    assert lib.admmq_launch_count(None) == 0


def test_missing_library_fails_loudly(tmp_path):
    from paper_2605_11222_b200 import binding as B
    with pytest.raises(FileNotFoundError):
        B.load_library(str(tmp_path / "libadmmq.so"))


def test_product_path_does_not_import_the_oracle():
    for f in ("binding.py", "workloads.py", "__init__.py", "build.py", "sharding.py"):
        src = open(os.path.join(ROOT, "paper_2605_11222_b200", f)).read()
        assert "oracle" not in src.replace("no CPU", ""), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2605_11222_b200" not in open(os.path.join(ROOT, "oracle", f)).read()


# ------------------------------------------------------------------ workloads
def test_workloads_are_seeded_and_shaped():
    from paper_2605_11222_b200 import workloads as wl
    s = wl.small_case(64, 24, 300, n_outlier=3)
    a, b = wl.gen_x_chunk(s, 0), wl.gen_x_chunk(s, 0)
    assert a.dtype == torch.bfloat16 and a.shape == (300, 64) and torch.equal(a, b)
    assert torch.equal(wl.gen_weight(s), wl.gen_weight(s)) and wl.gen_weight(s).shape == (24, 64)
    ch = wl.outlier_channels(s)
    assert len(ch) == 3
    col_scale = a.float().abs().mean(0)
    others = torch.ones(64, dtype=torch.bool)
    others[ch] = False
    assert col_scale[ch].min() > 5 * col_scale[others].max()
    c1 = wl.config1()
    assert (c1.d_in, c1.d_out, c1.n_tokens, c1.T, c1.bits, c1.group_size) == (256, 256, 4096, 100, 3, 0)
    assert abs(c1.rho()[0] - 1e-2) < 1e-12 and abs(c1.rho()[-1] - 1e2) < 1e-9
    c2 = wl.config2()
    assert (c2.d_in, c2.d_out, c2.n_tokens, c2.T, c2.group_size, c2.outlier_count) == (4096, 4096, 262144, 300, 128, 41)
    assert [l.d_in for l in wl.config3()] == [4096, 4096, 12288]
    assert all(l.rotate and l.symmetric and l.bits == 2 and l.T == 500 for l in wl.config4())
    c5 = wl.config5()
    assert len(c5) == 252 and len({l.seed for l in c5}) == 252 and c5[6].d_in == 12288


def test_rotation_preserves_the_layer_output_and_flattens_outliers():
    from paper_2605_11222_b200 import workloads as wl
    kw = dict(x_dtype="f32", seed=3, n_outlier=2, group_size=0)
    s = wl.small_case(64, 8, 200, rotate=True, **kw)
    s0 = wl.small_case(64, 8, 200, rotate=False, **kw)
    X, W, X0, W0 = wl.gen_x_chunk(s, 0), wl.gen_weight(s), wl.gen_x_chunk(s0, 0), wl.gen_weight(s0)
    assert (X @ W.T - X0 @ W0.T).abs().max() < 1e-4
    assert X.abs().max() < 0.5 * X0.abs().max()


# ------------------------------------------------------------------ sharding across ranks (gloo, CPU)
_WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
from paper_2605_11222_b200 import sharding, workloads as wl
dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{sys.argv[2]}", rank=int(sys.argv[3]), world_size=2)
layers = wl.config5(n_blocks=2)
mine = sharding.shard_layers(layers, dist.get_rank(), dist.get_world_size())
names = [l.name for l in mine]
gathered = [None, None]
dist.all_gather_object(gathered, names)
t = sharding.max_over_ranks(1.0 + dist.get_rank())
total = sharding.sum_over_ranks(len(mine))
if dist.get_rank() == 0:
    print(json.dumps({"gathered": gathered, "tmax": t, "total": total, "all": [l.name for l in layers]}))
dist.destroy_process_group()
"""


def test_layer_sharding_two_ranks_gloo(tmp_path):
    import json
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, str(port), str(r)],
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    a, b = res["gathered"]
    assert set(a).isdisjoint(b) and sorted(a + b) == sorted(res["all"])
    assert abs(len(a) - len(b)) <= 1
    assert res["tmax"] == 2.0 and res["total"] == len(res["all"])


def test_shard_layers_balances_cost():
    from paper_2605_11222_b200 import sharding, workloads as wl
    layers = wl.config5(n_blocks=4)
    for world in (1, 2, 4, 8):
        shards = [sharding.shard_layers(layers, r, world) for r in range(world)]
        assert sorted(l.name for s in shards for l in s) == sorted(l.name for l in layers)
        costs = [sum(sharding.layer_cost(l) for l in s) for s in shards]
        assert max(costs) <= 1.35 * (sum(costs) / world) + max(sharding.layer_cost(l) for l in layers)
