"""The allocation-free error report (admmq_objective_static) against the context-based one and the oracle.

Runs last on purpose: it shares a fixed scratch array inside the library with nothing else, and a
failure here must not hide the other GPU tests from a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

from oracle import admmq_oracle as O
from paper_2605_11222_b200 import binding as B
from paper_2605_11222_b200 import workloads as wl
from tests.helpers import np64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_objective_static_matches_context_objective_twice_in_a_row():
    from paper_2605_11222_b200 import build
    build.build()
    spec = wl.small_case(512, 200, 4096, T=12)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    sol.hessian_accumulate(wl.gen_x_chunk(spec, 0, DEV))
    sol.factor(rho=spec.rho())
    codes, scale, zero, _ = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    H, _ = sol.get_hessian()
    out = torch.full((1,), -1.0, dtype=torch.float64, device=DEV)

    # call 1: all channels, the ADMM codes
    ref1 = sol.objective(W, spec.group_size, codes, scale, zero)
    assert B.objective_static(H, W, spec.group_size, codes, scale, zero, out) == B.OK
    torch.cuda.synchronize()
    got1 = out.item()
    assert abs(got1 - ref1) <= 1e-4 * ref1, (got1, ref1)
    Hn, Wn = np64(H), np64(W)
    ora1 = O.objective(Hn, Wn, O.dequantize(codes.cpu().numpy(), np64(scale), np64(zero)))
    assert abs(got1 - ora1) <= 1e-5 * ora1, (got1, ora1)

    # call 2, right after: fewer channels and other codes -- stale scratch from call 1 must not leak in
    sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero)
    m = 77
    Wm, cm = W[:m].contiguous(), codes[:m].contiguous()
    sm, zm = scale[:m].contiguous(), zero[:m].contiguous()
    ref2 = sol.objective(Wm, spec.group_size, cm, sm, zm)
    torch.cuda.synchronize()
    free_before, alloc_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    assert B.objective_static(H, Wm, spec.group_size, cm, sm, zm, out) == B.OK
    torch.cuda.synchronize()
    # the call took no device memory, neither from the driver nor from torch's pool
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == alloc_before
    got2 = out.item()
    assert abs(got2 - ref2) <= 1e-4 * ref2, (got2, ref2)
    assert got2 < got1
    ora2 = O.objective(Hn, Wn[:m], O.dequantize(cm.cpu().numpy(), np64(sm), np64(zm)))
    assert abs(got2 - ora2) <= 1e-5 * ora2, (got2, ora2)

    # sizes beyond the fixed scratch are refused, nothing runs
    big = B.load_library().admmq_objective_static
    st = big(B._ptr(H), H.shape[0], B._ptr(W), 16385, spec.group_size, B._ptr(codes), B._ptr(scale),
             B._ptr(zero), B._ptr(out), None)
    assert st == B.ERR_SHAPE
    torch.cuda.synchronize()
    assert out.item() == got2
    assert sol.last_device_status() == B.OK
