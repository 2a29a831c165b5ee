"""Shared helpers of the GPU parity tests: run the fp64 oracle on a seeded workload."""
import numpy as np
import torch

from oracle import admmq_oracle as O
from paper_2605_11222_b200 import workloads as wl


def oracle_hessian(spec, device="cpu"):
    """Damped fp64 Hessian of a workload, from the same chunks the GPU path receives."""
    Hr = None
    for c in range(spec.n_chunks):
        x = wl.gen_x_chunk(spec, c, device)
        Hr = O.hessian_accumulate(Hr, x.float().cpu().numpy())
    return O.hessian_finalize(Hr, spec.n_tokens)


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def to_dev(a: np.ndarray, dtype, device):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dtype).to(device)
