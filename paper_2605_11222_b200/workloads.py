"""Seeded synthetic layer workloads (inputs only -- no solver arithmetic lives here).

Shapes follow the linear layers of an 8B-class decoder (hidden 4096, MLP 12288,
KV width 1024); values follow the "outlier channel" structure of LLM activations:
most input channels are N(0,1), a few carry much larger magnitudes.  Calibration
rows are generated in fixed chunks of `CHUNK_ROWS`, each chunk from its own seed, so
any consumer (GPU resident, host streamed) sees the same rows.

Everything is produced by torch generators on the requested device; the same call
serves the CUDA path and the CPU checker, which then see bit-identical inputs.
"""
from __future__ import annotations

import dataclasses
import math

import torch

CHUNK_ROWS = 8192


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    name: str
    d_in: int
    d_out: int
    n_tokens: int
    x_dtype: str = "bf16"          # "bf16" | "f32"
    x_kind: str = "normal"         # "normal" | "silu_like" (|z1|*z2)
    outlier: str = "student_t"     # "student_t" (x30, nu=3) | "scale20" | "none"
    n_outlier: int = -1            # -1: 1 % of d_in
    bits: int = 3
    group_size: int = 128          # 0: one group per output channel
    symmetric: bool = False
    T: int = 300
    rho0: float = 0.1
    gamma: float = 1.1
    rotate: bool = False           # seeded +-1 Hadamard rotation of X and W
    seed: int = 0

    def rho(self):
        return [self.rho0 * self.gamma ** t for t in range(self.T)]

    @property
    def outlier_count(self) -> int:
        if self.outlier == "none":
            return 0
        return self.n_outlier if self.n_outlier >= 0 else max(1, round(0.01 * self.d_in))

    @property
    def n_chunks(self) -> int:
        return (self.n_tokens + CHUNK_ROWS - 1) // CHUNK_ROWS


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def outlier_channels(spec: LayerSpec) -> torch.Tensor:
    """Indices of the outlier input channels (seeded permutation, CPU)."""
    g = _gen(spec.seed * 7919 + 3, "cpu")
    return torch.randperm(spec.d_in, generator=g)[: spec.outlier_count].sort().values


def hadamard_signs(spec: LayerSpec) -> torch.Tensor:
    g = _gen(spec.seed * 7919 + 5, "cpu")
    return (torch.randint(0, 2, (spec.d_in,), generator=g) * 2 - 1).to(torch.float32)


def fwht_(x: torch.Tensor) -> torch.Tensor:
    """Unnormalised Walsh-Hadamard transform (Sylvester order) along the last dim."""
    n = x.shape[-1]
    assert n & (n - 1) == 0
    h = 1
    lead = x.shape[:-1]
    while h < n:
        y = x.reshape(*lead, n // (2 * h), 2, h)
        a = y[..., 0, :] + y[..., 1, :]
        b = y[..., 0, :] - y[..., 1, :]
        x = torch.stack((a, b), dim=-2).reshape(*lead, n)
        h *= 2
    return x


def rotate_rows(a: torch.Tensor, signs: torch.Tensor) -> torch.Tensor:
    """a @ R with R = diag(signs) * Hadamard / sqrt(n), along the last dim (fp32)."""
    n = a.shape[-1]
    return fwht_(a.to(torch.float32) * signs.to(a.device)) / math.sqrt(n)


def gen_weight(spec: LayerSpec, device="cpu") -> torch.Tensor:
    """Pre-trained weights, [d_out, d_in] fp32, N(0, 0.02^2) (rotated if spec.rotate)."""
    g = _gen(spec.seed * 7919 + 1, device)
    w = torch.randn(spec.d_out, spec.d_in, generator=g, device=device, dtype=torch.float32) * 0.02
    if spec.rotate:
        w = rotate_rows(w, hadamard_signs(spec))
    return w.contiguous()


def gen_x_chunk(spec: LayerSpec, c: int, device="cpu") -> torch.Tensor:
    """Rows [c*CHUNK_ROWS, ...) of the calibration activations, [rows, d_in]."""
    rows = min(CHUNK_ROWS, spec.n_tokens - c * CHUNK_ROWS)
    assert rows > 0
    g = _gen(spec.seed * 7919 + 1000 + c, device)
    n = spec.d_in
    x = torch.randn(rows, n, generator=g, device=device, dtype=torch.float32)
    if spec.x_kind == "silu_like":
        x = x.abs() * torch.randn(rows, n, generator=g, device=device, dtype=torch.float32)
    m = spec.outlier_count
    if m:
        ch = outlier_channels(spec).to(device)
        if spec.outlier == "scale20":
            x[:, ch] *= 20.0
        else:  # Student-t, nu = 3: z / sqrt(chi2_3 / 3), scaled by 30
            z = torch.randn(rows, m, 4, generator=g, device=device, dtype=torch.float32)
            t = z[..., 0] / torch.sqrt((z[..., 1:] ** 2).sum(-1) / 3.0)
            x[:, ch] = 30.0 * t
    if spec.rotate:
        x = rotate_rows(x, hadamard_signs(spec))
    if spec.x_dtype == "bf16":
        x = x.to(torch.bfloat16)
    return x.contiguous()


# ---------------------------------------------------------------------------
# The five benchmark configurations and a few small parity cases.
# ---------------------------------------------------------------------------
def config1() -> LayerSpec:
    T = 100
    return LayerSpec("cfg1_256x256", 256, 256, 4096, x_dtype="f32", outlier="scale20", n_outlier=4,
                     bits=3, group_size=0, symmetric=False, T=T, rho0=1e-2,
                     gamma=(1e2 / 1e-2) ** (1.0 / (T - 1)), seed=0)


def config2(n_tokens: int = 262144) -> LayerSpec:
    return LayerSpec("cfg2_q_proj_4096x4096", 4096, 4096, n_tokens, seed=2000)


def config3(n_tokens: int = 262144):
    return [
        LayerSpec("cfg3_gate_proj", 4096, 12288, n_tokens, seed=3000),
        LayerSpec("cfg3_up_proj", 4096, 12288, n_tokens, seed=3001),
        LayerSpec("cfg3_down_proj", 12288, 4096, n_tokens, x_kind="silu_like", seed=3002),
    ]


def config4(n_tokens: int = 262144):
    kw = dict(bits=2, group_size=0, symmetric=True, T=500, rotate=True)
    return [
        LayerSpec("cfg4_k_proj", 4096, 1024, n_tokens, seed=4000, **kw),
        LayerSpec("cfg4_v_proj", 4096, 1024, n_tokens, seed=4001, **kw),
        LayerSpec("cfg4_o_proj", 4096, 4096, n_tokens, seed=4002, **kw),
    ]


def config5(n_blocks: int = 36, n_tokens: int = 131072):
    shapes = [("q", 4096, 4096, "normal"), ("k", 4096, 1024, "normal"), ("v", 4096, 1024, "normal"),
              ("o", 4096, 4096, "normal"), ("gate", 4096, 12288, "normal"),
              ("up", 4096, 12288, "normal"), ("down", 12288, 4096, "silu_like")]
    out = []
    for b in range(n_blocks):
        for i, (nm, n, p, kind) in enumerate(shapes):
            out.append(LayerSpec(f"cfg5_b{b}_{nm}", n, p, n_tokens, x_kind=kind, bits=4,
                                 seed=5000 + 7 * b + i))
    return out


def named_workload(name: str) -> LayerSpec:
    """One layer of the benchmark configurations by name: cfg1, cfg2, cfg3_<gate|up|down>,
    cfg4_<k|v|o>, cfg5_<q|k|v|o|gate|up|down> (block 0 of the 36-block stack)."""
    if name == "cfg1":
        return config1()
    if name == "cfg2":
        return config2()
    table = {}
    for s in config3() + config4():
        table[s.name.replace("_proj", "")] = s
    for s in config5(n_blocks=1):
        table[s.name.replace("_b0", "")] = s
    if name not in table:
        raise KeyError(f"unknown workload {name!r}; known: cfg1, cfg2, {', '.join(sorted(table))}")
    return table[name]


def small_case(d_in=512, d_out=384, n_tokens=6144, **kw) -> LayerSpec:
    """Mid-size parity case: several tiles and a ragged tail, seconds on the CPU checker."""
    base = dict(x_dtype="bf16", bits=3, group_size=128, T=40, rho0=0.1, gamma=1.25, seed=77,
                n_outlier=5)
    base.update(kw)
    return LayerSpec(f"small_{d_in}x{d_out}", d_in, d_out, n_tokens, **base)
