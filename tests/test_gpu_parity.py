"""GPU parity: every step of the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs.  Tolerances (spec bars; the W-update and Hessian ones follow from fp32
accumulation of 22-bit two-plane operands and of exact bf16 products):
  * integer codes: exact on the tiny / brute-force cases, >= 99.9 % equal on larger layers;
  * layer reconstruction error within 1e-3 relative of the oracle's;
  * one W-update from identical (D, V): 1e-4 relative Frobenius;
  * Hessian entries: 1e-4 relative to the Frobenius norm (fp32 accumulation of bf16 products).
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import admmq_oracle as O
from paper_2605_11222_b200 import binding as B
from paper_2605_11222_b200 import workloads as wl
from tests.helpers import np64, oracle_hessian, to_dev

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

W_UPDATE_TOL = 1e-4
CODE_AGREEMENT = 0.999
ERR_TOL = 1e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2605_11222_b200 import build
    build.build()
    B.load_library()


def _solve_gpu(spec, gemm_kind=B.GEMM_TENSOR, local_search=True, precondition=True):
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=max(spec.T, 2))
    sol.set_gemm_kind(gemm_kind)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho(), precondition=precondition)
    resid = torch.zeros(spec.T, 2, device=DEV)
    Wq = torch.empty_like(W)
    codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, Wq=Wq,
                                                 resid=resid)
    out = dict(sol=sol, W=W, codes_admm=codes.clone(), scale=scale, zero=zero, rep=rep,
               resid=resid.cpu().numpy(), Wq_admm=Wq.clone())
    if local_search:
        rep2, st = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero, Wq=Wq)
        out.update(codes_final=codes, rep_ls=rep2, st_ls=st, Wq_final=Wq)
    assert sol.last_device_status() == B.OK
    return out


def _solve_oracle(spec, H=None, cols=None):
    Wn = np64(wl.gen_weight(spec, DEV))
    if cols is not None:
        Wn = Wn[cols]
    H = oracle_hessian(spec, DEV) if H is None else H
    res = O.quantize_layer(H, Wn, spec.bits, spec.group_size, spec.symmetric, np.array(spec.rho()))
    return H, Wn, res


# ------------------------------------------------------------------ step 1-2: Hessian, damping, scaling
@pytest.mark.parametrize("x_dtype,n,N", [("bf16", 520, 6000), ("f32", 264, 9000), ("bf16", 64, 100)])
@pytest.mark.parametrize("kind", [B.GEMM_TENSOR, B.GEMM_SIMT])
def test_hessian_parity(x_dtype, n, N, kind):
    spec = wl.small_case(n, 16, N, x_dtype=x_dtype, group_size=0, T=2)
    sol = B.Solver(n, 16, T_max=2)
    sol.set_gemm_kind(kind)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=[0.1, 0.2])
    Hg, sg = sol.get_hessian()
    Ho = oracle_hessian(spec, DEV)
    Hg = np64(Hg)
    assert np.array_equal(Hg, Hg.T)
    assert np.linalg.norm(Hg - Ho) <= 1e-4 * np.linalg.norm(Ho)
    assert np.abs(np64(sg) - np.sqrt(np.diag(Ho))).max() <= 1e-4 * np.sqrt(np.diag(Ho)).max()
    # sampled entries against the entry-wise definition H_ab = sum_t X_ta X_tb / N (+ damping on a = b)
    X = torch.cat([wl.gen_x_chunk(spec, c, DEV) for c in range(spec.n_chunks)]).double()
    lam = 0.01 * float((X * X).sum(0).mean() / N)
    for a, b in [(0, 0), (n - 1, 3), (n // 2, n // 2 + 1), (n - 1, n - 1)]:
        ref = float((X[:, a] * X[:, b]).sum() / N) + (lam if a == b else 0.0)
        assert abs(Hg[a, b] - ref) <= 1e-4 * max(abs(ref), np.sqrt(Ho[a, a] * Ho[b, b]) * 1e-2)
    assert sol.last_device_status() == B.OK


def test_hessian_chunking_is_immaterial():
    spec = wl.small_case(256, 16, 5000, group_size=0, T=2)
    X = torch.cat([wl.gen_x_chunk(spec, c, DEV) for c in range(spec.n_chunks)])
    outs = []
    for pieces in ([5000], [1234, 3766], [100] * 50):
        sol = B.Solver(256, 16, T_max=2)
        sol.hessian_reset()
        a = 0
        for m in pieces:
            sol.hessian_accumulate(X[a:a + m])
            a += m
        sol.factor(rho=[0.1, 0.2])
        outs.append(np64(sol.get_hessian()[0]))
    for o in outs[1:]:
        assert np.linalg.norm(o - outs[0]) <= 2e-5 * np.linalg.norm(outs[0])


# ------------------------------------------------------------------ step 5-6: one W-update from identical (D, V)
@pytest.mark.parametrize("n,p,gs", [(512, 384, 128), (328, 130, 0)])
@pytest.mark.parametrize("kind", [B.GEMM_TENSOR, B.GEMM_SIMT])
def test_w_update_parity(n, p, gs, kind):
    spec = wl.small_case(n, p, 4096, group_size=gs, T=2)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(n, p, T_max=2)
    sol.set_gemm_kind(kind)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=[0.1, 0.2])
    Ho = oracle_hessian(spec, DEV)
    Wn = np64(W)
    delta, z0 = O.grid_fit(Wn, spec.bits, gs, False)
    s, Ht, Ws = O.precondition(Ho, Wn)
    lam, U = O.eig_factor(Ht)
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 1 << spec.bits, size=Wn.shape).astype(np.uint8)
    V = (0.01 * np.abs(Ws).mean() * rng.standard_normal(Wn.shape)).astype(np.float32)
    D = s[None, :] * O.dequantize(codes, delta, z0)
    for rho in (0.05, 0.1, 1.0, 37.0, 1e4):
        Wo = O.w_update(lam, U, Ws @ Ht, D, V.astype(np.float64), rho)
        Wg = sol.w_update(W, gs, to_dev(codes, torch.uint8, DEV), to_dev(delta, torch.float32, DEV),
                          to_dev(z0, torch.float32, DEV), to_dev(V, torch.float32, DEV), rho)
        rel = np.linalg.norm(np64(Wg) - Wo) / np.linalg.norm(Wo)
        assert rel <= W_UPDATE_TOL, (rho, rel)
    assert sol.last_device_status() == B.OK


@pytest.mark.parametrize("n,p", [(520, 264), (1024, 512)])
def test_w_update_as_truncated_series_at_large_penalties(n, p):
    """rho (H~ + rho I)^{-1} = c (I + E + E^2 + ...), E = (mu I - H~) / (mu + rho) (Eq. 7 rearranged).  The late
    iterations keep c R + c R E, those before them one more term; what they drop is bounded by gamma^2 ||R||
    (gamma^3) with gamma = max |mu - lambda| / (mu + rho).  Checked against the fp64 W-update of the oracle at
    penalties on both sides of the solver's switches (gamma <= 2^-13, 2^-9): the error follows the bound where the
    truncation dominates and sits at the level of the route through the factorisation where it does not."""
    spec = wl.small_case(n, p, 4096, group_size=0, T=2)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(n, p, T_max=2)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=[0.1, 0.2])
    Ho = oracle_hessian(spec, DEV)
    Wn = np64(W)
    delta, z0 = O.grid_fit(Wn, spec.bits, 0, False)
    s, Ht, Ws = O.precondition(Ho, Wn)
    lam, U = O.eig_factor(Ht)
    mu = float(np.trace(Ht)) / n
    rng = np.random.default_rng(11)
    codes = rng.integers(0, 1 << spec.bits, size=Wn.shape).astype(np.uint8)
    V = (0.01 * np.abs(Ws).mean() * rng.standard_normal(Wn.shape)).astype(np.float32)
    D = s[None, :] * O.dequantize(codes, delta, z0)
    args = (W, 0, to_dev(codes, torch.uint8, DEV), to_dev(delta, torch.float32, DEV),
            to_dev(z0, torch.float32, DEV), to_dev(V, torch.float32, DEV))
    spread = max(abs(mu - lam.min()), abs(mu - lam.max()))
    for gamma in (2.0 ** -6, 2.0 ** -9, 2.0 ** -10, 2.0 ** -13, 2.0 ** -16, 2.0 ** -26, 2.0 ** -29):
        rho = spread / gamma - mu
        Zo = O.w_update(lam, U, Ws @ Ht, D, V.astype(np.float64), rho) - Ws      # W - W_hat' in fp64
        R = D - V.astype(np.float64) / rho - Ws
        Ze = np64(sol.w_update_correction(*args, rho))
        err_exact = np.linalg.norm(Ze - Zo) / np.linalg.norm(R)
        assert err_exact <= 4e-7, (gamma, err_exact)
        Z1 = np64(sol.w_update_series(*args, rho, terms=1))
        Z2 = np64(sol.w_update_series(*args, rho, terms=2))
        err1 = np.linalg.norm(Z1 - Zo) / np.linalg.norm(R)
        err2 = np.linalg.norm(Z2 - Zo) / np.linalg.norm(R)
        # truncation (<= gamma^(terms+1) / (1 - gamma)) plus the rounding of the products: a one-plane product of
        # relative size gamma (one term), a two-plane one of size gamma and a one-plane one of size gamma^2 (two)
        assert err1 <= gamma ** 2 / (1 - gamma) + gamma * 2.0 ** -11 + 4e-7, (gamma, err1)
        assert err2 <= gamma ** 3 / (1 - gamma) + gamma * 2.0 ** -20 + gamma ** 2 * 2.0 ** -11 + 4e-7, (gamma, err2)
        Z0 = np64(sol.w_update_series(*args, rho, terms=0))      # c R alone
        err0 = np.linalg.norm(Z0 - Zo) / np.linalg.norm(R)
        assert err0 <= gamma / (1 - gamma) + 4e-7, (gamma, err0)
        if gamma <= 2.0 ** -26:                                  # where the solver drops the product
            assert err0 <= 2.0 ** -22, (gamma, err0)
        if gamma <= 2.0 ** -13:                                  # where the solver uses one term: fp32 resolution
            assert err1 <= 2.0 ** -22, (gamma, err1)
        if gamma <= 2.0 ** -9:                                   # ... and two terms
            assert err2 <= 2.0 ** -22, (gamma, err2)
    assert sol.last_device_status() == B.OK


# ------------------------------------------------------------------ whole layer, mid size
@pytest.mark.parametrize("kw", [
    dict(d_in=512, d_out=384, n_tokens=6144),                                   # g128, asym, 3 bit
    dict(d_in=328, d_out=130, n_tokens=3000, group_size=0, bits=4),             # ragged tiles, per-channel
    dict(d_in=256, d_out=200, n_tokens=3000, group_size=0, bits=2, symmetric=True, rotate=True),
    dict(d_in=384, d_out=64, n_tokens=2048, group_size=64, x_kind="silu_like"),
])
def test_layer_parity_mid_size(kw):
    spec = wl.small_case(**kw)
    g = _solve_gpu(spec)
    H, Wn, res = _solve_oracle(spec)
    a = res.admm
    assert np.allclose(g["scale"].cpu().numpy(), a.delta, rtol=2e-7, atol=0)
    assert np.allclose(g["zero"].cpu().numpy(), a.z0, rtol=1e-7, atol=0)
    cg = g["codes_admm"].cpu().numpy()
    assert cg.max() <= (1 << spec.bits) - 1
    assert (cg == a.codes).mean() >= CODE_AGREEMENT
    # reconstruction error of the GPU's codes, evaluated by the oracle, against the oracle's own
    e_g = O.objective(H, Wn, O.dequantize(cg, a.delta, a.z0))
    assert abs(e_g - res.err_admm) <= ERR_TOL * res.err_admm
    assert abs(g["rep"].err_before - e_g) <= ERR_TOL * e_g                   # the GPU's own error report
    # dequantised output is the grid point of its codes
    assert np.allclose(g["Wq_admm"].cpu().numpy(), O.dequantize(cg, a.delta, a.z0), rtol=1e-6, atol=3e-8)
    # residual traces (Theorem 1 quantities); the fp32 floor shows only once they are ~1e-6 of the start
    r = g["resid"]
    assert np.abs(r[:, 0] - a.r).max() <= 1e-3 * a.r.max()
    assert np.abs(r[:, 1] - a.sres).max() <= 2e-2 * a.sres.max()
    # after local search
    cf = g["codes_final"].cpu().numpy()
    assert (cf == res.ls.codes).mean() >= CODE_AGREEMENT
    e_f = O.objective(H, Wn, O.dequantize(cf, a.delta, a.z0))
    assert abs(e_f - res.err_final) <= ERR_TOL * res.err_final
    assert e_f <= e_g * (1 + 1e-9)
    assert abs(g["rep_ls"].err_after - e_f) <= ERR_TOL * e_f
    # the GPU's final point is a 1-move local optimum in the oracle's fp64 arithmetic, up to fp32 slack
    again = O.local_search(H, Wn, cf, a.delta, a.z0, spec.bits, tau=1e-6)
    assert again.moves.sum() <= 1e-3 * cf.size
    assert O.objective(H, Wn, again.Wq) >= e_f * (1 - 1e-5)


def test_local_search_from_identical_codes():
    spec = wl.small_case(512, 96, 4096, bits=3)
    g = _solve_gpu(spec, local_search=False)
    H, Wn, _ = _solve_oracle(spec)
    codes = g["codes_admm"].clone()
    cg = codes.cpu().numpy()
    delta, z0 = O.grid_fit(Wn, spec.bits, spec.group_size, spec.symmetric)
    ls = O.local_search(H, Wn, cg, delta, z0, spec.bits)
    rep, st = g["sol"].local_search(g["W"], spec.bits, spec.group_size, codes, g["scale"], g["zero"])
    assert st == B.OK
    assert (codes.cpu().numpy() == ls.codes).mean() >= 0.9999
    assert abs(rep.moves - int(ls.moves.sum())) <= max(3, 1e-3 * ls.moves.sum())
    e = O.objective(H, Wn, ls.Wq)
    assert abs(rep.err_after - e) <= ERR_TOL * e
    # move cap: a warning status, never more than the cap per column
    codes2 = g["codes_admm"].clone()
    rep2, st2 = g["sol"].local_search(g["W"], spec.bits, spec.group_size, codes2, g["scale"], g["zero"],
                                      max_moves_per_col=2)
    assert st2 == B.WARN_MOVE_CAP and rep2.capped_columns > 0 and rep2.moves <= 2 * spec.d_out
    ls2 = O.local_search(H, Wn, cg, delta, z0, spec.bits, max_moves=2)
    assert (codes2.cpu().numpy() == ls2.codes).mean() >= 0.9999


def test_tensor_and_simt_products_agree():
    spec = wl.small_case(512, 256, 4096)
    a = _solve_gpu(spec, B.GEMM_TENSOR)
    b = _solve_gpu(spec, B.GEMM_SIMT)
    assert (a["codes_admm"] == b["codes_admm"]).float().mean().item() >= CODE_AGREEMENT
    assert abs(a["rep"].err_before - b["rep"].err_before) <= ERR_TOL * b["rep"].err_before


# ------------------------------------------------------------------ config 1 in full
def test_config1_full():
    spec = wl.config1()
    g = _solve_gpu(spec)
    H, Wn, res = _solve_oracle(spec)
    cg = g["codes_admm"].cpu().numpy()
    assert (cg == res.admm.codes).mean() >= CODE_AGREEMENT
    cf = g["codes_final"].cpu().numpy()
    assert (cf == res.ls.codes).mean() >= CODE_AGREEMENT
    e_f = O.objective(H, Wn, O.dequantize(cf, res.admm.delta, res.admm.z0))
    assert abs(e_f - res.err_final) <= ERR_TOL * res.err_final
    rtn = O.dequantize(O.project(Wn, np.ones(spec.d_in), res.admm.delta, res.admm.z0, spec.bits)[0],
                       res.admm.delta, res.admm.z0)
    assert e_f < O.objective(H, Wn, rtn)


# ------------------------------------------------------------------ tiny cases: exact codes, brute force
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_tiny_exact_and_brute_force(seed):
    n, p, bits = 8, 5, 2
    rng = np.random.default_rng(200 + seed)
    X = rng.standard_normal((64, n))
    X[:, seed % n] *= 5.0
    Hn = (X.T @ X / 64).astype(np.float32)                       # undamped Hessian, handed over directly
    Wn = (0.02 * rng.standard_normal((p, n))).astype(np.float32)
    rho = O.rho_schedule(40, 0.05, 1.3)
    sol = B.Solver(n, p, T_max=40)
    sol.hessian_set(to_dev(Hn, torch.float32, DEV))
    sol.factor(rho=list(rho))
    W = to_dev(Wn, torch.float32, DEV)
    codes, scale, zero, rep = sol.quantize_layer(W, bits, 0, False)
    H = O.hessian_finalize(Hn.astype(np.float64), 1)
    res = O.quantize_layer(H, Wn.astype(np.float64), bits, 0, False, rho)
    assert np.array_equal(codes.cpu().numpy(), res.admm.codes)
    sol.local_search(W, bits, 0, codes, scale, zero)
    mine = codes.cpu().numpy()
    assert np.array_equal(mine, res.ls.codes)
    # brute force over all 4^8 assignments per column: 1-move local optimum
    all_codes = np.array(list(itertools.product(range(4), repeat=n)))
    delta, z0 = res.admm.delta, res.admm.z0
    for j in range(p):
        E = z0[j, 0] + delta[j, 0] * all_codes - Wn[j].astype(np.float64)[None, :]
        loss = np.einsum("ci,ik,ck->c", E, H, E)
        w = 4 ** np.arange(n - 1, -1, -1)
        my = loss[int(mine[j].astype(int) @ w)]
        assert my >= loss.min() - 1e-15
        for i in range(n):
            for sg in (1, -1):
                nb = mine[j].astype(int).copy()
                nb[i] += sg
                if 0 <= nb[i] <= 3:
                    assert loss[int(nb @ w)] >= my - 1e-6 * H[i, i] * delta[j, 0] ** 2 - 1e-12
    assert sol.last_device_status() == B.OK


def test_diagonal_hessian_gives_rtn():
    n, p, bits = 64, 24, 3
    rng = np.random.default_rng(12)
    Wn = (0.02 * rng.standard_normal((p, n))).astype(np.float32)
    Hn = np.diag(np.exp(rng.standard_normal(n))).astype(np.float32)
    W = to_dev(Wn, torch.float32, DEV)
    delta, z0 = O.grid_fit(Wn.astype(np.float64), bits, 0, False)
    rtn = O.project(Wn.astype(np.float64), np.ones(n), delta, z0, bits)[0]
    for rho in ([1.0 * 1.2 ** t for t in range(30)], [0.05]):                 # rho >= 1 always; T = 1
        sol = B.Solver(n, p, T_max=30)
        sol.hessian_set(to_dev(Hn, torch.float32, DEV))
        sol.factor(rho=rho, damp_frac=0.0)
        codes, scale, zero, _ = sol.quantize_layer(W, bits, 0, False)
        assert np.array_equal(codes.cpu().numpy(), rtn)
    sol = B.Solver(n, p, T_max=60)                                           # any schedule + local search
    sol.hessian_set(to_dev(Hn, torch.float32, DEV))
    sol.factor(rho=[0.01 * 1.2 ** t for t in range(60)], damp_frac=0.0)
    codes, scale, zero, _ = sol.quantize_layer(W, bits, 0, False)
    sol.local_search(W, bits, 0, codes, scale, zero)
    assert np.array_equal(codes.cpu().numpy(), rtn)


# ------------------------------------------------------------------ edge cases and error paths (no GPU fault)
def test_degenerate_inputs():
    n, p = 64, 3
    spec = wl.small_case(n, p, 512, group_size=16, T=5)
    W = wl.gen_weight(spec, DEV)
    W[1, 16:32] = 0.0125                                          # a constant group: Delta = 1, codes 0
    W[2, :] = 0.0                                                 # a constant channel
    sol = B.Solver(n, p, T_max=5)
    sol.hessian_reset()
    sol.hessian_accumulate(wl.gen_x_chunk(spec, 0, DEV))
    sol.hessian_accumulate(wl.gen_x_chunk(spec, 0, DEV)[:0])      # an empty chunk is a no-op
    sol.factor(rho=spec.rho())
    codes, scale, zero, rep = sol.quantize_layer(W, 3, 16, False)
    assert scale[1, 1].item() == 1.0 and zero[1, 1].item() == pytest.approx(0.0125)
    assert codes[1, 16:32].max().item() == 0 and codes[2].max().item() == 0
    sol.local_search(W, 3, 16, codes, scale, zero)
    assert codes[1, 16:32].max().item() == 0 and codes[2].max().item() == 0
    assert sol.last_device_status() == B.OK
    # caller-supplied grid is honoured
    Hh, _ = sol.get_hessian()
    sc = torch.full((p, n // 16), 0.01, device=DEV)
    zr = torch.full((p, n // 16), -0.035, device=DEV)
    c2, s2, z2, _ = sol.quantize_layer(W, 3, 16, False, scale=sc, zero=zr, use_caller_grid=True)
    assert torch.equal(s2, sc) and torch.equal(z2, zr) and c2.max().item() <= 7


def test_error_paths():
    n, p = 64, 4
    spec = wl.small_case(n, p, 256, group_size=0, T=3)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(n, p, T_max=3)
    lib = sol.lib
    with pytest.raises(B.AdmmqError) as e:                        # factor before any Hessian
        sol.factor(rho=[0.1])
    assert e.value.status == B.ERR_STATE
    with pytest.raises(B.AdmmqError) as e:                        # accumulate before reset
        sol.hessian_accumulate(wl.gen_x_chunk(spec, 0, DEV))
    assert e.value.status == B.ERR_STATE
    sol.hessian_reset()
    sol.hessian_accumulate(wl.gen_x_chunk(spec, 0, DEV))
    with pytest.raises(B.AdmmqError) as e:                        # quantize before factor
        sol.quantize_layer(W, 3)
    assert e.value.status == B.ERR_STATE
    for bad in (dict(rho=[0.1, -1.0]), dict(rho=[0.1] * 4), dict(rho=[0.1], kind=2)):
        with pytest.raises(B.AdmmqError) as e:
            sol.factor(**bad)
        assert e.value.status in (B.ERR_INVALID_ARG, B.ERR_SHAPE, B.ERR_UNSUPPORTED)
    sol.factor(rho=[0.1, 0.2, 0.4])
    for kw in (dict(bits=1), dict(bits=9), dict(bits=3, group_size=48)):
        with pytest.raises(B.AdmmqError) as e:
            sol.quantize_layer(W, **kw)
        assert e.value.status == B.ERR_SHAPE
    with pytest.raises(B.AdmmqError) as e:                        # more output channels than the context holds
        sol.quantize_layer(torch.zeros(p + 1, n, device=DEV), 3)
    assert e.value.status == B.ERR_SHAPE
    with pytest.raises(B.AdmmqError) as e:                        # misaligned pointer
        sol.quantize_layer(torch.zeros(p * n + 1, device=DEV)[1:].view(p, n), 3)
    assert e.value.status == B.ERR_INVALID_ARG
    # non-finite weights: reported through the device status word, nothing faults
    Wbad = W.clone()
    Wbad[0, 0] = float("nan")
    with pytest.raises(B.AdmmqError) as e:
        sol.quantize_layer(Wbad, 3)
    assert e.value.status == B.ERR_NONFINITE
    # the error was reported once: the same context, on the same factorisation, then solves a valid matrix
    assert sol.last_device_status() == B.OK
    codes, scale, zero, rep = sol.quantize_layer(W, 3)
    rep_ls, st = sol.local_search(W, 3, 0, codes, scale, zero)
    assert st == B.OK and sol.last_device_status() == B.OK
    Ho = oracle_hessian(spec, DEV)
    res = O.quantize_layer(Ho, np64(W), 3, 0, False, np.array([0.1, 0.2, 0.4]))
    assert (codes.cpu().numpy() == res.ls.codes).mean() >= CODE_AGREEMENT
    # a Hessian with a non-positive diagonal entry: NOT_SPD through the status word
    sol2 = B.Solver(n, p, T_max=3)
    Hbad = torch.eye(n, device=DEV)
    Hbad[5, 5] = -1.0
    sol2.hessian_set(Hbad)
    sol2.factor(rho=[0.1], damp_frac=0.0)
    assert sol2.last_device_status() == B.ERR_NOT_SPD
    # the context is still usable afterwards
    sol2.hessian_set(torch.eye(n, device=DEV))
    sol2.factor(rho=[0.1], damp_frac=0.0)
    assert sol2.last_device_status() == B.OK


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """Failure detection without a fault: the product kernel's producer withholds its loads (a barrier that
    nothing completes), the bound of the waits is set to about a millisecond, and every CTA must leave through
    its time-out path -- status ADMMQ_ERR_TIMEOUT, tensor memory freed, kernel returned.  The same context, with
    the hook off again, then solves the layer and matches the oracle."""
    spec = wl.small_case(512, 384, 4096, T=4)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    assert sol.last_device_status() == B.OK
    sol.test_set_wait(2_000_000, hold_loads=True)
    with pytest.raises(B.AdmmqError) as e:
        sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    assert e.value.status == B.ERR_TIMEOUT
    torch.cuda.synchronize()
    sol.test_set_wait()                                           # default bound, loads on
    assert sol.last_device_status() == B.OK                       # the time-out was reported once
    codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    rep_ls, st = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero)
    assert st == B.OK and sol.last_device_status() == B.OK
    H, Wn, res = _solve_oracle(spec)
    assert (codes.cpu().numpy() == res.ls.codes).mean() >= CODE_AGREEMENT
    with pytest.raises(B.AdmmqError):
        sol.test_set_wait(10)                                     # bounds below 1000 cycles are refused
    # the same for the one-plane products of large penalties (another instantiation of the kernel)
    sol.factor(rho=[1e7, 2e7, 4e7])
    sol.test_set_wait(2_000_000, hold_loads=True)
    with pytest.raises(B.AdmmqError) as e:
        sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    assert e.value.status == B.ERR_TIMEOUT
    torch.cuda.synchronize()
    sol.test_set_wait()
    c3, _, _, rep3 = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    assert sol.last_device_status() == B.OK and rep3.one_plane_iters >= 2
    ref3 = O.admm(H, Wn, spec.bits, spec.group_size, spec.symmetric, np.array([1e7, 2e7, 4e7]))
    assert (c3.cpu().numpy() == ref3.codes).mean() >= CODE_AGREEMENT


# ------------------------------------------------------------------ pair-swap refinement (Sec. 3.5, Eq. 11 in full)
@pytest.mark.parametrize("kw", [dict(d_in=512, d_out=96, n_tokens=4096, bits=3),
                                dict(d_in=264, d_out=70, n_tokens=3000, bits=2, group_size=0, symmetric=True)])
def test_pair_swap_parity(kw):
    spec = wl.small_case(**kw)
    g = _solve_gpu(spec)                                         # ADMM + single-entry local search on the GPU
    H, Wn, _ = _solve_oracle(spec)
    codes = g["codes_final"].clone()
    c0 = codes.cpu().numpy()
    delta, z0 = O.grid_fit(Wn, spec.bits, spec.group_size, spec.symmetric)
    rng = np.random.default_rng(9)
    pairs = rng.integers(0, spec.d_in, size=(5, 512, 2)).astype(np.int32)
    pairs[0, 0] = (7, 7)                                         # not a pair: ignored on both sides
    ref = O.pair_swap(H, Wn, c0, delta, z0, spec.bits, pairs)
    Wq = g["Wq_final"].clone()
    rep, st = g["sol"].pair_swap(g["W"], spec.bits, spec.group_size, codes, g["scale"], g["zero"],
                                 to_dev(pairs, torch.int32, DEV), Wq=Wq)
    assert st == B.OK and g["sol"].last_device_status() == B.OK
    cg = codes.cpu().numpy()
    e0 = O.objective(H, Wn, O.dequantize(c0, delta, z0))
    e_g = O.objective(H, Wn, O.dequantize(cg, delta, z0))
    e_o = O.objective(H, Wn, ref.Wq)
    assert e_g <= e0 * (1 + 1e-9)                                # never worse than the start
    assert abs(e_g - e_o) <= ERR_TOL * e_o
    assert abs(rep.err_after - e_g) <= ERR_TOL * e_g and abs(rep.err_before - e0) <= ERR_TOL * e0
    assert (cg == ref.codes).mean() >= CODE_AGREEMENT
    # only the rows of candidate pairs can have moved, by one level
    assert np.abs(cg.astype(int) - c0.astype(int)).max() <= 5
    moved_rows = set(np.nonzero((cg != c0).any(axis=0))[0])
    assert moved_rows <= set(pairs.reshape(-1).tolist())
    assert rep.iters_run == sum(1 for b in ref.chosen if b >= 0) or abs(e_g - e_o) <= 1e-6 * e_o
    assert np.allclose(Wq.cpu().numpy(), O.dequantize(cg, delta, z0), rtol=1e-6, atol=3e-8)
    # no rounds, no batch: a no-op
    c2 = codes.clone()
    rep2, _ = g["sol"].pair_swap(g["W"], spec.bits, spec.group_size, c2, g["scale"], g["zero"],
                                 torch.zeros(0, 0, 2, dtype=torch.int32, device=DEV))
    assert torch.equal(c2, codes) and rep2.moves == 0


# ------------------------------------------------------------------ grid refresh (Sec. 3.3 "Grid refresh", App. B)
@pytest.mark.parametrize("kw,attempts", [
    (dict(d_in=512, d_out=384, n_tokens=6144), list(range(1, 40))),          # g128, asym: first accepted attempt
    (dict(d_in=264, d_out=70, n_tokens=3000, bits=2, group_size=0, symmetric=True), [4]),
    (dict(d_in=256, d_out=64, n_tokens=2048, group_size=64), [0]),            # at t = 0 the refit sees W_hat: no change
    # a long schedule: an attempt inside the last iterations, which otherwise form no product and run in one pass
    (dict(d_in=256, d_out=96, n_tokens=2048, group_size=64, T=130, gamma=1.25), [3, 126]),
])
def test_grid_refresh_parity(kw, attempts):
    spec = wl.small_case(**kw)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    resid = torch.zeros(spec.T, 2, device=DEV)
    codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, resid=resid,
                                                 refresh_at=attempts)
    assert sol.last_device_status() == B.OK
    H = oracle_hessian(spec, DEV)
    Wn = np64(W)
    ref = O.admm(H, Wn, spec.bits, spec.group_size, spec.symmetric, np.array(spec.rho()), refresh_at=attempts)
    # The accepted attempt is a comparison of two sums over the whole matrix.  At t = 0 the target is W_hat
    # itself, both grids coincide and the two sums are equal up to rounding: either answer is right there.
    if attempts != [0]:
        assert rep.refreshed_iter == ref.refreshed_at
    assert np.allclose(scale.cpu().numpy(), ref.delta, rtol=2e-5, atol=0)
    assert np.allclose(zero.cpu().numpy(), ref.z0, rtol=2e-5, atol=1e-7)
    cg = codes.cpu().numpy()
    assert cg.max() <= (1 << spec.bits) - 1
    assert (cg == ref.codes).mean() >= CODE_AGREEMENT
    e_g = O.objective(H, Wn, O.dequantize(cg, ref.delta, ref.z0))
    e_o = O.objective(H, Wn, ref.Wq)
    assert abs(e_g - e_o) <= ERR_TOL * e_o
    assert abs(rep.err_before - e_g) <= 2 * ERR_TOL * e_g
    r = resid.cpu().numpy()
    assert np.abs(r[:, 0] - ref.r).max() <= 1e-3 * ref.r.max()
    if attempts == [0]:
        base = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)[0]
        assert (base == codes).float().mean().item() >= 0.9999
    # a refresh needs groups of at least two entries
    with pytest.raises(B.AdmmqError) as e:
        sol.quantize_layer(W, spec.bits, 1, spec.symmetric, refresh_at=[3])
    assert e.value.status == B.ERR_UNSUPPORTED


# ------------------------------------------------------------------ MSE search for the clipping ratio (Sec. 3.4, App. D)
@pytest.mark.parametrize("kw", [
    dict(d_in=256, d_out=96, n_tokens=2048, bits=3, group_size=64),
    dict(d_in=512, d_out=40, n_tokens=1536, bits=4, group_size=128, symmetric=True),
    dict(d_in=264, d_out=70, n_tokens=3000, bits=2, group_size=0),              # one group per channel, ragged n
    dict(d_in=384, d_out=33, n_tokens=1200, bits=3, group_size=384),           # group longer than the register path
])
def test_mse_clip_search_parity(kw):
    spec = wl.small_case(**kw)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, clip_points=100,
                                                 clip_min_ratio=0.8)
    assert sol.last_device_status() == B.OK
    Wn = np64(W)
    d_o, z_o = O.grid_fit_mse(Wn, spec.bits, spec.group_size, spec.symmetric, points=100, min_ratio=0.8)
    d_g, z_g = np64(scale), np64(zero)
    # The chosen candidate is an argmin over sums that can lie within rounding of each other: the grid must
    # agree for almost every group, and where it does not the GPU's choice must be as good as the optimum.
    same = np.isclose(d_g, d_o, rtol=1e-6, atol=0) & np.isclose(z_g, z_o, rtol=1e-6, atol=1e-12)
    assert same.mean() >= 0.98, same.mean()
    levels = (1 << spec.bits) - 1
    gs = spec.d_in if spec.group_size in (0, spec.d_in) else spec.group_size
    Wg = Wn.reshape(spec.d_out, spec.d_in // gs, gs)

    def mse(d, z):
        k = np.clip(np.rint((Wg - z[..., None]) / d[..., None]), 0, levels)
        return ((z[..., None] + d[..., None] * k - Wg) ** 2).sum(axis=2)

    e_g, e_o = mse(d_g, z_g), mse(d_o, z_o)
    assert (e_g <= e_o * (1 + 1e-4) + 1e-30).all()
    # every GPU grid is one of the candidates: ratio = Delta / Delta_minmax in [0.8, 1]
    d_mm, _ = O.grid_fit(Wn, spec.bits, spec.group_size, spec.symmetric)
    ratio = d_g / d_mm
    assert (ratio >= 0.8 - 1e-6).all() and (ratio <= 1 + 1e-6).all()
    assert (ratio < 0.999).mean() > 0.2                      # the search does clip on these weights
    # the ADMM run on that grid matches the oracle's run on the same grid
    H = oracle_hessian(spec, DEV)
    ref = O.admm(H, Wn, spec.bits, spec.group_size, spec.symmetric, np.array(spec.rho()), grid=(d_g, z_g))
    cg = codes.cpu().numpy()
    assert (cg == ref.codes).mean() >= CODE_AGREEMENT
    e_a = O.objective(H, Wn, O.dequantize(cg, d_g, z_g))
    assert abs(e_a - O.objective(H, Wn, ref.Wq)) <= ERR_TOL * e_a
    # one candidate is the min-max grid, bit for bit
    _, s1, z1, _ = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, clip_points=1)
    _, s0, z0, _ = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    assert torch.equal(s1, s0) and torch.equal(z1, z0)
    with pytest.raises(B.AdmmqError):
        sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, clip_points=100, clip_min_ratio=0.0)


def test_fused_and_row_pass_element_update_agree():
    """The element update of Eq. 8-10 inside the product's epilogue and in the row pass is the same arithmetic
    on the same accumulators: codes, grid and residual trace are identical."""
    spec = wl.small_case(d_in=520, d_out=200, n_tokens=2048, bits=3, group_size=0)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    out = []
    for fused in (False, True):
        resid = torch.zeros(spec.T, 2, device=DEV)
        # (both runs through the factorisation in every iteration: the fused variant has no series route)
        codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, resid=resid,
                                                     fused_epilogue=fused, wupdate_series=1)
        assert sol.last_device_status() == B.OK
        out.append((codes.clone(), scale.clone(), zero.clone(), resid.cpu().numpy(), rep.err_before))
    assert torch.equal(out[0][0], out[1][0])
    assert torch.equal(out[0][1], out[1][1]) and torch.equal(out[0][2], out[1][2])
    assert np.allclose(out[0][3], out[1][3], rtol=1e-5, atol=0)
    assert abs(out[0][4] - out[1][4]) <= 1e-12 * out[0][4]     # the error sum is accumulated atomically


@pytest.mark.parametrize("kw", [dict(d_in=256, d_out=640, n_tokens=4096, bits=4, group_size=128),
                                dict(d_in=264, d_out=400, n_tokens=3000, bits=3, group_size=0)])
def test_explicit_operator_route_against_oracle_and_two_product_route(kw):
    """Layers with more output than input channels form the n x n operator of the W-update once per iteration and
    apply it in one product.  Same operator, other rounding: both routes meet the oracle's bars, and a context
    too narrow for the explicit route refuses it."""
    spec = wl.small_case(**kw)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    H, Wn, res = _solve_oracle(spec)
    errs = []
    for route in (1, 2, 0):
        resid = torch.zeros(spec.T, 2, device=DEV)
        codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, resid=resid,
                                                     wupdate_route=route)
        assert sol.last_device_status() == B.OK
        assert (codes.cpu().numpy() == res.admm.codes).mean() >= CODE_AGREEMENT, route
        assert abs(rep.err_before - res.err_admm) <= ERR_TOL * res.err_admm
        assert np.allclose(resid.cpu().numpy()[:, 0], res.admm.r, rtol=2e-3, atol=1e-6 * res.admm.r.max())
        errs.append(rep.err_before)
    assert abs(errs[0] - errs[1]) <= ERR_TOL * errs[0]
    narrow = B.Solver(spec.d_in, spec.d_in, T_max=spec.T)           # d_out_max = d_in: no room for the operator
    narrow.hessian_reset()
    narrow.hessian_accumulate(wl.gen_x_chunk(spec, 0, DEV))
    narrow.factor(rho=spec.rho())
    with pytest.raises(B.AdmmqError) as e:
        narrow.quantize_layer(W[: spec.d_in].contiguous(), spec.bits, spec.group_size, spec.symmetric, wupdate_route=2)
    assert e.value.status == B.ERR_UNSUPPORTED


def test_one_plane_products_of_the_late_iterations():
    """Once the penalty is large the products carry a part of the W-update so small that one fp16 plane per
    operand resolves it below fp32, then so small that a truncated series replaces the route through the
    factorisation, and at the end none at all: the default run switches there, a run forced to two planes does
    not, a run without the series keeps the factorisation, and all give the oracle's codes."""
    spec = wl.small_case(d_in=520, d_out=264, n_tokens=4096, bits=4, group_size=0, T=130, gamma=1.25)
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    H, Wn, res = _solve_oracle(spec)
    c0, s0, z0, rep0 = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    c2, s2, z2, rep2 = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, product_planes=2)
    assert sol.last_device_status() == B.OK
    c1, s1, z1, rep1 = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric, wupdate_series=1)
    assert 10 <= rep0.one_plane_iters < spec.T and rep2.one_plane_iters == 0
    # by default those iterations are evaluated as the truncated series; wupdate_series = 1 keeps them on the
    # factorisation (one-plane products and the row solve)
    assert rep0.one_plane_iters - 1 <= rep0.series_iters + rep0.series0_iters <= rep0.one_plane_iters
    assert rep2.series_iters == 0 and rep2.series0_iters == 0 and rep1.series0_iters == 0
    assert rep0.series0_iters >= 5                          # the run ends with iterations that form no product
    assert rep0.series2_iters >= 5 and rep1.series2_iters == 0 and rep2.series2_iters == 0
    assert rep1.one_plane_iters == rep0.one_plane_iters and rep1.series_iters == 0
    assert (c0.cpu().numpy() == res.admm.codes).mean() >= CODE_AGREEMENT
    assert (c1.cpu().numpy() == res.admm.codes).mean() >= CODE_AGREEMENT
    assert (c2.cpu().numpy() == res.admm.codes).mean() >= CODE_AGREEMENT
    assert (c0 == c2).float().mean().item() >= 0.9995
    assert (c1 == c2).float().mean().item() >= 0.9995
    assert abs(rep0.err_before - res.err_admm) <= ERR_TOL * res.err_admm


def test_stacked_layers_share_one_factorisation():
    """Projections that read the same activations share H: stacking their weights into one call gives, channel
    by channel, exactly what separate calls on the same factorisation give (output channels are independent
    problems given H; Sec. 3.1)."""
    spec = wl.small_case(d_in=512, d_out=320, n_tokens=2048, bits=4, group_size=128)
    sizes = [192, 64, 64]                                   # a q / k / v split
    W = wl.gen_weight(spec, DEV)
    sol = B.Solver(spec.d_in, spec.d_out, T_max=spec.T)
    sol.hessian_reset()
    for c in range(spec.n_chunks):
        sol.hessian_accumulate(wl.gen_x_chunk(spec, c, DEV))
    sol.factor(rho=spec.rho())
    codes, scale, zero, rep = sol.quantize_layer(W, spec.bits, spec.group_size, spec.symmetric)
    rep_ls, _ = sol.local_search(W, spec.bits, spec.group_size, codes, scale, zero)
    r0, err_sum, err_ls_sum = 0, 0.0, 0.0
    for p_i in sizes:
        Wi = W[r0:r0 + p_i].contiguous()
        ci, si, zi, ri = sol.quantize_layer(Wi, spec.bits, spec.group_size, spec.symmetric)
        assert torch.equal(si, scale[r0:r0 + p_i]) and torch.equal(zi, zero[r0:r0 + p_i])
        ri_ls, _ = sol.local_search(Wi, spec.bits, spec.group_size, ci, si, zi)
        assert torch.equal(ci, codes[r0:r0 + p_i])
        err_sum += ri.err_before
        err_ls_sum += ri_ls.err_after
        r0 += p_i
    assert abs(err_sum - rep.err_before) <= 1e-9 * rep.err_before
    assert abs(err_ls_sum - rep_ls.err_after) <= 1e-9 * rep_ls.err_after
    assert sol.last_device_status() == B.OK
