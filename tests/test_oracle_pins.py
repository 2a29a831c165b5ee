"""Pins for the fp64 oracle: each check fixes a piece of oracle/admmq_oracle.py
against something other than itself -- hand-worked values (tests/golden), closed
forms, brute force on tiny inputs, library routines, and invariants the paper
proves.  All CPU, no GPU, a few seconds each.
"""
import itertools
import os

import numpy as np
import pytest
import scipy.linalg

from oracle import admmq_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = np.array([float(x) for x in v])
    return out


def _problem(n, p, N, seed, outliers=2, scale=20.0):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((N, n))
    X[:, rng.permutation(n)[:outliers]] *= scale
    W = 0.02 * rng.standard_normal((p, n))
    H = O.hessian_finalize(O.hessian_accumulate(None, X), N)
    return X, W, H


# ------------------------------------------------------------------ golden, hand-worked
def test_w_update_hand_worked_2x2():
    g = _read_kv("w_update_2x2.txt")
    H = g["H"].reshape(2, 2)
    lam, U = O.eig_factor(H)
    Wh = g["W_hat"][None, :]
    W = O.w_update(lam, U, Wh @ H, g["D"][None, :], g["V"][None, :], float(g["rho"][0]))
    assert np.allclose(W[0], g["W"], rtol=0, atol=1e-14)
    W2 = O.w_update_cholesky(H, Wh @ H, g["D"][None, :], g["V"][None, :], float(g["rho"][0]))
    assert np.allclose(W2[0], g["W"], rtol=0, atol=1e-14)


def test_projection_hand_worked():
    rows = [l.split() for l in open(os.path.join(GOLD, "projection_cases.txt"))
            if l.strip() and not l.startswith("#")]
    wt = np.array([[float(r[0]) for r in rows]])
    k, D = O.project(wt, np.full(len(rows), 2.0), np.array([[0.5]]), np.array([[-1.0]]), 2)
    assert k[0].tolist() == [int(r[1]) for r in rows]
    assert np.allclose(D[0], [float(r[2]) for r in rows], atol=1e-15)


def test_move_cost_hand_worked():
    g = _read_kv("move_cost_2x2.txt")
    H = g["H"].reshape(2, 2)
    # grid: Delta = 0.5, z0 = -1, 3 bits; W_q = [0.5, 0.0] (codes 3, 2); W_hat = W_q - eps
    delta, z0 = np.array([[0.5]]), np.array([[-1.0]])
    codes = np.array([[3, 2]], dtype=np.uint8)
    Wq = O.dequantize(codes, delta, z0)
    W_hat = Wq - g["eps"][None, :]
    assert abs(O.objective(H, W_hat, Wq) - g["loss"][0]) < 1e-15
    ls = O.local_search(H, W_hat, codes, delta, z0, bits=3, max_moves=1)
    # the best single move is the hand-worked one (entry 0, -Delta): costs of the 4 candidates are
    # (0,+): 2*.5*.75+.5 = 1.25 ; (0,-): -0.25 ; (1,+-): 0 +- 0 + .5 = 0.5
    assert ls.codes.tolist() == [[2, 2]]
    assert np.allclose(ls.g[0], g["g_new"], atol=1e-15)
    assert abs(O.objective(H, W_hat, ls.Wq) - (g["loss"][0] + g["change"][0])) < 1e-15


# ------------------------------------------------------------------ Hessian, damping, scaling
def test_rho_schedule_is_geometric_with_the_stated_ends():
    """Sec. 3.6: rho_t = rho_0 gamma^t.  Pinned on the two schedules the workloads use: the paper's default
    (rho_0 = 0.1, gamma = 1.1, T = 300: the last penalty is 0.1 * 1.1^299) and the 100-step schedule from 1e-2
    to 1e2 of the small configuration (gamma = 1e4^(1/99)), and on the product workloads.py hands the GPU."""
    from paper_2605_11222_b200 import workloads as wl
    r = O.rho_schedule(300, 0.1, 1.1)
    assert r[0] == 0.1 and len(r) == 300
    assert np.allclose(r[1:] / r[:-1], 1.1, rtol=1e-14)
    assert abs(r[-1] / (0.1 * 1.1 ** 299) - 1) < 1e-12 and 2.3e11 < r[-1] < 2.4e11
    g = 1e4 ** (1.0 / 99)
    r1 = O.rho_schedule(100, 1e-2, g)
    assert r1[0] == 1e-2 and abs(r1[-1] - 1e2) < 1e-9 and np.all(np.diff(r1) > 0)
    for spec in (wl.config1(), wl.config2()):
        assert np.allclose(np.array(spec.rho()), O.rho_schedule(spec.T, spec.rho0, spec.gamma), rtol=1e-13)


def test_hessian_chunked_equals_one_shot_and_entry_definition():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((300, 12))
    Hc = None
    for a in range(0, 300, 64):
        Hc = O.hessian_accumulate(Hc, X[a:a + 64])
    H1 = O.hessian_accumulate(None, X)
    assert np.allclose(Hc, H1, rtol=1e-13, atol=1e-12)
    # entry-by-entry definition H_ab = sum_t X_ta X_tb
    for a, b in [(0, 0), (3, 7), (11, 2)]:
        assert abs(H1[a, b] - sum(X[t, a] * X[t, b] for t in range(300))) < 1e-10


def test_damping_is_one_percent_of_mean_diagonal():
    rng = np.random.default_rng(2)
    X = rng.standard_normal((50, 6))
    Hr = O.hessian_accumulate(None, X)
    H = O.hessian_finalize(Hr, 50, 0.01)
    lam = 0.01 * np.mean(np.diag(Hr / 50))
    assert np.allclose(H - Hr / 50, lam * np.eye(6), atol=1e-15)
    Hl = O.hessian_finalize(Hr, 50, 0.01, literal_trace=True)
    assert np.allclose(Hl - Hr / 50, 6 * lam * np.eye(6), atol=1e-14)
    assert np.all(np.linalg.eigvalsh(H) > 0)


def test_preconditioning_unit_diagonal_and_objective_identity():
    _, W, H = _problem(16, 5, 200, 3)
    s, Ht, Ws = O.precondition(H, W)
    assert np.allclose(np.diag(Ht), 1.0, atol=1e-14)
    assert np.all(np.linalg.eigvalsh(Ht) > 0)
    # Eq. 3: the scaled objective equals the unscaled one for any candidate
    rng = np.random.default_rng(4)
    Wc = W + 0.01 * rng.standard_normal(W.shape)
    unscaled = O.objective(H, W, Wc)
    scaled = O.objective(Ht, Ws, Wc * s[None, :])
    assert abs(unscaled - scaled) <= 1e-12 * abs(unscaled)


# ------------------------------------------------------------------ grid and projection
@pytest.mark.parametrize("bits,gs,sym", [(2, 0, True), (3, 4, False), (4, 8, False), (3, 8, True)])
def test_grid_fit_brute_force(bits, gs, sym):
    rng = np.random.default_rng(5)
    W = rng.standard_normal((6, 16)) * 0.02
    W[2, 4:8] = 0.0125  # a constant group
    delta, z0 = O.grid_fit(W, bits, gs, sym)
    g = 16 if gs == 0 else gs
    L = (1 << bits) - 1
    for j in range(6):
        for q in range(16 // g):
            blk = W[j, q * g:(q + 1) * g]
            lo, hi = (-(np.abs(blk).max()), np.abs(blk).max()) if sym else (blk.min(), blk.max())
            if hi == lo:
                assert delta[j, q] == 1.0 and z0[j, q] == lo
                continue
            assert abs(delta[j, q] - (hi - lo) / L) < 1e-18 and z0[j, q] == lo
            # every weight inside the grid's range, RTN error at most Delta/2
            k, D = O.project(blk[None, :], np.ones(g), delta[j:j + 1, q:q + 1], z0[j:j + 1, q:q + 1], bits)
            assert np.all(np.abs(D[0] - blk) <= delta[j, q] / 2 * (1 + 1e-12))


def test_projection_is_nearest_grid_point_brute_force():
    rng = np.random.default_rng(6)
    p, n, bits, gs = 7, 24, 3, 8
    W = rng.standard_normal((p, n)) * 0.02
    delta, z0 = O.grid_fit(W, bits, gs, False)
    s = np.exp(rng.standard_normal(n))
    Wt = (W + 0.05 * rng.standard_normal((p, n))) * s[None, :]   # also exercises the clamp
    k, D = O.project(Wt, s, delta, z0, bits)
    for j in range(p):
        for i in range(n):
            levels = s[i] * (z0[j, i // gs] + delta[j, i // gs] * np.arange(1 << bits))
            kb = int(np.argmin(np.abs(levels - Wt[j, i])))
            assert kb == k[j, i] and abs(levels[kb] - D[j, i]) < 1e-15
    assert k.max() == (1 << bits) - 1 and k.min() == 0


# ------------------------------------------------------------------ W-update
def test_w_update_solves_linear_system_and_matches_cholesky():
    _, W, H = _problem(48, 9, 400, 7)
    s, Ht, Ws = O.precondition(H, W)
    lam, U = O.eig_factor(Ht)
    rng = np.random.default_rng(8)
    D = Ws + 0.01 * rng.standard_normal(Ws.shape)
    V = 0.01 * rng.standard_normal(Ws.shape)
    HW = Ws @ Ht
    for rho in (1e-2, 0.1, 3.0, 1e4):
        Wn = O.w_update(lam, U, HW, D, V, rho)
        rhs = HW + rho * D - V
        res = Wn @ (Ht + rho * np.eye(48)) - rhs          # transposed system
        assert np.linalg.norm(res) <= 1e-10 * np.linalg.norm(rhs)
        Wc = O.w_update_cholesky(Ht, HW, D, V, rho)
        assert np.linalg.norm(Wn - Wc) <= 1e-10 * np.linalg.norm(Wc)
        # and against an independent library solve of the untransposed system
        Wl = np.linalg.solve(Ht + rho * np.eye(48), rhs.T).T
        assert np.linalg.norm(Wn - Wl) <= 1e-10 * np.linalg.norm(Wl)


# ------------------------------------------------------------------ ADMM as a whole
def _rtn_codes(W, bits, gs, sym):
    delta, z0 = O.grid_fit(W, bits, gs, sym)
    n = W.shape[1]
    k, _ = O.project(W, np.ones(n), delta, z0, bits)
    return k


@pytest.mark.parametrize("precond", [True, False])
def test_first_iteration_is_rtn_for_any_hessian(precond):
    _, W, H = _problem(32, 11, 300, 9)
    a = O.admm(H, W, 3, 8, False, np.array([0.37]), precond=precond)
    assert np.array_equal(a.codes, _rtn_codes(W, 3, 8, False))


def test_key_inequality_feasibility_and_residual_trend():
    _, W, H = _problem(40, 13, 500, 10, outliers=3)
    bits, gs = 3, 8
    rho = O.rho_schedule(120, 0.1, 1.1)
    snaps = []
    a = O.admm(H, W, bits, gs, False, rho, probe=lambda t, st: snaps.append(
        (st["D"].copy(), st["V"].copy(), st["rho"], st["W"].copy())))
    delta, z0 = O.grid_fit(W, bits, gs, False)
    s = np.sqrt(np.diag(H))
    for t in range(1, len(snaps)):
        D_t, V_t, rt, W_t1 = snaps[t]
        tgt = W_t1 + V_t / rt
        _, D_t1 = O.project(tgt, s, delta, z0, bits)
        # Eq. 15: the new projection is at least as close to the target as the old D
        assert np.linalg.norm(D_t1 - tgt) <= np.linalg.norm(D_t - tgt) * (1 + 1e-12)
        # feasibility: D^(t), t >= 1, is on the grid with codes in range
        y = D_t / s[None, :]
        kk = (y - O._expand(z0, 40)) / O._expand(delta, 40)
        assert np.allclose(kk, np.rint(kk), atol=1e-8) and kk.min() > -1e-8 and kk.max() < 7 + 1e-8
    # Theorem 1: rho_t * residual stays bounded; codes freeze once rho is large
    tail = rho[60:] * np.maximum(a.r[60:], a.sres[60:])
    assert tail.max() <= 50 * max(tail[0], 1e-12) + 1e-9
    assert a.changed[-20:].sum() == 0
    assert a.r[-1] < 1e-3 * a.r[1]


def test_cholesky_route_gives_the_same_run():
    _, W, H = _problem(24, 6, 300, 11)
    rho = O.rho_schedule(30, 0.1, 1.3)
    a = O.admm(H, W, 3, 0, False, rho)
    b = O.admm(H, W, 3, 0, False, rho, use_cholesky=True)
    assert np.array_equal(a.codes, b.codes)
    assert np.allclose(a.r, b.r, rtol=1e-8, atol=1e-14)


def test_diagonal_hessian_gives_rtn():
    rng = np.random.default_rng(12)
    n, p, bits = 24, 9, 3
    W = 0.02 * rng.standard_normal((p, n))
    H = np.diag(np.exp(rng.standard_normal(n)))
    rtn = _rtn_codes(W, bits, 0, False)
    # (a) ADMM alone with rho_t >= 1 for every t
    a = O.admm(H, W, bits, 0, False, O.rho_schedule(40, 1.0, 1.2))
    assert np.array_equal(a.codes, rtn)
    # (b) any schedule followed by local search run to convergence
    res = O.quantize_layer(H, W, bits, 0, False, O.rho_schedule(60, 0.01, 1.2))
    assert np.array_equal(res.ls.codes, rtn)
    # (c) a single iteration
    assert np.array_equal(O.admm(H, W, bits, 0, False, np.array([0.05])).codes, rtn)


def test_fine_grid_limit_stays_next_to_dense_weights():
    # b = 8 on a per-channel grid: the constraint is nearly inactive, so ADMM on the strongly
    # convex quadratic must end within two grid steps of W_hat (the unconstrained minimiser)
    # in every entry -- a dropped term or wrong sign in the W- or V-update drifts far away.
    _, W, H = _problem(20, 5, 200, 13)
    a = O.admm(H, W, 8, 0, False, O.rho_schedule(150, 0.1, 1.1))
    assert np.all(np.abs(a.Wq - W) <= 2.0 * a.delta)
    # and with the grid made of W_hat's own values (caller grid, Delta -> levels hit W_hat exactly)
    # the fixed point is W_hat itself: codes of RTN, zero error
    delta, z0 = O.grid_fit(W, 8, 0, False)
    Wg = O.dequantize(_rtn_codes(W, 8, 0, False), delta, z0)           # weights already on the grid
    b = O.admm(H, Wg, 8, 0, False, O.rho_schedule(60, 0.1, 1.2), grid=(delta, z0))
    assert np.allclose(b.Wq, Wg, atol=1e-15) and b.r[-1] < 1e-9


def test_admm_beats_rtn_on_outlier_problem():
    _, W, H = _problem(64, 32, 2000, 14, outliers=3)
    res = O.quantize_layer(H, W, 3, 0, False, O.rho_schedule(150, 0.1, 1.1))
    rtn = O.dequantize(_rtn_codes(W, 3, 0, False), *O.grid_fit(W, 3, 0, False))
    e_rtn = O.objective(H, W, rtn)
    assert res.err_admm < e_rtn
    assert res.err_final <= res.err_admm


# ------------------------------------------------------------------ local search
def test_local_search_invariants():
    _, W, H = _problem(32, 10, 300, 15)
    delta, z0 = O.grid_fit(W, 3, 8, False)
    codes = _rtn_codes(W, 3, 8, False)
    e0 = O.objective(H, W, O.dequantize(codes, delta, z0))
    prev = e0
    cur = codes
    total = 0
    for _ in range(400):                      # one move at a time: strictly decreasing objective
        ls = O.local_search(H, W, cur, delta, z0, 3, max_moves=1)
        if ls.moves.sum() == 0:
            break
        e = O.objective(H, W, ls.Wq)
        assert e < prev
        # each column's decrease equals the closed-form cost of its move (checked in aggregate)
        prev, cur = e, ls.codes
        total += int(ls.moves.sum())
    full = O.local_search(H, W, codes, delta, z0, 3)
    assert np.array_equal(full.codes, cur) and int(full.moves.sum()) == total
    # maintained gradient equals the recomputed one
    assert np.allclose(full.g, (full.Wq - W) @ H, rtol=1e-10, atol=1e-12)
    # identity E = sum_j eps_j . g_j
    assert abs(np.sum((full.Wq - W) * full.g) - O.objective(H, W, full.Wq)) < 1e-12 * e0
    assert np.array_equal(full.Wq, O.dequantize(full.codes, delta, z0)) or \
        np.allclose(full.Wq, O.dequantize(full.codes, delta, z0), atol=1e-15)


def test_local_search_closed_form_cost_vs_recomputed_loss():
    _, W, H = _problem(12, 4, 100, 16)
    delta, z0 = O.grid_fit(W, 2, 0, False)
    codes = _rtn_codes(W, 2, 0, False)
    Wq = O.dequantize(codes, delta, z0)
    g = (Wq - W) @ H
    for j in range(4):
        e0 = (Wq[j] - W[j]) @ H @ (Wq[j] - W[j])
        for i in range(12):
            for sg in (+1, -1):
                d = sg * delta[j, 0]
                w2 = Wq[j].copy()
                w2[i] += d
                e1 = (w2 - W[j]) @ H @ (w2 - W[j])
                assert abs((e1 - e0) - (2 * d * g[j, i] + d * d * H[i, i])) < 1e-12 * max(e0, 1e-30) + 1e-18


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_local_search_brute_force_tiny(seed):
    """d_in = 8, 2 bits: enumerate all 4^8 assignments per column."""
    n, p, bits = 8, 3, 2
    _, W, H = _problem(n, p, 64, 100 + seed, outliers=1, scale=5.0)
    res = O.quantize_layer(H, W, bits, 0, False, O.rho_schedule(40, 0.05, 1.3))
    delta, z0 = res.admm.delta, res.admm.z0
    all_codes = np.array(list(itertools.product(range(4), repeat=n)))       # [65536, 8]
    tau = 1e-6
    for j in range(p):
        cand = z0[j, 0] + delta[j, 0] * all_codes                            # [65536, 8]
        E = cand - W[j][None, :]
        loss = np.einsum("ci,ik,ck->c", E, H, E)
        mine = res.ls.codes[j].astype(int)
        idx = int(np.dot(mine, 4 ** np.arange(n - 1, -1, -1)))
        assert np.array_equal(all_codes[idx], mine)
        my_loss = loss[idx]
        assert my_loss >= loss.min() - 1e-15
        # 1-move local optimum: no neighbour (one code +-1) improves by more than the threshold
        for i in range(n):
            for sg in (+1, -1):
                nb = mine.copy()
                nb[i] += sg
                if nb[i] < 0 or nb[i] > 3:
                    continue
                nidx = int(np.dot(nb, 4 ** np.arange(n - 1, -1, -1)))
                assert loss[nidx] >= my_loss - tau * H[i, i] * delta[j, 0] ** 2 - 1e-15
        # local search never made the column worse than the ADMM point
        aidx = int(np.dot(res.admm.codes[j].astype(int), 4 ** np.arange(n - 1, -1, -1)))
        assert my_loss <= loss[aidx] + 1e-15


def test_local_search_respects_move_cap_and_bounds():
    _, W, H = _problem(16, 6, 100, 17)
    delta, z0 = O.grid_fit(W, 2, 0, False)
    rng = np.random.default_rng(18)
    codes = rng.integers(0, 4, size=(6, 16)).astype(np.uint8)      # a poor start: many moves
    ls = O.local_search(H, W, codes, delta, z0, 2, max_moves=3)
    assert ls.moves.max() <= 3 and ls.capped.any()
    full = O.local_search(H, W, codes, delta, z0, 2)
    assert full.codes.max() <= 3 and not full.capped.any()
    assert O.objective(H, W, full.Wq) < O.objective(H, W, O.dequantize(codes, delta, z0))


# ------------------------------------------------------------------ pair-swap local search (Sec. 3.5, Eq. 11 in full)
def _pair_case(seed, n=10, p=6, bits=2):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((40, n))
    X[:, 1] = 0.9 * X[:, 0] + 0.1 * X[:, 1]              # correlated channels: cross terms matter
    H = O.hessian_finalize(X.T @ X, 40)
    W = 0.02 * rng.standard_normal((p, n))
    delta, z0 = O.grid_fit(W, bits, 0, False)
    codes = O.project(W, np.ones(n), delta, z0, bits)[0]
    return H, W, delta, z0, codes


def test_pair_cost_closed_form_equals_recomputed_loss():
    """Eq. 11: the closed-form change of eps^T H eps for every sign combination."""
    H, W, delta, z0, codes = _pair_case(3)
    Wq = O.dequantize(codes, delta, z0)
    g = (Wq - W) @ H
    j, i1, i2 = 2, 0, 1
    d = delta[j, 0]
    c = O.pair_move_costs(g[j, i1], g[j, i2], H[i1, i1], H[i2, i2], H[i1, i2], d, d)
    e0 = Wq[j] - W[j]
    for q, (a, b) in enumerate(O.PAIR_SIGNS):
        e1 = e0.copy()
        e1[i1] += a * d
        e1[i2] += b * d
        assert abs((e1 @ H @ e1 - e0 @ H @ e0) - c[q]) <= 1e-12 * abs(e0 @ H @ e0)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_pair_swap_brute_force_choice_and_invariants(seed):
    """One round over ALL row pairs: the applied pair and every column's sign combination are the best ones
    by direct evaluation of the loss; codes stay in range; the maintained gradient stays exact."""
    bits = 2
    H, W, delta, z0, codes0 = _pair_case(seed, bits=bits)
    p, n = codes0.shape
    codes = O.local_search(H, W, codes0, delta, z0, bits).codes          # start from a 1-move optimum
    pairs = np.array([[(a, b) for a in range(n) for b in range(a + 1, n)]])
    res = O.pair_swap(H, W, codes, delta, z0, bits, pairs)
    # brute force: total improvement of every pair, every column choosing freely among the 4 combos or none
    Wq = O.dequantize(codes, delta, z0)
    base = np.einsum("jn,nm,jm->j", Wq - W, H, Wq - W)
    best_total, best_pair = 0.0, -1
    for b, (i1, i2) in enumerate(pairs[0]):
        tot = 0.0
        for j in range(p):
            best = 0.0
            for a, s2 in O.PAIR_SIGNS:
                k1, k2 = codes[j, i1] + a, codes[j, i2] + s2
                if 0 <= k1 <= 3 and 0 <= k2 <= 3:
                    e = Wq[j] - W[j]
                    e = e.copy()
                    e[i1] += a * delta[j, 0]
                    e[i2] += s2 * delta[j, 0]
                    best = min(best, e @ H @ e - base[j])
            tot += best
        if tot < best_total - 1e-15:
            best_total, best_pair = tot, b
    assert res.chosen[0] == best_pair
    if best_pair >= 0:
        assert abs(res.totals[0] - best_total) <= 1e-9 * abs(best_total)
        assert abs((O.objective(H, W, res.Wq) - base.sum()) - best_total) <= 1e-9 * abs(base.sum())
        i1, i2 = pairs[0][best_pair]
        changed = np.nonzero((res.codes != codes).any(axis=1))[0]
        assert res.moves == changed.size
        assert set(np.nonzero((res.codes != codes).any(axis=0))[0]) <= {i1, i2}
    assert res.codes.max() <= 3
    assert np.allclose(res.g, (res.Wq - W) @ H, rtol=0, atol=1e-12 * np.abs(res.g).max())
    assert np.allclose(res.Wq, O.dequantize(res.codes, delta, z0), rtol=0, atol=1e-15)


def test_pair_swap_monotone_and_diagonal_hessian_declines():
    bits = 3
    H, W, delta, z0, codes0 = _pair_case(5, n=16, p=12, bits=bits)
    codes = O.local_search(H, W, codes0, delta, z0, bits).codes
    rng = np.random.default_rng(1)
    pairs = rng.integers(0, 16, size=(5, 40, 2))
    res = O.pair_swap(H, W, codes, delta, z0, bits, pairs)
    errs = [O.objective(H, W, O.dequantize(codes, delta, z0))]
    c = codes
    for r in range(5):                                            # round by round: never increases
        c = O.pair_swap(H, W, c, delta, z0, bits, pairs[r:r + 1]).codes
        errs.append(O.objective(H, W, O.dequantize(c, delta, z0)))
    assert all(b <= a * (1 + 1e-12) for a, b in zip(errs, errs[1:]))
    assert np.array_equal(c, res.codes)
    assert all(t <= 0 for t in res.totals)
    # separable problem: the 1-move optimum is the nearest grid point and no pair move can improve it
    Hd = np.diag(np.diag(H))
    cd = O.local_search(Hd, W, codes0, delta, z0, bits).codes
    rd = O.pair_swap(Hd, W, cd, delta, z0, bits, pairs)
    assert rd.moves == 0 and rd.chosen == [-1] * 5 and np.array_equal(rd.codes, cd)


# ------------------------------------------------------------------ grid refresh (Sec. 3.3 "Grid refresh", App. B)
def _refresh_case(seed=4, n=48, p=10, bits=3, gs=16):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((200, n))
    X[:, :3] *= 8.0
    H = O.hessian_finalize(X.T @ X, 200)
    W = 0.02 * rng.standard_normal((p, n))
    rho = O.rho_schedule(40, 0.05, 1.25)
    return H, W, bits, gs, rho


def test_grid_refresh_at_first_iteration_changes_nothing():
    """W^1 = W_hat and V^0 = 0, so the refit sees the dense weights: same grid, accepted with equality."""
    H, W, bits, gs, rho = _refresh_case()
    a = O.admm(H, W, bits, gs, False, rho)
    b = O.admm(H, W, bits, gs, False, rho, refresh_at=[0])
    assert b.refreshed_at == 0
    assert np.allclose(a.delta, b.delta, rtol=1e-12) and np.allclose(a.z0, b.z0, rtol=1e-12, atol=1e-18)
    assert np.array_equal(a.codes, b.codes)


def test_grid_refresh_acceptance_dual_consistency_and_single_acceptance():
    H, W, bits, gs, rho = _refresh_case()
    snaps = {}
    O.admm(H, W, bits, gs, False, rho, probe=lambda t, st: snaps.setdefault(t, {k: (v.copy() if hasattr(v, "copy") else v) for k, v in st.items()}))
    res = O.admm(H, W, bits, gs, False, rho, refresh_at=range(3, 40))
    t = res.refreshed_at
    assert t >= 3                                                   # some attempt is accepted on this problem
    # up to the accepted attempt the run is the fixed-grid run: rebuild that iteration by hand
    st = snaps[t]
    s, Ht, Ws = O.precondition(H, W)
    Wt = st["W"] + st["V"] / st["rho"]
    d_old, z_old = O.grid_fit(W, bits, gs, False)
    k_old, D_old = O.project(Wt, s, d_old, z_old, bits)
    k_new, D_new = O.project(Wt, s, res.delta, res.z0, bits)
    assert np.sum((D_new - Wt) ** 2) <= np.sum((D_old - Wt) ** 2)   # the acceptance criterion held
    y = Wt / s[None, :]
    d_fit, z_fit = O.grid_fit(y, bits, gs, False)
    assert np.allclose(d_fit, res.delta, rtol=1e-12) and np.allclose(z_fit, res.z0, rtol=1e-12, atol=1e-18)
    lo = z_fit.repeat(gs, axis=1)
    hi = lo + 7 * d_fit.repeat(gs, axis=1)
    assert (y >= lo - 1e-15).all() and (y <= hi + 1e-12).all()      # the new grid spans the target
    # dual consistency: Eq. 9 with D_old, then V += rho (D_old - D_new), equals the update with D_new
    V_two_step = st["V"] + st["rho"] * (st["W"] - D_old) + st["rho"] * (D_old - D_new)
    snaps2 = {}
    O.admm(H, W, bits, gs, False, rho, refresh_at=[t],
           probe=lambda tt, s2: snaps2.setdefault(tt, {k: (v.copy() if hasattr(v, "copy") else v) for k, v in s2.items()}))
    assert np.allclose(snaps2[t + 1]["V"], V_two_step, rtol=0, atol=1e-12 * np.abs(V_two_step).max())
    assert np.array_equal(snaps2[t + 1]["codes"], k_new)
    # feasibility on the final grid, exactly one accepted refresh
    assert res.codes.max() <= 7
    assert np.allclose(res.Wq, O.dequantize(res.codes, res.delta, res.z0))
    again = O.admm(H, W, bits, gs, False, rho, refresh_at=[t])
    assert np.array_equal(again.codes, res.codes) and again.refreshed_at == t


@pytest.mark.parametrize("seed", [4, 5])
def test_grid_refresh_first_accepted_attempt_and_declined_ones(seed):
    """Attempts at every iteration from 1 on: each attempt before the accepted one fails Eq. (refresh
    criterion) when rebuilt by hand from the fixed-grid run, the accepted one passes it; without attempts the
    run is the fixed-grid run."""
    H, W, bits, gs, rho = _refresh_case(seed=seed)
    snaps = {}
    base = O.admm(H, W, bits, gs, False, rho,
                  probe=lambda t, st: snaps.setdefault(t, {k: (v.copy() if hasattr(v, "copy") else v) for k, v in st.items()}))
    res = O.admm(H, W, bits, gs, False, rho, refresh_at=range(1, 40))
    t_acc = res.refreshed_at
    assert t_acc > 1                                                # these seeds decline at least one attempt
    s, _, _ = O.precondition(H, W)
    d_old, z_old = O.grid_fit(W, bits, gs, False)
    for t in range(1, t_acc + 1):
        st = snaps[t]
        Wt = st["W"] + st["V"] / st["rho"]
        _, D_old = O.project(Wt, s, d_old, z_old, bits)
        d2, z2 = O.grid_fit(Wt / s[None, :], bits, gs, False)
        _, D2 = O.project(Wt, s, d2, z2, bits)
        accepted = np.sum((D2 - Wt) ** 2) <= np.sum((D_old - Wt) ** 2)
        assert accepted == (t == t_acc), t
    never = O.admm(H, W, bits, gs, False, rho, refresh_at=[])
    assert np.array_equal(never.codes, base.codes) and never.refreshed_at == -1


# ------------------------------------------------------------------ MSE search for the clipping ratio (Sec. 3.4, App. D)
def test_mse_clip_search_brute_force_and_limits():
    rng = np.random.default_rng(21)
    p, n, gs, bits = 6, 64, 16, 3
    W = 0.02 * rng.standard_normal((p, n))
    W[0, 3] = 0.2                                               # an outlier: clipping it pays
    delta, z0 = O.grid_fit_mse(W, bits, gs, False)
    d_mm, z_mm = O.grid_fit(W, bits, gs, False)
    levels = 7
    ratios = [1.0 - 0.2 * i / 99 for i in range(100)]

    def group_err(w, lo, dl):
        k = np.clip(np.rint((w - lo) / dl), 0, levels)
        return float(((lo + dl * k - w) ** 2).sum())

    for j in range(p):
        for g in range(n // gs):
            w = W[j, g * gs:(g + 1) * gs]
            errs = [group_err(w, r * w.min(), (r * w.max() - r * w.min()) / levels) for r in ratios]
            i_best = int(np.argmin(errs))                        # first minimum = largest ratio
            r = ratios[i_best]
            assert abs(z0[j, g] - r * w.min()) <= 1e-15
            assert abs(delta[j, g] - r * (w.max() - w.min()) / levels) <= 1e-15
            assert errs[i_best] <= group_err(w, z_mm[j, g], d_mm[j, g]) + 1e-18   # never worse than min-max
    assert delta[0, 0] < d_mm[0, 0]                              # the outlier group is clipped
    # one candidate = the min-max grid; a constant group keeps Delta = 1
    d1, z1 = O.grid_fit_mse(W, bits, gs, False, points=1)
    assert np.array_equal(d1, d_mm) and np.array_equal(z1, z_mm)
    Wc = W.copy()
    Wc[1, :gs] = 0.5
    dc, zc = O.grid_fit_mse(Wc, bits, gs, False)
    assert dc[1, 0] == 1.0
    # symmetric: the grid stays symmetric around zero
    ds, zs = O.grid_fit_mse(W, bits, gs, True)
    assert np.allclose(zs, -0.5 * levels * ds)
