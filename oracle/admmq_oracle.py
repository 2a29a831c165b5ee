"""Plain fp64 CPU oracle for the ADMM-Q layer-wise quantization solver.

TEST INFRASTRUCTURE ONLY -- the product path never imports this module, and
this module imports nothing from the CUDA package.  Every function follows
one passage of the paper, named in its docstring, in the paper's order and
notation (n = input channels, p = output channels, N = calibration rows).
Arithmetic is numpy float64 throughout; LAPACK routines (eigh, Cholesky
solve) are used only as whole steps.

Memory layout: every n-by-p matrix of the paper (W-hat, W, D, V, W_q) is held
TRANSPOSED as an array of shape [p, n] (one row per output channel, input
channels contiguous), which is the layout of a linear layer's weight.  The
mathematics is unchanged: row j of the array is column j of the paper's
matrix.

Pin status (what fixes each function independently of itself is in
tests/test_oracle_pins.py):
  hessian / damping / preconditioning ... closed forms and identities
  grid_fit, project .................... brute force over the 2^b levels
  w_update ............................. linear-system residual, Cholesky route,
                                         hand-worked 2x2 example (tests/golden)
  admm ................................. T=1 gives RTN for any H; key inequality
                                         of the convergence proof; diagonal-H
                                         cases; large-b limit
  local_search ......................... brute-force enumeration on tiny columns
  Whole-pipeline VALUES: parity unpinned (the paper prints no numbers for any
  layer); pinned only through the invariants above.
"""
from __future__ import annotations

import dataclasses
from typing import Sequence, Callable, Optional

import numpy as np
import scipy.linalg

F64 = np.float64


# --------------------------------------------------------------------------
# Step 1-2: Hessian (Sec. 3.1, text after Eq. 1) and damping (App. D)
# --------------------------------------------------------------------------
def hessian_accumulate(H_raw: Optional[np.ndarray], X_chunk: np.ndarray) -> np.ndarray:
    """H_raw += X_c^T X_c for one chunk of calibration rows (Sec. 3.1: H = X^T X)."""
    Xc = np.asarray(X_chunk, dtype=F64)
    G = Xc.T @ Xc
    return G if H_raw is None else H_raw + G


def hessian_finalize(H_raw: np.ndarray, n_tokens: int, damp_frac: float = 0.01,
                     literal_trace: bool = False) -> np.ndarray:
    """H = H_raw / N + lambda I  (Eq. 1's lambda is the damping of App. D).

    Reading: lambda = damp_frac * mean(diag(H_raw / N)).  App. D prints
    0.01 * Tr(X^T X); `literal_trace=True` gives that literal form.
    """
    H = np.asarray(H_raw, dtype=F64) / float(n_tokens)
    n = H.shape[0]
    tr = float(np.trace(H))
    lam = damp_frac * (tr if literal_trace else tr / n)
    return H + lam * np.eye(n)


# --------------------------------------------------------------------------
# Step 3: diagonal scaling (Sec. 3.2, Eq. 3; Algorithm 1 lines 1-2)
# --------------------------------------------------------------------------
def precondition(H: np.ndarray, W_hat: np.ndarray, enable: bool = True):
    """Sigma = Diag(H)^(-1/2).  Returns (s, H_tilde, W_hat_scaled) with
    s_i = sqrt(H_ii) = 1/Sigma_ii, H_tilde = Sigma H Sigma, and
    W_hat_scaled = Sigma^{-1} W_hat  (array [p, n]: column i times s_i)."""
    n = H.shape[0]
    if enable:
        s = np.sqrt(np.diag(H).astype(F64))
    else:
        s = np.ones(n, dtype=F64)
    Ht = H / s[:, None] / s[None, :]
    Ws = np.asarray(W_hat, dtype=F64) * s[None, :]
    return s, Ht, Ws


# --------------------------------------------------------------------------
# Step 4: grid (Sec. 3.5 "Setup": levels z + k*Delta, 0 <= k <= 2^b - 1;
#          Sec. 3.4 "Clipping": Delta = (max - min) / (2^b - 1))
# --------------------------------------------------------------------------
def grid_fit(W_hat: np.ndarray, bits: int, group_size: int, symmetric: bool):
    """Min-max grid on the UNSCALED weights, per (output channel j, group of
    `group_size` consecutive input channels).  Returns (Delta, z0), each [p, n/gs].

    asymmetric: lo = min, hi = max;  symmetric: hi = max|w|, lo = -hi.
    Delta = (hi - lo) / (2^b - 1), z0 = lo; a constant group gets Delta = 1.
    """
    W = np.asarray(W_hat, dtype=F64)
    p, n = W.shape
    gs = n if group_size in (0, n) else group_size
    assert n % gs == 0
    Wg = W.reshape(p, n // gs, gs)
    if symmetric:
        hi = np.abs(Wg).max(axis=2)
        lo = -hi
    else:
        hi = Wg.max(axis=2)
        lo = Wg.min(axis=2)
    levels = (1 << bits) - 1
    delta = (hi - lo) / levels
    delta = np.where(hi - lo == 0.0, 1.0, delta)
    return delta, lo.copy()


def grid_fit_mse(W_hat: np.ndarray, bits: int, group_size: int, symmetric: bool, points: int = 100,
                 min_ratio: float = 0.8):
    """MSE search for the clipping ratio (Sec. 3.4 "Clipping Heuristics"; App. D: 100 grid points, maximum
    shrink ratio 0.8).  Per (output channel, group): candidates r_i = 1 - (1 - min_ratio) i / (points - 1),
    i = 0 .. points-1; the min-max range is shrunk to [r lo, r hi] (symmetric: +-r max|w|), Delta and z0
    follow as in grid_fit, the group is rounded to that grid with clamping, and the candidate with the
    smallest sum of squared rounding errors is kept (the largest ratio on ties).
    Readings: the ratio scales both ends of the range towards zero; the candidates run from 1.0 down to
    min_ratio inclusive; the error is the plain squared error of the unscaled weights."""
    W = np.asarray(W_hat, dtype=F64)
    p, n = W.shape
    gs = n if group_size in (0, n) else group_size
    Wg = W.reshape(p, n // gs, gs)
    if symmetric:
        hi0 = np.abs(Wg).max(axis=2)
        lo0 = -hi0
    else:
        hi0 = Wg.max(axis=2)
        lo0 = Wg.min(axis=2)
    levels = (1 << bits) - 1
    best_err = np.full(hi0.shape, np.inf)
    best_delta = np.ones(hi0.shape)
    best_z0 = lo0.copy()
    for i in range(points):
        r = 1.0 - (1.0 - min_ratio) * i / max(points - 1, 1)
        lo, hi = r * lo0, r * hi0
        delta = np.where(hi - lo == 0.0, 1.0, (hi - lo) / levels)
        k = np.clip(np.rint((Wg - lo[..., None]) / delta[..., None]), 0, levels)
        err = ((lo[..., None] + delta[..., None] * k - Wg) ** 2).sum(axis=2)
        take = err < best_err
        best_err = np.where(take, err, best_err)
        best_delta = np.where(take, delta, best_delta)
        best_z0 = np.where(take, lo, best_z0)
    return best_delta, best_z0


def _expand(g: np.ndarray, n: int) -> np.ndarray:
    """[p, n/gs] per-group values -> [p, n]."""
    return np.repeat(g, n // g.shape[1], axis=1)


def project(W_tilde: np.ndarray, s: np.ndarray, delta: np.ndarray, z0: np.ndarray, bits: int):
    """D-update, Eq. 8 / Eq. 10 (Algorithm 1 line 7): nearest grid point of
    Sigma*W_tilde, returned in scaled coordinates.

    y = W_tilde / s (unscaled coordinates), k = clamp(rint((y - z0)/Delta), 0, 2^b-1)
    with round-half-to-even, D = s * (z0 + Delta * k).  Returns (k uint8, D)."""
    p, n = W_tilde.shape
    dl = _expand(delta, n)
    zz = _expand(z0, n)
    y = W_tilde / s[None, :]
    k = np.rint((y - zz) / dl)
    k = np.clip(k, 0, (1 << bits) - 1)
    D = s[None, :] * (zz + dl * k)
    return k.astype(np.uint8), D


def dequantize(codes: np.ndarray, delta: np.ndarray, z0: np.ndarray) -> np.ndarray:
    """W_q = z0 + Delta * k in unscaled coordinates (= Sigma D, Algorithm 1 line 11)."""
    p, n = codes.shape
    return _expand(z0, n) + _expand(delta, n) * codes.astype(F64)


# --------------------------------------------------------------------------
# Step 5-6: factorisation and W-update (Eq. 7; "Efficient W-update"; Alg. 1 l.3, l.6)
# --------------------------------------------------------------------------
def eig_factor(Ht: np.ndarray):
    """H_tilde = U Lambda U^T  (Algorithm 1 line 3)."""
    lam, U = scipy.linalg.eigh(Ht)
    return lam, U


def w_update(lam: np.ndarray, U: np.ndarray, HW: np.ndarray, D: np.ndarray, V: np.ndarray,
             rho: float) -> np.ndarray:
    """Eq. 7 in the eigen form of Algorithm 1 line 6:
    W = U (Lambda + rho I)^{-1} U^T (H W_hat + rho D - V).
    Arrays are [p, n] (transposed), so the products act from the right."""
    rhs = HW + rho * D - V
    return ((rhs @ U) / (lam + rho)[None, :]) @ U.T


def w_update_cholesky(Ht: np.ndarray, HW: np.ndarray, D: np.ndarray, V: np.ndarray,
                      rho: float) -> np.ndarray:
    """Eq. 7 solved directly: (H + rho I) W = H W_hat + rho D - V by Cholesky."""
    n = Ht.shape[0]
    c = scipy.linalg.cho_factor(Ht + rho * np.eye(n), lower=True)
    rhs = HW + rho * D - V
    return scipy.linalg.cho_solve(c, rhs.T).T


def rho_schedule(T: int, rho0: float, gamma: float) -> np.ndarray:
    """rho_t = rho0 * gamma^t (Sec. 3.6, text after Theorem 1)."""
    return rho0 * gamma ** np.arange(T, dtype=F64)


@dataclasses.dataclass
class AdmmResult:
    codes: np.ndarray        # [p, n] uint8, codes of D^(T)
    delta: np.ndarray        # [p, n/gs]
    z0: np.ndarray           # [p, n/gs]
    Wq: np.ndarray           # [p, n] unscaled quantized weights (Alg. 1 line 11)
    r: np.ndarray            # [T]  ||W^(t+1) - D^(t+1)||_F
    sres: np.ndarray         # [T]  ||D^(t+1) - D^(t)||_F
    changed: np.ndarray      # [T]  number of codes that changed (t >= 1)
    s: np.ndarray            # [n]  sqrt(diag H)
    V: np.ndarray            # [p, n] final dual
    W: np.ndarray            # [p, n] final continuous iterate (scaled)
    refreshed_at: int = -1   # iteration of the accepted grid refresh, -1: none


def admm(H: np.ndarray, W_hat: np.ndarray, bits: int, group_size: int, symmetric: bool,
         rho: np.ndarray, precond: bool = True, use_cholesky: bool = False,
         grid: Optional[tuple] = None,
         probe: Optional[Callable[[int, dict], None]] = None,
         refresh_at: Sequence[int] = ()) -> AdmmResult:
    """Algorithm 1 lines 1-11.

    H is the damped, unscaled Hessian; W_hat is [p, n].  `rho` is the array of
    penalties, one per iteration.  `probe(t, state)` is called each iteration
    with the state BEFORE the W-update (D, V, rho) and the W it produces.

    Grid refresh (Sec. 3.3 "Grid refresh", App. B): at the iterations listed in `refresh_at`, until one
    attempt is accepted, the grid (Delta, z0) is refitted by the initial fitting routine on the unscaled
    projection target Sigma W~ = (W + V/rho) / s, the same target is projected again, and the new grid is
    kept iff || D_new - W~ ||_F^2 <= || D_old - W~ ||_F^2 (whole matrix, scaled coordinates).  The dual
    update then uses D_new, which is the paper's V <- V + rho (D_old - D_new) applied after Eq. 9.
    Readings: when the refresh is attempted is the caller's choice; the fit uses the projected point W~
    (the paper says "the current continuous weights"); at most one refresh is accepted.
    """
    W_hat = np.asarray(W_hat, dtype=F64)
    p, n = W_hat.shape
    s, Ht, Ws = precondition(H, W_hat, precond)               # lines 1-2
    delta, z0 = grid if grid is not None else grid_fit(W_hat, bits, group_size, symmetric)
    if not use_cholesky:
        lam, U = eig_factor(Ht)                                # line 3
    HW = Ws @ Ht                                               # (H W_hat)^T, H symmetric
    D = Ws.copy()                                              # line 4: D^0 = W_hat
    V = np.zeros_like(Ws)                                      #         V^0 = 0
    T = len(rho)
    r = np.zeros(T)
    sres = np.zeros(T)
    changed = np.zeros(T, dtype=np.int64)
    codes = None
    W = Ws
    refresh_set = set(int(x) for x in refresh_at)
    refreshed_at = -1
    for t in range(T):
        rt = float(rho[t])
        if use_cholesky:
            W = w_update_cholesky(Ht, HW, D, V, rt)
        else:
            W = w_update(lam, U, HW, D, V, rt)                 # line 6
        if probe is not None:
            probe(t, dict(D=D, V=V, rho=rt, W=W, codes=codes))
        W_tilde = W + V / rt
        k_new, D_new = project(W_tilde, s, delta, z0, bits)    # line 7
        if refreshed_at < 0 and t in refresh_set:
            d2, z2 = grid_fit(W_tilde / s[None, :], bits, group_size, symmetric)
            k2, D2 = project(W_tilde, s, d2, z2, bits)
            if np.sum((D2 - W_tilde) ** 2) <= np.sum((D_new - W_tilde) ** 2):
                delta, z0, k_new, D_new = d2, z2, k2, D2
                refreshed_at = t
        r[t] = np.linalg.norm(W - D_new)
        sres[t] = np.linalg.norm(D_new - D)
        if codes is not None:
            changed[t] = int((k_new != codes).sum())
        V = V + rt * (W - D_new)                               # line 8, Eq. 9
        D = D_new
        codes = k_new
    Wq = dequantize(codes, delta, z0)                          # line 11
    return AdmmResult(codes, delta, z0, Wq, r, sres, changed, s, V, W, refreshed_at)


# --------------------------------------------------------------------------
# Objective (Eq. 2 without the 1/2, as in Sec. 3.5: L = sum_j eps_j^T H eps_j)
# --------------------------------------------------------------------------
def objective(H: np.ndarray, W_hat: np.ndarray, Wq: np.ndarray) -> float:
    E = np.asarray(Wq, dtype=F64) - np.asarray(W_hat, dtype=F64)   # [p, n]
    return float(np.einsum("jn,jn->", E @ H, E))


# --------------------------------------------------------------------------
# Local search: single-entry moves = Eq. 11 with the second perturbation zero
# --------------------------------------------------------------------------
@dataclasses.dataclass
class LocalSearchResult:
    codes: np.ndarray
    Wq: np.ndarray
    g: np.ndarray            # maintained gradient H (W_q - W_hat), [p, n]
    moves: np.ndarray        # [p] moves applied per column
    capped: np.ndarray       # [p] bool: stopped at the move cap


def local_search(H: np.ndarray, W_hat: np.ndarray, codes: np.ndarray, delta: np.ndarray,
                 z0: np.ndarray, bits: int, max_moves: int = 0, tau: float = 1e-6
                 ) -> LocalSearchResult:
    """Greedy single-entry local search, every output column independently.

    With g = H (W_q - W_hat) (the paper's G with the sign flipped), moving entry
    i of a column by d = +/-Delta changes that column's loss eps^T H eps by
      c = 2 d g_i + d^2 H_ii                       (Eq. 11 with delta_{i2} = 0).
    Each step applies the move of smallest c among those that keep the code in
    [0, 2^b - 1] (ties: smallest i, then +Delta before -Delta), as long as
    c < -tau * H_ii * Delta^2; then g += d * H[:, i] (rank-1 form of the paper's
    rank-2 gradient correction).  H is the unscaled damped Hessian.
    """
    H = np.asarray(H, dtype=F64)
    W_hat = np.asarray(W_hat, dtype=F64)
    p, n = codes.shape
    kmax = (1 << bits) - 1
    cap = max_moves if max_moves > 0 else 8 * n
    dl = _expand(delta, n)
    hd = np.diag(H).copy()
    k = codes.astype(np.int64).copy()
    Wq = dequantize(codes, delta, z0)
    g = (Wq - W_hat) @ H                                       # [p, n]
    moves = np.zeros(p, dtype=np.int64)
    capped = np.zeros(p, dtype=bool)
    active = np.arange(p)
    while active.size:
        ga, ka, da = g[active], k[active], dl[active]
        quad = da * da * hd[None, :]
        c_plus = np.where(ka < kmax, 2.0 * da * ga + quad, np.inf)
        c_minus = np.where(ka > 0, -2.0 * da * ga + quad, np.inf)
        # candidate order (i, +) before (i, -): interleave so argmin's first-hit
        # rule implements "smallest i, then + before -".
        c = np.stack([c_plus, c_minus], axis=2).reshape(active.size, 2 * n)
        best = np.argmin(c, axis=1)
        cbest = c[np.arange(active.size), best]
        i_star = best // 2
        sign = np.where(best % 2 == 0, 1.0, -1.0)
        d_star = sign * da[np.arange(active.size), i_star]
        thresh = -tau * hd[i_star] * d_star * d_star
        go = cbest < thresh
        if not go.any():
            break
        cols = active[go]
        ii = i_star[go]
        dd = d_star[go]
        k[cols, ii] += sign[go].astype(np.int64)
        Wq[cols, ii] += dd
        g[cols] += dd[:, None] * H[ii, :]
        moves[cols] += 1
        hit = moves[cols] >= cap
        capped[cols[hit]] = True
        active = cols[~hit]
    return LocalSearchResult(k.astype(np.uint8), Wq, g, moves, capped)


# --------------------------------------------------------------------------
# Pair-swap local search (Sec. 3.5 "Algorithm"; Eq. 11 in full)
# --------------------------------------------------------------------------
@dataclasses.dataclass
class PairSwapResult:
    codes: np.ndarray
    Wq: np.ndarray
    g: np.ndarray            # maintained gradient H (W_q - W_hat), [p, n]
    chosen: list             # per round: index of the applied pair in that round's batch, or -1
    totals: list             # per round: total loss change of the applied pair (0 if none)
    moves: int               # (pair, column) moves applied


PAIR_SIGNS = ((1.0, 1.0), (1.0, -1.0), (-1.0, 1.0), (-1.0, -1.0))


def pair_move_costs(g1, g2, h11, h22, h12, d1, d2):
    """Eq. 11 for the four sign combinations, with g = H (W_q - W_hat) = -G:
      c = 2 a d1 g1 + d1^2 H11 + 2 b d2 g2 + d2^2 H22 + 2 a b d1 d2 H12,  (a, b) in PAIR_SIGNS.
    Arrays broadcast; returns an array with a leading axis of length 4."""
    out = []
    for a, b in PAIR_SIGNS:
        out.append(2.0 * a * d1 * g1 + d1 * d1 * h11 + 2.0 * b * d2 * g2 + d2 * d2 * h22
                   + 2.0 * a * b * d1 * d2 * h12)
    return np.stack(out)


def pair_swap(H: np.ndarray, W_hat: np.ndarray, codes: np.ndarray, delta: np.ndarray, z0: np.ndarray,
              bits: int, pairs: np.ndarray, tau: float = 1e-6) -> PairSwapResult:
    """The paper's pair-swap refinement.  `pairs` is [rounds, batch, 2]: the row pairs sampled for every
    round (the random draws are an input).  Each round: for every candidate pair (i1, i2), i1 != i2, and
    every output column independently, the best of the four sign combinations that keep both codes in
    [0, 2^b - 1] is found by Eq. 11; a column takes part only if that cost is below
    -tau (d1^2 H11 + d2^2 H22); the pair's total is the sum of the participating columns' costs.  The pair
    with the smallest total is applied in all participating columns (ties: first in the batch; nothing is
    applied when no total is negative) and the gradient takes the rank-2 correction
    g_j += d1 H[:, i1] + d2 H[:, i2].  H is the unscaled damped Hessian.
    Readings: one pair applied per round (the paper's step (iv)); a column may decline; sign combinations
    are tried in the order (+,+), (+,-), (-,+), (-,-) and the first minimum wins."""
    H = np.asarray(H, dtype=F64)
    W_hat = np.asarray(W_hat, dtype=F64)
    p, n = codes.shape
    kmax = (1 << bits) - 1
    dl = _expand(delta, n)
    k = codes.astype(np.int64).copy()
    Wq = dequantize(codes, delta, z0)
    g = (Wq - W_hat) @ H
    chosen, totals, moves = [], [], 0

    def evaluate(i1, i2):
        d1, d2 = dl[:, i1], dl[:, i2]
        c = pair_move_costs(g[:, i1], g[:, i2], H[i1, i1], H[i2, i2], H[i1, i2], d1, d2)   # [4, p]
        for q, (a, b) in enumerate(PAIR_SIGNS):
            ok = (k[:, i1] + a >= 0) & (k[:, i1] + a <= kmax) & (k[:, i2] + b >= 0) & (k[:, i2] + b <= kmax)
            c[q] = np.where(ok, c[q], np.inf)
        q_best = np.argmin(c, axis=0)
        c_best = c[q_best, np.arange(p)]
        take = c_best < -tau * (d1 * d1 * H[i1, i1] + d2 * d2 * H[i2, i2])
        return q_best, c_best, take

    for batch in np.asarray(pairs):
        best_t, best_b = 0.0, -1
        for b_idx, (i1, i2) in enumerate(batch):
            i1, i2 = int(i1), int(i2)
            if i1 == i2:
                continue
            _, c_best, take = evaluate(i1, i2)
            t = float(np.sum(np.where(take, c_best, 0.0)))
            if t < best_t:
                best_t, best_b = t, b_idx
        chosen.append(best_b)
        totals.append(best_t)
        if best_b < 0:
            continue
        i1, i2 = int(batch[best_b][0]), int(batch[best_b][1])
        q_best, _, take = evaluate(i1, i2)
        sa = np.array([s[0] for s in PAIR_SIGNS])[q_best]
        sb = np.array([s[1] for s in PAIR_SIGNS])[q_best]
        cols = np.nonzero(take)[0]
        da = sa[cols] * dl[cols, i1]
        db = sb[cols] * dl[cols, i2]
        k[cols, i1] += sa[cols].astype(np.int64)
        k[cols, i2] += sb[cols].astype(np.int64)
        Wq[cols, i1] += da
        Wq[cols, i2] += db
        g[cols] += da[:, None] * H[i1, :][None, :] + db[:, None] * H[i2, :][None, :]
        moves += int(cols.size)
    return PairSwapResult(k.astype(np.uint8), Wq, g, chosen, totals, moves)


# --------------------------------------------------------------------------
# Whole layer: Algorithm 1
# --------------------------------------------------------------------------
@dataclasses.dataclass
class LayerResult:
    admm: AdmmResult
    ls: Optional[LocalSearchResult]
    H: np.ndarray
    err_admm: float
    err_final: float


def quantize_layer(H: np.ndarray, W_hat: np.ndarray, bits: int, group_size: int,
                   symmetric: bool, rho: np.ndarray, do_local_search: bool = True,
                   precond: bool = True, max_moves: int = 0, tau: float = 1e-6,
                   probe=None, grid: Optional[tuple] = None) -> LayerResult:
    """Algorithm 1 on a damped Hessian H: ADMM loop, then local search (line 12).
    `grid` = (Delta, z0), each [p, n/gs]: run on this grid instead of fitting one (passed on to `admm`)."""
    a = admm(H, W_hat, bits, group_size, symmetric, rho, precond=precond, probe=probe, grid=grid)
    e0 = objective(H, W_hat, a.Wq)
    ls = None
    e1 = e0
    if do_local_search:
        ls = local_search(H, W_hat, a.codes, a.delta, a.z0, bits, max_moves, tau)
        e1 = objective(H, W_hat, ls.Wq)
    return LayerResult(a, ls, H, e0, e1)
