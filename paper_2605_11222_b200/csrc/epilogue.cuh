// Epilogues of the matrix-product kernels: what happens to an accumulator tile before it
// leaves the SM.  Shared by the tensor-core and the SIMT product kernels so that both
// apply identical arithmetic.
#pragma once
#include "common.cuh"

namespace admmq {

enum EpiKind : int {
  EPI_STORE = 0,   // C = acc
  EPI_ACCUM = 1,   // C += acc                     (Hessian accumulation)
  EPI_ADMM = 2     // projection + dual update + residuals + next right-hand side (Eq. 8-10)
};

struct EpiParams {
  int kind;
  float* C;                 // STORE / ACCUM: output [M][ldc]
  long long ldc;
  int lower_only;           // ACCUM: skip elements with col > row (symmetric product)
  // ---- ADMM state, all [p][n] row-major with leading dimension n ----
  const float* W0;          // W_hat, unscaled, as the caller passed it (ADMM element update)
  float* V;                 // dual V (in/out)
  unsigned char* codes;     // codes of D (in: D^(t), out: D^(t+1))
  const float* s;           // [n] s_i = sqrt(H_ii)
  const float* inv_s;       // [n] 1 / s_i, fp32
  const float* delta;       // [p][n_groups]
  const float* zero;        // [p][n_groups]
  int group_size, n_groups;
  int kmax;                 // 2^bits - 1
  int first_iter;           // 1: D^(0) = W_hat' (Algorithm 1 line 4), codes not yet defined
  double rho, inv_rho, inv_rho_next;
  const double* shift_c;    // device scalar c = rho / (mu + rho) of this iteration: the product's output is the
                            // W-update correction WITHOUT its c R part, which the element update adds
  float* Rnext;             // next right-hand side D - V/rho_next - W_hat' (fp32; split into planes by a row pass)
  float* partials;          // [slots][2]: per-CTA sums of (W-D)^2 and (D-D_old)^2
  // ---- undoing the operands' power-of-two scales: value = acc * row_inv[row] * a_inv[0] * b_inv[0] ----
  const float* row_inv;     // [M] or nullptr
  const float* a_inv;       // device scalar or nullptr
  const float* b_inv;       // device scalar or nullptr
};

// Factor that turns an accumulator of output row `row` back into the unscaled product.
__device__ __forceinline__ float epi_row_factor(const EpiParams& P, int row) {
  float f = 1.0f;
  if (P.row_inv) f = P.row_inv[row];
  if (P.a_inv) f *= P.a_inv[0];
  if (P.b_inv) f *= P.b_inv[0];
  return f;
}

// One element of the ADMM update (Eq. 8-10).  zp is the product's output, z = zp + c R the W-update of Eq. 7
// written for the error W - W_hat'.
//
// Every quantity here is kept RELATIVE to the pre-trained weight, i.e. at the size of a grid step, never at
// the size of the weight itself: in unscaled coordinates the projection target is
//     Sigma W~ = w_hat + (z + V/rho) / s,
// so the code is k = rint(((w_hat - z0) + (z + V/rho)/s) / Delta), and the grid point enters only through its
// distance from the weight, D - W_hat' = s (z0 + Delta k - w_hat).  (In plain fp32 the sums W_hat' + z,
// s (z0 + Delta k) and y - z0 each round at the weight's magnitude, up to 2^(bits-1) grid steps: ~1e-6 of a
// step per iteration at 4 bits, which decided most of the codes that differed from an fp64 run.)
//
// The two places where numbers of the weight's size meet are evaluated without rounding, in fp32:
//   a = w_hat - z0 as the unevaluated sum a_hi + a_lo of an error-free subtraction;
//   Delta k as p + pe with p = fl(Delta k) and pe = fma(Delta, k, -p), so that Delta k - a comes out with the
//   relative accuracy of a grid-step-sized number.
// The rounding decision itself is first taken on the fp32 value of (a + u) / Delta, which is good to ~1e-6 of a
// step; only when that lands within ROUND_MARGIN of a half-integer is it retaken in fp64 from the same fp32
// inputs, like the oracle's.  (An all-fp64 element update was measured: row pass 113 us instead of 72 us, the
// conversions between the two formats being the cost, and no fewer differing codes.)
struct AdmmElem {
  unsigned char code;
  float v_new, r_next, dr2, ds2;
};
// Constants of one (channel, group): Delta, z0 and 1 / Delta.
struct GridG {
  float dl, z0, inv_dl;
};
__device__ __forceinline__ GridG grid_g(float dl, float z0) {
  GridG g;
  g.dl = dl;
  g.z0 = z0;
  g.inv_dl = __frcp_rn(dl);
  return g;
}
constexpr float ROUND_MARGIN = 1e-4f;

// w_hat - z0 = hi + lo exactly (branch-free two-sum).  The intrinsics keep the compiler from contracting or
// reordering the steps: each must round exactly once, as written.
__device__ __forceinline__ void diff_exact(float w0, float z0, float& hi, float& lo) {
  hi = __fsub_rn(w0, z0);
  const float bb = __fsub_rn(hi, w0);
  lo = __fsub_rn(__fsub_rn(w0, __fsub_rn(hi, bb)), __fadd_rn(z0, bb));
}
// s (Delta k - a) for a = a_hi + a_lo: the distance of grid point k from the weight, scaled coordinates.
__device__ __forceinline__ float grid_offset(float s, float dl, float k, float a_hi, float a_lo) {
  const float p = __fmul_rn(dl, k);
  const float pe = __fmaf_rn(dl, k, -p);                  // Delta k = p + pe exactly
  // (the product by s rounds once, here: left to the compiler it may be contracted into the caller's next
  // subtraction, and two evaluations of the same grid point would then no longer cancel exactly)
  return __fmul_rn(s, __fsub_rn(__fadd_rn(__fsub_rn(p, a_hi), pe), a_lo));
}

// g: the grid the new code is taken on; g_old: the grid code_old refers to (the same one, except in the
// iteration that accepts a grid refresh).
// The iteration's scalars in the precision the update uses them in.
struct IterF {
  float rho, inv_rho, inv_rho_next;
  int first_iter, kmax;
};
__device__ __forceinline__ IterF iter_f(const EpiParams& P) {
  IterF q;
  q.rho = (float)P.rho;
  q.inv_rho = (float)P.inv_rho;
  q.inv_rho_next = (float)P.inv_rho_next;
  q.first_iter = P.first_iter;
  q.kmax = P.kmax;
  return q;
}

__device__ __forceinline__ AdmmElem admm_elem(float zp, float w0, float v, int code_old, float s, float inv_s,
                                              const GridG& g, const GridG& g_old, float cshift, const IterF& P) {
  AdmmElem o;
  float a_hi, a_lo;
  diff_exact(w0, g.z0, a_hi, a_lo);
  float e_old = 0.0f;                                      // D^(0) = W_hat'
  if (!P.first_iter) {
    float b_hi = a_hi, b_lo = a_lo;
    if (g_old.z0 != g.z0) diff_exact(w0, g_old.z0, b_hi, b_lo);
    e_old = grid_offset(s, g_old.dl, (float)code_old, b_hi, b_lo);
  }
  const float inv_rho = P.inv_rho;
  // z = c R + (product output), R = D^(t) - V/rho - W_hat' exactly as the right-hand side was formed
  const float z = fmaf(cshift, fmaf(-v, inv_rho, e_old), zp);
  const float u = fmaf(v, inv_rho, z) * inv_s;             // (W~ - W_hat') / s: target minus weight  (Eq. 8)
  const float x = __fadd_rn(__fadd_rn(a_hi, u), a_lo) * g.inv_dl;   // (Sigma W~ - z0) / Delta, good to ~1e-6
  float k = rintf(x);                                      // nearest level, ties to even    (Eq. 10)
  if (fabsf(fabsf(x - k) - 0.5f) < ROUND_MARGIN)           // too close to a tie for fp32: decide in fp64
    k = (float)rint((((double)w0 - (double)g.z0) + (double)u) / (double)g.dl);
  k = fminf(fmaxf(k, 0.0f), (float)P.kmax);
  const float e_new = grid_offset(s, g.dl, k, a_hi, a_lo); // D^(t+1) - W_hat'
  const float wd = z - e_new;                              // W^(t+1) - D^(t+1)
  const float dd = e_new - e_old;                          // D^(t+1) - D^(t)
  o.code = (unsigned char)(int)k;
  o.v_new = fmaf(P.rho, wd, v);                            // V += rho (W - D)               (Eq. 9)
  o.r_next = fmaf(-o.v_new, P.inv_rho_next, e_new);        // next R = D - V/rho' - W_hat'
  o.dr2 = wd * wd;
  o.ds2 = dd * dd;
  return o;
}
__device__ __forceinline__ AdmmElem admm_elem(float zp, float w0, float v, int code_old, float s, float inv_s,
                                              const GridG& g, const GridG& g_old, float cshift, const EpiParams& P) {
  return admm_elem(zp, w0, v, code_old, s, inv_s, g, g_old, cshift, iter_f(P));
}

// Scalar epilogue for one output element (used by the SIMT kernel and for ragged edges).
__device__ __forceinline__ void epi_scalar(const EpiParams& P, int row, int col, int n_cols, float acc,
                                           float& r2, float& s2) {
  acc *= epi_row_factor(P, row);
  if (P.kind == EPI_STORE) {
    P.C[(long long)row * P.ldc + col] = acc;
  } else if (P.kind == EPI_ACCUM) {
    if (!P.lower_only || col <= row) P.C[(long long)row * P.ldc + col] += acc;
  } else {
    const long long idx = (long long)row * n_cols + col;
    const int g = col / P.group_size;
    const float dl = P.delta[(long long)row * P.n_groups + g];
    const float z0 = P.zero[(long long)row * P.n_groups + g];
    const GridG gg = grid_g(dl, z0);
    AdmmElem e = admm_elem(acc, P.W0[idx], P.V[idx], P.first_iter ? 0 : (int)P.codes[idx], P.s[col],
                           P.inv_s[col], gg, gg, (float)P.shift_c[0], P);
    P.codes[idx] = e.code;
    P.V[idx] = e.v_new;
    P.Rnext[idx] = e.r_next;
    r2 += e.dr2;
    s2 += e.ds2;
  }
}

}  // namespace admmq
