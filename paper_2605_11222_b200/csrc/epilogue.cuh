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
  const double* s;          // [n] s_i = sqrt(H_ii), fp64
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

// One element of the ADMM update (Eq. 8-10).  z = [Q (T/rho + I)^{-1} Q^T R]_{ji} is the product's output, so
// that W = W_hat' + z is the W-update of Eq. 7 written for the error W - W_hat'.
//
// Every quantity here is kept RELATIVE to the pre-trained weight, i.e. at the size of a grid step, never at
// the size of the weight itself: in unscaled coordinates the projection target is
//     Sigma W~ = w_hat + (z + V/rho) / s,
// so the code is k = rint(((w_hat - z0) + (z + V/rho)/s) / Delta), and the grid point enters only through its
// distance from the weight, D - W_hat' = s (z0 + Delta k - w_hat).  The two places where numbers of the
// weight's size meet -- (w_hat - z0) and (Delta k - (w_hat - z0)) -- are evaluated in fp64, where both are
// exact; the rounding decision of Eq. 10 is taken in fp64 like the oracle's.  (In plain fp32 the sums
// W_hat' + z, s (z0 + Delta k) and y - z0 each round at the weight's magnitude, up to 2^(bits-1) grid steps:
// ~1e-6 of a step per iteration at 4 bits, which is what decided most of the codes that differed from an
// fp64 run.)
struct AdmmElem {
  unsigned char code;
  float v_new, r_next, dr2, ds2;
};
// Constants of one (channel, group): Delta, z0 and 1 / Delta in fp64.
struct GridG {
  float dl, z0;
  double inv_dl;
};
__device__ __forceinline__ GridG grid_g(float dl, float z0) {
  GridG g;
  g.dl = dl;
  g.z0 = z0;
  g.inv_dl = 1.0 / (double)dl;
  return g;
}
// g: the grid the new code is taken on; g_old: the grid code_old refers to (the same one, except in the
// iteration that accepts a grid refresh).  fp64 is used where numbers of the weight's size meet and for the
// rounding decision; the grid-step-sized quantities around them (z, V/rho, the residuals) are fp32, which is the
// precision they are stored in anyway (measured on the 12288-wide layers: the correction W - W_hat' reaches the
// decision with an error of 2e-8 to 6e-8 of a grid step rms, the rounding of its own fp32 storage).
__device__ __forceinline__ AdmmElem admm_elem(float zp, float w0, float v, int code_old, double s, float inv_s,
                                              const GridG& g, const GridG& g_old, float cshift, const EpiParams& P) {
  AdmmElem o;
  const double a = (double)w0 - (double)g.z0;              // w_hat - z0, exact
  const float e_old = P.first_iter ? 0.0f                  // D^(0) = W_hat'
                                   : (float)(s * fma((double)g_old.dl, (double)code_old,
                                                     (double)g_old.z0 - (double)w0));
  const float inv_rho = (float)P.inv_rho;
  // z = c R + (product output), R = D^(t) - V/rho - W_hat' exactly as the right-hand side was formed
  const float z = fmaf(cshift, fmaf(-v, inv_rho, e_old), zp);
  const float u = fmaf(v, inv_rho, z) * inv_s;             // (W~ - W_hat') / s: target minus weight  (Eq. 8)
  double k = rint((a + (double)u) * g.inv_dl);             // nearest level, ties to even    (Eq. 10)
  k = fmin(fmax(k, 0.0), (double)P.kmax);
  const float e_new = (float)(s * fma((double)g.dl, k, -a));               // D^(t+1) - W_hat'
  const float wd = z - e_new;                              // W^(t+1) - D^(t+1)
  const float dd = e_new - e_old;                          // D^(t+1) - D^(t)
  o.code = (unsigned char)(int)k;
  o.v_new = fmaf((float)P.rho, wd, v);                     // V += rho (W - D)               (Eq. 9)
  o.r_next = fmaf(-o.v_new, (float)P.inv_rho_next, e_new); // next R = D - V/rho' - W_hat'
  o.dr2 = wd * wd;
  o.ds2 = dd * dd;
  return o;
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
