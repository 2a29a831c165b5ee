// Epilogues of the matrix-product kernels: what happens to an accumulator tile before it
// leaves the SM.  Shared by the tensor-core and the SIMT product kernels so that both
// apply identical arithmetic.
#pragma once
#include "common.cuh"

namespace admmq {

enum EpiKind : int {
  EPI_STORE = 0,   // C = acc
  EPI_ACCUM = 1,   // C += acc                     (Hessian accumulation)
  EPI_ADMM = 2,    // projection + dual update + residuals + next right-hand side (Eq. 8-10)
  EPI_WOUT = 3     // C = W_hat' + acc             (W-update of Eq. 7 alone)
};

struct EpiParams {
  int kind;
  float* C;                 // STORE / ACCUM / WOUT: output [M][ldc]
  long long ldc;
  int lower_only;           // ACCUM: skip elements with col > row (symmetric product)
  // ---- ADMM state, all [p][n] row-major with leading dimension n ----
  const float* Whs;         // W_hat' = s_i * W_hat  (scaled pre-trained weights)
  float* V;                 // dual V (in/out)
  unsigned char* codes;     // codes of D (in: D^(t), out: D^(t+1))
  const float* s;           // [n] s_i = sqrt(H_ii)
  const float* inv_s;       // [n] 1 / s_i
  const float* delta;       // [p][n_groups]
  const float* zero;        // [p][n_groups]
  int group_size, n_groups;
  int kmax;                 // 2^bits - 1
  int first_iter;           // 1: D^(0) = W_hat' (Algorithm 1 line 4), codes not yet defined
  float rho, inv_rho, inv_rho_next;
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

// One element of the fused ADMM epilogue.  z = [Q (T/rho + I)^{-1} Q^T R]_{ji} is the accumulator, so
// that W = W_hat' + z is the W-update of Eq. 7 written for the error W - W_hat'.
struct AdmmElem {
  unsigned char code;
  float v_new, r_next, dr2, ds2;
};
// The two divisions of the projection are taken as products with 1 / s_i and 1 / Delta (each correctly
// rounded): the epilogue runs on the critical path of every tile, and a full-precision division costs as
// much as the rest of the element.
__device__ __forceinline__ AdmmElem admm_elem(float z, float wh, float v, int code_old, float s, float inv_s,
                                              float dl, float inv_dl, float z0, const EpiParams& P) {
  AdmmElem o;
  const float w = wh + z;                                  // W^(t+1)
  const float wt = fmaf(v, P.inv_rho, w);                  // target W~ = W + V/rho          (Eq. 8)
  const float y = wt * inv_s;                              // unscaled coordinate Sigma W~
  float k = rintf((y - z0) * inv_dl);                      // nearest level, ties to even    (Eq. 10)
  k = fminf(fmaxf(k, 0.0f), (float)P.kmax);
  const float d_new = s * (z0 + dl * k);                   // D^(t+1), scaled coordinates
  const float d_old = P.first_iter ? wh : s * (z0 + dl * (float)code_old);
  const float wd = w - d_new;
  const float dd = d_new - d_old;
  o.code = (unsigned char)k;
  o.v_new = v + P.rho * wd;                                // V += rho (W - D)               (Eq. 9)
  o.r_next = d_new - o.v_new * P.inv_rho_next - wh;        // next R = D - V/rho' - W_hat'
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
  } else if (P.kind == EPI_WOUT) {
    P.C[(long long)row * P.ldc + col] = P.Whs[(long long)row * n_cols + col] + acc;
  } else {
    const long long idx = (long long)row * n_cols + col;
    const int g = col / P.group_size;
    const float dl = P.delta[(long long)row * P.n_groups + g];
    const float z0 = P.zero[(long long)row * P.n_groups + g];
    AdmmElem e = admm_elem(acc, P.Whs[idx], P.V[idx], P.first_iter ? 0 : (int)P.codes[idx], P.s[col],
                           P.inv_s[col], dl, __frcp_rn(dl), z0, P);
    P.codes[idx] = e.code;
    P.V[idx] = e.v_new;
    P.Rnext[idx] = e.r_next;
    r2 += e.dr2;
    s2 += e.ds2;
  }
}

}  // namespace admmq
