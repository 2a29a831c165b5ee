// Host-side declarations shared by the translation units of libadmmq.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "epilogue.cuh"

namespace admmq {

typedef __nv_bfloat16 bf16;

// One operand of a product C = A * B^T: up to two bf16 planes (hi, lo) whose sum is the value.
// Row-major [rows][ld], the contraction index contiguous ("K-major").
struct Planes {
  const bf16* hi;           // 16-bit storage: bf16 values, or fp16 values when f16 != 0
  const bf16* lo;           // nullptr: single plane
  long long ld;
  int f16;                  // 1: planes hold fp16 values that were scaled by a power of two first
  const float* row_inv;     // [rows] inverse of each row's scale (device), or nullptr
  const float* all_inv;     // inverse of a scale common to all elements (device scalar), or nullptr
};
inline Planes planes_bf16(const bf16* hi, const bf16* lo, long long ld) { return Planes{hi, lo, ld, 0, nullptr, nullptr}; }
inline Planes planes_f16(const bf16* hi, const bf16* lo, long long ld, const float* row_inv, const float* all_inv) {
  return Planes{hi, lo, ld, 1, row_inv, all_inv};
}

struct Ctx {
  int n = 0, p_max = 0, T_max = 0;
  cudaStream_t stream = nullptr;
  int num_sms = 148;
  int gemm_kind = 0;
  int state = 0;            // 0 created, 1 hessian open, 2 factored
  long long n_tokens = 0;
  int T = 0;
  int precondition = 1;
  double rho_host[4096];
  unsigned char planes_host[4096];  // per iteration: operand planes the W-update products need (1 or 2)
  unsigned char series_host[4096];  // per iteration: terms of E the truncated series needs to be accurate to fp32 (1, 2), 0: not usable
  double mu_host = 1.0, lam_lo = 0.0, lam_hi = 0.0;   // mean and Gershgorin bounds of the spectrum of H~ (host copies)
  long long launches = 0;
  long long wait_limit_cycles = 2000000000LL;   // bound of every device-side wait, about a second
  int pair_clusters = 0;
  int use_pair_kernel = 1;
  int one_plane_flush_kb = 1 << 20;   // K blocks per flush of the one-plane fp16 products (whole K by default)
  int hold_loads = 0;           // failure-handling tests only: the product kernel's producer issues no loads
  // ---- workspace carve-up (device) ----
  char* ws = nullptr;
  size_t ws_bytes = 0;
  int* status = nullptr;        // device status word (+ padding)
  float* H_raw = nullptr;       // [n][n] fp32 accumulator of X^T X (lower triangle valid until finalize)
  float* H = nullptr;           // [n][n] fp32 damped, unscaled
  float* s = nullptr;           // [n]
  float* inv_s = nullptr;       // [n] 1 / s_i
  double* s64 = nullptr;        // [n] s_i in fp64 (the element update works in fp64)
  double* inv_s64 = nullptr;    // [n] 1 / s_i in fp64
  float* hdiag = nullptr;       // [n] diag of damped H
  double* A64 = nullptr;        // [n][n] fp64 working copy of H~, reflectors afterwards
  double* P64 = nullptr;        // [n][n] fp64 Q^T
  double* td = nullptr;         // [n] tridiagonal diagonal
  double* te = nullptr;         // [n] tridiagonal off-diagonal
  double* beta = nullptr;       // [n] reflector scalars
  double* pvec = nullptr;       // [n] matrix-vector scratch of the reduction
  float* stage_l = nullptr;     // [T_max+1][stage_factor_stride(n)] LDL^T multipliers per penalty
  float* stage_invd = nullptr;  // [T_max+1][stage_factor_stride(n)] LDL^T inverse pivots per penalty, times 1 / (mu + rho)
  double* shift_c = nullptr;    // [T_max+1] c = rho / (mu + rho) per penalty (shifted W-update operator)
  bf16* N_hi = nullptr;         // [n][n] one fp16 plane of mu I - H~ (operand of the truncated-series W-update), scale in fscal[9..11]
  bf16* N_lo = nullptr;         // its lo plane (first-order term of the two-term series, which needs two planes)
  float* series_g = nullptr;    // [T_max+1] per penalty: 1 / (mu + rho) times the inverse scale of the N planes
  float* series_f = nullptr;    // [T_max+1] per penalty: rho / (mu + rho)^2 times the inverse scale of N_hi
  float* Qs32 = nullptr;        // [n][n] fp32 Q (mu I - T), or nullptr: input of the explicit-operator route (p_max > n only)
  double* ps_totals = nullptr;  // [PAIR_BATCH_MAX] totals of the candidate pairs of a pair-swap round
  int* ps_chosen = nullptr;     // [1] index of the applied pair, -1: none
  float* ps_d = nullptr;        // [2][p] applied perturbations of the two rows
  double* trd_ws = nullptr;     // scratch of the blocked reduction (tridiag_blocked_scratch_doubles)
  double* wy_s = nullptr;       // [ceil(n/32)][32][32] triangular factors of the reflector blocks
  bf16 *Q_hi = nullptr, *Q_lo = nullptr;    // [n][n] Q   (row i, col m)
  bf16 *QT_hi = nullptr, *QT_lo = nullptr;  // [n][n] Q^T (row m, col k)
  bf16 *H_hi = nullptr, *H_lo = nullptr;    // [n][n] split planes of the damped unscaled H
  float* V = nullptr;           // [p][n]
  bf16 *R_hi = nullptr, *R_lo = nullptr;    // [p][n]
  float* Y = nullptr;           // [p][n] (also the local-search gradient g)
  bf16 *Y_hi = nullptr, *Y_lo = nullptr;    // [p][n]
  float* partials = nullptr;    // [T_max][slots][2]
  int partial_slots = 0;
  double* scal = nullptr;       // small fp64 scalars (objective, counters)
  float* fscal = nullptr;       // [0] 1 / scale of the Q planes, [1] 1 / scale of the H planes, [2] scale of the H planes,
                                // [3] 1 / scale and [4] scale of the shifted Q^T planes, [5] their largest magnitude,
                                // [6..8] 1 / scale, scale, largest magnitude of the explicit operator's planes; [9..11] the same of N_hi
  float* rs_R = nullptr;        // [p] inverse row scales of the R (and E) planes
  float* rs_Y = nullptr;        // [p] inverse row scales of the Y' planes
  bf16 *XT_hi = nullptr, *XT_lo = nullptr;  // [n][XT_ROWS] transposed chunk of X
  void* tmaps = nullptr;        // reserved
};

constexpr int XT_ROWS = 16384;   // calibration rows handled per Hessian launch

// Raises a kernel's dynamic shared-memory limit to at least `bytes` on the CURRENT device.  The attribute
// belongs to a (kernel, device) pair, so the record of what was already set is kept per pair, under a
// mutex: contexts on several GPUs of one process, and host threads, each get a correctly set-up kernel.
cudaError_t ensure_dynamic_smem(const void* kernel, int bytes);

// ---- elem.cu ----
void launch_zero(Ctx* c, void* ptr, size_t bytes);
void launch_transpose_split(Ctx* c, const void* X, int is_bf16, long long rows, long long ldx, int n,
                            bf16* XT_hi, bf16* XT_lo, long long ldt);
void launch_finalize(Ctx* c, double damp_frac, int precondition);
void launch_symmetric_copy(Ctx* c, float* out);      // H_raw (lower triangle valid) -> full symmetric matrix
void launch_grid_fit(Ctx* c, const float* W0, int p, int bits, int gs, int symmetric, float* delta,
                     float* zero);
void launch_admm_rows(Ctx* c, const EpiParams& P, int p, bf16* hi, bf16* lo, float* row_inv);
void launch_grid_fit_mse(Ctx* c, const float* W0, int p, int bits, int gs, int symmetric, int points,
                         double min_ratio, float* delta, float* zero);
void launch_scale_weights(Ctx* c, const float* W0, int p);   // start of a layer: V = 0, R = 0, finite check of W_hat
void launch_operand_scales(Ctx* c);   // fscal from diag(H)
void launch_split_f64(Ctx* c, const double* src, int n, bf16* hi, bf16* lo, bf16* thi, bf16* tlo);
void launch_split_f32(Ctx* c, const float* src, long long count, bf16* hi, bf16* lo);
void launch_global_split(Ctx* c, const float* src, long long count, float* slot, bf16* hi, bf16* lo);
void launch_shifted_qt(Ctx* c);       // mu = mean(td) -> scal[8]; planes of [Q (mu I - T)]^T -> QT_hi / QT_lo, scales -> fscal[3..5]
void launch_w_out(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes, const float* delta,
                  const float* zero, const float* V_in, double inv_rho, const double* shift_c, const float* z,
                  float* W_out, int correction_only);
void launch_row_split(Ctx* c, const float* src, int p, bf16* hi, bf16* lo, float* row_inv);
void launch_init_rhs(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes, const float* delta,
                     const float* zero, const float* V_in, double inv_rho, float* R_out);
void launch_reduce_partials(Ctx* c, int T, float* resid);
void launch_dequant(Ctx* c, int p, int gs, const unsigned char* codes, const float* delta,
                    const float* zero, float* Wq);
void launch_error_planes(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes,
                         const float* delta, const float* zero, bf16* Ehi, bf16* Elo, float* row_inv);
void launch_grid_refresh(Ctx* c, const EpiParams& P, int p, int bits, int symmetric, int iter, float* delta,
                         float* zero, int* flags);
void launch_objective_dot(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes,
                          const float* delta, const float* zero, const float* g, double* out);

// ---- gemm_simt.cu / gemm_tc.cu:  C[M][N] (epilogue)= A[M][K] * B[N][K]^T ----
cudaError_t gemm_simt(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi);
cudaError_t gemm_tc(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi);
int gemm_tc_partial_slots(int num_sms);

// ---- tridiag.cu ----
cudaError_t tridiag_reduce(Ctx* c);                 // A64 -> td, te, reflectors, beta
cudaError_t tridiag_reduce_blocked(Ctx* c);         // the same result, panels of 32 columns
size_t tridiag_blocked_scratch_doubles(int n);
cudaError_t tridiag_form_qt(Ctx* c);                // reflectors -> P64 = Q^T
size_t stage_factor_stride(int n);                  // floats per penalty in stage_l / stage_invd
void launch_stage_factors(Ctx* c, const double* rho_dev, int first, int count);
void launch_admm_tail(Ctx* c, const EpiParams& P, int p, const double* rho_dev, int first, int count, int T);
void launch_series_operand(Ctx* c);   // A64 = H~ (before the reduction overwrites it) -> N_hi, fscal[9..11]; mean of its diagonal -> scal[11]
void launch_tridiag_solve(Ctx* c, const float* Y, int p, int stage, bf16* hi, bf16* lo, float* row_inv);

// ---- local_search.cu ----
cudaError_t launch_local_search(Ctx* c, const float* W0, int p, int bits, int gs, long long max_moves,
                                float tau, unsigned char* codes, const float* delta,
                                const float* zero, float* Wq, float* g, long long* d_moves,
                                int* d_capped);

// ---- pair_swap.cu ----
constexpr int PAIR_BATCH_MAX = 65536;
cudaError_t launch_pair_round(Ctx* c, int p, int bits, int gs, float tau, unsigned char* codes,
                              const float* delta, const float* zero, float* Wq, float* g, const int* pairs,
                              int batch, long long* d_moves, int* d_rounds);

}  // namespace admmq
