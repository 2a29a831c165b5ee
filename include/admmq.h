/*
 * admmq.h -- C ABI of the B200 (sm_100a) ADMM-Q layer-wise quantization solver.
 *
 * The library solves, for one linear layer,
 *     min_W  Tr((W - W_hat)^T H (W - W_hat))   s.t.  W on a low-bit uniform grid,
 *     H = X^T X / N + lambda I                                        (Eq. 1, Eq. 2)
 * by the operator-splitting iteration of Algorithm 1 followed by a greedy
 * local search (Sec. 3.5).  Paper notation: n = d_in (input channels, size of H),
 * p = d_out (output channels), N = calibration rows.
 *
 * Conventions shared by every call
 *  - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller owns
 *    every buffer, including the workspace; the library never allocates or frees
 *    device memory (admmq_create allocates only a small host struct).
 *  - Every n-by-p matrix of the paper (W_hat, codes, W_q) is passed TRANSPOSED as a
 *    row-major [d_out][d_in] array (the layout of a linear layer's weight): row j is
 *    output channel j, input channels are contiguous.
 *  - Work is enqueued on the CUDA stream given to admmq_create and is asynchronous
 *    unless a call says that it synchronises.  No call throws, aborts or traps.
 *  - Argument, shape and call-order errors are returned at once, with nothing
 *    enqueued.  Numerical failures found on the device (non-finite input, a
 *    non-positive Hessian diagonal or pivot, a wait that ran out) are recorded in a
 *    device status word: admmq_last_device_status synchronises and returns it, and a
 *    call given a non-NULL host report returns it too.  The word keeps the first error
 *    raised since it was last read, and reading it clears it: the error is returned
 *    once, and the next call on the context (for example quantize_layer with a valid
 *    weight matrix after one that held a NaN, on the same factorisation) starts from
 *    ADMMQ_OK.  admmq_hessian_reset and admmq_hessian_set clear it as well.  Outputs
 *    are unspecified after an error.
 *  - Device pointers must be 16-byte aligned; d_in must be a multiple of 8 and at
 *    most ADMMQ_MAX_D_IN; d_in must be a multiple of the group size.
 *  - Call order: create -> hessian_reset -> hessian_accumulate* -> factor ->
 *    (quantize_layer -> local_search)* -> destroy.  Several weight matrices that
 *    share one H may reuse one factor.  A call out of order returns ADMMQ_ERR_STATE.
 */
#ifndef ADMMQ_H_
#define ADMMQ_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ADMMQ_MAX_D_IN 14336
#define ADMMQ_MAX_BITS 8

typedef struct admmq_ctx admmq_ctx; /* opaque */

typedef enum {
  ADMMQ_OK = 0,
  ADMMQ_ERR_INVALID_ARG = 1,  /* NULL pointer, bad enum, bad struct_size, misaligned pointer */
  ADMMQ_ERR_SHAPE = 2,        /* sizes outside the supported range or not divisible as required */
  ADMMQ_ERR_STATE = 3,        /* call out of order */
  ADMMQ_ERR_WORKSPACE = 4,    /* workspace too small */
  ADMMQ_ERR_NOT_SPD = 5,      /* non-positive Hessian diagonal or pivot (device status) */
  ADMMQ_ERR_NONFINITE = 6,    /* NaN/Inf met in H or W_hat (device status) */
  ADMMQ_ERR_TIMEOUT = 7,      /* a bounded device-side wait ran out (device status) */
  ADMMQ_ERR_CUDA = 8,         /* a CUDA runtime/driver call failed */
  ADMMQ_ERR_UNSUPPORTED = 9,  /* valid request that this build does not implement */
  ADMMQ_WARN_MOVE_CAP = 10    /* local search stopped at max_moves_per_col in some column */
} admmq_status;

typedef enum { ADMMQ_F32 = 0, ADMMQ_BF16 = 1 } admmq_dtype;

/* How the product (H~ + rho I)^{-1} of the W-update (Eq. 7) is applied.
 * TRIDIAG: one orthogonal reduction H~ = Q T Q^T (T tridiagonal), reused for every rho, with an O(n)
 *          LDL^T of T + rho I per penalty value -- the role the single eigendecomposition plays in
 *          Algorithm 1 line 3.  It is the only kind; the field exists so that the struct need not
 *          change if another is added. */
typedef enum { ADMMQ_FACTOR_TRIDIAG = 0 } admmq_factor_kind;

/* Which matrix-product kernels run.  TENSOR: tcgen05 tensor-core kernels on two-plane 16-bit operands
 * (power-of-two scaled fp16 hi + lo for the W-update and gradient products, bf16 for the calibration
 * activations) with fp32 accumulation: the product path.  SIMT: plain fp32 FMA kernels on the same
 * operands, kept as an on-device cross-check. */
typedef enum { ADMMQ_GEMM_TENSOR = 0, ADMMQ_GEMM_SIMT = 1 } admmq_gemm_kind;

const char* admmq_status_string(admmq_status s);

/* Bytes of device workspace a context needs for layers with d_in input channels, at most d_out_max
 * output channels and at most T_max ADMM iterations.  Returns 0 for unsupported sizes. */
size_t admmq_workspace_bytes(int d_in, int d_out_max, int T_max);

/* Creates a context for one value of d_in.  d_workspace: device memory of at least
 * admmq_workspace_bytes(...) bytes, 256-byte aligned, owned by the caller and kept alive until
 * admmq_destroy.  cuda_stream: a cudaStream_t (NULL = the default stream).  Synchronous. */
admmq_status admmq_create(admmq_ctx** ctx, int d_in, int d_out_max, int T_max, void* d_workspace,
                          size_t workspace_bytes, void* cuda_stream);
admmq_status admmq_destroy(admmq_ctx* ctx); /* frees the host struct only */
admmq_status admmq_set_gemm_kind(admmq_ctx* ctx, admmq_gemm_kind kind);

/* Synchronises the stream, returns the device status word (ADMMQ_OK if none was raised) and clears it. */
admmq_status admmq_last_device_status(admmq_ctx* ctx);

/* ---- Step 1: Hessian accumulation, H_raw += X^T X, N += n_tokens  (Sec. 3.1: H = X^T X). ----------
 * d_X: [n_tokens][ldx] row-major, dtype fp32 or bf16; the first d_in columns of each row are used;
 * ldx >= d_in, and ldx * sizeof(element) a multiple of 16.  Only read.  May be called any number of
 * times after admmq_hessian_reset; accumulation is in fp32.  n_tokens == 0 is a no-op. */
admmq_status admmq_hessian_reset(admmq_ctx* ctx);
admmq_status admmq_hessian_accumulate(admmq_ctx* ctx, const void* d_X, admmq_dtype dtype,
                                      long long n_tokens, long long ldx);
/* Alternative to accumulation: the caller supplies the UNDAMPED Hessian X^T X / N directly
 * (Algorithm 1 takes H as its input).  d_H: [d_in][d_in] fp32, symmetric.  Counts as N = 1. */
admmq_status admmq_hessian_set(admmq_ctx* ctx, const float* d_H);

/* The accumulated state of step 1, for a Hessian whose calibration rows are spread over several contexts
 * (for instance one per GPU, each fed its share of the tokens): every context exports its sum, the caller
 * adds the sums element by element (an all-reduce) and imports the total, with the total row count, into
 * every context before admmq_factor.  H = X^T X is a plain sum over the rows (Sec. 3.1), so the result is
 * the Hessian of all rows.
 * export: d_Hraw_out [d_in][d_in] fp32 receives sum_t x_t x_t^T of the rows accumulated so far (full
 *         symmetric matrix, not divided by N); *h_tokens (host) receives the row count.  Synchronises.
 * import: replaces the accumulated sum by d_Hraw (symmetric, same meaning) and the row count by n_tokens
 *         (>= 1); like admmq_hessian_reset it may be the first call after admmq_create.  Asynchronous. */
admmq_status admmq_hessian_export(admmq_ctx* ctx, float* d_Hraw_out, long long* h_tokens);
admmq_status admmq_hessian_import(admmq_ctx* ctx, const float* d_Hraw, long long n_tokens);

/* ---- Step 2: damping, diagonal scaling, factorisation.  Synchronises (it reads three scalars of the
 * factorisation back: the mean and two bounds of the spectrum of H~). --------------------------------
 * H = H_raw / N + damp_frac * mean(diag(H_raw / N)) I                         (App. D, damping)
 * s_i = sqrt(H_ii),  H~ = diag(1/s) H diag(1/s)                   (Sec. 3.2; Algorithm 1 lines 1-2)
 * then the one-time factorisation of H~ (Algorithm 1 line 3) and the per-penalty factors for
 * rho[0..T).  rho: HOST array of T penalties, or NULL for rho0 * gamma^t (Sec. 3.6). */
typedef struct {
  size_t struct_size;     /* sizeof(admmq_factor_cfg) */
  double damp_frac;       /* 0.01 in the paper */
  int precondition;       /* 1: diagonal scaling on (paper default); 0: s_i = 1 */
  int kind;               /* admmq_factor_kind; any other value: ADMMQ_ERR_INVALID_ARG */
  int T;                  /* number of ADMM iterations, 1..T_max */
  const double* h_rho;    /* host array [T] or NULL */
  double rho0, gamma;     /* used when h_rho == NULL */
} admmq_factor_cfg;
admmq_status admmq_factor(admmq_ctx* ctx, const admmq_factor_cfg* cfg);

/* ---- Step 3: the ADMM loop (Algorithm 1 lines 4-11; Eq. 7-10). -------------------------------------
 * d_W0: pre-trained weights [d_out][d_in] fp32 (unscaled), only read.
 * Outputs, caller-allocated:
 *   d_codes [d_out][d_in] uint8     codes k of D^(T), 0 <= k <= 2^bits - 1
 *   d_scale, d_zero [d_out][d_in/group] fp32   grid Delta and z0 (inputs when use_caller_grid)
 *   d_Wq [d_out][d_in] fp32 or NULL  W_q = z0 + Delta * k  (Algorithm 1 line 11)
 *   d_resid [T][2] fp32 or NULL      (||W^(t+1) - D^(t+1)||_F, ||D^(t+1) - D^(t)||_F), Theorem 1
 * The grid is the min-max grid of the unscaled weights (Sec. 3.4): asymmetric lo = min, hi = max;
 * symmetric hi = max|w|, lo = -hi; Delta = (hi - lo)/(2^bits - 1), z0 = lo; Delta = 1 for a constant
 * group.  Rounding is to nearest, ties to even, then clamped to the grid's range.
 * Grid refresh: at the listed iterations, until one attempt is accepted, (Delta, z0) are refitted by the same
 * rule on the unscaled projection target (W + V/rho)/s, the target is projected on both grids, and the new grid
 * replaces the old one (in d_scale / d_zero) iff ||D_new - W~||_F^2 <= ||D_old - W~||_F^2 over the whole matrix;
 * the dual update then uses D_new.  Needs a group size >= 2.
 * h_report NULL: nothing is synchronised.  Non-NULL: the call synchronises, fills the report and
 * returns the device status. */
typedef struct {
  size_t struct_size;   /* sizeof(admmq_quant_cfg) */
  int bits;             /* 2..8 */
  int group_size;       /* along d_in; 0 or d_in: one group per output channel */
  int symmetric;        /* 0 asymmetric, 1 symmetric */
  int use_caller_grid;  /* 1: d_scale / d_zero are inputs */
  int n_refresh;        /* grid refresh (Sec. 3.3, App. B): number of iterations at which it is attempted, 0: never */
  const int* h_refresh_iters; /* HOST array [n_refresh] of iteration indices t in [0, T) */
  int clip_points;      /* MSE search for the clipping ratio (Sec. 3.4 "Clipping Heuristics", App. D): number of
                           candidate ratios, 0: plain min-max grid; the paper uses 100.  Ignored with a caller grid. */
  double clip_min_ratio;/* smallest candidate ratio in (0, 1]; the paper uses 0.8.  Candidates are
                           r_i = 1 - (1 - clip_min_ratio) i / (clip_points - 1); each scales both ends of the group's
                           min-max range (symmetric: +-r max|w|), and the candidate with the smallest sum of squared
                           rounding errors of the group is kept (the largest ratio on ties). */
  int fused_epilogue;   /* where the element update of Eq. 8-10 runs.  0 (default): the second product stores
                           W^(t+1) - W_hat' and one row pass does projection, dual update, residual sums and the
                           split of the next right-hand side (the faster of the two as measured on B200).
                           1: inside the second product's epilogue, W never leaves the SM.  Same arithmetic per
                           element, so both settings give the same codes. */
  int wupdate_route;    /* how the W-update of Eq. 7 is evaluated.  1: two products per iteration through the basis
                           of the factorisation, R Q -> row solve -> Q^T (2 p n^2 multiply-adds).  2: the n x n operator
                           (H~/rho + I)^{-1} is formed each iteration (a row solve of n rows and one n^3 product) and
                           applied in one product (n^3 + p n^2): fewer operations when d_out > d_in; needs a context
                           created with d_out_max >= 1.25 d_in, otherwise ADMMQ_ERR_UNSUPPORTED.  0: route 2 when
                           d_out >= 1.5 d_in and the context allows it, else route 1.  Both evaluate the same
                           operator; their results differ by rounding only. */
  int product_planes;   /* operand precision of the W-update products.  The products carry only the part of the
                           W-update that is not c R (c = rho / (mu + rho), mu the mean of the spectrum of H~), whose
                           relative size gamma(rho) = max |mu - lambda| / (lambda + rho) over the spectrum shrinks as the
                           penalty grows.  0: two fp16 planes per operand (about 22 bits) while gamma > 2^-13, one
                           plane (11 bits, a third of the tensor-core work) afterwards, where the rounding of one
                           plane is below the fp32 resolution of the W-update.  2: two planes in every iteration. */
  int wupdate_series;   /* the later iterations' W-update as a truncated series.  With E = (mu I - H~) / (mu + rho) the
                           operator of Eq. 7 is rho (H~ + rho I)^{-1} = c (I - E)^{-1} = c (I + E + E^2 + ...), and
                           ||E|| = max |mu - lambda| / (mu + rho) shrinks as the penalty grows.  0: once ||E|| <= 2^-13
                           (in effect the iterations that run on one plane) the update is evaluated as c R + c R E --
                           ONE product with the fixed operand mu I - H~ instead of two products and a row solve; for
                           2^-13 < ||E|| <= 2^-9 as c R + c R E + c R E^2 -- the first product on two planes, the
                           second (of relative size ||E||^2) on one; and once ||E|| <= 2^-26 as c R alone, without a
                           product.  The dropped terms are below 2^-26 of the
                           right-hand side, under the fp32 resolution of the stored iterate.  1: never (every
                           iteration goes through the factorisation).  Ignored with product_planes = 2 or
                           fused_epilogue = 1, which keep every iteration on the two-plane route through the
                           factorisation. */
} admmq_quant_cfg;
typedef struct {
  double err_before;    /* Tr(E^T H E), E = W_q - W_hat, at entry (local search) / of the ADMM result */
  double err_after;     /* same, at exit (local search only; = err_before for quantize_layer) */
  long long moves;      /* local-search moves applied, all columns */
  int iters_run;        /* ADMM iterations run */
  int capped_columns;   /* columns that hit max_moves_per_col */
  float ms;             /* device time of the call, CUDA events */
  int refreshed_iter;   /* quantize_layer: iteration of the accepted grid refresh, -1: none */
  int one_plane_iters;  /* quantize_layer: iterations whose products ran on one fp16 plane per operand */
  int series_iters;     /* quantize_layer: iterations evaluated as the series with one term of E (one product) */
  int series2_iters;    /* quantize_layer: iterations evaluated as the series with two terms of E (two products) */
  int series0_iters;    /* quantize_layer: iterations evaluated as c R alone (||E|| <= 2^-26: no product) */
} admmq_report;
admmq_status admmq_quantize_layer(admmq_ctx* ctx, const float* d_W0, int d_out,
                                  const admmq_quant_cfg* cfg, unsigned char* d_codes, float* d_scale,
                                  float* d_zero, float* d_Wq, float* d_resid, admmq_report* h_report);

/* One W-update (Eq. 7) from a caller-supplied state, for step-by-step checking:
 * d_codes [d_out][d_in] uint8 defines D = s * (z0 + Delta k); d_V [d_out][d_in] fp32 is the dual in
 * scaled coordinates; d_W_out [d_out][d_in] fp32 receives W^(t+1) (scaled coordinates).  Needs a prior
 * admmq_factor; the penalty may be any rho > 0 (its per-penalty factor is computed on the fly). */
admmq_status admmq_w_update(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                            const unsigned char* d_codes, const float* d_scale, const float* d_zero,
                            const float* d_V, double rho, float* d_W_out);

/* ---- Step 4: local search (Sec. 3.5, Eq. 11 restricted to one perturbed entry). --------------------
 * Every output channel independently: with g = H (W_q - W_hat) (unscaled damped H held by the
 * context), moving entry i by d = +-Delta changes the loss by c = 2 d g_i + d^2 H_ii.  The move of
 * smallest c that keeps the code in range (ties: smallest i, then +Delta first) is applied while
 * c < -accept_tol * H_ii * Delta^2, then g += d H[:, i].  Codes (and d_Wq if non-NULL) are updated in
 * place.  Returns ADMMQ_WARN_MOVE_CAP (a success) through the report path if a column hit the cap. */
typedef struct {
  size_t struct_size;           /* sizeof(admmq_ls_cfg) */
  int bits;
  int group_size;
  long long max_moves_per_col;  /* 0: 8 * d_in */
  double accept_tol;            /* relative threshold tau; the paper gives none, 1e-6 by default */
} admmq_ls_cfg;
admmq_status admmq_local_search(admmq_ctx* ctx, const float* d_W0, int d_out, const admmq_ls_cfg* cfg,
                                unsigned char* d_codes, const float* d_scale, const float* d_zero,
                                float* d_Wq, admmq_report* h_report);

/* ---- Pair-swap refinement (Sec. 3.5 "Algorithm"; Eq. 11 with both perturbations). --------------------
 * cfg->d_pairs: DEVICE array [rounds][batch][2] of row indices in [0, d_in): the candidate row pairs of
 * every round, drawn by the caller (entries with equal or out-of-range indices are ignored).  Per round,
 * with g = H (W_q - W_hat): for a pair (i1, i2) every output channel finds the best of the four sign
 * combinations d1 = +-Delta, d2 = +-Delta that keep both codes in range,
 *   c = 2 d1 g_i1 + d1^2 H_i1i1 + 2 d2 g_i2 + d2^2 H_i2i2 + 2 d1 d2 H_i1i2
 * (order (+,+), (+,-), (-,+), (-,-), first minimum), and takes part if
 * c < -accept_tol (d1^2 H_i1i1 + d2^2 H_i2i2).  The pair with the smallest sum of c over the channels that
 * take part (first in the batch on ties; none if no sum is negative) is applied in those channels, then
 * g += d1 H[:, i1] + d2 H[:, i2].  One pair per round, as the paper's step (iv); the paper runs at most 5
 * rounds.  Codes (and d_Wq if non-NULL) are updated in place.  Usually called after admmq_local_search.
 * Report: err_before / err_after as for local search, moves = (pair, channel) moves applied, iters_run =
 * rounds in which a pair was applied. */
typedef struct {
  size_t struct_size;           /* sizeof(admmq_pairswap_cfg) */
  int bits;
  int group_size;
  int rounds;                   /* >= 0 */
  int batch;                    /* candidate pairs per round, 0..65536 */
  const int* d_pairs;           /* device, [rounds][batch][2] */
  double accept_tol;            /* relative threshold tau, 1e-6 by default */
} admmq_pairswap_cfg;
admmq_status admmq_pair_swap(admmq_ctx* ctx, const float* d_W0, int d_out, const admmq_pairswap_cfg* cfg,
                             unsigned char* d_codes, const float* d_scale, const float* d_zero,
                             float* d_Wq, admmq_report* h_report);

/* Tr(E^T H E) with E = (z0 + Delta k) - W_hat and the unscaled damped H (Eq. 2 without the 1/2, as in
 * Sec. 3.5).  Synchronises; the value is written to *h_err (host). */
admmq_status admmq_objective(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                             const unsigned char* d_codes, const float* d_scale, const float* d_zero,
                             double* h_err);

/* Copies of internal state for checking (synchronise).  d_H_out [d_in][d_in] fp32: the damped unscaled
 * H; d_s_out [d_in] fp32: s_i = sqrt(H_ii) (1 when preconditioning is off).  Either may be NULL. */
admmq_status admmq_get_hessian(admmq_ctx* ctx, float* d_H_out, float* d_s_out);

/* The one-time factorisation H~ = Q T Q^T (Algorithm 1 line 3 in its tridiagonal form), for checking
 * (synchronises).  d_QT_out [d_in][d_in] fp64: Q^T, row m = m-th basis vector; d_diag_out [d_in] and
 * d_offdiag_out [d_in] fp64: diagonal of T and its off-diagonal (entry i couples i and i+1; the last is 0).
 * Any of them may be NULL. */
admmq_status admmq_get_factor(admmq_ctx* ctx, double* d_QT_out, double* d_diag_out, double* d_offdiag_out);

/* Number of kernels this context has launched so far (host counter). */
long long admmq_launch_count(const admmq_ctx* ctx);

/* Per-kernel device timing for measurement.  With timing on, the library brackets each launch of the
 * kinds below with CUDA events on its stream.  admmq_get_timing synchronises, adds up the elapsed time
 * and the number of launches of one kind since the last admmq_reset_timing, and keeps the records. */
typedef enum {
  ADMMQ_T_HESSIAN_PRODUCT = 0,  /* X^T X product kernel                                   (step 1) */
  ADMMQ_T_TRANSPOSE = 1,        /* X chunk -> K-major planes                              (step 1) */
  ADMMQ_T_FACTOR = 2,           /* finalisation + tridiagonal reduction + Q + stage factors (step 2) */
  ADMMQ_T_WUPDATE_PRODUCT1 = 3, /* Y = R Q                                                (step 3) */
  ADMMQ_T_TRIDIAG_SOLVE = 4,    /* (T/rho + I)^{-1} row solve                             (step 3) */
  ADMMQ_T_WUPDATE_PRODUCT2 = 5, /* Z = Y' Q^T (with fused_epilogue: plus projection/dual/residuals) (step 3) */
  ADMMQ_T_GRADIENT_PRODUCT = 6, /* g = E H                                                (step 4) */
  ADMMQ_T_LOCAL_SEARCH = 7,     /* move loop kernel                                       (step 4) */
  ADMMQ_T_ROW_SPLIT = 8,        /* row pass: projection, dual update, residuals (unless fused into product 2) and
                                   next right-hand side -> scaled fp16 operand planes     (step 3) */
  ADMMQ_T_WUPDATE_ONE_PLANE = 9, /* either W-update product when it runs on one fp16 plane per operand (step 3) */
  ADMMQ_T_KINDS = 10
} admmq_timing_kind;
admmq_status admmq_set_timing(admmq_ctx* ctx, int on);
admmq_status admmq_reset_timing(admmq_ctx* ctx);
admmq_status admmq_get_timing(admmq_ctx* ctx, int kind, double* h_total_ms, long long* h_count);

/* ---- Error report without a context, a workspace or any allocation. ---------------------------------
 * (The paper has no counterpart: this entry point exists for deployment, not for the method.)
 * Computes Tr(E^T H E), E = (z0 + Delta k) - W_hat, like admmq_objective, for callers that cannot obtain
 * device memory of their own: a job sharing the GPU with an engine that has already claimed all free
 * HBM for its pool, code hosted by a framework that forbids allocations outside its arena, or a thread
 * that must not cause the device-wide synchronisation an allocation may imply.  The caller passes only
 * inputs and the output; the per-channel scratch of the reduction is a fixed array inside the library
 * (ADMMQ_STATIC_MAX_D_OUT doubles = 128 KiB on every GPU that loads the library, until process exit).
 *   d_H [d_in][d_in] fp32  damped unscaled Hessian (e.g. from admmq_get_hessian), symmetric
 *   d_W0, d_codes [d_out][d_in]; d_scale, d_zero [d_out][d_in/group]; d_err: one DEVICE double (output)
 *   cuda_stream: stream to enqueue on (NULL = default).  Asynchronous: read *d_err after the stream
 *   has finished.
 * Limits: d_out <= ADMMQ_STATIC_MAX_D_OUT and d_in <= ADMMQ_MAX_D_IN, otherwise ADMMQ_ERR_SHAPE and
 * nothing is enqueued.  The call makes no cudaMalloc/cudaFree and calls no allocating routine.
 * The scratch is shared by all calls and keeps the last call's contents (each call overwrites the
 * entries it later reads, so nothing needs clearing): calls that overlap on the GPU -- different
 * streams or threads without an ordering between them -- race; serialise them.  The first call on a
 * device also looks up the scratch address and raises the kernel's shared-memory limit; make that first
 * call outside any stream capture.  The device that owns the pointers and the stream must be the
 * current device of the calling thread: the scratch address is looked up for the current device.  With
 * lazy module loading the array and the kernels are placed in device memory at that first call, so a
 * caller that expects a co-tenant to claim the remaining HBM should make it before that happens. */
#define ADMMQ_STATIC_MAX_D_OUT 16384
admmq_status admmq_objective_static(const float* d_H, int d_in, const float* d_W0, int d_out,
                                    int group_size, const unsigned char* d_codes, const float* d_scale,
                                    const float* d_zero, double* d_err, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ADMMQ_H_ */
