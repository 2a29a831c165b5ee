// extern "C" entry points of libadmmq: argument checks, workspace carve-up and the host-side
// sequencing of the kernels.  All numerical work runs in the CUDA kernels of this library.
#include <math.h>
#include <map>
#include <mutex>
#include <new>
#include <string.h>
#include <utility>
#include <vector>

#include "../../include/admmq.h"
#include "../../include/admmq_testing.h"
#include "internal.h"

using namespace admmq;

namespace admmq {
cudaError_t ensure_dynamic_smem(const void* kernel, int bytes) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, int> done;   // (kernel, device) -> limit already set
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  int& have = done[std::make_pair(kernel, dev)];
  if (have >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) have = bytes;
  return e;
}
}  // namespace admmq

struct admmq_ctx {
  Ctx c;
  double* rho_dev = nullptr;
  long long* d_moves = nullptr;
  int* d_capped = nullptr;
  int slots_cap = 0;
  double rho_adhoc = 0.0;
  // ---- optional per-kernel timing ----
  int timing_on = 0;
  struct Rec { cudaEvent_t a, b; int kind; };
  std::vector<Rec> recs;          // records in use
  std::vector<Rec> pool;          // created events available for reuse
};

namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Carver {
  char* base;
  size_t off = 0;
  template <typename T>
  T* take(size_t count) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

// The explicit-operator route of the W-update needs an n x n fp32 copy of Q (mu I - T) and pays off only for
// layers with clearly more output than input channels.
bool explicit_operator_possible(int n, int p_max) { return (long long)4 * p_max >= (long long)5 * n; }

int slots_cap_for(int n, int p) {
  const int simt = ((p + 63) / 64) * ((n + 63) / 64);
  return simt > 256 ? simt : 256;
}

// Lays the workspace out; with base == nullptr only measures it.
size_t carve(admmq_ctx* a, char* base, int n, int p, int T) {
  Carver cv{base};
  Ctx dummy;
  Ctx& c = a ? a->c : dummy;
  const size_t nn = (size_t)n * n, pn = (size_t)p * n;
  c.status = cv.take<int>(64);
  c.scal = cv.take<double>(32);
  c.fscal = cv.take<float>(16);
  c.rs_R = cv.take<float>((size_t)p);
  c.rs_Y = cv.take<float>((size_t)p);
  long long* moves = cv.take<long long>(8);
  int* capped = cv.take<int>(16);
  double* rho_dev = cv.take<double>((size_t)T + 1);
  c.H_raw = cv.take<float>(nn);
  c.H = cv.take<float>(nn);
  c.s = cv.take<float>(n);
  c.inv_s = cv.take<float>(n);
  c.s64 = cv.take<double>(n);
  c.inv_s64 = cv.take<double>(n);
  c.hdiag = cv.take<float>(n);
  c.A64 = cv.take<double>(nn);
  c.P64 = cv.take<double>(nn);
  c.td = cv.take<double>(n);
  c.te = cv.take<double>(n);
  c.beta = cv.take<double>(n);
  c.pvec = cv.take<double>(n);
  c.stage_l = cv.take<float>((size_t)(T + 1) * stage_factor_stride(n));
  c.stage_invd = cv.take<float>((size_t)(T + 1) * stage_factor_stride(n));
  c.shift_c = cv.take<double>((size_t)T + 1);
  c.Qs32 = explicit_operator_possible(n, p) ? cv.take<float>(nn) : nullptr;
  c.N_hi = cv.take<bf16>(nn);
  c.N_lo = cv.take<bf16>(nn);
  c.series_g = cv.take<float>((size_t)T + 1);
  c.series_f = cv.take<float>((size_t)T + 1);
  c.ps_totals = cv.take<double>(PAIR_BATCH_MAX);
  c.ps_chosen = cv.take<int>(16);
  c.ps_d = cv.take<float>((size_t)2 * p);
  c.trd_ws = cv.take<double>(tridiag_blocked_scratch_doubles(n));
  c.wy_s = cv.take<double>((size_t)((n + 31) / 32) * 1024);
  c.Q_hi = cv.take<bf16>(nn);
  c.Q_lo = cv.take<bf16>(nn);
  c.QT_hi = cv.take<bf16>(nn);
  c.QT_lo = cv.take<bf16>(nn);
  c.H_hi = cv.take<bf16>(nn);
  c.H_lo = cv.take<bf16>(nn);
  c.V = cv.take<float>(pn);
  c.Y = cv.take<float>(pn);
  c.R_hi = cv.take<bf16>(pn);
  c.R_lo = cv.take<bf16>(pn);
  c.Y_hi = cv.take<bf16>(pn);
  c.Y_lo = cv.take<bf16>(pn);
  const int slots = slots_cap_for(n, p);
  c.partials = cv.take<float>((size_t)T * slots * 2);
  c.partial_slots = slots;
  c.XT_hi = cv.take<bf16>((size_t)n * XT_ROWS);
  c.XT_lo = cv.take<bf16>((size_t)n * XT_ROWS);
  if (a) {
    a->rho_dev = rho_dev;
    a->d_moves = moves;
    a->d_capped = capped;
    a->slots_cap = slots;
  }
  return align_up(cv.off, 256);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool sizes_ok(int d_in, int d_out, int T) {
  return d_in >= 8 && d_in <= ADMMQ_MAX_D_IN && (d_in % 8) == 0 && d_out >= 1 && d_out <= (1 << 20) &&
         T >= 1 && T <= 4096;
}

cudaError_t product(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& e) {
  return c->gemm_kind == ADMMQ_GEMM_SIMT ? gemm_simt(c, A, B, M, N, K, e) : gemm_tc(c, A, B, M, N, K, e);
}

// Reads the device status word and clears it: an error is reported once, by the first call that reads
// it, and later calls on the context start from ADMMQ_OK again.
admmq_status read_status(admmq_ctx* a) {
  int st = 0;
  if (cudaStreamSynchronize(a->c.stream) != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (cudaMemcpy(&st, a->c.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (st != 0 && cudaMemsetAsync(a->c.status, 0, sizeof(int), a->c.stream) != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (cudaGetLastError() != cudaSuccess) return ADMMQ_ERR_CUDA;
  return (admmq_status)st;
}

// Brackets a region of launches with events when timing is on.
struct Timed {
  admmq_ctx* a;
  bool live = false;
  admmq_ctx::Rec r{};
  Timed(admmq_ctx* ctx, int kind) : a(ctx) {
    if (!a->timing_on) return;
    if (!a->pool.empty()) {
      r = a->pool.back();
      a->pool.pop_back();
    } else if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) {
      return;
    }
    r.kind = kind;
    live = true;
    cudaEventRecord(r.a, a->c.stream);
  }
  ~Timed() {
    if (!live) return;
    cudaEventRecord(r.b, a->c.stream);
    a->recs.push_back(r);
  }
};

int group_of(int d_in, int gs) { return (gs == 0 || gs == d_in) ? d_in : gs; }

// Operand descriptors: Q, Q^T and H are stored once per factorisation as fp16 planes with a common
// power-of-two scale; R, Y' and E carry one scale per row (output channel).
Planes op_Q(Ctx* c) { return planes_f16(c->Q_hi, c->Q_lo, c->n, nullptr, c->fscal + 0); }
// operand of the first product: planes of [Q (mu I - T)]^T with their own scale (shifted operator, elem.cu)
Planes op_QT(Ctx* c) { return planes_f16(c->QT_hi, c->QT_lo, c->n, nullptr, c->fscal + 3); }
Planes op_H(Ctx* c) { return planes_f16(c->H_hi, c->H_lo, c->n, nullptr, c->fscal + 1); }
Planes op_R(Ctx* c) { return planes_f16(c->R_hi, c->R_lo, c->n, c->rs_R, nullptr); }
Planes op_Y(Ctx* c) { return planes_f16(c->Y_hi, c->Y_lo, c->n, c->rs_Y, nullptr); }

// g = E H with E = W_q - W_hat, into c->Y; E planes go through the R buffers.
cudaError_t gradient(admmq_ctx* a, const float* W0, int p, int gs, const unsigned char* codes,
                     const float* delta, const float* zero) {
  Ctx* c = &a->c;
  launch_error_planes(c, W0, p, gs, codes, delta, zero, c->R_hi, c->R_lo, c->rs_R);
  EpiParams e{};
  e.kind = EPI_STORE;
  e.C = c->Y;
  e.ldc = c->n;
  Timed t(a, ADMMQ_T_GRADIENT_PRODUCT);
  return product(c, op_R(c), op_H(c), p, c->n, c->n, e);
}

}  // namespace

extern "C" {

const char* admmq_status_string(admmq_status s) {
  switch (s) {
    case ADMMQ_OK: return "ok";
    case ADMMQ_ERR_INVALID_ARG: return "invalid argument";
    case ADMMQ_ERR_SHAPE: return "unsupported shape";
    case ADMMQ_ERR_STATE: return "call out of order";
    case ADMMQ_ERR_WORKSPACE: return "workspace too small";
    case ADMMQ_ERR_NOT_SPD: return "Hessian not positive definite";
    case ADMMQ_ERR_NONFINITE: return "non-finite value in the input";
    case ADMMQ_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case ADMMQ_ERR_CUDA: return "CUDA call failed";
    case ADMMQ_ERR_UNSUPPORTED: return "not implemented in this build";
    case ADMMQ_WARN_MOVE_CAP: return "local search stopped at the move cap";
  }
  return "unknown status";
}

size_t admmq_workspace_bytes(int d_in, int d_out_max, int T_max) {
  if (!sizes_ok(d_in, d_out_max, T_max)) return 0;
  return carve(nullptr, nullptr, d_in, d_out_max, T_max);
}

admmq_status admmq_create(admmq_ctx** ctx, int d_in, int d_out_max, int T_max, void* d_workspace,
                          size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !d_workspace) return ADMMQ_ERR_INVALID_ARG;
  *ctx = nullptr;
  if (!sizes_ok(d_in, d_out_max, T_max)) return ADMMQ_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255u) return ADMMQ_ERR_INVALID_ARG;
  if (workspace_bytes < admmq_workspace_bytes(d_in, d_out_max, T_max)) return ADMMQ_ERR_WORKSPACE;
  admmq_ctx* a = new (std::nothrow) admmq_ctx();
  if (!a) return ADMMQ_ERR_CUDA;
  a->c.n = d_in;
  a->c.p_max = d_out_max;
  a->c.T_max = T_max;
  a->c.stream = (cudaStream_t)cuda_stream;
  a->c.ws = (char*)d_workspace;
  a->c.ws_bytes = workspace_bytes;
  carve(a, (char*)d_workspace, d_in, d_out_max, T_max);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
    delete a;
    return ADMMQ_ERR_CUDA;
  }
  a->c.num_sms = sms;
  if (cudaMemsetAsync(a->c.status, 0, 256, a->c.stream) != cudaSuccess) {
    delete a;
    return ADMMQ_ERR_CUDA;
  }
  *ctx = a;
  return ADMMQ_OK;
}

admmq_status admmq_destroy(admmq_ctx* ctx) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  for (auto* v : {&ctx->recs, &ctx->pool})
    for (auto& r : *v) {
      cudaEventDestroy(r.a);
      cudaEventDestroy(r.b);
    }
  delete ctx;
  return ADMMQ_OK;
}

admmq_status admmq_set_gemm_kind(admmq_ctx* ctx, admmq_gemm_kind kind) {
  if (!ctx || (kind != ADMMQ_GEMM_TENSOR && kind != ADMMQ_GEMM_SIMT)) return ADMMQ_ERR_INVALID_ARG;
  ctx->c.gemm_kind = (int)kind;
  return ADMMQ_OK;
}

admmq_status admmq_last_device_status(admmq_ctx* ctx) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  return read_status(ctx);
}

long long admmq_launch_count(const admmq_ctx* ctx) { return ctx ? ctx->c.launches : 0; }

admmq_status admmq_test_set_wait(admmq_ctx* ctx, long long wait_limit_cycles, int hold_loads) {
  if (!ctx || wait_limit_cycles < 1000) return ADMMQ_ERR_INVALID_ARG;
  ctx->c.wait_limit_cycles = wait_limit_cycles;
  ctx->c.hold_loads = hold_loads ? 1 : 0;
  return ADMMQ_OK;
}

admmq_status admmq_hessian_reset(admmq_ctx* ctx) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  launch_zero(c, c->H_raw, (size_t)c->n * c->n * sizeof(float));
  launch_zero(c, c->status, 256);
  c->n_tokens = 0;
  c->state = 1;
  return cudaGetLastError() == cudaSuccess ? ADMMQ_OK : ADMMQ_ERR_CUDA;
}

admmq_status admmq_hessian_accumulate(admmq_ctx* ctx, const void* d_X, admmq_dtype dtype,
                                      long long n_tokens, long long ldx) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  if (dtype != ADMMQ_F32 && dtype != ADMMQ_BF16) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->state != 1) return ADMMQ_ERR_STATE;
  if (n_tokens == 0) return ADMMQ_OK;                    // an empty chunk adds nothing
  if (!d_X || !aligned16(d_X)) return ADMMQ_ERR_INVALID_ARG;
  const size_t esz = dtype == ADMMQ_BF16 ? 2 : 4;
  if (n_tokens < 0 || ldx < c->n || ((size_t)ldx * esz) % 16 != 0) return ADMMQ_ERR_SHAPE;
  const int n = c->n;
  for (long long r0 = 0; r0 < n_tokens; r0 += XT_ROWS) {
    const long long rows = (n_tokens - r0 < XT_ROWS) ? (n_tokens - r0) : XT_ROWS;
    const char* xp = (const char*)d_X + (size_t)r0 * ldx * esz;
    bf16* lo = dtype == ADMMQ_BF16 ? nullptr : c->XT_lo;
    {
      Timed t(ctx, ADMMQ_T_TRANSPOSE);
      launch_transpose_split(c, xp, dtype == ADMMQ_BF16, rows, ldx, n, c->XT_hi, lo, XT_ROWS);
    }
    EpiParams e{};
    e.kind = EPI_ACCUM;
    e.C = c->H_raw;
    e.ldc = n;
    e.lower_only = 1;
    Planes P = planes_bf16(c->XT_hi, lo, XT_ROWS);
    Timed t(ctx, ADMMQ_T_HESSIAN_PRODUCT);
    if (product(c, P, P, n, n, (int)rows, e) != cudaSuccess) return ADMMQ_ERR_CUDA;
  }
  c->n_tokens += n_tokens;
  return cudaGetLastError() == cudaSuccess ? ADMMQ_OK : ADMMQ_ERR_CUDA;
}

admmq_status admmq_hessian_set(admmq_ctx* ctx, const float* d_H) {
  if (!ctx || !d_H || !aligned16(d_H)) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (cudaMemcpyAsync(c->H_raw, d_H, (size_t)c->n * c->n * sizeof(float), cudaMemcpyDeviceToDevice,
                      c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  launch_zero(c, c->status, 256);
  c->n_tokens = 1;
  c->state = 1;
  return ADMMQ_OK;
}

admmq_status admmq_hessian_export(admmq_ctx* ctx, float* d_Hraw_out, long long* h_tokens) {
  if (!ctx || !d_Hraw_out || !h_tokens || !aligned16(d_Hraw_out)) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->state < 1) return ADMMQ_ERR_STATE;
  launch_symmetric_copy(c, d_Hraw_out);
  *h_tokens = c->n_tokens;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess || cudaGetLastError() != cudaSuccess) return ADMMQ_ERR_CUDA;
  return ADMMQ_OK;
}

admmq_status admmq_hessian_import(admmq_ctx* ctx, const float* d_Hraw, long long n_tokens) {
  if (!ctx || !d_Hraw || !aligned16(d_Hraw)) return ADMMQ_ERR_INVALID_ARG;
  if (n_tokens < 1) return ADMMQ_ERR_SHAPE;
  Ctx* c = &ctx->c;
  if (cudaMemcpyAsync(c->H_raw, d_Hraw, (size_t)c->n * c->n * sizeof(float), cudaMemcpyDeviceToDevice,
                      c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  launch_zero(c, c->status, 256);
  c->n_tokens = n_tokens;
  c->state = 1;
  return ADMMQ_OK;
}

admmq_status admmq_factor(admmq_ctx* ctx, const admmq_factor_cfg* cfg) {
  if (!ctx || !cfg || cfg->struct_size != sizeof(admmq_factor_cfg)) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->state < 1 || c->n_tokens < 1) return ADMMQ_ERR_STATE;
  if (cfg->kind != ADMMQ_FACTOR_TRIDIAG) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->T < 1 || cfg->T > c->T_max) return ADMMQ_ERR_SHAPE;
  if (!(cfg->damp_frac >= 0.0) || !isfinite(cfg->damp_frac)) return ADMMQ_ERR_INVALID_ARG;
  for (int t = 0; t < cfg->T; ++t) {
    const double r = cfg->h_rho ? cfg->h_rho[t] : cfg->rho0 * pow(cfg->gamma, (double)t);
    if (!(r > 0.0) || !isfinite(r)) return ADMMQ_ERR_INVALID_ARG;
    c->rho_host[t] = r;
  }
  c->T = cfg->T;
  c->precondition = cfg->precondition ? 1 : 0;
  const int n = c->n;
  Timed tfac(ctx, ADMMQ_T_FACTOR);
  launch_finalize(c, cfg->damp_frac, c->precondition);
  launch_operand_scales(c);
  launch_split_f32(c, c->H, (long long)n * n, c->H_hi, c->H_lo);
  launch_series_operand(c);                                // plane of mu I - H~, before the reduction overwrites H~
  if (tridiag_reduce(c) != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (tridiag_form_qt(c) != cudaSuccess) return ADMMQ_ERR_CUDA;
  launch_split_f64(c, c->P64, n, nullptr, nullptr, c->Q_hi, c->Q_lo);   // planes of Q (second product)
  launch_shifted_qt(c);                                    // planes of [Q (mu I - T)]^T (first product)
  if (cudaMemcpyAsync(ctx->rho_dev, c->rho_host, sizeof(double) * c->T, cudaMemcpyHostToDevice,
                      c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  launch_stage_factors(c, ctx->rho_dev, 0, c->T);
  if (cudaGetLastError() != cudaSuccess) return ADMMQ_ERR_CUDA;
  // Operand precision per iteration.  The products carry only the part of the W-update that is not c R, of
  // relative size gamma(rho) = max over the spectrum of |mu - lambda| / (lambda + rho).  Rounding the four
  // operands to one fp16 plane costs about 2^-11.8 of that part; once gamma <= 2^-13 this is below 2^-24 of the
  // W-update itself, under the rounding of its fp32 storage, and one plane per operand (one MMA per K step
  // instead of three) loses nothing.  The bounds come back from the device here: this call synchronises.
  double spec[3] = {1.0, 0.0, 0.0};
  if (cudaMemcpy(spec, c->scal + 8, sizeof(spec), cudaMemcpyDeviceToHost) != cudaSuccess) return ADMMQ_ERR_CUDA;
  c->mu_host = spec[0];
  c->lam_lo = spec[1] > 0.0 ? spec[1] : 0.0;                // H~ is positive semidefinite
  c->lam_hi = spec[2];
  for (int t = 0; t < c->T; ++t) {
    const double r = c->rho_host[t];
    const double g = fmax(fabs(c->mu_host - c->lam_lo) / (c->lam_lo + r), fabs(c->mu_host - c->lam_hi) / (c->lam_hi + r));
    c->planes_host[t] = (isfinite(g) && g <= 1.0 / 8192.0) ? 1 : 2;
    // truncated series c (I + E) R: ||E|| = max |mu - lambda| / (mu + rho); its remainder is below ||E||^2 of R
    const double e = fmax(fabs(c->mu_host - c->lam_lo), fabs(c->mu_host - c->lam_hi)) / (c->mu_host + r);
    // one term of E (one plane) once ||E|| <= 2^-13; two terms -- the first on two planes, the second, of relative
    // size ||E||^2, on one -- once ||E|| <= 2^-9 (remainder below ||E||^3 <= 2^-27)
    c->series_host[t] = !isfinite(e) ? 0 : (c->planes_host[t] == 1 && e <= 1.0 / 8192.0) ? 1 : (e <= 1.0 / 512.0 ? 2 : 0);
    // ... and no term at all once ||E|| itself is below 2^-26: the W-update is c R to the same accuracy
    if (c->series_host[t] == 1 && e <= 1.0 / 67108864.0) c->series_host[t] = 3;
  }
  c->state = 2;
  return ADMMQ_OK;
}

static admmq_status check_layer_args(admmq_ctx* ctx, const float* d_W0, int d_out, int bits, int group_size,
                                     const void* codes, const void* scale, const void* zero) {
  if (!ctx || !d_W0 || !codes || !scale || !zero) return ADMMQ_ERR_INVALID_ARG;
  if (!aligned16(d_W0) || !aligned16(codes) || !aligned16(scale) || !aligned16(zero))
    return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->state != 2) return ADMMQ_ERR_STATE;
  if (d_out < 1 || d_out > c->p_max) return ADMMQ_ERR_SHAPE;
  if (bits < 2 || bits > ADMMQ_MAX_BITS) return ADMMQ_ERR_SHAPE;
  if (group_size < 0 || group_size > c->n) return ADMMQ_ERR_SHAPE;
  const int gs = group_of(c->n, group_size);
  if (c->n % gs != 0) return ADMMQ_ERR_SHAPE;
  return ADMMQ_OK;
}

// One W-update in the error form of Eq. 7:  W - W_hat' = Q (T/rho + I)^{-1} Q^T R,
// R = D - V/rho - W_hat'.  Product 1 -> solve -> product 2 (whose epilogue is `epi`).
// One plane of an operand pair (the hi plane alone: the value rounded to fp16).
static Planes hi_only(Planes P) {
  P.lo = nullptr;
  return P;
}

static cudaError_t w_update_products(admmq_ctx* a, int p, int stage, const EpiParams& epi, int planes) {
  Ctx* c = &a->c;
  const int n = c->n;
  const bool one = planes == 1 && epi.kind == EPI_STORE;   // the fused epilogue exists for two planes only
  EpiParams e1{};
  e1.kind = EPI_STORE;
  e1.C = c->Y;
  e1.ldc = n;
  cudaError_t err;
  {
    Timed t(a, one ? ADMMQ_T_WUPDATE_ONE_PLANE : ADMMQ_T_WUPDATE_PRODUCT1);
    err = one ? product(c, hi_only(op_R(c)), hi_only(op_QT(c)), p, n, n, e1) : product(c, op_R(c), op_QT(c), p, n, n, e1);
  }
  if (err != cudaSuccess) return err;
  {
    Timed t(a, ADMMQ_T_TRIDIAG_SOLVE);
    launch_tridiag_solve(c, c->Y, p, stage, c->Y_hi, c->Y_lo, c->rs_Y);
  }
  Timed t(a, one ? ADMMQ_T_WUPDATE_ONE_PLANE : ADMMQ_T_WUPDATE_PRODUCT2);
  return one ? product(c, hi_only(op_Y(c)), hi_only(op_Q(c)), p, n, n, epi) : product(c, op_Y(c), op_Q(c), p, n, n, epi);
}

// The same W-update with the operator formed explicitly, for layers with more output than input channels:
//   M' = [Q (mu I - T)] (T/rho + I)^{-1} Q^T / (mu + rho)       (n x n: one row solve of n rows + one n^3 product)
//   W - W_hat' - c R = R M'                                      (one p n^2 product)
// n^3 + p n^2 multiply-adds per iteration instead of 2 p n^2.  M' is symmetric (a function of H~), so its rows
// serve as the second product's operand; it takes one power-of-two scale for the whole matrix.
static cudaError_t w_update_explicit(admmq_ctx* a, int p, int stage, const EpiParams& epi, int planes) {
  Ctx* c = &a->c;
  const int n = c->n;
  const bool one = planes == 1 && epi.kind == EPI_STORE;
  {
    Timed t(a, ADMMQ_T_TRIDIAG_SOLVE);
    launch_tridiag_solve(c, c->Qs32, n, stage, c->Y_hi, c->Y_lo, c->rs_Y);
  }
  EpiParams e1{};
  e1.kind = EPI_STORE;
  e1.C = c->Y;
  e1.ldc = n;
  cudaError_t err;
  {
    Timed t(a, ADMMQ_T_WUPDATE_PRODUCT1);
    err = one ? product(c, hi_only(op_Y(c)), hi_only(op_Q(c)), n, n, n, e1) : product(c, op_Y(c), op_Q(c), n, n, n, e1);
  }
  if (err != cudaSuccess) return err;
  {
    Timed t(a, ADMMQ_T_ROW_SPLIT);
    launch_global_split(c, c->Y, (long long)n * n, c->fscal + 6, c->Y_hi, c->Y_lo);
  }
  Timed t(a, one ? ADMMQ_T_WUPDATE_ONE_PLANE : ADMMQ_T_WUPDATE_PRODUCT2);
  const Planes Mp = planes_f16(c->Y_hi, c->Y_lo, n, nullptr, c->fscal + 6);
  return one ? product(c, hi_only(op_R(c)), hi_only(Mp), p, n, n, epi) : product(c, op_R(c), Mp, p, n, n, epi);
}

// The late iterations' W-update as the series c (I + E + ...) truncated after E = (mu I - H~) / (mu + rho):
//   W - W_hat' - c R = c R E = [rho / (mu + rho)^2] R (mu I - H~)
// one p n^2 product of the one-plane right-hand side with the fixed one-plane operand; the dropped terms are
// below gamma(rho)^2 of R.  mu I - H~ is symmetric, so its rows serve as the operand.
static cudaError_t w_update_series(admmq_ctx* a, int p, int stage, const EpiParams& epi) {
  Ctx* c = &a->c;
  const int n = c->n;
  Timed t(a, ADMMQ_T_WUPDATE_ONE_PLANE);
  const Planes Np = planes_f16(c->N_hi, nullptr, n, nullptr, c->series_f + stage);
  return product(c, hi_only(op_R(c)), Np, p, n, n, epi);
}

// Two terms, c R E + c R E^2, for the iterations just before: the first term is the product above on two planes per
// operand (its rounding must stay below 2^-24 / ||E|| of itself), the second -- of relative size ||E||^2 <= 2^-18 --
// a one-plane product of the first with the same operand, added into the stored result.
static cudaError_t w_update_series2(admmq_ctx* a, int p, int stage, const EpiParams& epi) {
  Ctx* c = &a->c;
  const int n = c->n;
  cudaError_t err;
  {
    Timed t(a, ADMMQ_T_WUPDATE_PRODUCT2);
    const Planes Np = planes_f16(c->N_hi, c->N_lo, n, nullptr, c->series_f + stage);
    err = product(c, op_R(c), Np, p, n, n, epi);            // epi.C = c R E
  }
  if (err != cudaSuccess) return err;
  {
    Timed t(a, ADMMQ_T_ROW_SPLIT);
    launch_row_split(c, epi.C, p, c->Y_hi, c->Y_lo, c->rs_Y);
  }
  EpiParams e2 = epi;
  e2.kind = EPI_ACCUM;
  e2.lower_only = 0;
  Timed t(a, ADMMQ_T_WUPDATE_ONE_PLANE);
  const Planes Ng = planes_f16(c->N_hi, nullptr, n, nullptr, c->series_g + stage);
  return product(c, hi_only(op_Y(c)), Ng, p, n, n, e2);     // epi.C += (c R E) E
}

static cudaError_t w_update_any(admmq_ctx* a, int p, int stage, const EpiParams& epi, bool explicit_op, int planes,
                                int series = 0) {
  if (series == 1 && planes == 1 && epi.kind == EPI_STORE) return w_update_series(a, p, stage, epi);
  if (series == 2 && epi.kind == EPI_STORE && epi.ldc == a->c.n) return w_update_series2(a, p, stage, epi);
  return explicit_op ? w_update_explicit(a, p, stage, epi, planes) : w_update_products(a, p, stage, epi, planes);
}

// Two events for the device time of a call; destroyed on every exit path.
struct CallEvents {
  cudaEvent_t a = nullptr, b = nullptr;
  bool create() { return cudaEventCreate(&a) == cudaSuccess && cudaEventCreate(&b) == cudaSuccess; }
  ~CallEvents() {
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
  }
};

admmq_status admmq_quantize_layer(admmq_ctx* ctx, const float* d_W0, int d_out, const admmq_quant_cfg* cfg,
                                  unsigned char* d_codes, float* d_scale, float* d_zero, float* d_Wq,
                                  float* d_resid, admmq_report* h_report) {
  if (!cfg || cfg->struct_size != sizeof(admmq_quant_cfg)) return ADMMQ_ERR_INVALID_ARG;
  admmq_status st = check_layer_args(ctx, d_W0, d_out, cfg->bits, cfg->group_size, d_codes, d_scale, d_zero);
  if (st != ADMMQ_OK) return st;
  if ((d_Wq && !aligned16(d_Wq)) || (d_resid && !aligned16(d_resid))) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->n_refresh < 0 || (cfg->n_refresh > 0 && !cfg->h_refresh_iters)) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->clip_points < 0 || cfg->clip_points > 4096) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->clip_points > 0 && !(cfg->clip_min_ratio > 0.0 && cfg->clip_min_ratio <= 1.0)) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->n_refresh > 0 && group_of(ctx->c.n, cfg->group_size) < 2) return ADMMQ_ERR_UNSUPPORTED;
  if (cfg->wupdate_route < 0 || cfg->wupdate_route > 2) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->product_planes != 0 && cfg->product_planes != 2) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->wupdate_series != 0 && cfg->wupdate_series != 1) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (cfg->wupdate_route == 2 && !c->Qs32) return ADMMQ_ERR_UNSUPPORTED;
  const int n = c->n, p = d_out, gs = group_of(n, cfg->group_size), T = c->T;
  // explicit operator: asked for, or worth it (n^3 + p n^2 against 2 p n^2, plus three small kernels per iteration)
  const bool explicit_op = cfg->wupdate_route == 2 || (cfg->wupdate_route == 0 && c->Qs32 && 2 * p >= 3 * n);
  CallEvents ev;
  if (h_report) {
    if (!ev.create()) return ADMMQ_ERR_CUDA;
    cudaEventRecord(ev.a, c->stream);
  }
  if (!cfg->use_caller_grid) {
    if (cfg->clip_points > 0)
      launch_grid_fit_mse(c, d_W0, p, cfg->bits, gs, cfg->symmetric, cfg->clip_points, cfg->clip_min_ratio,
                          d_scale, d_zero);
    else
      launch_grid_fit(c, d_W0, p, cfg->bits, gs, cfg->symmetric, d_scale, d_zero);
  }
  launch_scale_weights(c, d_W0, p);                        // V = 0, R = 0 (Algorithm 1 l.4)
  launch_zero(c, c->partials, (size_t)T * c->partial_slots * 2 * sizeof(float));
  int* refresh_flags = c->ps_chosen + 4;                   // [0] this attempt accepted, [1] 1 + accepted iteration
  launch_zero(c, c->ps_chosen, 64);
  EpiParams e{};
  e.kind = EPI_ADMM;
  e.W0 = d_W0;
  e.V = c->V;
  e.codes = d_codes;
  e.s = c->s;
  e.inv_s = c->inv_s;
  e.delta = d_scale;
  e.zero = d_zero;
  e.group_size = gs;
  e.n_groups = n / gs;
  e.kmax = (1 << cfg->bits) - 1;
  e.Rnext = c->Y;                                          // Y is free once its planes exist
  int one_plane_iters = 0, series_iters = 0, series2_iters = 0, series0_iters = 0;
  const bool series = cfg->wupdate_series == 0 && !cfg->fused_epilogue && cfg->product_planes != 2;
  auto series_of = [&](int t) { return series ? (int)c->series_host[t] : 0; };
  auto refresh_at = [&](int t) {
    for (int q = 0; q < cfg->n_refresh; ++q)
      if (cfg->h_refresh_iters[q] == t) return true;
    return false;
  };
  // the run's last iterations, if none of them forms a product (or is a refresh attempt), go in one pass
  int t_tail = T;
  while (t_tail > 1 && series_of(t_tail - 1) == 3 && !refresh_at(t_tail - 1)) --t_tail;
  if (T - t_tail < 2) t_tail = T;
  for (int t = 0; t < T; ++t) {
    if (t == t_tail) {
      Timed tt(ctx, ADMMQ_T_ROW_SPLIT);
      launch_admm_tail(c, e, p, ctx->rho_dev, t, T - t, T);
      one_plane_iters += T - t;
      series0_iters += T - t;
      break;
    }
    const double rho = c->rho_host[t];
    const double rho_next = (t + 1 < T) ? c->rho_host[t + 1] : rho;
    e.first_iter = (t == 0);
    e.rho = rho;
    e.inv_rho = 1.0 / rho;
    e.inv_rho_next = 1.0 / rho_next;
    e.partials = c->partials + (size_t)t * c->partial_slots * 2;
    e.shift_c = c->shift_c + t;
    const int planes = (cfg->product_planes == 2 || cfg->fused_epilogue) ? 2 : c->planes_host[t];
    one_plane_iters += planes == 1;
    // terms of E this iteration's W-update keeps (0: through the factorisation)
    int series_t = series_of(t);
    const bool refresh = refresh_at(t);
    if (series_t == 3 && refresh) series_t = 1;             // a refresh attempt wants the product stored
    series_iters += series_t == 1;
    series2_iters += series_t == 2;
    series0_iters += series_t == 3;
    if (refresh) {
      // grid refresh attempt: z = W^(t+1) - W_hat' is stored by the plain epilogue, then evaluated on both grids
      EpiParams w = e;
      w.kind = EPI_STORE;
      w.C = c->Y;
      w.ldc = n;
      if (w_update_any(ctx, p, t, w, explicit_op, planes, series_t) != cudaSuccess) return ADMMQ_ERR_CUDA;
      launch_grid_refresh(c, e, p, cfg->bits, cfg->symmetric, t, d_scale, d_zero, refresh_flags);
      if (t + 1 < T) {
        Timed tt(ctx, ADMMQ_T_ROW_SPLIT);
        launch_row_split(c, c->Y, p, c->R_hi, c->R_lo, c->rs_R);
      }
    } else if (cfg->fused_epilogue) {
      // projection, dual update and residuals inside the second product's epilogue; the next right-hand side
      // leaves it in fp32 and a row pass splits it into planes
      if (w_update_any(ctx, p, t, e, explicit_op, planes) != cudaSuccess) return ADMMQ_ERR_CUDA;
      if (t + 1 < T) {
        Timed tt(ctx, ADMMQ_T_ROW_SPLIT);
        launch_row_split(c, c->Y, p, c->R_hi, c->R_lo, c->rs_R);
      }
    } else {
      // the product stores z = W^(t+1) - W_hat'; one row pass does the element update and the plane split
      EpiParams w = e;
      w.kind = EPI_STORE;
      w.C = c->Y;
      w.ldc = n;
      if (series_t == 3)
        w.C = nullptr;                                       // W^(t+1) - W_hat' = c R: nothing to add in the row pass
      else if (w_update_any(ctx, p, t, w, explicit_op, planes, series_t) != cudaSuccess)
        return ADMMQ_ERR_CUDA;
      Timed tt(ctx, ADMMQ_T_ROW_SPLIT);
      w.kind = EPI_ADMM;
      // the lo plane of the next right-hand side is written only if the next iteration's products read it
      const bool next_two = t + 1 >= T || cfg->product_planes == 2 || series_of(t + 1) == 2 ||
                            (series_of(t + 1) == 0 && c->planes_host[t + 1] != 1);
      // ... and none of its planes when the next iteration forms no product (or there is none): the element update
      // rebuilds R from the codes and the dual
      const bool next_none = t + 1 >= T || (series_of(t + 1) == 3 && !refresh_at(t + 1));
      launch_admm_rows(c, w, p, next_none ? nullptr : c->R_hi, next_two && !next_none ? c->R_lo : nullptr, c->rs_R);
    }
  }
  if (d_resid) launch_reduce_partials(c, T, d_resid);
  if (d_Wq) launch_dequant(c, p, gs, d_codes, d_scale, d_zero, d_Wq);
  if (cudaGetLastError() != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (!h_report) return ADMMQ_OK;
  cudaEventRecord(ev.b, c->stream);
  memset(h_report, 0, sizeof(*h_report));
  if (gradient(ctx, d_W0, p, gs, d_codes, d_scale, d_zero) != cudaSuccess) return ADMMQ_ERR_CUDA;
  launch_objective_dot(c, d_W0, p, gs, d_codes, d_scale, d_zero, c->Y, c->scal + 1);
  st = read_status(ctx);
  double err = 0.0;
  cudaMemcpy(&err, c->scal + 1, sizeof(double), cudaMemcpyDeviceToHost);
  cudaEventElapsedTime(&h_report->ms, ev.a, ev.b);
  int flags[2] = {0, 0};
  cudaMemcpy(flags, refresh_flags, sizeof(flags), cudaMemcpyDeviceToHost);
  h_report->err_before = err;
  h_report->err_after = err;
  h_report->iters_run = T;
  h_report->refreshed_iter = flags[1] - 1;
  h_report->one_plane_iters = one_plane_iters;
  h_report->series_iters = series_iters;
  h_report->series2_iters = series2_iters;
  h_report->series0_iters = series0_iters;
  return st;
}

static admmq_status w_update_call(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                                  const unsigned char* d_codes, const float* d_scale, const float* d_zero,
                                  const float* d_V, double rho, float* d_W_out, int correction_only);

admmq_status admmq_w_update(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                            const unsigned char* d_codes, const float* d_scale, const float* d_zero,
                            const float* d_V, double rho, float* d_W_out) {
  return w_update_call(ctx, d_W0, d_out, group_size, d_codes, d_scale, d_zero, d_V, rho, d_W_out, 0);
}

admmq_status admmq_test_w_update_correction(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                                            const unsigned char* d_codes, const float* d_scale,
                                            const float* d_zero, const float* d_V, double rho, float* d_Z_out) {
  return w_update_call(ctx, d_W0, d_out, group_size, d_codes, d_scale, d_zero, d_V, rho, d_Z_out, 1);
}

admmq_status admmq_test_w_update_series(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                                        const unsigned char* d_codes, const float* d_scale,
                                        const float* d_zero, const float* d_V, double rho, int terms,
                                        float* d_Z_out) {
  if (terms < 0 || terms > 2) return ADMMQ_ERR_INVALID_ARG;
  return w_update_call(ctx, d_W0, d_out, group_size, d_codes, d_scale, d_zero, d_V, rho, d_Z_out, terms == 0 ? 4 : 1 + terms);
}

// correction_only: 0 the whole W-update, 1 the correction W - W_hat', 2 / 3 / 4 the correction by the series with
// one / two / no terms of E
static admmq_status w_update_call(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                                  const unsigned char* d_codes, const float* d_scale, const float* d_zero,
                                  const float* d_V, double rho, float* d_W_out, int correction_only) {
  admmq_status st = check_layer_args(ctx, d_W0, d_out, 2, group_size, d_codes, d_scale, d_zero);
  if (st != ADMMQ_OK) return st;
  if (!d_V || !d_W_out || !aligned16(d_V) || !aligned16(d_W_out)) return ADMMQ_ERR_INVALID_ARG;
  if (!(rho > 0.0) || !isfinite(rho)) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  const int n = c->n, p = d_out, gs = group_of(n, group_size);
  launch_scale_weights(c, d_W0, p);
  launch_init_rhs(c, d_W0, p, gs, d_codes, d_scale, d_zero, d_V, 1.0 / rho, c->Y);
  launch_row_split(c, c->Y, p, c->R_hi, c->R_lo, c->rs_R);
  const int stage = c->T_max;                              // spare slot for an ad-hoc penalty
  ctx->rho_adhoc = rho;
  if (cudaMemcpyAsync(ctx->rho_dev + stage, &ctx->rho_adhoc, sizeof(double), cudaMemcpyHostToDevice,
                      c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  launch_stage_factors(c, ctx->rho_dev, stage, 1);
  EpiParams e{};
  e.kind = EPI_STORE;
  e.C = c->Y;                                               // free once its planes exist
  e.ldc = n;
  const cudaError_t err = correction_only == 2            ? w_update_series(ctx, p, stage, e)
                          : correction_only == 3            ? w_update_series2(ctx, p, stage, e)
                          : correction_only == 4            ? cudaMemsetAsync(c->Y, 0, (size_t)p * n * sizeof(float), c->stream)
                                                            : w_update_products(ctx, p, stage, e, 2);
  if (err != cudaSuccess) return ADMMQ_ERR_CUDA;
  launch_w_out(c, d_W0, p, gs, d_codes, d_scale, d_zero, d_V, 1.0 / rho, c->shift_c + stage, c->Y, d_W_out,
               correction_only != 0);
  return cudaGetLastError() == cudaSuccess ? ADMMQ_OK : ADMMQ_ERR_CUDA;
}

admmq_status admmq_local_search(admmq_ctx* ctx, const float* d_W0, int d_out, const admmq_ls_cfg* cfg,
                                unsigned char* d_codes, const float* d_scale, const float* d_zero,
                                float* d_Wq, admmq_report* h_report) {
  if (!cfg || cfg->struct_size != sizeof(admmq_ls_cfg)) return ADMMQ_ERR_INVALID_ARG;
  admmq_status st = check_layer_args(ctx, d_W0, d_out, cfg->bits, cfg->group_size, d_codes, d_scale, d_zero);
  if (st != ADMMQ_OK) return st;
  if (d_Wq && !aligned16(d_Wq)) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->max_moves_per_col < 0 || !(cfg->accept_tol >= 0.0)) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  const int n = c->n, p = d_out, gs = group_of(n, cfg->group_size);
  const long long cap = cfg->max_moves_per_col > 0 ? cfg->max_moves_per_col : 8LL * n;
  CallEvents ev;
  if (h_report) {
    if (!ev.create()) return ADMMQ_ERR_CUDA;
    cudaEventRecord(ev.a, c->stream);
  }
  if (gradient(ctx, d_W0, p, gs, d_codes, d_scale, d_zero) != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (h_report) launch_objective_dot(c, d_W0, p, gs, d_codes, d_scale, d_zero, c->Y, c->scal + 1);
  launch_zero(c, ctx->d_moves, 64);
  launch_zero(c, ctx->d_capped, 64);
  {
    Timed t(ctx, ADMMQ_T_LOCAL_SEARCH);
    if (launch_local_search(c, d_W0, p, cfg->bits, gs, cap, (float)cfg->accept_tol, d_codes, d_scale,
                            d_zero, d_Wq, c->Y, ctx->d_moves, ctx->d_capped) != cudaSuccess)
      return ADMMQ_ERR_CUDA;
  }
  if (!h_report) return ADMMQ_OK;
  cudaEventRecord(ev.b, c->stream);
  memset(h_report, 0, sizeof(*h_report));
  if (gradient(ctx, d_W0, p, gs, d_codes, d_scale, d_zero) != cudaSuccess) return ADMMQ_ERR_CUDA;
  launch_objective_dot(c, d_W0, p, gs, d_codes, d_scale, d_zero, c->Y, c->scal + 2);
  st = read_status(ctx);
  double errs[2] = {0, 0};
  long long moves = 0;
  int capped = 0;
  cudaMemcpy(errs, c->scal + 1, 2 * sizeof(double), cudaMemcpyDeviceToHost);
  cudaMemcpy(&moves, ctx->d_moves, sizeof(long long), cudaMemcpyDeviceToHost);
  cudaMemcpy(&capped, ctx->d_capped, sizeof(int), cudaMemcpyDeviceToHost);
  cudaEventElapsedTime(&h_report->ms, ev.a, ev.b);
  h_report->err_before = errs[0];
  h_report->err_after = errs[1];
  h_report->moves = moves;
  h_report->capped_columns = capped;
  if (st == ADMMQ_OK && capped > 0) st = ADMMQ_WARN_MOVE_CAP;
  return st;
}

admmq_status admmq_pair_swap(admmq_ctx* ctx, const float* d_W0, int d_out, const admmq_pairswap_cfg* cfg,
                             unsigned char* d_codes, const float* d_scale, const float* d_zero, float* d_Wq,
                             admmq_report* h_report) {
  if (!cfg || cfg->struct_size != sizeof(admmq_pairswap_cfg)) return ADMMQ_ERR_INVALID_ARG;
  admmq_status st = check_layer_args(ctx, d_W0, d_out, cfg->bits, cfg->group_size, d_codes, d_scale, d_zero);
  if (st != ADMMQ_OK) return st;
  if (d_Wq && !aligned16(d_Wq)) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->rounds < 0 || cfg->batch < 0 || !(cfg->accept_tol >= 0.0)) return ADMMQ_ERR_INVALID_ARG;
  if (cfg->batch > PAIR_BATCH_MAX) return ADMMQ_ERR_SHAPE;
  if (cfg->rounds > 0 && cfg->batch > 0 && (!cfg->d_pairs || !aligned16(cfg->d_pairs))) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  const int n = c->n, p = d_out, gs = group_of(n, cfg->group_size);
  CallEvents ev;
  if (h_report) {
    if (!ev.create()) return ADMMQ_ERR_CUDA;
    cudaEventRecord(ev.a, c->stream);
  }
  if (gradient(ctx, d_W0, p, gs, d_codes, d_scale, d_zero) != cudaSuccess) return ADMMQ_ERR_CUDA;
  if (h_report) launch_objective_dot(c, d_W0, p, gs, d_codes, d_scale, d_zero, c->Y, c->scal + 1);
  launch_zero(c, ctx->d_moves, 64);
  launch_zero(c, ctx->d_capped, 64);
  for (int r = 0; r < cfg->rounds && cfg->batch > 0; ++r)
    if (launch_pair_round(c, p, cfg->bits, gs, (float)cfg->accept_tol, d_codes, d_scale, d_zero, d_Wq, c->Y,
                          cfg->d_pairs + (size_t)r * cfg->batch * 2, cfg->batch, ctx->d_moves,
                          ctx->d_capped) != cudaSuccess)
      return ADMMQ_ERR_CUDA;
  if (!h_report) return ADMMQ_OK;
  cudaEventRecord(ev.b, c->stream);
  memset(h_report, 0, sizeof(*h_report));
  if (gradient(ctx, d_W0, p, gs, d_codes, d_scale, d_zero) != cudaSuccess) return ADMMQ_ERR_CUDA;
  launch_objective_dot(c, d_W0, p, gs, d_codes, d_scale, d_zero, c->Y, c->scal + 2);
  st = read_status(ctx);
  double errs[2] = {0, 0};
  long long moves = 0;
  int rounds_applied = 0;
  cudaMemcpy(errs, c->scal + 1, 2 * sizeof(double), cudaMemcpyDeviceToHost);
  cudaMemcpy(&moves, ctx->d_moves, sizeof(long long), cudaMemcpyDeviceToHost);
  cudaMemcpy(&rounds_applied, ctx->d_capped, sizeof(int), cudaMemcpyDeviceToHost);
  cudaEventElapsedTime(&h_report->ms, ev.a, ev.b);
  h_report->err_before = errs[0];
  h_report->err_after = errs[1];
  h_report->moves = moves;
  h_report->iters_run = rounds_applied;
  return st;
}

admmq_status admmq_objective(admmq_ctx* ctx, const float* d_W0, int d_out, int group_size,
                             const unsigned char* d_codes, const float* d_scale, const float* d_zero,
                             double* h_err) {
  admmq_status st = check_layer_args(ctx, d_W0, d_out, 2, group_size, d_codes, d_scale, d_zero);
  if (st != ADMMQ_OK) return st;
  if (!h_err) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  const int gs = group_of(c->n, group_size);
  if (gradient(ctx, d_W0, d_out, gs, d_codes, d_scale, d_zero) != cudaSuccess) return ADMMQ_ERR_CUDA;
  launch_objective_dot(c, d_W0, d_out, gs, d_codes, d_scale, d_zero, c->Y, c->scal + 1);
  st = read_status(ctx);
  if (cudaMemcpy(h_err, c->scal + 1, sizeof(double), cudaMemcpyDeviceToHost) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  return st;
}

admmq_status admmq_set_timing(admmq_ctx* ctx, int on) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  ctx->timing_on = on ? 1 : 0;
  return ADMMQ_OK;
}

admmq_status admmq_reset_timing(admmq_ctx* ctx) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->c.stream) != cudaSuccess) return ADMMQ_ERR_CUDA;
  for (auto& r : ctx->recs) ctx->pool.push_back(r);
  ctx->recs.clear();
  return ADMMQ_OK;
}

admmq_status admmq_get_timing(admmq_ctx* ctx, int kind, double* h_total_ms, long long* h_count) {
  if (!ctx || !h_total_ms || !h_count || kind < 0 || kind >= ADMMQ_T_KINDS) return ADMMQ_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->c.stream) != cudaSuccess) return ADMMQ_ERR_CUDA;
  double total = 0.0;
  long long count = 0;
  for (auto& r : ctx->recs) {
    if (r.kind != kind) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) return ADMMQ_ERR_CUDA;
    total += ms;
    ++count;
  }
  *h_total_ms = total;
  *h_count = count;
  return ADMMQ_OK;
}

admmq_status admmq_get_hessian(admmq_ctx* ctx, float* d_H_out, float* d_s_out) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->state != 2) return ADMMQ_ERR_STATE;
  if (d_H_out && cudaMemcpyAsync(d_H_out, c->H, (size_t)c->n * c->n * sizeof(float),
                                 cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  if (d_s_out && cudaMemcpyAsync(d_s_out, c->s, (size_t)c->n * sizeof(float), cudaMemcpyDeviceToDevice,
                                 c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  return read_status(ctx);
}

admmq_status admmq_get_factor(admmq_ctx* ctx, double* d_QT_out, double* d_diag_out, double* d_offdiag_out) {
  if (!ctx) return ADMMQ_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->state != 2) return ADMMQ_ERR_STATE;
  const size_t n = (size_t)c->n;
  if (d_QT_out && cudaMemcpyAsync(d_QT_out, c->P64, n * n * sizeof(double), cudaMemcpyDeviceToDevice,
                                  c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  if (d_diag_out && cudaMemcpyAsync(d_diag_out, c->td, n * sizeof(double), cudaMemcpyDeviceToDevice,
                                    c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  if (d_offdiag_out && cudaMemcpyAsync(d_offdiag_out, c->te, n * sizeof(double), cudaMemcpyDeviceToDevice,
                                       c->stream) != cudaSuccess)
    return ADMMQ_ERR_CUDA;
  return read_status(ctx);
}

}  // extern "C"
