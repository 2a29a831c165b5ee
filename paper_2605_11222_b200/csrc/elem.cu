// Bandwidth-bound kernels of the ADMM-Q path: layout changes, Hessian finalisation (damping, diagonal
// scaling), grid fit, operand splitting and the small reductions.
#include "internal.h"

namespace admmq {

#define LAUNCH(c) ((c)->launches++)

void launch_zero(Ctx* c, void* ptr, size_t bytes) { cudaMemsetAsync(ptr, 0, bytes, c->stream); }

// ------------------------------------------------------------------------------------------------
// X chunk [rows][ldx] -> X^T planes [n][ldt] (token index contiguous), so that the Hessian product
// H_raw += X^T X contracts over a contiguous index.  fp32 input is split into two bf16 planes.
// ------------------------------------------------------------------------------------------------
template <typename TIn>
__global__ void transpose_split_kernel(const TIn* __restrict__ X, long long rows, long long ldx, int n,
                                       bf16* __restrict__ Thi, bf16* __restrict__ Tlo, long long ldt) {
  __shared__ float tile[32][33];
  const long long r0 = (long long)blockIdx.x * 32;
  const int c0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const long long r = r0 + i;
    const int cc = c0 + threadIdx.x;
    float v = 0.f;
    if (r < rows && cc < n) {
      if constexpr (sizeof(TIn) == 2) v = __bfloat162float(X[r * ldx + cc]);
      else v = X[r * ldx + cc];
    }
    tile[i][threadIdx.x] = v;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int cc = c0 + i;
    const long long r = r0 + threadIdx.x;
    if (cc < n && r < rows) {
      const float v = tile[threadIdx.x][i];
      if (Tlo) {
        bf16 hi, lo;
        split_bf16(v, hi, lo);
        Thi[(long long)cc * ldt + r] = hi;
        Tlo[(long long)cc * ldt + r] = lo;
      } else {
        Thi[(long long)cc * ldt + r] = __float2bfloat16_rn(v);
      }
    }
  }
}

// The bf16 case on 64 x 64 tiles, two elements per thread: every warp access is 128 contiguous bytes on both
// sides (the generic kernel moves 64).  Needs even leading dimensions (4-byte accesses).
__global__ void transpose_bf16_kernel(const bf16* __restrict__ X, long long rows, long long ldx, int n,
                                      bf16* __restrict__ T, long long ldt) {
  __shared__ unsigned short tile[64][66];
  const long long r0 = (long long)blockIdx.x * 64;
  const int c0 = blockIdx.y * 64;
  const int tx = threadIdx.x;
  for (int i = threadIdx.y; i < 64; i += blockDim.y) {
    const long long r = r0 + i;
    const int cc = c0 + 2 * tx;
    unsigned int v = 0u;
    if (r < rows && cc < n) v = *reinterpret_cast<const unsigned int*>(X + r * ldx + cc);   // n is even
    tile[i][2 * tx] = (unsigned short)(v & 0xffffu);
    tile[i][2 * tx + 1] = (unsigned short)(v >> 16);
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 64; i += blockDim.y) {
    const int cc = c0 + i;
    const long long r = r0 + 2 * tx;
    if (cc < n && r < rows) {
      const unsigned int lo = tile[2 * tx][i], hi = tile[2 * tx + 1][i];
      bf16* dst = T + (long long)cc * ldt + r;
      if (r + 1 < rows) *reinterpret_cast<unsigned int*>(dst) = lo | (hi << 16);
      else *reinterpret_cast<unsigned short*>(dst) = (unsigned short)lo;
    }
  }
}

void launch_transpose_split(Ctx* c, const void* X, int is_bf16, long long rows, long long ldx, int n,
                            bf16* XT_hi, bf16* XT_lo, long long ldt) {
  if (is_bf16 && (ldx & 1) == 0 && (ldt & 1) == 0 && (reinterpret_cast<uintptr_t>(X) & 3) == 0) {
    dim3 grid64((unsigned)((rows + 63) / 64), (unsigned)((n + 63) / 64)), block64(32, 8);
    transpose_bf16_kernel<<<grid64, block64, 0, c->stream>>>((const bf16*)X, rows, ldx, n, XT_hi, ldt);
    LAUNCH(c);
    return;
  }
  dim3 grid((unsigned)((rows + 31) / 32), (unsigned)((n + 31) / 32)), block(32, 8);
  if (is_bf16)
    transpose_split_kernel<bf16><<<grid, block, 0, c->stream>>>((const bf16*)X, rows, ldx, n, XT_hi,
                                                                nullptr, ldt);
  else
    transpose_split_kernel<float><<<grid, block, 0, c->stream>>>((const float*)X, rows, ldx, n, XT_hi,
                                                                 XT_lo, ldt);
  LAUNCH(c);
}

// ------------------------------------------------------------------------------------------------
// Finalisation: H = H_raw/N + damp * mean(diag(H_raw/N)) I (App. D), s_i = sqrt(H_ii),
// H~ = diag(1/s) H diag(1/s) in fp64 (Sec. 3.2).  H_raw holds the lower triangle.
// ------------------------------------------------------------------------------------------------
__global__ void diag_sum_kernel(const float* __restrict__ Hraw, int n, double inv_N, double* out) {
  __shared__ double scratch[32];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) acc += (double)Hraw[(long long)i * n + i] * inv_N;
  acc = block_sum(acc, scratch);
  if (threadIdx.x == 0) out[0] = acc;
}

__global__ void finalize_diag_kernel(const float* __restrict__ Hraw, int n, double inv_N,
                                     double damp_frac, int precondition, const double* __restrict__ dsum,
                                     float* __restrict__ hdiag, float* __restrict__ s,
                                     float* __restrict__ inv_s, double* s64, double* inv_s64, int* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const double lam = damp_frac * dsum[0] / n;
  const float hii = (float)((double)Hraw[(long long)i * n + i] * inv_N + lam);
  hdiag[i] = hii;
  if (!(hii > 0.f) || !isfinite(hii)) {
    raise_status(status, isfinite(hii) ? ST_NOT_SPD : ST_NONFINITE);
    s[i] = 1.f;
    inv_s[i] = 1.f;
    s64[i] = 1.0;
    inv_s64[i] = 1.0;
    return;
  }
  const double sv = precondition ? sqrt((double)hii) : 1.0;
  s64[i] = sv;
  inv_s64[i] = 1.0 / sv;
  s[i] = (float)sv;
  inv_s[i] = (float)(1.0 / sv);
}

__global__ void finalize_full_kernel(const float* __restrict__ Hraw, int n, double inv_N,
                                     const float* __restrict__ hdiag, const double* __restrict__ s64,
                                     float* __restrict__ H, double* __restrict__ A64, int* status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  const int a = blockIdx.y;
  if (b >= n) return;
  const int lo = min(a, b), hi = max(a, b);
  float h = (float)((double)Hraw[(long long)hi * n + lo] * inv_N);
  if (a == b) h = hdiag[a];
  if (!isfinite(h)) raise_status(status, ST_NONFINITE);
  H[(long long)a * n + b] = h;
  A64[(long long)a * n + b] = (double)h / (s64[a] * s64[b]);
}

// Full symmetric copy of the accumulator, whose lower triangle is the valid half.
__global__ void symmetric_copy_kernel(const float* __restrict__ Hraw, int n, float* __restrict__ out) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  const int a = blockIdx.y;
  if (b >= n) return;
  const int lo = min(a, b), hi = max(a, b);
  out[(long long)a * n + b] = Hraw[(long long)hi * n + lo];
}

void launch_symmetric_copy(Ctx* c, float* out) {
  dim3 grid((c->n + 255) / 256, c->n);
  symmetric_copy_kernel<<<grid, 256, 0, c->stream>>>(c->H_raw, c->n, out);
  LAUNCH(c);
}

void launch_finalize(Ctx* c, double damp_frac, int precondition) {
  const int n = c->n;
  const double inv_N = 1.0 / (double)c->n_tokens;
  double* s64 = c->s64;
  diag_sum_kernel<<<1, 1024, 0, c->stream>>>(c->H_raw, n, inv_N, c->scal);
  LAUNCH(c);
  finalize_diag_kernel<<<(n + 255) / 256, 256, 0, c->stream>>>(c->H_raw, n, inv_N, damp_frac,
                                                              precondition, c->scal, c->hdiag, c->s,
                                                              c->inv_s, s64, c->inv_s64, c->status);
  LAUNCH(c);
  dim3 grid((n + 255) / 256, n);
  finalize_full_kernel<<<grid, 256, 0, c->stream>>>(c->H_raw, n, inv_N, c->hdiag, s64, c->H, c->A64,
                                                    c->status);
  LAUNCH(c);
}

// ------------------------------------------------------------------------------------------------
// Grid fit (Sec. 3.4: Delta = (max - min)/(2^b - 1); Sec. 3.5: levels z0 + k Delta): one warp per
// (output channel, group) of the unscaled weights.
// ------------------------------------------------------------------------------------------------
__global__ void grid_fit_kernel(const float* __restrict__ W0, int p, int n, int gs, int levels,
                                int symmetric, float* __restrict__ delta, float* __restrict__ zero) {
  const int ng = n / gs;
  const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (gw >= (long long)p * ng) return;
  const int j = (int)(gw / ng), g = (int)(gw % ng);
  const float* w = W0 + (long long)j * n + (long long)g * gs;
  float lo = INFINITY, hi = -INFINITY;
  for (int i = lane; i < gs; i += 32) {
    const float v = w[i];
    lo = fminf(lo, v);
    hi = fmaxf(hi, v);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  if (lane == 0) {
    if (symmetric) {
      hi = fmaxf(fabsf(lo), fabsf(hi));
      lo = -hi;
    }
    float d = (hi - lo) / (float)levels;
    if (hi - lo == 0.f) d = 1.f;
    delta[gw] = d;
    zero[gw] = lo;
  }
}

void launch_grid_fit(Ctx* c, const float* W0, int p, int bits, int gs, int symmetric, float* delta,
                     float* zero) {
  const long long warps = (long long)p * (c->n / gs);
  const int threads = 256;
  const long long blocks = (warps * 32 + threads - 1) / threads;
  grid_fit_kernel<<<(unsigned)blocks, threads, 0, c->stream>>>(W0, p, c->n, gs, (1 << bits) - 1,
                                                                symmetric, delta, zero);
  LAUNCH(c);
}

// Grid fit with an MSE search for the clipping ratio (Sec. 3.4 "Clipping Heuristics"; App. D: 100 grid
// points, maximum shrink ratio 0.8): candidates r_i = 1 - (1 - min_ratio) i / (points - 1) scale both ends
// of the min-max range; the candidate with the smallest sum of squared rounding errors of the group wins
// (strict <, so the largest ratio on ties).  One warp per (output channel, group); a group of up to
// 32 * CLIP_REG values is held in registers, longer ones are re-read (they stay in L1/L2).
constexpr int CLIP_REG = 8;
__global__ void grid_fit_mse_kernel(const float* __restrict__ W0, int p, int n, int gs, int levels,
                                    int symmetric, int points, double min_ratio,
                                    float* __restrict__ delta, float* __restrict__ zero) {
  const int ng = n / gs;
  const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (gw >= (long long)p * ng) return;
  const int j = (int)(gw / ng), g = (int)(gw % ng);
  const float* w = W0 + (long long)j * n + (long long)g * gs;
  const bool in_regs = gs <= 32 * CLIP_REG;
  float wr[CLIP_REG];
  float lo0 = INFINITY, hi0 = -INFINITY;
  if (in_regs) {
#pragma unroll
    for (int q = 0; q < CLIP_REG; ++q) {
      const int i = lane + 32 * q;
      wr[q] = i < gs ? w[i] : NAN;
      if (i < gs) {
        lo0 = fminf(lo0, wr[q]);
        hi0 = fmaxf(hi0, wr[q]);
      }
    }
  } else {
    for (int i = lane; i < gs; i += 32) {
      const float v = w[i];
      lo0 = fminf(lo0, v);
      hi0 = fmaxf(hi0, v);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo0 = fminf(lo0, __shfl_xor_sync(0xffffffffu, lo0, o));
    hi0 = fmaxf(hi0, __shfl_xor_sync(0xffffffffu, hi0, o));
  }
  if (symmetric) {
    hi0 = fmaxf(fabsf(lo0), fabsf(hi0));
    lo0 = -hi0;
  }
  const float fl = (float)levels;
  double best = INFINITY;
  float best_d = 1.f, best_lo = lo0;
  const double step = points > 1 ? (1.0 - min_ratio) / (double)(points - 1) : 0.0;
  for (int c = 0; c < points; ++c) {
    const double r = 1.0 - step * (double)c;
    const float lo = (float)(r * (double)lo0), hi = (float)(r * (double)hi0);
    float d = (hi - lo) / fl;
    if (hi - lo == 0.f) d = 1.f;
    const float inv_d = 1.f / d;
    double acc = 0.0;
    if (in_regs) {
#pragma unroll
      for (int q = 0; q < CLIP_REG; ++q) {
        if (lane + 32 * q < gs) {
          const float k = fminf(fmaxf(rintf((wr[q] - lo) * inv_d), 0.f), fl);
          const float e = fmaf(d, k, lo) - wr[q];
          acc += (double)e * (double)e;
        }
      }
    } else {
      for (int i = lane; i < gs; i += 32) {
        const float v = w[i];
        const float k = fminf(fmaxf(rintf((v - lo) * inv_d), 0.f), fl);
        const float e = fmaf(d, k, lo) - v;
        acc += (double)e * (double)e;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (acc < best) {
      best = acc;
      best_d = d;
      best_lo = lo;
    }
  }
  if (lane == 0) {
    delta[gw] = best_d;
    zero[gw] = best_lo;
  }
}

void launch_grid_fit_mse(Ctx* c, const float* W0, int p, int bits, int gs, int symmetric, int points,
                         double min_ratio, float* delta, float* zero) {
  const long long warps = (long long)p * (c->n / gs);
  const int threads = 128;
  const long long blocks = (warps * 32 + threads - 1) / threads;
  grid_fit_mse_kernel<<<(unsigned)blocks, threads, 0, c->stream>>>(
      W0, p, c->n, gs, (1 << bits) - 1, symmetric, points, min_ratio, delta, zero);
  LAUNCH(c);
}

// Start of a layer: V^(0) = 0 and the first right-hand side R = D^(0) - W_hat' = 0 (all-zero planes, row scale 1;
// Algorithm 1 line 4).  W_hat' = Sigma^{-1} W_hat (line 2) is never stored: every later step works with
// differences from it.  Also the place where non-finite weights are caught.
__global__ void init_state_kernel(const float* __restrict__ W0, long long total, int n, float* __restrict__ V,
                                  bf16* __restrict__ Rhi, bf16* __restrict__ Rlo, float* __restrict__ row_inv,
                                  int* status) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  if (!isfinite(W0[i])) raise_status(status, ST_NONFINITE);
  V[i] = 0.f;
  Rhi[i] = __float2bfloat16_rn(0.f);                      // the all-zero pattern is zero in fp16 as well
  Rlo[i] = __float2bfloat16_rn(0.f);
  if (i % n == 0) row_inv[i / n] = 1.0f;
}

void launch_scale_weights(Ctx* c, const float* W0, int p) {
  const long long total = (long long)p * c->n;
  init_state_kernel<<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(W0, total, c->n, c->V, c->R_hi, c->R_lo,
                                                                          c->rs_R, c->status);
  LAUNCH(c);
}

// ------------------------------------------------------------------------------------------------
// Operand splitting: matrices -> (hi, lo) fp16 planes of the value times a power of two.
// Q has entries of magnitude <= 1 and takes the fixed scale 2^13; H takes the scale that brings its
// largest entry (on the diagonal: H is positive definite) to [2^13, 2^14).
// ------------------------------------------------------------------------------------------------
constexpr float Q_PLANE_SCALE = 8192.0f;

__device__ __forceinline__ void store_f16_pair(bf16* hi, bf16* lo, long long idx, float scaled) {
  __half h, l;
  split_f16(scaled, h, l);
  reinterpret_cast<__half*>(hi)[idx] = h;
  reinterpret_cast<__half*>(lo)[idx] = l;
}

__global__ void operand_scales_kernel(const float* __restrict__ hdiag, int n, float* __restrict__ fscal) {
  __shared__ float scratch[32];
  float m = 0.0f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) m = fmaxf(m, fabsf(hdiag[i]));
  m = block_max(m, scratch);
  if (threadIdx.x == 0) {
    float inv;
    const float sc = pow2_scale_for(m, &inv);
    fscal[0] = 1.0f / Q_PLANE_SCALE;
    fscal[1] = inv;
    fscal[2] = sc;
  }
}

void launch_operand_scales(Ctx* c) {
  operand_scales_kernel<<<1, 1024, 0, c->stream>>>(c->hdiag, c->n, c->fscal);
  LAUNCH(c);
}

__global__ void split_f64_kernel(const double* __restrict__ src, int n, bf16* __restrict__ hi,
                                 bf16* __restrict__ lo, bf16* __restrict__ thi, bf16* __restrict__ tlo) {
  __shared__ float tile[32][33];
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int r = r0 + i, cc = c0 + threadIdx.x;
    float v = 0.f;
    if (r < n && cc < n) {
      v = (float)(src[(long long)r * n + cc] * (double)Q_PLANE_SCALE);
      if (hi) store_f16_pair(hi, lo, (long long)r * n + cc, v);            // planes of src itself: optional
    }
    tile[i][threadIdx.x] = v;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int cc = c0 + i, r = r0 + threadIdx.x;   // element (r, cc) of src -> (cc, r) of the transpose
    if (cc < n && r < n) store_f16_pair(thi, tlo, (long long)cc * n + r, tile[threadIdx.x][i]);
  }
}

void launch_split_f64(Ctx* c, const double* src, int n, bf16* hi, bf16* lo, bf16* thi, bf16* tlo) {
  dim3 grid((n + 31) / 32, (n + 31) / 32), block(32, 8);
  split_f64_kernel<<<grid, block, 0, c->stream>>>(src, n, hi, lo, thi, tlo);
  LAUNCH(c);
}

// ------------------------------------------------------------------------------------------------
// Shifted form of the W-update operator.  With mu = trace(T) / n (= 1 when H~ has unit diagonal) and
// c = rho / (mu + rho),
//     (T/rho + I)^{-1} = c I + (T/rho + I)^{-1} (mu I - T) / (mu + rho),
// so that  Q (T/rho + I)^{-1} Q^T R = c R + Q (T/rho + I)^{-1} [Q (mu I - T)]^T R / (mu + rho).
// The first term is exact and stays in each element's own column; only the second goes through the products,
// whose rounding errors are relative to the whole row of R (a few input channels with a large diagonal scale
// s_i dominate it) -- and that term is small: of relative size |mu - lambda| / (lambda + rho) for an eigenvalue
// lambda of H~, and O(1/rho) for the large penalties of the late iterations.  The operand of the first product
// is therefore row m of  Qs^T = mu P[m] - td[m] P[m] - te[m-1] P[m-1] - te[m] P[m+1]  (P = Q^T), formed in fp64
// and split into fp16 planes with a power-of-two scale of its own; 1 / (mu + rho) is folded into the inverse
// pivots of the per-penalty factor, and the element update adds c R.
// ------------------------------------------------------------------------------------------------
__global__ void shift_mean_kernel(const double* __restrict__ td, int n, double* __restrict__ mu_out,
                                  float* __restrict__ fscal) {
  __shared__ double scratch[32];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) acc += td[i];
  acc = block_sum(acc, scratch);
  if (threadIdx.x == 0) {
    mu_out[0] = acc / (double)n;
    reinterpret_cast<unsigned int*>(fscal)[5] = 0u;        // running maximum of |Qs^T|, as float bits
  }
}

// Gershgorin bounds of the spectrum of T (= that of H~): out[0] <= lambda <= out[1].
__global__ void spectrum_bounds_kernel(const double* __restrict__ td, const double* __restrict__ te, int n,
                                       double* __restrict__ out) {
  __shared__ double scratch[32];
  double lo = INFINITY, hi = -INFINITY;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const double r = fabs(te[i]) + (i > 0 ? fabs(te[i - 1]) : 0.0);
    lo = fmin(lo, td[i] - r);
    hi = fmax(hi, td[i] + r);
  }
  lo = -block_max_f64(-lo, scratch);
  hi = block_max_f64(hi, scratch);
  if (threadIdx.x == 0) {
    out[0] = lo;
    out[1] = hi;
  }
}

__device__ __forceinline__ double shifted_qt_elem(const double* __restrict__ P, const double* __restrict__ td,
                                                  const double* __restrict__ te, double mu, int n, int m, int k) {
  double v = (mu - td[m]) * P[(size_t)m * n + k];
  if (m > 0) v -= te[m - 1] * P[(size_t)(m - 1) * n + k];
  if (m + 1 < n) v -= te[m] * P[(size_t)(m + 1) * n + k];
  return v;
}

__global__ void shifted_qt_max_kernel(const double* __restrict__ P, const double* __restrict__ td,
                                      const double* __restrict__ te, const double* __restrict__ mu_p, int n,
                                      float* __restrict__ fscal) {
  __shared__ float scratch[32];
  const double mu = mu_p[0];
  const int m = blockIdx.x;
  float mx = 0.0f;
  for (int k = threadIdx.x; k < n; k += blockDim.x)
    mx = fmaxf(mx, fabsf((float)shifted_qt_elem(P, td, te, mu, n, m, k)));
  mx = block_max(mx, scratch);
  if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned int*>(fscal) + 5, __float_as_uint(mx));
}

__global__ void shifted_qt_scale_kernel(float* __restrict__ fscal) {
  float inv;
  const float sc = pow2_scale_for(fscal[5], &inv);
  fscal[3] = inv;
  fscal[4] = sc;
}

__global__ void shifted_qt_split_kernel(const double* __restrict__ P, const double* __restrict__ td,
                                        const double* __restrict__ te, const double* __restrict__ mu_p, int n,
                                        const float* __restrict__ fscal, bf16* __restrict__ hi,
                                        bf16* __restrict__ lo) {
  const double mu = mu_p[0];
  const double sc = (double)fscal[4];
  const int m = blockIdx.x;
  for (int k = threadIdx.x; k < n; k += blockDim.x)
    store_f16_pair(hi, lo, (long long)m * n + k, (float)(shifted_qt_elem(P, td, te, mu, n, m, k) * sc));
}

// Q (mu I - T) itself, [k][m] in fp32 (the transpose of what shifted_qt_split_kernel splits): the input of the
// row solve that builds the explicit operator.
__global__ void shifted_q32_kernel(const double* __restrict__ P, const double* __restrict__ td,
                                   const double* __restrict__ te, const double* __restrict__ mu_p, int n,
                                   float* __restrict__ out) {
  __shared__ float tile[32][33];
  const double mu = mu_p[0];
  const int m0 = blockIdx.y * 32, k0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int m = m0 + i, k = k0 + threadIdx.x;
    tile[i][threadIdx.x] = (m < n && k < n) ? (float)shifted_qt_elem(P, td, te, mu, n, m, k) : 0.0f;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int k = k0 + i, m = m0 + threadIdx.x;
    if (k < n && m < n) out[(size_t)k * n + m] = tile[threadIdx.x][i];
  }
}

void launch_shifted_qt(Ctx* c) {
  const int n = c->n;
  shift_mean_kernel<<<1, 1024, 0, c->stream>>>(c->td, n, c->scal + 8, c->fscal);
  spectrum_bounds_kernel<<<1, 1024, 0, c->stream>>>(c->td, c->te, n, c->scal + 9);
  shifted_qt_max_kernel<<<n, 256, 0, c->stream>>>(c->P64, c->td, c->te, c->scal + 8, n, c->fscal);
  shifted_qt_scale_kernel<<<1, 1, 0, c->stream>>>(c->fscal);
  shifted_qt_split_kernel<<<n, 256, 0, c->stream>>>(c->P64, c->td, c->te, c->scal + 8, n, c->fscal, c->QT_hi,
                                                    c->QT_lo);
  c->launches += 5;
  if (c->Qs32) {
    dim3 grid((n + 31) / 32, (n + 31) / 32), block(32, 8);
    shifted_q32_kernel<<<grid, block, 0, c->stream>>>(c->P64, c->td, c->te, c->scal + 8, n, c->Qs32);
    LAUNCH(c);
  }
}

// W^(t+1) = W_hat' + c R + z for the one-step entry point: R = D - V/rho - W_hat' is rebuilt from the caller's
// state as init_rhs_kernel built it, z is the product's output.
__global__ void w_out_kernel(long long total, int n, int gs, int ng, const unsigned char* __restrict__ codes,
                             const float* __restrict__ delta, const float* __restrict__ zero,
                             const float* __restrict__ V, double inv_rho, const double* __restrict__ s,
                             const float* __restrict__ W0, const double* __restrict__ shift_c, const float* __restrict__ z,
                             float* __restrict__ W_out, int correction_only) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int col = (int)(idx % n);
  const long long gi = (idx / n) * ng + col / gs;
  const double e = s[col] * fma((double)delta[gi], (double)codes[idx], (double)zero[gi] - (double)W0[idx]);
  const double r = fma(-(double)V[idx], inv_rho, e);
  const double corr = fma(shift_c[0], r, (double)z[idx]);                     // W^(t+1) - W_hat'
  W_out[idx] = (float)(correction_only ? corr : fma(s[col], (double)W0[idx], corr));
}

void launch_w_out(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes, const float* delta,
                  const float* zero, const float* V_in, double inv_rho, const double* shift_c, const float* z,
                  float* W_out, int correction_only) {
  const long long total = (long long)p * c->n;
  w_out_kernel<<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(
      total, c->n, gs, c->n / gs, codes, delta, zero, V_in, inv_rho, c->s64, W0, shift_c, z, W_out, correction_only);
  LAUNCH(c);
}

__global__ void split_f32_kernel(const float* __restrict__ src, long long count,
                                 const float* __restrict__ fscal, bf16* __restrict__ hi,
                                 bf16* __restrict__ lo) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  store_f16_pair(hi, lo, i, src[i] * fscal[2]);
}

void launch_split_f32(Ctx* c, const float* src, long long count, bf16* hi, bf16* lo) {
  split_f32_kernel<<<(unsigned)((count + 255) / 256), 256, 0, c->stream>>>(src, count, c->fscal, hi, lo);
  LAUNCH(c);
}

// A whole fp32 matrix -> fp16 planes with ONE power-of-two scale (from its largest magnitude): the form an
// operand needs when its rows are the output columns of a product.  slot: three floats, [0] receives 1 / scale,
// [1] the scale, [2] is the running maximum (float bits).
__global__ void absmax_kernel(const float* __restrict__ src, long long count, float* __restrict__ slot) {
  __shared__ float scratch[32];
  float m = 0.0f;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < count;
       i += (long long)gridDim.x * blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(src + i);       // count is a multiple of 4
    m = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(m, fmaxf(fabsf(v.z), fabsf(v.w))));
  }
  m = block_max(m, scratch);
  if (threadIdx.x == 0 && isfinite(m)) atomicMax(reinterpret_cast<unsigned int*>(slot) + 2, __float_as_uint(m));
}
__global__ void scale_from_max_kernel(float* __restrict__ slot) {
  float inv;
  const float sc = pow2_scale_for(slot[2], &inv);
  slot[0] = inv;
  slot[1] = sc;
}
__global__ void split_scaled_kernel(const float* __restrict__ src, long long count, const float* __restrict__ slot,
                                    bf16* __restrict__ hi, bf16* __restrict__ lo) {
  const float sc = slot[1];
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < count;
       i += (long long)gridDim.x * blockDim.x * 8) {
    const float4 a = *reinterpret_cast<const float4*>(src + i), b = *reinterpret_cast<const float4*>(src + i + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    __align__(16) __half hh[8];
    __align__(16) __half ll[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) split_f16(v[e] * sc, hh[e], ll[e]);
    *reinterpret_cast<uint4*>(hi + i) = *reinterpret_cast<const uint4*>(hh);
    *reinterpret_cast<uint4*>(lo + i) = *reinterpret_cast<const uint4*>(ll);
  }
}

// ------------------------------------------------------------------------------------------------
// Operand of the truncated-series W-update: N = mu0 I - H~ as fp16 planes (hi, lo) with a power-of-two scale for
// the whole matrix, mu0 the mean of the diagonal of H~ (1 up to rounding when H~ has been scaled to unit diagonal).
// H~ + rho I = (mu0 + rho) (I - N / (mu0 + rho)), so rho (H~ + rho I)^{-1} = c (I + E + E^2 + ...) with
// E = N / (mu0 + rho); the later iterations keep c R + c R E (+ c R E^2 somewhat earlier).  Read from the fp64 copy of H~ before
// the reduction overwrites it.
// ------------------------------------------------------------------------------------------------
__global__ void series_mean_kernel(const double* __restrict__ A, int n, double* __restrict__ mu_out) {
  __shared__ double scratch[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) s += A[(size_t)i * n + i];
  s = block_sum(s, scratch);
  if (threadIdx.x == 0) mu_out[0] = s / (double)n;
}
__global__ void series_max_kernel(const double* __restrict__ A, int n, const double* __restrict__ mu,
                                  float* __restrict__ slot) {
  __shared__ float scratch[32];
  const int a = blockIdx.x;
  const double m0 = mu[0];
  float m = 0.0f;
  for (int b = threadIdx.x; b < n; b += blockDim.x) {
    const double v = (a == b ? m0 : 0.0) - A[(size_t)a * n + b];
    m = fmaxf(m, fabsf((float)v));
  }
  m = block_max(m, scratch);
  if (threadIdx.x == 0 && isfinite(m)) atomicMax(reinterpret_cast<unsigned int*>(slot) + 2, __float_as_uint(m));
}
__global__ void series_split_kernel(const double* __restrict__ A, int n, const double* __restrict__ mu,
                                    const float* __restrict__ slot, bf16* __restrict__ hi,
                                    bf16* __restrict__ lo) {
  const int a = blockIdx.x;
  const double m0 = mu[0], sc = (double)slot[1];
  __half* oh = reinterpret_cast<__half*>(hi) + (size_t)a * n;
  __half* ol = reinterpret_cast<__half*>(lo) + (size_t)a * n;
  for (int b = threadIdx.x; b < n; b += blockDim.x) {
    const double v = ((a == b ? m0 : 0.0) - A[(size_t)a * n + b]) * sc;
    split_f16((float)v, oh[b], ol[b]);
  }
}

void launch_series_operand(Ctx* c) {
  const int n = c->n;
  float* slot = c->fscal + 9;
  cudaMemsetAsync(slot + 2, 0, sizeof(float), c->stream);
  series_mean_kernel<<<1, 1024, 0, c->stream>>>(c->A64, n, c->scal + 11);
  series_max_kernel<<<n, 256, 0, c->stream>>>(c->A64, n, c->scal + 11, slot);
  scale_from_max_kernel<<<1, 1, 0, c->stream>>>(slot);
  series_split_kernel<<<n, 256, 0, c->stream>>>(c->A64, n, c->scal + 11, slot, c->N_hi, c->N_lo);
  c->launches += 4;
}

void launch_global_split(Ctx* c, const float* src, long long count, float* slot, bf16* hi, bf16* lo) {
  cudaMemsetAsync(slot + 2, 0, sizeof(float), c->stream);
  const int blocks = c->num_sms * 8;
  absmax_kernel<<<blocks, 256, 0, c->stream>>>(src, count, slot);
  scale_from_max_kernel<<<1, 1, 0, c->stream>>>(slot);
  split_scaled_kernel<<<blocks, 256, 0, c->stream>>>(src, count, slot, hi, lo);
  c->launches += 3;
}

// ------------------------------------------------------------------------------------------------
// Row pass: one fp32 row -> its largest magnitude -> power-of-two scale -> (hi, lo) fp16 planes and
// the inverse scale.  One CTA per row at a time, the row staged in shared memory.  `make` yields
// element i of row j.
// ------------------------------------------------------------------------------------------------
constexpr int ROW_THREADS = 256;

template <typename Make>
__device__ __forceinline__ void row_split_body(int p, int n, Make make, bf16* __restrict__ hi,
                                               bf16* __restrict__ lo, float* __restrict__ row_inv) {
  extern __shared__ float rowbuf[];
  __shared__ float scratch[32];
  for (int j = blockIdx.x; j < p; j += gridDim.x) {
    float m = 0.0f;
    for (int i = threadIdx.x * 4; i < n; i += ROW_THREADS * 4) {          // n is a multiple of 8
      const float4 v = make(j, i);
      *reinterpret_cast<float4*>(rowbuf + i) = v;
      m = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(m, fmaxf(fabsf(v.z), fabsf(v.w))));
    }
    m = block_max(m, scratch);
    float inv;
    const float sc = pow2_scale_for(m, &inv);
    if (threadIdx.x == 0) row_inv[j] = inv;
    for (int i = threadIdx.x * 8; i < n; i += ROW_THREADS * 8) {
      __align__(16) __half hh[8];
      __align__(16) __half ll[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) split_f16(rowbuf[i + e] * sc, hh[e], ll[e]);
      *reinterpret_cast<uint4*>(hi + (size_t)j * n + i) = *reinterpret_cast<const uint4*>(hh);
      *reinterpret_cast<uint4*>(lo + (size_t)j * n + i) = *reinterpret_cast<const uint4*>(ll);
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(ROW_THREADS)
row_split_kernel(const float* __restrict__ src, int p, int n, bf16* __restrict__ hi, bf16* __restrict__ lo,
                 float* __restrict__ row_inv) {
  row_split_body(p, n, [&](int j, int i) { return *reinterpret_cast<const float4*>(src + (size_t)j * n + i); },
                 hi, lo, row_inv);
}

static int row_pass_blocks(Ctx* c, int p, size_t smem) {
  int per_sm = (int)((200 * 1024) / (smem + 1024));
  if (per_sm > 8) per_sm = 8;
  if (per_sm < 1) per_sm = 1;
  const int blocks = c->num_sms * per_sm;
  return blocks < p ? blocks : p;
}

void launch_row_split(Ctx* c, const float* src, int p, bf16* hi, bf16* lo, float* row_inv) {
  const size_t smem = (size_t)c->n * sizeof(float);
  if (ensure_dynamic_smem((const void*)row_split_kernel, 64 * 1024) != cudaSuccess) return;   // the launch error check reports it
  row_split_kernel<<<row_pass_blocks(c, p, smem), ROW_THREADS, smem, c->stream>>>(src, p, c->n, hi, lo, row_inv);
  LAUNCH(c);
}

// Right-hand side of the error-form W-update from a caller-supplied state:
// R = D - V/rho - W_hat', D = s (z0 + Delta k).
__global__ void init_rhs_kernel(long long total, int n, int gs, int ng,
                                const unsigned char* __restrict__ codes,
                                const float* __restrict__ delta, const float* __restrict__ zero,
                                const float* __restrict__ V, double inv_rho, const double* __restrict__ s,
                                const float* __restrict__ W0, float* __restrict__ R) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int col = (int)(idx % n);
  const long long row = idx / n;
  const long long gi = row * ng + col / gs;
  // D - W_hat' = s (z0 + Delta k - w_hat): the difference of weight-sized numbers is taken in fp64
  const double e = s[col] * fma((double)delta[gi], (double)codes[idx], (double)zero[gi] - (double)W0[idx]);
  R[idx] = (float)fma(-(double)V[idx], inv_rho, e);
}

void launch_init_rhs(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes, const float* delta,
                     const float* zero, const float* V_in, double inv_rho, float* R_out) {
  const long long total = (long long)p * c->n;
  init_rhs_kernel<<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(
      total, c->n, gs, c->n / gs, codes, delta, zero, V_in, inv_rho, c->s64, W0, R_out);
  LAUNCH(c);
}

// Fixed-order second stage of the residual sums: resid[t] = (sqrt(sum (W-D)^2), sqrt(sum (D-D_old)^2)).
__global__ void reduce_partials_kernel(const float* __restrict__ partials, int slots, int T,
                                       float* __restrict__ resid) {
  __shared__ double scratch[32];
  const int t = blockIdx.x;
  if (t >= T) return;
  double a = 0.0, b = 0.0;
  for (int i = threadIdx.x; i < slots; i += blockDim.x) {
    a += (double)partials[((long long)t * slots + i) * 2 + 0];
    b += (double)partials[((long long)t * slots + i) * 2 + 1];
  }
  a = block_sum(a, scratch);
  b = block_sum(b, scratch);
  if (threadIdx.x == 0) {
    resid[2 * t + 0] = (float)sqrt(a);
    resid[2 * t + 1] = (float)sqrt(b);
  }
}

void launch_reduce_partials(Ctx* c, int T, float* resid) {
  reduce_partials_kernel<<<T, 128, 0, c->stream>>>(c->partials, c->partial_slots, T, resid);
  LAUNCH(c);
}

// W_q = z0 + Delta k (Algorithm 1 line 11, unscaled coordinates).
__global__ void dequant_kernel(long long total, int n, int gs, int ng,
                               const unsigned char* __restrict__ codes, const float* __restrict__ delta,
                               const float* __restrict__ zero, float* __restrict__ Wq) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const long long gi = (idx / n) * ng + (idx % n) / gs;
  Wq[idx] = zero[gi] + delta[gi] * (float)codes[idx];
}

void launch_dequant(Ctx* c, int p, int gs, const unsigned char* codes, const float* delta,
                    const float* zero, float* Wq) {
  const long long total = (long long)p * c->n;
  dequant_kernel<<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(total, c->n, gs, c->n / gs,
                                                                         codes, delta, zero, Wq);
  LAUNCH(c);
}

// E = W_q - W_hat as two bf16 planes (operand of the gradient product g = E H, Sec. 3.5).
__global__ void __launch_bounds__(ROW_THREADS)
error_planes_kernel(int p, int n, int gs, int ng, const float* __restrict__ W0,
                    const unsigned char* __restrict__ codes, const float* __restrict__ delta,
                    const float* __restrict__ zero, bf16* __restrict__ Ehi, bf16* __restrict__ Elo,
                    float* __restrict__ row_inv) {
  row_split_body(p, n,
                 [&](int j, int i) {
                   const size_t idx = (size_t)j * n + i;
                   const float4 w = *reinterpret_cast<const float4*>(W0 + idx);
                   const uchar4 k = *reinterpret_cast<const uchar4*>(codes + idx);
                   float4 e;
                   size_t gi = (size_t)j * ng + i / gs;
                   e.x = (zero[gi] + delta[gi] * (float)k.x) - w.x;
                   gi = (size_t)j * ng + (i + 1) / gs;
                   e.y = (zero[gi] + delta[gi] * (float)k.y) - w.y;
                   gi = (size_t)j * ng + (i + 2) / gs;
                   e.z = (zero[gi] + delta[gi] * (float)k.z) - w.z;
                   gi = (size_t)j * ng + (i + 3) / gs;
                   e.w = (zero[gi] + delta[gi] * (float)k.w) - w.w;
                   return e;
                 },
                 Ehi, Elo, row_inv);
}

void launch_error_planes(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes,
                         const float* delta, const float* zero, bf16* Ehi, bf16* Elo, float* row_inv) {
  const size_t smem = (size_t)c->n * sizeof(float);
  if (ensure_dynamic_smem((const void*)error_planes_kernel, 64 * 1024) != cudaSuccess) return;   // the launch error check reports it
  error_planes_kernel<<<row_pass_blocks(c, p, smem), ROW_THREADS, smem, c->stream>>>(
      p, c->n, gs, c->n / gs, W0, codes, delta, zero, Ehi, Elo, row_inv);
  LAUNCH(c);
}

// ------------------------------------------------------------------------------------------------
// Grid refresh (Sec. 3.3 "Grid refresh", App. B) at one iteration, from the stored product z = W^(t+1) - W_hat':
//   eval:   per (channel, group) refit (Delta', z0') on the unscaled target Sigma W~ = w_hat + (z + V/rho)/s by
//           the initial fitting rule, project the target on the old and on the new grid, sum both squared distances;
//   decide: new grid kept iff its sum <= the old one (Eq. of App. B) and no refresh was accepted before;
//   apply:  the ADMM element update (projection, dual, residual sums, next right-hand side) with the grid
//           that was kept.  Same arithmetic as the row pass: targets and grid points relative to the weight,
//           weight-sized differences and the rounding decisions in fp64.
// ------------------------------------------------------------------------------------------------
// (W~ - W_hat') / s of one element: the product's output plus its c R part (R rebuilt from the codes and the dual
// as in the element update), plus V/rho.
__device__ __forceinline__ double refresh_target(float zp, float w0, float v, int code_old, int first_iter, float s,
                                                 float inv_s, float dl, float z0, float cshift, float inv_rho) {
  float a_hi, a_lo;
  diff_exact(w0, z0, a_hi, a_lo);
  const float e_old = first_iter ? 0.0f : grid_offset(s, dl, (float)code_old, a_hi, a_lo);
  const float z = fmaf(cshift, fmaf(-v, inv_rho, e_old), zp);
  return (double)(fmaf(v, inv_rho, z) * inv_s);           // the same fp32 steps as the element update
}

__global__ void __launch_bounds__(256)
refresh_eval_kernel(const float* __restrict__ Zc, const float* __restrict__ W0, const float* __restrict__ V,
                    const unsigned char* __restrict__ codes, int first_iter, const double* __restrict__ shift_c,
                    const float* __restrict__ s, const float* __restrict__ inv_s, int p, int n, int gs, int kmax,
                    int symmetric, double inv_rho, const float* __restrict__ delta, const float* __restrict__ zero,
                    float* __restrict__ cand_delta, float* __restrict__ cand_zero, double* __restrict__ partial) {
  __shared__ double scratch[32];
  const int ng = n / gs, lane = threadIdx.x & 31;
  const long long groups = (long long)p * ng;
  const float cs = (float)shift_c[0];
  const float inv_rho_f = (float)inv_rho;
  double e_old = 0.0, e_new = 0.0;
  for (long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; gw < groups;
       gw += ((long long)gridDim.x * blockDim.x) >> 5) {
    const int j = (int)(gw / ng), gq = (int)(gw % ng);
    const size_t base = (size_t)j * n + (size_t)gq * gs;
    const float d0 = delta[gw], z0 = zero[gw];
    double lo = INFINITY, hi = -INFINITY;
    for (int i = lane; i < gs; i += 32) {
      const double u = refresh_target(Zc[base + i], W0[base + i], V[base + i], first_iter ? 0 : (int)codes[base + i],
                                      first_iter, s[gq * gs + i], inv_s[gq * gs + i], d0, z0, cs, inv_rho_f);
      const double y = (double)W0[base + i] + u;
      lo = fmin(lo, y);
      hi = fmax(hi, y);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (symmetric) {
      hi = fmax(fabs(lo), fabs(hi));
      lo = -hi;
    }
    float dn = (float)((hi - lo) / (double)kmax);          // the grid is stored in fp32
    if (hi - lo == 0.0) dn = 1.f;
    const float zn = (float)lo;
    if (lane == 0) {
      cand_delta[gw] = dn;
      cand_zero[gw] = zn;
    }
    const double id0 = 1.0 / (double)d0, idn = 1.0 / (double)dn;
    double a = 0.0, b = 0.0;
    for (int i = lane; i < gs; i += 32) {
      const double sv = (double)s[gq * gs + i];
      const double u = refresh_target(Zc[base + i], W0[base + i], V[base + i],
                                              first_iter ? 0 : (int)codes[base + i], first_iter, s[gq * gs + i],
                                              inv_s[gq * gs + i], d0, z0, cs, inv_rho_f);
      const double w = (double)W0[base + i];
      const double k0 = fmin(fmax(rint(((w - (double)z0) + u) * id0), 0.0), (double)kmax);
      const double kn = fmin(fmax(rint(((w - (double)zn) + u) * idn), 0.0), (double)kmax);
      // D - W~ in scaled coordinates: s ((z0 + Delta k - w_hat) - u)
      const double eo = sv * (fma((double)d0, k0, (double)z0 - w) - u);
      const double en = sv * (fma((double)dn, kn, (double)zn - w) - u);
      a = fma(eo, eo, a);
      b = fma(en, en, b);
    }
    e_old += warp_sum(a);
    e_new += warp_sum(b);
  }
  e_old = block_sum(e_old, scratch);       // every lane of a warp carries its warp's sums: divide by 32 below
  e_new = block_sum(e_new, scratch);
  if (threadIdx.x == 0) {
    partial[2 * blockIdx.x] = e_old / 32.0;
    partial[2 * blockIdx.x + 1] = e_new / 32.0;
  }
}

// flags[0]: 1 if this attempt is accepted; flags[1]: 1 + iteration of the accepted refresh (0: none so far)
__global__ void refresh_decide_kernel(const double* __restrict__ partial, int blocks, int iter, int* flags) {
  __shared__ double scratch[32];
  double a = 0.0, b = 0.0;
  for (int i = threadIdx.x; i < blocks; i += blockDim.x) {
    a += partial[2 * i];
    b += partial[2 * i + 1];
  }
  a = block_sum(a, scratch);
  b = block_sum(b, scratch);
  if (threadIdx.x == 0) {
    const int ok = (flags[1] == 0 && b <= a) ? 1 : 0;
    flags[0] = ok;
    if (ok) flags[1] = iter + 1;
  }
}

// After this kernel (delta, zero) is the grid in force and (cand_delta, cand_zero) the grid the codes of D^(t)
// refer to: the two are exchanged when the attempt is accepted, and equal otherwise.
__global__ void refresh_commit_kernel(long long groups, const int* __restrict__ flags,
                                      float* __restrict__ cand_delta, float* __restrict__ cand_zero,
                                      float* __restrict__ delta, float* __restrict__ zero) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= groups) return;
  const float d_old = delta[i], z_old = zero[i];
  if (flags[0]) {
    delta[i] = cand_delta[i];
    zero[i] = cand_zero[i];
  }
  cand_delta[i] = d_old;
  cand_zero[i] = z_old;
}

// The ADMM element update from the stored product z = W^(t+1) - W_hat' (in P.Rnext, overwritten by the next
// right-hand side).
__global__ void __launch_bounds__(256) admm_elementwise_kernel(EpiParams P, const float* __restrict__ old_delta,
                                                               const float* __restrict__ old_zero, long long total,
                                                               int n) {
  __shared__ float red[32];
  float r2 = 0.f, s2 = 0.f;
  const float cs = (float)P.shift_c[0];
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int col = (int)(idx % n);
    const long long row = idx / n;
    const long long gi = row * P.n_groups + col / P.group_size;
    AdmmElem e = admm_elem(P.Rnext[idx], P.W0[idx], P.V[idx], P.first_iter ? 0 : (int)P.codes[idx], P.s[col],
                           P.inv_s[col], grid_g(P.delta[gi], P.zero[gi]), grid_g(old_delta[gi], old_zero[gi]), cs, P);
    P.codes[idx] = e.code;
    P.V[idx] = e.v_new;
    P.Rnext[idx] = e.r_next;
    r2 += e.dr2;
    s2 += e.ds2;
  }
  r2 = block_sum(r2, red);
  s2 = block_sum(s2, red);
  if (threadIdx.x == 0) {
    P.partials[2 * blockIdx.x + 0] = r2;
    P.partials[2 * blockIdx.x + 1] = s2;
  }
}

// The ADMM element update (Eq. 8-10) of whole rows from the stored product z = W^(t+1) - W_hat' (in P.C), merged
// with the split of the next right-hand side into its scaled fp16 planes: the row of R = D - V/rho' - W_hat'
// stays in shared memory between the two halves, so it makes no trip through memory of its own.
__global__ void __launch_bounds__(ROW_THREADS)
admm_row_kernel(EpiParams P, int p, int n, bf16* __restrict__ hi, bf16* __restrict__ lo,
                float* __restrict__ row_inv) {
  extern __shared__ float rowbuf[];
  __shared__ float scratch[32];
  float r2 = 0.f, s2 = 0.f;
  const int gs = P.group_size;
  const int gsh = (gs & (gs - 1)) == 0 ? 31 - __clz(gs) : -1;      // group index by shift when the size allows
  const float cs = (float)P.shift_c[0];
  for (int j = blockIdx.x; j < p; j += gridDim.x) {
    const size_t base = (size_t)j * n;
    const float* dlt = P.delta + (size_t)j * P.n_groups;
    const float* zr = P.zero + (size_t)j * P.n_groups;
    float m = 0.0f;
    for (int i = threadIdx.x * 4; i < n; i += ROW_THREADS * 4) {          // n is a multiple of 8
      // P.C == nullptr: the product's part of the W-update is below fp32 resolution and was not formed
      const float4 z = P.C ? *reinterpret_cast<const float4*>(P.C + base + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      const float4 wh = *reinterpret_cast<const float4*>(P.W0 + base + i);
      const float4 v = *reinterpret_cast<const float4*>(P.V + base + i);
      const float4 sv = *reinterpret_cast<const float4*>(P.s + i);
      const float4 si = *reinterpret_cast<const float4*>(P.inv_s + i);
      uchar4 k = make_uchar4(0, 0, 0, 0);
      if (!P.first_iter) k = *reinterpret_cast<const uchar4*>(P.codes + base + i);
      const int g0 = gsh >= 0 ? i >> gsh : i / gs;
      const int g3 = gsh >= 0 ? (i + 3) >> gsh : (i + 3) / gs;
      const GridG gg = grid_g(dlt[g0], zr[g0]);
      AdmmElem e0 = admm_elem(z.x, wh.x, v.x, k.x, sv.x, si.x, gg, gg, cs, P);
      AdmmElem e1, e2, e3;
      if (g3 == g0) {
        e1 = admm_elem(z.y, wh.y, v.y, k.y, sv.y, si.y, gg, gg, cs, P);
        e2 = admm_elem(z.z, wh.z, v.z, k.z, sv.z, si.z, gg, gg, cs, P);
        e3 = admm_elem(z.w, wh.w, v.w, k.w, sv.w, si.w, gg, gg, cs, P);
      } else {
        const int g1 = (i + 1) / gs, g2 = (i + 2) / gs;
        const GridG q1 = grid_g(dlt[g1], zr[g1]), q2 = grid_g(dlt[g2], zr[g2]), q3 = grid_g(dlt[g3], zr[g3]);
        e1 = admm_elem(z.y, wh.y, v.y, k.y, sv.y, si.y, q1, q1, cs, P);
        e2 = admm_elem(z.z, wh.z, v.z, k.z, sv.z, si.z, q2, q2, cs, P);
        e3 = admm_elem(z.w, wh.w, v.w, k.w, sv.w, si.w, q3, q3, cs, P);
      }
      *reinterpret_cast<uchar4*>(P.codes + base + i) = make_uchar4(e0.code, e1.code, e2.code, e3.code);
      *reinterpret_cast<float4*>(P.V + base + i) = make_float4(e0.v_new, e1.v_new, e2.v_new, e3.v_new);
      r2 += (e0.dr2 + e1.dr2) + (e2.dr2 + e3.dr2);
      s2 += (e0.ds2 + e1.ds2) + (e2.ds2 + e3.ds2);
      if (!hi) continue;                                   // no product reads the next right-hand side: no planes
      *reinterpret_cast<float4*>(rowbuf + i) = make_float4(e0.r_next, e1.r_next, e2.r_next, e3.r_next);
      m = fmaxf(fmaxf(fabsf(e0.r_next), fabsf(e1.r_next)), fmaxf(m, fmaxf(fabsf(e2.r_next), fabsf(e3.r_next))));
    }
    if (!hi) continue;                                     // (uniform in the grid)
    m = block_max(m, scratch);
    float inv;
    const float sc = pow2_scale_for(m, &inv);
    if (threadIdx.x == 0) row_inv[j] = inv;
    for (int i = threadIdx.x * 8; i < n; i += ROW_THREADS * 8) {
      __align__(16) __half hh[8];
      __align__(16) __half ll[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) split_f16(rowbuf[i + e] * sc, hh[e], ll[e]);
      *reinterpret_cast<uint4*>(hi + base + i) = *reinterpret_cast<const uint4*>(hh);
      if (lo) *reinterpret_cast<uint4*>(lo + base + i) = *reinterpret_cast<const uint4*>(ll);   // nullptr: one plane
    }
    __syncthreads();
  }
  r2 = block_sum(r2, scratch);
  s2 = block_sum(s2, scratch);
  if (threadIdx.x == 0) {
    P.partials[2 * blockIdx.x + 0] = r2;
    P.partials[2 * blockIdx.x + 1] = s2;
  }
}

// The last iterations of a run, in which no product is formed (||E|| <= 2^-26: W - W_hat' = c R): every element
// then evolves on its own -- R is rebuilt from its code and dual, the update reads nothing else -- so `count`
// iterations starting at `first` run in one pass over the state, the element held in registers throughout.  Same
// arithmetic per element and iteration as admm_row_kernel.  The residual sums of every iteration (Theorem 1) are
// taken per warp in shared memory and written per CTA at the end, in a fixed order.
constexpr int TAIL_MAX = 512;                 // iterations per launch (shared memory: 8 warps x 2 sums each)
__global__ void __launch_bounds__(256)
admm_tail_kernel(EpiParams P, long long total, int n, const double* __restrict__ rho, const double* __restrict__ shift_c,
                 int first, int count, int T, float* __restrict__ partials, int slots) {
  __shared__ float it_rho[TAIL_MAX], it_inv[TAIL_MAX], it_inv_next[TAIL_MAX], it_c[TAIL_MAX];
  __shared__ float wsum[8][TAIL_MAX][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int q = threadIdx.x; q < count; q += blockDim.x) {
    const int t = first + q;
    const double r = rho[t], rn = rho[t + 1 < T ? t + 1 : t];
    it_rho[q] = (float)r;
    it_inv[q] = (float)(1.0 / r);
    it_inv_next[q] = (float)(1.0 / rn);
    it_c[q] = (float)shift_c[t];
  }
  for (int q = threadIdx.x; q < 8 * count; q += blockDim.x) {
    wsum[q / count][q % count][0] = 0.0f;
    wsum[q / count][q % count][1] = 0.0f;
  }
  __syncthreads();
  const int gs = P.group_size;
  // whole warps take part in the butterflies: the loop bound is rounded up to a multiple of the grid's stride
  const long long groups = total / 4, stride = (long long)gridDim.x * blockDim.x;
  for (long long g0 = (long long)blockIdx.x * blockDim.x; g0 < groups; g0 += stride) {
    const long long gq = g0 + threadIdx.x;
    const bool live = gq < groups;
    const long long idx = live ? gq * 4 : 0;
    const int col = (int)(idx % n);
    const long long row = idx / n;
    const float4 w4 = *reinterpret_cast<const float4*>(P.W0 + idx);
    float4 v4 = *reinterpret_cast<const float4*>(P.V + idx);
    const float4 s4 = *reinterpret_cast<const float4*>(P.s + col);
    const float4 i4 = *reinterpret_cast<const float4*>(P.inv_s + col);
    uchar4 k4 = *reinterpret_cast<const uchar4*>(P.codes + idx);
    GridG gg[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const long long gi = row * P.n_groups + (col + e) / gs;
      gg[e] = grid_g(P.delta[gi], P.zero[gi]);
    }
    float w[4] = {w4.x, w4.y, w4.z, w4.w}, v[4] = {v4.x, v4.y, v4.z, v4.w};
    const float sv[4] = {s4.x, s4.y, s4.z, s4.w}, si[4] = {i4.x, i4.y, i4.z, i4.w};
    int k[4] = {k4.x, k4.y, k4.z, k4.w};
    IterF it;
    it.first_iter = 0;
    it.kmax = P.kmax;
    for (int q = 0; q < count; ++q) {
      it.rho = it_rho[q];
      it.inv_rho = it_inv[q];
      it.inv_rho_next = it_inv_next[q];
      const float cs = it_c[q];
      float r2 = 0.f, s2 = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const AdmmElem o = admm_elem(0.0f, w[e], v[e], k[e], sv[e], si[e], gg[e], gg[e], cs, it);
        v[e] = o.v_new;
        k[e] = o.code;
        r2 += o.dr2;
        s2 += o.ds2;
      }
      if (!live) r2 = s2 = 0.f;
      r2 = warp_sum(r2);
      s2 = warp_sum(s2);
      if (lane == 0) {
        wsum[warp][q][0] += r2;
        wsum[warp][q][1] += s2;
      }
    }
    if (live) {
      *reinterpret_cast<float4*>(P.V + idx) = make_float4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<uchar4*>(P.codes + idx) = make_uchar4(k[0], k[1], k[2], k[3]);
    }
  }
  __syncthreads();
  for (int q = threadIdx.x; q < count; q += blockDim.x) {
    float a = 0.f, b = 0.f;
    for (int wq = 0; wq < 8; ++wq) {
      a += wsum[wq][q][0];
      b += wsum[wq][q][1];
    }
    float* ps = partials + ((size_t)(first + q) * slots + blockIdx.x) * 2;
    ps[0] = a;
    ps[1] = b;
  }
}

// Iterations [first, first + count) of a run, none of which forms a product (and none is the first).
void launch_admm_tail(Ctx* c, const EpiParams& P, int p, const double* rho_dev, int first, int count, int T) {
  const long long total = (long long)p * c->n;
  int blocks = c->num_sms * 4;
  if (blocks > c->partial_slots) blocks = c->partial_slots;
  for (int done = 0; done < count; done += TAIL_MAX) {
    const int m = count - done < TAIL_MAX ? count - done : TAIL_MAX;
    admm_tail_kernel<<<blocks, 256, 0, c->stream>>>(P, total, c->n, rho_dev, c->shift_c, first + done, m, T,
                                                   c->partials, c->partial_slots);
    LAUNCH(c);
  }
}

void launch_admm_rows(Ctx* c, const EpiParams& P, int p, bf16* hi, bf16* lo, float* row_inv) {
  const size_t smem = (size_t)c->n * sizeof(float);
  if (ensure_dynamic_smem((const void*)admm_row_kernel, 64 * 1024) != cudaSuccess) return;   // the launch error check reports it
  int blocks = row_pass_blocks(c, p, smem);
  if (blocks > c->partial_slots) blocks = c->partial_slots;
  admm_row_kernel<<<blocks, ROW_THREADS, smem, c->stream>>>(P, p, c->n, hi, lo, row_inv);
  LAUNCH(c);
}

void launch_grid_refresh(Ctx* c, const EpiParams& P, int p, int bits, int symmetric, int iter, float* delta,
                         float* zero, int* flags) {
  const int n = c->n, gs = P.group_size, ng = n / gs;
  const long long groups = (long long)p * ng;
  float* cand_delta = reinterpret_cast<float*>(c->R_hi);      // the R planes are free between the products
  float* cand_zero = reinterpret_cast<float*>(c->R_lo);       // and the row pass that rewrites them
  long long want = (groups * 32 + 255) / 256;
  const int blocks = (int)(want < 1184 ? want : 1184);
  refresh_eval_kernel<<<blocks, 256, 0, c->stream>>>(P.Rnext, P.W0, P.V, P.codes, P.first_iter, P.shift_c, P.s,
                                                     P.inv_s, p, n, gs, (1 << bits) - 1,
                                                     symmetric, P.inv_rho, delta, zero, cand_delta, cand_zero,
                                                     c->ps_totals);
  refresh_decide_kernel<<<1, 256, 0, c->stream>>>(c->ps_totals, blocks, iter, flags);
  refresh_commit_kernel<<<(unsigned)((groups + 255) / 256), 256, 0, c->stream>>>(groups, flags, cand_delta,
                                                                                 cand_zero, delta, zero);
  const long long total = (long long)p * n;
  int eb = c->partial_slots < 1184 ? c->partial_slots : 1184;
  if ((long long)eb * 256 > total) eb = (int)((total + 255) / 256);
  admm_elementwise_kernel<<<eb, 256, 0, c->stream>>>(P, cand_delta, cand_zero, total, n);
  c->launches += 4;
}

// sum_j eps_j . g_j  =  Tr(E^T H E)  when g = H E  (fp64 accumulation).
__global__ void objective_dot_kernel(long long total, int n, int gs, int ng, const float* __restrict__ W0,
                                     const unsigned char* __restrict__ codes,
                                     const float* __restrict__ delta, const float* __restrict__ zero,
                                     const float* __restrict__ g, double* out) {
  __shared__ double scratch[32];
  double acc = 0.0;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const long long gi = (idx / n) * ng + (idx % n) / gs;
    const float e = (zero[gi] + delta[gi] * (float)codes[idx]) - W0[idx];
    acc += (double)e * (double)g[idx];
  }
  acc = block_sum(acc, scratch);
  if (threadIdx.x == 0) atomicAdd(out, acc);
}

void launch_objective_dot(Ctx* c, const float* W0, int p, int gs, const unsigned char* codes,
                          const float* delta, const float* zero, const float* g, double* out) {
  const long long total = (long long)p * c->n;
  cudaMemsetAsync(out, 0, sizeof(double), c->stream);
  long long blocks = (total + 255) / 256;
  if (blocks > 4 * 148) blocks = 4 * 148;
  objective_dot_kernel<<<(unsigned)blocks, 256, 0, c->stream>>>(total, c->n, gs, c->n / gs, W0, codes,
                                                                delta, zero, g, out);
  LAUNCH(c);
}

}  // namespace admmq
