// One-time factorisation of the scaled Hessian (Algorithm 1 line 3) and its per-penalty part.
//
// The paper diagonalises H~ once so that (H~ + rho I)^{-1} is available for every rho.  Here the
// orthogonal reduction stops at tridiagonal form, H~ = Q T Q^T (Householder), which serves the same
// purpose: (H~ + rho I)^{-1} = Q (T + rho I)^{-1} Q^T, and T + rho I is solved in O(n) per column by an
// LDL^T factorisation computed once per penalty value.  The reduction runs in fp64 so that the
// operator is accurate far below the split-bf16 product error.
#include <cooperative_groups.h>

#include "internal.h"

namespace cg = cooperative_groups;

namespace admmq {

// ------------------------------------------------------------------------------------------------
// Householder tridiagonalisation of the symmetric matrix A (full storage, fp64), cooperative launch.
// Step k: x = A[k, k+1:], reflector H_k = I - beta u u^T with u = x - alpha e_1, trailing update
// A22 <- A22 - u w^T - w u^T, w = p - (beta u^T p / 2) u, p = beta A22 u.  Row r is always handled by
// the same warp (r mod #warps), so a warp re-reads only rows it wrote itself; row k and p cross CTAs
// and are read with cache-global loads after a grid-wide barrier.
// Output: td/te (diagonal / off-diagonal of T), reflector k in A[k, k+1:], beta[k].
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024, 1)
tridiag_reduce_kernel(double* __restrict__ A, int n, double* __restrict__ td, double* __restrict__ te,
                      double* __restrict__ beta, double* __restrict__ pvec) {
  cg::grid_group grid = cg::this_grid();
  extern __shared__ double sm[];
  double* u = sm;
  double* w = sm + n;
  __shared__ double scratch[32];
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int gw = blockIdx.x * wpb + (threadIdx.x >> 5);
  const int GW = gridDim.x * wpb;

  for (int k = 0; k < n - 2; ++k) {
    const int m = n - k - 1;
    const int c0 = k + 1;
    const double* rowk = A + (long long)k * n + c0;
    // ---- reflector (identical in every CTA) ----
    double tail = 0.0;
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
      const double x = __ldcg(rowk + i);
      u[i] = x;
      if (i > 0) tail += x * x;
    }
    tail = block_sum(tail, scratch);
    __syncthreads();
    const double x0 = u[0];
    double alpha = x0, bt = 0.0;
    if (tail > 0.0) {
      const double nrm = sqrt(x0 * x0 + tail);
      alpha = (x0 >= 0.0) ? -nrm : nrm;
      bt = 1.0 / (nrm * nrm - x0 * alpha);          // 2 / (u^T u)
    }
    __syncthreads();
    if (threadIdx.x == 0) u[0] = x0 - alpha;
    __syncthreads();
    // ---- p = beta * A22 u over the rows this warp owns ----
    int r = c0 + (((gw - c0) % GW) + GW) % GW;
    for (; r < n; r += GW) {
      const double* row = A + (long long)r * n + c0;
      double acc = 0.0;
      for (int i = lane; i < m; i += 32) acc += row[i] * u[i];
      acc = warp_sum(acc);
      if (lane == 0) pvec[r - c0] = bt * acc;
    }
    grid.sync();
    // ---- w = p - (beta u^T p / 2) u ----
    double up = 0.0;
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
      const double pi = __ldcg(pvec + i);
      w[i] = pi;
      up += pi * u[i];
    }
    up = block_sum(up, scratch);
    const double kc = 0.5 * bt * up;
    __syncthreads();
    for (int i = threadIdx.x; i < m; i += blockDim.x) w[i] -= kc * u[i];
    __syncthreads();
    // ---- rank-2 update of the rows this warp owns ----
    r = c0 + (((gw - c0) % GW) + GW) % GW;
    for (; r < n; r += GW) {
      double* row = A + (long long)r * n + c0;
      const double ur = u[r - c0], wr = w[r - c0];
      for (int i = lane; i < m; i += 32) row[i] -= ur * w[i] + wr * u[i];
    }
    if (blockIdx.x == 0) {
      double* rk = A + (long long)k * n + c0;
      for (int i = threadIdx.x; i < m; i += blockDim.x) rk[i] = u[i];
      if (threadIdx.x == 0) {
        td[k] = __ldcg(A + (long long)k * n + k);
        te[k] = alpha;
        beta[k] = bt;
      }
    }
    grid.sync();
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (n >= 2) {
      td[n - 2] = __ldcg(A + (long long)(n - 2) * n + (n - 2));
      te[n - 2] = __ldcg(A + (long long)(n - 2) * n + (n - 1));
      beta[n - 2] = 0.0;
    }
    td[n - 1] = __ldcg(A + (long long)(n - 1) * n + (n - 1));
    te[n - 1] = 0.0;
    beta[n - 1] = 0.0;
  }
}

cudaError_t tridiag_reduce(Ctx* c) {
  const int n = c->n;
  const size_t smem = (size_t)2 * n * sizeof(double);
  cudaError_t e = cudaFuncSetAttribute(tridiag_reduce_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tridiag_reduce_kernel, 1024, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  int blocks = c->num_sms;   // one CTA per SM: co-residency is what the cooperative launch checks
  double* A = c->A64;
  int nn = n;
  void* args[] = {&A, &nn, &c->td, &c->te, &c->beta, &c->pvec};
  e = cudaLaunchCooperativeKernel((void*)tridiag_reduce_kernel, dim3(blocks), dim3(1024), args, smem,
                                  c->stream);
  c->launches++;
  return e;
}

// ------------------------------------------------------------------------------------------------
// Q^T = H_{n-3} ... H_1 H_0 built row by row: P <- P H_k for k descending touches each row of P
// independently, so one warp keeps one row in shared memory and applies every reflector to it.
// ------------------------------------------------------------------------------------------------
__global__ void form_qt_kernel(const double* __restrict__ A, const double* __restrict__ beta, int n,
                               double* __restrict__ P, int rows_per_block) {
  extern __shared__ double sm[];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int r = n - 1 - (blockIdx.x * rows_per_block + wid);   // heavy rows first
  if (wid >= rows_per_block || r < 0) return;
  double* row = sm + (size_t)wid * n;
  for (int i = lane; i < n; i += 32) row[i] = (i == r) ? 1.0 : 0.0;
  __syncwarp();
  for (int k = min(r - 1, n - 3); k >= 0; --k) {
    const double bt = beta[k];
    if (bt == 0.0) continue;
    const int c0 = k + 1, m = n - c0;
    const double* u = A + (long long)k * n + c0;
    double acc = 0.0;
    for (int i = lane; i < m; i += 32) acc += row[c0 + i] * u[i];
    acc = bt * warp_sum(acc);
    for (int i = lane; i < m; i += 32) row[c0 + i] -= acc * u[i];
    __syncwarp();
  }
  double* out = P + (long long)r * n;
  for (int i = lane; i < n; i += 32) out[i] = row[i];
}

cudaError_t tridiag_form_qt(Ctx* c) {
  const int n = c->n;
  int rpb = (int)((200 * 1024) / ((size_t)n * sizeof(double)));
  if (rpb > 8) rpb = 8;
  if (rpb < 1) return cudaErrorInvalidValue;
  const size_t smem = (size_t)rpb * n * sizeof(double);
  cudaError_t e = cudaFuncSetAttribute(form_qt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  form_qt_kernel<<<(n + rpb - 1) / rpb, rpb * 32, smem, c->stream>>>(c->A64, c->beta, n, c->P64, rpb);
  c->launches++;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Per-penalty factor: LDL^T of T/rho + I (unit lower bidiagonal L, diagonal D), one thread per
// penalty value.  (T/rho + I) is the W-update matrix of Eq. 7 divided by rho, in the Q basis.
// ------------------------------------------------------------------------------------------------
__global__ void stage_factors_kernel(const double* __restrict__ td, const double* __restrict__ te, int n,
                                     const double* __restrict__ rho, int first, int count,
                                     double* __restrict__ L, double* __restrict__ invD, int* status) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= count) return;
  const int stage = first + t;
  const double inv_r = 1.0 / rho[stage];
  double* l = L + (long long)stage * n;
  double* id = invD + (long long)stage * n;
  double piv = 1.0 + td[0] * inv_r;
  bool bad = false;
  for (int i = 0; i < n; ++i) {
    if (!(piv > 0.0)) bad = true;
    const double ip = 1.0 / piv;
    id[i] = ip;
    if (i < n - 1) {
      const double b = te[i] * inv_r;
      const double li = b * ip;
      l[i] = li;
      piv = (1.0 + td[i + 1] * inv_r) - li * b;
    } else {
      l[i] = 0.0;
    }
  }
  if (bad) raise_status(status, ST_NOT_SPD);
}

void launch_stage_factors(Ctx* c, const double* rho_dev, int first, int count) {
  stage_factors_kernel<<<(count + 63) / 64, 64, 0, c->stream>>>(c->td, c->te, c->n, rho_dev, first, count,
                                                               c->stage_l, c->stage_invd, c->status);
  c->launches++;
}

// ------------------------------------------------------------------------------------------------
// Y' = (T/rho + I)^{-1} Y row by row (one warp per output channel).  Both substitutions are first-
// order linear recurrences x_i = y_i - l x_{i-1}; each lane runs its contiguous segment once to get
// the segment's affine map, the 32 maps are combined by a warp scan, and a second run applies the
// carry.  The factor (l, 1/d) of this penalty is staged once per CTA in shared memory in the same
// padded layout as the rows, so every lane's walk through its segment is bank-conflict free.
// fp64 registers, fp32 shared memory, result written as two bf16 planes.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int pad_index(int i, int seg, int stride) { return (i / seg) * stride + (i % seg); }

__global__ void tridiag_solve_kernel(const float* __restrict__ Y, int p, int n,
                                     const double* __restrict__ L, const double* __restrict__ invD,
                                     bf16* __restrict__ Yhi, bf16* __restrict__ Ylo, int seg, int stride) {
  extern __shared__ float smf[];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, wpb = blockDim.x >> 5;
  float* sl = smf;                         // l_i,     padded
  float* sd = smf + stride * 32;           // 1 / d_i, padded
  float* rs = smf + (size_t)(2 + wid) * stride * 32;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int q = pad_index(i, seg, stride);
    sl[q] = (float)L[i];
    sd[q] = (float)invD[i];
  }
  __syncthreads();
  const int a = min(n, lane * seg), b = min(n, (lane + 1) * seg);
  const int len = b - a;
  float* mine = rs + lane * stride;        // mine[t] is element a + t
  const float* ml = sl + lane * stride;    // ml[t] = l_{a+t}
  const float* md = sd + lane * stride;
  // l_{a-1}: the multiplier that couples this segment to the previous one
  const double l_prev = (a > 0 && a < n) ? (double)sl[pad_index(a - 1, seg, stride)] : 0.0;

  for (int j = blockIdx.x * wpb + wid; j < p; j += gridDim.x * wpb) {
    const float* y = Y + (long long)j * n;
    for (int i = lane; i < n; i += 32) rs[pad_index(i, seg, stride)] = y[i];
    __syncwarp();
    // ---- forward substitution  x_i = y_i - l_{i-1} x_{i-1} ----
    {
      double cc = 0.0, mm = 1.0, lp = l_prev;
#pragma unroll 4
      for (int t = 0; t < len; ++t) {
        cc = (double)mine[t] - lp * cc;
        mm *= -lp;
        lp = (double)ml[t];
      }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const double c2 = __shfl_up_sync(0xffffffffu, cc, off);
        const double m2 = __shfl_up_sync(0xffffffffu, mm, off);
        if (lane >= off) {
          cc = cc + mm * c2;
          mm = mm * m2;
        }
      }
      double x = __shfl_up_sync(0xffffffffu, cc, 1);
      if (lane == 0) x = 0.0;
      lp = l_prev;
#pragma unroll 4
      for (int t = 0; t < len; ++t) {
        x = (double)mine[t] - lp * x;
        lp = (double)ml[t];
        mine[t] = (float)(x * (double)md[t]);
      }
    }
    __syncwarp();
    // ---- backward substitution  z_i = x_i - l_i z_{i+1} ----
    {
      double cc = 0.0, mm = 1.0;
#pragma unroll 4
      for (int t = len - 1; t >= 0; --t) {
        const double li = (double)ml[t];
        cc = (double)mine[t] - li * cc;
        mm *= -li;
      }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const double c2 = __shfl_down_sync(0xffffffffu, cc, off);
        const double m2 = __shfl_down_sync(0xffffffffu, mm, off);
        if (lane + off < 32) {
          cc = cc + mm * c2;
          mm = mm * m2;
        }
      }
      double z = __shfl_down_sync(0xffffffffu, cc, 1);
      if (lane == 31) z = 0.0;
#pragma unroll 4
      for (int t = len - 1; t >= 0; --t) {
        z = (double)mine[t] - (double)ml[t] * z;
        mine[t] = (float)z;
      }
    }
    __syncwarp();
    for (int i = lane; i < n; i += 32) {
      bf16 h, l;
      split_bf16(rs[pad_index(i, seg, stride)], h, l);
      Yhi[(long long)j * n + i] = h;
      Ylo[(long long)j * n + i] = l;
    }
    __syncwarp();
  }
}

void launch_tridiag_solve(Ctx* c, int p, int stage) {
  const int n = c->n;
  const int seg = (n + 31) / 32;
  const int stride = seg | 1;
  const size_t per_row = (size_t)stride * 32 * sizeof(float);
  int wpb = (int)((200 * 1024) / per_row) - 2;
  if (wpb > 16) wpb = 16;
  if (wpb < 1) wpb = 1;
  const size_t smem = per_row * (wpb + 2);
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(tridiag_solve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
    attr_set = true;
  }
  int blocks = (p + wpb - 1) / wpb;
  if (blocks > c->num_sms) blocks = c->num_sms;
  tridiag_solve_kernel<<<blocks, wpb * 32, smem, c->stream>>>(
      c->Y, p, n, c->stage_l + (long long)stage * n, c->stage_invd + (long long)stage * n, c->Y_hi,
      c->Y_lo, seg, stride);
  c->launches++;
}

}  // namespace admmq
