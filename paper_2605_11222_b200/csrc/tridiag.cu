// One-time factorisation of the scaled Hessian (Algorithm 1 line 3) and its per-penalty part.
//
// The paper diagonalises H~ once so that (H~ + rho I)^{-1} is available for every rho.  Here the
// orthogonal reduction stops at tridiagonal form, H~ = Q T Q^T (Householder), which serves the same
// purpose: (H~ + rho I)^{-1} = Q (T + rho I)^{-1} Q^T, and T + rho I is solved in O(n) per column by an
// LDL^T factorisation computed once per penalty value.  The reduction and Q run in fp64 so that the
// operator is accurate far below the split-bf16 product error.
#include <cooperative_groups.h>

#include "internal.h"

namespace cg = cooperative_groups;

namespace admmq {

// ------------------------------------------------------------------------------------------------
// Householder tridiagonalisation of the symmetric matrix A (full storage, fp64), cooperative launch.
//
// Step k uses the reflector H_k = I - beta u u^T built from row k (u = x - alpha e_1, x = A[k, k+1:])
// and updates the trailing matrix A22 <- A22 - u w^T - w u^T with w = p - (beta u^T p / 2) u,
// p = beta A22 u.  The matrix is read and written ONCE per step: the pass of step k applies the
// rank-2 update of step k-1 to every element and, in the same sweep, accumulates that element's
// contribution to p of step k.  This is possible because the next reflector needs only one row of
// the updated matrix, which every CTA rebuilds for itself from the stored row and the two update
// vectors.  One grid-wide barrier per step (for p).
//
// Rows are dealt cyclically to row groups of CTAs, so the load stays balanced as the trailing matrix
// shrinks; a row group has C CTAs, each sweeping one chunk of the columns (C = 1 up to n = 9216,
// where the three length-n vectors fit in shared memory; above that each CTA keeps the full vectors
// in a private global scratch and only its column chunk in shared memory).
// Output: td/te (diagonal / off-diagonal of T), reflector k in A[k, k+1:], beta[k].
// ------------------------------------------------------------------------------------------------
constexpr int TRD_THREADS = 1024;
constexpr int TRD_BLOCKED_FROM = 4096;
constexpr int TRD_PSUM = 512;

struct TrdArgs {
  double* A;
  int n;
  double* td;
  double* te;
  double* beta;
  double* pbuf;   // [2][C][n]: per-chunk row sums of A22 u, double-buffered by the parity of the step
  double* priv;   // [grid][3][n]: full-length vectors of each CTA (C > 1 only)
  int C;          // column chunks per row group
  int cap;        // doubles per shared-memory vector
};

__global__ void __launch_bounds__(TRD_THREADS, 1) tridiag_reduce_kernel(TrdArgs a) {
  cg::grid_group grid = cg::this_grid();
  extern __shared__ double sm[];
  __shared__ double scratch[32];
  __shared__ double psum[TRD_PSUM];
  const int n = a.n, C = a.C;
  const int Gr = gridDim.x / C, g = blockIdx.x / C, h = blockIdx.x % C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool alias = (C == 1);
  // shared copies (column chunk) and full-length versions of: pending u, pending w, current reflector
  double *Sup = sm, *Swp = sm + a.cap, *Suc = sm + 2 * (size_t)a.cap;
  double *Fup = Sup, *Fwp = Swp, *Fuc = Suc;
  if (!alias) {
    double* base = a.priv + (size_t)blockIdx.x * 3 * n;
    Fup = base;
    Fwp = base + n;
    Fuc = base + 2 * (size_t)n;
  }
  for (int i = tid; i < n; i += TRD_THREADS) {
    Fup[i] = 0.0;
    Fwp[i] = 0.0;
    Fuc[i] = 0.0;
  }
  __syncthreads();
  double beta_k = 0.0, alpha_k = 0.0;   // belong to the current reflector u_k (in Fuc)

  for (int k = -1; k <= n - 2; ++k) {
    const int c0 = k + 1;
    if (k >= 0) {
      // ================= fused pass over rows / columns >= k+1 =================
      const int m = n - c0;
      int cb = c0, ce = n;
      if (!alias) {
        const int per = (((m + C - 1) / C) + 1) & ~1;
        cb = c0 + h * per;
        if (cb > n) cb = n;
        ce = cb + per < n ? cb + per : n;
      }
      const int base = alias ? 0 : (cb & ~1);
      if (!alias) {
        const int iend = (ce + 1) & ~1;
        for (int i = base + tid; i < iend; i += TRD_THREADS) {
          Sup[i - base] = Fup[i];
          Swp[i - base] = Fwp[i];
          Suc[i - base] = Fuc[i];
        }
        __syncthreads();
      }
      const int r_first = c0 + (((g - c0) % Gr) + Gr) % Gr;
      const int nr = (r_first < n) ? (n - r_first + Gr - 1) / Gr : 0;
      const int i_lo = cb & ~1;
      const int width = ce > i_lo ? ce - i_lo : 0;
      const int nseg = (width + 255) >> 8;
      int Sf = 1;                                   // parts a row is split into, so that every warp has work
      while (nr * Sf < 32 && Sf < nseg) Sf <<= 1;
      const int sp = (nseg + Sf - 1) / Sf;
      const int items = nr * Sf;
      for (int it = warp; it < items; it += 32) {
        const int rl = it / Sf, part = it - rl * Sf;
        const int r = r_first + rl * Gr;
        const double ur = Fup[r], wr = Fwp[r];
        double* arow = a.A + (size_t)r * n;
        double acc = 0.0;
        const int s_end = (part + 1) * sp < nseg ? (part + 1) * sp : nseg;
        for (int sg = part * sp; sg < s_end; ++sg) {
          const int i0 = i_lo + (sg << 8) + lane * 2;
          double2 av[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int i = i0 + q * 64;
            av[q] = make_double2(0.0, 0.0);
            if (i < ce) av[q] = __ldcg(reinterpret_cast<const double2*>(arow + i));
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int i = i0 + q * 64;
            if (i < ce) {
              const double2 up2 = *reinterpret_cast<const double2*>(Sup + (i - base));
              const double2 wp2 = *reinterpret_cast<const double2*>(Swp + (i - base));
              const double2 uc2 = *reinterpret_cast<const double2*>(Suc + (i - base));
              const double x = av[q].x - (ur * wp2.x + wr * up2.x);
              const double y = av[q].y - (ur * wp2.y + wr * up2.y);
              const bool vx = (i >= cb), vy = (i + 1 < ce);
              if (vx && vy) {
                __stcg(reinterpret_cast<double2*>(arow + i), make_double2(x, y));
                acc += x * uc2.x + y * uc2.y;
              } else if (vx) {
                arow[i] = x;
                acc += x * uc2.x;
              } else if (vy) {
                arow[i + 1] = y;
                acc += y * uc2.y;
              }
            }
          }
        }
        acc = warp_sum(acc);
        if (lane == 0) psum[it] = acc;
      }
      __syncthreads();
      double* pb = a.pbuf + ((size_t)(k & 1) * C + h) * n;
      for (int t = tid; t < nr; t += TRD_THREADS) {
        double s = 0.0;
        for (int q = 0; q < Sf; ++q) s += psum[t * Sf + q];
        pb[r_first + t * Gr] = s;
      }
      grid.sync();
    }
    // ================= vector phase (identical in every CTA) =================
    // w_k = p - (beta u^T p / 2) u,  p = beta A22 u
    double up = 0.0;
    if (k >= 0) {
      const double* pb = a.pbuf + (size_t)(k & 1) * C * n;
      for (int i = c0 + tid; i < n; i += TRD_THREADS) {
        double p = 0.0;
        for (int hh = 0; hh < C; ++hh) p += __ldcg(pb + (size_t)hh * n + i);
        p *= beta_k;
        Fwp[i] = p;                      // w_{k-1} is dead: this CTA's pass has used it
        up += p * Fuc[i];
      }
    }
    up = block_sum(up, scratch);
    const double kc = 0.5 * beta_k * up;
    if (k >= 0)
      for (int i = c0 + tid; i < n; i += TRD_THREADS) Fwp[i] -= kc * Fuc[i];
    __syncthreads();
    // row k+1 of the matrix after update k, rebuilt locally: source of the next reflector and of td[k+1]
    const int r1 = k + 1;
    const double u1 = Fuc[r1], w1 = Fwp[r1];
    const double* row = a.A + (size_t)r1 * n;
    double tail = 0.0;
    for (int i = r1 + 1 + tid; i < n; i += TRD_THREADS) {
      const double x = __ldcg(row + i) - u1 * Fwp[i] - w1 * Fuc[i];
      Fup[i] = x;                        // u_{k-1} is dead
      if (i > r1 + 1) tail += x * x;
    }
    tail = block_sum(tail, scratch);
    __syncthreads();
    const double x0 = (r1 + 1 < n) ? Fup[r1 + 1] : 0.0;
    double alpha = x0, bt = 0.0;
    if (tail > 0.0) {
      const double nrm = sqrt(x0 * x0 + tail);
      alpha = (x0 >= 0.0) ? -nrm : nrm;
      bt = 1.0 / (nrm * nrm - x0 * alpha);          // 2 / (u^T u)
    }
    const double diag = __ldcg(row + r1) - 2.0 * u1 * w1;
    __syncthreads();
    if (tid == 0) {
      if (r1 + 1 < n) Fup[r1 + 1] = x0 - alpha;
      Fup[r1] = 0.0;
    }
    if (blockIdx.x == 0) {
      if (k >= 0) {
        double* rk = a.A + (size_t)k * n;
        for (int i = c0 + tid; i < n; i += TRD_THREADS) rk[i] = Fuc[i];
        if (tid == 0) {
          a.te[k] = alpha_k;
          a.beta[k] = beta_k;
        }
      }
      if (tid == 0) a.td[r1] = diag;
    }
    // (u_k, w_k) become the pending update, the new reflector becomes current
    double* t = Fup;
    Fup = Fuc;
    Fuc = t;
    if (alias) {
      Sup = Fup;
      Suc = Fuc;
    }
    alpha_k = alpha;
    beta_k = bt;
    __syncthreads();
  }
  if (blockIdx.x == 0 && tid == 0) {
    a.te[n - 1] = 0.0;
    a.beta[n - 1] = 0.0;
  }
}

static int trd_cap(int n, int C) {
  if (C == 1) return n;
  return ((((n - 1 + C - 1) / C) + 1) & ~1) + 4;
}

cudaError_t tridiag_reduce(Ctx* c) {
  const int n = c->n;
  // The blocked kernel halves the traffic per column but pays a second grid barrier and more serial
  // work per column; measured, it wins from n = 4096 on (whole factorisation at n = 4096: 98.7 ms vs 102.0 ms;
  // reduction alone at n = 12288: 1.36 s vs 2.0 s).
  if (n >= TRD_BLOCKED_FROM) {
    const cudaError_t eb = tridiag_reduce_blocked(c);
    if (eb != cudaErrorInvalidConfiguration) return eb;    // too large for its shared memory: fall through
  }
  int C = 1;
  while ((size_t)3 * 8 * trd_cap(n, C) > (size_t)216 * 1024 && C < 4) C *= 2;
  int blocks = (c->num_sms / C) * C;   // one CTA per SM: co-residency is what the cooperative launch checks
  if (blocks < C) return cudaErrorLaunchOutOfResources;
  TrdArgs a;
  a.A = c->A64;
  a.n = n;
  a.td = c->td;
  a.te = c->te;
  a.beta = c->beta;
  a.C = C;
  a.cap = trd_cap(n, C);
  // scratch inside the (not yet written) Q^T buffer
  a.pbuf = c->P64;
  a.priv = c->P64 + (((size_t)2 * C * n + 31) & ~(size_t)31);
  if (C > 1 && (size_t)2 * C * n + 32 + (size_t)blocks * 3 * n > (size_t)n * n) return cudaErrorInvalidValue;
  const size_t smem = (size_t)3 * a.cap * sizeof(double);
  cudaError_t e = cudaFuncSetAttribute(tridiag_reduce_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tridiag_reduce_kernel, TRD_THREADS, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  void* args[] = {&a};
  e = cudaLaunchCooperativeKernel((void*)tridiag_reduce_kernel, dim3(blocks), dim3(TRD_THREADS), args, smem,
                                  c->stream);
  c->launches++;
  return e;
}

// ------------------------------------------------------------------------------------------------
// Q^T = H_{n-3} ... H_1 H_0, accumulated in blocks of WY_NB reflectors in compact WY form:
//   H_kb H_{kb+1} ... H_{kb+nb-1} = I - Y S Y^T,  Y = [u_kb ... u_{kb+nb-1}], S upper triangular,
//   S_jj = beta_j,  S_{0:j,j} = -beta_j S_{0:j,0:j} (Y_{:,0:j}^T u_j).
// Row r of P = Q^T starts as e_r^T and receives the blocks in descending order:
//   X <- X (I - Y S^T Y^T) = X - ((X Y) S^T) Y^T   on the rows r > kb and columns > kb,
// independently of every other row, so each CTA owns a cyclic set of rows and needs no grid barrier.
// Both products run on the fp64 tensor-core MMA (m8n8k4).
// ------------------------------------------------------------------------------------------------
constexpr int WY_NB = 32;
constexpr int QT_KC = 64;            // columns per staged chunk
constexpr int QT_LD = QT_KC + 4;     // stride == 4 (mod 16) doubles: fragment loads hit every bank pair twice
constexpr int QT_LDZ = WY_NB + 4;
constexpr int QT_RS_MAX = 128;       // row slots per CTA
constexpr int QT_THREADS = 1024;


// S of every block: one CTA per block.
__global__ void __launch_bounds__(1024)
wy_factor_kernel(const double* __restrict__ A, const double* __restrict__ beta, int n,
                 double* __restrict__ Sall) {
  __shared__ double Ys[WY_NB][65];
  __shared__ double Gs[WY_NB][WY_NB + 1];
  __shared__ double Ss[WY_NB][WY_NB + 1];
  const int b = blockIdx.x, kb = b * WY_NB;
  const int nrefl = n - 2;                                 // reflectors k = 0 .. n-3
  const int nbk = nrefl - kb < WY_NB ? nrefl - kb : WY_NB;
  const int tid = threadIdx.x, j1 = tid >> 5, j2 = tid & 31;
  double acc = 0.0;
  for (int cs = kb + 1; cs < n; cs += 64) {
    for (int idx = tid; idx < WY_NB * 64; idx += 1024) {
      const int j = idx >> 6, cl = idx & 63, cc = cs + cl;
      double v = 0.0;
      if (j < nbk && cc < n && cc >= kb + j + 1) v = A[(size_t)(kb + j) * n + cc];
      Ys[j][cl] = v;
    }
    __syncthreads();
#pragma unroll 8
    for (int cl = 0; cl < 64; ++cl) acc += Ys[j1][cl] * Ys[j2][cl];
    __syncthreads();
  }
  Gs[j1][j2] = acc;
  Ss[j1][j2] = 0.0;
  __syncthreads();
  if (tid < 32) {
    const int i = tid;                                     // lane i builds row i of S
    for (int j = 0; j < WY_NB; ++j) {
      const double bj = (j < nbk) ? beta[kb + j] : 0.0;
      if (i == j) Ss[i][j] = bj;
      if (i < j) {
        double s = 0.0;
        for (int l = i; l < j; ++l) s += Ss[i][l] * Gs[l][j];
        Ss[i][j] = -bj * s;
      }
    }
  }
  __syncthreads();
  Sall[(size_t)b * WY_NB * WY_NB + tid] = Ss[j1][j2];
}

__global__ void set_identity_kernel(double* __restrict__ P, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) P[(size_t)i * n + i] = 1.0;
}

__global__ void __launch_bounds__(QT_THREADS, 1)
form_qt_kernel(const double* __restrict__ A, const double* __restrict__ Sall, int n, int nblk,
               double* __restrict__ P) {
  extern __shared__ double smq[];
  double* Ys = smq;                                        // [WY_NB][QT_LD]
  double* Xs = Ys + WY_NB * QT_LD;                         // [QT_RS_MAX][QT_LD]
  double* Zp = Xs + QT_RS_MAX * QT_LD;                     // [ks][RS][QT_LDZ], ks * RS <= 128
  double* Z1 = Zp + QT_RS_MAX * QT_LDZ;                    // [RS][QT_LDZ]  (X Y), then -(X Y) S^T
  double* Ss = Z1 + QT_RS_MAX * QT_LDZ;                    // [WY_NB][WY_NB + 1]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int G = gridDim.x, c = blockIdx.x;
  if (c >= n) return;
  const int Rtot = (n - c + G - 1) / G;                    // rows c, c + G, c + 2G, ...
  const int nrefl = n - 2;

  for (int b = nblk - 1; b >= 0; --b) {
    const int kb = b * WY_NB;
    const int nbk = nrefl - kb < WY_NB ? nrefl - kb : WY_NB;
    int t0 = (kb + 1 - c + G - 1) / G;                     // first own row with r >= kb + 1
    if (kb + 1 - c <= 0) t0 = 0;
    const int Ract = Rtot - t0;
    if (Ract <= 0) continue;                               // uniform in the CTA
    const int RS = (Ract + 7) & ~7;
    const int nrt = RS >> 3;
    int KS = 1;
    while (KS < 4 && 2 * KS * RS <= QT_RS_MAX) KS <<= 1;
    const int kspan = QT_KC / KS;
    const int cbeg = ((kb + 1) / QT_KC) * QT_KC;

    for (int idx = tid; idx < WY_NB * WY_NB; idx += QT_THREADS)
      Ss[(idx >> 5) * (WY_NB + 1) + (idx & 31)] = Sall[(size_t)b * WY_NB * WY_NB + idx];

    // ---------------- Z = X Y ----------------
    const int units_z = nrt * 4 * KS;                      // (k split, row tile, column tile of 8)
    double z00 = 0.0, z01 = 0.0, z10 = 0.0, z11 = 0.0;     // accumulators of units warp and warp + 32
    for (int cs = cbeg; cs < n; cs += QT_KC) {
      for (int idx = tid; idx < WY_NB * QT_KC; idx += QT_THREADS) {
        const int j = idx >> 6, cl = idx & 63, cc = cs + cl;
        double v = 0.0;
        if (j < nbk && cc < n && cc >= kb + j + 1) v = A[(size_t)(kb + j) * n + cc];
        Ys[j * QT_LD + cl] = v;
      }
      for (int idx = tid; idx < RS * QT_KC; idx += QT_THREADS) {
        const int rl = idx >> 6, cl = idx & 63, cc = cs + cl;
        double v = 0.0;
        if (rl < Ract && cc < n) v = P[(size_t)(c + (size_t)(t0 + rl) * G) * n + cc];
        Xs[rl * QT_LD + cl] = v;
      }
      __syncthreads();
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        const int u = warp + 32 * s;
        if (u < units_z) {
          const int ks = u / (nrt * 4), rem = u - ks * nrt * 4;
          const int rt = rem >> 2, jt = rem & 3;
          const double* xa = Xs + (rt * 8 + gid) * QT_LD + ks * kspan + tig;
          const double* yb = Ys + (jt * 8 + gid) * QT_LD + ks * kspan + tig;
          double d0 = s ? z10 : z00, d1 = s ? z11 : z01;
          for (int kk = 0; kk < kspan; kk += 4) dmma_8x8x4(d0, d1, xa[kk], yb[kk]);
          if (s) {
            z10 = d0;
            z11 = d1;
          } else {
            z00 = d0;
            z01 = d1;
          }
        }
      }
      __syncthreads();
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      const int u = warp + 32 * s;
      if (u < units_z) {
        const int ks = u / (nrt * 4), rem = u - ks * nrt * 4;
        const int rt = rem >> 2, jt = rem & 3;
        double* zp = Zp + (ks * RS + rt * 8 + gid) * QT_LDZ + jt * 8 + 2 * tig;
        zp[0] = s ? z10 : z00;
        zp[1] = s ? z11 : z01;
      }
    }
    __syncthreads();
    for (int idx = tid; idx < RS * WY_NB; idx += QT_THREADS) {
      const int rl = idx >> 5, j = idx & 31;
      double z = 0.0;
      for (int ks = 0; ks < KS; ++ks) z += Zp[(ks * RS + rl) * QT_LDZ + j];
      Z1[rl * QT_LDZ + j] = z;
    }
    __syncthreads();
    // ---------------- Z2 = -(Z S^T):  Z2[rl][j] = -sum_{j' >= j} Z[rl][j'] S[j][j'] ----------------
    double z2v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int idx = tid + q * QT_THREADS;
      z2v[q] = 0.0;
      if (idx < RS * WY_NB) {
        const int rl = idx >> 5, j = idx & 31;
        double z = 0.0;
        for (int jp = j; jp < WY_NB; ++jp) z += Z1[rl * QT_LDZ + jp] * Ss[j * (WY_NB + 1) + jp];
        z2v[q] = -z;
      }
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int idx = tid + q * QT_THREADS;
      if (idx < RS * WY_NB) Z1[(idx >> 5) * QT_LDZ + (idx & 31)] = z2v[q];
    }
    __syncthreads();
    // ---------------- X += Z2 Y^T ----------------
    const int units_u = nrt * 8;                           // (row tile, column tile of 8 inside the chunk)
    for (int cs = cbeg; cs < n; cs += QT_KC) {
      for (int idx = tid; idx < WY_NB * QT_KC; idx += QT_THREADS) {
        const int j = idx >> 6, cl = idx & 63, cc = cs + cl;
        double v = 0.0;
        if (j < nbk && cc < n && cc >= kb + j + 1) v = A[(size_t)(kb + j) * n + cc];
        Ys[j * QT_LD + cl] = v;
      }
      __syncthreads();
      for (int u = warp; u < units_u; u += 32) {
        const int rt = u >> 3, nt = u & 7;
        const int rl = rt * 8 + gid;
        const int cc = cs + nt * 8 + 2 * tig;
        const bool live = (rl < Ract) && (cc < n);         // n is even: cc + 1 < n as well
        double* xp = P + (size_t)(c + (size_t)(t0 + (rl < Ract ? rl : 0)) * G) * n + cc;
        double2 cv = make_double2(0.0, 0.0);
        if (live) cv = *reinterpret_cast<const double2*>(xp);
        const double* za = Z1 + rl * QT_LDZ + tig;
        const double* yb = Ys + tig * QT_LD + nt * 8 + gid;
#pragma unroll
        for (int kk = 0; kk < WY_NB; kk += 4) dmma_8x8x4(cv.x, cv.y, za[kk], yb[kk * QT_LD]);
        if (live) *reinterpret_cast<double2*>(xp) = cv;
      }
      __syncthreads();
    }
  }
}

// ---- the same accumulation for CTAs with at most QT_PIPE_ROWS own rows (d_in <= QT_PIPE_ROWS x CTAs): the
// chunks of Y and X are staged by asynchronous copies several chunks ahead, so that the sweep over the columns
// no longer waits for a round trip to L2 at every chunk.
constexpr int QT_PIPE_ROWS = 32;
constexpr int QT_PIPE_DEPTH = 3;
__device__ __forceinline__ void cp_async8(double* dst_smem, const double* src, bool valid) {
  const unsigned int d = (unsigned int)__cvta_generic_to_shared(dst_smem);
  const int bytes = valid ? 8 : 0;                         // 0: the destination is filled with zeros
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__global__ void __launch_bounds__(QT_THREADS, 1)
form_qt_pipe_kernel(const double* __restrict__ A, const double* __restrict__ Sall, int n, int nblk,
               double* __restrict__ P) {
  extern __shared__ double smq[];
  constexpr int BUF = (WY_NB + QT_PIPE_ROWS) * QT_LD;      // one staged chunk: Y block, then the own rows of X
  double* Zp = smq + QT_PIPE_DEPTH * BUF;                  // [ks][RS][QT_LDZ], ks * RS <= 128
  double* Z1 = Zp + QT_RS_MAX * QT_LDZ;                    // [RS][QT_LDZ]  (X Y), then -(X Y) S^T
  double* Ss = Z1 + QT_PIPE_ROWS * QT_LDZ;                 // [WY_NB][WY_NB + 1]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int G = gridDim.x, c = blockIdx.x;
  if (c >= n) return;
  const int Rtot = (n - c + G - 1) / G;                    // rows c, c + G, c + 2G, ...
  const int nrefl = n - 2;

  for (int b = nblk - 1; b >= 0; --b) {
    const int kb = b * WY_NB;
    const int nbk = nrefl - kb < WY_NB ? nrefl - kb : WY_NB;
    int t0 = (kb + 1 - c + G - 1) / G;                     // first own row with r >= kb + 1
    if (kb + 1 - c <= 0) t0 = 0;
    const int Ract = Rtot - t0;
    if (Ract <= 0) continue;                               // uniform in the CTA
    const int RS = (Ract + 7) & ~7;
    const int nrt = RS >> 3;
    int KS = 1;
    while (KS < 4 && 2 * KS * RS <= QT_RS_MAX) KS <<= 1;
    const int kspan = QT_KC / KS;
    const int cbeg = ((kb + 1) / QT_KC) * QT_KC;

    for (int idx = tid; idx < WY_NB * WY_NB; idx += QT_THREADS)
      Ss[(idx >> 5) * (WY_NB + 1) + (idx & 31)] = Sall[(size_t)b * WY_NB * WY_NB + idx];

    // ---------------- Z = X Y ----------------
    const int units_z = nrt * 4 * KS;                      // (k split, row tile, column tile of 8)
    double z00 = 0.0, z01 = 0.0, z10 = 0.0, z11 = 0.0;     // accumulators of units warp and warp + 32
    const int nch = (n - cbeg + QT_KC - 1) / QT_KC;
    // chunk ci of the columns, staged by asynchronous copies QT_PIPE_DEPTH - 1 chunks ahead of its use
    auto issue = [&](int ci, bool with_x) {
      if (ci < nch) {
        const int cs = cbeg + ci * QT_KC;
        double* Yb = smq + (ci % QT_PIPE_DEPTH) * BUF;
        double* Xb = Yb + WY_NB * QT_LD;
        for (int idx = tid; idx < WY_NB * QT_KC; idx += QT_THREADS) {
          const int j = idx >> 6, cl = idx & 63, cc = cs + cl;
          const bool ok = j < nbk && cc < n && cc >= kb + j + 1;
          cp_async8(Yb + j * QT_LD + cl, ok ? A + (size_t)(kb + j) * n + cc : A, ok);
        }
        if (with_x)
          for (int idx = tid; idx < RS * QT_KC; idx += QT_THREADS) {
            const int rl = idx >> 6, cl = idx & 63, cc = cs + cl;
            const bool ok = rl < Ract && cc < n;
            cp_async8(Xb + rl * QT_LD + cl, ok ? P + (size_t)(c + (size_t)(t0 + rl) * G) * n + cc : P, ok);
          }
      }
      cp_async_commit();                                   // an empty group keeps the count uniform
    };
    for (int d = 0; d < QT_PIPE_DEPTH - 1; ++d) issue(d, true);
    for (int ci = 0; ci < nch; ++ci) {
      issue(ci + QT_PIPE_DEPTH - 1, true);                 // its buffer was released by the barrier below
      cp_async_wait<QT_PIPE_DEPTH - 1>();
      __syncthreads();
      const double* Ys = smq + (ci % QT_PIPE_DEPTH) * BUF;
      const double* Xs = Ys + WY_NB * QT_LD;
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        const int u = warp + 32 * s;
        if (u < units_z) {
          const int ks = u / (nrt * 4), rem = u - ks * nrt * 4;
          const int rt = rem >> 2, jt = rem & 3;
          const double* xa = Xs + (rt * 8 + gid) * QT_LD + ks * kspan + tig;
          const double* yb = Ys + (jt * 8 + gid) * QT_LD + ks * kspan + tig;
          double d0 = s ? z10 : z00, d1 = s ? z11 : z01;
          for (int kk = 0; kk < kspan; kk += 4) dmma_8x8x4(d0, d1, xa[kk], yb[kk]);
          if (s) {
            z10 = d0;
            z11 = d1;
          } else {
            z00 = d0;
            z01 = d1;
          }
        }
      }
      __syncthreads();
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      const int u = warp + 32 * s;
      if (u < units_z) {
        const int ks = u / (nrt * 4), rem = u - ks * nrt * 4;
        const int rt = rem >> 2, jt = rem & 3;
        double* zp = Zp + (ks * RS + rt * 8 + gid) * QT_LDZ + jt * 8 + 2 * tig;
        zp[0] = s ? z10 : z00;
        zp[1] = s ? z11 : z01;
      }
    }
    __syncthreads();
    for (int idx = tid; idx < RS * WY_NB; idx += QT_THREADS) {
      const int rl = idx >> 5, j = idx & 31;
      double z = 0.0;
      for (int ks = 0; ks < KS; ++ks) z += Zp[(ks * RS + rl) * QT_LDZ + j];
      Z1[rl * QT_LDZ + j] = z;
    }
    __syncthreads();
    // ---------------- Z2 = -(Z S^T):  Z2[rl][j] = -sum_{j' >= j} Z[rl][j'] S[j][j'] ----------------
    double z2v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int idx = tid + q * QT_THREADS;
      z2v[q] = 0.0;
      if (idx < RS * WY_NB) {
        const int rl = idx >> 5, j = idx & 31;
        double z = 0.0;
        for (int jp = j; jp < WY_NB; ++jp) z += Z1[rl * QT_LDZ + jp] * Ss[j * (WY_NB + 1) + jp];
        z2v[q] = -z;
      }
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int idx = tid + q * QT_THREADS;
      if (idx < RS * WY_NB) Z1[(idx >> 5) * QT_LDZ + (idx & 31)] = z2v[q];
    }
    __syncthreads();
    // ---------------- X += Z2 Y^T ----------------
    const int units_u = nrt * 8;                           // (row tile, column tile of 8 inside the chunk)
    __syncthreads();                                       // every warp is done with the buffers of the first sweep
    // one unit per warp at most (QT_PIPE_ROWS = 32 rows): its tile of X for the next chunk is loaded a chunk ahead
    const int rt_u = warp >> 3, nt_u = warp & 7;
    const int rl_u = rt_u * 8 + gid;
    const bool has_u = warp < units_u;
    auto xptr = [&](int ci) {
      return P + (size_t)(c + (size_t)(t0 + (rl_u < Ract ? rl_u : 0)) * G) * n + cbeg + ci * QT_KC + nt_u * 8 + 2 * tig;
    };
    auto xlive = [&](int ci) { return has_u && rl_u < Ract && cbeg + ci * QT_KC + nt_u * 8 + 2 * tig < n; };
    double2 cvn = make_double2(0.0, 0.0);
    if (xlive(0)) cvn = *reinterpret_cast<const double2*>(xptr(0));
    for (int d = 0; d < QT_PIPE_DEPTH - 1; ++d) issue(d, false);
    for (int ci = 0; ci < nch; ++ci) {
      issue(ci + QT_PIPE_DEPTH - 1, false);
      cp_async_wait<QT_PIPE_DEPTH - 1>();
      __syncthreads();
      const double* Ys = smq + (ci % QT_PIPE_DEPTH) * BUF;
      double2 cv = cvn;
      if (ci + 1 < nch && xlive(ci + 1)) cvn = *reinterpret_cast<const double2*>(xptr(ci + 1));
      if (has_u) {
        const double* za = Z1 + rl_u * QT_LDZ + tig;
        const double* yb = Ys + tig * QT_LD + nt_u * 8 + gid;
#pragma unroll
        for (int kk = 0; kk < WY_NB; kk += 4) dmma_8x8x4(cv.x, cv.y, za[kk], yb[kk * QT_LD]);
        if (xlive(ci)) *reinterpret_cast<double2*>(xptr(ci)) = cv;
      }
      __syncthreads();
    }
  }
}

cudaError_t tridiag_form_qt(Ctx* c) {
  const int n = c->n;
  const int nrefl = n - 2;
  const int nblk = (nrefl + WY_NB - 1) / WY_NB;
  double* Sall = c->wy_s;
  cudaError_t e = cudaMemsetAsync(c->P64, 0, (size_t)n * n * sizeof(double), c->stream);
  if (e != cudaSuccess) return e;
  set_identity_kernel<<<(n + 255) / 256, 256, 0, c->stream>>>(c->P64, n);
  c->launches++;
  wy_factor_kernel<<<nblk, 1024, 0, c->stream>>>(c->A64, c->beta, n, Sall);
  c->launches++;
  const size_t smem = (size_t)(WY_NB * QT_LD + QT_RS_MAX * QT_LD + 2 * QT_RS_MAX * QT_LDZ +
                               WY_NB * (WY_NB + 1)) * sizeof(double);
  e = cudaFuncSetAttribute(form_qt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int grid = c->num_sms;
  if ((n + grid - 1) / grid <= QT_PIPE_ROWS) {
    const size_t smem_p = (size_t)(QT_PIPE_DEPTH * (WY_NB + QT_PIPE_ROWS) * QT_LD + QT_RS_MAX * QT_LDZ +
                                   QT_PIPE_ROWS * QT_LDZ + WY_NB * (WY_NB + 1)) * sizeof(double);
    e = cudaFuncSetAttribute(form_qt_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_p);
    if (e != cudaSuccess) return e;
    form_qt_pipe_kernel<<<grid, QT_THREADS, smem_p, c->stream>>>(c->A64, Sall, n, nblk, c->P64);
    c->launches++;
    return cudaGetLastError();
  }
  while ((n + grid - 1) / grid > QT_RS_MAX) grid += c->num_sms;   // at most 128 rows per CTA
  form_qt_kernel<<<grid, QT_THREADS, smem, c->stream>>>(c->A64, Sall, n, nblk, c->P64);
  c->launches++;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Per-penalty factor: LDL^T of T/rho + I (unit lower bidiagonal L, diagonal D), one thread per
// penalty value, fp64 arithmetic.  (T/rho + I) is the W-update matrix of Eq. 7 divided by rho, in the
// Q basis.  The factor is stored in fp32 in the order the solve kernel reads it: element
// i = t * ept + e (thread t, e-th element of its segment) at [e * SOLVE_THREADS + t].
// ------------------------------------------------------------------------------------------------
constexpr int SOLVE_THREADS = 256;
constexpr int SOLVE_ROWS = 2;               // rows solved together by the register-resident kernel

// elements per thread of the solve kernel: n / 256 rounded up to a multiple of 8 (16-byte plane stores)
int solve_ept(int n) { return (((n + SOLVE_THREADS - 1) / SOLVE_THREADS) + 7) & ~7; }
size_t stage_factor_stride(int n) { return (size_t)solve_ept(n) * SOLVE_THREADS; }

__global__ void stage_factors_kernel(const double* __restrict__ td, const double* __restrict__ te, int n,
                                     const double* __restrict__ rho, const double* __restrict__ mu_p, int first,
                                     int count, int ept, float* __restrict__ L, float* __restrict__ invD,
                                     double* __restrict__ shift_c, const float* __restrict__ series_inv,
                                     float* __restrict__ series_f, float* __restrict__ series_g, int* status) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= count) return;
  const int stage = first + t;
  const double inv_r = 1.0 / rho[stage];
  // shifted operator: the solve returns (T/rho + I)^{-1} y / (mu + rho); c = rho / (mu + rho) goes to the element update
  const double wshift = 1.0 / (mu_p[0] + rho[stage]);
  shift_c[stage] = rho[stage] * wshift;
  // truncated series c (I + E), E = (mu I - H~) / (mu + rho): factor of the product R (mu I - H~), with the inverse
  // of the operand plane's scale folded in
  series_f[stage] = (float)(rho[stage] * wshift * wshift * (double)series_inv[0]);
  series_g[stage] = (float)(wshift * (double)series_inv[0]);   // one more factor E: (c R E) (mu I - H~) / (mu + rho)
  const size_t stride = (size_t)ept * SOLVE_THREADS;
  float* l = L + (size_t)stage * stride;
  float* id = invD + (size_t)stage * stride;
  double piv = 1.0 + td[0] * inv_r;
  bool bad = false;
  for (int i = 0; i < n; ++i) {
    if (!(piv > 0.0)) bad = true;
    const double ip = 1.0 / piv;
    const size_t q = (size_t)(i % ept) * SOLVE_THREADS + i / ept;
    id[q] = (float)(ip * wshift);
    if (i < n - 1) {
      const double b = te[i] * inv_r;
      const double li = b * ip;
      l[q] = (float)li;
      piv = (1.0 + td[i + 1] * inv_r) - li * b;
    } else {
      l[q] = 0.0f;
    }
  }
  if (bad) raise_status(status, ST_NOT_SPD);
}

void launch_stage_factors(Ctx* c, const double* rho_dev, int first, int count) {
  stage_factors_kernel<<<(count + 63) / 64, 64, 0, c->stream>>>(c->td, c->te, c->n, rho_dev, c->scal + 8, first,
                                                               count, solve_ept(c->n), c->stage_l, c->stage_invd,
                                                               c->shift_c, c->fscal + 9, c->series_f, c->series_g, c->status);
  c->launches++;
}

// ------------------------------------------------------------------------------------------------
// Y' = (T/rho + I)^{-1} Y row by row.  Both substitutions are first-order linear recurrences
// x_i = y_i - l x_{i-1}.  One CTA per row at a time: every thread owns a contiguous segment of EPT
// elements in registers, runs it once to get the segment's affine map x_out = c + m x_in, the 256 maps
// are combined by a block-wide scan, and a second run applies the carry.  The LDL^T substitution of a
// positive definite matrix is backward stable, so fp32 arithmetic keeps the result at the accuracy of
// the fp32 right-hand side.  Result written as two fp16 planes of the row times a power of two
// (largest magnitude brought to [2^13, 2^14)), with the inverse scale per row.
// ------------------------------------------------------------------------------------------------
struct Affine {
  float c, m;
};
// map `second` applied after map `first`
__device__ __forceinline__ Affine then(Affine first, Affine second) {
  Affine r;
  r.c = fmaf(second.m, first.c, second.c);
  r.m = second.m * first.m;
  return r;
}

template <int EPT>
__global__ void __launch_bounds__(SOLVE_THREADS)
tridiag_solve_kernel(const float* __restrict__ Y, int p, int n, const float* __restrict__ lT,
                     const float* __restrict__ dT, bf16* __restrict__ Yhi, bf16* __restrict__ Ylo,
                     float* __restrict__ row_inv) {
  extern __shared__ float fac[];                           // this penalty's factor: l then 1/d, [e][thread]
  __shared__ Affine wtot[SOLVE_THREADS / 32];
  __shared__ float mscratch[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float* sl = fac;
  float* sd = fac + EPT * SOLVE_THREADS;
  for (int i = tid; i < EPT * SOLVE_THREADS; i += SOLVE_THREADS) {
    sl[i] = lT[i];
    sd[i] = dT[i];
  }
  __syncthreads();
  const int a0 = tid * EPT;
  const int len = a0 >= n ? 0 : (n - a0 < EPT ? n - a0 : EPT);      // a multiple of 8
  const float l_before = (tid > 0 && len > 0) ? sl[(EPT - 1) * SOLVE_THREADS + tid - 1] : 0.0f;

  constexpr bool PREFETCH = (EPT <= 24);                   // next row's segment requested a row ahead
  float xn[PREFETCH ? EPT : 4];
  auto load_row = [&](int j, float* dst) {
    const float* y = Y + (size_t)j * n + a0;
#pragma unroll
    for (int e = 0; e < EPT; e += 4) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e < len) v = *reinterpret_cast<const float4*>(y + e);
      dst[e] = v.x; dst[e + 1] = v.y; dst[e + 2] = v.z; dst[e + 3] = v.w;
    }
  };
  if (PREFETCH && (int)blockIdx.x < p) load_row(blockIdx.x, xn);
  for (int j = blockIdx.x; j < p; j += gridDim.x) {
    float x[EPT];
    if (PREFETCH) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) x[e] = xn[e];
      if (j + (int)gridDim.x < p) load_row(j + gridDim.x, xn);
    } else {
      load_row(j, x);
    }
    // ---- forward substitution x_i = y_i - l_{i-1} x_{i-1}, then the diagonal ----
    {
      Affine f{0.0f, 1.0f};
      float lp = l_before;
#pragma unroll
      for (int t = 0; t < EPT; ++t)
        if (t < len) {
          f.c = fmaf(-lp, f.c, x[t]);
          f.m *= -lp;
          lp = sl[t * SOLVE_THREADS + tid];
        }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        Affine o;
        o.c = __shfl_up_sync(0xffffffffu, f.c, off);
        o.m = __shfl_up_sync(0xffffffffu, f.m, off);
        if (lane >= off) f = then(o, f);
      }
      if (lane == 31) wtot[warp] = f;
      __syncthreads();
      Affine pre{0.0f, 1.0f};
      for (int w = 0; w < warp; ++w) pre = then(pre, wtot[w]);
      float xin = __shfl_up_sync(0xffffffffu, then(pre, f).c, 1);
      if (lane == 0) xin = pre.c;
      lp = l_before;
#pragma unroll
      for (int t = 0; t < EPT; ++t)
        if (t < len) {
          xin = fmaf(-lp, xin, x[t]);
          lp = sl[t * SOLVE_THREADS + tid];
          x[t] = xin * sd[t * SOLVE_THREADS + tid];
        }
      __syncthreads();
    }
    // ---- backward substitution z_i = x_i - l_i z_{i+1} ----
    float zmax = 0.0f;
    {
      Affine f{0.0f, 1.0f};
#pragma unroll
      for (int t = EPT - 1; t >= 0; --t)
        if (t < len) {
          const float li = sl[t * SOLVE_THREADS + tid];
          f.c = fmaf(-li, f.c, x[t]);
          f.m *= -li;
        }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        Affine o;
        o.c = __shfl_down_sync(0xffffffffu, f.c, off);
        o.m = __shfl_down_sync(0xffffffffu, f.m, off);
        if (lane + off < 32) f = then(o, f);
      }
      if (lane == 0) wtot[warp] = f;
      __syncthreads();
      Affine post{0.0f, 1.0f};
      for (int w = SOLVE_THREADS / 32 - 1; w > warp; --w) post = then(post, wtot[w]);
      float z = __shfl_down_sync(0xffffffffu, then(post, f).c, 1);
      if (lane == 31) z = post.c;
#pragma unroll
      for (int t = EPT - 1; t >= 0; --t)
        if (t < len) {
          z = fmaf(-sl[t * SOLVE_THREADS + tid], z, x[t]);
          x[t] = z;
          zmax = fmaxf(zmax, fabsf(z));
        }
    }
    zmax = block_max(zmax, mscratch);                      // its barriers also separate the rows' use of wtot
    float inv;
    const float sc = pow2_scale_for(zmax, &inv);
    if (tid == 0) row_inv[j] = inv;
#pragma unroll
    for (int e = 0; e < EPT; e += 8) {
      if (e < len) {
        __align__(16) __half hh[8];
        __align__(16) __half ll[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) split_f16(x[e + k] * sc, hh[k], ll[k]);
        *reinterpret_cast<uint4*>(Yhi + (size_t)j * n + a0 + e) = *reinterpret_cast<const uint4*>(hh);
        *reinterpret_cast<uint4*>(Ylo + (size_t)j * n + a0 + e) = *reinterpret_cast<const uint4*>(ll);
      }
    }
  }
}

// The same solve for R rows at a time, for d_in <= 4096 (EPT <= 16).  The one-row kernel is bound by latency,
// not by memory: every step of its four recurrences waits for the previous one (and for a shared-memory load of
// the factor).  Here the thread's part of the factor sits in registers for all rows, and the R rows give every
// step R independent chains; the multipliers of the affine maps, the barriers and the loop overhead are shared by
// the rows.  Every row sees exactly the operations, in the same order, as in the one-row kernel.
template <int R>
struct AffineR {
  float c[R];
  float m;
};

template <int EPT, int R, bool FULL>
__global__ void __launch_bounds__(SOLVE_THREADS, 3)
tridiag_solve_rows_kernel(const float* __restrict__ Y, int p, int n, const float* __restrict__ lT,
                          const float* __restrict__ dT, bf16* __restrict__ Yhi, bf16* __restrict__ Ylo,
                          float* __restrict__ row_inv) {
  __shared__ AffineR<R> wtot[SOLVE_THREADS / 32];
  __shared__ float mscratch[R][32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float sl[EPT], sd[EPT];
#pragma unroll
  for (int t = 0; t < EPT; ++t) {
    sl[t] = lT[t * SOLVE_THREADS + tid];
    sd[t] = dT[t * SOLVE_THREADS + tid];
  }
  const int a0 = tid * EPT;
  // FULL: d_in = EPT * SOLVE_THREADS, every thread has a whole segment and the guards below fold away
  const int len = FULL ? EPT : (a0 >= n ? 0 : (n - a0 < EPT ? n - a0 : EPT));      // a multiple of 8
  const float l_before = (tid > 0 && len > 0) ? lT[(EPT - 1) * SOLVE_THREADS + tid - 1] : 0.0f;
  const int groups = (p + R - 1) / R;

  for (int jg = blockIdx.x; jg < groups; jg += gridDim.x) {
    const int j0 = jg * R;
    float x[R][EPT];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int j = j0 + r < p ? j0 + r : p - 1;           // rows past the end repeat the last one, unsaved
      const float* y = Y + (size_t)j * n + a0;
#pragma unroll
      for (int e = 0; e < EPT; e += 4) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < len) v = *reinterpret_cast<const float4*>(y + e);
        x[r][e] = v.x; x[r][e + 1] = v.y; x[r][e + 2] = v.z; x[r][e + 3] = v.w;
      }
    }
    // ---- forward substitution x_i = y_i - l_{i-1} x_{i-1}, then the diagonal ----
    {
      AffineR<R> f;
#pragma unroll
      for (int r = 0; r < R; ++r) f.c[r] = 0.0f;
      f.m = 1.0f;
      float lp = l_before;
#pragma unroll
      for (int t = 0; t < EPT; ++t)
        if (t < len) {
#pragma unroll
          for (int r = 0; r < R; ++r) f.c[r] = fmaf(-lp, f.c[r], x[r][t]);
          f.m *= -lp;
          lp = sl[t];
        }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        float oc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) oc[r] = __shfl_up_sync(0xffffffffu, f.c[r], off);
        const float om = __shfl_up_sync(0xffffffffu, f.m, off);
        if (lane >= off) {
#pragma unroll
          for (int r = 0; r < R; ++r) f.c[r] = fmaf(f.m, oc[r], f.c[r]);
          f.m = f.m * om;
        }
      }
      if (lane == 31) wtot[warp] = f;
      __syncthreads();
      float prec[R], prem = 1.0f;
#pragma unroll
      for (int r = 0; r < R; ++r) prec[r] = 0.0f;
      for (int w = 0; w < warp; ++w) {
        const float wm = wtot[w].m;
#pragma unroll
        for (int r = 0; r < R; ++r) prec[r] = fmaf(wm, prec[r], wtot[w].c[r]);
        prem = wm * prem;
      }
      float xin[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float tot = fmaf(f.m, prec[r], f.c[r]);      // map of everything up to this thread
        xin[r] = __shfl_up_sync(0xffffffffu, tot, 1);
        if (lane == 0) xin[r] = prec[r];
      }
      lp = l_before;
#pragma unroll
      for (int t = 0; t < EPT; ++t)
        if (t < len) {
#pragma unroll
          for (int r = 0; r < R; ++r) {
            xin[r] = fmaf(-lp, xin[r], x[r][t]);
            x[r][t] = xin[r] * sd[t];
          }
          lp = sl[t];
        }
      __syncthreads();
    }
    // ---- backward substitution z_i = x_i - l_i z_{i+1} ----
    float zmax[R];
#pragma unroll
    for (int r = 0; r < R; ++r) zmax[r] = 0.0f;
    {
      AffineR<R> f;
#pragma unroll
      for (int r = 0; r < R; ++r) f.c[r] = 0.0f;
      f.m = 1.0f;
#pragma unroll
      for (int t = EPT - 1; t >= 0; --t)
        if (t < len) {
#pragma unroll
          for (int r = 0; r < R; ++r) f.c[r] = fmaf(-sl[t], f.c[r], x[r][t]);
          f.m *= -sl[t];
        }
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        float oc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) oc[r] = __shfl_down_sync(0xffffffffu, f.c[r], off);
        const float om = __shfl_down_sync(0xffffffffu, f.m, off);
        if (lane + off < 32) {
#pragma unroll
          for (int r = 0; r < R; ++r) f.c[r] = fmaf(f.m, oc[r], f.c[r]);
          f.m = f.m * om;
        }
      }
      if (lane == 0) wtot[warp] = f;
      __syncthreads();
      float postc[R], postm = 1.0f;
#pragma unroll
      for (int r = 0; r < R; ++r) postc[r] = 0.0f;
      for (int w = SOLVE_THREADS / 32 - 1; w > warp; --w) {
        const float wm = wtot[w].m;
#pragma unroll
        for (int r = 0; r < R; ++r) postc[r] = fmaf(wm, postc[r], wtot[w].c[r]);
        postm = wm * postm;
      }
      float z[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float tot = fmaf(f.m, postc[r], f.c[r]);
        z[r] = __shfl_down_sync(0xffffffffu, tot, 1);
        if (lane == 31) z[r] = postc[r];
      }
#pragma unroll
      for (int t = EPT - 1; t >= 0; --t)
        if (t < len) {
#pragma unroll
          for (int r = 0; r < R; ++r) {
            z[r] = fmaf(-sl[t], z[r], x[r][t]);
            x[r][t] = z[r];
            zmax[r] = fmaxf(zmax[r], fabsf(z[r]));
          }
        }
    }
    // all row maxima through one pair of barriers (they also separate the row groups' use of wtot)
#pragma unroll
    for (int r = 0; r < R; ++r) zmax[r] = warp_max(zmax[r]);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r) mscratch[r][warp] = zmax[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (j0 + r >= p) break;
      const int j = j0 + r;
      const float zm = warp_max(lane < SOLVE_THREADS / 32 ? mscratch[r][lane] : 0.0f);
      float inv;
      const float sc = pow2_scale_for(zm, &inv);
      if (tid == 0) row_inv[j] = inv;
#pragma unroll
      for (int e = 0; e < EPT; e += 8) {
        if (e < len) {
          __align__(16) __half hh[8];
          __align__(16) __half ll[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) split_f16(x[r][e + k] * sc, hh[k], ll[k]);
          *reinterpret_cast<uint4*>(Yhi + (size_t)j * n + a0 + e) = *reinterpret_cast<const uint4*>(hh);
          *reinterpret_cast<uint4*>(Ylo + (size_t)j * n + a0 + e) = *reinterpret_cast<const uint4*>(ll);
        }
      }
    }
  }
}

template <int EPT, int R>
static void launch_solve_rows_t(Ctx* c, const float* Y, int p, int stage, int ctas_per_sm, bf16* hi, bf16* lo,
                                float* row_inv) {
  const size_t fs = stage_factor_stride(c->n);
  const int groups = (p + R - 1) / R;
  int blocks = c->num_sms * ctas_per_sm;
  if (blocks > groups) blocks = groups;
  if (c->n == EPT * SOLVE_THREADS)
    tridiag_solve_rows_kernel<EPT, R, true><<<blocks, SOLVE_THREADS, 0, c->stream>>>(
        Y, p, c->n, c->stage_l + (size_t)stage * fs, c->stage_invd + (size_t)stage * fs, hi, lo, row_inv);
  else
    tridiag_solve_rows_kernel<EPT, R, false><<<blocks, SOLVE_THREADS, 0, c->stream>>>(
        Y, p, c->n, c->stage_l + (size_t)stage * fs, c->stage_invd + (size_t)stage * fs, hi, lo, row_inv);
}

template <int EPT>
static void launch_solve_t(Ctx* c, const float* Y, int p, int stage, int blocks, bf16* hi, bf16* lo,
                           float* row_inv) {
  const size_t fs = stage_factor_stride(c->n);
  const size_t smem = (size_t)2 * EPT * SOLVE_THREADS * sizeof(float);
  if (ensure_dynamic_smem((const void*)tridiag_solve_kernel<EPT>, (int)smem) != cudaSuccess) return;
  tridiag_solve_kernel<EPT><<<blocks, SOLVE_THREADS, smem, c->stream>>>(
      Y, p, c->n, c->stage_l + (size_t)stage * fs, c->stage_invd + (size_t)stage * fs, hi, lo, row_inv);
}

// rows [0, p) of Y (fp32, [p][n]) -> planes hi / lo with one inverse scale per row
void launch_tridiag_solve(Ctx* c, const float* Y, int p, int stage, bf16* hi, bf16* lo, float* row_inv) {
  int blocks = c->num_sms * 3;                             // resident CTAs; each loads the factor once
  if (blocks > p) blocks = p;
  switch (solve_ept(c->n)) {
    case 8: launch_solve_rows_t<8, SOLVE_ROWS>(c, Y, p, stage, 3, hi, lo, row_inv); break;
    case 16: launch_solve_rows_t<16, SOLVE_ROWS>(c, Y, p, stage, 3, hi, lo, row_inv); break;
    case 24: launch_solve_t<24>(c, Y, p, stage, blocks, hi, lo, row_inv); break;
    case 32: launch_solve_t<32>(c, Y, p, stage, blocks, hi, lo, row_inv); break;
    case 40: launch_solve_t<40>(c, Y, p, stage, blocks, hi, lo, row_inv); break;
    case 48: launch_solve_t<48>(c, Y, p, stage, blocks, hi, lo, row_inv); break;
    default: launch_solve_t<56>(c, Y, p, stage, blocks, hi, lo, row_inv); break;     // n <= 14336
  }
  c->launches++;
}

}  // namespace admmq
