// Blocked Householder tridiagonalisation of the scaled Hessian (Algorithm 1 line 3 in its tridiagonal
// form, H~ = Q T Q^T), fp64, cooperative launch.
//
// Columns are reduced in panels of TB_NB.  Inside a panel the trailing matrix is NOT touched: column k is
// brought up to date on the fly from the panel's vectors,
//     a = A[:, k] - V W[k, :]^T - W V[k, :]^T,
// the reflector v (beta) is built from it, and
//     w = beta (A22 v - V (W^T v) - W (V^T v)) - (beta^2 / 2) (v^T A22 v - 2 (V^T v).(W^T v)) v
// so that A22 is read exactly once per column (8 bytes per element) instead of being read and written.
// While the trailing matrix is large (the panels that start with TB_SYM_MIN rows or more, in matrices of at least
// TB_SYM_N; one launch of its own) only its lower triangle is read and kept up to date: a CTA forms, from the
// entries a_rj (j <= r) of its own rows, the part  sum_{j <= r} a_rj v_j  of y_r and, per column j, the part
// sum_{own r > j} a_rj v_r  of y_j.  The column parts of all CTAs are published; after the second barrier every
// CTA adds up one block of columns (fixed order) and a third barrier hands the complete y to the rows' owners.
// 4 bytes per element and column instead of 8.  The launch for the smaller rest first mirrors the lower triangle
// into the upper one and then reads whole rows, which is faster once the matrix fits the L2.
// After the panel the trailing matrix takes the rank-2*TB_NB update A22 -= V W^T + W V^T on the fp64
// tensor-core MMA.
//
// Rows are dealt cyclically to the CTAs (row r belongs to CTA r mod G) and a CTA only ever reads and
// writes its own rows of A (the one-time mirror reads finished entries of other rows), so the matrix needs no
// grid-wide ordering at all.  What crosses CTAs is small:
// the current column and its squared norm (barrier 1), the product A22 v and the partial inner products
// with the panel (barrier 2), and the finished panel before the update (one barrier per panel).  The rows
// of V and W that later columns of the panel need (at most TB_NB of them) are rebuilt by every CTA for
// itself.  All cross-CTA sums are taken in a fixed order, so the result does not depend on timing.
// Output: td/te (diagonal / off-diagonal of T), reflector k in A[k, k+1:], beta[k].
#include <cooperative_groups.h>

#include "internal.h"

namespace cg = cooperative_groups;

namespace admmq {

constexpr int TB_NB = 32;
constexpr int TB_LDP = TB_NB + 4;            // row stride of the own-row panels: == 4 (mod 16) doubles
constexpr int TB_CB = 64;                    // columns per staged block of the trailing update
constexpr int TB_LDC = TB_CB + 4;
constexpr int TB_LDT = TB_NB + 1;            // row stride of the broadcast-row tables
constexpr int TB_PART = 2 * TB_NB + 2;       // partial inner products per CTA: W^T v, V^T v, v^T A22 v
constexpr int TB_THREADS = 1024;
constexpr int TB_PSUM = 512;
constexpr int TB_MAX_GRID = 256;
constexpr int TB_SYM_MIN = 4096;             // lower-triangle sweep for the panels that start with n - k0 >= this ...
constexpr int TB_SYM_N = 5120;               // ... in matrices of at least this size
constexpr int TB_CHUNK = 2 * TB_THREADS;     // columns per pass of the lower-triangle sweep (two per thread)

struct TrbArgs {
  double* A;
  int n;
  double* td;
  double* te;
  double* beta;
  double* colbuf;     // [n] current column, brought up to date
  double* ybuf;       // [n] A22 v
  double* part;       // [TB_PART][grid]: the partials of one inner product are contiguous
  double* normpart;   // [grid]
  double* Vg;         // [n][TB_NB] finished panel, row-major
  double* Wg;         // [n][TB_NB]
  double* colpart;    // [grid][n] column parts of A22 v from the lower-triangle sweep
  double* ycol;       // [n] complete A22 v of the lower-triangle sweep
  int rows_cap;       // own rows per CTA, rounded up to 8, plus 8
};

size_t tridiag_blocked_scratch_doubles(int n) {
  return (size_t)2 * n + (size_t)2 * n * TB_NB + (size_t)TB_MAX_GRID * (TB_PART + 1) + 64 +
         (n >= TB_SYM_N ? (size_t)TB_MAX_GRID * n + n : 0);
}

// y = A22 v from the lower triangle of A22 (own rows r = c + (tA + t) G, t < nr; columns c1 .. r).  Publishes the row
// parts (ybuf, yown) and this CTA's column parts (colpart); returns sum_j v_j (column part)_j over the block.  A
// function of its own so that its loop gets the whole register file: `vown` ([cap]) takes v at the own rows.
__device__ __noinline__ double sweep_lower(const double* __restrict__ A, double* __restrict__ colpart,
                                           double* __restrict__ ybuf, int n, const double* v, double* rowpart,
                                           double* yown, double* vown, double* scratch, int k, int c1, int tA, int nr, int cap) {
  const int G = gridDim.x, c = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // Lower triangle only.  A thread owns two adjacent columns of each TB_CHUNK-wide pass and walks down the own
  // rows four at a time: the entries (r, col..col+1) of four rows feed four row sums (reduced over the warp
  // in one transposing butterfly and kept per warp in shared memory) and the thread's two column sums.
  // rowpart: [32][cap], the staging area of the trailing update, idle here
  for (int idx = tid; idx < 32 * cap; idx += TB_THREADS) rowpart[idx] = 0.0;
  for (int t = tid; t < cap; t += TB_THREADS) vown[t] = t < nr ? v[c + (tA + t) * G] : 0.0;
  __syncthreads();
  const int i_lo = c1 & ~1;
  const int nch = (n - i_lo + TB_CHUNK - 1) / TB_CHUNK;
  const int nb4 = (nr + 3) >> 2;
  const size_t rstride2 = (size_t)G * n / 2;          // one own row further, in 16-byte units (n is even)
  const bool back = (k & 1) != 0;                    // see the full sweep below
  const bool hi16 = (lane & 16) != 0, hi8 = (lane & 8) != 0;
  double vcol = 0.0;
  for (int qq = 0; qq < nch; ++qq) {
    const int q = back ? nch - 1 - qq : qq;
    const int S = i_lo + q * TB_CHUNK;
    const int col = S + 2 * tid;
    double2 vc = make_double2(0.0, 0.0);
    if (col < n) vc = *reinterpret_cast<const double2*>(v + col);
    double2 cacc = make_double2(0.0, 0.0);
    int tlo = S - c - tA * G;                        // first own row r = c + (tA + t) G that reaches column S
    tlo = tlo > 0 ? (tlo + G - 1) / G : 0;
    const int b_lo = tlo >> 2;
    for (int bb = b_lo; bb < nb4; ++bb) {
      const int t0 = (back ? nb4 - 1 + b_lo - bb : bb) << 2;
      const int r0 = c + (tA + t0) * G;
      double2 av[4];
      double racc[4];
      if (r0 >= S + TB_CHUNK && t0 + 3 < nr) {       // all four rows lie wholly below the diagonal in this pass
        const double2* ap = reinterpret_cast<const double2*>(A + (size_t)r0 * n + col);
#pragma unroll
        for (int j = 0; j < 4; ++j) av[j] = __ldcg(ap + j * rstride2);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const double vr = vown[t0 + j];
          racc[j] = av[j].x * vc.x + av[j].y * vc.y;
          cacc.x += av[j].x * vr;
          cacc.y += av[j].y * vr;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = r0 + j * G;
          av[j] = make_double2(0.0, 0.0);
          if (t0 + j < nr && col <= r) av[j] = __ldcg(reinterpret_cast<const double2*>(A + (size_t)r * n + col));
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = r0 + j * G;
          const double vr = vown[t0 + j];              // zero beyond the last own row
          const double ay = (col + 1 <= r) ? av[j].y : 0.0;   // right of the diagonal: upper triangle
          racc[j] = av[j].x * vc.x + ay * vc.y;
          if (col < r) cacc.x += av[j].x * vr;
          if (col + 1 < r) cacc.y += ay * vr;
        }
      }
      // four sums over 32 lanes: halve the set of sums a lane carries twice, then finish over 8 lanes
      double k0s = hi16 ? racc[2] : racc[0], k1s = hi16 ? racc[3] : racc[1];
      k0s += __shfl_xor_sync(0xffffffffu, hi16 ? racc[0] : racc[2], 16);
      k1s += __shfl_xor_sync(0xffffffffu, hi16 ? racc[1] : racc[3], 16);
      double ks = hi8 ? k1s : k0s;
      ks += __shfl_xor_sync(0xffffffffu, hi8 ? k0s : k1s, 8);
      ks += __shfl_xor_sync(0xffffffffu, ks, 4);
      ks += __shfl_xor_sync(0xffffffffu, ks, 2);
      ks += __shfl_xor_sync(0xffffffffu, ks, 1);
      if ((lane & 7) == 0) rowpart[warp * cap + t0 + (lane >> 3)] += ks;   // lane 8 j holds row t0 + j
    }
    if (col < n) {
      __stcg(reinterpret_cast<double2*>(colpart + (size_t)c * n + col), cacc);
      vcol += cacc.x * vc.x + cacc.y * vc.y;
    }
  }
  __syncthreads();
  for (int t = tid; t < nr; t += TB_THREADS) {
    double s = 0.0;
#pragma unroll 8
    for (int w = 0; w < 32; ++w) s += rowpart[w * cap + t];
    ybuf[c + (size_t)(tA + t) * G] = s;
    yown[tA + t] = s;
  }
  vcol = block_sum(vcol, scratch);
  __syncthreads();
  return vcol;
}

// Panels k0 in [k_begin, k_end).  SYM: every column of these panels takes the lower-triangle sweep.
template <bool SYM>
__global__ void __launch_bounds__(TB_THREADS, 1) tridiag_blocked_kernel(TrbArgs a, int k_begin, int k_end) {
  cg::grid_group grid = cg::this_grid();
  extern __shared__ double sm[];
  __shared__ double scratch[32];
  __shared__ double bc[4];
  const int n = a.n, G = gridDim.x, c = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int cap = a.rows_cap;
  double* v = sm;                               // [n] current reflector (absolute index)
  double* Vs = v + n;                           // [cap][TB_LDP] own rows of V
  double* Ws = Vs + (size_t)cap * TB_LDP;       // [cap][TB_LDP] own rows of W
  double* Cst = Ws + (size_t)cap * TB_LDP;      // [2 TB_NB][TB_LDC] staged W^T / V^T block of the update
  double* Vt = Cst + 2 * TB_NB * TB_LDC;        // [TB_NB][TB_LDT] rows k0+1 .. of V (every CTA)
  double* Wt = Vt + TB_NB * TB_LDT;             // [TB_NB][TB_LDT] rows k0+1 .. of W
  double* red = Wt + TB_NB * TB_LDT;            // [TB_PART] W^T v | V^T v | v^T A22 v
  double* yown = red + TB_PART;                 // [cap]
  double* psum = yown + cap;                    // [TB_PSUM]
  const int Rtot = (c < n) ? (n - c + G - 1) / G : 0;       // own rows c, c + G, ...

  if (!SYM && k_begin > 0) {
    // the launch before this one kept only the lower triangle of the trailing matrix up to date: own rows take
    // their upper part from the columns below the diagonal (one pass, once)
    for (int t = warp; t < Rtot; t += 32) {
      const int r = c + t * G;
      if (r < k_begin) continue;
      for (int col = r + 1 + lane; col < n; col += 32) a.A[(size_t)r * n + col] = __ldcg(a.A + (size_t)col * n + r);
    }
    __syncthreads();
  }
  for (int k0 = k_begin; k0 < n - 2 && k0 < k_end; k0 += TB_NB) {
    const int nbk = n - 2 - k0 < TB_NB ? n - 2 - k0 : TB_NB;
    for (int i = tid; i < cap * TB_LDP; i += TB_THREADS) {
      Vs[i] = 0.0;
      Ws[i] = 0.0;
    }
    for (int i = tid; i < TB_NB * TB_LDT; i += TB_THREADS) {
      Vt[i] = 0.0;
      Wt[i] = 0.0;
    }
    __syncthreads();

    for (int i = 0; i < nbk; ++i) {
      const int k = k0 + i;
      constexpr bool sym = SYM;
      double vcolsum = 0.0;
      // ================= A: column k up to date, own rows r >= k =================
      double nrm2 = 0.0;
      if (tid < Rtot) {
        const int r = c + tid * G;
        if (r >= k) {
          double av = __ldcg(a.A + (size_t)r * n + k);
          const double* vr = Vs + (size_t)tid * TB_LDP;
          const double* wr = Ws + (size_t)tid * TB_LDP;
          const double* vk = Vt + (i > 0 ? i - 1 : 0) * TB_LDT;
          const double* wk = Wt + (i > 0 ? i - 1 : 0) * TB_LDT;
          for (int j = 0; j < i; ++j) av -= vr[j] * wk[j] + wr[j] * vk[j];
          a.colbuf[r] = av;
          if (r >= k + 2) nrm2 = av * av;
        }
      }
      nrm2 = block_sum(nrm2, scratch);
      if (tid == 0) a.normpart[c] = nrm2;
      grid.sync();
      // ================= B: reflector (identical in every CTA) =================
      if (warp == 0) {
        double t = 0.0;
        for (int b = lane; b < G; b += 32) t += __ldcg(a.normpart + b);
        t = warp_sum(t);
        if (lane == 0) bc[0] = t;
      }
      for (int idx = k + 1 + tid; idx < n; idx += TB_THREADS) v[idx] = __ldcg(a.colbuf + idx);
      __syncthreads();
      const double tail = bc[0];
      const double x0 = v[k + 1];
      double alpha = x0, bt = 0.0;
      if (tail > 0.0) {
        const double nrm = sqrt(x0 * x0 + tail);
        alpha = (x0 >= 0.0) ? -nrm : nrm;
        bt = 1.0 / (nrm * nrm - x0 * alpha);          // 2 / (v^T v)
      }
      __syncthreads();
      if (tid == 0) {
        v[k + 1] = x0 - alpha;
        if (sym) v[k] = 0.0;                              // the lower-triangle sweep starts at an even column
      }
      __syncthreads();
      if (tid < Rtot) {
        const int r = c + tid * G;
        Vs[(size_t)tid * TB_LDP + i] = (r >= k + 1) ? v[r] : 0.0;
      }
      if (c == k % G) {                                 // row k is dead: it keeps the reflector
        double* rk = a.A + (size_t)k * n;
        for (int idx = k + 1 + tid; idx < n; idx += TB_THREADS) rk[idx] = v[idx];
        if (tid == 0) {
          a.td[k] = __ldcg(a.colbuf + k);
          a.te[k] = alpha;
          a.beta[k] = bt;
        }
      }
      // ================= C: y = A22 v over own rows r >= k + 1 =================
      const int c1 = k + 1;
      int tA = (c1 - c + G - 1) / G;
      if (c1 - c <= 0) tA = 0;
      const int nr = Rtot - tA > 0 ? Rtot - tA : 0;
      if (sym) {
        vcolsum = sweep_lower(a.A, a.colpart, a.ybuf, n, v, Cst, yown, psum + 64, scratch, k, c1, tA, nr, cap);
      } else {
        const int i_lo = c1 & ~1;
        const int nseg = (n - i_lo + 255) >> 8;
        int Sf = 1;
        while (nr * Sf < 32 && Sf < nseg) Sf <<= 1;
        const int sp = (nseg + Sf - 1) / Sf;
        const int items = nr * Sf;
        // Odd columns sweep the matrix backwards (last row first, last segment first): the end of one sweep is
        // the start of the next, so whatever part of the trailing matrix the L2 still holds is read from there
        // before anything is fetched from HBM again.
        const bool back = (k & 1) != 0;
        for (int itw = warp; itw < items; itw += 32) {
          const int it = back ? items - 1 - itw : itw;
          const int rq = it / Sf, part = it - rq * Sf;
          const double* arow = a.A + (size_t)(c + (size_t)(tA + rq) * G) * n;
          double acc = 0.0;
          const int s_beg = part * sp, s_end = (part + 1) * sp < nseg ? (part + 1) * sp : nseg;
          for (int sq = s_beg; sq < s_end; ++sq) {
            const int sg = back ? s_beg + s_end - 1 - sq : sq;
            const int i0 = i_lo + (sg << 8) + lane * 2;
            double2 av[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int idx = i0 + q * 64;
              av[q] = make_double2(0.0, 0.0);
              if (idx < n) av[q] = __ldcg(reinterpret_cast<const double2*>(arow + idx));
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int idx = i0 + q * 64;
              if (idx < n) {
                const double2 v2 = *reinterpret_cast<const double2*>(v + idx);
                if (idx >= c1) acc += av[q].x * v2.x;
                acc += av[q].y * v2.y;
              }
            }
          }
          acc = warp_sum(acc);
          if (lane == 0) psum[it] = acc;
        }
        __syncthreads();
        for (int t = tid; t < nr; t += TB_THREADS) {
          double s = 0.0;
          for (int q = 0; q < Sf; ++q) s += psum[t * Sf + q];
          a.ybuf[c + (size_t)(tA + t) * G] = s;
          yown[tA + t] = s;
        }
        __syncthreads();
      }
      if (tid <= 2 * i) {                                // partial inner products over the own rows
        double s = 0.0;
        if (tid < i) {
          for (int t = 0; t < nr; ++t) s += Ws[(size_t)(tA + t) * TB_LDP + tid] * v[c + (tA + t) * G];
          a.part[(size_t)tid * G + c] = s;
        } else if (tid < 2 * i) {
          const int j = tid - i;
          for (int t = 0; t < nr; ++t) s += Vs[(size_t)(tA + t) * TB_LDP + j] * v[c + (tA + t) * G];
          a.part[(size_t)(TB_NB + j) * G + c] = s;
        } else {
          for (int t = 0; t < nr; ++t) s += yown[tA + t] * v[c + (tA + t) * G];
          a.part[(size_t)(2 * TB_NB) * G + c] = s + vcolsum;
        }
      }
      grid.sync();
      // ================= D: w, own rows and the panel's broadcast rows =================
      // sums o < i (W^T v), TB_NB + o < TB_NB + i (V^T v) and 2 TB_NB (v^T A22 v) in one round: the two halves of
      // warp w take w and TB_NB + w; the last warp, whose two are never needed (i < TB_NB), takes the third kind
      double* ybc = psum;                                // [TB_NB] complete y of the panel's broadcast rows
      if (sym) {
        // y_j = row part (its owner's) + the column parts of all CTAs.  Every CTA adds up one block of columns
        // (coalesced reads of the 148 published vectors, fixed order), publishes the complete entries, and after
        // a third barrier the owners and the panel's broadcast rows pick theirs.
        const int blk = (n - c1 + G - 1) / G;
        const int jb = c1 + c * blk;
        double* cpart = Cst;                             // [32][cap]; blk <= cap
        for (int jj = lane; jj < blk; jj += 32) {
          const int j = jb + jj;
          double s = 0.0;
          if (j < n)
            for (int b = warp; b < G; b += 32) s += __ldcg(a.colpart + (size_t)b * n + j);
          cpart[warp * cap + jj] = s;
        }
        __syncthreads();
        for (int jj = tid; jj < blk; jj += TB_THREADS) {
          const int j = jb + jj;
          if (j < n) {
            double s = __ldcg(a.ybuf + j);
#pragma unroll 8
            for (int w = 0; w < 32; ++w) s += cpart[w * cap + jj];
            a.ycol[j] = s;
          }
        }
        grid.sync();
        for (int t = tid; t < nr; t += TB_THREADS) yown[tA + t] = __ldcg(a.ycol + c + (size_t)(tA + t) * G);
        if (tid < TB_NB - i && k0 + 1 + i + tid < n) ybc[i + tid] = __ldcg(a.ycol + k0 + 1 + i + tid);
      }
      {
        const int half = lane >> 4, sub = lane & 15;
        int o = warp + TB_NB * half;
        if (warp == 31) o = 2 * TB_NB;                   // both halves: the same sum, written once
        const bool need = (o < TB_NB) ? (o < i) : (o < 2 * TB_NB ? (o - TB_NB < i) : true);
        double s = 0.0;
        if (need)
          for (int b = sub; b < G; b += 16) s += __ldcg(a.part + (size_t)o * G + b);
        s += __shfl_xor_sync(0xffffffffu, s, 8);
        s += __shfl_xor_sync(0xffffffffu, s, 4);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        if (need && sub == 0 && (warp != 31 || half == 0)) red[o] = s;
      }
      __syncthreads();
      const double* Wv = red;                            // W^T v
      const double* Vv = red + TB_NB;                    // V^T v
      double vyc = red[2 * TB_NB];
      for (int j = 0; j < i; ++j) vyc -= 2.0 * Vv[j] * Wv[j];
      const double al = 0.5 * bt * bt * vyc;
      if (tid < Rtot && tid >= tA) {
        const int r = c + tid * G;
        const double* vr = Vs + (size_t)tid * TB_LDP;
        double* wr = Ws + (size_t)tid * TB_LDP;
        double yc = yown[tid];
        for (int j = 0; j < i; ++j) yc -= vr[j] * Wv[j] + wr[j] * Vv[j];
        wr[i] = bt * yc - al * v[r];
      }
      if (tid >= TB_THREADS - TB_NB) {                   // rows k0+1+tr of V and W for the later columns
        const int tr = tid - (TB_THREADS - TB_NB);
        const int row = k0 + 1 + tr;
        if (tr >= i && row < n) {
          double* vt = Vt + tr * TB_LDT;
          double* wt = Wt + tr * TB_LDT;
          double yc = sym ? ybc[tr] : __ldcg(a.ybuf + row);
          for (int j = 0; j < i; ++j) yc -= vt[j] * Wv[j] + wt[j] * Vv[j];
          vt[i] = v[row];
          wt[i] = bt * yc - al * v[row];
        }
      }
      __syncthreads();
    }

    // ================= panel end: A22 -= V W^T + W V^T on rows / columns >= kn =================
    const int kn = k0 + nbk;
    int t0 = (kn - c + G - 1) / G;
    if (kn - c <= 0) t0 = 0;
    const int Ract = Rtot - t0 > 0 ? Rtot - t0 : 0;
    for (int idx = tid; idx < Ract * TB_NB; idx += TB_THREADS) {
      const int t = idx / TB_NB, j = idx - t * TB_NB;
      const size_t r = c + (size_t)(t0 + t) * G;
      a.Vg[r * TB_NB + j] = Vs[(size_t)(t0 + t) * TB_LDP + j];
      a.Wg[r * TB_NB + j] = Ws[(size_t)(t0 + t) * TB_LDP + j];
    }
    grid.sync();
    const int nrt = (Ract + 7) >> 3;
    for (int cs = (kn / TB_CB) * TB_CB; cs < n; cs += TB_CB) {
      // SYM: only the lower triangle is kept up to date -- the tiles of 8 own rows whose largest row reaches
      // this block of columns
      int rt_lo = 0;
      if (SYM) {
        const int need = cs - c - (t0 + 7) * G;
        rt_lo = need > 0 ? (need + 8 * G - 1) / (8 * G) : 0;
        if (rt_lo >= nrt) continue;
      }
      for (int idx = tid; idx < 2 * TB_NB * TB_CB; idx += TB_THREADS) {
        const int cc = idx >> 6, jj = idx & 63;          // jj fastest: 32 contiguous doubles of one panel row
        const int col = cs + cc;
        double val = 0.0;
        if (col >= kn && col < n)
          val = (jj < TB_NB) ? __ldcg(a.Wg + (size_t)col * TB_NB + jj) : __ldcg(a.Vg + (size_t)col * TB_NB + jj - TB_NB);
        Cst[jj * TB_LDC + cc] = val;
      }
      __syncthreads();
      for (int u = warp; u < (nrt - rt_lo) * (TB_CB / 8); u += 32) {
        const int rt = rt_lo + (u >> 3), nt = u & 7;
        if (SYM && cs + nt * 8 > c + (t0 + rt * 8 + 7) * G) continue;   // tile wholly above the diagonal
        const int rq = rt * 8 + gid;
        const int cc = cs + nt * 8 + 2 * tig;
        const bool live = (rq < Ract) && (cc < n);       // n is even: cc + 1 < n as well
        const int rl = t0 + (rq < Ract ? rq : 0);
        double* xp = a.A + (size_t)(c + (size_t)rl * G) * n + cc;
        double2 cv = make_double2(0.0, 0.0);
        if (live) cv = __ldcg(reinterpret_cast<const double2*>(xp));
        const double* va = Vs + (size_t)rl * TB_LDP + tig;
        const double* wa = Ws + (size_t)rl * TB_LDP + tig;
        const double* cb = Cst + tig * TB_LDC + nt * 8 + gid;
#pragma unroll
        for (int kk = 0; kk < TB_NB; kk += 4) dmma_8x8x4(cv.x, cv.y, -va[kk], cb[kk * TB_LDC]);
#pragma unroll
        for (int kk = 0; kk < TB_NB; kk += 4) dmma_8x8x4(cv.x, cv.y, -wa[kk], cb[(TB_NB + kk) * TB_LDC]);
        if (live) __stcg(reinterpret_cast<double2*>(xp), cv);
      }
      __syncthreads();
    }
  }
  // the last 2 x 2 block, held by the owners of rows n-2 and n-1
  if (tid == 0 && k_end >= n - 2) {
    if (c == (n - 2) % G) {
      a.td[n - 2] = __ldcg(a.A + (size_t)(n - 2) * n + (n - 2));
      a.te[n - 2] = __ldcg(a.A + (size_t)(n - 2) * n + (n - 1));
      a.beta[n - 2] = 0.0;
    }
    if (c == (n - 1) % G) {
      a.td[n - 1] = __ldcg(a.A + (size_t)(n - 1) * n + (n - 1));
      a.te[n - 1] = 0.0;
      a.beta[n - 1] = 0.0;
    }
  }
}

cudaError_t tridiag_reduce_blocked(Ctx* c) {
  const int n = c->n;
  int blocks = c->num_sms < TB_MAX_GRID ? c->num_sms : TB_MAX_GRID;
  TrbArgs a;
  a.A = c->A64;
  a.n = n;
  a.td = c->td;
  a.te = c->te;
  a.beta = c->beta;
  double* w = c->trd_ws;
  a.colbuf = w;
  a.ybuf = w + n;
  a.Vg = w + 2 * (size_t)n;
  a.Wg = a.Vg + (size_t)n * TB_NB;
  a.part = a.Wg + (size_t)n * TB_NB;
  a.normpart = a.part + (size_t)TB_MAX_GRID * TB_PART;
  a.colpart = a.normpart + TB_MAX_GRID + 64;
  a.ycol = a.colpart + (size_t)TB_MAX_GRID * n;
  a.rows_cap = ((((n + blocks - 1) / blocks) + 7) & ~7) + 8;
  // the lower-triangle sweep keeps 32 x rows_cap row sums in the update's staging area and needs n even
  const bool sym_ok = n >= TB_SYM_N && 32 * a.rows_cap <= 2 * TB_NB * TB_LDC && (n & 1) == 0;
  // panels whose first column still has n - k0 >= the threshold take the lower-triangle sweep
  const int k_switch = sym_ok ? ((n - TB_SYM_MIN) / TB_NB + 1) * TB_NB : 0;
  const size_t doubles = (size_t)n + (size_t)2 * a.rows_cap * TB_LDP + 2 * TB_NB * TB_LDC + 2 * TB_NB * TB_LDT +
                         TB_PART + a.rows_cap + TB_PSUM;
  const size_t smem = doubles * sizeof(double);
  if (smem > (size_t)226 * 1024) return cudaErrorInvalidConfiguration;   // caller takes the unblocked kernel
  const void* kernels[2] = {(const void*)tridiag_blocked_kernel<true>, (const void*)tridiag_blocked_kernel<false>};
  int begin[2] = {0, k_switch}, end[2] = {k_switch, n};
  for (int q = 0; q < 2; ++q) {
    if (begin[q] >= end[q] || begin[q] >= n - 2) continue;
    cudaError_t e = cudaFuncSetAttribute(kernels[q], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernels[q], TB_THREADS, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    void* args[] = {&a, &begin[q], &end[q]};
    e = cudaLaunchCooperativeKernel(kernels[q], dim3(blocks), dim3(TB_THREADS), args, smem, c->stream);
    c->launches++;
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace admmq
