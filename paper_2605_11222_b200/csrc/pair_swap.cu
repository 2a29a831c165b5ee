// Pair-swap local search (Sec. 3.5 "Algorithm"; Eq. 11 with both perturbations).
// A round evaluates a batch of candidate row pairs: for a pair (i1, i2) every output channel picks the best
// of the four sign combinations (+-Delta on each of the two entries) that keep both codes in range, and
// takes part only if that lowers its loss; the pair's total is the sum over the channels that take part.
// The pair with the smallest total is applied in those channels and the gradient g = H (w_q - w_hat) takes
// the rank-2 correction g += d1 H[:, i1] + d2 H[:, i2].  The candidate pairs are an input (the caller draws
// them), so the pass is deterministic.
#include "internal.h"

namespace admmq {

// Best feasible sign combination of one channel for the pair; combinations are tried in the order
// (+,+), (+,-), (-,+), (-,-) and the first minimum wins.  Returns the combination (0..3) or -1 when the
// channel declines (no feasible combination lowers the loss by more than tau (d1^2 H11 + d2^2 H22)).
__device__ __forceinline__ int best_pair_move(float g1, float g2, float h11, float h22, float h12, float d1,
                                              float d2, int k1, int k2, int kmax, float tau, float* cost) {
  const float q = d1 * d1 * h11 + d2 * d2 * h22;
  const float l1 = 2.0f * d1 * g1, l2 = 2.0f * d2 * g2, x = 2.0f * d1 * d2 * h12;
  const float c[4] = {l1 + l2 + q + x, l1 - l2 + q - x, -l1 + l2 + q - x, -l1 - l2 + q + x};
  const bool up1 = k1 < kmax, dn1 = k1 > 0, up2 = k2 < kmax, dn2 = k2 > 0;
  const bool ok[4] = {up1 && up2, up1 && dn2, dn1 && up2, dn1 && dn2};
  float best = INFINITY;
  int which = -1;
#pragma unroll
  for (int s = 0; s < 4; ++s)
    if (ok[s] && c[s] < best) {
      best = c[s];
      which = s;
    }
  *cost = best;
  if (which < 0 || !(best < -tau * q)) return -1;
  return which;
}

__global__ void __launch_bounds__(256)
pair_eval_kernel(const float* __restrict__ H, const float* __restrict__ hdiag, int n, int p, int gs, int kmax,
                 float tau, const unsigned char* __restrict__ codes, const float* __restrict__ delta,
                 const float* __restrict__ g, const int* __restrict__ pairs, double* __restrict__ totals) {
  __shared__ double scratch[32];
  const int b = blockIdx.x;
  const int i1 = pairs[2 * b], i2 = pairs[2 * b + 1];
  if (i1 == i2 || i1 < 0 || i2 < 0 || i1 >= n || i2 >= n) {          // not a pair: never chosen
    if (threadIdx.x == 0) totals[b] = 0.0;
    return;
  }
  const int ng = n / gs;
  const float h11 = hdiag[i1], h22 = hdiag[i2], h12 = H[(size_t)i1 * n + i2];
  double acc = 0.0;
  for (int j = threadIdx.x; j < p; j += blockDim.x) {
    const size_t r = (size_t)j * n;
    float cost;
    const int w = best_pair_move(g[r + i1], g[r + i2], h11, h22, h12, delta[(size_t)j * ng + i1 / gs],
                                 delta[(size_t)j * ng + i2 / gs], codes[r + i1], codes[r + i2], kmax, tau, &cost);
    if (w >= 0) acc += (double)cost;
  }
  acc = block_sum(acc, scratch);
  if (threadIdx.x == 0) totals[b] = acc;
}

// Smallest total, first in the batch on ties; -1 when no total is negative.
__global__ void pair_select_kernel(const double* __restrict__ totals, int batch, int* __restrict__ chosen) {
  __shared__ double sv[256];
  __shared__ int si[256];
  double best = 0.0;
  int bi = -1;
  for (int b = threadIdx.x; b < batch; b += blockDim.x) {
    const double t = totals[b];
    if (t < best) {
      best = t;
      bi = b;
    }
  }
  sv[threadIdx.x] = best;
  si[threadIdx.x] = bi;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int t = 1; t < (int)blockDim.x; ++t)
      if (si[t] >= 0 && (sv[t] < best || (sv[t] == best && (bi < 0 || si[t] < bi)))) {
        best = sv[t];
        bi = si[t];
      }
    chosen[0] = bi;
  }
}

__global__ void __launch_bounds__(256)
pair_apply_kernel(const float* __restrict__ H, const float* __restrict__ hdiag, int n, int p, int gs, int kmax,
                  float tau, unsigned char* __restrict__ codes, const float* __restrict__ delta,
                  const float* __restrict__ zero, float* __restrict__ Wq, const float* __restrict__ g,
                  const int* __restrict__ pairs, const int* __restrict__ chosen, float* __restrict__ d1buf,
                  float* __restrict__ d2buf, long long* __restrict__ moves, int* __restrict__ rounds_applied) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = chosen[0];
  if (j >= p) return;
  d1buf[j] = 0.0f;
  d2buf[j] = 0.0f;
  if (b < 0) return;
  const int i1 = pairs[2 * b], i2 = pairs[2 * b + 1];
  const int ng = n / gs;
  const size_t r = (size_t)j * n;
  const float dl1 = delta[(size_t)j * ng + i1 / gs], dl2 = delta[(size_t)j * ng + i2 / gs];
  float cost;
  const int w = best_pair_move(g[r + i1], g[r + i2], hdiag[i1], hdiag[i2], H[(size_t)i1 * n + i2], dl1, dl2,
                               codes[r + i1], codes[r + i2], kmax, tau, &cost);
  if (j == 0) atomicAdd(rounds_applied, 1);
  if (w < 0) return;
  const int a1 = (w < 2) ? 1 : -1, a2 = (w & 1) ? -1 : 1;
  const int k1 = (int)codes[r + i1] + a1, k2 = (int)codes[r + i2] + a2;
  codes[r + i1] = (unsigned char)k1;
  codes[r + i2] = (unsigned char)k2;
  if (Wq) {
    Wq[r + i1] = zero[(size_t)j * ng + i1 / gs] + dl1 * (float)k1;
    Wq[r + i2] = zero[(size_t)j * ng + i2 / gs] + dl2 * (float)k2;
  }
  d1buf[j] = (float)a1 * dl1;
  d2buf[j] = (float)a2 * dl2;
  atomicAdd((unsigned long long*)moves, 1ULL);
}

// g[j, :] += d1[j] H[i1, :] + d2[j] H[i2, :]
__global__ void __launch_bounds__(256)
pair_gradient_kernel(const float* __restrict__ H, int n, int p, const int* __restrict__ pairs,
                     const int* __restrict__ chosen, const float* __restrict__ d1buf,
                     const float* __restrict__ d2buf, float* __restrict__ g) {
  const int b = chosen[0];
  if (b < 0) return;
  const float* h1 = H + (size_t)pairs[2 * b] * n;
  const float* h2 = H + (size_t)pairs[2 * b + 1] * n;
  // channels on grid.x (any d_out), column segments on grid.y
  for (int j = blockIdx.x; j < p; j += gridDim.x) {
    const float d1 = d1buf[j], d2 = d2buf[j];
    if (d1 == 0.0f && d2 == 0.0f) continue;
    float* gr = g + (size_t)j * n;
    for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < n; i += gridDim.y * blockDim.x)
      gr[i] = fmaf(d2, h2[i], fmaf(d1, h1[i], gr[i]));
  }
}

cudaError_t launch_pair_round(Ctx* c, int p, int bits, int gs, float tau, unsigned char* codes,
                              const float* delta, const float* zero, float* Wq, float* g, const int* pairs,
                              int batch, long long* d_moves, int* d_rounds) {
  const int n = c->n, kmax = (1 << bits) - 1;
  pair_eval_kernel<<<batch, 256, 0, c->stream>>>(c->H, c->hdiag, n, p, gs, kmax, tau, codes, delta, g, pairs,
                                                 c->ps_totals);
  pair_select_kernel<<<1, 256, 0, c->stream>>>(c->ps_totals, batch, c->ps_chosen);
  pair_apply_kernel<<<(p + 255) / 256, 256, 0, c->stream>>>(c->H, c->hdiag, n, p, gs, kmax, tau, codes, delta,
                                                            zero, Wq, g, pairs, c->ps_chosen, c->ps_d,
                                                            c->ps_d + p, d_moves, d_rounds);
  dim3 grid(p, (n + 1023) / 1024);
  pair_gradient_kernel<<<grid, 256, 0, c->stream>>>(c->H, n, p, pairs, c->ps_chosen, c->ps_d, c->ps_d + p, g);
  c->launches += 4;
  return cudaGetLastError();
}

}  // namespace admmq
