// Greedy single-entry local search (Sec. 3.5; Eq. 11 with the second perturbation zero).
// One CTA per output channel: its gradient g = H (w_q - w_hat) and its codes stay in shared memory (the
// quadratic term of a move, Delta_i^2 H_ii, is formed from the cached diagonal on the fly: five bytes per entry
// instead of nine let more channels share an SM); every step scans the 2 n
// candidate moves, a block-wide argmin picks the best one, and the gradient takes the rank-1 correction g += d H[:, i] (row i of the symmetric H, contiguous).
#include "internal.h"

namespace admmq {

struct Cand {
  float cost;
  int idx;   // 2 * i + (0 for +Delta, 1 for -Delta); ties resolve to the smallest idx
};

__device__ __forceinline__ Cand better(Cand a, Cand b) {
  if (b.cost < a.cost || (b.cost == a.cost && b.idx < a.idx)) return b;
  return a;
}

// Near-ties are settled exactly.  The scan works on an fp32 gradient that has taken hundreds of rank-1
// corrections (and started from a product of 22-bit operands): good to ~1e-6 of a move's cost, which decides
// the order of two candidates whose costs differ by less than that.  Such a misorder is harmless for the loss
// but sends the search to another local optimum.  So the scan also keeps the second-smallest cost, and whenever
// that is within TIE_MARGIN of the smallest, or the smallest is within TIE_MARGIN of the acceptance threshold,
// the candidates in that margin are collected, the entries of the gradient they need are recomputed from their
// definition g_i = sum_k H_ik (w_q - w_hat)_k in fp64, and the decision is taken on those values.
constexpr float TIE_MARGIN = 1e-4f;
constexpr int TIE_SLOTS = 8;

__global__ void __launch_bounds__(512)
local_search_kernel(const float* __restrict__ H, const float* __restrict__ hdiag, int n, int p, int gs,
                    int kmax, long long max_moves, float tau, const float* __restrict__ W0,
                    unsigned char* __restrict__ codes, const float* __restrict__ delta,
                    const float* __restrict__ zero, float* __restrict__ Wq, float* __restrict__ g_glob,
                    long long* __restrict__ moves_out, int* __restrict__ capped_out) {
  extern __shared__ float smf[];
  float* g = smf;                  // [n]
  float* sdl = smf + n;            // [n / gs]  this channel's Delta per group
  float* szr = sdl + n / gs;       // [n / gs]  this channel's z0 per group
  unsigned char* kc = (unsigned char*)(szr + n / gs);   // [n]
  __shared__ Cand wbest[16];
  __shared__ float wsecond[16];
  __shared__ Cand chosen;
  __shared__ float tie_limit;      // candidates with a cost up to this value are settled exactly; < 0 cost scale: see below
  __shared__ int tie_on, tie_count;
  __shared__ int tie_idx[TIE_SLOTS];
  __shared__ double tie_g[TIE_SLOTS];
  __shared__ double dscratch[32];
  const int j = blockIdx.x;
  if (j >= p) return;
  const int ng = n / gs;
  const float* dl = delta + (long long)j * ng;
  const float* w0 = W0 + (long long)j * n;
  const int shift = (gs & (gs - 1)) == 0 ? __ffs(gs) - 1 : -1;   // group of entry i: i >> shift, or i / gs
  for (int i = threadIdx.x; i < ng; i += blockDim.x) {
    sdl[i] = dl[i];
    szr[i] = zero[(long long)j * ng + i];
  }
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    g[i] = g_glob[(long long)j * n + i];
    kc[i] = codes[(long long)j * n + i];
  }
  __syncthreads();
  long long moves = 0;
  int capped = 0;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  // The gradient update of the move just applied and the scan for the next move share one sweep over the
  // entries: d_move = 0 on the first sweep (nothing to apply yet).
  int i_move = -1, k_step = 0;
  float d_move = 0.0f;
  const float* hrow = H;
  while (true) {
    Cand best;
    best.cost = INFINITY;
    best.idx = 0x7fffffff;
    float second = INFINITY;       // second-smallest cost met by this thread
    // a thread meets its candidates in increasing index order, so a strict "<" keeps the earliest;
    // four consecutive entries per step (n is a multiple of 8)
    for (int i4 = threadIdx.x * 4; i4 < n; i4 += blockDim.x * 4) {
      float4 g4 = *reinterpret_cast<const float4*>(g + i4);
      const float4 q4 = __ldg(reinterpret_cast<const float4*>(hdiag + i4));   // H_ii; times Delta_i^2 below
      uchar4 k4 = *reinterpret_cast<const uchar4*>(kc + i4);
      if (i_move >= 0) {
        const float4 h4 = *reinterpret_cast<const float4*>(hrow + i4);   // g += d H[:, i_move] (H symmetric)
        g4.x = fmaf(d_move, h4.x, g4.x);
        g4.y = fmaf(d_move, h4.y, g4.y);
        g4.z = fmaf(d_move, h4.z, g4.z);
        g4.w = fmaf(d_move, h4.w, g4.w);
        *reinterpret_cast<float4*>(g + i4) = g4;
        if ((i_move & ~3) == i4) {
          const int e = i_move & 3;
          if (e == 0) k4.x = (unsigned char)((int)k4.x + k_step);
          if (e == 1) k4.y = (unsigned char)((int)k4.y + k_step);
          if (e == 2) k4.z = (unsigned char)((int)k4.z + k_step);
          if (e == 3) k4.w = (unsigned char)((int)k4.w + k_step);
          *reinterpret_cast<uchar4*>(kc + i4) = k4;
        }
      }
      const float gv[4] = {g4.x, g4.y, g4.z, g4.w};
      const float qv[4] = {q4.x, q4.y, q4.z, q4.w};
      const int kv[4] = {k4.x, k4.y, k4.z, k4.w};
      float d = sdl[shift >= 0 ? (i4 >> shift) : (i4 / gs)];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = i4 + e;
        if (e > 0 && (gs & 3) != 0) d = sdl[shift >= 0 ? (i >> shift) : (i / gs)];
        const float lin = 2.0f * d * gv[e];
        const float qd = d * d * qv[e];                     // Delta_i^2 H_ii, the quadratic term of a move of entry i
        const float cp = kv[e] < kmax ? lin + qd : INFINITY;
        const float cm = kv[e] > 0 ? qd - lin : INFINITY;
        second = fminf(second, fmaxf(cp, best.cost));
        if (cp < best.cost) {
          best.cost = cp;
          best.idx = 2 * i;
        }
        second = fminf(second, fmaxf(cm, best.cost));
        if (cm < best.cost) {
          best.cost = cm;
          best.idx = 2 * i + 1;
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Cand other;
      other.cost = __shfl_xor_sync(0xffffffffu, best.cost, o);
      other.idx = __shfl_xor_sync(0xffffffffu, best.idx, o);
      const float osec = __shfl_xor_sync(0xffffffffu, second, o);
      second = fminf(fminf(second, osec), fmaxf(best.cost, other.cost));
      best = better(best, other);
    }
    if (lane == 0) {
      wbest[wid] = best;
      wsecond[wid] = second;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      Cand b = wbest[0];
      float sec = wsecond[0];
      for (int w = 1; w < nw; ++w) {
        sec = fminf(fminf(sec, wsecond[w]), fmaxf(b.cost, wbest[w].cost));
        b = better(b, wbest[w]);
      }
      tie_on = 0;
      tie_count = 0;
      if (b.idx != 0x7fffffff) {
        const int i = b.idx >> 1;
        const float di = sdl[shift >= 0 ? (i >> shift) : (i / gs)];
        const float qi = di * di * hdiag[i];
        const float thr = -tau * qi;
        const float tol = TIE_MARGIN * fmaxf(fabsf(b.cost), qi);
        if (sec - b.cost <= tol || fabsf(b.cost - thr) <= tol) {   // too close to call in fp32
          tie_on = 1;
          tie_limit = b.cost + tol;
        }
        if (!(b.cost < thr)) b.idx = -1;                    // no improving move: stop
      } else {
        b.idx = -1;
      }
      chosen = b;
    }
    __syncthreads();
    if (tie_on) {
      // collect the candidates within the margin (the gradient already holds the last move's correction)
      const float lim = tie_limit;
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float d = sdl[shift >= 0 ? (i >> shift) : (i / gs)];
        const float lin = 2.0f * d * g[i];
        const int k = kc[i];
        const float qi = d * d * hdiag[i];
        if (k < kmax && lin + qi <= lim) {
          const int slot = atomicAdd(&tie_count, 1);
          if (slot < TIE_SLOTS) tie_idx[slot] = 2 * i;
        }
        if (k > 0 && qi - lin <= lim) {
          const int slot = atomicAdd(&tie_count, 1);
          if (slot < TIE_SLOTS) tie_idx[slot] = 2 * i + 1;
        }
      }
      __syncthreads();
      // more candidates than slots (many equal costs): the fp32 choice, smallest index first, stands
      const int nc = tie_count <= TIE_SLOTS ? tie_count : 0;
      // g_i = sum_k H_ik e_k, e = w_q - w_hat of this channel as it stands, for every row in question
      for (int q = 0; q < nc; ++q) {
        const float* hq = H + (long long)(tie_idx[q] >> 1) * n;
        double acc = 0.0;
        for (int k = threadIdx.x; k < n; k += blockDim.x) {
          const int gq = shift >= 0 ? (k >> shift) : (k / gs);
          const double e = fma((double)sdl[gq], (double)kc[k], (double)szr[gq]) - (double)w0[k];
          acc = fma(e, (double)hq[k], acc);
        }
        acc = block_sum(acc, dscratch);
        if (threadIdx.x == 0) tie_g[q] = acc;
      }
      __syncthreads();
      if (threadIdx.x == 0 && nc > 0) {
        Cand pick;
        pick.idx = -1;
        pick.cost = 0.0f;
        double cbest = INFINITY;
        for (int q = 0; q < nc; ++q) {
          const int idx = tie_idx[q], i = idx >> 1;
          const double d = ((idx & 1) ? -1.0 : 1.0) * (double)sdl[shift >= 0 ? (i >> shift) : (i / gs)];
          const double c = 2.0 * d * tie_g[q] + d * d * (double)hdiag[i];
          if (c < cbest || (c == cbest && idx < pick.idx)) {
            cbest = c;
            pick.idx = idx;
          }
          g[i] = (float)tie_g[q];                           // the recomputed entry replaces the drifted one
        }
        if (pick.idx >= 0) {
          const int i = pick.idx >> 1;
          const double d = (double)sdl[shift >= 0 ? (i >> shift) : (i / gs)];
          if (!(cbest < -(double)tau * (double)hdiag[i] * d * d)) pick.idx = -1;
        }
        chosen = pick;
      }
      __syncthreads();
    }
    const Cand c = chosen;
    if (moves >= max_moves) {                              // the move that reached the cap has been applied
      capped = 1;
      break;
    }
    if (c.idx < 0) break;
    i_move = c.idx >> 1;
    k_step = (c.idx & 1) ? -1 : 1;
    d_move = (float)k_step * dl[i_move / gs];
    hrow = H + (long long)i_move * n;
    ++moves;
  }
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const long long idx = (long long)j * n + i;
    codes[idx] = kc[i];
    g_glob[idx] = g[i];
    if (Wq) Wq[idx] = zero[(long long)j * ng + i / gs] + dl[i / gs] * (float)kc[i];
  }
  if (threadIdx.x == 0) {
    atomicAdd((unsigned long long*)moves_out, (unsigned long long)moves);
    if (capped) atomicAdd(capped_out, 1);
  }
}

cudaError_t launch_local_search(Ctx* c, const float* W0, int p, int bits, int gs, long long max_moves,
                                float tau, unsigned char* codes, const float* delta, const float* zero,
                                float* Wq, float* g, long long* d_moves, int* d_capped) {
  const int n = c->n;
  const size_t smem = (size_t)n * 5 + (size_t)(n / gs) * 8 + 16;
  const int threads = n >= 8192 ? 512 : 256;               // long rows: more warps per channel
  cudaError_t e = cudaFuncSetAttribute(local_search_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  local_search_kernel<<<p, threads, smem, c->stream>>>(c->H, c->hdiag, n, p, gs, (1 << bits) - 1, max_moves,
                                                   tau, W0, codes, delta, zero, Wq, g, d_moves, d_capped);
  c->launches++;
  return cudaGetLastError();
}

}  // namespace admmq
