// Greedy single-entry local search (Sec. 3.5; Eq. 11 with the second perturbation zero).
// One CTA per output channel: its gradient g = H (w_q - w_hat), its codes and diag(H) stay in shared
// memory (the diagonal as Delta_i^2 H_ii, the quadratic term of a move); every step scans the 2 n
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

__global__ void __launch_bounds__(512)
local_search_kernel(const float* __restrict__ H, const float* __restrict__ hdiag, int n, int p, int gs,
                    int kmax, long long max_moves, float tau, const float* __restrict__ W0,
                    unsigned char* __restrict__ codes, const float* __restrict__ delta,
                    const float* __restrict__ zero, float* __restrict__ Wq, float* __restrict__ g_glob,
                    long long* __restrict__ moves_out, int* __restrict__ capped_out) {
  extern __shared__ float smf[];
  float* g = smf;                  // [n]
  float* quad = smf + n;           // [n]  Delta_i^2 H_ii, the quadratic term of a move of entry i
  float* sdl = smf + 2 * n;        // [n / gs]  this channel's Delta per group
  unsigned char* kc = (unsigned char*)(smf + 2 * n + n / gs);   // [n]
  __shared__ Cand wbest[16];
  __shared__ Cand chosen;
  const int j = blockIdx.x;
  if (j >= p) return;
  const int ng = n / gs;
  const float* dl = delta + (long long)j * ng;
  const int shift = (gs & (gs - 1)) == 0 ? __ffs(gs) - 1 : -1;   // group of entry i: i >> shift, or i / gs
  for (int i = threadIdx.x; i < ng; i += blockDim.x) sdl[i] = dl[i];
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const float d = dl[i / gs];
    g[i] = g_glob[(long long)j * n + i];
    quad[i] = d * d * hdiag[i];
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
    // a thread meets its candidates in increasing index order, so a strict "<" keeps the earliest;
    // four consecutive entries per step (n is a multiple of 8)
    for (int i4 = threadIdx.x * 4; i4 < n; i4 += blockDim.x * 4) {
      float4 g4 = *reinterpret_cast<const float4*>(g + i4);
      const float4 q4 = *reinterpret_cast<const float4*>(quad + i4);
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
        const float cp = lin + qv[e], cm = qv[e] - lin;
        if (kv[e] < kmax && cp < best.cost) {
          best.cost = cp;
          best.idx = 2 * i;
        }
        if (kv[e] > 0 && cm < best.cost) {
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
      best = better(best, other);
    }
    if (lane == 0) wbest[wid] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
      Cand b = wbest[0];
      for (int w = 1; w < nw; ++w) b = better(b, wbest[w]);
      if (b.idx != 0x7fffffff) {
        const int i = b.idx >> 1;
        if (!(b.cost < -tau * quad[i])) b.idx = -1;         // no improving move: stop
      } else {
        b.idx = -1;
      }
      chosen = b;
    }
    __syncthreads();
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
  const size_t smem = (size_t)n * 9 + (size_t)(n / gs) * 4 + 16;
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
