// Shared device helpers for the ADMM-Q kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace admmq {

// Device status codes: numerically equal to admmq_status in admmq.h.
constexpr int ST_OK = 0, ST_NOT_SPD = 5, ST_NONFINITE = 6, ST_TIMEOUT = 7;

// First error wins; the word stays 0 on success.
__device__ __forceinline__ void raise_status(int* status, int code) { atomicCAS(status, 0, code); }

// a ~= hi + lo with hi = bf16(a), lo = bf16(a - hi): 16 mantissa bits in two tensor-core operands.
__device__ __forceinline__ void split_bf16(float a, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(a);
  lo = __float2bfloat16_rn(a - __bfloat162float(hi));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block, result in every thread.  `scratch` holds >= 32 elements.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();  // scratch may still be read from a previous call
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  T t = (lane < nw) ? scratch[lane] : T(0);
  t = warp_sum(t);
  return t;
}

}  // namespace admmq
