// Shared device helpers for the ADMM-Q kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
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

// fp16 counterpart for operands that were first multiplied by a power of two which brings their
// largest magnitude to [2^13, 2^14): a ~= hi + lo keeps 22 mantissa bits for every element within
// 2^17 of that maximum (lo stays a normal fp16 number), and 2^-25 absolute below.  The clamp only
// guards the conversion against non-finite results.
__device__ __forceinline__ void split_f16(float a, __half& hi, __half& lo) {
  a = fminf(fmaxf(a, -60000.0f), 60000.0f);
  hi = __float2half_rn(a);
  lo = __float2half_rn(a - __half2float(hi));
}
// Power of two S with maxabs * S in [2^13, 2^14); 1 for a zero or non-finite maximum.  *inv = 1 / S.
__device__ __forceinline__ float pow2_scale_for(float maxabs, float* inv) {
  if (!(maxabs > 0.0f) || !isfinite(maxabs)) {
    *inv = 1.0f;
    return 1.0f;
  }
  int e;
  frexpf(maxabs, &e);
  *inv = ldexpf(1.0f, e - 14);
  return ldexpf(1.0f, 14 - e);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Maximum over the block, result in every thread.  `scratch` holds >= 32 floats.
__device__ __forceinline__ float block_max(float v, float* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  float t = (lane < nw) ? scratch[lane] : 0.0f;
  return warp_max(t);
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

// D (8x8, fp64) += A (8x4) B (4x8) on the fp64 tensor-core MMA.  Lane l holds A[l / 4][l % 4],
// B[l % 4][l / 4] and D[l / 4][2 (l % 4) .. + 1].
__device__ __forceinline__ void dmma_8x8x4(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d0), "+d"(d1)
               : "d"(a), "d"(b));
}

// Maximum of a double over the block, result in every thread.  `scratch` holds >= 32 doubles.
__device__ __forceinline__ double block_max_f64(double v, double* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  double t = (lane < nw) ? scratch[lane] : -INFINITY;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t = fmax(t, __shfl_xor_sync(0xffffffffu, t, o));
  return t;
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
