// admmq_objective_static: the layer error Tr(E^T H E) for callers that cannot allocate device memory.
//
// Who that is: a quantization job that shares its GPU with a serving engine which has already handed
// every free byte of HBM to its own memory pool (cudaMalloc would fail or evict), a plug-in running
// under a host framework whose rules forbid driver allocations outside its arena, or a monitoring
// thread that must not trigger the implicit device-wide synchronisation an allocation can cause.
// Such a caller already owns its inputs (H, the weights, the codes, the grid) and one double for the
// result; what it lacks is the per-channel scratch the reduction needs.  That scratch lives here, in
// a fixed array inside the library image.
//
// Consequences the caller must know about:
//  * the array is ADMMQ_STATIC_MAX_D_OUT doubles (128 KiB) of device memory on every GPU that loads
//    the library, held until the process exits;
//  * it is shared by every call, from every thread and stream: two calls that overlap on the GPU
//    race on it.  Serialise them (one stream, or an event between them);
//  * it keeps the previous call's contents.  Nothing has to be cleared: a call with d_out channels
//    writes entries [0, d_out) before its second kernel reads exactly those;
//  * the first call on each device looks the array's device address up (cudaGetSymbolAddress) and
//    raises the kernel's shared-memory limit.  Make that first call before any stream capture begins.
#include <mutex>

#include "../../include/admmq.h"
#include "common.cuh"

namespace {

// In host code this name is only a handle for the runtime; the address kernels may use comes from
// cudaGetSymbolAddress, once per device.
static __device__ __align__(256) double g_channel_err[ADMMQ_STATIC_MAX_D_OUT];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
double* g_scratch_ptr[kMaxDevices] = {};

// One CTA per output channel j: e = (z0 + Delta k) - w_hat in shared memory, then
// q_j = sum_i e_i (H[i, :] . e), one warp per row i of H.  Result to scratch[j].
__global__ void __launch_bounds__(256)
channel_error_kernel(const float* __restrict__ H, int n, const float* __restrict__ W0, int p, int gs,
                     const unsigned char* __restrict__ codes, const float* __restrict__ delta,
                     const float* __restrict__ zero, double* __restrict__ scratch) {
  extern __shared__ float e[];
  __shared__ double red[32];
  const int ng = n / gs;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int j = blockIdx.x; j < p; j += gridDim.x) {
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const long long idx = (long long)j * n + i;
      const long long gi = (long long)j * ng + i / gs;
      e[i] = (zero[gi] + delta[gi] * (float)codes[idx]) - W0[idx];
    }
    __syncthreads();
    double acc = 0.0;
    for (int i = wid; i < n; i += nw) {
      const float* hrow = H + (long long)i * n;
      float d = 0.f;
      for (int c = lane; c < n; c += 32) d = fmaf(hrow[c], e[c], d);
      acc += (double)e[i] * (double)d;          // every lane keeps its share of row i's dot product
    }
    acc = admmq::block_sum(acc, red);
    if (threadIdx.x == 0) scratch[j] = acc;
  }
}

// Fixed-order sum of the per-channel values.
__global__ void sum_channels_kernel(const double* __restrict__ scratch, int p, double* __restrict__ out) {
  __shared__ double red[32];
  double acc = 0.0;
  for (int j = threadIdx.x; j < p; j += blockDim.x) acc += scratch[j];
  acc = admmq::block_sum(acc, red);
  if (threadIdx.x == 0) *out = acc;
}

// Once per device, with that device current: resolve the scratch address, raise the smem limit.
admmq_status setup_device(int dev, double** ptr_out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    double* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_channel_err) != cudaSuccess || !ptr) return ADMMQ_ERR_CUDA;
    if (cudaFuncSetAttribute(channel_error_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ADMMQ_MAX_D_IN * (int)sizeof(float)) != cudaSuccess)
      return ADMMQ_ERR_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *ptr_out = g_scratch_ptr[dev];
  return ADMMQ_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" admmq_status admmq_objective_static(const float* d_H, int d_in, const float* d_W0, int d_out,
                                               int group_size, const unsigned char* d_codes,
                                               const float* d_scale, const float* d_zero, double* d_err,
                                               void* cuda_stream) {
  if (!d_H || !d_W0 || !d_codes || !d_scale || !d_zero || !d_err) return ADMMQ_ERR_INVALID_ARG;
  if (!aligned16(d_H) || !aligned16(d_W0) || !aligned16(d_codes) || !aligned16(d_scale) ||
      !aligned16(d_zero) || (reinterpret_cast<uintptr_t>(d_err) & 7u))
    return ADMMQ_ERR_INVALID_ARG;
  if (d_in < 8 || d_in > ADMMQ_MAX_D_IN || (d_in % 8) != 0) return ADMMQ_ERR_SHAPE;
  if (d_out < 1 || d_out > ADMMQ_STATIC_MAX_D_OUT) return ADMMQ_ERR_SHAPE;   // beyond the fixed scratch
  const int gs = (group_size == 0 || group_size == d_in) ? d_in : group_size;
  if (gs < 0 || gs > d_in || d_in % gs != 0) return ADMMQ_ERR_SHAPE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ADMMQ_ERR_CUDA;
  double* scratch = nullptr;
  admmq_status st = setup_device(dev, &scratch);
  if (st != ADMMQ_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const int blocks = d_out < 1184 ? d_out : 1184;
  channel_error_kernel<<<blocks, 256, (size_t)d_in * sizeof(float), stream>>>(
      d_H, d_in, d_W0, d_out, gs, d_codes, d_scale, d_zero, scratch);
  sum_channels_kernel<<<1, 256, 0, stream>>>(scratch, d_out, d_err);
  return cudaGetLastError() == cudaSuccess ? ADMMQ_OK : ADMMQ_ERR_CUDA;
}
