// Plain fp32 FMA product kernel on the same split-bf16 operands as the tensor-core kernel:
// C[M][N] (epilogue)= A[M][K] * B[N][K]^T with a = hi + lo rebuilt in fp32.  It is the on-device
// cross-check of the tcgen05 kernel and serves shapes too small to matter.
#include "internal.h"

namespace admmq {

constexpr int ST = 64, SK = 16;

__device__ __forceinline__ float plane_value(const bf16* plane, long long idx, int f16) {
  return f16 ? __half2float(reinterpret_cast<const __half*>(plane)[idx]) : __bfloat162float(plane[idx]);
}

__global__ void __launch_bounds__(256)
gemm_simt_kernel(Planes A, Planes B, int M, int N, int K, EpiParams epi) {
  __shared__ float As[SK][ST + 1];
  __shared__ float Bs[SK][ST + 1];
  __shared__ float red[32];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int m0 = blockIdx.y * ST, n0 = blockIdx.x * ST;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SK) {
    for (int e = threadIdx.x; e < ST * SK; e += 256) {
      const int r = e / SK, kk = e % SK;
      float a = 0.f, b = 0.f;
      if (m0 + r < M && k0 + kk < K) {
        const long long ia = (long long)(m0 + r) * A.ld + k0 + kk;
        a = plane_value(A.hi, ia, A.f16);
        if (A.lo) a += plane_value(A.lo, ia, A.f16);
      }
      if (n0 + r < N && k0 + kk < K) {
        const long long ib = (long long)(n0 + r) * B.ld + k0 + kk;
        b = plane_value(B.hi, ib, B.f16);
        if (B.lo) b += plane_value(B.lo, ib, B.f16);
      }
      As[kk][r] = a;
      Bs[kk][r] = b;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  float r2 = 0.f, s2 = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int row = m0 + ty * 4 + i, col = n0 + tx * 4 + j;
      if (row < M && col < N) epi_scalar(epi, row, col, N, acc[i][j], r2, s2);
    }
  if (epi.kind == EPI_ADMM) {
    r2 = block_sum(r2, red);
    s2 = block_sum(s2, red);
    if (threadIdx.x == 0) {
      const int slot = blockIdx.y * gridDim.x + blockIdx.x;
      epi.partials[2 * slot + 0] = r2;
      epi.partials[2 * slot + 1] = s2;
    }
  }
}

cudaError_t gemm_simt(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi_in) {
  EpiParams epi = epi_in;
  epi.row_inv = A.row_inv;
  epi.a_inv = A.all_inv;
  epi.b_inv = B.all_inv;
  dim3 grid((N + ST - 1) / ST, (M + ST - 1) / ST);
  gemm_simt_kernel<<<grid, 256, 0, c->stream>>>(A, B, M, N, K, epi);
  c->launches++;
  return cudaGetLastError();
}

}  // namespace admmq
