// Tensor-core product kernel for sm_100a:  C[M][N] (epilogue)= A[M][K] * B[N][K]^T.
//
// Operands are bf16 planes, one (plain bf16 data) or two (hi + lo split of an fp32 value) per operand;
// with two planes the product is hi*hi + hi*lo + lo*hi, three tcgen05.mma per K step into one fp32
// accumulator in tensor memory, which keeps ~16 mantissa bits of each operand.
//
// One persistent CTA per SM, 192 threads:
//   warp 0     TMA producer: cp.async.bulk.tensor loads of 128B-swizzled K-major tiles into a ring
//              of shared-memory stages, completion counted by mbarriers;
//   warp 1     MMA issuer: one elected thread issues tcgen05.mma (M=128, N=256, K=16 per instruction)
//              and tcgen05.commit, which releases stages and publishes finished accumulators;
//   warps 2-5  epilogue: tcgen05.ld the accumulator (lane = output row) and apply the epilogue --
//              for the ADMM iteration the projection, dual update, residual sums and the next
//              right-hand side -- while the issuer already works on the next tile in the second
//              accumulator (2 x 256 columns of tensor memory).
// Every wait is bounded: on expiry the kernel records ADMMQ_ERR_TIMEOUT, stops issuing work, lets
// copies in flight land, frees tensor memory and returns.
#include <cuda.h>

#include "internal.h"

namespace admmq {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int TC_THREADS = 192;
constexpr long long WAIT_LIMIT_CYCLES = 2000000000LL;   // about a second

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.b32 %0, 1, 0, p;\n}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done;
}
// Bounded wait.  Returns false (and raises the abort flag + device status) when the limit runs out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (++spins >= 32) {
      spins = 0;
      if (*abort_flag || clock64() - t0 > WAIT_LIMIT_CYCLES) {
        *abort_flag = 1;
        raise_status(status, ST_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile with 128-byte rows and 128B swizzle: groups of
// 8 rows are 1024 bytes apart (stride byte offset), the leading byte offset is unused for swizzled
// K-major tiles, descriptor version 1 (sm_100), layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, N = 256, M = 128.
constexpr uint32_t IDESC_BF16_128x256 =
    (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

struct TcMaps {
  CUtensorMap a[2];
  CUtensorMap b[2];
};

// ------------------------------------------------------------------ vectorised epilogue pieces
__device__ __forceinline__ void epi_chunk32(const EpiParams& P, int row, int col0, int M, int N,
                                            const uint32_t (&acc)[32], float& r2, float& s2) {
  if (row >= M || col0 >= N) return;
  const bool full = (col0 + 32 <= N);
  if (P.kind == EPI_ADMM) {
    const long long base = (long long)row * N + col0;
    const bool one_group = full && ((P.group_size & 31) == 0);
    if (one_group) {
      const long long gi = (long long)row * P.n_groups + col0 / P.group_size;
      const float dl = P.delta[gi], z0 = P.zero[gi];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const long long o = base + q * 8;
        const float4 w0 = *reinterpret_cast<const float4*>(P.Whs + o);
        const float4 w1 = *reinterpret_cast<const float4*>(P.Whs + o + 4);
        const float4 v0 = *reinterpret_cast<const float4*>(P.V + o);
        const float4 v1 = *reinterpret_cast<const float4*>(P.V + o + 4);
        const float4 s0 = *reinterpret_cast<const float4*>(P.s + col0 + q * 8);
        const float4 s1 = *reinterpret_cast<const float4*>(P.s + col0 + q * 8 + 4);
        uint2 cold = make_uint2(0u, 0u);
        if (!P.first_iter) cold = *reinterpret_cast<const uint2*>(P.codes + o);
        const float wh[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
        const float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        const float ss[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
        float vn[8];
        uint32_t cn[2] = {0u, 0u};
        __align__(16) bf16 rh[8];
        __align__(16) bf16 rl[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t word = (e < 4) ? cold.x : cold.y;
          const int code_old = (int)((word >> (8 * (e & 3))) & 0xffu);
          AdmmElem r = admm_elem(__uint_as_float(acc[q * 8 + e]), wh[e], vv[e], code_old, ss[e], dl, z0, P);
          vn[e] = r.v_new;
          cn[e >> 2] |= (uint32_t)r.code << (8 * (e & 3));
          split_bf16(r.r_next, rh[e], rl[e]);
          r2 += r.dr2;
          s2 += r.ds2;
        }
        *reinterpret_cast<float4*>(P.V + o) = make_float4(vn[0], vn[1], vn[2], vn[3]);
        *reinterpret_cast<float4*>(P.V + o + 4) = make_float4(vn[4], vn[5], vn[6], vn[7]);
        *reinterpret_cast<uint2*>(P.codes + o) = make_uint2(cn[0], cn[1]);
        *reinterpret_cast<uint4*>(P.Rhi + o) = *reinterpret_cast<const uint4*>(rh);
        *reinterpret_cast<uint4*>(P.Rlo + o) = *reinterpret_cast<const uint4*>(rl);
      }
      return;
    }
    for (int e = 0; e < 32; ++e)
      if (col0 + e < N) epi_scalar(P, row, col0 + e, N, __uint_as_float(acc[e]), r2, s2);
    return;
  }
  // STORE / ACCUM / WOUT
  float* crow = P.C + (long long)row * P.ldc + col0;
  const bool vec_ok = full && ((P.ldc & 3) == 0) && (P.kind != EPI_ACCUM || !P.lower_only || col0 + 31 <= row);
  if (vec_ok) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      float4 o = make_float4(__uint_as_float(acc[4 * q]), __uint_as_float(acc[4 * q + 1]),
                             __uint_as_float(acc[4 * q + 2]), __uint_as_float(acc[4 * q + 3]));
      if (P.kind == EPI_ACCUM) {
        const float4 c = *reinterpret_cast<const float4*>(crow + 4 * q);
        o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w;
      } else if (P.kind == EPI_WOUT) {
        const float4 c = *reinterpret_cast<const float4*>(P.Whs + (long long)row * N + col0 + 4 * q);
        o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w;
      }
      *reinterpret_cast<float4*>(crow + 4 * q) = o;
    }
    return;
  }
  for (int e = 0; e < 32; ++e)
    if (col0 + e < N) epi_scalar(P, row, col0 + e, N, __uint_as_float(acc[e]), r2, s2);
}

// ------------------------------------------------------------------ the kernel
template <int NA, int NB>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ TcMaps maps, int M, int N, int K, EpiParams epi, int* status) {
  constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
  constexpr int STAGE_BYTES = NA * A_BYTES + NB * B_BYTES;
  constexpr int STAGES = (NA + NB == 2) ? 4 : 2;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ float red[8];

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;

  const uint32_t full0 = smem_u32(&bars[0]);
  const uint32_t empty0 = smem_u32(&bars[STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[2 * STAGES]);
  const uint32_t tempty0 = smem_u32(&bars[2 * STAGES + 2]);

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull0 + 8 * a, 1);
      mbar_init(tempty0 + 8 * a, 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(
                     smem_u32(&tmem_base_slot))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  const int tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN - 1) / BN;
  const int num_tiles = tiles_m * tiles_n;
  const int num_kb = (K + BK - 1) / BK;
  const bool lower = (epi.kind == EPI_ACCUM) && epi.lower_only;

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        if (lower && tn * BN > tm * BM + BM - 1) continue;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag, status);
          if (!ok) break;
          const uint32_t sbase = tiles_base + stage * STAGE_BYTES;
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, STAGE_BYTES);
#pragma unroll
          for (int pl = 0; pl < NA; ++pl) tma_load_2d(sbase + pl * A_BYTES, &maps.a[pl], fb, kb * BK, tm * BM);
#pragma unroll
          for (int pl = 0; pl < NB; ++pl)
            tma_load_2d(sbase + NA * A_BYTES + pl * B_BYTES, &maps.b[pl], fb, kb * BK, tn * BN);
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        if (lower && tn * BN > tm * BM + BM - 1) continue;
        const int acc = it & 1;
        ok = mbar_wait(tempty0 + 8 * acc, (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        uint32_t accumulate = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sbase = tiles_base + stage * STAGE_BYTES;
          const uint64_t a_hi = make_kmajor_sw128_desc(sbase);
          const uint64_t a_lo = make_kmajor_sw128_desc(sbase + A_BYTES);
          const uint64_t b_hi = make_kmajor_sw128_desc(sbase + NA * A_BYTES);
          const uint64_t b_lo = make_kmajor_sw128_desc(sbase + NA * A_BYTES + B_BYTES);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16) {
            const uint64_t koff = (uint64_t)((k16 * 32) >> 4);   // 16 bf16 = 32 bytes along K
            tc_mma_bf16(d_tmem, a_hi + koff, b_hi + koff, IDESC_BF16_128x256, accumulate);
            accumulate = 1;
            if (NB == 2) tc_mma_bf16(d_tmem, a_hi + koff, b_lo + koff, IDESC_BF16_128x256, 1);
            if (NA == 2) tc_mma_bf16(d_tmem, a_lo + koff, b_hi + koff, IDESC_BF16_128x256, 1);
          }
          tc_commit(empty0 + 8 * stage);     // stage reusable once these MMAs have read it
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        tc_commit(tfull0 + 8 * acc);         // accumulator complete
        ++it;
      }
    }
  } else {
    // ===================== epilogue warps =====================
    const int q = warp & 3;                  // tensor-memory lane quarter this warp may read
    float r2 = 0.f, s2 = 0.f;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      const int tm = tile / tiles_n, tn = tile % tiles_n;
      if (lower && tn * BN > tm * BM + BM - 1) continue;
      const int acc = it & 1;
      ok = mbar_wait(tfull0 + 8 * acc, ((uint32_t)it >> 1) & 1u, abort_flag, status);
      if (!ok) break;
      tc_fence_after();
      const int row = tm * BM + q * 32 + lane;
      const uint32_t taddr = tmem_base + (uint32_t)acc * BN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int cchunk = 0; cchunk < BN / 32; ++cchunk) {
        uint32_t v[32];
        tc_ld32(taddr + cchunk * 32, v);
        epi_chunk32(epi, row, tn * BN + cchunk * 32, M, N, v, r2, s2);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
      ++it;
    }
    if (epi.kind == EPI_ADMM) {
      r2 = warp_sum(r2);
      s2 = warp_sum(s2);
      if (lane == 0) {
        red[2 * q] = r2;
        red[2 * q + 1] = s2;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (abort_flag_s) {                        // give copies in flight time to land before the CTA exits
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {
    }
    __syncthreads();
  }
  if (epi.kind == EPI_ADMM && threadIdx.x == 0) {
    // fixed order over the four lane quarters (warps 2,3,4,5 hold quarters 2,3,0,1)
    epi.partials[2 * blockIdx.x + 0] = ((red[0] + red[2]) + red[4]) + red[6];
    epi.partials[2 * blockIdx.x + 1] = ((red[1] + red[3]) + red[5]) + red[7];
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// Row-major bf16 matrix [rows][ld], K = `cols` contiguous; box = box_rows x 64 elements, 128B swizzle;
// out-of-range elements read as zero.
static bool encode_plane(CUtensorMap* map, const bf16* ptr, long long rows, long long cols, long long ld,
                         int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(bf16)};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)ptr, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int gemm_tc_partial_slots(int num_sms) { return num_sms; }

template <int NA, int NB>
static cudaError_t launch_tc(Ctx* c, const TcMaps& maps, int M, int N, int K, const EpiParams& epi) {
  constexpr int STAGE_BYTES = NA * BM * BK * 2 + NB * BN * BK * 2;
  constexpr int STAGES = (NA + NB == 2) ? 4 : 2;
  const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<NA, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  const int grid = tiles < c->num_sms ? tiles : c->num_sms;
  gemm_tc_kernel<NA, NB><<<grid, TC_THREADS, smem, c->stream>>>(maps, M, N, K, epi, c->status);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t gemm_tc(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi) {
  const int na = A.lo ? 2 : 1, nb = B.lo ? 2 : 1;
  if (na != nb) return cudaErrorInvalidValue;
  if ((A.ld & 7) || (B.ld & 7)) return cudaErrorInvalidValue;
  TcMaps maps;
  bool ok = encode_plane(&maps.a[0], A.hi, M, K, A.ld, BM) && encode_plane(&maps.b[0], B.hi, N, K, B.ld, BN);
  if (na == 2) ok = ok && encode_plane(&maps.a[1], A.lo, M, K, A.ld, BM);
  else maps.a[1] = maps.a[0];
  if (nb == 2) ok = ok && encode_plane(&maps.b[1], B.lo, N, K, B.ld, BN);
  else maps.b[1] = maps.b[0];
  if (!ok) return cudaErrorInvalidValue;
  if (epi.kind == EPI_ADMM) {
    // unused partial slots of this launch must read as zero
    const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
    (void)tiles;
  }
  return (na == 2) ? launch_tc<2, 2>(c, maps, M, N, K, epi) : launch_tc<1, 1>(c, maps, M, N, K, epi);
}

}  // namespace admmq
