// Tensor-core product kernel for sm_100a:  C[M][N] (epilogue)= A[M][K] * B[N][K]^T.
//
// Operands are 16-bit planes, one (plain bf16 data) or two (hi + lo split of an fp32 value) per
// operand; with two planes the product is hi*hi + hi*lo + lo*hi, three tcgen05.mma per K step.
//
// Accumulation.  The tensor core adds into its fp32 accumulator with truncation, so a long chain of
// accumulating MMAs drifts toward zero (measured ~3e-5 relative after the 768 steps of K = 4096).
// The chain is therefore kept short: one flush = 12 MMA steps (one 64-wide K block with two planes,
// three with one plane) goes into one of four 128-column accumulators in tensor memory, and the
// worker warps add each finished partial into fp32 registers with round-to-nearest adds.
//
// One persistent CTA per SM, 576 threads, output tiles of 128 x 128:
//   warp 0       TMA producer: cp.async.bulk.tensor loads of 128B-swizzled K-major tiles into a ring
//                of shared-memory stages, completion counted by mbarriers;
//   warp 1       MMA issuer: one elected thread issues tcgen05.mma (M = 128, N = 128, K = 16 per
//                instruction) and tcgen05.commit, which releases stages and publishes partials;
//   warps 2-9    worker group 0, warps 10-17 worker group 1.  The groups take alternate tiles.  A
//                group drains the partials of its tile (tcgen05.ld, lane = output row; the two
//                warps of a lane quarter split the 128 columns) and then runs the epilogue from its
//                registers -- for the ADMM iteration the projection, dual update, residual sums and
//                the next right-hand side -- while the other group drains the next tile.
// Every wait is bounded: on expiry the kernel records ADMMQ_ERR_TIMEOUT, stops issuing work, lets
// copies in flight land, frees tensor memory and returns.
#include <cuda.h>

#include "internal.h"

namespace admmq {

constexpr int BM = 128, BN = 128, BK = 64;
constexpr int NPART = 4;                 // partial accumulators in tensor memory (4 x 128 columns)
constexpr int GROUP_WARPS = 8;
constexpr int TC_THREADS = 32 * (2 + 2 * GROUP_WARPS);
constexpr int COLS_PER_THREAD = BN / 2;  // 64
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
// The same wait for a whole warp: lane 0 polls, the others sleep at the shuffle, so that the 16 worker
// warps do not all hammer one barrier word.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int* status) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
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
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 consecutive accumulator columns of this warp's 32 lanes (lane = row), issued without waiting.
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&v)[32]) {
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
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

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
// Instruction descriptor: fp32 accumulate, A and B of the same 16-bit type (format 1 = bf16, 0 = fp16),
// both K-major, N = 128, M = 128.
__host__ __device__ constexpr uint32_t idesc_128x128(uint32_t fmt) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// Tile order.  Consecutive tiles (the ones resident at the same time) form bands of RASTER_M tile rows
// walked column by column, so that one wave of CTAs touches about 12 x 12 tiles: ~12 row blocks of A and
// ~12 row blocks of B stay in L2 instead of a whole operand being streamed from HBM by every wave.
constexpr int RASTER_M = 12;
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int band = tile / (RASTER_M * tiles_n);
  const int first = band * RASTER_M;
  const int rows = tiles_m - first < RASTER_M ? tiles_m - first : RASTER_M;
  const int in_band = tile - band * RASTER_M * tiles_n;
  tn = in_band / rows;
  tm = first + in_band - tn * rows;
}

struct TcMaps {
  CUtensorMap a[2];
  CUtensorMap b[2];
};

// ------------------------------------------------------------------ epilogue
// A worker warp holds a 32-row x 64-column block of products, one row per lane.  Global accesses in
// that ownership would touch 32 different lines per instruction, 16 bytes each, and choke the
// load/store queue next to the draining warps.  So the block goes through a small per-warp staging
// buffer in pieces of 8 columns: each lane writes its 8 values, then takes 4 consecutive values of
// another row (lane / 2 + 16 i, columns 4 (lane & 1) ...), so that every global instruction covers 16
// rows x 32 bytes in whole sectors.
constexpr int PIECE_COLS = 8;
constexpr int STAGE_FLOATS = 32 * PIECE_COLS;            // per worker warp

// Four consecutive elements (row, col .. col + 3) of the output, products in `acc` (unscaled values).
template <int EPI>
__device__ __forceinline__ void epi_elem4(const EpiParams& P, int row, int col, int N, const float4 acc,
                                          float& r2, float& s2) {
  const float a[4] = {acc.x, acc.y, acc.z, acc.w};
  if (EPI == EPI_ADMM) {
    const long long o = (long long)row * N + col;
    const float4 w = *reinterpret_cast<const float4*>(P.Whs + o);
    const float4 v = *reinterpret_cast<const float4*>(P.V + o);
    const float4 s = *reinterpret_cast<const float4*>(P.s + col);
    uint32_t codes = 0u;
    if (!P.first_iter) codes = *reinterpret_cast<const uint32_t*>(P.codes + o);
    const float wh[4] = {w.x, w.y, w.z, w.w};
    const float vv[4] = {v.x, v.y, v.z, v.w};
    const float ss[4] = {s.x, s.y, s.z, s.w};
    const bool one_group = (P.group_size & 3) == 0;        // then the 4 columns share (Delta, z0)
    long long gi = (long long)row * P.n_groups + col / P.group_size;
    float dl = P.delta[gi], z0 = P.zero[gi];
    float vn[4], rn[4];
    uint32_t cn = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (!one_group && e > 0) {
        gi = (long long)row * P.n_groups + (col + e) / P.group_size;
        dl = P.delta[gi];
        z0 = P.zero[gi];
      }
      const int code_old = (int)((codes >> (8 * e)) & 0xffu);
      AdmmElem r = admm_elem(a[e], wh[e], vv[e], code_old, ss[e], dl, z0, P);
      vn[e] = r.v_new;
      cn |= (uint32_t)r.code << (8 * e);
      rn[e] = r.r_next;
      r2 += r.dr2;
      s2 += r.ds2;
    }
    *reinterpret_cast<float4*>(P.V + o) = make_float4(vn[0], vn[1], vn[2], vn[3]);
    *reinterpret_cast<uint32_t*>(P.codes + o) = cn;
    *reinterpret_cast<float4*>(P.Rnext + o) = make_float4(rn[0], rn[1], rn[2], rn[3]);
    return;
  }
  float* cp = P.C + (long long)row * P.ldc + col;
  float o[4] = {a[0], a[1], a[2], a[3]};
  if (EPI == EPI_WOUT) {
    const float4 c = *reinterpret_cast<const float4*>(P.Whs + (long long)row * N + col);
    o[0] += c.x; o[1] += c.y; o[2] += c.z; o[3] += c.w;
  }
  if (EPI == EPI_ACCUM) {
    if (P.lower_only && col + 3 > row) {                   // the tile straddles the diagonal
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (col + e <= row) cp[e] += o[e];
      return;
    }
    const float4 c = *reinterpret_cast<const float4*>(cp);
    o[0] += c.x; o[1] += c.y; o[2] += c.z; o[3] += c.w;
  }
  *reinterpret_cast<float4*>(cp) = make_float4(o[0], o[1], o[2], o[3]);
}

// The block rows [row0, row0 + 32) x columns [col0, col0 + 64) held by one warp.  All sizes on this path
// keep N and the leading dimensions multiples of 4, so a group of 4 columns is inside or outside.
template <int EPI>
__device__ __forceinline__ void epilogue_block(const EpiParams& P, int row0, int col0, int M, int N,
                                               const float (&sums)[COLS_PER_THREAD], float* stage, int lane,
                                               float& r2, float& s2) {
  const float sc = (row0 + lane < M) ? epi_row_factor(P, row0 + lane) : 0.0f;
#pragma unroll
  for (int pc = 0; pc < COLS_PER_THREAD / PIECE_COLS; ++pc) {
    float* mine = stage + lane * PIECE_COLS;
    *reinterpret_cast<float4*>(mine) = make_float4(sums[pc * 8] * sc, sums[pc * 8 + 1] * sc,
                                                   sums[pc * 8 + 2] * sc, sums[pc * 8 + 3] * sc);
    *reinterpret_cast<float4*>(mine + 4) = make_float4(sums[pc * 8 + 4] * sc, sums[pc * 8 + 5] * sc,
                                                       sums[pc * 8 + 6] * sc, sums[pc * 8 + 7] * sc);
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int r = (lane >> 1) + 16 * i, c4 = (lane & 1) * 4;
      const float4 acc = *reinterpret_cast<const float4*>(stage + r * PIECE_COLS + c4);
      const int row = row0 + r, col = col0 + pc * PIECE_COLS + c4;
      if (row < M && col < N) epi_elem4<EPI>(P, row, col, N, acc, r2, s2);
    }
    __syncwarp();
  }
}

// ------------------------------------------------------------------ the kernel
// NP: planes per operand (1 or 2).  EPI: epilogue kind (compile-time copy of epi.kind).
template <int NP, int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ TcMaps maps, int M, int N, int K, uint32_t idesc, EpiParams epi,
               int* status) {
  constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
  constexpr int STAGE_BYTES = NP * (A_BYTES + B_BYTES);
  constexpr int STAGES = (NP == 1) ? 6 : 3;
  constexpr int KB_PER_FLUSH = (NP == 1) ? 3 : 1;        // 12 accumulating MMA steps per flush either way
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 2 * NPART + 2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ float red[2 * GROUP_WARPS * 2];
  __shared__ __align__(16) float stage_all[2 * GROUP_WARPS * STAGE_FLOATS];

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;

  const uint32_t full0 = smem_u32(&bars[0]);
  const uint32_t empty0 = smem_u32(&bars[STAGES]);
  const uint32_t pfull0 = smem_u32(&bars[2 * STAGES]);
  const uint32_t pempty0 = smem_u32(&bars[2 * STAGES + NPART]);
  const uint32_t drained0 = smem_u32(&bars[2 * STAGES + 2 * NPART]);   // [group]: that group has drained a tile

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < NPART; ++a) {
      mbar_init(pfull0 + 8 * a, 1);
      mbar_init(pempty0 + 8 * a, GROUP_WARPS);
    }
    for (int a = 0; a < 2; ++a) mbar_init(drained0 + 8 * a, GROUP_WARPS);
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
  const int num_flush = (num_kb + KB_PER_FLUSH - 1) / KB_PER_FLUSH;
  const bool lower = (EPI == EPI_ACCUM) && epi.lower_only;

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int tm, tn;
        tile_coords(tile, tiles_m, tiles_n, tm, tn);
        if (lower && tn * BN > tm * BM + BM - 1) continue;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag, status);
          if (!ok) break;
          const uint32_t sbase = tiles_base + stage * STAGE_BYTES;
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, STAGE_BYTES);
#pragma unroll
          for (int pl = 0; pl < NP; ++pl) tma_load_2d(sbase + pl * A_BYTES, &maps.a[pl], fb, kb * BK, tm * BM);
#pragma unroll
          for (int pl = 0; pl < NP; ++pl)
            tma_load_2d(sbase + NP * A_BYTES + pl * B_BYTES, &maps.b[pl], fb, kb * BK, tn * BN);
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
      uint32_t g = 0;                        // flush counter, shared sequence with the workers
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int tm, tn;
        tile_coords(tile, tiles_m, tiles_n, tm, tn);
        if (lower && tn * BN > tm * BM + BM - 1) continue;
        uint32_t d_tmem = 0, accumulate = 0;
        int pb = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (kb % KB_PER_FLUSH == 0) {
            pb = (int)(g % NPART);
            ok = mbar_wait(pempty0 + 8 * pb, ((g / NPART) & 1u) ^ 1u, abort_flag, status);
            if (!ok) break;
            tc_fence_after();
            d_tmem = tmem_base + (uint32_t)pb * BN;
            accumulate = 0;
          }
          ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sbase = tiles_base + stage * STAGE_BYTES;
          const uint64_t a_hi = make_kmajor_sw128_desc(sbase);
          const uint64_t a_lo = make_kmajor_sw128_desc(sbase + A_BYTES);
          const uint64_t b_hi = make_kmajor_sw128_desc(sbase + NP * A_BYTES);
          const uint64_t b_lo = make_kmajor_sw128_desc(sbase + NP * A_BYTES + B_BYTES);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16) {
            const uint64_t koff = (uint64_t)((k16 * 32) >> 4);   // 16 elements = 32 bytes along K
            // small terms first, so that they meet a small accumulator
            if (NP == 2) {
              tc_mma_f16(d_tmem, a_hi + koff, b_lo + koff, idesc, accumulate);
              tc_mma_f16(d_tmem, a_lo + koff, b_hi + koff, idesc, 1);
              accumulate = 1;
            }
            tc_mma_f16(d_tmem, a_hi + koff, b_hi + koff, idesc, accumulate);
            accumulate = 1;
          }
          tc_commit(empty0 + 8 * stage);     // stage reusable once these MMAs have read it
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1u;
          }
          if (kb % KB_PER_FLUSH == KB_PER_FLUSH - 1 || kb == num_kb - 1) {
            tc_commit(pfull0 + 8 * pb);      // partial complete
            ++g;
          }
        }
      }
    }
  } else {
    // ===================== worker groups =====================
    const int gsel = (warp - 2) / GROUP_WARPS;             // 0 or 1
    const int wi = (warp - 2) % GROUP_WARPS;
    const int q = warp & 3;                                // tensor-memory lane quarter this warp may read
    const int half = wi >> 2;                              // which 64 of the 128 columns
    float r2 = 0.f, s2 = 0.f;
    uint32_t g = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int tm, tn;
        tile_coords(tile, tiles_m, tiles_n, tm, tn);
      if (lower && tn * BN > tm * BM + BM - 1) continue;
      if ((it & 1) != gsel) {                              // the other group's tile
        g += (uint32_t)num_flush;
        ++it;
        continue;
      }
      // A parity wait cannot tell a phase from the one two completions later, so a group starts
      // watching the partial barriers only once the other group has drained the tile before this one.
      if (it > 0) {
        ok = mbar_wait_warp(drained0 + 8 * (1 - gsel), (uint32_t)((it - 1) >> 1) & 1u, abort_flag, status);
        if (!ok) break;
      }
      float sums[COLS_PER_THREAD];
#pragma unroll
      for (int e = 0; e < COLS_PER_THREAD; ++e) sums[e] = 0.f;
      for (int f = 0; f < num_flush; ++f) {
        const int pb = (int)(g % NPART);
        ok = mbar_wait_warp(pfull0 + 8 * pb, (g / NPART) & 1u, abort_flag, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + (uint32_t)pb * BN + (uint32_t)(half * COLS_PER_THREAD) +
                               ((uint32_t)(q * 32) << 16);
        uint32_t v[32];
        tc_ld32_issue(taddr, v);
        tc_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; ++e) sums[e] += __uint_as_float(v[e]);
        tc_ld32_issue(taddr + 32, v);
        tc_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(pempty0 + 8 * pb);      // the partial is in registers: buffer free
#pragma unroll
        for (int e = 0; e < 32; ++e) sums[32 + e] += __uint_as_float(v[e]);
        ++g;
      }
      if (!ok) break;
      if (lane == 0) mbar_arrive(drained0 + 8 * gsel);
      epilogue_block<EPI>(epi, tm * BM + q * 32, tn * BN + half * COLS_PER_THREAD, M, N, sums,
                          stage_all + (warp - 2) * STAGE_FLOATS, lane, r2, s2);
      ++it;
    }
    if (EPI == EPI_ADMM) {
      r2 = warp_sum(r2);
      s2 = warp_sum(s2);
      if (lane == 0) {
        red[2 * (warp - 2)] = r2;
        red[2 * (warp - 2) + 1] = s2;
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
  if (EPI == EPI_ADMM && threadIdx.x == 0) {
    float a = 0.f, b = 0.f;                  // fixed order over the worker warps
    for (int w = 0; w < 2 * GROUP_WARPS; ++w) {
      a += red[2 * w];
      b += red[2 * w + 1];
    }
    epi.partials[2 * blockIdx.x + 0] = a;
    epi.partials[2 * blockIdx.x + 1] = b;
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

// Row-major 16-bit matrix [rows][ld], K = `cols` contiguous; box = box_rows x 64 elements, 128B swizzle;
// out-of-range elements read as zero.
static bool encode_plane(CUtensorMap* map, const bf16* ptr, long long rows, long long cols, long long ld,
                         int box_rows, int f16) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(bf16)};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)ptr,
                  dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int gemm_tc_partial_slots(int num_sms) { return num_sms; }

template <int NP, int EPI>
static cudaError_t launch_tc(Ctx* c, const TcMaps& maps, int M, int N, int K, uint32_t idesc,
                             const EpiParams& epi) {
  constexpr int STAGE_BYTES = NP * (BM * BK * 2 + BN * BK * 2);
  constexpr int STAGES = (NP == 1) ? 6 : 3;
  const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<NP, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  const int grid = tiles < c->num_sms ? tiles : c->num_sms;
  gemm_tc_kernel<NP, EPI><<<grid, TC_THREADS, smem, c->stream>>>(maps, M, N, K, idesc, epi, c->status);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t gemm_tc(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi_in) {
  const int na = A.lo ? 2 : 1, nb = B.lo ? 2 : 1;
  if (na != nb || A.f16 != B.f16) return cudaErrorInvalidValue;   // one MMA takes A and B of one type
  if ((A.ld & 7) || (B.ld & 7)) return cudaErrorInvalidValue;
  TcMaps maps;
  bool ok = encode_plane(&maps.a[0], A.hi, M, K, A.ld, BM, A.f16) &&
            encode_plane(&maps.b[0], B.hi, N, K, B.ld, BN, B.f16);
  if (na == 2) ok = ok && encode_plane(&maps.a[1], A.lo, M, K, A.ld, BM, A.f16);
  else maps.a[1] = maps.a[0];
  if (nb == 2) ok = ok && encode_plane(&maps.b[1], B.lo, N, K, B.ld, BN, B.f16);
  else maps.b[1] = maps.b[0];
  if (!ok) return cudaErrorInvalidValue;
  EpiParams epi = epi_in;
  epi.row_inv = A.row_inv;
  epi.a_inv = A.all_inv;
  epi.b_inv = B.all_inv;
  const uint32_t idesc = idesc_128x128(A.f16 ? 0u : 1u);
  if (na == 1) {
    if (epi.kind == EPI_ACCUM) return launch_tc<1, EPI_ACCUM>(c, maps, M, N, K, idesc, epi);
    if (epi.kind == EPI_STORE) return launch_tc<1, EPI_STORE>(c, maps, M, N, K, idesc, epi);
    return cudaErrorInvalidValue;
  }
  switch (epi.kind) {
    case EPI_STORE: return launch_tc<2, EPI_STORE>(c, maps, M, N, K, idesc, epi);
    case EPI_ACCUM: return launch_tc<2, EPI_ACCUM>(c, maps, M, N, K, idesc, epi);
    case EPI_ADMM: return launch_tc<2, EPI_ADMM>(c, maps, M, N, K, idesc, epi);
    case EPI_WOUT: return launch_tc<2, EPI_WOUT>(c, maps, M, N, K, idesc, epi);
  }
  return cudaErrorInvalidValue;
}

}  // namespace admmq
