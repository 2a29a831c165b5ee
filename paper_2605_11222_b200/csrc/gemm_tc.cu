// Tensor-core product kernel for sm_100a:  C[M][N] (epilogue)= A[M][K] * B[N][K]^T.
//
// Operands are 16-bit planes, one (plain bf16 data) or two (hi + lo split of an fp32 value) per
// operand; with two planes the product is hi*hi + hi*lo + lo*hi, three tcgen05.mma per K step.
//
// Accumulation.  The tensor core adds into its fp32 accumulator with truncation, so a long chain of
// accumulating MMAs drifts toward zero (measured ~3e-5 relative after the 768 steps of K = 4096).
// The chain is therefore kept short: one flush = 12 MMA steps (one 64-wide K block with two planes,
// three with one plane) goes into one of two 256-column accumulators in tensor memory, and the
// worker warps add each finished partial into fp32 registers with round-to-nearest adds.
//
// Tiles.  An MMA reads its operands from shared memory at (M + N) * 32 bytes per 16-deep step, and
// the next stage is written into the same memory meanwhile; at 128 x 128 that traffic alone caps the
// tensor pipe near 60 %.  Output tiles are therefore 128 x 256 (one MMA of N = 256).  The tiles that
// would form a last, partly filled wave are cut into 128 x 128 halves, so that the wave costs half a
// tile time instead of a whole one.
//
// One persistent CTA per SM, 576 threads:
//   warp 0       TMA producer: cp.async.bulk.tensor loads of 128B-swizzled K-major tiles into a ring
//                of shared-memory stages, completion counted by mbarriers; with two planes the lo planes of
//                a stage are refilled as soon as the cross products of its K block are done, the hi planes
//                after the hi x hi products (only two stages fit, so every cycle of head start counts);
//   warp 1       MMA issuer: one elected thread issues tcgen05.mma (M = 128, N = 256 or 128, K = 16 per
//                instruction) and tcgen05.commit, which releases stages and publishes partials;
//   warps 2-17   workers: warp w owns tensor-memory lanes 32 (w mod 4) .. +31 (output rows) and 64 of
//                the 256 columns.  They drain every partial (tcgen05.ld) into 64 register sums per
//                thread and, when the tile is complete, run the epilogue from those registers -- for the
//                ADMM iteration the projection, dual update, residual sums and the next right-hand
//                side -- through a per-warp staging buffer that makes the global accesses coalesced.
//                The issuer runs up to two flushes into the next tile meanwhile.
// Every wait is bounded: on expiry the kernel records ADMMQ_ERR_TIMEOUT, stops issuing work, waits (again
// bounded) until the stage fills and MMAs already issued have completed, frees tensor memory and returns.
#include <cuda.h>

#include "internal.h"

namespace admmq {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int BN_BOX = 128;              // rows of B per TMA box (a tile takes two, a half tile one)
constexpr int NPART = 2;                 // partial accumulators in tensor memory (2 x 256 columns)
constexpr int WORKER_WARPS = 16;
constexpr int TC_THREADS = 32 * (2 + WORKER_WARPS);
constexpr int COLS_PER_THREAD = BN / 4;  // 64
constexpr long long DRAIN_LIMIT_CYCLES = 20000000LL;    // bound of each wait of the abort path (~10 ms)

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
                                          int* status, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (++spins >= 32) {
      spins = 0;
      if (*abort_flag || clock64() - t0 > limit) {
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
                                               int* status, long long limit) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status, limit) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// Wait of the abort path: bounded, raises nothing (the status is already set).
__device__ __forceinline__ void mbar_wait_quiet(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity) && clock64() - t0 < DRAIN_LIMIT_CYCLES) {
  }
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
// 8 consecutive accumulator columns of this warp's 32 lanes (lane = row), issued without waiting.  The
// drain uses this narrow form on purpose: a thread already holds 64 running sums, and with 16 or 32
// temporaries on top the worker loop spills (the register file gives 96 registers per thread at 18 warps),
// which cost 12 % of the launch.
__device__ __forceinline__ void tc_ld8_issue(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
      : "r"(taddr)
      : "memory");
}
// sums[0..7] += v[0..7] as four packed fp32 additions (round to nearest, the same result as eight scalar ones).
__device__ __forceinline__ void add8(float* sums, const uint32_t (&v)[8]) {
#pragma unroll
  for (int e = 0; e < 8; e += 2) {
    const float2 r = __fadd2_rn(make_float2(sums[e], sums[e + 1]),
                                make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])));
    sums[e] = r.x;
    sums[e + 1] = r.y;
  }
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
// both K-major, M = 128, N columns.
__host__ __device__ constexpr uint32_t idesc_m128(uint32_t fmt, uint32_t n_cols) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((n_cols >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
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

// Work units of the persistent loop: whole 128 x 256 tiles, except that the tiles of a last wave that
// would fill at most half of the CTAs are cut into two 128 x 128 units.
struct Schedule {
  int tiles_m, tiles_n, full_units, num_units;
};
__device__ __forceinline__ Schedule make_schedule(int M, int N, int ctas) {
  Schedule s;
  s.tiles_m = (M + BM - 1) / BM;
  s.tiles_n = (N + BN - 1) / BN;
  const int tiles = s.tiles_m * s.tiles_n;
  const int waves = tiles / ctas, rem = tiles - waves * ctas;
  const bool split = rem > 0 && 2 * rem <= ctas;
  s.full_units = split ? waves * ctas : tiles;
  s.num_units = split ? waves * ctas + 2 * rem : tiles;
  return s;
}
struct Unit {
  int tm, col0, ncols;   // first column and width (256 or 128)
};
__device__ __forceinline__ Unit unit_of(const Schedule& s, int u) {
  Unit x;
  int tile = u, off = 0;
  x.ncols = BN;
  if (u >= s.full_units) {
    const int h = u - s.full_units;
    tile = s.full_units + (h >> 1);
    off = (h & 1) * BN_BOX;
    x.ncols = BN_BOX;
  }
  int tn;
  tile_coords(tile, s.tiles_m, s.tiles_n, x.tm, tn);
  x.col0 = tn * BN + off;
  return x;
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
    const float4 w = *reinterpret_cast<const float4*>(P.W0 + o);
    const float4 v = *reinterpret_cast<const float4*>(P.V + o);
    const float4 s = *reinterpret_cast<const float4*>(P.s + col);
    const float4 is = *reinterpret_cast<const float4*>(P.inv_s + col);
    uint32_t codes = 0u;
    if (!P.first_iter) codes = *reinterpret_cast<const uint32_t*>(P.codes + o);
    const float wh[4] = {w.x, w.y, w.z, w.w};
    const float vv[4] = {v.x, v.y, v.z, v.w};
    const float ss[4] = {s.x, s.y, s.z, s.w};
    const float si[4] = {is.x, is.y, is.z, is.w};
    const bool one_group = (P.group_size & 3) == 0;        // then the 4 columns share (Delta, z0)
    const float cshift = (float)P.shift_c[0];
    long long gi = (long long)row * P.n_groups + col / P.group_size;
    GridG gg = grid_g(P.delta[gi], P.zero[gi]);
    float vn[4], rn[4];
    uint32_t cn = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (!one_group && e > 0) {
        gi = (long long)row * P.n_groups + (col + e) / P.group_size;
        gg = grid_g(P.delta[gi], P.zero[gi]);
      }
      const int code_old = (int)((codes >> (8 * e)) & 0xffu);
      AdmmElem r = admm_elem(a[e], wh[e], vv[e], code_old, ss[e], si[e], gg, gg, cshift, P);
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

// Asks L2 for the lines the epilogue of (row, [col0, col0 + 64)) will read, a few flushes ahead.
template <int EPI>
__device__ __forceinline__ void epilogue_prefetch(const EpiParams& P, int row, int col0, int M, int N) {
  if (row >= M || col0 + COLS_PER_THREAD > N) return;
  if (EPI == EPI_ADMM) {
    const long long o = (long long)row * N + col0;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(P.W0 + o));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(P.W0 + o + 32));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(P.V + o));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(P.V + o + 32));
    if (!P.first_iter) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.codes + o));
  } else if (EPI == EPI_ACCUM) {
    const float* c = P.C + (long long)row * P.ldc + col0;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(c));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(c + 32));
  }
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
gemm_tc_kernel(const __grid_constant__ TcMaps maps, int M, int N, int K, uint32_t fmt, EpiParams epi,
               int* status, long long wait_limit, int hold_loads, int flush_kb) {
  constexpr int A_BYTES = BM * BK * 2, BOX_BYTES = BN_BOX * BK * 2, B_BYTES = 2 * BOX_BYTES;
  constexpr int STAGE_BYTES = NP * (A_BYTES + B_BYTES);
  constexpr int STAGES = (NP == 1) ? 4 : 2;
  // K blocks accumulated in tensor memory before the workers take the partial: 12 MMA steps (one block with two
  // planes, three with one) where the result must be good to fp32, as many as the caller allows (flush_kb) where the
  // operands' own rounding is far above the accumulator's truncation (the one-plane products of the late iterations)
  const int KB_PER_FLUSH = (NP == 1) ? (flush_kb > 0 ? flush_kb : 3) : 1;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[3 * STAGES + 2 * NPART + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ uint32_t fill_state[3];       // producer's record for the abort path: armed / parity / half-armed stages
  __shared__ float red[WORKER_WARPS * 2];
  __shared__ __align__(16) float stage_all[WORKER_WARPS * STAGE_FLOATS];

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;

  const uint32_t full0 = smem_u32(&bars[0]);
  const uint32_t empty0 = smem_u32(&bars[STAGES]);
  const uint32_t pfull0 = smem_u32(&bars[2 * STAGES]);
  const uint32_t pempty0 = smem_u32(&bars[2 * STAGES + NPART]);
  const uint32_t elo0 = smem_u32(&bars[2 * STAGES + 2 * NPART]);   // two planes: the lo planes of a stage are free
  const uint32_t drain_bar = smem_u32(&bars[3 * STAGES + 2 * NPART]);  // abort path: all issued MMAs have completed

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    fill_state[0] = fill_state[1] = fill_state[2] = 0u;
    mbar_init(drain_bar, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, NP == 2 ? 2 : 1);           // two planes: the lo and the hi half arrive separately
      mbar_init(empty0 + 8 * s, 1);
      mbar_init(elo0 + 8 * s, 1);
    }
    for (int a = 0; a < NPART; ++a) {
      mbar_init(pfull0 + 8 * a, 1);
      mbar_init(pempty0 + 8 * a, WORKER_WARPS);
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

  const Schedule sched = make_schedule(M, N, gridDim.x);
  const int num_kb = (K + BK - 1) / BK;
  const int num_flush = (num_kb + KB_PER_FLUSH - 1) / KB_PER_FLUSH;
  const bool lower = (EPI == EPI_ACCUM) && epi.lower_only;

  if (warp == 0) {
    // ===================== TMA producer =====================
    // hold_loads (failure-handling tests only): the producer issues nothing, so the issuer's first wait runs out
    // with no copy in flight.
    if (lane == 0 && !hold_loads) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // latest fill of every stage, for the abort path: bit s of `armed`: stage s was armed, of `par`: with which
      // phase parity, of `half`: only the first of its two arrivals has been made
      uint32_t armed = 0u, par = 0u, half = 0u;
      for (int u = blockIdx.x; u < sched.num_units && ok; u += gridDim.x) {
        const Unit un = unit_of(sched, u);
        if (lower && un.col0 > un.tm * BM + BM - 1) continue;
        const int boxes = un.ncols / BN_BOX;
        for (int kb = 0; kb < num_kb; ++kb) {
          const uint32_t sbase = tiles_base + stage * STAGE_BYTES;
          const uint32_t fb = full0 + 8 * stage;
          const uint32_t bit = 1u << stage;
          if (NP == 2) {
            // the lo planes of a stage are released after the two cross products of its K block, a third of the
            // block's MMA time before the hi planes: their refill starts that much earlier
            ok = mbar_wait(elo0 + 8 * stage, phase ^ 1u, abort_flag, status, wait_limit);
            if (!ok) break;
            mbar_expect_tx(fb, A_BYTES + boxes * BOX_BYTES);
            armed |= bit;
            half |= bit;
            par = (par & ~bit) | (phase << stage);
            tma_load_2d(sbase + A_BYTES, &maps.a[1], fb, kb * BK, un.tm * BM);
            for (int bx = 0; bx < boxes; ++bx)
              tma_load_2d(sbase + NP * A_BYTES + B_BYTES + bx * BOX_BYTES, &maps.b[1], fb, kb * BK,
                          un.col0 + bx * BN_BOX);
          }
          ok = mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag, status, wait_limit);
          if (!ok) break;
          mbar_expect_tx(fb, A_BYTES + boxes * BOX_BYTES);
          armed |= bit;
          half &= ~bit;
          par = (par & ~bit) | (phase << stage);
          tma_load_2d(sbase, &maps.a[0], fb, kb * BK, un.tm * BM);
          for (int bx = 0; bx < boxes; ++bx)
            tma_load_2d(sbase + NP * A_BYTES + bx * BOX_BYTES, &maps.b[0], fb, kb * BK, un.col0 + bx * BN_BOX);
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      fill_state[0] = armed;
      fill_state[1] = par;
      fill_state[2] = half;
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t g = 0;                        // flush counter, shared sequence with the workers
      bool ok = true;
      for (int u = blockIdx.x; u < sched.num_units && ok; u += gridDim.x) {
        const Unit un = unit_of(sched, u);
        if (lower && un.col0 > un.tm * BM + BM - 1) continue;
        const uint32_t idesc = idesc_m128(fmt, (uint32_t)un.ncols);
        uint32_t d_tmem = 0, accumulate = 0;
        int pb = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (kb % KB_PER_FLUSH == 0) {
            pb = (int)(g % NPART);
            ok = mbar_wait(pempty0 + 8 * pb, ((g / NPART) & 1u) ^ 1u, abort_flag, status, wait_limit);
            if (!ok) break;
            tc_fence_after();
            d_tmem = tmem_base + (uint32_t)pb * BN;
            accumulate = 0;
          }
          ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, status, wait_limit);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sbase = tiles_base + stage * STAGE_BYTES;
          const uint64_t a_hi = make_kmajor_sw128_desc(sbase);
          const uint64_t a_lo = make_kmajor_sw128_desc(sbase + A_BYTES);
          const uint64_t b_hi = make_kmajor_sw128_desc(sbase + NP * A_BYTES);
          const uint64_t b_lo = make_kmajor_sw128_desc(sbase + NP * A_BYTES + B_BYTES);
          // the small cross terms of the whole K block first (they meet a small accumulator, and the lo planes
          // become free for the next load), then the hi x hi terms
          if (NP == 2) {
#pragma unroll
            for (int k16 = 0; k16 < BK / 16; ++k16) {
              const uint64_t koff = (uint64_t)((k16 * 32) >> 4);   // 16 elements = 32 bytes along K
              tc_mma_f16(d_tmem, a_hi + koff, b_lo + koff, idesc, accumulate);
              tc_mma_f16(d_tmem, a_lo + koff, b_hi + koff, idesc, 1);
              accumulate = 1;
            }
            tc_commit(elo0 + 8 * stage);
          }
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16) {
            const uint64_t koff = (uint64_t)((k16 * 32) >> 4);
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
    // ===================== workers =====================
    const int q = warp & 3;                                // tensor-memory lane quarter this warp may read
    const int cq = (warp - 2) >> 2;                        // which 64 of the 256 columns
    float r2 = 0.f, s2 = 0.f;
    uint32_t g = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < sched.num_units && ok; u += gridDim.x) {
      const Unit un = unit_of(sched, u);
      if (lower && un.col0 > un.tm * BM + BM - 1) continue;
      const bool mine = cq * COLS_PER_THREAD < un.ncols;   // a half unit has columns for cq = 0, 1 only
      const int row0 = un.tm * BM + q * 32, col0 = un.col0 + cq * COLS_PER_THREAD;
      const int pf_at = num_flush > 6 ? num_flush - 6 : 0;
      float sums[COLS_PER_THREAD];
#pragma unroll
      for (int e = 0; e < COLS_PER_THREAD; ++e) sums[e] = 0.f;
      for (int f = 0; f < num_flush; ++f) {
        if (f == pf_at && mine) epilogue_prefetch<EPI>(epi, row0 + lane, col0, M, N);
        const int pb = (int)(g % NPART);
        ok = mbar_wait_warp(pfull0 + 8 * pb, (g / NPART) & 1u, abort_flag, status, wait_limit);
        if (!ok) break;
        tc_fence_after();
        if (mine) {
          const uint32_t taddr = tmem_base + (uint32_t)pb * BN + (uint32_t)(cq * COLS_PER_THREAD) +
                                 ((uint32_t)(q * 32) << 16);
          // two alternating groups of 8 columns: the adds of one group run while the next load is in flight
          uint32_t va[8], vb[8];
          tc_ld8_issue(taddr, va);
#pragma unroll
          for (int h = 0; h < 3; ++h) {
            tc_ld8_issue(taddr + 16 * h + 8, vb);
            tc_ld_wait();
            add8(sums + 16 * h, va);
            tc_ld8_issue(taddr + 16 * h + 16, va);
            add8(sums + 16 * h + 8, vb);
          }
          tc_ld8_issue(taddr + 56, vb);
          tc_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(pempty0 + 8 * pb);    // the partial is in registers: buffer free
          add8(sums + 48, va);
          add8(sums + 56, vb);
        } else {
          tc_fence_before();
          if (lane == 0) mbar_arrive(pempty0 + 8 * pb);
        }
        ++g;
      }
      if (!ok) break;
      if (mine)
        epilogue_block<EPI>(epi, row0, col0, M, N, sums, stage_all + (warp - 2) * STAGE_FLOATS, lane, r2, s2);
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
  if (abort_flag_s) {
    // A wait ran out and every role has stopped.  Before shared and tensor memory are given back: (thread 0, the
    // producer) every stage fill that was armed must have landed -- a stage with only the first of its two
    // arrivals gets the second one here, without bytes, so that its barrier can complete; (thread 32, the
    // issuer) every MMA issued so far must have completed, which a commit to a barrier of its own reports.
    // These waits are bounded as well and raise nothing: the status word already holds the timeout.
    if (threadIdx.x == 0) {
      const uint32_t armed = fill_state[0], par = fill_state[1], half = fill_state[2];
      for (int s = 0; s < STAGES; ++s)
        if (armed >> s & 1u) {
          if (half >> s & 1u) mbar_arrive(full0 + 8 * s);
          mbar_wait_quiet(full0 + 8 * s, par >> s & 1u);
        }
    }
    if (threadIdx.x == 32) {
      tc_commit(drain_bar);
      mbar_wait_quiet(drain_bar, 0u);
    }
    __syncthreads();
  }
  if (EPI == EPI_ADMM && threadIdx.x == 0) {
    float a = 0.f, b = 0.f;                  // fixed order over the worker warps
    for (int w = 0; w < WORKER_WARPS; ++w) {
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

// ------------------------------------------------------------------ one-plane products on CTA pairs
// The W-update products of the late iterations run on one fp16 plane per operand: one MMA per K step, so a
// 128 x 256 tile asks its SM for 48 KB of operands per 512 tensor-core cycles, more than the shared memory of one
// SM can keep in flight against the latency of L2 (measured: 57-60 % of the tensor peak).  Here two SMs work as a
// pair (a cluster of two CTAs, tcgen05.mma.cta_group::2) on a 256 x 256 tile: each CTA stages its own 128 rows of
// A and 128 of the 256 rows of B, 32 KB per K block, and the tensor cores of both read B from both shared
// memories.  The result of such a product need not be better than the 2^-12 of its operands, so the whole K range
// accumulates in tensor memory (one of two 256-column buffers per tile) and the workers take it once per tile,
// while the issuer already works on the next tile in the other buffer.
//   warp 0       TMA producer in both CTAs; the bytes of both are counted by the leader's (rank 0) mbarriers, which
//                the leader's producer alone arms;
//   warp 1       MMA issuer in the leader only: tcgen05.mma M = 256 and tcgen05.commit, which arrives on the
//                barriers of both CTAs;
//   warps 2-17   workers in both CTAs, each CTA on its own 128 rows: tensor memory -> registers -> staging buffer ->
//                coalesced stores, then an arrival on the leader's "buffer free" barrier.
// No multicast load anywhere: every CTA fetches its own tiles.  Waits are bounded as in the single-CTA kernel;
// both CTAs always reach the cluster barrier at the end, so an expired wait in one cannot strand the other.
constexpr int PAIR_M = 2 * BM;
constexpr int PAIR_BOX = 64;             // rows of B per TMA box (a CTA takes two per tile, one per half tile)
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_A_BYTES = BM * BK * 2, PAIR_B_BYTES = (BN / 2) * BK * 2;
constexpr int PAIR_STAGE_BYTES = PAIR_A_BYTES + PAIR_B_BYTES;   // 32 KB

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrivals on a barrier that may live in the other CTA of the pair (cluster addresses).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// Tile load of one CTA of a pair into its own shared memory; the completion bytes go to `cluster_bar`, the
// leader's barrier.  (A plain load: no multicast.)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar,
                                                 int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(x), "r"(y)
      : "memory");
}
// Arrives, once the MMAs issued so far are complete, on the barrier at this offset in both CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "{\n.reg .b16 m;\nmov.b16 m, 3;\n"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n}"
      ::"r"(bar)
      : "memory");
}
__device__ __forceinline__ void tc_mma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__host__ __device__ constexpr uint32_t idesc_m256(uint32_t fmt, uint32_t n_cols) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((n_cols >> 3) << 17) | ((uint32_t)(PAIR_M >> 4) << 24);
}

// Work units of a pair: whole 256 x 256 tiles, except that the tiles of a last wave that would fill at most half
// of the pairs are cut into two 256 x 128 units.
__device__ __forceinline__ Schedule make_pair_schedule(int M, int N, int pairs) {
  Schedule s;
  s.tiles_m = (M + PAIR_M - 1) / PAIR_M;
  s.tiles_n = (N + BN - 1) / BN;
  const int tiles = s.tiles_m * s.tiles_n;
  const int waves = tiles / pairs, rem = tiles - waves * pairs;
  const bool split = rem > 0 && 2 * rem <= pairs;
  s.full_units = split ? waves * pairs : tiles;
  s.num_units = split ? waves * pairs + 2 * rem : tiles;
  return s;
}

template <int EPI>                          // EPI_STORE, or EPI_ACCUM (C += the product, whole tiles)
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ TcMaps maps, int M, int N, int K, uint32_t fmt, EpiParams epi,
                    int* status, long long wait_limit, int hold_loads) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * PAIR_STAGES + 2 * NPART + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ uint32_t fill_state[2];       // producer's record for the abort path: armed stages / their parities
  __shared__ __align__(16) float stage_all[WORKER_WARPS * STAGE_FLOATS];

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;
  const uint32_t rank = cluster_ctarank();                 // 0: leader of the pair
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  const uint32_t full0 = smem_u32(&bars[0]);
  const uint32_t empty0 = smem_u32(&bars[PAIR_STAGES]);
  const uint32_t pfull0 = smem_u32(&bars[2 * PAIR_STAGES]);
  const uint32_t pempty0 = smem_u32(&bars[2 * PAIR_STAGES + NPART]);
  const uint32_t drain_bar = smem_u32(&bars[2 * PAIR_STAGES + 2 * NPART]);

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    fill_state[0] = fill_state[1] = 0u;
    mbar_init(drain_bar, 1);
    for (int s = 0; s < PAIR_STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);                         // the leader's producer arrives, expecting the bytes of both
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < NPART; ++a) {
      mbar_init(pfull0 + 8 * a, 1);
      mbar_init(pempty0 + 8 * a, 2 * WORKER_WARPS);        // the workers of both CTAs (the leader's is used)
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(
                     smem_u32(&tmem_base_slot))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                      // the peer's barriers exist before any remote arrival
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  const Schedule sched = make_pair_schedule(M, N, num_pairs);
  const int num_kb = (K + BK - 1) / BK;

  if (warp == 0) {
    // ===================== TMA producer (both CTAs) =====================
    if (lane == 0 && !hold_loads) {
      int stage = 0;
      uint32_t phase = 0, armed = 0u, par = 0u;
      bool ok = true;
      for (int u = pair; u < sched.num_units && ok; u += num_pairs) {
        const Unit un = unit_of(sched, u);
        const int half_cols = un.ncols / 2;                // B rows staged by this CTA
        const int boxes = half_cols / PAIR_BOX;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag, status, wait_limit);
          if (!ok) break;
          const uint32_t sbase = tiles_base + stage * PAIR_STAGE_BYTES;
          const uint32_t fb = map_to_cta(full0 + 8 * stage, 0);           // the leader's barrier
          // The leader expects the bytes of both CTAs (each loads the same amount) with a local arrival; the peer
          // only issues its loads, whose completion bytes go to the leader's barrier.  (An arrival of the peer on
          // the leader's barrier for every stage, with cluster-scope release, was measured: it held the producer
          // ~1500 cycles per K block and the tensor pipe at 28 %.)
          if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * (PAIR_A_BYTES + boxes * PAIR_BOX * BK * 2));
          armed |= 1u << stage;
          par = (par & ~(1u << stage)) | (phase << stage);
          tma_load_2d_pair(sbase, &maps.a[0], fb, kb * BK, un.tm * PAIR_M + (int)rank * BM);
          // this CTA's half of B: one box of 128 rows for a whole tile (map b[1]), one of 64 for a half tile (b[0])
          tma_load_2d_pair(sbase + PAIR_A_BYTES, boxes == 2 ? &maps.b[1] : &maps.b[0], fb, kb * BK,
                           un.col0 + (int)rank * half_cols);
          if (++stage == PAIR_STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      fill_state[0] = armed;
      fill_state[1] = par;
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (leader CTA) =====================
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t g = 0;                        // unit counter, shared sequence with the workers
      bool ok = true;
      for (int u = pair; u < sched.num_units && ok; u += num_pairs) {
        const Unit un = unit_of(sched, u);
        const uint32_t idesc = idesc_m256(fmt, (uint32_t)un.ncols);
        const int pb = (int)(g % NPART);
        ok = mbar_wait(pempty0 + 8 * pb, ((g / NPART) & 1u) ^ 1u, abort_flag, status, wait_limit);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)pb * BN;
        uint32_t accumulate = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, status, wait_limit);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sbase = tiles_base + stage * PAIR_STAGE_BYTES;
          const uint64_t a_desc = make_kmajor_sw128_desc(sbase);
          const uint64_t b_desc = make_kmajor_sw128_desc(sbase + PAIR_A_BYTES);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16) {
            const uint64_t koff = (uint64_t)((k16 * 32) >> 4);   // 16 elements = 32 bytes along K
            tc_mma_f16_pair(d_tmem, a_desc + koff, b_desc + koff, idesc, accumulate);
            accumulate = 1;
          }
          tc_commit_pair(empty0 + 8 * stage);   // stage reusable in both CTAs once these MMAs have read it
          if (++stage == PAIR_STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        tc_commit_pair(pfull0 + 8 * pb);        // the tile is complete in both CTAs
        ++g;
      }
    }
  } else {
    // ===================== workers (both CTAs) =====================
    const int q = warp & 3;                                // tensor-memory lane quarter this warp may read
    const int cq = (warp - 2) >> 2;                        // which 64 of the 256 columns
    float r2 = 0.f, s2 = 0.f;
    uint32_t g = 0;
    bool ok = true;
    const uint32_t pempty_leader = map_to_cta(pempty0, 0);
    for (int u = pair; u < sched.num_units && ok; u += num_pairs) {
      const Unit un = unit_of(sched, u);
      const bool mine = cq * COLS_PER_THREAD < un.ncols;   // a half unit has columns for cq = 0, 1 only
      const int row0 = un.tm * PAIR_M + (int)rank * BM + q * 32, col0 = un.col0 + cq * COLS_PER_THREAD;
      const int pb = (int)(g % NPART);
      ok = mbar_wait_warp(pfull0 + 8 * pb, (g / NPART) & 1u, abort_flag, status, wait_limit);
      if (!ok) break;
      tc_fence_after();
      float sums[COLS_PER_THREAD];
      if (mine) {
        const uint32_t taddr = tmem_base + (uint32_t)pb * BN + (uint32_t)(cq * COLS_PER_THREAD) +
                               ((uint32_t)(q * 32) << 16);
#pragma unroll
        for (int h = 0; h < COLS_PER_THREAD / 8; ++h) {
          uint32_t v[8];
          tc_ld8_issue(taddr + 8 * h, v);
          tc_ld_wait();
#pragma unroll
          for (int e = 0; e < 8; ++e) sums[8 * h + e] = __uint_as_float(v[e]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(pempty_leader + 8 * pb);   // in registers: the buffer is free
      ++g;
      if (mine)
        epilogue_block<EPI>(epi, row0, col0, M, N, sums, stage_all + (warp - 2) * STAGE_FLOATS, lane, r2, s2);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (abort_flag_s) {
    // as in the single-CTA kernel: the fills this CTA armed must have landed (they are counted on the leader's
    // barriers, which the leader waits for, the peer being held at the cluster barrier below meanwhile), and the
    // MMAs issued must have completed, before shared and tensor memory are given back
    if (threadIdx.x == 0 && rank == 0) {
      const uint32_t armed = fill_state[0], par = fill_state[1];
      for (int s = 0; s < PAIR_STAGES; ++s)
        if (armed >> s & 1u) mbar_wait_quiet(full0 + 8 * s, par >> s & 1u);
    }
    if (threadIdx.x == 32 && rank == 0) {
      tc_commit_pair(drain_bar);             // (every tcgen05 instruction of a kernel names the same CTA group)
      mbar_wait_quiet(drain_bar, 0u);
    }
    if (threadIdx.x == 64) {                 // loads of this CTA that the leader never armed a barrier for: let them land
      const long long t0 = clock64();
      while (clock64() - t0 < 100000LL) {
      }
    }
    __syncthreads();
  }
  cluster_sync_all();                        // both CTAs are done with tensor memory and with remote arrivals
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
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
static cudaError_t launch_tc(Ctx* c, const TcMaps& maps, int M, int N, int K, uint32_t fmt,
                             const EpiParams& epi, int flush_kb = 0) {
  constexpr int STAGE_BYTES = NP * (BM * BK * 2 + BN * BK * 2);
  constexpr int STAGES = (NP == 1) ? 4 : 2;
  const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
  const cudaError_t ea = ensure_dynamic_smem((const void*)gemm_tc_kernel<NP, EPI>, (int)smem);
  if (ea != cudaSuccess) return ea;
  const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  const int grid = tiles < c->num_sms ? tiles : c->num_sms;
  gemm_tc_kernel<NP, EPI><<<grid, TC_THREADS, smem, c->stream>>>(maps, M, N, K, fmt, epi, c->status,
                                                                   c->wait_limit_cycles, c->hold_loads, flush_kb);
  c->launches++;
  return cudaGetLastError();
}

// Row-major 16-bit plane -> tensor map with the given box height (defined below).
static bool encode_plane(CUtensorMap* map, const bf16* ptr, long long rows, long long cols, long long ld,
                         int box_rows, int f16);

static cudaError_t launch_tc_pair(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi) {
  TcMaps maps;
  if (!encode_plane(&maps.a[0], A.hi, M, K, A.ld, BM, A.f16) ||
      !encode_plane(&maps.b[0], B.hi, N, K, B.ld, PAIR_BOX, B.f16) ||
      !encode_plane(&maps.b[1], B.hi, N, K, B.ld, 2 * PAIR_BOX, B.f16))
    return cudaErrorInvalidValue;
  maps.a[1] = maps.a[0];
  const size_t smem = (size_t)PAIR_STAGES * PAIR_STAGE_BYTES + 1024;
  const bool accum = epi.kind == EPI_ACCUM;
  auto kernel = accum ? gemm_tc_pair_kernel<EPI_ACCUM> : gemm_tc_pair_kernel<EPI_STORE>;
  const cudaError_t ea = ensure_dynamic_smem((const void*)kernel, (int)smem);
  if (ea != cudaSuccess) return ea;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (c->num_sms / 2));
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // pairs that can be resident at once: a persistent kernel must not launch more, or the surplus would run after
  // the others (asked once per context, which belongs to one device)
  if (c->pair_clusters == 0) {
    int nc = 0;
    if (cudaOccupancyMaxActiveClusters(&nc, kernel, &cfg) != cudaSuccess || nc < 1) {
      c->pair_clusters = -1;
      cudaGetLastError();
    } else {
      c->pair_clusters = nc < c->num_sms / 2 ? nc : c->num_sms / 2;
    }
  }
  if (c->pair_clusters < 1) return cudaErrorNotSupported;
  const int tiles = ((M + PAIR_M - 1) / PAIR_M) * ((N + BN - 1) / BN);
  const int pairs = tiles < c->pair_clusters ? tiles : c->pair_clusters;
  cfg.gridDim = dim3(2 * pairs);
  const uint32_t fmt = A.f16 ? 0u : 1u;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, maps, M, N, K, fmt, epi, c->status,
                                     c->wait_limit_cycles, c->hold_loads);
  c->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t gemm_tc(Ctx* c, Planes A, Planes B, int M, int N, int K, const EpiParams& epi_in) {
  const int na = A.lo ? 2 : 1, nb = B.lo ? 2 : 1;
  if (na != nb || A.f16 != B.f16) return cudaErrorInvalidValue;   // one MMA takes A and B of one type
  if ((A.ld & 7) || (B.ld & 7)) return cudaErrorInvalidValue;
  TcMaps maps;
  bool ok = encode_plane(&maps.a[0], A.hi, M, K, A.ld, BM, A.f16) &&
            encode_plane(&maps.b[0], B.hi, N, K, B.ld, BN_BOX, B.f16);
  if (na == 2) ok = ok && encode_plane(&maps.a[1], A.lo, M, K, A.ld, BM, A.f16);
  else maps.a[1] = maps.a[0];
  if (nb == 2) ok = ok && encode_plane(&maps.b[1], B.lo, N, K, B.ld, BN_BOX, B.f16);
  else maps.b[1] = maps.b[0];
  if (!ok) return cudaErrorInvalidValue;
  EpiParams epi = epi_in;
  epi.row_inv = A.row_inv;
  epi.a_inv = A.all_inv;
  epi.b_inv = B.all_inv;
  const uint32_t idesc = A.f16 ? 0u : 1u;                  // operand format: 0 = fp16, 1 = bf16
  // one fp16 plane and a plain store (or a sum into whole tiles of C), large enough for 256 x 256 tiles: the
  // CTA-pair kernel
  const bool pair_epi = epi.kind == EPI_STORE || (epi.kind == EPI_ACCUM && !epi.lower_only);
  if (na == 1 && A.f16 && pair_epi && c->use_pair_kernel && M >= PAIR_M && N >= BN && c->num_sms >= 2) {
    const cudaError_t ep = launch_tc_pair(c, A, B, M, N, K, epi);
    if (ep != cudaErrorNotSupported) return ep;           // no room for a pair on this device: single-CTA kernel
  }
  if (na == 1) {
    if (epi.kind == EPI_ACCUM) return launch_tc<1, EPI_ACCUM>(c, maps, M, N, K, idesc, epi);
    // one fp16 plane and a plain store: a W-update product of the late iterations, whose result need not be better
    // than the 2^-12 of its operands: the whole K range accumulates in tensor memory
    if (epi.kind == EPI_STORE) return launch_tc<1, EPI_STORE>(c, maps, M, N, K, idesc, epi, A.f16 ? c->one_plane_flush_kb : 0);
    return cudaErrorInvalidValue;
  }
  switch (epi.kind) {
    case EPI_STORE: return launch_tc<2, EPI_STORE>(c, maps, M, N, K, idesc, epi);
    case EPI_ACCUM: return launch_tc<2, EPI_ACCUM>(c, maps, M, N, K, idesc, epi);
    case EPI_ADMM: return launch_tc<2, EPI_ADMM>(c, maps, M, N, K, idesc, epi);
  }
  return cudaErrorInvalidValue;
}

}  // namespace admmq
