// fp32-accurate dense products on the sm_100a tensor cores.
//
// Every product C = A * B is issued as three fp16 MMAs on a scaled two-term split of the operands,
//     xs = x * 2^e                      (e per matrix, from max|x|, so that max|xs| lies in [2^14, 2^15))
//     x_hi = xs rounded to 11 significant bits      (exact in fp16 down to 2^-14)
//     x_lo = (xs - x_hi) * 2^11, rounded to fp16    (xs - x_hi is exact in fp32; the factor keeps it out of the
//                                                    fp16 subnormals, so the pair carries 22 bits down to 2^-14
//                                                    and at least 11 bits down to 2^-25 of the scaled range)
//     A * B ~= 2^-(eA+eB) [ A_hi B_hi + 2^-11 (A_hi B_lo + A_lo B_hi) ]      (the dropped lo*lo term is 2^-24 relative)
// Products of two 11-bit numbers are exact in the fp32 accumulator, so the split is as accurate as the same
// split on tf32 operands at twice the tensor-core rate and half the shared-memory footprint per operand.
//
// TMA brings fp32 tiles of the node-sized operand into shared memory; converter warps turn them into the two
// fp16 planes, which they write to tensor memory; the small operand (a weight matrix) arrives as two precomputed
// fp16 planes (K-major, 128-byte swizzle).  One thread issues tcgen05.mma; completion is tracked with mbarriers;
// two sets of four accumulate warps take the output tiles of a block in turn: a set reads each K block's main term
// from tensor memory, adds it to a register accumulator and finally applies the scaling and the fused epilogue --
// while it is in that epilogue the other set already accumulates the next tile, so the tensor pipe never waits for
// a store phase.
//
// Tile: 128 x 128 outputs per CTA, 64-deep K blocks, 3 stages of 64 KB.  Tensor memory (512 columns): two
// accumulator tiles for the main term, one for the correction terms, two slots for the planes of A.
// Every wait is bounded; a wait that expires raises an error word in global memory and the CTA drains and exits.
#pragma once

#include <cuda_fp16.h>

#include <type_traits>

#include "common.cuh"
#include "gemm_simt.cuh"   // epilogue functors
#include "tc_ptx.cuh"

namespace pd {

constexpr int TC_BM = 128, TC_BN = 128, TC_BK = 64, TC_STAGES = 3;
constexpr int TC_KSTEPS = TC_BK / 16;                          // MMAs (K = 16) per pair of planes and K block
constexpr int TC_FLUSH = 1;                                    // K blocks per read-out of the main accumulator
constexpr int TC_PLANE_BYTES = 128 * TC_BK * 2;                // 16 KB: one 128 x 64 fp16 operand plane
constexpr int TC_STAGE_BYTES = 4 * TC_PLANE_BYTES;             // A_hi, A_lo, B_hi, B_lo (= two fp32 tiles of 128 x 64)
// Four warpgroups (register budgets are set per warpgroup): 0 = TMA warp, MMA warp and two idle warps; 1 = four
// converter warps (one 32-lane quarter of tensor memory each); 2, 3 = the two accumulate sets, four warps each (a
// warp owns one quarter of the tile's rows and all 128 columns: 128 accumulators per thread).
// Registers: the block is launched with 512 x 128 = 65536; warpgroup 0 keeps 40 per thread, the converters 112, the
// accumulate sets take 168 (the compiler spills least there): 128 (40 + 112 + 2 x 168) = 62464 <= 65536, so every increase is satisfiable.
constexpr int TC_CONV_WARPS = 4;
constexpr int TC_CONV0 = 4, TC_ACC0 = 8;                      // first converter warp, first accumulate warp
constexpr int TC_THREADS = 512;
constexpr int TC_ACC_THREADS = 128;                            // threads of one accumulate set
constexpr int TC_REGS_LAUNCH = 128, TC_REGS_CTRL = 40, TC_REGS_CONV = 112, TC_REGS_ACC = 168;
static_assert(TC_THREADS * TC_REGS_LAUNCH <= 65536, "register file");
static_assert(128 * (TC_REGS_CTRL + TC_REGS_CONV + 2 * TC_REGS_ACC) <= TC_THREADS * TC_REGS_LAUNCH,
              "the warpgroups' register shares exceed what the block is launched with: an increase would wait for ever");
constexpr int TC_ACC_BUFS = 2;                                 // main-term accumulator tiles in tensor memory
static_assert(TC_ACC_BUFS == 2, "the accumulate warps keep one phase counter per buffer");
constexpr int TC_A_SLOTS = 2;                                  // K blocks of A planes in tensor memory
constexpr int TC_TMEM_COLS = 512;                              // 2 main tiles, 1 correction tile, 2 x (A_hi, A_lo)
constexpr uint32_t TC_COL_CORR = TC_ACC_BUFS * TC_BN;          // first column of the correction tile
constexpr uint32_t TC_COL_A = TC_COL_CORR + TC_BN;             // A slot a: columns + 64 a (hi), + 64 a + 32 (lo)
constexpr int TC_TR_BYTES = 8 * 32 * 32 * 4;                   // epilogue transpose: 8 warps x 32 rows x 32 columns
constexpr int TC_SMEM_BYTES = TC_STAGES * TC_STAGE_BYTES + TC_TR_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

__device__ __forceinline__ float tc_pow2(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

// One scaled value -> its two planes (as floats that fp16 holds exactly inside the normal range).
__device__ __forceinline__ void tc_split(float x, float scale, float &hi, float &lo) {
  const float xs = x * scale;
  hi = __uint_as_float((__float_as_uint(xs) + 0x1000u) & 0xFFFFE000u);     // 11 significant bits, nearest
  lo = (xs - hi) * 2048.0f;
}
// Eight consecutive values -> 16 bytes of the hi plane and 16 bytes of the lo plane.
__device__ __forceinline__ void tc_split8(const float (&x)[8], float scale, uint4 &h, uint4 &l) {
  float hi[8], lo[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) tc_split(x[i], scale, hi[i], lo[i]);
  auto pack = [](float a, float b) {
    const __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t *>(&v);
  };
  h = make_uint4(pack(hi[0], hi[1]), pack(hi[2], hi[3]), pack(hi[4], hi[5]), pack(hi[6], hi[7]));
  l = make_uint4(pack(lo[0], lo[1]), pack(lo[2], lo[3]), pack(lo[4], lo[5]), pack(lo[6], lo[7]));
}

// Epilogues store their result unless they say otherwise (kStore = false).
template <class Epi, class = void> struct epi_stores { static constexpr bool value = true; };
template <class Epi> struct epi_stores<Epi, std::enable_if_t<!Epi::kStore>> { static constexpr bool value = false; };
// An epilogue that wants nothing but the sum of squares of the product may say kCoarse = true: the product is then
// issued as the main term A_hi B_hi alone (one MMA instead of three).  Each term then carries an independent relative
// rounding of 2^-11 instead of 2^-22; over the 1e6..1e9 squares of the sum these average out to far below the
// single-precision accuracy of the sum itself.
// An epilogue whose sum of squares is that of the product itself, not of what it stores, says kSumsqOfAcc = true.
template <class Epi, class = void> struct epi_sumsq_acc { static constexpr bool value = false; };
template <class Epi> struct epi_sumsq_acc<Epi, std::enable_if_t<Epi::kSumsqOfAcc>> { static constexpr bool value = true; };
// An epilogue that can also leave an fp16 copy of its result (see EpiGradT) says kHalfCopy = true.
template <class Epi, class = void> struct epi_half_copy { static constexpr bool value = false; };
template <class Epi> struct epi_half_copy<Epi, std::enable_if_t<Epi::kHalfCopy>> { static constexpr bool value = true; };
template <class Epi, class = void> struct epi_coarse { static constexpr bool value = false; };
template <class Epi> struct epi_coarse<Epi, std::enable_if_t<Epi::kCoarse>> { static constexpr bool value = true; };

struct TcParams {
  int M, N, K;            // output rows, output columns, contraction length
  int k_chunk;            // contraction slice (multiple of TC_BK); K rounded up if not split
  int n_split;            // number of contraction slices; slice z writes its own partial output
  size_t c_split_stride;  // elements between the partial outputs of consecutive slices
  int *error;             // set to 1 if a bounded wait expired
  const uint32_t *amax_a; // bit pattern of max|A| (device word) when A is converted in the kernel; nullptr = no scaling
  const uint32_t *amax_b; // the same for B when B is converted in the kernel (TC_RAW_MN)
  const int *exp_a;       // scaling exponent stored with the precomputed planes of A (TC_PLANES)
  const int *exp_b;       // scaling exponent stored with the precomputed planes of B
  // Tail balancing (n_split == 1 only): output tiles from tail_begin on are cut into tail_split contraction
  // slices, one work unit each, so that the last, partly filled round of the persistent grid is shorter.
  // A slice leaves its accumulators in tail_ws; the warp that finds itself last (tail_count) adds the slices
  // in slice order and runs the epilogue.  tail_split <= 1 switches this off.
  int tail_begin, tail_split;
  float *tail_ws;         // [tiles from tail_begin][tail_split][4 row quarters][128][32] floats
  int *tail_count;        // [tiles from tail_begin][4 row quarters], zero before and after every launch
  float mul = 1.0f;       // factor applied to the result after the power-of-two scalings (integer operands, see ZERO)
};

// MODE TC_RAW_K:  A is [M][K] fp32, contiguous along K (a node-major matrix, rows = nodes), converted in the kernel;
//                  B arrives as two fp16 planes [N][K] (map_b = hi, map_blo = lo), contiguous along K.
// The contraction over nodes of the W-gradient has both operands node-major, i.e. contiguous along their output
// index, A = [K][M], B = [K][N], and comes in two forms:
// MODE TC_RAW_MN:  both arrive as fp32 tiles and the converter warps transpose while they split (A to tensor
//                  memory, B in place in shared memory).  Every output tile converts its operand tiles again, so
//                  this form suits outputs with few tiles.
// MODE TC_PLANES:  both arrive as fp16 planes [M][K], [N][K] (map_a / map_alo, map_b / map_blo), transposed and
//                  split once by transpose_planes_kernel; the converter warps have nothing to do.
//
// Persistent: the grid has at most one block per SM and block i works on output tiles i, i + gridDim.x, ...
// (column tile fastest, so that neighbouring blocks share the streamed operand in L2).  All roles keep running
// counters over K blocks, so the producer prefetches the next tile while the current one is in its epilogue.
//
// The tensor cores add into their fp32 accumulator with truncation, which costs about 2^-24 of the
// accumulator per MMA and always in the same direction.  To keep fp32-class accuracy the main term
// A_hi B_hi is accumulated in tensor memory for ONE K block only (4 MMAs): after each block the accumulate
// warps read it out and add it to a register accumulator with round-to-nearest, while the MMAs of the next
// block fill the other buffer.  The two correction terms are 2^-11 of the main term, so they are summed over
// the whole contraction in a fourth tensor-memory tile and added once at the end.
//
// ZERO (TC_PLANES only): bit 0 = the lo plane of A is identically zero, bit 1 = the lo plane of B is.  An operand of
// pdADMM-G-Q that lies on a level set {c s} (the quantised p, or the difference of two of them) is the spacing s times
// a small integer, and integers up to 2048 are exact in one fp16 plane: its plane holds the integers, there is no lo
// plane to load and no MMA for it (two MMAs per product instead of three), and prm.mul = s restores the values.
enum : int { TC_RAW_K = 0, TC_RAW_MN = 1, TC_PLANES = 2 };
template <int MODE, class Epi, int ZERO = 0>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_alo,
               const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_blo,
               const TcParams prm, Epi epi, double *__restrict__ partials) {
  constexpr bool PP = MODE == TC_PLANES, MN = MODE == TC_RAW_MN, COARSE = epi_coarse<Epi>::value || ZERO == 3;
  // which lo planes are loaded and used (a product that only wants its squared norm uses neither, and lets the main
  // term accumulate in tensor memory over the whole contraction: the truncation of that accumulation, 1e-5 relative,
  // does not matter to a norm that only starts a search)
  constexpr bool A_LO = !(ZERO & 1) && !COARSE, B_LO = !(ZERO & 2) && !COARSE;
  constexpr int FLUSH = COARSE ? (1 << 30) : TC_FLUSH;        // K blocks per read-out of the main accumulator
  static_assert(ZERO == 0 || MODE == TC_PLANES, "operands without a lo plane come as planes");
  constexpr uint32_t STAGE_TX = MODE == TC_PLANES ? (uint32_t)(2 + (A_LO ? 1 : 0) + (B_LO ? 1 : 0)) * TC_PLANE_BYTES
                              : MODE == TC_RAW_K  ? (uint32_t)(3 + (B_LO ? 1 : 0)) * TC_PLANE_BYTES
                                                  : (uint32_t)TC_STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *tr_base = smem + TC_STAGES * TC_STAGE_BYTES;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tr_base + TC_TR_BYTES);
  uint64_t *full_bar = bars, *conv_bar = bars + TC_STAGES, *empty_bar = bars + 2 * TC_STAGES;
  uint64_t *acc_full = bars + 3 * TC_STAGES, *acc_empty = acc_full + 2 * TC_ACC_BUFS;     // acc_full: [set][buffer]
  uint64_t *corr_empty = acc_empty + TC_ACC_BUFS, *drain_bar = corr_empty + 1, *a_empty = drain_bar + 1;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(a_empty + TC_A_SLOTS);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  volatile int *skip_flag = abort_flag + 1;           // an earlier block gave up: this one does no work

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int ACC0 = TC_ACC0;                        // first accumulate warp
  const int tiles_n = (prm.N + TC_BN - 1) / TC_BN, tiles_m = (prm.M + TC_BM - 1) / TC_BM;
  const int n_out_tiles = tiles_n * tiles_m * prm.n_split;
  const bool tail_on = prm.tail_split > 1;
  const int tail_begin = tail_on ? prm.tail_begin : n_out_tiles;
  const int n_tiles = tail_begin + (n_out_tiles - tail_begin) * (tail_on ? prm.tail_split : 1);   // work units

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&conv_bar[s], 32 * TC_CONV_WARPS);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < TC_ACC_BUFS; ++b) {
      ptx::mbar_init(&acc_full[b], 1);
      ptx::mbar_init(&acc_full[TC_ACC_BUFS + b], 1);
      ptx::mbar_init(&acc_empty[b], TC_ACC_THREADS);
    }
    ptx::mbar_init(corr_empty, TC_ACC_THREADS);
    ptx::mbar_init(drain_bar, 1);
    for (int a = 0; a < TC_A_SLOTS; ++a) ptx::mbar_init(&a_empty[a], 1);
    *abort_flag = 0;
    // One thread reads the error word for the whole block, so that all warps take the same path: every block still
    // allocates and releases its tensor memory and passes both block-wide barriers.
    *skip_flag = *reinterpret_cast<volatile int *>(prm.error) != 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&map_a);
    ptx::prefetch_tmap(&map_b);
    ptx::prefetch_tmap(&map_blo);
    if (PP && A_LO) ptx::prefetch_tmap(&map_alo);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TC_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // scaling exponents of the two operands (written by earlier kernels of the stream)
  const int exp_a = PP ? (prm.exp_a ? *prm.exp_a : 0) : (prm.amax_a ? tc_scale_exp(*prm.amax_a) : 0);
  const int exp_b = MN ? (prm.amax_b ? tc_scale_exp(*prm.amax_b) : 0) : (prm.exp_b ? *prm.exp_b : 0);

  // work unit -> (row tile origin, column tile origin, first and number of K blocks); a unit is an output tile or,
  // in the tail, one contraction slice of an output tile
  auto tile_coords = [&](int unit, int &m0, int &n0, int &k_begin, int &n_kb, int &z) {
    int tile = unit, slice = 0;
    if (unit >= tail_begin) {
      tile = tail_begin + (unit - tail_begin) / prm.tail_split;
      slice = (unit - tail_begin) % prm.tail_split;
    }
    z = tile / (tiles_m * tiles_n);
    const int rem = tile - z * tiles_m * tiles_n;
    m0 = (rem / tiles_n) * TC_BM;
    n0 = (rem % tiles_n) * TC_BN;
    k_begin = z * prm.k_chunk;
    const int k_end = min(prm.K, k_begin + prm.k_chunk);
    n_kb = (max(k_end - k_begin, 0) + TC_BK - 1) / TC_BK;
    if (unit >= tail_begin) {
      const int kb0 = slice * n_kb / prm.tail_split, kb1 = (slice + 1) * n_kb / prm.tail_split;
      k_begin += kb0 * TC_BK;
      n_kb = kb1 - kb0;
    }
  };

  // Register budgets per warpgroup (every warp of a warpgroup executes the same instruction; the choice is
  // block-uniform, so a block that skips its work leaves the budgets alone).
  const bool skip = *skip_flag != 0;
  if (skip) {
    // nothing: do not queue work behind a block whose bounded wait expired
  } else if (warp < TC_CONV0) {
   ptx::setmaxnreg_dec<TC_REGS_CTRL>();
   if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (one lane)
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        int m0, n0, k_begin, n_kb, z;
        tile_coords(tile, m0, n0, k_begin, n_kb, z);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % TC_STAGES, use = it / TC_STAGES;
          if (use > 0 && !ptx::mbar_wait(&empty_bar[s], (use - 1) & 1, abort_flag)) { ok = false; break; }
          uint8_t *st = smem + s * TC_STAGE_BYTES;
          const int k0 = k_begin + kb * TC_BK;
          ptx::mbar_expect_tx(&full_bar[s], STAGE_TX);
          if (MN) {
            // fp32 [64 contraction rows][128 output indices], 512-byte rows, no swizzle (only the converters read it)
            ptx::tma_load_2d(st, &map_a, m0, k0, &full_bar[s]);
            ptx::tma_load_2d(st + 2 * TC_PLANE_BYTES, &map_b, n0, k0, &full_bar[s]);
          } else {
            if (PP) {
              ptx::tma_load_2d(st, &map_a, k0, m0, &full_bar[s]);
              if (A_LO) ptx::tma_load_2d(st + TC_PLANE_BYTES, &map_alo, k0, m0, &full_bar[s]);
            } else {
              // fp32 [128 rows][64 floats] as two 128-byte-swizzled boxes of 32 floats
              ptx::tma_load_2d(st, &map_a, k0, m0, &full_bar[s]);
              ptx::tma_load_2d(st + TC_PLANE_BYTES, &map_a, k0 + 32, m0, &full_bar[s]);
            }
            // fp16 planes of B as the MMA reads them
            ptx::tma_load_2d(st + 2 * TC_PLANE_BYTES, &map_b, k0, n0, &full_bar[s]);
            if (B_LO) ptx::tma_load_2d(st + 3 * TC_PLANE_BYTES, &map_blo, k0, n0, &full_bar[s]);
          }
        }
      }
      if (*abort_flag) {
        // copies in flight must land before the block's shared memory is released
        for (int j = max(it - TC_STAGES, 0); j < it; ++j)
          ptx::mbar_wait(&full_bar[j % TC_STAGES], (j / TC_STAGES) & 1, abort_flag, 200000000ll, false);
      }
    }
   } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_f16(TC_BM, TC_BN);
      const uint32_t d_corr = tmem_base + TC_COL_CORR;
      // A: tensor memory, 8 columns per K step.  B: shared-memory descriptors with a constant high word; the low
      // word of stage 0 advances by whole stages / K steps (K-major planes with 128-byte rows; 16 fp16 are 32 bytes)
      const uint32_t hi_b = ptx::smem_desc_hi(false, TC_BK * 2);
      const uint32_t lo_a0 = ptx::smem_desc_lo(ptx::smem_u32(smem), false, 0);       // PP: A planes in shared memory too
      const uint32_t lo_b0 = ptx::smem_desc_lo(ptx::smem_u32(smem) + 2 * TC_PLANE_BYTES, false, 0);
      uint64_t *const ready_bar = PP ? full_bar : conv_bar;      // what tells that a stage's operands are in place
      constexpr uint32_t step_b = 32u >> 4;
      bool ok = true;
      // running state: stage s with phase bit sp, accumulator buffer b with phase bit bp (of its *previous* use),
      // and whether the barriers of the coming K block were already seen complete by the probe below
      int s = 0, b = 0, ti = 0;
      uint32_t sp = 0, bp = 1, aslot = 0;
      bool first_round = true, seen_conv = false, seen_acc = false;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++ti) {
        int m0, n0, k_begin, n_kb, z;
        tile_coords(tile, m0, n0, k_begin, n_kb, z);
        for (int kb = 0; kb < n_kb && ok; ++kb) {
          const bool first = kb % FLUSH == 0, last = kb % FLUSH == FLUSH - 1 || kb == n_kb - 1;
          if (!seen_conv) ok = ptx::mbar_wait(&ready_bar[s], sp, abort_flag);
          if (ok && first && !first_round && !seen_acc) ok = ptx::mbar_wait(&acc_empty[b], bp, abort_flag);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t ta = tmem_base + TC_COL_A + aslot * 64u, lb = lo_b0 + (uint32_t)s * (TC_STAGE_BYTES >> 4);
          const uint32_t la = lo_a0 + (uint32_t)s * (TC_STAGE_BYTES >> 4);
          const uint32_t d = tmem_base + (uint32_t)(b * TC_BN);
          // next K block's stage and, if it starts a new group, its accumulator buffer
          const int s_next = s + 1 == TC_STAGES ? 0 : s + 1;
          const uint32_t sp_next = s + 1 == TC_STAGES ? sp ^ 1u : sp;
          const int b_next = b + 1 == TC_ACC_BUFS ? 0 : b + 1;
          const uint32_t bp_next = b + 1 == TC_ACC_BUFS ? bp ^ 1u : bp;
          const bool round_next = first_round && b + 1 != TC_ACC_BUFS;
          // the MMAs of K step kk: the two correction terms and / or the main term
          auto issue = [&](int kk, bool corr, bool main) {
            const uint32_t ah = ta + 8u * kk, al = ah + 32u;
            const uint64_t dbh = ptx::smem_desc(hi_b, lb + kk * step_b);
            const uint64_t dbl = ptx::smem_desc(hi_b, lb + (TC_PLANE_BYTES >> 4) + kk * step_b);
            if constexpr (PP) {
              const uint64_t dah = ptx::smem_desc(hi_b, la + kk * step_b);
              const uint64_t dal = ptx::smem_desc(hi_b, la + (TC_PLANE_BYTES >> 4) + kk * step_b);
              if (corr) {
                // the first correction MMA of a tile overwrites the tile, every later one accumulates
                if (A_LO) ptx::mma_f16(d_corr, dal, dbh, idesc, kb > 0 || kk > 0);
                if (B_LO) ptx::mma_f16(d_corr, dah, dbl, idesc, A_LO || kb > 0 || kk > 0);
              }
              if (main) ptx::mma_f16(d, dah, dbh, idesc, !first || kk > 0);
            } else {
              if (corr) {
                ptx::mma_f16_ts(d_corr, al, dbh, idesc, kb > 0 || kk > 0);
                ptx::mma_f16_ts(d_corr, ah, dbl, idesc, true);
              }
              if (main) ptx::mma_f16_ts(d, ah, dbh, idesc, !first || kk > 0);
            }
          };
          const bool split_first = !COARSE && kb == 0 && ti > 0;
          if (split_first) {
            // The correction tile still holds the previous output tile until the accumulate warps have read it:
            // the main-term MMAs of this block, which do not touch it, go first and keep the tensor pipe busy
            // while that read finishes.
#pragma unroll
            for (int kk = 0; kk < TC_KSTEPS; ++kk) issue(kk, false, true);
            ok = ptx::mbar_wait(corr_empty, (ti - 1) & 1, abort_flag);
            if (!ok) break;
            ptx::tc_fence_after_sync();
          }
#pragma unroll
          for (int kk = 0; kk < TC_KSTEPS; ++kk) {
            issue(kk, !COARSE, !split_first);
            if (kk == TC_KSTEPS - 2) {
              // probe the coming block's barriers while the tensor pipe still has work queued
              seen_conv = ptx::mbar_test_wait(&ready_bar[s_next], sp_next);
              seen_acc = last ? (round_next ? true : ptx::mbar_test_wait(&acc_empty[b_next], bp_next)) : true;
            }
          }
          ptx::mma_commit(&empty_bar[s]);          // stage can be refilled once these MMAs have read it
          if (!PP) {
            ptx::mma_commit(&a_empty[aslot]);      // and so can the A planes' slot in tensor memory
            aslot ^= 1u;
          }
          if (last) {
            // this group's partial product is complete.  Each accumulate set has its own pair of barriers: a set
            // is idle during the other set's tiles, and a waiter that lags by more than one phase of a barrier
            // would take an earlier completion of the same parity for its own.
            ptx::mma_commit(&acc_full[(ti & 1) * TC_ACC_BUFS + b]);
            if (b + 1 == TC_ACC_BUFS) first_round = false;
            b = b_next; bp = bp_next;
          }
          s = s_next; sp = sp_next;
        }
      }
      if (!ok) {
        // after an abandoned wait: let the MMAs already issued finish before tensor memory is released
        ptx::mma_commit(drain_bar);
        ptx::mbar_wait(drain_bar, 0, abort_flag, 200000000ll, false);
      }
    }
   }   // warps 2 and 3 of warpgroup 0 are spare
  } else if (warp < ACC0) {
    ptx::setmaxnreg_dec<TC_REGS_CONV>();
    // ---------------------------------------------------------------- converters (128 threads; idle with TC_PLANES)
    // The planes of A go to tensor memory, where the MMA reads them without touching shared memory: row i of the
    // tile lives in lane i, and a warp can only write the 32 lanes of its own quarter (warp index mod 4).  Thread
    // t = 32 (warp mod 4) + lane converts row t of the K block, 32 values at a time (16 + 16 columns per half).
    // TC_RAW_K:  the values come from the swizzled [128][64] fp32 tile (row t, 16-byte chunks).
    // TC_RAW_MN: the tile is [64][128] (contraction index first), so the thread reads a column; and B is converted
    //             too, in place in shared memory: thread tb reads the 64 values of output index tb, all 128 threads
    //             wait until everyone has read (the planes overwrite the fp32 tile), then the thread writes eight
    //             16-byte chunks of row tb of the hi and of the lo plane, chunk j at position j ^ (tb mod 8)
    //             (the 128-byte swizzle).
    if constexpr (!PP) {
      const int quarter = warp & 3;
      const int t = quarter * 32 + lane;
      const float scale_a = tc_pow2(exp_a), scale_b = tc_pow2(exp_b);
      const uint32_t sw = (uint32_t)(t & 7);
      bool ok = true;
      int it = 0;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        int m0, n0, k_begin, n_kb, z;
        tile_coords(tile, m0, n0, k_begin, n_kb, z);
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = it % TC_STAGES, use = it / TC_STAGES;
          ok = ptx::mbar_wait(&full_bar[s], use & 1, abort_flag);
          uint8_t *stage = smem + s * TC_STAGE_BYTES;
          const int aslot = it % TC_A_SLOTS, ause = it / TC_A_SLOTS;
          if (ok && ause > 0) ok = ptx::mbar_wait(&a_empty[aslot], (ause - 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);                  // the tensor-memory stores below are warp-wide
          if (ok) {
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              float v[32];
              if (MN) {
                const float *raw = reinterpret_cast<const float *>(stage);     // [64][128]
#pragma unroll
                for (int k = 0; k < 32; ++k) v[k] = raw[(32 * half + k) * 128 + t];
              } else {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                  const float4 q = *reinterpret_cast<const float4 *>(stage + half * TC_PLANE_BYTES + t * 128 +
                                                                     (((uint32_t)c ^ sw) << 4));
                  v[4 * c] = q.x; v[4 * c + 1] = q.y; v[4 * c + 2] = q.z; v[4 * c + 3] = q.w;
                }
              }
              uint32_t hreg[16], lreg[16];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                float x[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) x[i] = v[8 * j + i];
                uint4 h, l;
                tc_split8(x, scale_a, h, l);
                hreg[4 * j] = h.x; hreg[4 * j + 1] = h.y; hreg[4 * j + 2] = h.z; hreg[4 * j + 3] = h.w;
                lreg[4 * j] = l.x; lreg[4 * j + 1] = l.y; lreg[4 * j + 2] = l.z; lreg[4 * j + 3] = l.w;
              }
              const uint32_t col = tmem_base + ((uint32_t)(quarter * 32) << 16) + TC_COL_A + (uint32_t)aslot * 64u +
                                   16u * (uint32_t)half;
              ptx::tmem_st16(col, hreg);
              if constexpr (!COARSE) ptx::tmem_st16(col + 32u, lreg);
            }
          }
          if constexpr (MN) {
            uint8_t *region = stage + 2 * TC_PLANE_BYTES;
            const float *raw = reinterpret_cast<const float *>(region);      // [64][128]
            float v[64];
            if (ok) {
#pragma unroll
              for (int k = 0; k < 64; ++k) v[k] = raw[k * 128 + t];
            }
            // everyone has read its values of B (or someone gave up: then all stop here)
            if (ptx::named_barrier_or(1, 32 * TC_CONV_WARPS, !ok)) { ok = false; break; }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float x[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) x[i] = v[8 * j + i];
              uint4 h, l;
              tc_split8(x, scale_b, h, l);
              const uint32_t off = (uint32_t)t * 128u + (((uint32_t)j ^ sw) << 4);
              *reinterpret_cast<uint4 *>(region + off) = h;
              *reinterpret_cast<uint4 *>(region + TC_PLANE_BYTES + off) = l;
            }
            ptx::fence_proxy_async_smem();
          } else if (!ok) {
            break;
          }
          ptx::tmem_st_wait();
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&conv_bar[s]);
        }
      }
    }
  } else {
    ptx::setmaxnreg_inc<TC_REGS_ACC>();
    // ---------------------------------------------------------------- accumulate, then epilogue (2 sets x 128 threads)
    // The block's output tiles go to the two sets in turn.  Warp w of a set owns tensor-memory lanes 32 (w mod 4) ..
    // +31 = output rows m0 + that range, and all 128 columns of the tile.  Both sets count every K block, so that the
    // accumulator buffers and their barrier phases stay in step.
    const int aw = warp - ACC0, set = aw >> 2, quarter = warp & 3;
    const int lane_base = quarter * 32;
    float4 *tr = reinterpret_cast<float4 *>(tr_base) + (size_t)aw * 32 * 8;    // 32 rows x 8 float4 per warp
    // columns up to the leading dimension are written: those from N on come out as exact zeros (zero-filled
    // operand rows, zero padding of the epilogue inputs), which keeps the padding of every matrix zero
    const int n_pad = epi.ldc;
    bool ok = true;
    int it = 0, ti = 0;
    uint32_t uses0 = 0u, uses1 = 0u;                   // completions of this set's two acc_full barriers seen so far
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++ti) {
      int m0, n0, k_begin, n_kb, z;
      tile_coords(tile, m0, n0, k_begin, n_kb, z);
      const int n_grp = COARSE ? (n_kb > 0 ? 1 : 0) : n_kb;   // read-outs of the main accumulator for this tile
      if ((ti & 1) != set) { it += n_grp; continue; }    // the other set's tile
      if (m0 + lane_base + lane < prm.M) {          // this thread's row of the epilogue inputs, on its way to L2
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const int col = n0 + h * 32;
          if (col < n_pad) epi.prefetch(m0 + lane_base + lane, col);
        }
      }
      float acc[128];
#pragma unroll
      for (int j = 0; j < 128; ++j) acc[j] = 0.f;
      auto add_tile = [&](uint32_t col_base, float w) {       // acc += w * tile (w = 1: plain add)
        const uint32_t src = tmem_base + ((uint32_t)lane_base << 16) + col_base;
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          uint32_t v[32];
          ptx::tmem_ld32(src + 32u * h, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) acc[32 * h + j] = fmaf(w, __uint_as_float(v[j]), acc[32 * h + j]);
        }
      };
      for (int g = 0; g < n_grp && ok; ++g, ++it) {
        const int b = it % TC_ACC_BUFS;
        ok = ptx::mbar_wait(&acc_full[set * TC_ACC_BUFS + b], (b ? uses1 : uses0) & 1u, abort_flag);
        if (!ok) break;
        if (b) ++uses1; else ++uses0;
        ptx::tc_fence_after_sync();
        add_tile((uint32_t)(b * TC_BN), 1.0f);
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(&acc_empty[b]);
      }
      if (!ok) break;
      if (n_kb > 0) {
        if constexpr (!COARSE) {
          // correction terms: complete once the last block's commit has arrived (it covers every earlier MMA)
          add_tile(TC_COL_CORR, 1.0f / 2048.0f);
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(corr_empty);
        }
        // undo the operand scalings (two exact factors, so that neither leaves the range on its own)
        const int e1 = (exp_a + exp_b) / 2, e2 = exp_a + exp_b - e1;
        const float u1 = tc_pow2(-e1), u2 = tc_pow2(-e2);
#pragma unroll
        for (int j = 0; j < 128; ++j) acc[j] = (acc[j] * u1) * u2;
        if constexpr (ZERO != 0) {
          const float mul = prm.mul;
#pragma unroll
          for (int j = 0; j < 128; ++j) acc[j] *= mul;
        }
      }
      int out_tile = tile;
      if (tile >= tail_begin) {
        // contraction slice of a tail tile: park the accumulators; the last warp to arrive sums the slices
        const int u = tile - tail_begin, t_idx = u / prm.tail_split;
        out_tile = tail_begin + t_idx;
        float *mine = prm.tail_ws + ((size_t)u * 4 + quarter) * 4096;
#pragma unroll
        for (int j = 0; j < 128; ++j) mine[j * 32 + lane] = acc[j];
        __threadfence();
        __syncwarp();
        int prev = 0;
        if (lane == 0) prev = atomicAdd(prm.tail_count + t_idx * 4 + quarter, 1);
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev != prm.tail_split - 1) continue;
        __threadfence();
        if (lane == 0) prm.tail_count[t_idx * 4 + quarter] = 0;
#pragma unroll
        for (int j = 0; j < 128; ++j) acc[j] = 0.f;
        for (int sl = 0; sl < prm.tail_split; ++sl) {
          const float *part = prm.tail_ws + ((size_t)(t_idx * prm.tail_split + sl) * 4 + quarter) * 4096;
#pragma unroll
          for (int j = 0; j < 128; ++j) acc[j] += __ldcg(part + j * 32 + lane);
        }
      }
      // Epilogue.  Thread i of the warp holds row (lane_base + i), 128 columns.  The warp's piece goes through shared
      // memory 32 columns at a time: thread i writes its 8 float4 groups with the group index XOR-ed by (i mod 8)
      // (conflict-free 128-bit stores), then the warp reads the piece back transposed, so that the output is written,
      // and the inputs of the epilogue are read, in a coalesced pattern: the warp walks over its rows four at a
      // time, lanes 8g..8g+7 take row 4 step + g, 4 consecutive columns per lane.  The loads of four or eight steps
      // are issued together (rows past the end are clamped, their results dropped).
      double ss = 0.0;
      if constexpr (!epi_stores<Epi>::value) {
        // only the squared norm: straight from the registers (rows and columns outside the matrix hold exact zeros)
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 128; ++j) s4[j & 3] = fmaf(acc[j], acc[j], s4[j & 3]);
        ss = ((double)s4[0] + (double)s4[1]) + ((double)s4[2] + (double)s4[3]);
      } else {
        float *C = epi.C + (size_t)z * prm.c_split_stride;
        float ssf = 0.f;
        uint32_t mx = 0u;                  // largest magnitude stored by this thread
        float h_scale = 0.f;               // scaling of the fp16 copy, if one is wanted
        if constexpr (epi_half_copy<Epi>::value) {
          if (epi.H != nullptr) h_scale = tc_pow2(max(-100, min(100, *epi.h_exp)));
        }
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int jj = h * 8 + j;
            tr[lane * 8 + (j ^ (lane & 7))] = make_float4(acc[4 * jj], acc[4 * jj + 1], acc[4 * jj + 2], acc[4 * jj + 3]);
          }
          __syncwarp();
          const int col = n0 + h * 32 + 4 * (lane & 7);
          if (col < n_pad) {
            constexpr int BATCH = Epi::kInputs <= 1 ? 8 : 4;       // row steps whose loads are in flight together
#pragma unroll
            for (int s0 = 0; s0 < 8; s0 += BATCH) {
              float4 in[BATCH][Epi::kInputs > 0 ? Epi::kInputs : 1];
#pragma unroll
              for (int i = 0; i < BATCH; ++i) {
                const int r = 4 * (s0 + i) + (lane >> 3);
                if constexpr (!Epi::kDirect) epi.load(min(m0 + lane_base + r, prm.M - 1), col, in[i]);
              }
#pragma unroll
              for (int i = 0; i < BATCH; ++i) {
                const int r = 4 * (s0 + i) + (lane >> 3);
                const int row = m0 + lane_base + r;
                float4 o = tr[r * 8 + ((lane & 7) ^ (r & 7))];
                if constexpr (epi_sumsq_acc<Epi>::value) {
                  if (row < prm.M) ssf = fmaf(o.x, o.x, fmaf(o.y, o.y, fmaf(o.z, o.z, fmaf(o.w, o.w, ssf))));
                }
                if constexpr (!Epi::kDirect) o = epi.apply(col, o, in[i]);
                if (row < prm.M) {
                  if (Epi::kSumsq && !epi_sumsq_acc<Epi>::value) ssf = fmaf(o.x, o.x, fmaf(o.y, o.y, fmaf(o.z, o.z, fmaf(o.w, o.w, ssf))));
                  *reinterpret_cast<float4 *>(C + (size_t)row * epi.ldc + col) = o;
                  if constexpr (epi_half_copy<Epi>::value) {
                    if (epi.H != nullptr) {
                      float h0, h1, h2, h3, lo_unused;
                      tc_split(o.x, h_scale, h0, lo_unused); tc_split(o.y, h_scale, h1, lo_unused);
                      tc_split(o.z, h_scale, h2, lo_unused); tc_split(o.w, h_scale, h3, lo_unused);
                      const __half2 a = __floats2half2_rn(h0, h1), b = __floats2half2_rn(h2, h3);
                      *reinterpret_cast<uint2 *>(epi.H + (size_t)row * epi.ldc + col) =
                          make_uint2(*reinterpret_cast<const uint32_t *>(&a), *reinterpret_cast<const uint32_t *>(&b));
                    }
                  }
                  if constexpr (!Epi::kDirect) mx = max(mx, abs_bits(o));
                }
              }
            }
          }
        }
        ss = (double)ssf;
        if constexpr (!Epi::kDirect) {
          if (epi.amax != nullptr) commit_amax(mx, epi.amax);      // the output is an operand of a later product
        }
      }
      if (partials != nullptr) {          // one slot per tile and row quarter; a single block adds the slots in index order
        ss = warp_sum(ss);
        if (lane == 0) partials[(size_t)out_tile * 4 + quarter] = ss;
      }
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, TC_TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(prm.error, 1);
}

}  // namespace pd
