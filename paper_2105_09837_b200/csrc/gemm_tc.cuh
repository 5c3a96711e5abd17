// fp32-accurate dense products on the sm_100a tensor cores.
//
// Every product C = A * B is issued as three tf32 MMAs on an error-free split of the operands,
//     x = x_hi + x_lo,  x_hi = x rounded to tf32 (11 significant bits),  x_lo = x - x_hi (exact),
//     A * B ~= A_hi B_hi + A_hi B_lo + A_lo B_hi            (the dropped A_lo B_lo term is below 2^-24 relative),
// accumulated in fp32 in tensor memory.  TMA brings fp32 tiles into 128-byte-swizzled shared memory; four
// converter warps split the streamed operand in place (hi) and into a second buffer (lo); the small operand
// (a weight matrix) arrives as two precomputed planes.  One thread issues tcgen05.mma; completion is tracked
// with mbarriers; four more warps read each K block's partial product from tensor memory (each warp its own
// 32 lanes), add it to a register accumulator and finally apply the fused epilogue.
//
// Tile: 128 x 128 outputs per CTA, 32-float K blocks, 3 stages of 64 KB, two accumulator tiles in tensor memory.
// Every wait is bounded; a wait that expires raises an error word in global memory and the CTA drains and exits.
#pragma once

#include "common.cuh"
#include "gemm_simt.cuh"   // epilogue functors
#include "tc_ptx.cuh"

namespace pd {

constexpr int TC_BM = 128, TC_BN = 128, TC_BK = 32, TC_STAGES = 3;
constexpr int TC_FLUSH = 1;                                    // K blocks per read-out of the main accumulator
constexpr int TC_TILE_BYTES = 128 * TC_BK * 4;                 // 16 KB: one 128 x 32 fp32 operand tile
constexpr int TC_MN_CHUNK = TC_BK * 128;                       // MN-major tiles: 32 output indices x TC_BK rows
constexpr int TC_STAGE_BYTES = 4 * TC_TILE_BYTES;              // A_hi, A_lo, B_hi, B_lo
// warp 0: TMA, warp 1: MMA, then 4 (8) operand-split warps, then 8 accumulate + epilogue warps
// (two warps per 32-lane quarter of tensor memory, 64 columns each)
constexpr int TC_THREADS = 448;                                // 576 when both operands are split in the kernel
// number of operand-split warps: twice as many when both operands are split in shared memory (the contraction over
// nodes), where the split and not the MMA issue sets the pace
__host__ __device__ constexpr int tc_conv_warps(bool b_split) { return b_split ? 8 : 4; }
__host__ __device__ constexpr int tc_threads(bool b_split) { return 32 * (2 + tc_conv_warps(b_split) + 8); }
constexpr int TC_ACC_THREADS = 256;
constexpr int TC_ACC_BUFS = 3;                                 // main-term accumulator tiles in tensor memory
constexpr int TC_TMEM_COLS = 512;                              // 3 main tiles + 1 correction tile
constexpr int TC_TR_BYTES = 8 * 32 * 32 * 4;                   // epilogue transpose: 8 warps x 32 rows x 32 columns
constexpr int TC_SMEM_BYTES = TC_STAGES * TC_STAGE_BYTES + TC_TR_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

// x_hi: x rounded to the nearest tf32 number (11 significant bits).  x_lo = x - x_hi is then exact in fp32,
// at most 2^-12 |x| and of either sign, so what the MMA drops of it (its last bit) has no preferred direction.
__host__ __device__ __forceinline__ uint32_t tf32_hi(uint32_t bits) { return (bits + 0x1000u) & 0xFFFFE000u; }

struct TcParams {
  int M, N, K;            // output rows, output columns, contraction length
  int k_chunk;            // contraction slice (multiple of TC_BK); K rounded up if not split
  int n_split;            // number of contraction slices; slice z writes its own partial output
  size_t c_split_stride;  // elements between the partial outputs of consecutive slices
  int *error;             // set to 1 if a bounded wait expired
  // Tail balancing (n_split == 1 only): output tiles from tail_begin on are cut into tail_split contraction
  // slices, one work unit each, so that the last, partly filled round of the persistent grid is shorter.
  // A slice leaves its accumulators in tail_ws; the warp that finds itself last (tail_count) adds the slices
  // in slice order and runs the epilogue.  tail_split <= 1 switches this off.
  int tail_begin, tail_split;
  float *tail_ws;         // [tiles from tail_begin][tail_split][8 warps][64][32] floats
  int *tail_count;        // [tiles from tail_begin][8 warps], zero before and after every launch
};

// A_MN / B_MN: operand is stored contiguous along its output index (rows of the tile are K slices);
//              otherwise contiguous along K.
// B_SPLIT: B is one fp32 tensor split in shared memory like A; otherwise it arrives as two planes (map_b, map_blo).
//
// Persistent: the grid has at most one block per SM and block i works on output tiles i, i + gridDim.x, ...
// (column tile fastest, so that neighbouring blocks share the streamed operand in L2).  All roles keep running
// counters over K blocks, so the producer prefetches the next tile while the current one is in its epilogue.
//
// The tensor cores add into their fp32 accumulator with truncation, which costs about 2^-24 of the
// accumulator per MMA and always in the same direction.  To keep fp32-class accuracy the main term
// A_hi B_hi is accumulated in tensor memory for ONE K block only (4 MMAs): after each block the accumulate
// warps read it out and add it to a register accumulator with round-to-nearest, while the MMAs of the next
// block fill the other buffer.  The two correction terms are 2^-12 of the main term, so they are summed over
// the whole contraction in a third tensor-memory tile and added once at the end.
template <bool A_MN, bool B_MN, bool B_SPLIT, class Epi>
__global__ void __launch_bounds__(tc_threads(B_SPLIT), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_blo, const __grid_constant__ CUtensorMap map_c,
               const TcParams prm, Epi epi, double *__restrict__ partials) {
  if (*reinterpret_cast<volatile int *>(prm.error) != 0) return;   // an earlier block gave up: do not queue behind it
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *tr_base = smem + TC_STAGES * TC_STAGE_BYTES;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tr_base + TC_TR_BYTES);
  uint64_t *full_bar = bars, *conv_bar = bars + TC_STAGES, *empty_bar = bars + 2 * TC_STAGES;
  uint64_t *acc_full = bars + 3 * TC_STAGES, *acc_empty = acc_full + TC_ACC_BUFS;
  uint64_t *corr_empty = acc_empty + TC_ACC_BUFS, *drain_bar = corr_empty + 1;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(drain_bar + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int ACC0 = 2 + tc_conv_warps(B_SPLIT);              // first accumulate warp
  constexpr int CONV_T = 32 * tc_conv_warps(B_SPLIT);           // operand-split threads
  const int tiles_n = (prm.N + TC_BN - 1) / TC_BN, tiles_m = (prm.M + TC_BM - 1) / TC_BM;
  const int n_out_tiles = tiles_n * tiles_m * prm.n_split;
  const bool tail_on = prm.tail_split > 1;
  const int tail_begin = tail_on ? prm.tail_begin : n_out_tiles;
  const int n_tiles = tail_begin + (n_out_tiles - tail_begin) * (tail_on ? prm.tail_split : 1);   // work units

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&conv_bar[s], 32 * tc_conv_warps(B_SPLIT));
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < TC_ACC_BUFS; ++b) {
      ptx::mbar_init(&acc_full[b], 1);
      ptx::mbar_init(&acc_empty[b], TC_ACC_THREADS);
    }
    ptx::mbar_init(corr_empty, TC_ACC_THREADS);
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&map_a);
    ptx::prefetch_tmap(&map_b);
    if (!B_SPLIT) ptx::prefetch_tmap(&map_blo);
    if (Epi::kDirect) ptx::prefetch_tmap(&map_c);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TC_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

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
          ptx::mbar_expect_tx(&full_bar[s], (B_SPLIT ? 2 : 3) * TC_TILE_BYTES);
          if (A_MN) {
            ptx::tma_load_3d(st, &map_a, 0, k0, m0 / 32, &full_bar[s]);
          } else {
            ptx::tma_load_2d(st, &map_a, k0, m0, &full_bar[s]);
          }
          uint8_t *bh = st + 2 * TC_TILE_BYTES, *bl = st + 3 * TC_TILE_BYTES;
          if (B_MN) {
            ptx::tma_load_3d(bh, &map_b, 0, k0, n0 / 32, &full_bar[s]);
            if (!B_SPLIT) ptx::tma_load_3d(bl, &map_blo, 0, k0, n0 / 32, &full_bar[s]);
          } else {
            ptx::tma_load_2d(bh, &map_b, k0, n0, &full_bar[s]);
            if (!B_SPLIT) ptx::tma_load_2d(bl, &map_blo, k0, n0, &full_bar[s]);
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
      constexpr uint32_t idesc = ptx::idesc_tf32(TC_BM, TC_BN, A_MN, B_MN);
      const uint32_t d_corr = tmem_base + (uint32_t)(TC_ACC_BUFS * TC_BN);
      // descriptors: constant high words; the low word of stage 0 advances by whole stages / K steps
      const uint32_t hi_a = ptx::smem_desc_hi(A_MN, TC_BK * 4), hi_b = ptx::smem_desc_hi(B_MN, TC_BK * 4);
      const uint32_t lo_a0 = ptx::smem_desc_lo(ptx::smem_u32(smem), A_MN, TC_MN_CHUNK);
      const uint32_t lo_b0 = ptx::smem_desc_lo(ptx::smem_u32(smem) + 2 * TC_TILE_BYTES, B_MN, TC_MN_CHUNK);
      constexpr uint32_t step_a = (A_MN ? 1024u : 32u) >> 4, step_b = (B_MN ? 1024u : 32u) >> 4;
      bool ok = true;
      // running state: stage s with phase bit sp, accumulator buffer b with phase bit bp (of its *previous* use),
      // and whether the barriers of the coming K block were already seen complete by the probe below
      int s = 0, b = 0, ti = 0;
      uint32_t sp = 0, bp = 1;
      bool first_round = true, seen_conv = false, seen_acc = false;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++ti) {
        int m0, n0, k_begin, n_kb, z;
        tile_coords(tile, m0, n0, k_begin, n_kb, z);
        // the correction tile of the previous output tile must have been read before it is overwritten
        if (ti > 0 && n_kb > 0) ok = ptx::mbar_wait(corr_empty, (ti - 1) & 1, abort_flag);
        for (int kb = 0; kb < n_kb && ok; ++kb) {
          const bool first = kb % TC_FLUSH == 0, last = kb % TC_FLUSH == TC_FLUSH - 1 || kb == n_kb - 1;
          if (!seen_conv) ok = ptx::mbar_wait(&conv_bar[s], sp, abort_flag);
          if (ok && first && !first_round && !seen_acc) ok = ptx::mbar_wait(&acc_empty[b], bp, abort_flag);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t la = lo_a0 + (uint32_t)s * (TC_STAGE_BYTES >> 4), lb = lo_b0 + (uint32_t)s * (TC_STAGE_BYTES >> 4);
          const uint32_t d = tmem_base + (uint32_t)(b * TC_BN);
          // next K block's stage and, if it starts a new group, its accumulator buffer
          const int s_next = s + 1 == TC_STAGES ? 0 : s + 1;
          const uint32_t sp_next = s + 1 == TC_STAGES ? sp ^ 1u : sp;
          const int b_next = b + 1 == TC_ACC_BUFS ? 0 : b + 1;
          const uint32_t bp_next = b + 1 == TC_ACC_BUFS ? bp ^ 1u : bp;
          const bool round_next = first_round && b + 1 != TC_ACC_BUFS;
#pragma unroll
          for (int kk = 0; kk < TC_BK / 8; ++kk) {
            const uint64_t dah = ptx::smem_desc(hi_a, la + kk * step_a);
            const uint64_t dal = ptx::smem_desc(hi_a, la + (TC_TILE_BYTES >> 4) + kk * step_a);
            const uint64_t dbh = ptx::smem_desc(hi_b, lb + kk * step_b);
            const uint64_t dbl = ptx::smem_desc(hi_b, lb + (TC_TILE_BYTES >> 4) + kk * step_b);
            ptx::mma_tf32(d_corr, dal, dbh, idesc, kb > 0 || kk > 0);
            ptx::mma_tf32(d_corr, dah, dbl, idesc, true);
            ptx::mma_tf32(d, dah, dbh, idesc, !first || kk > 0);
            if (kk == TC_BK / 8 - 2) {
              // probe the coming block's barriers while the tensor pipe still has work queued
              seen_conv = ptx::mbar_test_wait(&conv_bar[s_next], sp_next);
              seen_acc = last ? (round_next ? true : ptx::mbar_test_wait(&acc_empty[b_next], bp_next)) : true;
            }
          }
          ptx::mma_commit(&empty_bar[s]);          // stage can be refilled once these MMAs have read it
          if (last) {
            ptx::mma_commit(&acc_full[b]);         // this group's partial product is complete
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
  } else if (warp < ACC0) {
    // ---------------------------------------------------------------- operand split (128 or 256 threads)
    const int t = threadIdx.x - 64;                       // 0 .. CONV_T-1
    bool ok = true;
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      int m0, n0, k_begin, n_kb, z;
      tile_coords(tile, m0, n0, k_begin, n_kb, z);
      for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
        const int s = it % TC_STAGES, use = it / TC_STAGES;
        ok = ptx::mbar_wait(&full_bar[s], use & 1, abort_flag);
        if (!ok) break;
        uint8_t *st = smem + s * TC_STAGE_BYTES;
        auto split = [&](uint8_t *hi_buf, uint8_t *lo_buf) {
          uint4 *hi = reinterpret_cast<uint4 *>(hi_buf), *lo = reinterpret_cast<uint4 *>(lo_buf);
#pragma unroll
          for (int i = 0; i < TC_TILE_BYTES / 16 / CONV_T; ++i) {
            const uint4 v = hi[t + CONV_T * i];
            uint4 h, l;
            h.x = tf32_hi(v.x); h.y = tf32_hi(v.y); h.z = tf32_hi(v.z); h.w = tf32_hi(v.w);
            l.x = __float_as_uint(__uint_as_float(v.x) - __uint_as_float(h.x));
            l.y = __float_as_uint(__uint_as_float(v.y) - __uint_as_float(h.y));
            l.z = __float_as_uint(__uint_as_float(v.z) - __uint_as_float(h.z));
            l.w = __float_as_uint(__uint_as_float(v.w) - __uint_as_float(h.w));
            hi[t + CONV_T * i] = h;
            lo[t + CONV_T * i] = l;
          }
        };
        split(st, st + TC_TILE_BYTES);
        if (B_SPLIT) split(st + 2 * TC_TILE_BYTES, st + 3 * TC_TILE_BYTES);
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(&conv_bar[s]);
      }
    }
  } else {
    // ---------------------------------------------------------------- accumulate, then epilogue (256 threads)
    // warp w owns tensor-memory lanes 32 (w mod 4) .. +31 = output rows m0 + that range, and the column half
    // (w - 6) / 4 of the tile (64 columns)
    const int lane_base = (warp & 3) * 32;
    const int chalf = (warp - ACC0) >> 2;
    float4 *tr = reinterpret_cast<float4 *>(tr_base) + (size_t)(warp - ACC0) * 32 * 8;    // 32 rows x 8 float4 per warp
    const int n_pad = (prm.N + 3) & ~3;
    bool ok = true;
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      int m0, n0, k_begin, n_kb, z;
      tile_coords(tile, m0, n0, k_begin, n_kb, z);
      if (m0 + lane_base + lane < prm.M) {          // this thread's row of the epilogue inputs, on its way to L2
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int col = n0 + chalf * 64 + h * 32;
          if (col < n_pad) epi.prefetch(m0 + lane_base + lane, col);
        }
      }
      float acc[64];
#pragma unroll
      for (int j = 0; j < 64; ++j) acc[j] = 0.f;
      auto add_tile = [&](uint32_t col_base) {
        const uint32_t src = tmem_base + ((uint32_t)lane_base << 16) + col_base + (uint32_t)(chalf * 64);
        if constexpr (B_SPLIT) {
          // 576 threads leave 96 registers per thread: 16 columns at a time
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            uint32_t v[16];
            ptx::tmem_ld16(src + 16u * h, v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) acc[16 * h + j] += __uint_as_float(v[j]);
          }
        } else {
          uint32_t v0[32], v1[32];
          ptx::tmem_ld32(src, v0);
          ptx::tmem_ld32(src + 32u, v1);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) { acc[j] += __uint_as_float(v0[j]); acc[32 + j] += __uint_as_float(v1[j]); }
        }
      };
      const int n_grp = (n_kb + TC_FLUSH - 1) / TC_FLUSH;
      for (int g = 0; g < n_grp && ok; ++g, ++it) {
        const int b = it % TC_ACC_BUFS, buse = it / TC_ACC_BUFS;
        ok = ptx::mbar_wait(&acc_full[b], buse & 1, abort_flag);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        add_tile((uint32_t)(b * TC_BN));
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(&acc_empty[b]);
      }
      if (!ok) break;
      if (n_kb > 0) {
        // correction terms: complete once the last block's commit has arrived (it covers every earlier MMA)
        add_tile((uint32_t)(TC_ACC_BUFS * TC_BN));
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(corr_empty);
      }
      int out_tile = tile;
      if (tile >= tail_begin) {
        // contraction slice of a tail tile: park the accumulators; the last warp to arrive sums the slices
        const int u = tile - tail_begin, t_idx = u / prm.tail_split;
        out_tile = tail_begin + t_idx;
        float *mine = prm.tail_ws + ((size_t)u * 8 + (warp - ACC0)) * 2048;
#pragma unroll
        for (int j = 0; j < 64; ++j) mine[j * 32 + lane] = acc[j];
        __threadfence();
        __syncwarp();
        int prev = 0;
        if (lane == 0) prev = atomicAdd(prm.tail_count + t_idx * 8 + (warp - ACC0), 1);
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev != prm.tail_split - 1) continue;
        __threadfence();
        if (lane == 0) prm.tail_count[t_idx * 8 + (warp - ACC0)] = 0;
#pragma unroll
        for (int j = 0; j < 64; ++j) acc[j] = 0.f;
        for (int sl = 0; sl < prm.tail_split; ++sl) {
          const float *part = prm.tail_ws + ((size_t)(t_idx * prm.tail_split + sl) * 8 + (warp - ACC0)) * 2048;
#pragma unroll
          for (int j = 0; j < 64; ++j) acc[j] += __ldcg(part + j * 32 + lane);
        }
      }
      // Epilogue.  Thread i of the warp holds row (lane_base + i), 64 columns.  The warp's piece goes through shared
      // memory 32 columns at a time: thread i writes its 8 float4 groups with the group index XOR-ed by (i mod 8)
      // (conflict-free 128-bit stores; this is also the 128-byte swizzle of the output tensor map).
      double ss = 0.0;
      if constexpr (Epi::kDirect) {
        // The output is the accumulator: sum of squares straight from the registers (four fp32 partial sums of 16
        // squares each, added in double), and the 32 x 32 pieces leave shared memory as TMA stores, which clip at the
        // matrix edges.  Rows and columns outside the matrix hold exact zeros (zero-filled operand tiles).
        if constexpr (Epi::kSumsq) {
          float s4[4] = {0.f, 0.f, 0.f, 0.f};
          const int n_valid = prm.N - (n0 + chalf * 64);      // columns of this thread inside the matrix
#pragma unroll
          for (int j = 0; j < 64; ++j)
            if (j < n_valid) s4[j & 3] = fmaf(acc[j], acc[j], s4[j & 3]);
          ss = ((double)s4[0] + (double)s4[1]) + ((double)s4[2] + (double)s4[3]);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (lane == 0) ptx::bulk_wait_read();       // the previous store has read the staging buffer
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int jj = h * 8 + j;
            tr[lane * 8 + (j ^ (lane & 7))] = make_float4(acc[4 * jj], acc[4 * jj + 1], acc[4 * jj + 2], acc[4 * jj + 3]);
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            const int x = n0 + chalf * 64 + h * 32, y = m0 + lane_base;
            if (x < epi.ldc && y < prm.M) ptx::tma_store_3d(&map_c, tr, x, y, z);
            ptx::bulk_commit();
          }
        }
      } else {
        // Inputs of the epilogue are read with the same coalesced pattern as the output is written: the warp walks
        // over its rows four at a time, lanes 8g..8g+7 take row 4 step + g, 4 consecutive columns per lane.  The
        // loads of four or eight steps are issued together (rows past the end are clamped, their results dropped).
        float *C = epi.C + (size_t)z * prm.c_split_stride;
        float ssf = 0.f;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int jj = h * 8 + j;
            tr[lane * 8 + (j ^ (lane & 7))] = make_float4(acc[4 * jj], acc[4 * jj + 1], acc[4 * jj + 2], acc[4 * jj + 3]);
          }
          __syncwarp();
          const int col = n0 + chalf * 64 + h * 32 + 4 * (lane & 7);
          if (col < n_pad) {
            constexpr int BATCH = Epi::kInputs <= 1 ? 8 : 4;       // row steps whose loads are in flight together
#pragma unroll
            for (int s0 = 0; s0 < 8; s0 += BATCH) {
              float4 in[BATCH][Epi::kInputs > 0 ? Epi::kInputs : 1];
#pragma unroll
              for (int i = 0; i < BATCH; ++i) {
                const int r = 4 * (s0 + i) + (lane >> 3);
                epi.load(min(m0 + lane_base + r, prm.M - 1), col, in[i]);
              }
#pragma unroll
              for (int i = 0; i < BATCH; ++i) {
                const int r = 4 * (s0 + i) + (lane >> 3);
                const int row = m0 + lane_base + r;
                const float4 o = epi.apply(col, tr[r * 8 + ((lane & 7) ^ (r & 7))], in[i]);
                if (row < prm.M) {
                  if (Epi::kSumsq) ssf = fmaf(o.x, o.x, fmaf(o.y, o.y, fmaf(o.z, o.z, fmaf(o.w, o.w, ssf))));
                  *reinterpret_cast<float4 *>(C + (size_t)row * epi.ldc + col) = o;
                }
              }
            }
          }
        }
        ss = (double)ssf;
      }
      if (partials != nullptr) {          // one slot per tile and warp; the host adds the slots in index order
        ss = warp_sum(ss);
        if (lane == 0) partials[(size_t)out_tile * 8 + (warp - ACC0)] = ss;
      }
    }
    if (Epi::kDirect && lane == 0) ptx::bulk_wait_all();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, TC_TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(prm.error, 1);
}

// x -> (x_hi, x_lo) planes of a small matrix (weights): x_hi = x rounded to tf32, x_lo = x - x_hi.
__global__ void __launch_bounds__(256)
split_planes_kernel(const float *__restrict__ x, float *__restrict__ hi, float *__restrict__ lo, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const float v = x[i];
    const float h = __uint_as_float(tf32_hi(__float_as_uint(v)));
    hi[i] = h;
    lo[i] = v - h;
  }
}

}  // namespace pd
