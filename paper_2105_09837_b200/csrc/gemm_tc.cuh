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
constexpr int TC_TILE_BYTES = 128 * TC_BK * 4;                 // 16 KB: one 128 x 32 fp32 operand tile
constexpr int TC_STAGE_BYTES = 4 * TC_TILE_BYTES;              // A_hi, A_lo, B_hi, B_lo
// warp 0: TMA, warp 1: MMA, warps 2..5: operand split, warps 6..13: accumulate + epilogue
// (two warps per 32-lane quarter of tensor memory, 64 columns each)
constexpr int TC_THREADS = 448;
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
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_blo, const TcParams prm, Epi epi, double *__restrict__ partials) {
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
  const int tiles_n = (prm.N + TC_BN - 1) / TC_BN, tiles_m = (prm.M + TC_BM - 1) / TC_BM;
  const int n_tiles = tiles_n * tiles_m * prm.n_split;

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&conv_bar[s], 128);
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
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TC_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile -> (row tile origin, column tile origin, first and number of K blocks)
  auto tile_coords = [&](int tile, int &m0, int &n0, int &k_begin, int &n_kb, int &z) {
    z = tile / (tiles_m * tiles_n);
    const int rem = tile - z * tiles_m * tiles_n;
    m0 = (rem / tiles_n) * TC_BM;
    n0 = (rem % tiles_n) * TC_BN;
    k_begin = z * prm.k_chunk;
    const int k_end = min(prm.K, k_begin + prm.k_chunk);
    n_kb = (max(k_end - k_begin, 0) + TC_BK - 1) / TC_BK;
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
            for (int j = 0; j < 4; ++j) ptx::tma_load_2d(st + j * 4096, &map_a, m0 + 32 * j, k0, &full_bar[s]);
          } else {
            ptx::tma_load_2d(st, &map_a, k0, m0, &full_bar[s]);
          }
          uint8_t *bh = st + 2 * TC_TILE_BYTES, *bl = st + 3 * TC_TILE_BYTES;
          if (B_MN) {
            for (int j = 0; j < 4; ++j) ptx::tma_load_2d(bh + j * 4096, &map_b, n0 + 32 * j, k0, &full_bar[s]);
            if (!B_SPLIT)
              for (int j = 0; j < 4; ++j) ptx::tma_load_2d(bl + j * 4096, &map_blo, n0 + 32 * j, k0, &full_bar[s]);
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
      bool ok = true;
      int it = 0, ti = 0;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++ti) {
        int m0, n0, k_begin, n_kb, z;
        tile_coords(tile, m0, n0, k_begin, n_kb, z);
        // the correction tile of the previous output tile must have been read before it is overwritten
        if (ti > 0 && n_kb > 0) ok = ptx::mbar_wait(corr_empty, (ti - 1) & 1, abort_flag);
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = it % TC_STAGES, use = it / TC_STAGES;
          const int b = it % TC_ACC_BUFS, buse = it / TC_ACC_BUFS;
          ok = ptx::mbar_wait(&conv_bar[s], use & 1, abort_flag);
          if (ok && buse > 0) ok = ptx::mbar_wait(&acc_empty[b], (buse - 1) & 1, abort_flag);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t st = ptx::smem_u32(smem + s * TC_STAGE_BYTES);
          const uint32_t a_hi = st, a_lo = st + TC_TILE_BYTES, b_hi = st + 2 * TC_TILE_BYTES, b_lo = st + 3 * TC_TILE_BYTES;
          const uint32_t d = tmem_base + (uint32_t)(b * TC_BN);
#pragma unroll
          for (int kk = 0; kk < TC_BK / 8; ++kk) {
            const uint32_t ao = A_MN ? kk * 1024 : kk * 32, bo = B_MN ? kk * 1024 : kk * 32;
            const uint64_t dah = ptx::smem_desc(a_hi + ao, A_MN, 4096);
            const uint64_t dal = ptx::smem_desc(a_lo + ao, A_MN, 4096);
            const uint64_t dbh = ptx::smem_desc(b_hi + bo, B_MN, 4096);
            const uint64_t dbl = ptx::smem_desc(b_lo + bo, B_MN, 4096);
            ptx::mma_tf32(d_corr, dal, dbh, idesc, kb > 0 || kk > 0);
            ptx::mma_tf32(d_corr, dah, dbl, idesc, true);
            ptx::mma_tf32(d, dah, dbh, idesc, kk > 0);
          }
          ptx::mma_commit(&empty_bar[s]);          // stage can be refilled once these MMAs have read it
          ptx::mma_commit(&acc_full[b]);           // this block's partial product is complete
        }
      }
      if (!ok) {
        // after an abandoned wait: let the MMAs already issued finish before tensor memory is released
        ptx::mma_commit(drain_bar);
        ptx::mbar_wait(drain_bar, 0, abort_flag, 200000000ll, false);
      }
    }
  } else if (warp < 6) {
    // ---------------------------------------------------------------- operand split (128 threads)
    const int t = threadIdx.x - 64;
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
          for (int i = 0; i < TC_TILE_BYTES / 16 / 128; ++i) {
            const uint4 v = hi[t + 128 * i];
            uint4 h, l;
            h.x = tf32_hi(v.x); h.y = tf32_hi(v.y); h.z = tf32_hi(v.z); h.w = tf32_hi(v.w);
            l.x = __float_as_uint(__uint_as_float(v.x) - __uint_as_float(h.x));
            l.y = __float_as_uint(__uint_as_float(v.y) - __uint_as_float(h.y));
            l.z = __float_as_uint(__uint_as_float(v.z) - __uint_as_float(h.z));
            l.w = __float_as_uint(__uint_as_float(v.w) - __uint_as_float(h.w));
            hi[t + 128 * i] = h;
            lo[t + 128 * i] = l;
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
    const int chalf = (warp - 6) >> 2;
    float4 *tr = reinterpret_cast<float4 *>(tr_base) + (size_t)(warp - 6) * 32 * 8;    // 32 rows x 8 float4 per warp
    const int n_pad = (prm.N + 3) & ~3;
    bool ok = true;
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      int m0, n0, k_begin, n_kb, z;
      tile_coords(tile, m0, n0, k_begin, n_kb, z);
      float acc[64];
#pragma unroll
      for (int j = 0; j < 64; ++j) acc[j] = 0.f;
      auto add_tile = [&](uint32_t col_base) {
        const uint32_t src = tmem_base + ((uint32_t)lane_base << 16) + col_base + (uint32_t)(chalf * 64);
        uint32_t v0[32], v1[32];
        ptx::tmem_ld32(src, v0);
        ptx::tmem_ld32(src + 32u, v1);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) { acc[j] += __uint_as_float(v0[j]); acc[32 + j] += __uint_as_float(v1[j]); }
      };
      for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
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
      // Epilogue.  Thread i of the warp holds row (lane_base + i), 64 columns.  For coalesced global accesses the
      // warp's piece goes through shared memory 32 columns at a time: thread i writes its 8 float4 groups with the
      // group index XOR-ed by (i mod 8) (conflict-free 128-bit stores), then the warp walks over its rows four at a
      // time: lanes 8g..8g+7 take row 4 step + g, 4 consecutive columns per lane (one 128-byte line per row).
      double ss = 0.0;
      float *C = epi.C + (size_t)z * prm.c_split_stride;
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
#pragma unroll 4
          for (int step = 0; step < 8; ++step) {
            const int r = 4 * step + (lane >> 3);
            const int row = m0 + lane_base + r;
            if (row < prm.M) {
              const float4 a = tr[r * 8 + ((lane & 7) ^ (r & 7))];
              const float4 o = epi(row, col, a, ss);
              *reinterpret_cast<float4 *>(C + (size_t)row * epi.ldc + col) = o;
            }
          }
        }
      }
      if (partials != nullptr) {          // one slot per tile and warp; the host adds the slots in index order
        ss = warp_sum(ss);
        if (lane == 0) partials[(size_t)tile * 8 + (warp - 6)] = ss;
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
