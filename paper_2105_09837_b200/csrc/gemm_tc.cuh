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
// warp 0: TMA, warp 1: MMA, warps 2..5: operand split, warps 6..9: accumulate + epilogue
constexpr int TC_THREADS = 320;
constexpr int TC_ACC_BUFS = 2;                                 // main-term accumulator tiles in tensor memory
constexpr int TC_TMEM_COLS = 512;                              // 2 main tiles + 1 correction tile, power of two
constexpr int TC_SMEM_BYTES = TC_STAGES * TC_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

// x_hi: x rounded to the nearest tf32 number (11 significant bits).  x_lo = x - x_hi is then exact in fp32,
// at most 2^-12 |x| and of either sign, so what the MMA drops of it (its last bit) has no preferred direction.
__host__ __device__ __forceinline__ uint32_t tf32_hi(uint32_t bits) { return (bits + 0x1000u) & 0xFFFFE000u; }

struct TcParams {
  int M, N, K;            // output rows, output columns, contraction length
  int k_chunk;            // contraction slice per blockIdx.z (multiple of TC_BK); K if not split
  size_t c_split_stride;  // elements between the partial outputs of consecutive slices
  int *error;             // set to 1 if a bounded wait expired
};

// A_MN / B_MN: operand is stored contiguous along its output index (rows of the tile are K slices);
//              otherwise contiguous along K.
// B_SPLIT: B is one fp32 tensor split in shared memory like A; otherwise it arrives as two planes (map_b, map_blo).
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
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + TC_STAGES * TC_STAGE_BYTES);
  uint64_t *full_bar = bars, *conv_bar = bars + TC_STAGES, *empty_bar = bars + 2 * TC_STAGES;
  uint64_t *acc_full = bars + 3 * TC_STAGES, *acc_empty = acc_full + TC_ACC_BUFS, *drain_bar = acc_empty + TC_ACC_BUFS;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(drain_bar + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  double *red = reinterpret_cast<double *>(drain_bar + 2);                    // 4 doubles

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * TC_BM, n0 = blockIdx.x * TC_BN;
  const int k_begin = blockIdx.z * prm.k_chunk;
  const int k_end = min(prm.K, k_begin + prm.k_chunk);
  const int n_kb = (max(k_end - k_begin, 0) + TC_BK - 1) / TC_BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&conv_bar[s], 128);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < TC_ACC_BUFS; ++b) {
      ptx::mbar_init(&acc_full[b], 1);
      ptx::mbar_init(&acc_empty[b], 128);
    }
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

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (one lane)
    if (lane == 0) {
      int issued = 0;
      for (int kb = 0; kb < n_kb; ++kb) {
        const int s = kb % TC_STAGES, use = kb / TC_STAGES;
        if (use > 0 && !ptx::mbar_wait(&empty_bar[s], (use - 1) & 1, abort_flag)) break;
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
        issued = kb + 1;
      }
      if (*abort_flag) {
        // copies in flight must land before the block's shared memory is released
        for (int kb = max(issued - TC_STAGES, 0); kb < issued; ++kb)
          ptx::mbar_wait(&full_bar[kb % TC_STAGES], (kb / TC_STAGES) & 1, abort_flag, 200000000ll, false);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_tf32(TC_BM, TC_BN, A_MN, B_MN);
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % TC_STAGES, use = kb / TC_STAGES;
        const int b = kb % TC_ACC_BUFS, buse = kb / TC_ACC_BUFS;
        ok = ptx::mbar_wait(&conv_bar[s], use & 1, abort_flag);
        if (ok && buse > 0) ok = ptx::mbar_wait(&acc_empty[b], (buse - 1) & 1, abort_flag);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t st = ptx::smem_u32(smem + s * TC_STAGE_BYTES);
        const uint32_t a_hi = st, a_lo = st + TC_TILE_BYTES, b_hi = st + 2 * TC_TILE_BYTES, b_lo = st + 3 * TC_TILE_BYTES;
        const uint32_t d = tmem_base + (uint32_t)(b * TC_BN), d_corr = tmem_base + (uint32_t)(TC_ACC_BUFS * TC_BN);
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
    for (int kb = 0; kb < n_kb && ok; ++kb) {
      const int s = kb % TC_STAGES, use = kb / TC_STAGES;
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
  } else {
    // ---------------------------------------------------------------- accumulate, then epilogue (128 threads)
    // warp w owns tensor-memory lanes 32 (w mod 4) .. +31 = output rows m0 + that range
    const int lane_base = (warp & 3) * 32;
    float acc[TC_BN];
#pragma unroll
    for (int j = 0; j < TC_BN; ++j) acc[j] = 0.f;
    bool ok = true;
    for (int kb = 0; kb < n_kb && ok; ++kb) {
      const int b = kb % TC_ACC_BUFS, buse = kb / TC_ACC_BUFS;
      ok = ptx::mbar_wait(&acc_full[b], buse & 1, abort_flag);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const uint32_t src = tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(b * TC_BN);
#pragma unroll
      for (int c0 = 0; c0 < TC_BN; c0 += 32) {
        uint32_t v[32];
        ptx::tmem_ld32(src + (uint32_t)c0, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[c0 + j] += __uint_as_float(v[j]);
      }
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(&acc_empty[b]);
    }
    if (ok && n_kb > 0) {
      // correction terms: complete once the last block's commit has arrived (it covers every earlier MMA)
      const uint32_t src = tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(TC_ACC_BUFS * TC_BN);
#pragma unroll
      for (int c0 = 0; c0 < TC_BN; c0 += 32) {
        uint32_t v[32];
        ptx::tmem_ld32(src + (uint32_t)c0, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[c0 + j] += __uint_as_float(v[j]);
      }
    }
    double ss = 0.0;
    if (ok) {
      const int row = m0 + lane_base + lane;
      const int n_pad = (prm.N + 3) & ~3;
      float *C = epi.C + (size_t)blockIdx.z * prm.c_split_stride;
      if (row < prm.M) {
#pragma unroll
        for (int j = 0; j < TC_BN / 4; ++j) {
          const int col = n0 + 4 * j;
          if (col < n_pad) {
            const float4 a = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
            const float4 o = epi(row, col, a, ss);
            *reinterpret_cast<float4 *>(C + (size_t)row * epi.ldc + col) = o;
          }
        }
      }
    }
    if (partials != nullptr) {
      ss = warp_sum(ss);
      if (lane == 0) red[warp - 6] = ss;
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, TC_TMEM_COLS);
  }
  if (threadIdx.x == 0) {
    if (partials != nullptr)
      partials[(size_t)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = red[0] + red[1] + red[2] + red[3];
    if (*abort_flag) atomicExch(prm.error, 1);
  }
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
