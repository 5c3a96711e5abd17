// Graph pre-processing: CSR structure of A + I, values of the renormalised adjacency
// A~ = (D+I)^{-1/2}(A+I)(D+I)^{-1/2} (device), and the sparse product Y = A~ X used to build the
// multi-hop input X = [H; H A~; H A~^2; ...] (A~ is symmetric, so in node-major storage the
// k-th block is A~ times the (k-1)-th block).
#pragma once

#include <cstdint>

#include "common.cuh"

namespace pd {

// ---- CSR pattern of A + I on the device ---------------------------------------------------------------
// Undirected edge list -> rows with ascending, unique columns; self-loops and repeats in the input are
// dropped and every row gets its diagonal entry.  Steps: count the raw entries of each row, prefix-sum them,
// scatter the edges (any order within a row), sort each row and drop its repeats, prefix-sum the final row
// lengths and compact.  The result does not depend on the order in which the scatter's atomics land.
// meta[0] = error word (1 bad node id, 2 more than 2^31-1 entries, 3 a row above CSR_MAX_ROW),
// meta[1] = number of long rows; bad_edge = smallest index of an edge with a node id outside [0, n).

constexpr int CSR_WARP_ROW = 512;        // longer rows are sorted by a whole block
constexpr int CSR_MAX_ROW = 1 << 16;     // the row sort is quadratic in the row length

__global__ void edge_count_kernel(const int *__restrict__ src, const int *__restrict__ dst, long long n_edges, int n,
                                  int *__restrict__ deg, int *__restrict__ meta, unsigned long long *bad_edge) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_edges) return;
  const int a = src[e], b = dst[e];
  if ((unsigned)a >= (unsigned)n || (unsigned)b >= (unsigned)n) {
    meta[0] = 1;
    atomicMin(bad_edge, (unsigned long long)e);
    return;
  }
  if (a == b) return;
  atomicAdd(deg + a, 1);
  atomicAdd(deg + b, 1);
}

// out[i] = sum_{j<i} (in[j] + add) for i = 0..n (out[n] is the total); one block, chunks of blockDim.x.
__global__ void __launch_bounds__(1024)
exclusive_scan_kernel(const int *__restrict__ in, int n, int add, int *__restrict__ out, int *__restrict__ meta) {
  __shared__ int warp_sum[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long carry = 0;
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < n ? in[i] + add : 0;
    int x = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, d);
      if (lane >= d) x += y;
    }
    if (lane == 31) warp_sum[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int t = warp_sum[lane];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, t, d);
        if (lane >= d) t += y;
      }
      warp_sum[lane] = t;
    }
    __syncthreads();
    if (i < n) out[i] = (int)(carry + (warp ? warp_sum[warp - 1] : 0) + x - v);
    carry += warp_sum[31];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    out[n] = (int)carry;
    if (carry > (long long)INT32_MAX) meta[0] = 2;
  }
}

__global__ void edge_scatter_kernel(const int *__restrict__ src, const int *__restrict__ dst, long long n_edges, int n,
                                    const int *__restrict__ raw_ptr, int *__restrict__ cursor, int *__restrict__ raw) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_edges) return;
  const int a = src[e], b = dst[e];
  if ((unsigned)a >= (unsigned)n || (unsigned)b >= (unsigned)n || a == b) return;
  raw[raw_ptr[a] + atomicAdd(cursor + a, 1)] = b;
  raw[raw_ptr[b] + atomicAdd(cursor + b, 1)] = a;
}

// One row: raw[b .. b+d) holds the neighbours in any order, its last slot is free for the diagonal.
// Writes the distinct columns in ascending order to sorted[b ..] and their number to len[row].
// Each of the `nt` threads of the group (a warp or a block) takes the entries k = t, t+nt, ...
template <bool BLOCK>
__device__ __forceinline__ void sort_unique_row(int row, int b, int d, int *raw, int *sorted, int *len, int t, int nt) {
  auto group_sync = [] { if constexpr (BLOCK) __syncthreads(); else __syncwarp(); };
  if (t == 0) raw[b + d - 1] = row;
  group_sync();
  // an entry is a repeat when an equal column stands before it
  for (int k = t; k < d; k += nt) {
    const int ck = raw[b + k];
    int rep = 0;
    for (int j = 0; j < k; ++j) rep |= (raw[b + j] == ck);
    sorted[b + k] = rep;
  }
  group_sync();
  int kept = 0;
  for (int k = t; k < d; k += nt) {
    if (sorted[b + k]) raw[b + k] = INT32_MAX; else ++kept;
  }
  group_sync();
  // rank = number of distinct smaller columns (repeats now compare as +infinity)
  for (int k = t; k < d; k += nt) {
    const int ck = raw[b + k];
    if (ck == INT32_MAX) continue;
    int rank = 0;
    for (int j = 0; j < d; ++j) rank += (raw[b + j] < ck);
    sorted[b + rank] = ck;
  }
  if (kept) atomicAdd(len + row, kept);
}

// Rows up to CSR_WARP_ROW entries: one warp each.  Longer rows are appended to `long_rows`.
__global__ void __launch_bounds__(256)
row_sort_warp_kernel(const int *__restrict__ raw_ptr, int n, int *raw, int *sorted, int *__restrict__ len,
                     int *__restrict__ long_rows, int *__restrict__ meta) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (row >= n) return;
  const int b = raw_ptr[row], d = raw_ptr[row + 1] - b;
  if (d > CSR_MAX_ROW) { if (lane == 0) meta[0] = 3; return; }
  if (d > CSR_WARP_ROW) { if (lane == 0) long_rows[atomicAdd(meta + 1, 1)] = row; return; }
  sort_unique_row<false>(row, b, d, raw, sorted, len, lane, 32);
}

__global__ void __launch_bounds__(1024)
row_sort_block_kernel(const int *__restrict__ raw_ptr, int *raw, int *sorted, int *__restrict__ len,
                      const int *__restrict__ long_rows, const int *__restrict__ meta) {
  const int n_long = meta[1];
  for (int i = blockIdx.x; i < n_long; i += gridDim.x) {
    const int row = long_rows[i], b = raw_ptr[row], d = raw_ptr[row + 1] - b;
    sort_unique_row<true>(row, b, d, raw, sorted, len, threadIdx.x, blockDim.x);
    __syncthreads();
  }
}

__global__ void __launch_bounds__(256)
row_compact_kernel(const int *__restrict__ raw_ptr, const int *__restrict__ row_ptr, int n,
                   const int *__restrict__ sorted, int *__restrict__ col_idx) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (row >= n) return;
  const int src = raw_ptr[row], dst = row_ptr[row], d = row_ptr[row + 1] - dst;
  for (int k = lane; k < d; k += 32) col_idx[dst + k] = sorted[src + k];
}

// val[e] = 1 / sqrt((d_i + 1)(d_j + 1)) for the entry e = (i, j); d_i = row length - 1 (the self-loop).
__global__ void adjacency_values_kernel(const int *__restrict__ row_ptr, const int *__restrict__ col_idx, int n,
                                        float *__restrict__ val) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= n) return;
  const int b = row_ptr[warp], e = row_ptr[warp + 1];
  const float di = (float)(e - b);                       // d_i + 1
  for (int k = b + lane; k < e; k += 32) {
    const int j = col_idx[k];
    const float dj = (float)(row_ptr[j + 1] - row_ptr[j]);
    val[k] = 1.0f / sqrtf(di * dj);
  }
}

// Y[i][0:width] = sum_e val[e] * X[col[e]][0:width], one warp per row, entries in CSR order.
// X and Y are addressed with the same row stride ld (they are column blocks of one matrix).
// VEC = 4, 2 or 1 floats per lane and access, chosen by the alignment of the blocks.
// The gathered rows are what costs: the lanes first fetch up to 32 (column, value) pairs of the row together and hand
// them round by shuffle, and every lane keeps SPMM_CH column groups in flight per neighbour (independent loads), so a
// warp has 4 x 32 x VEC floats of a neighbour's row on their way at a time instead of 32 x VEC.
constexpr int SPMM_CH = 4;
template <int VEC>
__global__ void __launch_bounds__(256)
spmm_kernel(const int *__restrict__ row_ptr, const int *__restrict__ col_idx, const float *__restrict__ val,
            int n_rows, const float *__restrict__ X, float *__restrict__ Y, int width, int ld) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  const int b = row_ptr[row], e = row_ptr[row + 1];
  for (int base = 0; base < width; base += 32 * VEC * SPMM_CH) {
    float acc[SPMM_CH][VEC];
#pragma unroll
    for (int ch = 0; ch < SPMM_CH; ++ch)
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc[ch][v] = 0.f;
    for (int k0 = b; k0 < e; k0 += 32) {
      const int n = min(32, e - k0);
      // lanes past the end of the row repeat the chunk's first entry with the value 0: nothing is read that the row
      // does not read anyway
      const int my_col = __ldg(col_idx + k0 + (lane < n ? lane : 0));
      const float my_val = lane < n ? __ldg(val + k0 + lane) : 0.f;
      // four neighbours at a time: their loads are independent
      for (int j = 0; j < n; j += 4) {
        float a[4];
        const float *xr[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          a[t] = __shfl_sync(0xffffffffu, my_val, (j + t) & 31);
          xr[t] = X + (size_t)__shfl_sync(0xffffffffu, my_col, (j + t) & 31) * ld;
        }
#pragma unroll
        for (int ch = 0; ch < SPMM_CH; ++ch) {
          const int c0 = base + (ch * 32 + lane) * VEC;
          if (c0 >= width) continue;
          float x[4][VEC];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            if (VEC == 4) {
              const float4 q = *reinterpret_cast<const float4 *>(xr[t] + c0);
              x[t][0] = q.x; x[t][1 % VEC] = q.y; x[t][2 % VEC] = q.z; x[t][3 % VEC] = q.w;
            } else if (VEC == 2) {
              const float2 q = *reinterpret_cast<const float2 *>(xr[t] + c0);
              x[t][0] = q.x; x[t][1 % VEC] = q.y;
            } else {
              x[t][0] = xr[t][c0];
            }
          }
          // added in entry order, like a loop over single entries
#pragma unroll
          for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[ch][v] = fmaf(a[t], x[t][v], acc[ch][v]);
        }
      }
    }
#pragma unroll
    for (int ch = 0; ch < SPMM_CH; ++ch) {
      const int c0 = base + (ch * 32 + lane) * VEC;
      if (c0 >= width) continue;
      float *yr = Y + (size_t)row * ld + c0;
      if (VEC == 4) *reinterpret_cast<float4 *>(yr) = make_float4(acc[ch][0], acc[ch][1 % VEC], acc[ch][2 % VEC], acc[ch][3 % VEC]);
      else if (VEC == 2) *reinterpret_cast<float2 *>(yr) = make_float2(acc[ch][0], acc[ch][1 % VEC]);
      else *yr = acc[ch][0];
    }
  }
}

// Launch with the widest access the alignment of both blocks allows (width % VEC == 0 is required so
// that a lane never straddles the end of the block).
inline void launch_spmm(cudaStream_t st, const int *row_ptr, const int *col_idx, const float *val, int n_rows,
                        const float *X, float *Y, int width, int ld) {
  const int threads = 256, rows_per_block = threads / 32;
  const int grid = (int)ceil_div(n_rows, rows_per_block);
  const uintptr_t mis = (uintptr_t)X | (uintptr_t)Y | ((uintptr_t)ld * 4) | ((uintptr_t)width * 4);
  if (mis % 16 == 0) spmm_kernel<4><<<grid, threads, 0, st>>>(row_ptr, col_idx, val, n_rows, X, Y, width, ld);
  else if (mis % 8 == 0) spmm_kernel<2><<<grid, threads, 0, st>>>(row_ptr, col_idx, val, n_rows, X, Y, width, ld);
  else spmm_kernel<1><<<grid, threads, 0, st>>>(row_ptr, col_idx, val, n_rows, X, Y, width, ld);
}

}  // namespace pd
