// Graph pre-processing: CSR structure of A + I (host), values of the renormalised adjacency
// A~ = (D+I)^{-1/2}(A+I)(D+I)^{-1/2} (device), and the sparse product Y = A~ X used to build the
// multi-hop input X = [H; H A~; H A~^2; ...] (A~ is symmetric, so in node-major storage the
// k-th block is A~ times the (k-1)-th block).
#pragma once

#include <algorithm>
#include <vector>

#include "common.cuh"

namespace pd {

// Host: undirected edge list -> CSR pattern of A + I with ascending columns; repeats and self-loops
// in the input are dropped.  Returns EINVAL on an out-of-range node id.
inline int build_csr_pattern(int64_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                             std::vector<int32_t> &row_ptr, std::vector<int32_t> &col_idx) {
  std::vector<uint64_t> keys;
  keys.reserve((size_t)(2 * n_edges + n));
  for (int64_t e = 0; e < n_edges; ++e) {
    const int64_t a = src[e], b = dst[e];
    if (a < 0 || a >= n || b < 0 || b >= n)
      return fail(PDADMM_EINVAL, "edge %lld = (%lld, %lld) is outside [0, %lld)", (long long)e, (long long)a,
                  (long long)b, (long long)n);
    if (a == b) continue;
    keys.push_back((uint64_t)a * (uint64_t)n + (uint64_t)b);
    keys.push_back((uint64_t)b * (uint64_t)n + (uint64_t)a);
  }
  for (int64_t i = 0; i < n; ++i) keys.push_back((uint64_t)i * (uint64_t)n + (uint64_t)i);
  std::sort(keys.begin(), keys.end());
  keys.erase(std::unique(keys.begin(), keys.end()), keys.end());
  if (keys.size() > (size_t)INT32_MAX) return fail(PDADMM_EINVAL, "more than 2^31-1 non-zeros");
  row_ptr.assign((size_t)n + 1, 0);
  col_idx.resize(keys.size());
  for (size_t i = 0; i < keys.size(); ++i) {
    const uint64_t r = keys[i] / (uint64_t)n;
    col_idx[i] = (int32_t)(keys[i] % (uint64_t)n);
    row_ptr[r + 1]++;
  }
  for (int64_t i = 0; i < n; ++i) row_ptr[i + 1] += row_ptr[i];
  return PDADMM_OK;
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
template <int VEC>
__global__ void __launch_bounds__(256)
spmm_kernel(const int *__restrict__ row_ptr, const int *__restrict__ col_idx, const float *__restrict__ val,
            int n_rows, const float *__restrict__ X, float *__restrict__ Y, int width, int ld) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  const int b = row_ptr[row], e = row_ptr[row + 1];
  for (int c0 = lane * VEC; c0 < width; c0 += 32 * VEC) {
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    for (int k = b; k < e; ++k) {
      const float a = __ldg(val + k);
      const float *xr = X + (size_t)__ldg(col_idx + k) * ld + c0;
      if (VEC == 4) {
        const float4 x = *reinterpret_cast<const float4 *>(xr);
        acc[0] = fmaf(a, x.x, acc[0]); acc[1] = fmaf(a, x.y, acc[1]);
        acc[2 % VEC] = fmaf(a, x.z, acc[2 % VEC]); acc[3 % VEC] = fmaf(a, x.w, acc[3 % VEC]);
      } else if (VEC == 2) {
        const float2 x = *reinterpret_cast<const float2 *>(xr);
        acc[0] = fmaf(a, x.x, acc[0]); acc[1 % VEC] = fmaf(a, x.y, acc[1 % VEC]);
      } else {
        acc[0] = fmaf(a, *xr, acc[0]);
      }
    }
    float *yr = Y + (size_t)row * ld + c0;
    if (VEC == 4) *reinterpret_cast<float4 *>(yr) = make_float4(acc[0], acc[1 % VEC], acc[2 % VEC], acc[3 % VEC]);
    else if (VEC == 2) *reinterpret_cast<float2 *>(yr) = make_float2(acc[0], acc[1 % VEC]);
    else *yr = acc[0];
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
