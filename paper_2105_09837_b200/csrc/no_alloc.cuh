// An entry point that allocates nothing: the node-contracting product C = A^T B (the form of the W-gradient,
// r^T p) on caller-owned device buffers, with the partial tiles of its node slices kept in a fixed array that
// is part of the library image instead of in memory obtained from cudaMalloc.
//
// Who needs it: code that runs where device allocation is not allowed or not wanted -- between
// cudaStreamBeginCapture and cudaStreamEndCapture, inside a latency-critical loop that must not take the
// allocator's lock or trigger an implicit device synchronisation, or in a process whose memory budget was
// handed out up front and whose allocator is simply not reachable from the calling layer.
#pragma once

#include "common.cuh"
#include "elementwise.cuh"
#include "gemm_simt.cuh"

namespace pd {

// Partial tiles of the node slices: at most this many floats (4 MiB).  Every GPU that loads the library keeps
// the array for the life of the process.
constexpr size_t STATIC_SCRATCH_FLOATS = size_t(1) << 20;
static __device__ __align__(256) float g_static_scratch[STATIC_SCRATCH_FLOATS];

constexpr int STATIC_MAX_DEVICES = 64;
static float *g_static_scratch_ptr[STATIC_MAX_DEVICES];   // device address of the array, per device; null = not set up

// sum of the partial tiles in slice order (no scaling, no norm).  Rows of C are ldc = 4 * ldc4 floats wide with N
// valid columns: the padding columns are written as zero whatever the partial tiles hold there (the product reads
// the operand in groups of four columns, so those entries are products with the caller's padding of B).
__global__ void __launch_bounds__(EW_THREADS)
sum_partial_tiles_kernel(const float *__restrict__ part, int n_split, size_t n4, int ldc4, int N, float *__restrict__ C) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < n_split; ++s) {
      const float4 v = ld4(part + (size_t)s * n4 * 4, i);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    const int col = (int)(i % (size_t)ldc4) * 4;
    if (col + 1 >= N) a.y = 0.f;
    if (col + 2 >= N) a.z = 0.f;
    if (col + 3 >= N) a.w = 0.f;
    st4(C, i, a);
  }
}

}  // namespace pd

extern "C" int pdadmm_matmul_tn_static(int device, int M, int N, int K, const float *dA, int lda, const float *dB,
                                       int ldb, float *dC, void *stream) {
  using namespace pd;
  if (M < 1 || N < 1 || K < 1 || !dA || !dB || !dC) return fail(PDADMM_EINVAL, "bad argument");
  if (device < 0 || device >= STATIC_MAX_DEVICES) return fail(PDADMM_EINVAL, "device ordinal out of range");
  const int ldc = round_up(N, 4);
  if (lda < M || ldb < N || lda % 4 || ldb % 4) return fail(PDADMM_EINVAL, "lda >= M, ldb >= N, both multiples of 4");
  if (((uintptr_t)dA | (uintptr_t)dB | (uintptr_t)dC) & 15) return fail(PDADMM_EINVAL, "buffers must be 16-byte aligned");
  const size_t tile_floats = (size_t)M * ldc;
  if (tile_floats > STATIC_SCRATCH_FLOATS)
    return fail(PDADMM_EINVAL,
                "output of %d x %d needs %zu scratch floats per node slice; the built-in scratch holds %zu "
                "(use pdadmm_matmul, which allocates, for larger outputs)",
                M, N, tile_floats, STATIC_SCRATCH_FLOATS);
  int prev = 0;
  PD_CUDA(cudaGetDevice(&prev));
  PD_CUDA(cudaSetDevice(device));
  auto body = [&]() -> int {
    if (g_static_scratch_ptr[device] == nullptr) {
      // once per device, with that device current: the array's name is only a host-side handle, the kernel
      // needs the address the symbol has on THIS device
      float *p = nullptr;
      PD_CUDA(cudaGetSymbolAddress((void **)&p, g_static_scratch));
      g_static_scratch_ptr[device] = p;
    }
    float *part = g_static_scratch_ptr[device];
    // as many node slices as fit (at most 8, at least 256 nodes each)
    int split = (int)std::min<size_t>(8, STATIC_SCRATCH_FLOATS / tile_floats);
    split = std::max(1, std::min(split, (int)ceil_div(K, 256)));
    const int k_chunk = round_up((int)ceil_div(K, split), SG_BK);
    const int n_split = (int)ceil_div(K, k_chunk);
    cudaStream_t st = (cudaStream_t)stream;
    dim3 grid((unsigned)ceil_div(N, SG_BN), (unsigned)ceil_div(M, SG_BM), (unsigned)n_split);
    gemm_tn_kernel<<<grid, SG_THREADS, 0, st>>>(M, N, K, k_chunk, dA, lda, dB, ldb, part, ldc);
    const size_t n4 = tile_floats / 4;
    const int g = (int)std::max<size_t>(1, std::min<size_t>(ceil_div((int64_t)n4, EW_THREADS), 148 * 8));
    sum_partial_tiles_kernel<<<g, EW_THREADS, 0, st>>>(part, n_split, n4, ldc / 4, N, dC);
    PD_CUDA(cudaPeekAtLastError());
    return PDADMM_OK;
  };
  const int rc = body();
  cudaSetDevice(prev);
  return rc;
}
