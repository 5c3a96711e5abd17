// fp32 CUDA-core matrix products with fused epilogues.
//
// These kernels are the reference-precision GEMM path (selected with PDADMM_FLAG_SIMT_GEMM) and
// the cross-check of the tensor-core path.  Operands are row-major with padded leading dimensions
// (multiples of 4 floats, 16-byte aligned rows).
//
//   gemm_nt :  C[M][N] = A[M][K] * B[N][K]^T        (both operands contiguous along K)
//   gemm_tn :  C[M][N] = sum_k A[k][M]^T B[k][N]    (both contiguous along the output index;
//                                                     K = nodes, split over grid.z into partial tiles)
#pragma once

#include "common.cuh"

namespace pd {

constexpr int SG_BM = 128, SG_BN = 128, SG_BK = 8, SG_THREADS = 256;

// ---- epilogues: called with 4 consecutive columns of one row ------------------------------------
// prefetch(row, col): optional hint that the 128 bytes of every epilogue input at (row, col .. col+31) will be
// read soon (the tensor-core kernel issues it when it starts a tile).
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// kDirect: the output is the accumulator itself (the tensor-core kernel then stores the tile by TMA);
// kSumsq: the epilogue accumulates the sum of squares of the output.
// `amax` (epilogues that feed a later tensor-core product): word that receives max|C| as a bit pattern; may be null.
struct EpiStore {             // C = acc
  static constexpr bool kDirect = true, kSumsq = false;
  static constexpr int kInputs = 0;
  float *C; int ldc;
  __device__ __forceinline__ void prefetch(int, int) const {}
  __device__ __forceinline__ float4 operator()(int, int, float4 a, double &) const { return a; }
};
struct EpiStoreSumsq {        // C = acc, accumulates sum(acc^2)
  static constexpr bool kDirect = true, kSumsq = true;
  static constexpr int kInputs = 0;
  float *C; int ldc;
  __device__ __forceinline__ void prefetch(int, int) const {}
  __device__ __forceinline__ float4 operator()(int, int, float4 a, double &ss) const {
    ss += (double)a.x * a.x + (double)a.y * a.y + (double)a.z * a.z + (double)a.w * a.w;
    return a;
  }
};
struct EpiNormOnly {          // nothing is stored: only sum(acc^2) is wanted (||W g||^2 of the quantised update, whose
                              // step uses W d instead of W g)
  static constexpr bool kDirect = true, kSumsq = true, kStore = false, kCoarse = true;
  static constexpr int kInputs = 0;
  float *C; int ldc;          // ldc = padded width of the output; C is written by the CUDA-core kernels only
  __device__ __forceinline__ void prefetch(int, int) const {}
  __device__ __forceinline__ float4 operator()(int, int, float4 a, double &ss) const {
    ss += (double)a.x * a.x + (double)a.y * a.y + (double)a.z * a.z + (double)a.w * a.w;
    return a;
  }
};
struct EpiLinearResidual {    // C = acc + b[col] - Z[row][col]     (r = W p + b - z)
  static constexpr bool kDirect = false, kSumsq = false;
  static constexpr int kInputs = 1;        // float4 loads per output group: load() fetches, apply() combines
  float *C; int ldc; const float *bias; const float *Z; uint32_t *amax;
  __device__ __forceinline__ void prefetch(int row, int col) const { prefetch_l2(Z + (size_t)row * ldc + col); }
  __device__ __forceinline__ void load(int row, int col, float4 *in) const {
    in[0] = *reinterpret_cast<const float4 *>(Z + (size_t)row * ldc + col);
  }
  __device__ __forceinline__ float4 apply(int col, float4 a, const float4 *in) const {
    const float4 b = *reinterpret_cast<const float4 *>(bias + col);
    return make_float4(a.x + b.x - in[0].x, a.y + b.y - in[0].y, a.z + b.z - in[0].z, a.w + b.w - in[0].w);
  }
  __device__ __forceinline__ float4 operator()(int row, int col, float4 a, double &) const {
    const float4 z = *reinterpret_cast<const float4 *>(Z + (size_t)row * ldc + col);
    const float4 b = *reinterpret_cast<const float4 *>(bias + col);
    return make_float4(a.x + b.x - z.x, a.y + b.y - z.y, a.z + b.z - z.z, a.w + b.w - z.w);
  }
};
struct EpiAddSumsq {          // C = acc + R, accumulates sum(acc^2)     (the quantised step: r + W d beside ||W d||^2)
  static constexpr bool kDirect = false, kSumsq = true, kSumsqOfAcc = true;
  static constexpr int kInputs = 1;
  float *C; int ldc; const float *R; uint32_t *amax;
  __device__ __forceinline__ void prefetch(int row, int col) const { prefetch_l2(R + (size_t)row * ldc + col); }
  __device__ __forceinline__ void load(int row, int col, float4 *in) const {
    in[0] = *reinterpret_cast<const float4 *>(R + (size_t)row * ldc + col);
  }
  __device__ __forceinline__ float4 apply(int, float4 a, const float4 *in) const {
    return make_float4(a.x + in[0].x, a.y + in[0].y, a.z + in[0].z, a.w + in[0].w);
  }
  __device__ __forceinline__ float4 operator()(int row, int col, float4 a, double &ss) const {
    float4 in;
    load(row, col, &in);
    ss += (double)a.x * a.x + (double)a.y * a.y + (double)a.z * a.z + (double)a.w * a.w;
    return apply(col, a, &in);
  }
};
struct EpiBiasAct {           // C = acc + b[col], then f (selected by `slope`, see act_eval) if relu != 0   (z = W p + b, p' = f(z))
  static constexpr bool kDirect = false, kSumsq = false;
  static constexpr int kInputs = 0;
  float *C; int ldc; const float *bias; int relu; float slope; uint32_t *amax;
  __device__ __forceinline__ float f(float x) const { return act_eval(x, slope); }
  __device__ __forceinline__ void prefetch(int, int) const {}
  __device__ __forceinline__ void load(int, int, float4 *) const {}
  __device__ __forceinline__ float4 apply(int col, float4 a, const float4 *) const {
    const float4 b = *reinterpret_cast<const float4 *>(bias + col);
    float4 o = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
    if (relu) { o.x = f(o.x); o.y = f(o.y); o.z = f(o.z); o.w = f(o.w); }
    return o;
  }
  __device__ __forceinline__ float4 operator()(int, int col, float4 a, double &) const { return apply(col, a, nullptr); }
};
struct EpiGradT {             // C = nu*acc + T, accumulates sum(C^2); T = u_{l-1} + rho (p_l - q_{l-1}) is kept
                              // up to date by the kernel that updates q and u (p-gradient of Eq. "update p")
  static constexpr bool kDirect = false, kSumsq = true;
  static constexpr int kInputs = 1;
  float *C; int ldc; const float *T; float nu; uint32_t *amax;
  __device__ __forceinline__ void load(int row, int col, float4 *in) const {
    in[0] = *reinterpret_cast<const float4 *>(T + (size_t)row * ldc + col);
  }
  __device__ __forceinline__ float4 apply(int, float4 a, const float4 *in) const {
    return make_float4(fmaf(nu, a.x, in[0].x), fmaf(nu, a.y, in[0].y), fmaf(nu, a.z, in[0].z), fmaf(nu, a.w, in[0].w));
  }
  __device__ __forceinline__ void prefetch(int row, int col) const { prefetch_l2(T + (size_t)row * ldc + col); }
  __device__ __forceinline__ float4 operator()(int row, int col, float4 a, double &ss) const {
    float4 in;
    load(row, col, &in);
    const float4 g = apply(col, a, &in);
    ss += (double)g.x * g.x + (double)g.y * g.y + (double)g.z * g.z + (double)g.w * g.w;
    return g;
  }
};
struct EpiGradTCopy : EpiGradT {   // the same, and (tensor-core kernel only) the result once more as an fp16 plane H [rows][ldc],
                                   // scaled by 2^(*h_exp) and rounded to 11 bits like the hi plane of an operand
                                   // (rows_planes_kernel says what it is for)
  static constexpr bool kHalfCopy = true;
  __half *H; const int *h_exp;
};

// ---- NT kernel -----------------------------------------------------------------------------------
// Thread (tx, ty) of a 16x16 block owns rows {ty*4+i, 64+ty*4+i} and columns {tx*4+j, 64+tx*4+j}.
// Rows are padded to a multiple of 4 columns and every group of 4 columns starts at a multiple of 4,
// so a group is either inside the padded row or outside it.  Padding columns of the output come out
// as zero because the padding of every input (operand rows >= N, bias, Z, U, P, Q) is zero.
// B_NMAJOR = false: B is [N][ldb], contiguous along K.  B_NMAJOR = true: B is [K][ldb], contiguous along N.
template <bool B_NMAJOR, class Epi>
__global__ void __launch_bounds__(SG_THREADS)
gemm_nt_kernel(int M, int N, int K, const float *__restrict__ A, int lda, const float *__restrict__ B, int ldb,
               Epi epi, double *__restrict__ partials) {
  __shared__ float As[2][SG_BK][SG_BM + 4];
  __shared__ float Bs[2][SG_BK][SG_BN + 4];
  __shared__ double red[SG_THREADS / 32];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  // loader: thread -> (row = t/2, k = (t%2)*4), one float4 along K
  const int lr = t >> 1, lk = (t & 1) * 4;
  const float *a_ptr = A + (size_t)(m0 + lr) * lda + lk;
  const float *b_ptr = B + (size_t)(n0 + lr) * ldb + lk;
  const bool a_row_ok = (m0 + lr) < M, b_row_ok = (n0 + lr) < N;

  auto load = [&](const float *ptr, bool ok, int k0) -> float4 {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (ok) {
      const int k = k0 + lk;
      if (k + 3 < K) v = *reinterpret_cast<const float4 *>(ptr + k0);
      else {
        if (k < K) v.x = ptr[k0];
        if (k + 1 < K) v.y = ptr[k0 + 1];
        if (k + 2 < K) v.z = ptr[k0 + 2];
      }
    }
    return v;
  };
  auto stash = [&](float (*S)[SG_BM + 4], float4 v) {
    S[lk + 0][lr] = v.x; S[lk + 1][lr] = v.y; S[lk + 2][lr] = v.z; S[lk + 3][lr] = v.w;
  };

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  // loader of an N-major B: thread -> (k = t/32, 4 consecutive columns)
  const int bk = t >> 5, bn = (t & 31) * 4;
  const int n_lim = (N + 3) & ~3;
  auto load_bn = [&](int k0) -> float4 {
    const int k = k0 + bk, c = n0 + bn;
    if (k < K && c < n_lim) return *reinterpret_cast<const float4 *>(B + (size_t)k * ldb + c);
    return make_float4(0.f, 0.f, 0.f, 0.f);
  };
  auto put_b = [&](int buf, float4 v) {
    if (B_NMAJOR) *reinterpret_cast<float4 *>(&Bs[buf][bk][bn]) = v;
    else stash(Bs[buf], v);
  };

  float4 ra = load(a_ptr, a_row_ok, 0), rb = B_NMAJOR ? load_bn(0) : load(b_ptr, b_row_ok, 0);
  stash(As[0], ra); put_b(0, rb);
  __syncthreads();
  const int nk = (K + SG_BK - 1) / SG_BK;
  for (int kb = 0; kb < nk; ++kb) {
    const int cur = kb & 1;
    if (kb + 1 < nk) {
      ra = load(a_ptr, a_row_ok, (kb + 1) * SG_BK);
      rb = B_NMAJOR ? load_bn((kb + 1) * SG_BK) : load(b_ptr, b_row_ok, (kb + 1) * SG_BK);
    }
#pragma unroll
    for (int k = 0; k < SG_BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4 *>(&As[cur][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4 *>(&As[cur][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4 *>(&Bs[cur][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4 *>(&Bs[cur][k][64 + tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    if (kb + 1 < nk) { stash(As[cur ^ 1], ra); put_b(cur ^ 1, rb); }
    __syncthreads();
  }

  double ss = 0.0;
  const int n_pad = epi.ldc;        // padding columns are written too: they come out as exact zeros
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (row >= M) continue;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int col = n0 + h * 64 + tx * 4;
      if (col >= n_pad) continue;
      float4 a = make_float4(acc[i][h * 4 + 0], acc[i][h * 4 + 1], acc[i][h * 4 + 2], acc[i][h * 4 + 3]);
      float4 o = epi(row, col, a, ss);
      *reinterpret_cast<float4 *>(epi.C + (size_t)row * epi.ldc + col) = o;
    }
  }
  if (partials != nullptr) {
    const double tot = block_sum<SG_THREADS>(ss, red);
    if (t == 0) partials[blockIdx.y * gridDim.x + blockIdx.x] = tot;
  }
}

// ---- TN kernel (contraction over the node index), split over grid.z ------------------------------
// A is [K][lda] with M valid columns, B is [K][ldb] with N valid columns.  Slice z of the grid handles
// rows [z*k_chunk, min(K,(z+1)*k_chunk)) and writes its partial tile to part[z][M][ldc].
__global__ void __launch_bounds__(SG_THREADS)
gemm_tn_kernel(int M, int N, int K, int k_chunk, const float *__restrict__ A, int lda,
               const float *__restrict__ B, int ldb, float *__restrict__ part, int ldc) {
  __shared__ float As[2][SG_BK][SG_BM + 4];
  __shared__ float Bs[2][SG_BK][SG_BN + 4];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  const int k_begin = blockIdx.z * k_chunk, k_end = min(K, k_begin + k_chunk);
  const int lkk = t >> 5, lm = (t & 31) * 4;                 // loader: k = t/32, 4 consecutive output indices
  const int ma = (M + 3) & ~3, na = (N + 3) & ~3;

  auto load = [&](const float *P, int ld, int base, int lim, int k) -> float4 {
    const int kk = k + lkk, c = base + lm;
    if (kk < k_end && c < lim) return *reinterpret_cast<const float4 *>(P + (size_t)kk * ld + c);
    return make_float4(0.f, 0.f, 0.f, 0.f);
  };

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  float4 ra = load(A, lda, m0, ma, k_begin), rb = load(B, ldb, n0, na, k_begin);
  *reinterpret_cast<float4 *>(&As[0][lkk][lm]) = ra;
  *reinterpret_cast<float4 *>(&Bs[0][lkk][lm]) = rb;
  __syncthreads();
  const int nk = (max(k_end - k_begin, 0) + SG_BK - 1) / SG_BK;
  for (int kb = 0; kb < nk; ++kb) {
    const int cur = kb & 1;
    if (kb + 1 < nk) {
      ra = load(A, lda, m0, ma, k_begin + (kb + 1) * SG_BK);
      rb = load(B, ldb, n0, na, k_begin + (kb + 1) * SG_BK);
    }
#pragma unroll
    for (int k = 0; k < SG_BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4 *>(&As[cur][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4 *>(&As[cur][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4 *>(&Bs[cur][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4 *>(&Bs[cur][k][64 + tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    if (kb + 1 < nk) {
      *reinterpret_cast<float4 *>(&As[cur ^ 1][lkk][lm]) = ra;
      *reinterpret_cast<float4 *>(&Bs[cur ^ 1][lkk][lm]) = rb;
    }
    __syncthreads();
  }
  float *out = part + (size_t)blockIdx.z * M * ldc;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (row >= M) continue;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int col = n0 + h * 64 + tx * 4;
      if (col >= ldc) continue;      // padding columns are written too (exact zeros)
      *reinterpret_cast<float4 *>(out + (size_t)row * ldc + col) =
          make_float4(acc[i][h * 4 + 0], acc[i][h * 4 + 1], acc[i][h * 4 + 2], acc[i][h * 4 + 3]);
    }
  }
}

}  // namespace pd
