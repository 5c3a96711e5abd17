// Elementwise, reduction and per-node kernels of one pdADMM-G / pdADMM-G-Q iteration.
//
// All matrices are node-major [N][ld] float32 with ld a multiple of 4 and zero padding columns,
// so a matrix is processed as a flat array of N*ld/4 float4 values.  Every operation below maps
// zero padding to zero padding.  Sums are accumulated per block in double precision and written
// to a slot per block; a single-block kernel adds the slots in index order, so results do not
// depend on scheduling.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

namespace pd {

constexpr int EW_THREADS = 256;

// ---- largest magnitude of an array (see commit_amax) ---------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
absmax_kernel(const float *__restrict__ x, size_t n4, uint32_t *__restrict__ word) {
  uint32_t m = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x)
    m = max(m, abs_bits(reinterpret_cast<const float4 *>(x)[i]));
  commit_amax(m, word);
}

// Scalars of one layer that live on the device (so that an iteration needs no host round trip).
struct LayerScalars {
  double sum_g2;      // ||g||^2
  double sum_wg2;     // ||W g||^2
  double sum_d2;      // ||p+ - p||^2        (quantised trial)
  double sum_wd2;     // ||W (p+ - p)||^2    (quantised trial)
  double sum_G2;      // ||grad_W||^2
  double sum_Gp2;     // ||grad_W p+||^2
  double res2;        // ||p_{l+1} - q_l||^2
  double tau;         // tau_l
  double theta;       // theta_l (0 if grad_W = 0)
  float inv_tau;      // 1/tau
  float inv_theta;    // 1/theta, 0 if grad_W = 0
  int accepted;       // quantised trial: 1 if the stop condition held
  int trials;         // trials so far in this iteration
};

__device__ __forceinline__ float4 ld4(const float *p, size_t i) { return reinterpret_cast<const float4 *>(p)[i]; }
__device__ __forceinline__ float4 ld4f(const float *p, size_t i) { return reinterpret_cast<const float4 *>(p)[i]; }
__device__ __forceinline__ void st4(float *p, size_t i, float4 v) { reinterpret_cast<float4 *>(p)[i] = v; }

// ---- final, fixed-order reduction of per-block slots -------------------------------------------
// out[j] = sum_i slots[i * stride + j], j < n_out, i < n_slots.  One block of 256 threads: thread t adds the
// slots t, t+256, ... in that order, then the 256 partial sums are combined in a fixed tree, so the result
// does not depend on scheduling.
__global__ void __launch_bounds__(256)
reduce_slots_kernel(const double *__restrict__ slots, int n_slots, int stride, int n_out, double *__restrict__ out) {
  __shared__ double sh[256];
  for (int j = 0; j < n_out; ++j) {
    double s = 0.0;
    for (int i = threadIdx.x; i < n_slots; i += 256) s += slots[(size_t)i * stride + j];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
      if (threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
      __syncthreads();
    }
    if (threadIdx.x == 0) out[j] = sh[0];
    __syncthreads();
  }
}

// Quantisation to m uniform levels lo, lo + s, ... (Eq. "update p quantized", elementwise argmin):
// code = clamp(floor((x - lo)/s + 1/2), 0, m-1), value = lo + float(code) * s, every operation rounded once.
__device__ __forceinline__ float quantize_one(float x, float s, float lo, float top, unsigned &code) {
  float c = floorf(__fdiv_rn(__fsub_rn(x, lo), s) + 0.5f);
  c = fminf(fmaxf(c, 0.0f), top);
  code = (unsigned)c;
  return __fadd_rn(lo, __fmul_rn(c, s));
}

// Four consecutive values of a quantised matrix from its codes: lo + code * s, rounded as quantize_one rounds them,
// i.e. bit for bit the stored values (1 or 2 bytes read per value instead of 4).
__device__ __forceinline__ float4 levels_of4(const void *__restrict__ codes, int wide_codes, size_t i, float s, float lo) {
  float c0, c1, c2, c3;
  if (wide_codes) {
    const ushort4 o = reinterpret_cast<const ushort4 *>(codes)[i];
    c0 = o.x; c1 = o.y; c2 = o.z; c3 = o.w;
  } else {
    const uchar4 o = reinterpret_cast<const uchar4 *>(codes)[i];
    c0 = o.x; c1 = o.y; c2 = o.z; c3 = o.w;
  }
  return make_float4(__fadd_rn(lo, __fmul_rn(c0, s)), __fadd_rn(lo, __fmul_rn(c1, s)), __fadd_rn(lo, __fmul_rn(c2, s)),
                     __fadd_rn(lo, __fmul_rn(c3, s)));
}

// ---- y -= x * (*inv) ----------------------------------------------------------------------------
// p-update  p+ = p - g/tau  (Eq. "update p") and the matching update of the linear residual,
// r <- r - (W g)/tau, and r <- r - (grad_W p+)/theta after the W-update (Eq. "update W").
__global__ void __launch_bounds__(EW_THREADS)
axpy_neg_kernel(float *__restrict__ y, const float *__restrict__ x, const float *__restrict__ inv, size_t n4,
                uint32_t *__restrict__ amax /* receives max|y| (see commit_amax); may be null */) {
  const float a = *inv;
  uint32_t m = 0u;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  // four groups per pass: eight loads in flight per thread
  for (; i + 3 * stride < n4; i += 4 * stride) {
    float4 v[4], w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) { v[k] = ld4(y, i + k * stride); w[k] = ld4(x, i + k * stride); }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[k].x = fmaf(-a, w[k].x, v[k].x); v[k].y = fmaf(-a, w[k].y, v[k].y);
      v[k].z = fmaf(-a, w[k].z, v[k].z); v[k].w = fmaf(-a, w[k].w, v[k].w);
      st4(y, i + k * stride, v[k]);
      m = max(m, abs_bits(v[k]));
    }
  }
  for (; i < n4; i += stride) {
    float4 v = ld4(y, i);
    const float4 w = ld4(x, i);
    v.x = fmaf(-a, w.x, v.x); v.y = fmaf(-a, w.y, v.y); v.z = fmaf(-a, w.z, v.z); v.w = fmaf(-a, w.w, v.w);
    st4(y, i, v);
    m = max(m, abs_bits(v));
  }
  if (amax != nullptr) commit_amax(m, amax);
}

// ---- quantised trial step ------------------------------------------------------------------------
// x = p - g/tau; p_new = nearest level; d = p_new - p; codes; per-block sum of d^2.
// p lies on the level set, p = lo + code * scale bit for bit (quantize_one), so it is read as its 1- or 2-byte codes
// instead of as 4-byte values.
__global__ void __launch_bounds__(EW_THREADS)
quant_trial_kernel(const float *__restrict__ g, const LayerScalars *__restrict__ sc,
                   float scale, float lo, int levels, float *__restrict__ p_new, float *__restrict__ d /* may be null */,
                   void *__restrict__ codes, int wide_codes, size_t n4, double *__restrict__ slots,
                   uint32_t *__restrict__ amax_p /* max|p_new|, may be null */, uint32_t *__restrict__ amax_d /* max|d| */,
                   const void *__restrict__ codes_old /* codes of p */,
                   __half *__restrict__ pn_plane /* the new codes as fp16 integers (operand plane of p_new = code * scale) */,
                   __half *__restrict__ d_plane /* new code - old code as fp16 integers (operand plane of d) */) {
  __shared__ double red[EW_THREADS / 32];
  const float inv_tau = sc->inv_tau, top = (float)(levels - 1);
  double ss = 0.0;
  uint32_t mp = 0u, md = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 gv = ld4(g, i);
    int o0, o1, o2, o3;
    if (wide_codes) {
      const ushort4 o = reinterpret_cast<const ushort4 *>(codes_old)[i];
      o0 = o.x; o1 = o.y; o2 = o.z; o3 = o.w;
    } else {
      const uchar4 o = reinterpret_cast<const uchar4 *>(codes_old)[i];
      o0 = o.x; o1 = o.y; o2 = o.z; o3 = o.w;
    }
    const float4 pv = make_float4(__fadd_rn(lo, __fmul_rn((float)o0, scale)), __fadd_rn(lo, __fmul_rn((float)o1, scale)),
                                  __fadd_rn(lo, __fmul_rn((float)o2, scale)), __fadd_rn(lo, __fmul_rn((float)o3, scale)));
    unsigned c0, c1, c2, c3;
    float4 nv, dv;
    nv.x = quantize_one(fmaf(-inv_tau, gv.x, pv.x), scale, lo, top, c0);
    nv.y = quantize_one(fmaf(-inv_tau, gv.y, pv.y), scale, lo, top, c1);
    nv.z = quantize_one(fmaf(-inv_tau, gv.z, pv.z), scale, lo, top, c2);
    nv.w = quantize_one(fmaf(-inv_tau, gv.w, pv.w), scale, lo, top, c3);
    dv.x = nv.x - pv.x; dv.y = nv.y - pv.y; dv.z = nv.z - pv.z; dv.w = nv.w - pv.w;
    ss += (double)dv.x * dv.x + (double)dv.y * dv.y + (double)dv.z * dv.z + (double)dv.w * dv.w;
    st4(p_new, i, nv);
    if (d != nullptr) st4(d, i, dv);     // with the integer planes below the product W d reads d_plane instead
    mp = max(mp, abs_bits(nv)); md = max(md, abs_bits(dv));
    if (wide_codes)      // more than 256 levels: 16-bit codes
      reinterpret_cast<ushort4 *>(codes)[i] = make_ushort4((unsigned short)c0, (unsigned short)c1, (unsigned short)c2, (unsigned short)c3);
    else
      reinterpret_cast<uchar4 *>(codes)[i] = make_uchar4((unsigned char)c0, (unsigned char)c1, (unsigned char)c2, (unsigned char)c3);
    if (pn_plane != nullptr) {
      // integers below 2048 are exact in fp16: the planes hold the codes themselves and their change
      const __half2 a = __floats2half2_rn((float)c0, (float)c1), b = __floats2half2_rn((float)c2, (float)c3);
      const __half2 e = __floats2half2_rn((float)((int)c0 - o0), (float)((int)c1 - o1));
      const __half2 f = __floats2half2_rn((float)((int)c2 - o2), (float)((int)c3 - o3));
      reinterpret_cast<uint2 *>(pn_plane)[i] = make_uint2(*reinterpret_cast<const uint32_t *>(&a), *reinterpret_cast<const uint32_t *>(&b));
      reinterpret_cast<uint2 *>(d_plane)[i] = make_uint2(*reinterpret_cast<const uint32_t *>(&e), *reinterpret_cast<const uint32_t *>(&f));
    }
  }
  if (amax_p != nullptr) { commit_amax(mp, amax_p); commit_amax(md, amax_d); }
  const double tot = block_sum<EW_THREADS>(ss, red);
  if (threadIdx.x == 0) slots[blockIdx.x] = tot;
}

// Plain projection of an array (initial forward pass, pdadmm_quantize, pdadmm_set_tensor).
__global__ void __launch_bounds__(EW_THREADS)
quantize_kernel(const float *x, size_t n, float scale, float lo, int levels, float *p_out /* may be x itself */,
                void *__restrict__ codes_out, int wide_codes) {
  const float top = (float)(levels - 1);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    unsigned c;
    const float v = quantize_one(x[i], scale, lo, top, c);
    if (p_out) p_out[i] = v;
    if (codes_out) {
      if (wide_codes) reinterpret_cast<uint16_t *>(codes_out)[i] = (uint16_t)c;
      else reinterpret_cast<uint8_t *>(codes_out)[i] = (uint8_t)c;
    }
  }
}

// ---- operand planes of a quantised p from its codes ------------------------------------------------------------
// p = code * s with code < 2048: the fp16 plane of the integer codes is the whole operand (the products multiply by s).
// Same orientation [N][ld] ...
__global__ void __launch_bounds__(EW_THREADS)
codes_to_plane_kernel(const void *__restrict__ codes, int wide_codes, size_t n4, __half *__restrict__ plane) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float c0, c1, c2, c3;
    if (wide_codes) {
      const ushort4 o = reinterpret_cast<const ushort4 *>(codes)[i];
      c0 = o.x; c1 = o.y; c2 = o.z; c3 = o.w;
    } else {
      const uchar4 o = reinterpret_cast<const uchar4 *>(codes)[i];
      c0 = o.x; c1 = o.y; c2 = o.z; c3 = o.w;
    }
    const __half2 a = __floats2half2_rn(c0, c1), b = __floats2half2_rn(c2, c3);
    reinterpret_cast<uint2 *>(plane)[i] = make_uint2(*reinterpret_cast<const uint32_t *>(&a), *reinterpret_cast<const uint32_t *>(&b));
  }
}
// ... and transposed [cols][ldT] (node index contiguous), for the product that contracts over the nodes.  One block of
// 32 x 8 threads per tile of 32 nodes x 32 columns, through shared memory.
__global__ void __launch_bounds__(256)
transpose_codes_kernel(const void *__restrict__ codes, int wide_codes, int rows, int cols, int ld,
                       __half *__restrict__ planeT, int ldT) {
  __shared__ __half sh[32][33];
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + threadIdx.y + 8 * i, c = c0 + threadIdx.x;
    float v = 0.f;
    if (r < rows && c < cols) {
      const size_t o = (size_t)r * ld + c;
      v = wide_codes ? (float)reinterpret_cast<const uint16_t *>(codes)[o] : (float)reinterpret_cast<const uint8_t *>(codes)[o];
    }
    sh[threadIdx.y + 8 * i][threadIdx.x] = __float2half_rn(v);
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = c0 + threadIdx.y + 8 * i, r = r0 + threadIdx.x;
    if (c < cols && r < rows) planeT[(size_t)c * ldT + r] = sh[threadIdx.x][threadIdx.y + 8 * i];
  }
}

// ---- finalisers of the step parameters (one block of FIN_THREADS threads) ---------------------------------
// Fixed-order sum of n slots by one block of FIN_THREADS threads: thread t adds slots t, t + FIN_THREADS, ..., then a
// fixed tree.  Result in thread 0.
constexpr int FIN_THREADS = 1024;
__device__ __forceinline__ double block_sum_slots(const double *__restrict__ slots, int n, double *sh /* FIN_THREADS */) {
  // four independent partial sums per thread keep four loads in flight; the order of the additions is fixed
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  int i = threadIdx.x;
  for (; i + 3 * FIN_THREADS < n; i += 4 * FIN_THREADS) {
    s0 += slots[i]; s1 += slots[i + FIN_THREADS]; s2 += slots[i + 2 * FIN_THREADS]; s3 += slots[i + 3 * FIN_THREADS];
  }
  for (; i < n; i += FIN_THREADS) s0 += slots[i];
  const double s = (s0 + s1) + (s2 + s3);
  __syncthreads();
  sh[threadIdx.x] = s;
  __syncthreads();
  for (int w = FIN_THREADS / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
    __syncthreads();
  }
  return sh[0];
}
// ||g||^2 and ||W g||^2 from their slots, then
// tau = rho + nu ||W g||^2 / ||g||^2 : the smallest tau with phi(p - g/tau) <= U_l(p - g/tau; tau).
__global__ void __launch_bounds__(FIN_THREADS)
finalize_tau_kernel(LayerScalars *sc, double rho, double nu, const double *slots_g, int n_g, const double *slots_wg, int n_wg,
                    int *nonfinite, uint32_t *clear_word /* max|p| of the layer restarts with the coming p-step */,
                    const uint32_t *amax_g = nullptr, int *next_g_exp = nullptr /* scaling of the next iteration's fp16 copy of g */) {
  __shared__ double sh[FIN_THREADS];
  const double gg = block_sum_slots(slots_g, n_g, sh);
  const double wg = block_sum_slots(slots_wg, n_wg, sh);
  if (threadIdx.x == 0) {
    sc->sum_g2 = gg;
    sc->sum_wg2 = wg;
    if (!(isfinite(gg) && isfinite(wg))) *nonfinite = 1;      // a NaN or Inf anywhere in the state reaches these sums
    const double tau = gg > 0.0 ? rho + nu * wg / gg : rho;
    sc->tau = tau;
    sc->inv_tau = (float)(1.0 / tau);
    sc->accepted = 0;
    sc->trials = 0;
    if (clear_word != nullptr) *clear_word = 0u;
    if (next_g_exp != nullptr) *next_g_exp = tc_predict_exp(*amax_g);
  }
}
// Stop condition of the quantised step in its quadratic form: nu||W d||^2 + rho||d||^2 <= tau||d||^2 (1 + slack).
// Not accepted: tau is doubled for the next trial.
__global__ void __launch_bounds__(FIN_THREADS)
finalize_trial_kernel(LayerScalars *sc, double rho, double nu, double slack, const double *slots_d, int n_d,
                      const double *slots_wd, int n_wd) {
  __shared__ double sh[FIN_THREADS];
  const double dd = block_sum_slots(slots_d, n_d, sh);
  const double wd = block_sum_slots(slots_wd, n_wd, sh);
  if (threadIdx.x == 0) {
    sc->sum_d2 = dd;
    sc->sum_wd2 = wd;
    const bool ok = nu * wd + rho * dd <= sc->tau * dd * (1.0 + slack);
    sc->trials += 1;
    sc->accepted = ok ? 1 : 0;
    if (!ok) {
      sc->tau *= 2.0;
      sc->inv_tau = (float)(1.0 / sc->tau);
    }
  }
}
// ||grad_W||^2 and ||grad_W p+||^2 from their slots, then
// theta = nu ||grad_W p+||^2 / ||grad_W||^2 : the smallest theta with phi(W+) <= V_l(W+; theta).
__global__ void __launch_bounds__(FIN_THREADS)
finalize_theta_kernel(LayerScalars *sc, double nu, const double *slots_G, int n_G, const double *slots_Gp, int n_Gp,
                      int *nonfinite, uint32_t *clear_word /* max|r| of the layer restarts with the coming z-step */) {
  __shared__ double sh[FIN_THREADS];
  const double GG = block_sum_slots(slots_G, n_G, sh);
  const double Gp = block_sum_slots(slots_Gp, n_Gp, sh);
  if (threadIdx.x == 0) {
    sc->sum_G2 = GG;
    sc->sum_Gp2 = Gp;
    if (!(isfinite(GG) && isfinite(Gp))) *nonfinite = 1;
    const double theta = GG > 0.0 ? nu * Gp / GG : 0.0;
    sc->theta = theta;
    sc->inv_theta = theta > 0.0 ? (float)(1.0 / theta) : 0.0f;
    if (clear_word != nullptr) *clear_word = 0u;
  }
}

// ---- fp16 operand planes of a weight-sized matrix --------------------------------------------------
// x [rows][ld] fp32 -> hi, lo [rows][ldh] (same orientation) and, if asked for, hiT, loT [cols][ldhT] (transposed),
// so that every tensor-core product finds its small operand contiguous along the contraction index.
// xs = x 2^e with e from max|x| (`amax`, see tc_scale_exp); hi = xs rounded to 11 significant bits,
// lo = (xs - hi) 2^11; e is stored in *exp_out for the products that use the planes.
// One block of 32 x 8 threads per 32 x 32 tile.
__global__ void __launch_bounds__(256)
make_planes_kernel(const float *__restrict__ x, int rows, int cols, int ld, const uint32_t *__restrict__ amax,
                   int *__restrict__ exp_out, __half *__restrict__ hi, __half *__restrict__ lo, int ldh,
                   __half *__restrict__ hiT, __half *__restrict__ loT, int ldhT) {
  __shared__ __half sh_hi[32][33], sh_lo[32][33];
  const int e = tc_scale_exp(*amax);
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0 && threadIdx.y == 0) *exp_out = e;
  const float scale = __uint_as_float((uint32_t)(e + 127) << 23);
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + threadIdx.y + 8 * i, c = c0 + threadIdx.x;
    __half h = __float2half_rn(0.f), l = h;
    if (r < rows && c < cols) {
      const float xs = x[(size_t)r * ld + c] * scale;
      const float hf = __uint_as_float((__float_as_uint(xs) + 0x1000u) & 0xFFFFE000u);
      h = __float2half_rn(hf);
      l = __float2half_rn((xs - hf) * 2048.0f);
      if (hi != nullptr) { hi[(size_t)r * ldh + c] = h; lo[(size_t)r * ldh + c] = l; }
    }
    sh_hi[threadIdx.y + 8 * i][threadIdx.x] = h;
    sh_lo[threadIdx.y + 8 * i][threadIdx.x] = l;
  }
  if (hiT == nullptr) return;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = c0 + threadIdx.y + 8 * i, r = r0 + threadIdx.x;
    if (c < cols && r < rows) {
      hiT[(size_t)c * ldhT + r] = sh_hi[threadIdx.x][threadIdx.y + 8 * i];
      loT[(size_t)c * ldhT + r] = sh_lo[threadIdx.x][threadIdx.y + 8 * i];
    }
  }
}

// ---- fp16 planes of a node-major matrix, same orientation -------------------------------------------
// x [rows][ld] fp32 -> hi, lo [rows][ld] halves (the padding columns, zero in x, come out as zero): the streamed
// operand of a product whose output is several column tiles wide, split once here instead of once per column tile
// inside the product.  Scaling and split as in make_planes_kernel; the exponent goes to *exp_out.  A thread converts
// eight consecutive values (two 16-byte loads, one 16-byte store per plane).
// `predicted` (may be null): the hi plane was already written by the kernel that produced x, scaled by 2^(*predicted),
// an exponent chosen before max|x| was known (from the previous iteration's maximum, see tc_predict_exp).  If that
// scaling turned out usable -- no overflow, at least 11 bits left: max|x| 2^e in [2^4, 2^15) -- nothing is left to do
// but to publish the exponent; otherwise the plane is written again here with the exponent from the true maximum.
// Only for hi-plane-only operands (lo == nullptr): 11 bits are all such a product wants.
__global__ void __launch_bounds__(256)
rows_planes_kernel(const float *__restrict__ x, size_t n8, const uint32_t *__restrict__ amax, int *__restrict__ exp_out,
                   __half *__restrict__ hi, __half *__restrict__ lo, const int *__restrict__ predicted = nullptr) {
  if (predicted != nullptr && lo == nullptr && tc_prediction_usable(*amax, *predicted)) {
    if (blockIdx.x == 0 && threadIdx.x == 0) *exp_out = *predicted;
    return;
  }
  const int e = tc_scale_exp(*amax);
  if (blockIdx.x == 0 && threadIdx.x == 0) *exp_out = e;
  const float scale = __uint_as_float((uint32_t)(e + 127) << 23);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
    const float4 a = reinterpret_cast<const float4 *>(x)[2 * i], b = reinterpret_cast<const float4 *>(x)[2 * i + 1];
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float h[8], l[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float xs = v[k] * scale;
      h[k] = __uint_as_float((__float_as_uint(xs) + 0x1000u) & 0xFFFFE000u);
      l[k] = (xs - h[k]) * 2048.0f;
    }
    auto pack = [](float p, float q) {
      const __half2 t = __floats2half2_rn(p, q);
      return *reinterpret_cast<const uint32_t *>(&t);
    };
    reinterpret_cast<uint4 *>(hi)[i] = make_uint4(pack(h[0], h[1]), pack(h[2], h[3]), pack(h[4], h[5]), pack(h[6], h[7]));
    if (lo != nullptr)        // a product that only wants its squared norm uses the hi plane alone
      reinterpret_cast<uint4 *>(lo)[i] = make_uint4(pack(l[0], l[1]), pack(l[2], l[3]), pack(l[4], l[5]), pack(l[6], l[7]));
  }
}

// ---- fp16 planes of a node-major matrix, transposed -------------------------------------------------
// x [rows = nodes][ld] fp32 -> hiT, loT [cols][ldT] with the node index contiguous: operands of the product that
// contracts over the nodes (the W-gradient r^T p+), for layers where splitting them once here is cheaper than
// splitting them once per output tile inside that product.  Scaling and split as in make_planes_kernel; the
// exponent goes to *exp_out.
// A warp handles 32 nodes x 32 columns: lane (q, g) loads the 4 x 8 block of nodes 4q..4q+3, columns 8g..8g+7
// (eight 16-byte loads, 128 contiguous bytes per row and warp), transposes it in registers and stores, per column,
// the four nodes as 8 bytes of each plane (64 contiguous bytes per column and warp): whole sectors both ways, no
// shared memory.  Tiles are numbered with the node index fastest.
__global__ void __launch_bounds__(256)
transpose_planes_kernel(const float *__restrict__ x, int rows, int cols, int ld, const uint32_t *__restrict__ amax,
                        int *__restrict__ exp_out, __half *__restrict__ hiT, __half *__restrict__ loT, int ldT) {
  const int e = tc_scale_exp(*amax);
  if (blockIdx.x == 0 && threadIdx.x == 0) *exp_out = e;
  const float scale = __uint_as_float((uint32_t)(e + 127) << 23);
  const int lane = threadIdx.x & 31, q = lane & 7, g = lane >> 3;
  const long long row_tiles = (rows + 31) / 32, n_tiles = row_tiles * ((cols + 31) / 32);
  for (long long wt = blockIdx.x * 8ll + (threadIdx.x >> 5); wt < n_tiles; wt += gridDim.x * 8ll) {
    const int node0 = (int)(wt % row_tiles) * 32 + 4 * q, col = (int)(wt / row_tiles) * 32 + 8 * g;
    if (node0 >= rows || col >= cols) continue;
    float v[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float4 t0 = make_float4(0.f, 0.f, 0.f, 0.f), t1 = t0;
      if (node0 + i < rows) {                  // ld is a multiple of 4: a group of 4 columns is inside the row or not
        t0 = *reinterpret_cast<const float4 *>(x + (size_t)(node0 + i) * ld + col);
        if (col + 4 < ld) t1 = *reinterpret_cast<const float4 *>(x + (size_t)(node0 + i) * ld + col + 4);
      }
      v[i][0] = t0.x; v[i][1] = t0.y; v[i][2] = t0.z; v[i][3] = t0.w;
      v[i][4] = t1.x; v[i][5] = t1.y; v[i][6] = t1.z; v[i][7] = t1.w;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (col + j >= cols) break;
      float h[4], l[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float xs = v[i][j] * scale;
        h[i] = __uint_as_float((__float_as_uint(xs) + 0x1000u) & 0xFFFFE000u);
        l[i] = (xs - h[i]) * 2048.0f;
      }
      const __half2 h0 = __floats2half2_rn(h[0], h[1]), h1 = __floats2half2_rn(h[2], h[3]);
      const __half2 l0 = __floats2half2_rn(l[0], l[1]), l1 = __floats2half2_rn(l[2], l[3]);
      const size_t o = (size_t)(col + j) * ldT + node0;
      *reinterpret_cast<uint2 *>(hiT + o) = make_uint2(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1));
      *reinterpret_cast<uint2 *>(loT + o) = make_uint2(*reinterpret_cast<const uint32_t *>(&l0), *reinterpret_cast<const uint32_t *>(&l1));
    }
  }
}

// ---- reduction of the split partial tiles of grad_W, scaling by nu, ||grad_W||^2 ------------------
__global__ void __launch_bounds__(EW_THREADS)
reduce_gradW_kernel(const float *__restrict__ part, int n_split, size_t n4, float nu, float *__restrict__ G,
                    uint32_t *__restrict__ amax, double *__restrict__ slots) {
  __shared__ double red[EW_THREADS / 32];
  double ss = 0.0;
  uint32_t m = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < n_split; ++s) {
      const float4 v = ld4(part + (size_t)s * n4 * 4, i);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    a.x *= nu; a.y *= nu; a.z *= nu; a.w *= nu;
    ss += (double)a.x * a.x + (double)a.y * a.y + (double)a.z * a.z + (double)a.w * a.w;
    st4(G, i, a);
    m = max(m, abs_bits(a));
  }
  if (amax != nullptr) commit_amax(m, amax);        // for the fp16 planes of the tensor-core product G p+
  const double tot = block_sum<EW_THREADS>(ss, red);
  if (threadIdx.x == 0) slots[blockIdx.x] = tot;
}

// ---- column sums of r - gp * inv_theta  (for the b-update) ----------------------------------------
// Block b handles rows [b*rows_per_block, ...).  A thread owns one group of 4 columns (float4) and one row
// subgroup: with ld/4 <= 128 column groups the block's 256 threads cover several rows per pass.  The row
// subgroups' sums are combined in subgroup order, then written to slots[b][ld].
constexpr int COLSUM_MAX_SUB = 8;
__global__ void __launch_bounds__(EW_THREADS)
resid_colsum_kernel(float *__restrict__ r, const float *__restrict__ gp, const LayerScalars *__restrict__ sc,
                    int n_rows, int ld, int rows_per_block, double *__restrict__ slots) {
  extern __shared__ double colsum_sh[];                       // [n_sub][ld] when n_sub > 1
  const float a = sc->inv_theta;
  const int ld4 = ld >> 2;
  const int cols_per_pass = min(ld4, EW_THREADS);
  const int n_sub = min(EW_THREADS / cols_per_pass, COLSUM_MAX_SUB);
  const int sub = threadIdx.x / cols_per_pass, c0 = threadIdx.x % cols_per_pass;
  const int r0 = blockIdx.x * rows_per_block, r1 = min(n_rows, r0 + rows_per_block);
  double *out = slots + (size_t)blockIdx.x * ld;
  if (sub < n_sub) {
    for (int cg = c0; cg < ld4; cg += cols_per_pass) {
      double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
#pragma unroll 4
      for (int j = r0 + sub; j < r1; j += n_sub) {
        const size_t o = (size_t)j * ld4 + cg;
        float4 v = ld4f(r, o);
        const float4 g = ld4f(gp, o);
        v.x = fmaf(-a, g.x, v.x); v.y = fmaf(-a, g.y, v.y); v.z = fmaf(-a, g.z, v.z); v.w = fmaf(-a, g.w, v.w);
        st4(r, o, v);
        s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w;
      }
      double *dst = (n_sub > 1 ? colsum_sh + (size_t)sub * ld : out) + 4 * cg;
      dst[0] = s0; dst[1] = s1; dst[2] = s2; dst[3] = s3;
    }
  }
  if (n_sub > 1) {
    __syncthreads();
    for (int c = threadIdx.x; c < ld; c += blockDim.x) {
      double s = 0.0;
      for (int k = 0; k < n_sub; ++k) s += colsum_sh[(size_t)k * ld + c];
      out[c] = s;
    }
  }
}

// out[c] = sum over the blocks' slots of column c (the first half of finalize_bias_kernel, for a context that owns only
// part of the nodes: the totals are then added over the shards before the mean is taken).  Same thread layout.
constexpr int BIAS_GROUPS = 32;          // slot groups per block of the two kernels below (blockDim = (32, BIAS_GROUPS))
__global__ void __launch_bounds__(32 * BIAS_GROUPS)
colsum_total_kernel(const double *__restrict__ slots, int n_slots, int ld, double *__restrict__ out) {
  __shared__ double sh[BIAS_GROUPS][33];
  const int c = blockIdx.x * 32 + threadIdx.x;
  double s = 0.0;
  if (c < ld)
    for (int i = threadIdx.y; i < n_slots; i += BIAS_GROUPS) s += slots[(size_t)i * ld + c];
  sh[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && c < ld) {
    double t = 0.0;
    for (int k = 0; k < BIAS_GROUPS; ++k) t += sh[k][threadIdx.x];
    out[c] = t;
  }
}

// sum of squares (one slot per block) and largest magnitude of a weight-sized matrix
__global__ void __launch_bounds__(EW_THREADS)
sumsq_amax_kernel(const float *__restrict__ G, size_t n4, uint32_t *__restrict__ amax, double *__restrict__ slots) {
  __shared__ double red[EW_THREADS / 32];
  double ss = 0.0;
  uint32_t m = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 a = ld4(G, i);
    ss += (double)a.x * a.x + (double)a.y * a.y + (double)a.z * a.z + (double)a.w * a.w;
    m = max(m, abs_bits(a));
  }
  if (amax != nullptr) commit_amax(m, amax);
  const double tot = block_sum<EW_THREADS>(ss, red);
  if (threadIdx.x == 0) slots[blockIdx.x] = tot;
}

// b+ = b - mean_j r[j][:]  (Eq. "update b" with the step 1/(nu N), i.e. the exact minimiser);
// shift[c] = that mean, which the z-update subtracts from r.  blockDim = (32 columns, BIAS_GROUPS slot groups): group g
// adds the slots g, g + BIAS_GROUPS, ... of its column, the group sums are then added in group order (32 groups keep
// 32 rows of slots in flight per block; the kernel has only ld / 32 blocks).
__global__ void __launch_bounds__(32 * BIAS_GROUPS)
finalize_bias_kernel(const double *__restrict__ slots, int n_slots, int ld, int width, double inv_n,
                     float *__restrict__ b, float *__restrict__ shift) {
  __shared__ double sh[BIAS_GROUPS][33];
  const int c = blockIdx.x * 32 + threadIdx.x;
  double s = 0.0;
  if (c < ld)
    for (int i = threadIdx.y; i < n_slots; i += BIAS_GROUPS) s += slots[(size_t)i * ld + c];
  sh[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && c < ld) {
    double t = 0.0;
    for (int k = 0; k < BIAS_GROUPS; ++k) t += sh[k][threadIdx.x];
    const float m = c < width ? (float)(t * inv_n) : 0.0f;
    shift[c] = m;
    if (c < width) b[c] -= m;
  }
}

// ---- z-, q-, u-update of a hidden layer, fused ----------------------------------------------------
// a = W+ p+ + b+ = (r - shift) + z.  z+ by the ReLU closed form of Eq. "update z" (better of the two
// half-line minimisers; a tie keeps the non-positive one; slope > 0: leaky ReLU f(x) = slope x for x <= 0, whose
// minimiser on z <= 0 is (a + slope q + z)/(2 + slope^2)), q+ by Eq. "update q" (q_top >= 0: projected onto
// the level set of p_{l+1}, the variant at the end of Sec. "Quantization Extension"), residual p_{l+1} - q+,
// u+ by Eq. "update u", the linear residual of the next iteration r = a - z+, and t_{l+1} = u+ + rho (p_{l+1} - q+),
// the part of the next p-gradient that does not involve a product.
__global__ void __launch_bounds__(EW_THREADS)
zqu_kernel(float *__restrict__ r, float *__restrict__ z, float *__restrict__ q, float *__restrict__ u,
           const float *__restrict__ p_next, const float *__restrict__ shift, int ld4cols, size_t n4,
           float rho, float nu, float slope, float q_scale, float q_lo, float q_top, float *__restrict__ t_next,
           double *__restrict__ slots, uint32_t *__restrict__ amax_r /* max|r| (see commit_amax); may be null */,
           const void *__restrict__ codes_next = nullptr /* pdADMM-G-Q: codes of p_next, read instead of it */, int wide_codes = 0) {
  __shared__ double red[EW_THREADS / 32];
  const float inv_rn = 1.0f / (rho + nu), inv_neg = 1.0f / (2.0f + slope * slope);
  double ss = 0.0;
  uint32_t mr = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 sh = ld4(shift, i % ld4cols);
    const float4 rv = ld4(r, i), zv = ld4(z, i), qv = ld4(q, i), uv = ld4(u, i);
    const float4 pv = codes_next != nullptr ? levels_of4(codes_next, wide_codes, i, q_scale, q_lo) : ld4(p_next, i);
    float4 zn, qn, un, rn, tn;
#define PD_ZQU(f)                                                                   \
    {                                                                               \
      const float a = (rv.f - sh.f) + zv.f;                                         \
      const float zneg = fminf((fmaf(slope, qv.f, a) + zv.f) * inv_neg, 0.0f);      \
      const float zpos = fmaxf((a + qv.f + zv.f) * (1.0f / 3.0f), 0.0f);            \
      const float qneg = qv.f - slope * zneg;                                       \
      const float fneg = (zneg - a) * (zneg - a) + qneg * qneg + (zneg - zv.f) * (zneg - zv.f); \
      const float fpos = (zpos - a) * (zpos - a) + (qv.f - zpos) * (qv.f - zpos) + (zpos - zv.f) * (zpos - zv.f); \
      const float zz = fpos < fneg ? zpos : zneg;                                   \
      float qq = (rho * pv.f + uv.f + nu * (zz > 0.0f ? zz : slope * zz)) * inv_rn; \
      if (q_top >= 0.0f) { unsigned code; qq = quantize_one(qq, q_scale, q_lo, q_top, code); } \
      const float res = pv.f - qq;                                                  \
      zn.f = zz; qn.f = qq; un.f = fmaf(rho, res, uv.f); rn.f = a - zz;             \
      tn.f = fmaf(rho, res, un.f);                                                  \
      ss += (double)res * res;                                                      \
    }
    PD_ZQU(x) PD_ZQU(y) PD_ZQU(z) PD_ZQU(w)
#undef PD_ZQU
    st4(z, i, zn); st4(q, i, qn); st4(u, i, un); st4(r, i, rn); st4(t_next, i, tn);
    mr = max(mr, abs_bits(rn));
  }
  if (amax_r != nullptr) commit_amax(mr, amax_r);
  const double tot = block_sum<EW_THREADS>(ss, red);
  if (threadIdx.x == 0) slots[blockIdx.x] = tot;
}

// ---- the same for a smooth activation: z-update by lookup table ---------------------------------------------
// f = tanh or sigmoid has no closed-form z-update; the paper recommends a lookup table (remark after Eq. "update z").
// The table holds T equally spaced candidates z_i = lo + i h with f(z_i); z+ is the candidate with the smallest
// (z - a)^2 + (q - f(z))^2 + (z - z^k)^2 (the first one if equal), element by element.  q, u, r, t as in zqu_kernel.
// Dynamic shared memory: 2 T floats.
__global__ void __launch_bounds__(EW_THREADS)
zqu_table_kernel(float *__restrict__ r, float *__restrict__ z, float *__restrict__ q, float *__restrict__ u,
                 const float *__restrict__ p_next, const float *__restrict__ shift, int ld4cols, size_t n4,
                 float rho, float nu, float act, float t_lo, float t_step, int T, float q_scale, float q_lo, float q_top,
                 float *__restrict__ t_next, double *__restrict__ slots, uint32_t *__restrict__ amax_r,
                 const void *__restrict__ codes_next = nullptr, int wide_codes = 0) {
  extern __shared__ float table_sh[];              // z_i, then f(z_i)
  __shared__ double red[EW_THREADS / 32];
  for (int i = threadIdx.x; i < T; i += blockDim.x) {
    const float zi = __fadd_rn(t_lo, __fmul_rn((float)i, t_step));
    table_sh[i] = zi;
    table_sh[T + i] = act_eval(zi, act);
  }
  __syncthreads();
  const float inv_rn = 1.0f / (rho + nu);
  double ss = 0.0;
  uint32_t mr = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 sh = ld4(shift, i % ld4cols);
    const float4 rv = ld4(r, i), zv = ld4(z, i), qv = ld4(q, i), uv = ld4(u, i);
    const float4 pv = codes_next != nullptr ? levels_of4(codes_next, wide_codes, i, q_scale, q_lo) : ld4(p_next, i);
    const float a[4] = {(rv.x - sh.x) + zv.x, (rv.y - sh.y) + zv.y, (rv.z - sh.z) + zv.z, (rv.w - sh.w) + zv.w};
    const float zo[4] = {zv.x, zv.y, zv.z, zv.w}, qo[4] = {qv.x, qv.y, qv.z, qv.w};
    float best[4] = {3.0e38f, 3.0e38f, 3.0e38f, 3.0e38f}, zb[4] = {0.f, 0.f, 0.f, 0.f}, fb[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k = 0; k < T; ++k) {
      const float zi = table_sh[k], fi = table_sh[T + k];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float d0 = zi - a[e], d1 = qo[e] - fi, d2 = zi - zo[e];
        const float h = fmaf(d0, d0, fmaf(d1, d1, d2 * d2));
        if (h < best[e]) { best[e] = h; zb[e] = zi; fb[e] = fi; }
      }
    }
    const float pn[4] = {pv.x, pv.y, pv.z, pv.w}, uo[4] = {uv.x, uv.y, uv.z, uv.w};
    float zn[4], qn[4], un[4], rn[4], tn[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float qq = (rho * pn[e] + uo[e] + nu * fb[e]) * inv_rn;
      if (q_top >= 0.0f) { unsigned code; qq = quantize_one(qq, q_scale, q_lo, q_top, code); }
      const float res = pn[e] - qq;
      zn[e] = zb[e]; qn[e] = qq; un[e] = fmaf(rho, res, uo[e]); rn[e] = a[e] - zb[e];
      tn[e] = fmaf(rho, res, un[e]);
      ss += (double)res * res;
    }
    st4(z, i, make_float4(zn[0], zn[1], zn[2], zn[3])); st4(q, i, make_float4(qn[0], qn[1], qn[2], qn[3]));
    st4(u, i, make_float4(un[0], un[1], un[2], un[3]));
    const float4 r4 = make_float4(rn[0], rn[1], rn[2], rn[3]);
    st4(r, i, r4); st4(t_next, i, make_float4(tn[0], tn[1], tn[2], tn[3]));
    mr = max(mr, abs_bits(r4));
  }
  if (amax_r != nullptr) commit_amax(mr, amax_r);
  const double tot = block_sum<EW_THREADS>(ss, red);
  if (threadIdx.x == 0) slots[blockIdx.x] = tot;
}

// ---- z-update of the last layer -------------------------------------------------------------------
// One thread per node.  a = (r - shift) + z.  Labelled node: z+ = argmin CE(z; y) + (nu/2)||z - a||^2
// (Eq. "update zl"), the unique root of softmax(z) - e_y + nu (z - a) = 0, by damped Newton with the
// Hessian diag(s) + nu I - s s^T inverted through the rank-one update formula; double precision
// inside, since nu is small and the Hessian is close to singular along (1,..,1).  Unlabelled: z+ = a.
constexpr int ZL_MAX_C = 64;
__global__ void __launch_bounds__(128)
zlast_kernel(float *__restrict__ r, float *__restrict__ z, const float *__restrict__ shift,
             const int *__restrict__ labels, const uint8_t *__restrict__ mask, int n_rows, int C, int ld,
             double nu, int *__restrict__ not_converged, uint32_t *__restrict__ amax_r /* max|r|, may be null */,
             int least_squares /* R = 1/2 ||z - e_y||^2: z+ = (e_y + nu a)/(1 + nu) */) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_rows) return;
  float *rj = r + (size_t)j * ld, *zj = z + (size_t)j * ld;
  double a[ZL_MAX_C], x[ZL_MAX_C], s[ZL_MAX_C], st[ZL_MAX_C];
  for (int c = 0; c < C; ++c) { a[c] = (double)((rj[c] - shift[c]) + zj[c]); x[c] = a[c]; }
  if (mask[j] && least_squares) {
    const int y = labels[j];
    for (int c = 0; c < C; ++c) x[c] = ((c == y ? 1.0 : 0.0) + nu * a[c]) / (1.0 + nu);
  } else if (mask[j]) {
    const int y = labels[j];
    auto fval = [&](const double *v) {
      double m = v[0];
      for (int c = 1; c < C; ++c) m = fmax(m, v[c]);
      double se = 0.0, sq = 0.0;
      for (int c = 0; c < C; ++c) { se += exp(v[c] - m); sq += (v[c] - a[c]) * (v[c] - a[c]); }
      return m + log(se) - v[y] + 0.5 * nu * sq;
    };
    double fx = fval(x);
    bool done = false;
    for (int it = 0; it < 100 && !done; ++it) {
      double m = x[0];
      for (int c = 1; c < C; ++c) m = fmax(m, x[c]);
      double se = 0.0;
      for (int c = 0; c < C; ++c) { s[c] = exp(x[c] - m); se += s[c]; }
      double gmax = 0.0, s_mg = 0.0, s_ms = 0.0;
      for (int c = 0; c < C; ++c) {
        s[c] /= se;
        const double g = s[c] - (c == y ? 1.0 : 0.0) + nu * (x[c] - a[c]);
        gmax = fmax(gmax, fabs(g));
        const double mi = 1.0 / (s[c] + nu);
        st[c] = g;                       // gradient for now
        s_mg += s[c] * mi * g;
        s_ms += s[c] * mi * s[c];
      }
      if (gmax <= 1e-10) { done = true; break; }
      const double k = s_mg / (1.0 - s_ms);
      double slope = 0.0;
      for (int c = 0; c < C; ++c) {
        const double mi = 1.0 / (s[c] + nu);
        const double g = st[c];
        const double d = -(mi * g + mi * s[c] * k);
        slope += g * d;
        st[c] = d;                       // Newton step
      }
      const bool resolvable = -slope > 1e-9 * (1.0 + fabs(fx));
      double t = 1.0, ft;
      for (;;) {
        for (int c = 0; c < C; ++c) s[c] = x[c] + t * st[c];
        ft = fval(s);
        if (!resolvable || ft <= fx + 1e-4 * t * slope || t < 1e-12) break;
        t *= 0.5;
      }
      for (int c = 0; c < C; ++c) x[c] = s[c];
      fx = ft;
    }
    if (!done) atomicAdd(not_converged, 1);
  }
  uint32_t mr = 0u;
  for (int c = 0; c < C; ++c) {
    const float zn = (float)x[c];
    zj[c] = zn;
    const float rn = (float)(a[c] - (double)zn);
    rj[c] = rn;
    mr = max(mr, abs_bits(rn));
  }
  if (amax_r != nullptr) commit_amax(mr, amax_r);
}

// t = u + rho (p - q) from the stored iterates (after the start or after the caller has set a tensor); the same
// operations as in zqu_kernel, so both give the same bits.
__global__ void __launch_bounds__(EW_THREADS)
gradp_const_kernel(const float *__restrict__ u, const float *__restrict__ p, const float *__restrict__ q, float rho,
                   float *__restrict__ t, size_t n4) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 uv = ld4(u, i), pv = ld4(p, i), qv = ld4(q, i);
    float4 tv;
    tv.x = fmaf(rho, pv.x - qv.x, uv.x); tv.y = fmaf(rho, pv.y - qv.y, uv.y);
    tv.z = fmaf(rho, pv.z - qv.z, uv.z); tv.w = fmaf(rho, pv.w - qv.w, uv.w);
    st4(t, i, tv);
  }
}

// ---- elementwise helpers of the initial forward pass ---------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
relu_max_kernel(const float *__restrict__ z, float *__restrict__ q, size_t n4, float slope, float *__restrict__ block_max) {
  __shared__ float red[EW_THREADS / 32];
  float m = 0.0f;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 v = ld4(z, i);
    v.x = act_eval(v.x, slope); v.y = act_eval(v.y, slope); v.z = act_eval(v.z, slope); v.w = act_eval(v.w, slope);
    m = fmaxf(m, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
    st4(q, i, v);
  }
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < EW_THREADS / 32; ++i) m = fmaxf(m, red[i]);
    block_max[blockIdx.x] = m;
  }
}

// ---- objective pieces of one layer ---------------------------------------------------------------
// slots[b][0..3] = sum r^2, sum (q - relu z)^2, sum u (p_next - q), sum (p_next - q)^2 ; q == nullptr: only r^2.
__global__ void __launch_bounds__(EW_THREADS)
objective_layer_kernel(const float *__restrict__ r, const float *__restrict__ z, const float *__restrict__ q,
                       const float *__restrict__ u, const float *__restrict__ p_next, size_t n, float slope,
                       double *__restrict__ slots) {
  __shared__ double red[EW_THREADS / 32];
  double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const double rv = r[i];
    s0 += rv * rv;
    if (q != nullptr) {
      const float zv = z[i];
      const double qv = q[i], act = act_eval(zv, slope), res = (double)p_next[i] - qv;
      s1 += (qv - act) * (qv - act);
      s2 += (double)u[i] * res;
      s3 += res * res;
    }
  }
  double t;
  t = block_sum<EW_THREADS>(s0, red); if (threadIdx.x == 0) slots[blockIdx.x * 4 + 0] = t;
  t = block_sum<EW_THREADS>(s1, red); if (threadIdx.x == 0) slots[blockIdx.x * 4 + 1] = t;
  t = block_sum<EW_THREADS>(s2, red); if (threadIdx.x == 0) slots[blockIdx.x * 4 + 2] = t;
  t = block_sum<EW_THREADS>(s3, red); if (threadIdx.x == 0) slots[blockIdx.x * 4 + 3] = t;
}

// R(z_L; y): sum over masked nodes of -z_y + logsumexp(z), or of 1/2 ||z - e_y||^2 (least_squares).
// One thread per node, one slot per block.
__global__ void __launch_bounds__(EW_THREADS)
risk_kernel(const float *__restrict__ z, const int *__restrict__ labels, const uint8_t *__restrict__ mask,
            int n_rows, int C, int ld, double *__restrict__ slots, int least_squares) {
  __shared__ double red[EW_THREADS / 32];
  double acc = 0.0;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n_rows; j += gridDim.x * blockDim.x) {
    if (!mask[j]) continue;
    const float *zj = z + (size_t)j * ld;
    if (least_squares) {
      double sq = 0.0;
      for (int c = 0; c < C; ++c) {
        const double d = (double)zj[c] - (c == labels[j] ? 1.0 : 0.0);
        sq += d * d;
      }
      acc += 0.5 * sq;
      continue;
    }
    double m = zj[0];
    for (int c = 1; c < C; ++c) m = fmax(m, (double)zj[c]);
    double se = 0.0;
    for (int c = 0; c < C; ++c) se += exp((double)zj[c] - m);
    acc += m + log(se) - (double)zj[labels[j]];
  }
  const double t = block_sum<EW_THREADS>(acc, red);
  if (threadIdx.x == 0) slots[blockIdx.x] = t;
}

// Predicted class of every node: the largest of its C logits, the first one among equals.  counts[0..3] (zeroed
// by the caller) receive: correct and total over the nodes with mask = 1, correct and total over the others.
__global__ void __launch_bounds__(EW_THREADS)
argmax_kernel(const float *__restrict__ z, const int *__restrict__ labels, const uint8_t *__restrict__ mask, int n_rows,
              int C, int ld, int *__restrict__ pred, unsigned long long *__restrict__ counts) {
  unsigned long long c_in = 0, n_in = 0, c_out = 0, n_out = 0;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n_rows; j += gridDim.x * blockDim.x) {
    const float *zj = z + (size_t)j * ld;
    int best = 0;
    float vbest = zj[0];
    for (int c = 1; c < C; ++c) {
      const float v = zj[c];
      if (v > vbest) { vbest = v; best = c; }
    }
    pred[j] = best;
    const bool hit = best == labels[j];
    if (mask[j]) { ++n_in; c_in += hit; } else { ++n_out; c_out += hit; }
  }
  // integer sums: the order of the atomics does not matter
  c_in = warp_sum_u64(c_in); n_in = warp_sum_u64(n_in); c_out = warp_sum_u64(c_out); n_out = warp_sum_u64(n_out);
  if ((threadIdx.x & 31) == 0) {
    if (n_in) { atomicAdd(counts + 0, c_in); atomicAdd(counts + 1, n_in); }
    if (n_out) { atomicAdd(counts + 2, c_out); atomicAdd(counts + 3, n_out); }
  }
}

// W+ = W - grad_W * inv_theta  (Eq. "update W")
__global__ void __launch_bounds__(EW_THREADS)
wstep_kernel(float *__restrict__ W, const float *__restrict__ G, const LayerScalars *__restrict__ sc, size_t n4,
             uint32_t *__restrict__ amax) {
  const float a = sc->inv_theta;
  uint32_t m = 0u;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 v = ld4(W, i);
    const float4 g = ld4(G, i);
    v.x = fmaf(-a, g.x, v.x); v.y = fmaf(-a, g.y, v.y); v.z = fmaf(-a, g.z, v.z); v.w = fmaf(-a, g.w, v.w);
    st4(W, i, v);
    m = max(m, abs_bits(v));
  }
  if (amax != nullptr) commit_amax(m, amax);        // max|W+| for the fp16 planes of the tensor-core products
}

}  // namespace pd
