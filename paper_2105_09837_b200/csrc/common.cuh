// Shared host/device helpers of the pdADMM library: status codes, error text, reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdarg.h>
#include <stdint.h>
#include <stdio.h>
#include <string>

#include "../../include/pdadmm.h"

namespace pd {

// ---- thread-local error text ------------------------------------------------------------------
inline std::string &err_text() {
  static thread_local std::string s;
  return s;
}
inline int fail(int code, const char *fmt, ...) __attribute__((format(printf, 2, 3)));
inline int fail(int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  err_text() = buf;
  return code;
}

#define PD_CUDA(expr)                                                                             \
  do {                                                                                            \
    cudaError_t e__ = (expr);                                                                     \
    if (e__ != cudaSuccess)                                                                       \
      return pd::fail(e__ == cudaErrorMemoryAllocation ? PDADMM_ENOMEM : PDADMM_ECUDA,           \
                      "%s:%d: %s -> %s", __FILE__, __LINE__, #expr, cudaGetErrorString(e__));     \
  } while (0)

#define PD_TRY(expr)            \
  do {                          \
    int rc__ = (expr);          \
    if (rc__ != PDADMM_OK) return rc__; \
  } while (0)

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Exponent e of the scaling 2^e of a matrix whose largest magnitude has the bit pattern `amax_bits`:
// max|x| 2^e lies in [2^14, 2^15), below the fp16 overflow threshold (the operands of the tensor-core products
// are split into fp16 planes).  Zero, subnormal or non-finite maxima
// take e = 0 (a NaN or Inf then travels through the product unchanged); |e| <= 100 so that 2^e is a normal float.
__host__ __device__ __forceinline__ int tc_scale_exp(uint32_t amax_bits) {
  const int E = (int)((amax_bits >> 23) & 0xFFu);
  if (E == 0 || E == 255) return 0;
  const int e = 14 - (E - 127);
  return e < -100 ? -100 : (e > 100 ? 100 : e);
}
// An fp16 copy of a matrix written before its largest magnitude is known takes its exponent from the maximum of the
// previous iteration, two binary orders lower (room for a fourfold growth); TC_NO_PREDICTION if that maximum is no
// normal number.  The copy is usable if the true maximum, scaled, lies in [2^4, 2^15): no overflow and at least 11
// significant bits above the fp16 subnormals for the largest entries (it is used as a hi plane alone).
constexpr int TC_NO_PREDICTION = -1000;
__host__ __device__ __forceinline__ int tc_predict_exp(uint32_t amax_bits) {
  const int E = (int)((amax_bits >> 23) & 0xFFu);
  if (E == 0 || E == 255) return TC_NO_PREDICTION;
  return tc_scale_exp(amax_bits) - 2;
}
__host__ __device__ __forceinline__ bool tc_prediction_usable(uint32_t amax_bits, int predicted) {
  const int E = (int)((amax_bits >> 23) & 0xFFu);
  if (E == 0 || E == 255 || predicted < -100 || predicted > 100) return false;
  const int e = 14 - (E - 127);          // unclamped exponent of the exact scaling
  return predicted <= e && predicted >= e - 10;
}
// ---- largest magnitude of an array, as a bit pattern ---------------------------------------------
// The tensor-core products scale each operand by a power of two chosen from max|x|.  The maximum is kept as the
// bit pattern of |x| in an unsigned word (for non-negative floats the integer order is the float order, a NaN
// sorts above Inf), combined with atomicMax: the result does not depend on the order of the updates.
__device__ __forceinline__ uint32_t abs_bits(float v) { return __float_as_uint(v) & 0x7FFFFFFFu; }
__device__ __forceinline__ uint32_t abs_bits(float4 v) {
  return max(max(abs_bits(v.x), abs_bits(v.y)), max(abs_bits(v.z), abs_bits(v.w)));
}
// called by the threads of a warp that are still running, each with its own maximum: one atomic per warp
__device__ __forceinline__ void commit_amax(uint32_t m, uint32_t *__restrict__ word) {
  const unsigned active = __activemask();
  m = __reduce_max_sync(active, m);
  if ((int)(threadIdx.x & 31) == __ffs(active) - 1 && m != 0u) atomicMax(word, m);
}
// ---- f_l ----------------------------------------------------------------------------------------------------
// The activation travels through the kernels as one float: a value in [0, 1) is ReLU (0) or leaky ReLU with that slope
// for x <= 0; 2 is tanh, 3 the logistic sigmoid (the smooth activations, whose z-update searches a lookup table).
constexpr float ACT_TANH = 2.0f, ACT_SIGMOID = 3.0f;
__device__ __forceinline__ float act_eval(float x, float sel) {
  if (sel < 1.0f) return x > 0.f ? x : sel * x;
  if (sel == ACT_TANH) return tanhf(x);
  return 1.0f / (1.0f + expf(-x));
}

// ---- device reductions -------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Sum of one double per thread over the block; the result is valid in thread 0.
// Warps are combined in index order, so the result does not depend on scheduling.
template <int THREADS>
__device__ __forceinline__ double block_sum(double v, double *smem /* THREADS/32 doubles */) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) smem[w] = v;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < THREADS / 32; ++i) t += smem[i];
  }
  return t;
}

}  // namespace pd
