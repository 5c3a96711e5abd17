// pdADMM-G / pdADMM-G-Q on one B200: context, host orchestration of one iteration, C ABI.
//
// Data layout (device): every N x width matrix is node-major with its leading dimension padded to a
// multiple of 32 floats (128-byte rows) and zero padding columns.  Per layer l the context keeps p_l, z_l, q_l, u_l,
// W_l, b_l and the linear residual r_l = W_l p_l + b_l - z_l, which every step of the iteration
// updates in place instead of recomputing the product:
//     p+ = p - g/tau        =>  r <- r - (W g)/tau            (pdADMM-G-Q: r <- r + W (p+ - p))
//     W+ = W - G/theta      =>  r <- r - (G p+)/theta
//     b+ = b - mean_j r     =>  r <- r - mean_j r
//     z+                    =>  r <- (r + z) - z+
// so one iteration of a layer costs four dense products: W^T r (the p-gradient), W g (tau),
// r^T p+ (the W-gradient, contraction over the nodes) and G p+ (theta).
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <map>
#include <memory>
#include <tuple>
#include <vector>

#include "common.cuh"
#include "elementwise.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "graph.cuh"

namespace pd {

// ---- kernel classes for the per-kernel timing -----------------------------------------------------
enum KClass {
  KC_GEMM_RESID = 0,  // r = P W^T + b - z                    (after init / set_tensor only)
  KC_GEMM_GRADP,      // g = nu r W + u + rho (p - q), ||g||^2
  KC_GEMM_WG,         // W g (or W d), squared norm
  KC_GEMM_GRADW,      // partial tiles of r^T p+ over node slices
  KC_GRADW_REDUCE,    // sum of the partial tiles, nu, ||G||^2
  KC_GEMM_GP,         // G p+, squared norm
  KC_AXPY,            // p -= g/tau ; r -= (Wg)/tau ; r += W d
  KC_QUANT,           // quantised trial step
  KC_COLSUM,          // r -= (G p+)/theta with column sums
  KC_ZQU,             // fused z, q, u update of a hidden layer
  KC_ZLAST,           // z update of the last layer
  KC_WSTEP,           // W -= G/theta
  KC_SMALL,           // single-block finalisers
  KC_AMAX,            // largest magnitude of a product's node-sized operand (for its power-of-two scaling)
  KC_PLANES,          // fp16 planes of a weight-sized operand
  KC_COUNT
};
static const char *kclass_names[KC_COUNT] = {
    "gemm_resid", "gemm_gradp", "gemm_wg", "gemm_gradw", "gradw_reduce", "gemm_gp", "axpy",
    "quant_trial", "resid_colsum", "zqu", "zlast", "wstep", "finalize", "absmax", "make_planes"};

// fp16 hi/lo planes of a weight-sized matrix [rows][cols] for the tensor-core products, in the orientation(s)
// in which it is contracted, and the exponent of the power-of-two scaling they were made with.
struct Planes {
  __half *hi = nullptr, *lo = nullptr;     // [rows][ldh], ldh = cols rounded up to 8
  __half *hiT = nullptr, *loT = nullptr;   // [cols][ldhT], ldhT = rows rounded up to 8 (only where needed)
  int ldh = 0, ldhT = 0;
  int *exp = nullptr;                      // device word
};
// one operand of a tensor-core product as two fp16 planes [n][ld], contiguous along the contraction index
struct PlaneRef { const __half *hi, *lo; int ld; const int *exp; };
// an operand that is `mul` times small integers (a quantised p = code * s, or the difference of two): one fp16 plane
// of the integers [n][ld], no lo plane
struct IntPlane { const __half *plane; int ld; float mul; };

// Rows of every node-major matrix start on a 128-byte boundary (leading dimensions are multiples of 32 floats):
// tile copies and the coalesced stores of the epilogues then move whole 32-byte sectors.
constexpr int LD_ALIGN = 32;
// number of lanes for the concurrency across layers (measured on workload c2: 1 lane 241.8, 2 lanes 273.3 iterations/s)
#ifndef PDADMM_N_LANES
#define PDADMM_N_LANES 2
#endif

struct Layer {
  int n_in = 0, n_out = 0, ld_in = 0, ld_out = 0;
  float *p = nullptr;       // [N][ld_in]  (layer 1: X)
  float *W = nullptr;       // [n_out][ld_in]
  float *b = nullptr;       // [ld_out]
  float *z = nullptr, *r = nullptr;          // [N][ld_out]
  float *q = nullptr, *u = nullptr;          // [N][ld_out], hidden layers only
  float *t = nullptr;       // [N][ld_in], l >= 2: u_{l-1} + rho (p_l - q_{l-1}), the product-free part of grad_p phi
  float *gradW = nullptr;   // [n_out][ld_in]
  Planes Wp;                // fp16 planes of W: [n_out][ldh_in], and of W^T: [n_in][ldh_out] (tensor-core path)
  Planes Gp;                // fp16 planes of grad_W: [n_out][ldh_in]
  __half *xT_hi = nullptr, *xT_lo = nullptr;   // layer 1 only: transposed planes of p_1 = X, which never changes
  int *xT_exp = nullptr;
  __half *x_hi = nullptr, *x_lo = nullptr;     // layer 1 only: planes of X in its own orientation [N][ld_in]
  int *x_exp = nullptr;
  int *g_exp = nullptr;     // l >= 2: exponent predicted for the scaling of the next fp16 copy of g_l (tc_predict_exp)
  float *shift = nullptr;   // [ld_out] column means removed by the b-update
  uint8_t *codes = nullptr; // [N][ld_in] codes of 1 byte (up to 256 levels) or 2 bytes, quantised mode, l >= 2
  __half *p_plane = nullptr; // [N][ld_in] the codes as fp16 integers: operand plane of p_l = code * scale (see int_operands)
  float scale = 1.0f;       // level spacing s_l of p_l
  float lo = 0.0f;          // smallest level of p_l: -(levels below zero) * s_l
  LayerScalars *sc = nullptr;
  // Largest magnitudes (bit patterns) of the two node-sized operands of this layer's products, kept by the kernels
  // that write them: amax_p covers every p_l written since the last tau of the layer, amax_r every r_l written
  // since its last theta -- upper bounds of the current maxima, which is all the power-of-two scaling needs.
  uint32_t *amax_p = nullptr, *amax_r = nullptr;
  int n_split = 1, k_chunk = 0;
};

struct Scratch {
  cudaStream_t st = nullptr;
  float *s1 = nullptr;      // g, later G p+
  float *s2 = nullptr;      // W g, later W d
  float *p_new = nullptr;   // quantised trial
  float *d = nullptr;       // quantised trial
  uint8_t *codes_new = nullptr;
  __half *pn_plane = nullptr, *d_plane = nullptr;   // planes of the trial's codes and of their change (see int_operands)
  float *part = nullptr;    // partial tiles of grad_W
  double *slots = nullptr;  // per-block partial sums
  size_t n_slots = 0;
  double *red = nullptr;    // sums on their way through the reduction over shards (widest layer + 8 values)
  float *tail_ws = nullptr; // accumulators of the contraction slices of tail tiles (one tile per SM at most)
  int *tail_count = nullptr;
  uint32_t *amax_pool = nullptr;   // words for the largest magnitudes of product operands, handed out in stream order
  int amax_next = 0;
  // transposed fp16 planes ([width][ldT], node index contiguous) of r_l and p_l for the product over the nodes
  __half *rT_hi = nullptr, *rT_lo = nullptr, *pT_hi = nullptr, *pT_lo = nullptr;
  int *rT_exp = nullptr, *pT_exp = nullptr;
  // planes [N][ld] of the streamed operand of a product over several column tiles (split once per product)
  __half *a_hi = nullptr, *a_lo = nullptr;
  size_t a_cap = 0;                // elements each of the two holds
  int *a_exp = nullptr;
  // quantised mode: fp16 copy [N][ld] of g, written by the epilogue of the p-gradient's product with a predicted
  // scaling, for the norm-only product W g that follows (rows_planes_kernel)
  __half *g_hi = nullptr;
  int *g_hi_exp = nullptr;
  int *h_flag = nullptr;           // pinned word that receives the accept flag of the lane's quantised trial
  cudaEvent_t ev_flag = nullptr;   // recorded after the copy of that flag
};

struct ProfRec { int cls; cudaEvent_t e0, e1; double bytes, flops; };

}  // namespace pd

struct pdadmm_ctx {
  int device = 0;
  int64_t N = 0;                   // nodes this context owns
  int64_t N_total = 0, node_begin = 0;   // the whole graph; first owned node
  pdadmm_allreduce_fn reduce = nullptr;  // adds over the shards' contexts (null: this context holds every node)
  void *reduce_user = nullptr;
  int64_t comm_bytes = 0;
  int L = 0, d = 0, n_blocks = 0, n0 = 0, ld0 = 0, C = 0, levels = 0;
  int code_bytes = 1;              // 1 for up to 256 levels, else 2
  int neg_levels = 0;              // levels below zero
  float fixed_step = 0.f;          // > 0: the same level spacing for every layer
  bool quant_q = false;            // q_l is kept on the level set of p_{l+1} as well
  float slope = 0.f;               // f_l (see act_eval): [0, 1) = (leaky) ReLU with that slope for x <= 0, 2 = tanh, 3 = sigmoid
  float table_lo = 0.f, table_step = 0.f;   // lookup table of the z-update of a smooth activation: z_i = lo + i step
  int table_size = 0;
  bool ls_risk = false;            // R = least squares instead of cross-entropy
  float rho = 0, nu = 0;
  uint32_t flags = 0;
  int64_t nnz = 0;
  int *row_ptr = nullptr, *col_idx = nullptr;
  float *csr_val = nullptr;
  int *labels = nullptr;
  uint8_t *mask = nullptr;
  std::vector<pd::Layer> layers;
  pd::Scratch scr;                  // lane 0: the context's main stream and its scratch
  // Layer concurrency: the updates of different layers are independent inside each phase of an iteration, so
  // layer l's chain of kernels is queued on lane l mod n_lanes.  Every lane has its own stream and its own scratch
  // (product outputs, partial tiles, reduction slots), so that chains of different layers can overlap: the next
  // product starts on the SMs that the previous one has already left, and bandwidth-bound kernels run beside
  // tensor-bound ones.  `cur` is the lane that the host code is queueing on.
  std::vector<std::unique_ptr<pd::Scratch>> more_lanes;
  pd::Scratch *cur = &scr;
  std::vector<cudaEvent_t> ev_p;    // [L]: p_l of this iteration is complete
  std::vector<cudaEvent_t> ev_lane; // [n_lanes]: fork / join
  bool r_valid = false;
  bool t_valid = false;             // every layer's t matches the stored u, p, q
  int *d_flag = nullptr;            // device counter (z_L solver non-convergence)
  int *h_pinned = nullptr;          // pinned host words for small read-backs
  int64_t launches = 0;
  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
  double last_step_ms = 0.0;
  bool profiling = false;
  std::vector<pd::ProfRec> prof;
  std::vector<cudaEvent_t> ev_pool;
  double prof_ms[pd::KC_COUNT] = {0}, prof_bytes[pd::KC_COUNT] = {0}, prof_flops[pd::KC_COUNT] = {0};
  int64_t prof_n[pd::KC_COUNT] = {0};
  std::vector<void *> allocs;       // driver allocations: chunks and large arrays
  size_t bytes_handed_out = 0;      // device bytes handed out by dev_alloc so far
  char *arena_base = nullptr;       // current chunk
  size_t arena_cap = 0, arena_used = 0, arena_next = size_t(64) << 20;
  bool use_tc = true;               // dense products on the tensor cores
  // pdADMM-G-Q with at most 2048 levels starting at zero: p_l = code * s_l exactly, and the codes are exact in fp16, so
  // the products whose operand is p_l (or d = p+ - p) take one plane of integers instead of a hi and a lo plane of
  // the values: two MMAs per product instead of three, a quarter of the operand bytes, no split pass
  bool int_operands = false;
  cudaGraphExec_t iter_graph = nullptr;   // one captured pdADMM-G iteration (no host round trips in it)
  int64_t iter_graph_launches = 0;
  bool graph_failed = false;
  int n_sms = 148;
  bool w_planes_valid = false;
  bool amax_p_valid = false;        // every layer's amax_p covers the stored p
  bool xT_valid = false;            // the transposed planes of X match the stored X
  int ldT = 0;                      // leading dimension of transposed planes: N rounded up to 8
  std::map<std::tuple<const void *, uint64_t, uint64_t, uint64_t, uint32_t, uint32_t>, CUtensorMap> tmaps;
};

namespace pd {

// ---- allocation bookkeeping -------------------------------------------------------------------------
// Device memory of a context.  Arrays of up to 64 MB are carved out of chunks (64 MB at first, doubling up to
// 1 GB), 256-byte aligned: a context has some twenty arrays per layer, and one driver allocation each made
// pdadmm_init spend most of its time in the allocator.  Larger arrays get an allocation of their own, so that
// a chunk never wastes more than one small array at its end.  Everything is released by destroy().
constexpr size_t ARENA_MAX_ARRAY = size_t(64) << 20, ARENA_MAX_CHUNK = size_t(1) << 30;   // first chunk: arena_next
template <class T>
static int dev_alloc(pdadmm_ctx *c, T **ptr, size_t count, bool zero = true) {
  // slack: operand copies may read up to 31 floats past a matrix
  const size_t bytes = (count * sizeof(T) + 256 + 255) & ~size_t(255);
  char *p = nullptr;
  if (bytes <= ARENA_MAX_ARRAY && c->arena_used + bytes <= c->arena_cap) {
    p = c->arena_base + c->arena_used;
    c->arena_used += bytes;
  } else {
    const bool chunk = bytes <= ARENA_MAX_ARRAY;
    const size_t want = chunk ? std::max(bytes, c->arena_next) : bytes;
    void *q = nullptr;
    const cudaError_t e = cudaMalloc(&q, want);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return fail(PDADMM_ENOMEM, "cudaMalloc of %zu bytes failed: %s", want, cudaGetErrorString(e));
    }
    c->allocs.push_back(q);
    p = (char *)q;
    if (chunk) {
      c->arena_base = p; c->arena_cap = want; c->arena_used = bytes;
      c->arena_next = std::min(ARENA_MAX_CHUNK, 2 * want);
    }
  }
  if (zero) PD_CUDA(cudaMemsetAsync(p, 0, bytes, c->scr.st));   // same stream as every kernel that uses it
  c->bytes_handed_out += bytes;
  *ptr = (T *)p;
  return PDADMM_OK;
}

static inline int ew_grid(size_t n_items) {
  return (int)std::max<size_t>(1, std::min<size_t>(ceil_div((int64_t)n_items, EW_THREADS), 148 * 8));
}

// ---- sums over the shards' contexts ---------------------------------------------------------------------------
static int shard_sum(pdadmm_ctx *c, cudaStream_t st, void *buf, size_t count, int is_double, int op = 0) {
  if (c->reduce == nullptr) return PDADMM_OK;
  c->comm_bytes += (int64_t)(count * (is_double ? 8 : 4));
  const int rc = c->reduce(c->reduce_user, buf, count, is_double, op, (void *)st);
  if (rc != 0) return fail(PDADMM_ECUDA, "the reduction callback returned %d", rc);
  return PDADMM_OK;
}
// fixed-order totals of up to two slot arrays into red[0], red[1], then their sum over the shards
static int shard_sum_slots(pdadmm_ctx *c, cudaStream_t st, double *red, const double *a, int na, const double *b, int nb) {
  reduce_slots_kernel<<<1, 256, 0, st>>>(a, na, 1, 1, red);
  if (b != nullptr) reduce_slots_kernel<<<1, 256, 0, st>>>(b, nb, 1, 1, red + 1);
  return shard_sum(c, st, red, b != nullptr ? 2 : 1, 1);
}

// ---- profiling hooks ----------------------------------------------------------------------------------
static cudaEvent_t take_event(pdadmm_ctx *c) {
  cudaEvent_t e;
  if (!c->ev_pool.empty()) { e = c->ev_pool.back(); c->ev_pool.pop_back(); return e; }
  cudaEventCreate(&e);
  return e;
}
struct Launch {                    // brackets one kernel launch
  pdadmm_ctx *c; int cls; cudaStream_t st; double bytes, flops; cudaEvent_t e0 = nullptr;
  Launch(pdadmm_ctx *c_, int cls_, cudaStream_t st_, double bytes_, double flops_)
      : c(c_), cls(cls_), st(st_), bytes(bytes_), flops(flops_) {
    c->launches++;
    if (c->profiling) { e0 = take_event(c); cudaEventRecord(e0, st); }
  }
  ~Launch() {
    if (c->profiling) {
      cudaEvent_t e1 = take_event(c);
      cudaEventRecord(e1, st);
      c->prof.push_back({cls, e0, e1, bytes, flops});
    }
  }
};
static int prof_collect(pdadmm_ctx *c) {
  if (c->prof.empty()) return PDADMM_OK;
  PD_CUDA(cudaDeviceSynchronize());
  for (auto &r : c->prof) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, r.e0, r.e1);
    c->prof_ms[r.cls] += ms; c->prof_n[r.cls]++; c->prof_bytes[r.cls] += r.bytes; c->prof_flops[r.cls] += r.flops;
    c->ev_pool.push_back(r.e0); c->ev_pool.push_back(r.e1);
  }
  c->prof.clear();
  return PDADMM_OK;
}

// ---- tensor maps -------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}
// Operand tiles of the tensor-core products; elements outside the matrix read as zero.
//   TM_RAW_K:  fp32 [outer][inner], tile = box of 32 floats x 128 rows, 128-byte swizzle (the contraction index is the
//              inner one; a 64-deep K block is two such boxes)
//   TM_RAW_MN: fp32 [outer][inner], tile = 128 floats x 64 rows, no swizzle (the contraction index is the outer one;
//              only the converter warps read it)
//   TM_PLANE:  fp16 [outer][inner], tile = 64 halves x 128 rows, 128-byte swizzle (what the MMA reads)
enum TmapKind { TM_RAW_K = 0, TM_RAW_MN = 1, TM_PLANE = 2 };
static int get_tmap(pdadmm_ctx *c, const void *base, uint64_t inner, uint64_t outer, uint64_t ld, TmapKind kind,
                    CUtensorMap *out) {
  auto key = std::make_tuple(base, inner, outer, ld, (uint32_t)kind, 0u);
  auto it = c->tmaps.find(key);
  if (it != c->tmaps.end()) { *out = it->second; return PDADMM_OK; }
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return fail(PDADMM_ECUDA, "cuTensorMapEncodeTiled is not available in this driver");
  const uint64_t esize = kind == TM_PLANE ? 2 : 4;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * esize};
  cuuint32_t box[2] = {kind == TM_RAW_K ? 32u : (kind == TM_RAW_MN ? 128u : 64u), kind == TM_RAW_MN ? 64u : 128u};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  const CUresult r = fn(&m, kind == TM_PLANE ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                        const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        kind == TM_RAW_MN ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(PDADMM_ECUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  if (c->tmaps.size() > 4096) c->tmaps.clear();
  c->tmaps[key] = m;
  *out = m;
  return PDADMM_OK;
}

template <int MODE, class Epi, int ZERO = 0>
static int launch_tc(pdadmm_ctx *c, cudaStream_t st, const CUtensorMap &ma, const CUtensorMap &mal, const CUtensorMap &mb,
                     const CUtensorMap &mbl, const TcParams &prm, const Epi &epi, double *partials, int n_tiles) {
  auto kern = gemm_tc_kernel<MODE, Epi, ZERO>;
  const dim3 grid((unsigned)std::min(n_tiles, c->n_sms));
  // the attribute belongs to (kernel, device): one flag per device ordinal for this instantiation
  static bool configured[64] = {false};
  const int dev = c->device;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    // The kernel's warpgroups re-divide the registers the block is launched with; their shares were added up
    // against TC_REGS_LAUNCH per thread.  A build that launches with fewer would make an increase wait for ever:
    // refuse to launch it.
    cudaFuncAttributes attr;
    PD_CUDA(cudaFuncGetAttributes(&attr, kern));
    if (attr.numRegs != TC_REGS_LAUNCH)
      return fail(PDADMM_ECUDA, "tensor-core product kernel was built with %d registers per thread, %d expected",
                  attr.numRegs, TC_REGS_LAUNCH);
    PD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  kern<<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(ma, mal, mb, mbl, prm, epi, partials);
  return PDADMM_OK;
}

// ---- largest magnitudes of product operands ------------------------------------------------------------------
// Each tensor-core product scales its operands by powers of two taken from their largest magnitudes.  The words
// that receive them come from a pool that is cleared in stream order: at the start of every iteration (so that a
// captured iteration always uses the same words) and whenever it runs out.
constexpr int AMAX_POOL = 4096;
static int amax_reset(pdadmm_ctx *c, cudaStream_t st) {
  PD_CUDA(cudaMemsetAsync(c->cur->amax_pool, 0, AMAX_POOL * sizeof(uint32_t), st));
  c->cur->amax_next = 0;
  return PDADMM_OK;
}
// room for n more words that must stay valid together
static int amax_reserve(pdadmm_ctx *c, cudaStream_t st, int n) {
  if (c->cur->amax_next + n > AMAX_POOL) PD_TRY(amax_reset(c, st));
  return PDADMM_OK;
}
static uint32_t *amax_take(pdadmm_ctx *c) { return c->cur->amax_pool + c->cur->amax_next++; }
// max|x| of a matrix stored as n4 float4 values -> a fresh word
static uint32_t *amax_of(pdadmm_ctx *c, cudaStream_t st, const float *x, size_t n4) {
  uint32_t *w = amax_take(c);
  Launch l(c, KC_AMAX, st, 16.0 * (double)n4, 0);
  absmax_kernel<<<ew_grid(n4), EW_THREADS, 0, st>>>(x, n4, w);
  return w;
}

// fp16 planes of x [rows][ld] (cols valid columns) from the largest magnitude in *amax
static void make_planes(pdadmm_ctx *c, cudaStream_t st, const float *x, int rows, int cols, int ld, const uint32_t *amax,
                        Planes &pl) {
  Launch l(c, KC_PLANES, st, (4.0 + 4.0 + (pl.hiT ? 4.0 : 0.0)) * rows * cols, 0);
  const dim3 grid((unsigned)ceil_div(cols, 32), (unsigned)ceil_div(rows, 32));
  make_planes_kernel<<<grid, dim3(32, 8), 0, st>>>(x, rows, cols, ld, amax, pl.exp, pl.hi, pl.lo, pl.ldh, pl.hiT, pl.loT,
                                                   pl.ldhT);
}
// the same for a matrix whose largest magnitude is not known yet
static int split_planes(pdadmm_ctx *c, cudaStream_t st, const float *x, int rows, int cols, int ld, Planes &pl) {
  if (!c->use_tc) return PDADMM_OK;
  PD_TRY(amax_reserve(c, st, 1));
  const uint32_t *w = amax_of(c, st, x, (size_t)rows * ld / 4);
  make_planes(c, st, x, rows, cols, ld, w, pl);
  return PDADMM_OK;
}
static int alloc_planes(pdadmm_ctx *c, int rows, int cols, bool transposed_too, bool natural, Planes *pl) {
  pl->ldh = round_up(cols, 8); pl->ldhT = round_up(rows, 8);
  if (natural) {
    PD_TRY(dev_alloc(c, &pl->hi, (size_t)rows * pl->ldh));
    PD_TRY(dev_alloc(c, &pl->lo, (size_t)rows * pl->ldh));
  }
  if (transposed_too) {
    PD_TRY(dev_alloc(c, &pl->hiT, (size_t)cols * pl->ldhT));
    PD_TRY(dev_alloc(c, &pl->loT, (size_t)cols * pl->ldhT));
  }
  PD_TRY(dev_alloc(c, &pl->exp, 1));
  return PDADMM_OK;
}

// ---- dense products --------------------------------------------------------------------------------------
// C[M][N] = A[M][K] * op(B), fused epilogue; per-block sums of squares go to `partials` (or nullptr).
// B is given by its fp32 matrix (CUDA-core path; B_NMAJOR tells its orientation) and by its two fp16 planes
// [N][K] (tensor-core path).  `amax_a`: the largest magnitude of A if the caller has it, else it is computed here.
// The streamed operand A is split into its planes tile by tile inside the product, or once beforehand
// (rows_planes_kernel into the lane's scratch, or planes the caller keeps: `Ap`).  Inside, every column tile of the
// output converts the same rows of A again and the converters' tensor-memory stores slow the MMAs down (measured:
// 2640 cycles per 64-deep K block against 1610 with both operands as planes); beforehand costs one pass of
// 8 bytes per element at HBM speed.  Measured per product (split pass included): 4 column tiles 69 against 58 us,
// 8 tiles 1.18 against 1.21 ms, 16 tiles 2.42 against 2.29 ms -- beforehand wins from 16 column tiles on, and
// always where the planes are kept (X).  The norm-only product needs the hi plane alone (6 bytes per element) and
// wins from 8 column tiles on (workload c4: 9.42 -> 9.74 iterations/s).
constexpr int PLANES_FROM_COL_TILES = 16;
template <bool B_NMAJOR, class Epi>
static int gemm_nodes(pdadmm_ctx *c, int cls, cudaStream_t st, int M, int N, int K, const float *A, int lda,
                      const float *B, int ldb, const PlaneRef &Bp, const Epi &epi, double *partials,
                      int *n_partials, double extra_bytes, const uint32_t *amax_a = nullptr,
                      const PlaneRef *Ap = nullptr, const IntPlane *Ai = nullptr) {
  const double bytes = 4.0 * ((double)M * K + (double)N * K + (double)M * N) + extra_bytes;
  if (!c->use_tc) {
    dim3 grid((unsigned)ceil_div(N, SG_BN), (unsigned)ceil_div(M, SG_BM));
    if (n_partials) *n_partials = (int)(grid.x * grid.y);
    Launch l(c, cls, st, bytes, 2.0 * M * N * K);
    gemm_nt_kernel<B_NMAJOR, Epi><<<grid, SG_THREADS, 0, st>>>(M, N, K, A, lda, B, ldb, epi, partials);
    return PDADMM_OK;
  }
  const int n_tiles = (int)(ceil_div(N, TC_BN) * ceil_div(M, TC_BM));
  if (n_partials) *n_partials = 4 * n_tiles;        // one slot per tile and row quarter
  const bool a_int = Ai != nullptr && Ai->plane != nullptr;
  if (amax_a == nullptr && !a_int) {
    PD_TRY(amax_reserve(c, st, 1));
    amax_a = amax_of(c, st, A, (size_t)M * lda / 4);
  }
  PlaneRef a_planes{nullptr, nullptr, 0, nullptr};
  if (a_int) {
    a_planes = PlaneRef{Ai->plane, Ai->plane, Ai->ld, nullptr};
  } else if (Ap != nullptr && Ap->hi != nullptr) {
    a_planes = *Ap;
  } else if (c->cur->a_hi != nullptr && lda % 8 == 0 && (size_t)M * lda <= c->cur->a_cap &&
             (ceil_div(N, TC_BN) >= PLANES_FROM_COL_TILES || (epi_coarse<Epi>::value && ceil_div(N, TC_BN) >= PLANES_FROM_COL_TILES / 2))) {
    Scratch &sc = *c->cur;
    const size_t n8 = (size_t)M * lda / 8;
    constexpr bool coarse = epi_coarse<Epi>::value;
    Launch l(c, KC_PLANES, st, (coarse ? 6.0 : 8.0) * M * K, 0);
    rows_planes_kernel<<<ew_grid(n8), 256, 0, st>>>(A, n8, amax_a, sc.a_exp, sc.a_hi, coarse ? nullptr : sc.a_lo);
    a_planes = PlaneRef{sc.a_hi, sc.a_lo, lda, sc.a_exp};
  }
  const bool pp = a_planes.hi != nullptr;
  CUtensorMap ma, mal, mb, mbl;
  if (pp) {
    PD_TRY(get_tmap(c, a_planes.hi, (uint64_t)K, (uint64_t)M, (uint64_t)a_planes.ld, TM_PLANE, &ma));
    PD_TRY(get_tmap(c, a_planes.lo, (uint64_t)K, (uint64_t)M, (uint64_t)a_planes.ld, TM_PLANE, &mal));
  } else {
    PD_TRY(get_tmap(c, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, TM_RAW_K, &ma));
    mal = ma;
  }
  PD_TRY(get_tmap(c, Bp.hi, (uint64_t)K, (uint64_t)N, (uint64_t)Bp.ld, TM_PLANE, &mb));
  PD_TRY(get_tmap(c, Bp.lo, (uint64_t)K, (uint64_t)N, (uint64_t)Bp.ld, TM_PLANE, &mbl));
  TcParams prm{M, N, K, round_up(K, TC_BK), 1, 0, c->d_flag + 1, pp ? nullptr : amax_a, nullptr, pp ? a_planes.exp : nullptr, Bp.exp};
  // The persistent grid works through the tiles in rounds of n_sms; a last round that fills only part of the
  // SMs costs as much as a full one, so its tiles are cut along the contraction into as many slices as fit.
  int n_units = n_tiles;
  const int tail = n_tiles % c->n_sms, n_kb = (int)ceil_div(K, TC_BK);
  if (tail > 0 && c->cur->tail_ws != nullptr) {
    // at least 8 K blocks per slice: parking and merging the slices of a tile costs about as much as four K blocks,
    // and with two lanes the other layer's kernels fill the SMs that a short last round leaves idle (workload c2,
    // 8 K blocks per tile: 281 iterations/s with 4 slices of 2 blocks, 289 without)
    const int split = std::min(std::min(c->n_sms / tail, n_kb / 8), 8);
    if (split > 1) {
      prm.tail_begin = n_tiles - tail; prm.tail_split = split;
      prm.tail_ws = c->cur->tail_ws; prm.tail_count = c->cur->tail_count;
      n_units = prm.tail_begin + tail * split;
    }
  }
  Launch l(c, cls, st, bytes, 2.0 * M * N * K);
  if constexpr (std::is_same<Epi, EpiStoreSumsq>::value || std::is_same<Epi, EpiAddSumsq>::value) {
    if (a_int) {
      prm.mul = Ai->mul;
      return launch_tc<TC_PLANES, Epi, 1>(c, st, ma, ma, mb, mbl, prm, epi, partials, n_units);
    }
  } else {
    if (a_int) return fail(PDADMM_EINVAL, "no integer-operand form of this product is built");
  }
  if (pp) return launch_tc<TC_PLANES, Epi>(c, st, ma, mal, mb, mbl, prm, epi, partials, n_units);
  return launch_tc<TC_RAW_K, Epi>(c, st, ma, ma, mb, mbl, prm, epi, partials, n_units);
}

// transposed fp16 planes [cols][ldT] of a node-major matrix x [rows][ld] whose largest magnitude is in *amax
static void transpose_planes(pdadmm_ctx *c, cudaStream_t st, const float *x, int rows, int cols, int ld,
                             const uint32_t *amax, __half *hiT, __half *loT, int ldT, int *exp_out) {
  Launch l(c, KC_PLANES, st, 8.0 * rows * cols, 0);
  const int64_t warp_tiles = ceil_div(rows, 32) * ceil_div(cols, 32);
  const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(ceil_div(warp_tiles, 8), 148 * 16));
  transpose_planes_kernel<<<grid, 256, 0, st>>>(x, rows, cols, ld, amax, exp_out, hiT, loT, ldT);
}

// C parts [n_split][M][ldc] = A^T B over node slices, both operands given by their transposed planes:
// A^T = [M][K nodes], B^T = [N][K nodes]
// b_mul > 0: B^T is one plane of integers (Bt.hi; the transposed codes of a quantised p) times b_mul
static int gemm_over_nodes_tc(pdadmm_ctx *c, int cls, cudaStream_t st, int M, int N, int K, const PlaneRef &At,
                              const PlaneRef &Bt, float *part, int ldc, int k_chunk, int n_split, float b_mul = 0.f) {
  const int n_tiles = (int)(ceil_div(N, TC_BN) * ceil_div(M, TC_BM)) * n_split;
  CUtensorMap ma, mal, mb, mbl;
  PD_TRY(get_tmap(c, At.hi, (uint64_t)K, (uint64_t)M, (uint64_t)At.ld, TM_PLANE, &ma));
  PD_TRY(get_tmap(c, At.lo, (uint64_t)K, (uint64_t)M, (uint64_t)At.ld, TM_PLANE, &mal));
  PD_TRY(get_tmap(c, Bt.hi, (uint64_t)K, (uint64_t)N, (uint64_t)Bt.ld, TM_PLANE, &mb));
  if (b_mul > 0.f) mbl = mb;
  else PD_TRY(get_tmap(c, Bt.lo, (uint64_t)K, (uint64_t)N, (uint64_t)Bt.ld, TM_PLANE, &mbl));
  TcParams prm{M, N, K, k_chunk, n_split, (size_t)M * ldc, c->d_flag + 1, nullptr, nullptr, At.exp, b_mul > 0.f ? nullptr : Bt.exp};
  EpiStore epi{part, ldc};
  Launch k(c, cls, st, 4.0 * ((double)K * N + (double)K * M), 2.0 * K * N * M);
  if (b_mul > 0.f) {
    prm.mul = b_mul;
    return launch_tc<TC_PLANES, EpiStore, 2>(c, st, ma, mal, mb, mb, prm, epi, nullptr, n_tiles);
  }
  return launch_tc<TC_PLANES, EpiStore>(c, st, ma, mal, mb, mbl, prm, epi, nullptr, n_tiles);
}

// The same from the fp32 operands themselves, A = [K][lda] (M valid columns), B = [K][ldb] (N valid columns), which
// the product transposes and splits tile by tile; wa, wb: their largest magnitudes.
static int gemm_over_nodes_raw(pdadmm_ctx *c, int cls, cudaStream_t st, int M, int N, int K, const float *A, int lda,
                               const float *B, int ldb, float *part, int ldc, int k_chunk, int n_split,
                               const uint32_t *wa, const uint32_t *wb) {
  const int n_tiles = (int)(ceil_div(N, TC_BN) * ceil_div(M, TC_BM)) * n_split;
  CUtensorMap ma, mb;
  PD_TRY(get_tmap(c, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, TM_RAW_MN, &ma));
  PD_TRY(get_tmap(c, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, TM_RAW_MN, &mb));
  TcParams prm{M, N, K, k_chunk, n_split, (size_t)M * ldc, c->d_flag + 1, wa, wb, nullptr, nullptr};
  EpiStore epi{part, ldc};
  Launch k(c, cls, st, 4.0 * ((double)K * N + (double)K * M), 2.0 * K * N * M);
  return launch_tc<TC_RAW_MN, EpiStore>(c, st, ma, ma, mb, mb, prm, epi, nullptr, n_tiles);
}

// Which form the product over the nodes takes for an M x N output.  Splitting the operands inside the product
// costs every output tile its own conversion of the operand tiles (the converter warps then set the pace, about
// twice the time of the MMAs); splitting them beforehand costs one bandwidth-bound pass per operand.  Measured on
// the B200: 16 output tiles (500 x 500) 88 us inside against 53 + 2 x 21 us beforehand; 64 tiles and more are
// faster beforehand (workloads c4, c5: +2 % and +6 % per iteration), and so is layer 1, whose second operand X
// never changes and keeps its planes.
static bool planes_beforehand(int M, int N, bool second_operand_cached) {
  const int64_t tiles = ceil_div(M, TC_BM) * ceil_div(N, TC_BN);
  return tiles >= 16 || (second_operand_cached && tiles >= 8);
}

}  // namespace pd

namespace pd {

// ---- pieces of one iteration -------------------------------------------------------------------------------

// planes of W_l as the operand of a product with rows n_out contracted over n_in (P W^T, g W^T) ...
static PlaneRef planes_W(const Layer &ly) { return PlaneRef{ly.Wp.hi, ly.Wp.lo, ly.Wp.ldh, ly.Wp.exp}; }
// ... and of W_l^T, rows n_in contracted over n_out (r W)
static PlaneRef planes_WT(const Layer &ly) { return PlaneRef{ly.Wp.hiT, ly.Wp.loT, ly.Wp.ldhT, ly.Wp.exp}; }
static PlaneRef planes_G(const Layer &ly) { return PlaneRef{ly.Gp.hi, ly.Gp.lo, ly.Gp.ldh, ly.Gp.exp}; }

// planes of p_1 = X, which never changes, in its own orientation (null planes if the layer does not keep them)
static PlaneRef planes_X(const Layer &ly) { return PlaneRef{ly.x_hi, ly.x_lo, ly.ld_in, ly.x_exp}; }

// r_l = P_l W_l^T + b_l - z_l from scratch (only when the cached residual is not valid).
static int refresh_residual(pdadmm_ctx *c, Layer &ly, cudaStream_t st) {
  PD_CUDA(cudaMemsetAsync(ly.amax_r, 0, sizeof(uint32_t), st));
  EpiLinearResidual epi{ly.r, ly.ld_out, ly.b, ly.z, ly.amax_r};
  const PlaneRef xp = planes_X(ly);
  PD_TRY(gemm_nodes<false>(c, KC_GEMM_RESID, st, (int)c->N, ly.n_out, ly.n_in, ly.p, ly.ld_in, ly.W, ly.ld_in,
                           planes_W(ly), epi, nullptr, nullptr, 4.0 * c->N * ly.n_out, ly.amax_p, &xp));
  if (!c->use_tc) {       // the CUDA-core product does not track the maximum of what it stores
    Launch l(c, KC_AMAX, st, 4.0 * c->N * ly.ld_out, 0);
    absmax_kernel<<<ew_grid((size_t)c->N * ly.ld_out / 4), EW_THREADS, 0, st>>>(ly.r, (size_t)c->N * ly.ld_out / 4, ly.amax_r);
  }
  return PDADMM_OK;
}

// g = nu r W + u_{l-1} + rho (p - q_{l-1}) -> s1, ||g||^2 ; W g -> s2, ||W g||^2 ; tau.
static int p_gradient_and_tau(pdadmm_ctx *c, int l /*0-based, >= 1*/) {
  Layer &ly = c->layers[l];
  Layer &prev = c->layers[l - 1];
  Scratch &s = *c->cur;
  const int N = (int)c->N;
  int np = 0;
  (void)prev;
  uint32_t *w_g = nullptr;                 // max|g|, kept by the epilogue that writes g
  if (c->use_tc) { PD_TRY(amax_reserve(c, s.st, 1)); w_g = amax_take(c); }
  // Quantised update, wide layers: the norm-only product W g takes g as one fp16 plane.  The epilogue that writes g
  // writes that plane too, scaled by an exponent predicted from the previous iteration's max|g| (the true one is known
  // only when the product has finished); rows_planes_kernel then confirms the prediction or, if max|g| moved by more
  // than the plane can take, splits g again (6 bytes per element, the cost of every iteration before this).
  const bool copy_g = c->levels && c->use_tc && s.g_hi != nullptr && (size_t)N * ly.ld_in <= s.a_cap &&
                      ceil_div(ly.n_out, TC_BN) >= PLANES_FROM_COL_TILES / 2;
  if (copy_g) {
    EpiGradTCopy epi{{s.s1, ly.ld_in, ly.t, c->nu, w_g}, s.g_hi, ly.g_exp};
    PD_TRY(gemm_nodes<true>(c, KC_GEMM_GRADP, s.st, N, ly.n_in, ly.n_out, ly.r, ly.ld_out, ly.W, ly.ld_in, planes_WT(ly),
                            epi, s.slots, &np, 6.0 * N * ly.n_in, ly.amax_r));
  } else {
    EpiGradT epi{s.s1, ly.ld_in, ly.t, c->nu, w_g};
    PD_TRY(gemm_nodes<true>(c, KC_GEMM_GRADP, s.st, N, ly.n_in, ly.n_out, ly.r, ly.ld_out, ly.W, ly.ld_in, planes_WT(ly),
                            epi, s.slots, &np, 4.0 * N * ly.n_in, ly.amax_r));
  }
  int np2 = 0;
  double *slots_b = s.slots + s.n_slots / 2;          // second half of the slot buffer
  if (c->levels && c->use_tc) {
    // the quantised update only needs ||W g||^2 (for the first tau); its residual update uses W d
    EpiNormOnly epi2{s.s2, ly.ld_out};
    PlaneRef gp{nullptr, nullptr, 0, nullptr};
    if (copy_g) {
      const size_t n8 = (size_t)N * ly.ld_in / 8;
      Launch k(c, KC_PLANES, s.st, 0.0, 0);          // normally only publishes the exponent
      rows_planes_kernel<<<ew_grid(n8), 256, 0, s.st>>>(s.s1, n8, w_g, s.g_hi_exp, s.g_hi, nullptr, ly.g_exp);
      gp = PlaneRef{s.g_hi, s.g_hi, ly.ld_in, s.g_hi_exp};
    }
    PD_TRY(gemm_nodes<false>(c, KC_GEMM_WG, s.st, N, ly.n_out, ly.n_in, s.s1, ly.ld_in, ly.W, ly.ld_in, planes_W(ly),
                             epi2, slots_b, &np2, 0, w_g, &gp));
  } else {
    EpiStoreSumsq epi2{s.s2, ly.ld_out};
    PD_TRY(gemm_nodes<false>(c, KC_GEMM_WG, s.st, N, ly.n_out, ly.n_in, s.s1, ly.ld_in, ly.W, ly.ld_in, planes_W(ly),
                             epi2, slots_b, &np2, 0, w_g));
  }
  if (c->reduce != nullptr) {
    // ||g||^2 and ||W g||^2 are sums over nodes: this shard's totals, added over the shards, then tau
    PD_TRY(shard_sum_slots(c, s.st, s.red, s.slots, np, slots_b, np2));
    finalize_tau_kernel<<<1, FIN_THREADS, 0, s.st>>>(ly.sc, (double)c->rho, (double)c->nu, s.red, 1, s.red + 1, 1, c->d_flag + 2,
                                             ly.amax_p, w_g, copy_g ? ly.g_exp : nullptr);
    return PDADMM_OK;
  }
  {
    Launch k(c, KC_SMALL, s.st, 8.0 * (np + np2), 0);
    finalize_tau_kernel<<<1, FIN_THREADS, 0, s.st>>>(ly.sc, (double)c->rho, (double)c->nu, s.slots, np, slots_b, np2, c->d_flag + 2,
                                             ly.amax_p, w_g, copy_g ? ly.g_exp : nullptr);
  }
  return PDADMM_OK;
}

// pdADMM-G: p <- p - g/tau, r <- r - (W g)/tau.
static void p_step_plain(pdadmm_ctx *c, int l) {
  Layer &ly = c->layers[l];
  Scratch &s = *c->cur;
  const size_t n4p = (size_t)c->N * ly.ld_in / 4, n4r = (size_t)c->N * ly.ld_out / 4;
  {
    Launch k(c, KC_AXPY, s.st, 12.0 * c->N * ly.n_in, 0);
    axpy_neg_kernel<<<ew_grid(n4p), EW_THREADS, 0, s.st>>>(ly.p, s.s1, &ly.sc->inv_tau, n4p, ly.amax_p);
  }
  {
    Launch k(c, KC_AXPY, s.st, 12.0 * c->N * ly.n_out, 0);
    axpy_neg_kernel<<<ew_grid(n4r), EW_THREADS, 0, s.st>>>(ly.r, s.s2, &ly.sc->inv_tau, n4r, ly.amax_r);
  }
}

// pdADMM-G-Q: project p - g/tau on the level set, doubling tau until the stop condition holds.  Each trial ends
// with a copy of the accept flag to the host, which decides whether another trial is needed (the only host round
// trips of an iteration).  The two halves below let the caller queue another layer's work on the other lane before
// it waits for the flag.
// One trial: trial p, d = trial p - p and its codes, W d with its squared norm, the accept test, the flag's copy.
static int q_trial(pdadmm_ctx *c, int l) {
  Layer &ly = c->layers[l];
  Scratch &s = *c->cur;
  const int N = (int)c->N;
  const size_t n4p = (size_t)N * ly.ld_in / 4;
  const int grid = ew_grid(n4p);
  uint32_t *w_d = nullptr;               // max|d| of this trial
  if (c->use_tc) { PD_TRY(amax_reserve(c, s.st, 1)); w_d = amax_take(c); }
  {
    // reads g and the codes of p; writes p+, the new codes and d -- as fp32, or, with integer operands, as the two
    // fp16 planes of integers: 14 bytes per element with one-byte codes either way
    Launch k(c, KC_QUANT, s.st, 14.0 * N * ly.n_in, 0);
    quant_trial_kernel<<<grid, EW_THREADS, 0, s.st>>>(s.s1, ly.sc, ly.scale, ly.lo, c->levels, s.p_new,
                                                     c->int_operands ? nullptr : s.d,
                                                     s.codes_new, c->code_bytes == 2, n4p, s.slots,
                                                     c->use_tc ? ly.amax_p : nullptr, w_d,
                                                     ly.codes, s.pn_plane, s.d_plane);
  }
  int np = 0;
  double *slots_b = s.slots + s.n_slots / 2;
  // the trial's residual r + W d is written beside r (the two trade places when the trial is taken), with ||W d||^2;
  // max|r| takes the trial's values too, which keeps it an upper bound whether or not the trial is taken
  EpiAddSumsq epi{s.s2, ly.ld_out, ly.r, c->use_tc ? ly.amax_r : nullptr};
  const IntPlane di{c->int_operands ? s.d_plane : nullptr, ly.ld_in, ly.scale};      // d = (new code - old code) s
  PD_TRY(gemm_nodes<false>(c, KC_GEMM_WG, s.st, N, ly.n_out, ly.n_in, s.d, ly.ld_in, ly.W, ly.ld_in, planes_W(ly), epi,
                           slots_b, &np, 4.0 * N * ly.n_out, w_d, nullptr, &di));
  if (c->reduce != nullptr) {
    PD_TRY(shard_sum_slots(c, s.st, s.red, s.slots, grid, slots_b, np));
    finalize_trial_kernel<<<1, FIN_THREADS, 0, s.st>>>(ly.sc, (double)c->rho, (double)c->nu, 1e-6, s.red, 1, s.red + 1, 1);
  } else {
    Launch k(c, KC_SMALL, s.st, 8.0 * (grid + np), 0);
    finalize_trial_kernel<<<1, FIN_THREADS, 0, s.st>>>(ly.sc, (double)c->rho, (double)c->nu, 1e-6, s.slots, grid, slots_b, np);
  }
  PD_CUDA(cudaMemcpyAsync(s.h_flag, &ly.sc->accepted, sizeof(int), cudaMemcpyDeviceToHost, s.st));
  PD_CUDA(cudaEventRecord(s.ev_flag, s.st));
  return PDADMM_OK;
}
// After the first trial of layer l was queued on the current lane: wait for its flag, run further trials while it
// says no, then take the trial: p, codes <- trial, r <- r + W d.
static int q_finish(pdadmm_ctx *c, int l, bool *hit_cap) {
  Layer &ly = c->layers[l];
  Scratch &s = *c->cur;
  const int max_trials = 30;
  for (int trial = 0;; ++trial) {
    PD_CUDA(cudaEventSynchronize(s.ev_flag));
    if (*s.h_flag || trial + 1 >= max_trials) {
      if (!*s.h_flag) *hit_cap = true;
      break;
    }
    PD_TRY(q_trial(c, l));
  }
  std::swap(ly.p, s.p_new);
  std::swap(ly.codes, s.codes_new);
  std::swap(ly.p_plane, s.pn_plane);
  std::swap(ly.r, s.s2);                // r <- r + W d, written by the trial's product
  return PDADMM_OK;
}

// G = nu r^T p+ (contraction over nodes), theta, W <- W - G/theta, r <- r - (G p+)/theta,
// b <- b - mean_j r, shift = mean_j r.
static int w_and_b_step(pdadmm_ctx *c, int l) {
  Layer &ly = c->layers[l];
  Scratch &s = *c->cur;
  const int N = (int)c->N;
  if (!c->use_tc) {
    dim3 grid((unsigned)ceil_div(ly.n_in, SG_BN), (unsigned)ceil_div(ly.n_out, SG_BM), (unsigned)ly.n_split);
    Launch k(c, KC_GEMM_GRADW, s.st, 4.0 * ((double)N * ly.n_in + (double)N * ly.n_out), 2.0 * N * ly.n_in * ly.n_out);
    gemm_tn_kernel<<<grid, SG_THREADS, 0, s.st>>>(ly.n_out, ly.n_in, N, ly.k_chunk, ly.r, ly.ld_out, ly.p, ly.ld_in,
                                                 s.part, ly.ld_in);
  } else {
    // both operands are node-major, i.e. contiguous along their output index (r is [nodes][n_out], p+ is
    // [nodes][n_in]): transposed and split into planes beforehand, or tile by tile inside the product
    if (planes_beforehand(ly.n_out, ly.n_in, l == 0)) {
      transpose_planes(c, s.st, ly.r, N, ly.n_out, ly.ld_out, ly.amax_r, s.rT_hi, s.rT_lo, c->ldT, s.rT_exp);
      PlaneRef Bt{s.pT_hi, s.pT_lo, c->ldT, s.pT_exp};
      float b_mul = 0.f;
      if (l == 0) {        // p_1 = X never changes: its planes are kept (made before the first iteration)
        Bt = PlaneRef{ly.xT_hi, ly.xT_lo, c->ldT, ly.xT_exp};
      } else if (c->int_operands) {
        // p+ = code * s: the transposed codes are the whole operand (1 byte read, 2 written per element instead of 4 + 4)
        Launch k(c, KC_PLANES, s.st, 3.0 * N * ly.n_in, 0);
        const dim3 grid((unsigned)ceil_div(ly.n_in, 32), (unsigned)ceil_div(N, 32));
        transpose_codes_kernel<<<grid, dim3(32, 8), 0, s.st>>>(ly.codes, c->code_bytes == 2, N, ly.n_in, ly.ld_in, s.pT_hi, c->ldT);
        b_mul = ly.scale;
      } else {
        transpose_planes(c, s.st, ly.p, N, ly.n_in, ly.ld_in, ly.amax_p, s.pT_hi, s.pT_lo, c->ldT, s.pT_exp);
      }
      PD_TRY(gemm_over_nodes_tc(c, KC_GEMM_GRADW, s.st, ly.n_out, ly.n_in, N,
                                PlaneRef{s.rT_hi, s.rT_lo, c->ldT, s.rT_exp}, Bt, s.part, ly.ld_in, ly.k_chunk, ly.n_split, b_mul));
    } else {
      PD_TRY(gemm_over_nodes_raw(c, KC_GEMM_GRADW, s.st, ly.n_out, ly.n_in, N, ly.r, ly.ld_out, ly.p, ly.ld_in, s.part,
                                 ly.ld_in, ly.k_chunk, ly.n_split, ly.amax_r, ly.amax_p));
    }
  }
  const size_t n4w = (size_t)ly.n_out * ly.ld_in / 4;
  const int gw = ew_grid(n4w);
  {
    Launch k(c, KC_GRADW_REDUCE, s.st, 4.0 * (ly.n_split + 1.0) * ly.n_out * ly.n_in, 0);
    uint32_t *w = nullptr;
    if (c->use_tc) { PD_TRY(amax_reserve(c, s.st, 1)); w = amax_take(c); }
    reduce_gradW_kernel<<<gw, EW_THREADS, 0, s.st>>>(s.part, ly.n_split, n4w, c->nu, ly.gradW, w, s.slots);
    if (c->reduce != nullptr) {
      // nabla_W phi is a sum over nodes: add the shards' parts, then take the norm and the largest magnitude of the total
      PD_TRY(shard_sum(c, s.st, ly.gradW, n4w * 4, 0));
      if (c->use_tc) { PD_TRY(amax_reserve(c, s.st, 1)); w = amax_take(c); }
      sumsq_amax_kernel<<<gw, EW_THREADS, 0, s.st>>>(ly.gradW, n4w, w, s.slots);
    }
    if (c->use_tc) make_planes(c, s.st, ly.gradW, ly.n_out, ly.n_in, ly.ld_in, w, ly.Gp);
  }
  int np = 0;
  double *slots_b = s.slots + s.n_slots / 2;
  EpiStoreSumsq epi{s.s1, ly.ld_out};
  const PlaneRef xp = planes_X(ly);
  const IntPlane pi{(c->int_operands && l > 0) ? ly.p_plane : nullptr, ly.ld_in, ly.scale};          // p+ = code * s
  PD_TRY(gemm_nodes<false>(c, KC_GEMM_GP, s.st, N, ly.n_out, ly.n_in, ly.p, ly.ld_in, ly.gradW, ly.ld_in, planes_G(ly),
                           epi, slots_b, &np, 0, ly.amax_p, &xp, &pi));
  if (c->reduce != nullptr) {
    // ||G p+||^2 is a sum over nodes (||G||^2 is the same on every shard already)
    PD_TRY(shard_sum_slots(c, s.st, s.red, slots_b, np, nullptr, 0));
    finalize_theta_kernel<<<1, FIN_THREADS, 0, s.st>>>(ly.sc, (double)c->nu, s.slots, gw, s.red, 1, c->d_flag + 2, ly.amax_r);
  } else {
    Launch k(c, KC_SMALL, s.st, 8.0 * (gw + np), 0);
    finalize_theta_kernel<<<1, FIN_THREADS, 0, s.st>>>(ly.sc, (double)c->nu, s.slots, gw, slots_b, np, c->d_flag + 2, ly.amax_r);
  }
  {
    Launch k(c, KC_WSTEP, s.st, 20.0 * ly.n_out * ly.n_in, 0);
    uint32_t *w = nullptr;
    if (c->use_tc) { PD_TRY(amax_reserve(c, s.st, 1)); w = amax_take(c); }
    wstep_kernel<<<gw, EW_THREADS, 0, s.st>>>(ly.W, ly.gradW, ly.sc, n4w, w);
    if (c->use_tc) make_planes(c, s.st, ly.W, ly.n_out, ly.n_in, ly.ld_in, w, ly.Wp);
  }
  const int n_blocks = (int)std::min<int64_t>(c->n_sms * 4, ceil_div(N, 16));
  const int rows_per_block = (int)ceil_div(N, n_blocks);
  const int used_blocks = (int)ceil_div(N, rows_per_block);
  {
    const int ld4 = ly.ld_out / 4, cols_per_pass = std::min(ld4, EW_THREADS);
    const int n_sub = std::min(EW_THREADS / cols_per_pass, COLSUM_MAX_SUB);
    const size_t sh = n_sub > 1 ? (size_t)n_sub * ly.ld_out * sizeof(double) : 0;
    Launch k(c, KC_COLSUM, s.st, 12.0 * N * ly.n_out, 0);
    resid_colsum_kernel<<<used_blocks, EW_THREADS, sh, s.st>>>(ly.r, s.s1, ly.sc, N, ly.ld_out, rows_per_block, s.slots);
  }
  if (c->reduce != nullptr) {
    // the column sums run over all nodes: this shard's sums, added over the shards, then the mean over |V|
    colsum_total_kernel<<<(int)ceil_div(ly.ld_out, 32), dim3(32, BIAS_GROUPS), 0, s.st>>>(s.slots, used_blocks, ly.ld_out, s.red);
    PD_TRY(shard_sum(c, s.st, s.red, (size_t)ly.ld_out, 1));
    finalize_bias_kernel<<<(int)ceil_div(ly.ld_out, 32), dim3(32, BIAS_GROUPS), 0, s.st>>>(s.red, 1, ly.ld_out, ly.n_out,
                                                                                1.0 / (double)c->N_total, ly.b, ly.shift);
  } else {
    Launch k(c, KC_SMALL, s.st, 8.0 * used_blocks * ly.ld_out, 0);
    finalize_bias_kernel<<<(int)ceil_div(ly.ld_out, 32), dim3(32, BIAS_GROUPS), 0, s.st>>>(s.slots, used_blocks, ly.ld_out, ly.n_out,
                                                                                1.0 / (double)N, ly.b, ly.shift);
  }
  return PDADMM_OK;
}

// z (and q, u for hidden layers) of layer l; needs p_{l+1} of this iteration.
static void zqu_step(pdadmm_ctx *c, int l) {
  Layer &ly = c->layers[l];
  Scratch &s = *c->cur;
  const int N = (int)c->N;
  if (l + 1 < c->L) {
    const size_t n4 = (size_t)N * ly.ld_out / 4;
    const int grid = ew_grid(n4);
    if (c->table_size > 0) {
      Launch k(c, KC_ZQU, s.st, (c->levels ? 37.0 : 40.0) * N * ly.n_out, 0);
      const Layer &nx = c->layers[l + 1];
      zqu_table_kernel<<<grid, EW_THREADS, 2 * c->table_size * sizeof(float), s.st>>>(
          ly.r, ly.z, ly.q, ly.u, nx.p, ly.shift, ly.ld_out / 4, n4, c->rho, c->nu, c->slope, c->table_lo, c->table_step,
          c->table_size, nx.scale, nx.lo, c->quant_q ? (float)(c->levels - 1) : -1.0f, nx.t, s.slots, ly.amax_r,
          c->levels ? nx.codes : nullptr, c->code_bytes == 2);
    } else {
      Launch k(c, KC_ZQU, s.st, (c->levels ? 37.0 : 40.0) * N * ly.n_out, 0);      // p_{l+1} as one-byte codes
      const Layer &nx = c->layers[l + 1];
      zqu_kernel<<<grid, EW_THREADS, 0, s.st>>>(ly.r, ly.z, ly.q, ly.u, nx.p, ly.shift, ly.ld_out / 4, n4, c->rho, c->nu,
                                               c->slope, nx.scale, nx.lo, c->quant_q ? (float)(c->levels - 1) : -1.0f, nx.t,
                                               s.slots, ly.amax_r, c->levels ? nx.codes : nullptr, c->code_bytes == 2);
    }
  } else {
    Launch k(c, KC_ZLAST, s.st, 16.0 * N * ly.n_out, 0);
    zlast_kernel<<<(int)ceil_div(N, 128), 128, 0, s.st>>>(ly.r, ly.z, ly.shift, c->labels, c->mask, N, ly.n_out,
                                                          ly.ld_out, (double)c->nu, c->d_flag, ly.amax_r, c->ls_risk ? 1 : 0);
  }
}

static Scratch &lane(pdadmm_ctx *c, int i) { return i == 0 ? c->scr : *c->more_lanes[i - 1]; }

static int iterate_once(pdadmm_ctx *c, bool *hit_cap) {
  // per-kernel timing wants one kernel at a time: a single lane then
  const int S = c->profiling ? 1 : 1 + (int)c->more_lanes.size();
  auto lane_of = [&](int l) -> Scratch & { return lane(c, l % S); };
  struct Restore { pdadmm_ctx *c; ~Restore() { c->cur = &c->scr; } } restore{c};
  // the other lanes start after everything queued on the main stream so far
  if (S > 1) {
    PD_CUDA(cudaEventRecord(c->ev_lane[0], c->scr.st));
    for (int i = 1; i < S; ++i) PD_CUDA(cudaStreamWaitEvent(lane(c, i).st, c->ev_lane[0], 0));
  }
  if (c->use_tc)
    for (int i = 0; i < S; ++i) { c->cur = &lane(c, i); PD_TRY(amax_reset(c, c->cur->st)); }
  // p-update of layers 2..L from the iterates of the previous iteration.  The quantised update reads an accept
  // flag on the host after every trial: the host queues layer l's gradient and first trial on its lane, and only
  // then waits for the flag of the layer that it queued on that lane before (layer l - S), so that the GPU always
  // has the other lane's work while a flag travels.
  std::vector<int> waiting(S, -1);                   // layer whose first trial is in flight on each lane
  for (int l = 1; l < c->L; ++l) {
    c->cur = &lane_of(l);
    if (c->levels) {
      int &w = waiting[l % S];
      if (w >= 0) {
        PD_TRY(q_finish(c, w, hit_cap));
        if (S > 1) PD_CUDA(cudaEventRecord(c->ev_p[w], c->cur->st));
      }
      PD_TRY(p_gradient_and_tau(c, l));
      PD_TRY(q_trial(c, l));
      w = l;
    } else {
      PD_TRY(p_gradient_and_tau(c, l));
      p_step_plain(c, l);
      if (S > 1) PD_CUDA(cudaEventRecord(c->ev_p[l], c->cur->st));
    }
  }
  for (int i = 0; i < S && c->levels; ++i) {
    if (waiting[i] < 0) continue;
    c->cur = &lane(c, i);
    PD_TRY(q_finish(c, waiting[i], hit_cap));
    if (S > 1) PD_CUDA(cudaEventRecord(c->ev_p[waiting[i]], c->cur->st));
  }
  // W- and b-update of every layer with the new p
  for (int l = 0; l < c->L; ++l) {
    c->cur = &lane_of(l);
    PD_TRY(w_and_b_step(c, l));
  }
  // z-, q-, u-update (q_l and u_l need p_{l+1} of this iteration, which another lane may have written)
  for (int l = 0; l < c->L; ++l) {
    c->cur = &lane_of(l);
    if (S > 1 && l + 1 < c->L) PD_CUDA(cudaStreamWaitEvent(c->cur->st, c->ev_p[l + 1], 0));
    zqu_step(c, l);
  }
  // join: the main stream continues after every lane
  for (int i = 1; i < S; ++i) {
    PD_CUDA(cudaEventRecord(c->ev_lane[i], lane(c, i).st));
    PD_CUDA(cudaStreamWaitEvent(c->scr.st, c->ev_lane[i], 0));
  }
  return PDADMM_OK;
}

}  // namespace pd

namespace pd {

// ---- construction ---------------------------------------------------------------------------------------------

static int check_config(const pdadmm_config *cfg) {
  if (!cfg) return fail(PDADMM_EINVAL, "config is null");
  if (cfg->n_nodes < 1 || cfg->n_nodes > (int64_t)INT32_MAX / 2) return fail(PDADMM_EINVAL, "n_nodes out of range");
  if (cfg->n_edges < 0 || (cfg->n_edges > 0 && (!cfg->edge_src || !cfg->edge_dst)))
    return fail(PDADMM_EINVAL, "edge list missing");
  if (cfg->feat_dim < 1 || !cfg->features) return fail(PDADMM_EINVAL, "features missing");
  if (cfg->n_hops < 0 || cfg->n_hops > 16) return fail(PDADMM_EINVAL, "n_hops must be in [0, 16]");
  if (cfg->n_layers < 1 || !cfg->layer_widths || !cfg->init_W) return fail(PDADMM_EINVAL, "layers missing");
  if (cfg->n_layers > 1024) return fail(PDADMM_EINVAL, "at most 1024 layers");
  if (cfg->n_classes < 2 || cfg->n_classes > ZL_MAX_C)
    return fail(PDADMM_EINVAL, "n_classes must be in [2, %d]", ZL_MAX_C);
  if (cfg->layer_widths[cfg->n_layers - 1] != cfg->n_classes)
    return fail(PDADMM_EINVAL, "last layer width must equal n_classes");
  for (int l = 0; l < cfg->n_layers; ++l) {
    if (cfg->layer_widths[l] < 1) return fail(PDADMM_EINVAL, "layer width %d is not positive", l + 1);
    if (!cfg->init_W[l]) return fail(PDADMM_EINVAL, "init_W[%d] is null", l);
  }
  if (!cfg->labels || !cfg->train_mask) return fail(PDADMM_EINVAL, "labels or mask missing");
  if (!(cfg->rho > 0.f) || !(cfg->nu > 0.f)) return fail(PDADMM_EINVAL, "rho and nu must be positive");
  if (cfg->quant_levels != 0 && (cfg->quant_levels < 2 || cfg->quant_levels > 65536))
    return fail(PDADMM_EINVAL, "quant_levels must be 0 or in [2, 65536]");
  if (cfg->quant_neg_levels < 0 || cfg->quant_neg_levels >= std::max(cfg->quant_levels, 1))
    return fail(PDADMM_EINVAL, "quant_neg_levels must be in [0, quant_levels)");
  if (cfg->quant_step < 0.f || (cfg->quant_neg_levels > 0 && !(cfg->quant_step > 0.f)))
    return fail(PDADMM_EINVAL, "quant_step must be >= 0, and > 0 when quant_neg_levels > 0");
  if (!(cfg->leaky_slope >= 0.f && cfg->leaky_slope < 1.f))
    return fail(PDADMM_EINVAL, "leaky_slope must be in [0, 1)");
  if (cfg->activation < 0 || cfg->activation > 2) return fail(PDADMM_EINVAL, "activation must be 0, 1 or 2");
  if (cfg->activation != 0) {
    if (cfg->leaky_slope != 0.f) return fail(PDADMM_EINVAL, "leaky_slope belongs to activation 0");
    if (cfg->table_size < 2 || cfg->table_size > 4096 || !(cfg->table_hi > cfg->table_lo))
      return fail(PDADMM_EINVAL, "a smooth activation needs table_size in [2, 4096] and table_lo < table_hi");
  }
  if ((cfg->flags & PDADMM_FLAG_QUANT_Q) && cfg->quant_levels == 0)
    return fail(PDADMM_EINVAL, "PDADMM_FLAG_QUANT_Q needs quant_levels >= 2");
  for (int64_t j = 0; j < cfg->n_nodes; ++j)
    if (cfg->labels[j] < 0 || cfg->labels[j] >= cfg->n_classes)
      return fail(PDADMM_EINVAL, "label of node %lld is outside [0, %d)", (long long)j, cfg->n_classes);
  return PDADMM_OK;
}

// Host -> device copies go through the context's stream, so that they are ordered with its kernels
// (the stream does not synchronise with the default stream).
static int upload_rows(cudaStream_t st, float *dst, int ld, const float *src, int width, int64_t rows) {
  PD_CUDA(cudaMemcpy2DAsync(dst, (size_t)ld * 4, src, (size_t)width * 4, (size_t)width * 4, (size_t)rows,
                            cudaMemcpyHostToDevice, st));
  PD_CUDA(cudaStreamSynchronize(st));
  return PDADMM_OK;
}

// Temporary device buffers of the CSR construction, released when the builder returns.
struct TempBuffers {
  std::vector<void *> ptrs;
  ~TempBuffers() { for (void *p : ptrs) cudaFree(p); }
  template <class T>
  int get(T **out, size_t count) {
    void *p = nullptr;
    const size_t bytes = std::max<size_t>(count * sizeof(T), 16);
    const cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return fail(PDADMM_ENOMEM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
    }
    ptrs.push_back(p);
    *out = (T *)p;
    return PDADMM_OK;
  }
};

// Edge list (host) -> c->row_ptr, c->col_idx (device), c->nnz; c->csr_val is allocated, not filled.
static int build_csr(pdadmm_ctx *c, const pdadmm_config *cfg) {
  const int64_t N = c->N, E = cfg->n_edges;
  const size_t raw_cap = (size_t)(2 * E + N);
  if (raw_cap > (size_t)INT32_MAX) return fail(PDADMM_EINVAL, "more than 2^31-1 non-zeros");
  cudaStream_t st = c->scr.st;
  TempBuffers tmp;
  int *d_src, *d_dst, *deg, *cursor, *raw_ptr, *raw, *sorted, *len, *long_rows, *meta;
  unsigned long long *bad_edge;
  PD_TRY(tmp.get(&d_src, (size_t)E)); PD_TRY(tmp.get(&d_dst, (size_t)E));
  PD_TRY(tmp.get(&deg, (size_t)N)); PD_TRY(tmp.get(&cursor, (size_t)N)); PD_TRY(tmp.get(&len, (size_t)N));
  PD_TRY(tmp.get(&raw_ptr, (size_t)N + 1)); PD_TRY(tmp.get(&long_rows, (size_t)N));
  PD_TRY(tmp.get(&raw, raw_cap)); PD_TRY(tmp.get(&sorted, raw_cap));
  PD_TRY(tmp.get(&meta, 4)); PD_TRY(tmp.get(&bad_edge, 1));
  PD_TRY(dev_alloc(c, &c->row_ptr, (size_t)N + 1, false));
  PD_CUDA(cudaMemsetAsync(deg, 0, (size_t)N * 4, st));
  PD_CUDA(cudaMemsetAsync(cursor, 0, (size_t)N * 4, st));
  PD_CUDA(cudaMemsetAsync(len, 0, (size_t)N * 4, st));
  PD_CUDA(cudaMemsetAsync(meta, 0, 16, st));
  PD_CUDA(cudaMemsetAsync(bad_edge, 0xff, 8, st));
  const int e_grid = (int)std::max<int64_t>(1, ceil_div(E, 256)), r_grid = (int)ceil_div(N * 32, 256);
  if (E > 0) {
    PD_CUDA(cudaMemcpyAsync(d_src, cfg->edge_src, (size_t)E * 4, cudaMemcpyHostToDevice, st));
    PD_CUDA(cudaMemcpyAsync(d_dst, cfg->edge_dst, (size_t)E * 4, cudaMemcpyHostToDevice, st));
    edge_count_kernel<<<e_grid, 256, 0, st>>>(d_src, d_dst, (long long)E, (int)N, deg, meta, bad_edge);
  }
  exclusive_scan_kernel<<<1, 1024, 0, st>>>(deg, (int)N, 1, raw_ptr, meta);
  if (E > 0) edge_scatter_kernel<<<e_grid, 256, 0, st>>>(d_src, d_dst, (long long)E, (int)N, raw_ptr, cursor, raw);
  row_sort_warp_kernel<<<r_grid, 256, 0, st>>>(raw_ptr, (int)N, raw, sorted, len, long_rows, meta);
  row_sort_block_kernel<<<2 * c->n_sms, 1024, 0, st>>>(raw_ptr, raw, sorted, len, long_rows, meta);
  exclusive_scan_kernel<<<1, 1024, 0, st>>>(len, (int)N, 0, c->row_ptr, meta);
  int h_meta[4]; unsigned long long h_bad; int h_nnz;
  PD_CUDA(cudaMemcpyAsync(h_meta, meta, 16, cudaMemcpyDeviceToHost, st));
  PD_CUDA(cudaMemcpyAsync(&h_bad, bad_edge, 8, cudaMemcpyDeviceToHost, st));
  PD_CUDA(cudaMemcpyAsync(&h_nnz, c->row_ptr + N, 4, cudaMemcpyDeviceToHost, st));
  PD_CUDA(cudaStreamSynchronize(st));
  if (h_meta[0] == 1)
    return fail(PDADMM_EINVAL, "edge %llu = (%d, %d) is outside [0, %lld)", h_bad, cfg->edge_src[h_bad],
                cfg->edge_dst[h_bad], (long long)N);
  if (h_meta[0] == 2) return fail(PDADMM_EINVAL, "more than 2^31-1 non-zeros");
  if (h_meta[0] == 3) return fail(PDADMM_EINVAL, "a node has more than %d neighbours", CSR_MAX_ROW - 1);
  c->nnz = h_nnz;
  PD_TRY(dev_alloc(c, &c->col_idx, (size_t)c->nnz, false));
  PD_TRY(dev_alloc(c, &c->csr_val, (size_t)c->nnz, false));
  row_compact_kernel<<<r_grid, 256, 0, st>>>(raw_ptr, c->row_ptr, (int)N, sorted, c->col_idx);
  PD_CUDA(cudaGetLastError());
  PD_CUDA(cudaStreamSynchronize(st));     // the temporaries are released on return
  return PDADMM_OK;
}

// buffers of a lane's quantised trials: trial p, d, codes (they trade places with a layer's p and codes when a
// trial is taken, so all have one size), the pinned word and the event of the accept flag
static int alloc_trial_buffers(pdadmm_ctx *c, Scratch &s, size_t n) {
  PD_TRY(dev_alloc(c, &s.p_new, n));
  if (!c->int_operands) PD_TRY(dev_alloc(c, &s.d, n));       // with integer operands d exists as d_plane only
  PD_TRY(dev_alloc(c, &s.codes_new, n * c->code_bytes));
  if (c->int_operands) {
    PD_TRY(dev_alloc(c, &s.pn_plane, n));
    PD_TRY(dev_alloc(c, &s.d_plane, n));
  }
  PD_CUDA(cudaMallocHost((void **)&s.h_flag, sizeof(int)));
  PD_CUDA(cudaEventCreateWithFlags(&s.ev_flag, cudaEventDisableTiming));
  return PDADMM_OK;
}

// transposed planes of r_l (up to max_out columns) and of p_l, l >= 2 (up to max_in columns) of one lane
// planes of the streamed operand of a product, once per lane: as wide as the widest matrix the lane's s1 holds
static int alloc_row_planes(pdadmm_ctx *c, Scratch &s, size_t n) {
  PD_TRY(dev_alloc(c, &s.a_hi, n, false));
  PD_TRY(dev_alloc(c, &s.a_lo, n, false));
  PD_TRY(dev_alloc(c, &s.a_exp, 1));
  s.a_cap = n;
  if (c->levels) {
    PD_TRY(dev_alloc(c, &s.g_hi, n, false));
    PD_TRY(dev_alloc(c, &s.g_hi_exp, 1));
  }
  return PDADMM_OK;
}

static int alloc_transposed(pdadmm_ctx *c, Scratch &s, int max_out, int max_in) {
  if (max_out > 0) {
    PD_TRY(dev_alloc(c, &s.rT_hi, (size_t)max_out * c->ldT));
    PD_TRY(dev_alloc(c, &s.rT_lo, (size_t)max_out * c->ldT));
  }
  PD_TRY(dev_alloc(c, &s.rT_exp, 1));
  if (max_in > 0) {
    PD_TRY(dev_alloc(c, &s.pT_hi, (size_t)max_in * c->ldT));
    PD_TRY(dev_alloc(c, &s.pT_lo, (size_t)max_in * c->ldT));
  }
  PD_TRY(dev_alloc(c, &s.pT_exp, 1));
  return PDADMM_OK;
}

// Start of Algorithm 1 for layers first..L-1 (0-based) from the current p_first: b = 0, z_l = W_l p_l, q_l = f(z_l),
// p_{l+1} = q_l (projected in -Q mode, with the level spacing from max(q_l)), u = 0, r = 0.
static int feasible_start(pdadmm_ctx *c, int first) {
  const int64_t N = c->N;
  cudaStream_t st = c->scr.st;
  Scratch &s = c->scr;
  for (int l = first; l < c->L; ++l) {
    Layer &ly = c->layers[l];
    EpiStore epi{ly.z, ly.ld_out};
    PD_TRY(split_planes(c, st, ly.W, ly.n_out, ly.n_in, ly.ld_in, ly.Wp));
    PD_CUDA(cudaMemsetAsync(ly.amax_p, 0, sizeof(uint32_t), st));
    absmax_kernel<<<ew_grid((size_t)N * ly.ld_in / 4), EW_THREADS, 0, st>>>(ly.p, (size_t)N * ly.ld_in / 4, ly.amax_p);
    if (l == 0 && ly.x_hi != nullptr) {
      const size_t n8 = (size_t)N * ly.ld_in / 8;
      rows_planes_kernel<<<ew_grid(n8), 256, 0, st>>>(ly.p, n8, ly.amax_p, ly.x_exp, ly.x_hi, ly.x_lo);
    }
    const PlaneRef xp = planes_X(ly);
    PD_TRY(gemm_nodes<false>(c, KC_GEMM_RESID, st, (int)N, ly.n_out, ly.n_in, ly.p, ly.ld_in, ly.W, ly.ld_in, planes_W(ly),
                             epi, nullptr, nullptr, 0, ly.amax_p, &xp));
    PD_CUDA(cudaMemsetAsync(ly.b, 0, (size_t)ly.ld_out * 4, st));
    PD_CUDA(cudaMemsetAsync(ly.shift, 0, (size_t)ly.ld_out * 4, st));
    PD_CUDA(cudaMemsetAsync(ly.r, 0, (size_t)N * ly.ld_out * 4, st));
    PD_CUDA(cudaMemsetAsync(ly.amax_r, 0, sizeof(uint32_t), st));
    if (l + 1 == c->L) break;
    PD_CUDA(cudaMemsetAsync(ly.u, 0, (size_t)N * ly.ld_out * 4, st));
    Layer &nx = c->layers[l + 1];
    const size_t n4 = (size_t)N * ly.ld_out / 4;
    const int grid = ew_grid(n4);
    float *bm = reinterpret_cast<float *>(s.slots);
    relu_max_kernel<<<grid, EW_THREADS, 0, st>>>(ly.z, ly.q, n4, c->slope, bm);
    if (c->levels) {
      std::vector<float> hm(grid);
      PD_CUDA(cudaMemcpyAsync(hm.data(), bm, grid * sizeof(float), cudaMemcpyDeviceToHost, st));
      PD_CUDA(cudaStreamSynchronize(st));
      float mx = 0.f;
      for (float v : hm) mx = std::max(mx, v);
      if (c->reduce != nullptr) {            // the level spacing comes from the largest entry over all nodes
        PD_CUDA(cudaMemcpyAsync(s.red, &mx, 4, cudaMemcpyHostToDevice, st));
        PD_TRY(shard_sum(c, st, s.red, 1, 0, 1));
        PD_CUDA(cudaMemcpyAsync(&mx, s.red, 4, cudaMemcpyDeviceToHost, st));
        PD_CUDA(cudaStreamSynchronize(st));
      }
      nx.scale = c->fixed_step > 0.f ? c->fixed_step : (mx > 0.f ? mx / (float)(c->levels - 1) : 1.0f);
      nx.lo = -(float)c->neg_levels * nx.scale;
      quantize_kernel<<<ew_grid(n4 * 4), EW_THREADS, 0, st>>>(ly.q, n4 * 4, nx.scale, nx.lo, c->levels, nx.p, nx.codes,
                                                              c->code_bytes == 2);
      if (c->int_operands) codes_to_plane_kernel<<<ew_grid(n4), EW_THREADS, 0, st>>>(nx.codes, c->code_bytes == 2, n4, nx.p_plane);
      if (c->quant_q)      // start inside the level set: q_l = p_{l+1}
        PD_CUDA(cudaMemcpyAsync(ly.q, nx.p, n4 * 16, cudaMemcpyDeviceToDevice, st));
    } else {
      PD_CUDA(cudaMemcpyAsync(nx.p, ly.q, n4 * 16, cudaMemcpyDeviceToDevice, st));
    }
  }
  return PDADMM_OK;
}

static int build(pdadmm_ctx *c, const pdadmm_config *cfg, const pdadmm_shard *shard) {
  const int64_t Ntot = cfg->n_nodes;
  const bool sharded = shard != nullptr && shard->allreduce != nullptr;
  const int64_t N = sharded ? shard->node_count : Ntot;
  const int64_t node0 = sharded ? shard->node_begin : 0;
  c->N_total = Ntot; c->node_begin = node0;
  if (sharded) { c->reduce = shard->allreduce; c->reduce_user = shard->user; }
  // the graph stage works on all nodes: c->N is the whole graph until X is built
  c->device = cfg->device; c->N = Ntot; c->L = cfg->n_layers; c->d = cfg->feat_dim; c->n_blocks = cfg->n_hops + 1;
  c->n0 = c->n_blocks * c->d; c->ld0 = round_up(c->n0, LD_ALIGN); c->C = cfg->n_classes; c->levels = cfg->quant_levels;
  c->neg_levels = cfg->quant_neg_levels; c->fixed_step = cfg->quant_step;
  c->code_bytes = cfg->quant_levels > 256 ? 2 : 1;
  c->quant_q = (cfg->flags & PDADMM_FLAG_QUANT_Q) != 0;
  c->slope = cfg->activation == 1 ? ACT_TANH : (cfg->activation == 2 ? ACT_SIGMOID : cfg->leaky_slope);
  if (cfg->activation != 0) {
    c->table_size = cfg->table_size;
    c->table_lo = cfg->table_lo;
    c->table_step = (cfg->table_hi - cfg->table_lo) / (float)(cfg->table_size - 1);      // single precision, like the candidates
  }
  c->ls_risk = (cfg->flags & PDADMM_FLAG_LEAST_SQUARES) != 0;
  c->rho = cfg->rho; c->nu = cfg->nu; c->flags = cfg->flags;
  c->use_tc = (cfg->flags & PDADMM_FLAG_SIMT_GEMM) == 0;
  c->int_operands = c->use_tc && c->levels >= 2 && c->levels <= 2048 && c->neg_levels == 0;
  PD_CUDA(cudaSetDevice(cfg->device));
  PD_CUDA(cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, cfg->device));
  PD_CUDA(cudaStreamCreateWithFlags(&c->scr.st, cudaStreamNonBlocking));
  cudaStream_t st = c->scr.st;
  PD_CUDA(cudaMallocHost((void **)&c->h_pinned, 64 * sizeof(int)));
  PD_CUDA(cudaEventCreate(&c->ev_begin));
  PD_CUDA(cudaEventCreate(&c->ev_end));
  PD_TRY(dev_alloc(c, &c->d_flag, 4));

  // graph: CSR pattern, values and sparse products all on the device
  PD_TRY(build_csr(c, cfg));
  adjacency_values_kernel<<<(int)ceil_div(Ntot * 32, 256), 256, 0, st>>>(c->row_ptr, c->col_idx, (int)Ntot, c->csr_val);
  PD_TRY(dev_alloc(c, &c->labels, (size_t)N, false));
  PD_TRY(dev_alloc(c, &c->mask, (size_t)N, false));
  PD_CUDA(cudaMemcpyAsync(c->labels, cfg->labels + node0, (size_t)N * 4, cudaMemcpyHostToDevice, st));
  PD_CUDA(cudaMemcpyAsync(c->mask, cfg->train_mask + node0, (size_t)N, cudaMemcpyHostToDevice, st));
  PD_CUDA(cudaStreamSynchronize(st));
  // X = [H, A~ H, A~^2 H, ...] for all nodes (a shard needs its neighbours' features, and theirs, ...); a shard then
  // keeps the rows of its own nodes
  float *x_full = nullptr;
  void *x_full_alloc = nullptr;
  if (sharded) {
    const size_t bytes = (size_t)Ntot * c->ld0 * 4 + 256;
    if (cudaMalloc(&x_full_alloc, bytes) != cudaSuccess) {
      cudaGetLastError();
      return fail(PDADMM_ENOMEM, "cudaMalloc of %zu bytes failed", bytes);
    }
    x_full = (float *)x_full_alloc;
    PD_CUDA(cudaMemsetAsync(x_full, 0, bytes, st));
  }
  struct FreeLater { void *p; ~FreeLater() { if (p) cudaFree(p); } } free_x{x_full_alloc};
  c->N = N;                                  // from here on: the nodes this context owns

  // layers
  c->layers.resize(c->L);
  int max_in = 0, max_out = 0;
  size_t max_part = 0;
  for (int l = 1; l < c->L; ++l) max_in = std::max(max_in, round_up(cfg->layer_widths[l - 1], LD_ALIGN));
  for (int l = 0; l < c->L; ++l) max_out = std::max(max_out, round_up(cfg->layer_widths[l], LD_ALIGN));
  for (int l = 0; l < c->L; ++l) {
    Layer &ly = c->layers[l];
    ly.n_in = l == 0 ? c->n0 : cfg->layer_widths[l - 1];
    ly.n_out = cfg->layer_widths[l];
    ly.ld_in = round_up(ly.n_in, LD_ALIGN); ly.ld_out = round_up(ly.n_out, LD_ALIGN);
    max_out = std::max(max_out, ly.ld_out);
    const size_t e_out = (size_t)N * ly.ld_out;
    // quantised mode: p_l and its codes trade places with the trial buffers, so all share one size
    const size_t e_in = (size_t)N * ((c->levels && l > 0) ? max_in : ly.ld_in);
    PD_TRY(dev_alloc(c, &ly.p, e_in));
    PD_TRY(dev_alloc(c, &ly.W, (size_t)ly.n_out * ly.ld_in));
    PD_TRY(dev_alloc(c, &ly.gradW, (size_t)ly.n_out * ly.ld_in));
    if (c->use_tc) {
      PD_TRY(alloc_planes(c, ly.n_out, ly.n_in, l > 0, true, &ly.Wp));     // W^T only where a p-gradient is taken
      PD_TRY(alloc_planes(c, ly.n_out, ly.n_in, false, true, &ly.Gp));
    }
    PD_TRY(dev_alloc(c, &ly.b, (size_t)ly.ld_out));
    PD_TRY(dev_alloc(c, &ly.shift, (size_t)ly.ld_out));
    PD_TRY(dev_alloc(c, &ly.z, e_out));
    // quantised mode: r_l (l >= 2) trades places with the lane's buffer for the trial's r + W d, so all have one size
    PD_TRY(dev_alloc(c, &ly.r, (c->levels && l > 0) ? (size_t)N * max_out : e_out));
    if (l + 1 < c->L) { PD_TRY(dev_alloc(c, &ly.q, e_out)); PD_TRY(dev_alloc(c, &ly.u, e_out)); }
    if (c->levels && l > 0) PD_TRY(dev_alloc(c, &ly.codes, e_in * c->code_bytes));
    if (c->int_operands && l > 0) PD_TRY(dev_alloc(c, &ly.p_plane, e_in));
    if (l > 0) PD_TRY(dev_alloc(c, &ly.t, (size_t)N * ly.ld_in));
    PD_TRY(dev_alloc(c, &ly.sc, 1));
    if (l > 0) PD_TRY(dev_alloc(c, &ly.g_exp, 1));
    PD_TRY(dev_alloc(c, &ly.amax_p, 1));
    PD_TRY(dev_alloc(c, &ly.amax_r, 1));
    PD_TRY(upload_rows(st, ly.W, ly.ld_in, cfg->init_W[l], ly.n_in, ly.n_out));
    // Node slices of the W-gradient product (slices >= 256 nodes, at most 32).  The persistent grid works through
    // tiles x slices units in rounds of n_sms, so the count is chosen to fill its last round: the smallest number
    // of slices within 3 % (relative) of the best fill (fewer slices = fewer partial tiles to write and add up).
    const int64_t tiles = ceil_div(ly.n_in, SG_BN) * ceil_div(ly.n_out, SG_BM);   // same tile for both kernels
    const int max_split = (int)std::max<int64_t>(1, std::min<int64_t>(32, ceil_div(N, 256)));
    auto slices_for = [&](int want) { return (int)ceil_div(N, round_up((int)ceil_div(N, want), TC_BK)); };
    auto fill = [&](int want) {
      const int64_t units = tiles * slices_for(want);
      return (double)units / (double)(c->n_sms * ceil_div(units, c->n_sms));
    };
    double best = 0.0;
    for (int w = 1; w <= max_split; ++w) best = std::max(best, fill(w));
    int split = 1;
    while (split < max_split && fill(split) < 0.97 * best) ++split;
    ly.k_chunk = round_up((int)ceil_div(N, split), TC_BK);      // multiple of both kernels' K blocks
    ly.n_split = (int)ceil_div(N, ly.k_chunk);
    max_part = std::max(max_part, (size_t)ly.n_split * ly.n_out * ly.ld_in);
  }
  // scratch
  Scratch &s = c->scr;
  int tr_out = 0, tr_in = 0;
  const size_t bytes_before_scratch = c->bytes_handed_out;
  const size_t e_max = (size_t)N * std::max(max_in, max_out);
  PD_TRY(dev_alloc(c, &s.s1, e_max));
  PD_TRY(dev_alloc(c, &s.s2, (size_t)N * max_out));
  if (c->levels) PD_TRY(alloc_trial_buffers(c, s, (size_t)N * max_in));
  PD_TRY(dev_alloc(c, &s.part, max_part));
  s.n_slots = std::max<size_t>((size_t)c->n_sms * 4 * max_out, 8 * (size_t)ceil_div(N, SG_BM) * ceil_div(std::max(max_in, max_out), SG_BN) + 148 * 8 * 4);
  s.n_slots *= 2;                       // two halves: consecutive reductions of one layer use different halves
  PD_TRY(dev_alloc(c, &s.slots, s.n_slots));
  PD_TRY(dev_alloc(c, &s.red, (size_t)max_out + 8));
  if (c->use_tc) {
    PD_TRY(dev_alloc(c, &s.tail_ws, (size_t)c->n_sms * TC_BM * TC_BN, false));
    PD_TRY(dev_alloc(c, &s.tail_count, (size_t)c->n_sms * 8));
    PD_TRY(dev_alloc(c, &s.amax_pool, (size_t)AMAX_POOL));
    c->ldT = round_up((int)N, 8);
    // widest r_l and p_l (l >= 2) among the layers whose product over the nodes takes its operands as planes
    for (int l = 0; l < c->L; ++l) {
      const Layer &ly = c->layers[l];
      if (!planes_beforehand(ly.n_out, ly.n_in, l == 0)) continue;
      tr_out = std::max(tr_out, ly.n_out);
      if (l > 0) tr_in = std::max(tr_in, ly.n_in);
    }
    PD_TRY(alloc_transposed(c, s, tr_out, tr_in));
    // planes of streamed operands: needed if some layer's products are at least PLANES_FROM_COL_TILES column tiles wide
    bool want_row_planes = false;
    for (int l = 0; l < c->L; ++l)
      want_row_planes |= std::max(ceil_div(c->layers[l].n_out, TC_BN), l > 0 ? ceil_div(c->layers[l].n_in, TC_BN) : 0) >= PLANES_FROM_COL_TILES;
    want_row_planes |= c->levels > 0;       // the norm-only product of the quantised update always takes a hi plane
    if (want_row_planes) PD_TRY(alloc_row_planes(c, s, e_max));
    Layer &l0 = c->layers[0];
    if (ceil_div(l0.n_out, TC_BN) >= 2) {      // X is split once for ever: worth it from two column tiles on
      PD_TRY(dev_alloc(c, &l0.x_hi, (size_t)N * l0.ld_in, false));
      PD_TRY(dev_alloc(c, &l0.x_lo, (size_t)N * l0.ld_in, false));
      PD_TRY(dev_alloc(c, &l0.x_exp, 1));
    }
    if (planes_beforehand(l0.n_out, l0.n_in, true)) {
      PD_TRY(dev_alloc(c, &l0.xT_hi, (size_t)l0.n_in * c->ldT));
      PD_TRY(dev_alloc(c, &l0.xT_lo, (size_t)l0.n_in * c->ldT));
    }
    PD_TRY(dev_alloc(c, &l0.xT_exp, 1));
  }

  // further lanes for the concurrency across layers: own stream, product outputs, partial tiles, slots.
  // Small problems are bound by the latency of their chain of launches, which only more concurrent chains shorten
  // (workload c1, 10 layers: 2 lanes 0.40 ms per iteration); large ones gain little beyond two (c2: 2 lanes 273,
  // 4 lanes 278 iterations/s) and their scratch is gigabytes per lane.  So: as many lanes as 4 GB of scratch pay for,
  // at least PDADMM_N_LANES, at most one per layer (c3, 0.4 GB per lane: 6 lanes 280, 10 lanes 301 iterations/s;
  // c4, 5.5 GB per lane: 2 lanes 9.95, 4 lanes 9.99).
  const size_t lane_bytes = std::max<size_t>(c->bytes_handed_out - bytes_before_scratch, 1);
  const int affordable = (int)std::min<size_t>(64, (size_t(4) << 30) / lane_bytes);
  const int n_lanes = (cfg->flags & PDADMM_FLAG_ONE_LANE) ? 1 : std::min(c->L, std::max(PDADMM_N_LANES, affordable));
  for (int i = 1; i < n_lanes; ++i) {
    c->more_lanes.emplace_back(new Scratch());
    Scratch &x = *c->more_lanes.back();
    PD_CUDA(cudaStreamCreateWithFlags(&x.st, cudaStreamNonBlocking));
    PD_TRY(dev_alloc(c, &x.s1, e_max));
    PD_TRY(dev_alloc(c, &x.s2, (size_t)N * max_out));
    PD_TRY(dev_alloc(c, &x.part, max_part));
    if (c->levels) PD_TRY(alloc_trial_buffers(c, x, (size_t)N * max_in));
    x.n_slots = s.n_slots;
    PD_TRY(dev_alloc(c, &x.slots, x.n_slots));
    PD_TRY(dev_alloc(c, &x.red, (size_t)max_out + 8));
    if (c->use_tc) {
      PD_TRY(dev_alloc(c, &x.tail_ws, (size_t)c->n_sms * TC_BM * TC_BN, false));
      PD_TRY(dev_alloc(c, &x.tail_count, (size_t)c->n_sms * 8));
      PD_TRY(dev_alloc(c, &x.amax_pool, (size_t)AMAX_POOL));
      PD_TRY(alloc_transposed(c, x, tr_out, tr_in));
      if (s.a_hi != nullptr) PD_TRY(alloc_row_planes(c, x, e_max));
    }
  }
  c->ev_p.resize(c->L);
  for (auto &e : c->ev_p) PD_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  c->ev_lane.resize(n_lanes);
  for (auto &e : c->ev_lane) PD_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));

  // X = [H, A~ H, A~^2 H, ...] in the column blocks of p_1
  Layer &l0 = c->layers[0];
  {
    float *xb = sharded ? x_full : l0.p;
    PD_TRY(upload_rows(st, xb, l0.ld_in, cfg->features, c->d, Ntot));
    for (int k = 1; k < c->n_blocks; ++k)
      launch_spmm(st, c->row_ptr, c->col_idx, c->csr_val, (int)Ntot, xb + (size_t)(k - 1) * c->d, xb + (size_t)k * c->d,
                  c->d, l0.ld_in);
    if (sharded)
      PD_CUDA(cudaMemcpyAsync(l0.p, x_full + (size_t)node0 * l0.ld_in, (size_t)N * l0.ld_in * 4, cudaMemcpyDeviceToDevice, st));
  }

  PD_TRY(feasible_start(c, 0));
  PD_CUDA(cudaStreamSynchronize(st));
  PD_CUDA(cudaGetLastError());
  c->r_valid = true;                        // z = W p + b exactly by construction, r = 0 (allocated as zero)
  c->w_planes_valid = true;
  c->amax_p_valid = true;
  c->xT_valid = false;            // the transposed planes of X are made by the first step
  c->launches = 0;
  c->comm_bytes = 0;
  return PDADMM_OK;
}

static void destroy(pdadmm_ctx *c) {
  if (!c) return;
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  for (auto &r : c->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
  for (auto e : c->ev_pool) cudaEventDestroy(e);
  for (void *p : c->allocs) cudaFree(p);
  if (c->h_pinned) cudaFreeHost(c->h_pinned);
  if (c->ev_begin) cudaEventDestroy(c->ev_begin);
  if (c->ev_end) cudaEventDestroy(c->ev_end);
  if (c->iter_graph) cudaGraphExecDestroy(c->iter_graph);
  for (auto e : c->ev_p) cudaEventDestroy(e);
  for (auto e : c->ev_lane) cudaEventDestroy(e);
  for (int i = 0; i <= (int)c->more_lanes.size(); ++i) {
    pd::Scratch &x = i == 0 ? c->scr : *c->more_lanes[i - 1];
    if (x.h_flag) cudaFreeHost(x.h_flag);
    if (x.ev_flag) cudaEventDestroy(x.ev_flag);
  }
  for (auto &x : c->more_lanes) if (x->st) cudaStreamDestroy(x->st);
  if (c->scr.st) cudaStreamDestroy(c->scr.st);
  delete c;
}

}  // namespace pd

// ======================================================================================================
// C ABI
// ======================================================================================================
using namespace pd;

extern "C" const char *pdadmm_last_error(void) { return err_text().c_str(); }

extern "C" int pdadmm_init(const pdadmm_config *cfg, pdadmm_ctx **out) { return pdadmm_init_sharded(cfg, nullptr, out); }

extern "C" int pdadmm_comm_bytes(pdadmm_ctx *c, int64_t *bytes) {
  if (!c || !bytes) return fail(PDADMM_EINVAL, "null argument");
  *bytes = c->comm_bytes;
  return PDADMM_OK;
}

extern "C" int pdadmm_init_sharded(const pdadmm_config *cfg, const pdadmm_shard *shard, pdadmm_ctx **out) {
  if (!out) return fail(PDADMM_EINVAL, "out is null");
  *out = nullptr;
  PD_TRY(check_config(cfg));
  if (shard != nullptr) {
    if (shard->node_begin < 0 || shard->node_count < 1 || shard->node_begin + shard->node_count > cfg->n_nodes)
      return fail(PDADMM_EINVAL, "shard [%lld, +%lld) is not inside the %lld nodes", (long long)shard->node_begin,
                  (long long)shard->node_count, (long long)cfg->n_nodes);
    if (shard->allreduce == nullptr && (shard->node_begin != 0 || shard->node_count != cfg->n_nodes))
      return fail(PDADMM_EINVAL, "a shard that is not the whole graph needs an allreduce callback");
  }
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
    cudaGetLastError();
    return fail(PDADMM_ECUDA, "no CUDA device is available");
  }
  if (cfg->device < 0 || cfg->device >= n_dev) return fail(PDADMM_EINVAL, "device %d does not exist", cfg->device);
  pdadmm_ctx *c = new (std::nothrow) pdadmm_ctx();
  if (!c) return fail(PDADMM_ENOMEM, "out of host memory");
  int rc;
  try {
    rc = build(c, cfg, shard);
  } catch (const std::bad_alloc &) {
    rc = fail(PDADMM_ENOMEM, "out of host memory");
  }
  if (rc != PDADMM_OK) { destroy(c); return rc; }
  *out = c;
  return PDADMM_OK;
}

extern "C" int pdadmm_start_layers_from(pdadmm_ctx *c, int first_layer) {
  if (!c) return fail(PDADMM_EINVAL, "context is null");
  if (first_layer < 1 || first_layer > c->L) return fail(PDADMM_EINVAL, "first_layer must be in [1, %d]", c->L);
  PD_CUDA(cudaSetDevice(c->device));
  PD_TRY(feasible_start(c, first_layer - 1));
  PD_CUDA(cudaStreamSynchronize(c->scr.st));
  PD_CUDA(cudaGetLastError());
  // the linear residual of the restarted layers is zero by construction; everything derived from the other tensors
  // (the residual of the kept layers, t, planes, largest magnitudes) is rebuilt by the next call that needs it
  c->r_valid = false; c->t_valid = false; c->w_planes_valid = false; c->amax_p_valid = false;
  return PDADMM_OK;
}

extern "C" int pdadmm_destroy(pdadmm_ctx *c) {
  destroy(c);
  return PDADMM_OK;
}

static int ensure_residual(pdadmm_ctx *c) {
  if (!c->w_planes_valid) {
    for (auto &ly : c->layers) PD_TRY(split_planes(c, c->scr.st, ly.W, ly.n_out, ly.n_in, ly.ld_in, ly.Wp));
    c->w_planes_valid = true;
  }
  if (!c->amax_p_valid) {
    for (auto &ly : c->layers) {
      const size_t n4 = (size_t)c->N * ly.ld_in / 4;
      PD_CUDA(cudaMemsetAsync(ly.amax_p, 0, sizeof(uint32_t), c->scr.st));
      Launch k(c, KC_AMAX, c->scr.st, 16.0 * n4, 0);
      absmax_kernel<<<ew_grid(n4), EW_THREADS, 0, c->scr.st>>>(ly.p, n4, ly.amax_p);
    }
    c->amax_p_valid = true;
  }
  if (!c->xT_valid && c->use_tc) {          // both kinds of planes of X follow the stored X
    Layer &l0 = c->layers[0];
    if (planes_beforehand(l0.n_out, l0.n_in, true))
      transpose_planes(c, c->scr.st, l0.p, (int)c->N, l0.n_in, l0.ld_in, l0.amax_p, l0.xT_hi, l0.xT_lo, c->ldT, l0.xT_exp);
    if (l0.x_hi != nullptr) {
      const size_t n8 = (size_t)c->N * l0.ld_in / 8;
      Launch k(c, KC_PLANES, c->scr.st, 8.0 * c->N * l0.n_in, 0);
      rows_planes_kernel<<<ew_grid(n8), 256, 0, c->scr.st>>>(l0.p, n8, l0.amax_p, l0.x_exp, l0.x_hi, l0.x_lo);
    }
    c->xT_valid = true;
  }
  if (!c->t_valid) {
    for (int l = 1; l < c->L; ++l) {
      Layer &ly = c->layers[l];
      const Layer &pv = c->layers[l - 1];
      const size_t n4 = (size_t)c->N * ly.ld_in / 4;
      Launch k(c, KC_AXPY, c->scr.st, 16.0 * c->N * ly.n_in, 0);
      gradp_const_kernel<<<ew_grid(n4), EW_THREADS, 0, c->scr.st>>>(pv.u, ly.p, pv.q, c->rho, ly.t, n4);
    }
    c->t_valid = true;
  }
  if (c->r_valid) return PDADMM_OK;
  for (int l = 0; l < c->L; ++l) PD_TRY(refresh_residual(c, c->layers[l], c->scr.st));
  c->r_valid = true;
  return PDADMM_OK;
}

extern "C" int pdadmm_step(pdadmm_ctx *c, int n_iters) {
  if (!c) return fail(PDADMM_EINVAL, "context is null");
  if (n_iters < 0) return fail(PDADMM_EINVAL, "n_iters is negative");
  PD_CUDA(cudaSetDevice(c->device));
  PD_CUDA(cudaEventRecord(c->ev_begin, c->scr.st));
  PD_CUDA(cudaMemsetAsync(c->d_flag, 0, 3 * sizeof(int), c->scr.st));
  PD_TRY(ensure_residual(c));
  bool hit_cap = false;
  // pdADMM-G has no host decision inside an iteration, so after a first eager iteration the sequence of launches
  // is captured once into a CUDA graph and replayed; pointers and tensor maps never change in that mode.
  // pdADMM-G-Q reads the accept flag of every tau trial on the host, and per-kernel timing needs its events:
  // both stay eager.
  // A sharded context calls back for its sums over shards in the middle of an iteration: eager as well.
  const bool may_graph = c->levels == 0 && !c->profiling && !c->graph_failed && !(c->flags & PDADMM_FLAG_NO_GRAPH) &&
                         c->reduce == nullptr;
  int k = 0;
  if (may_graph && c->iter_graph == nullptr && n_iters > 1) {
    PD_TRY(iterate_once(c, &hit_cap));
    ++k;
    const int64_t before = c->launches;
    cudaGraph_t g = nullptr;
    if (cudaStreamBeginCapture(c->scr.st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
      const int rc = iterate_once(c, &hit_cap);
      const cudaError_t e = cudaStreamEndCapture(c->scr.st, &g);
      if (rc != PDADMM_OK || e != cudaSuccess || cudaGraphInstantiate(&c->iter_graph, g, 0) != cudaSuccess) {
        c->iter_graph = nullptr;
        c->graph_failed = true;
      }
      if (g) cudaGraphDestroy(g);
    } else {
      c->graph_failed = true;
    }
    cudaGetLastError();
    c->iter_graph_launches = c->launches - before;
    c->launches = before;                       // capturing launched nothing
  }
  for (; k < n_iters; ++k) {
    if (may_graph && c->iter_graph != nullptr) {
      PD_CUDA(cudaGraphLaunch(c->iter_graph, c->scr.st));
      c->launches += c->iter_graph_launches;
    } else {
      PD_TRY(iterate_once(c, &hit_cap));
    }
  }
  PD_CUDA(cudaMemcpyAsync(c->h_pinned + 8, c->d_flag, 3 * sizeof(int), cudaMemcpyDeviceToHost, c->scr.st));
  PD_CUDA(cudaEventRecord(c->ev_end, c->scr.st));
  PD_CUDA(cudaStreamSynchronize(c->scr.st));
  PD_CUDA(cudaGetLastError());
  {
    float ms = 0.f;
    PD_CUDA(cudaEventElapsedTime(&ms, c->ev_begin, c->ev_end));
    c->last_step_ms = ms;
  }
  if (c->profiling) PD_TRY(prof_collect(c));
  if (c->h_pinned[9] != 0) return fail(PDADMM_ETIMEOUT, "a bounded wait inside a tensor-core product expired");
  if (c->h_pinned[10] != 0) return fail(PDADMM_ENUMERIC, "a non-finite value reached the gradient norms: the state holds NaN or Inf");
  if (c->h_pinned[8] != 0)
    return fail(PDADMM_ENOTCONV, "the last-layer z solver did not converge on %d nodes", c->h_pinned[8]);
  if (hit_cap) return fail(PDADMM_ENOTCONV, "the tau search of a quantised p-update reached its trial cap");
  return PDADMM_OK;
}

static int read_slots(pdadmm_ctx *c, int n_slots, int stride, int n_out, double *host) {
  double *dst = c->scr.slots + c->scr.n_slots - 8;            // tail of the slot buffer: results
  reduce_slots_kernel<<<1, 256, 0, c->scr.st>>>(c->scr.slots, n_slots, stride, n_out, dst);
  PD_CUDA(cudaMemcpyAsync(host, dst, n_out * sizeof(double), cudaMemcpyDeviceToHost, c->scr.st));
  PD_CUDA(cudaStreamSynchronize(c->scr.st));
  return PDADMM_OK;
}

extern "C" int pdadmm_objective(pdadmm_ctx *c, double out[6]) {
  if (!c || !out) return fail(PDADMM_EINVAL, "null argument");
  PD_CUDA(cudaSetDevice(c->device));
  PD_TRY(ensure_residual(c));
  cudaStream_t st = c->scr.st;
  double lin = 0, act = 0, dual = 0, pen = 0, R = 0;
  for (int l = 0; l < c->L; ++l) {
    Layer &ly = c->layers[l];
    const size_t n = (size_t)c->N * ly.ld_out;
    const int grid = std::min(ew_grid(n), 512);
    const bool hidden = l + 1 < c->L;
    objective_layer_kernel<<<grid, EW_THREADS, 0, st>>>(ly.r, ly.z, hidden ? ly.q : nullptr, ly.u,
                                                       hidden ? c->layers[l + 1].p : nullptr, n, c->slope, c->scr.slots);
    double h[4];
    PD_TRY(read_slots(c, grid, 4, 4, h));
    lin += h[0]; act += h[1]; dual += h[2]; pen += h[3];
  }
  {
    Layer &ly = c->layers[c->L - 1];
    const int grid = (int)std::min<int64_t>(512, ceil_div(c->N, EW_THREADS));
    risk_kernel<<<grid, EW_THREADS, 0, st>>>(ly.z, c->labels, c->mask, (int)c->N, ly.n_out, ly.ld_out, c->scr.slots,
                                             c->ls_risk ? 1 : 0);
    PD_TRY(read_slots(c, grid, 1, 1, &R));
  }
  PD_CUDA(cudaGetLastError());
  if (c->reduce != nullptr) {                 // every component is a sum over nodes
    double h[5] = {R, lin, act, dual, pen};
    PD_CUDA(cudaMemcpyAsync(c->scr.red, h, sizeof h, cudaMemcpyHostToDevice, st));
    PD_TRY(shard_sum(c, st, c->scr.red, 5, 1));
    PD_CUDA(cudaMemcpyAsync(h, c->scr.red, sizeof h, cudaMemcpyDeviceToHost, st));
    PD_CUDA(cudaStreamSynchronize(st));
    R = h[0]; lin = h[1]; act = h[2]; dual = h[3]; pen = h[4];
  }
  out[0] = R; out[1] = 0.5 * c->nu * lin; out[2] = 0.5 * c->nu * act; out[3] = dual; out[4] = 0.5 * c->rho * pen;
  out[5] = out[0] + out[1] + out[2] + out[3] + out[4];
  return PDADMM_OK;
}

extern "C" int pdadmm_predict(pdadmm_ctx *c, float *logits_out, int32_t *pred_out, int64_t counts_out[4]) {
  if (!c) return fail(PDADMM_EINVAL, "context is null");
  PD_CUDA(cudaSetDevice(c->device));
  cudaStream_t st = c->scr.st;
  if (!c->w_planes_valid) {
    for (auto &ly : c->layers) PD_TRY(split_planes(c, st, ly.W, ly.n_out, ly.n_in, ly.ld_in, ly.Wp));
    c->w_planes_valid = true;
  }
  // forward pass with the constraints enforced: activations alternate between the two scratch matrices
  const int N = (int)c->N;
  const float *in = c->layers[0].p;
  float *bufs[2] = {c->scr.s1, c->scr.s2};
  float *out = nullptr;
  const uint32_t *w_in = nullptr;            // max|activations| of the layer's input
  if (c->use_tc) {
    PD_TRY(amax_reset(c, st));               // one word per layer output, all from one pass through the pool
    w_in = amax_of(c, st, in, (size_t)N * c->layers[0].ld_in / 4);
  }
  for (int l = 0; l < c->L; ++l) {
    Layer &ly = c->layers[l];
    out = bufs[l & 1];
    uint32_t *w_out = nullptr;
    if (c->use_tc) w_out = amax_take(c);
    EpiBiasAct epi{out, ly.ld_out, ly.b, l + 1 < c->L ? 1 : 0, c->slope, w_out};
    // the first layer's input is X: its planes are kept by the context while they match the stored X
    const PlaneRef xp = (l == 0 && c->xT_valid) ? planes_X(ly) : PlaneRef{nullptr, nullptr, 0, nullptr};
    PD_TRY(gemm_nodes<false>(c, KC_GEMM_RESID, st, N, ly.n_out, ly.n_in, in, ly.ld_in, ly.W, ly.ld_in, planes_W(ly),
                             epi, nullptr, nullptr, 0, w_in, &xp));
    w_in = w_out;
    in = out;
  }
  const Layer &last = c->layers[c->L - 1];
  int *d_pred = reinterpret_cast<int *>(bufs[c->L & 1]);              // the scratch matrix the logits are not in
  unsigned long long *d_counts = reinterpret_cast<unsigned long long *>(c->scr.slots);
  PD_CUDA(cudaMemsetAsync(d_counts, 0, 4 * sizeof(unsigned long long), st));
  argmax_kernel<<<(int)std::min<int64_t>(1184, ceil_div(N, EW_THREADS)), EW_THREADS, 0, st>>>(
      out, c->labels, c->mask, N, last.n_out, last.ld_out, d_pred, d_counts);
  PD_CUDA(cudaGetLastError());
  if (logits_out)
    PD_CUDA(cudaMemcpy2DAsync(logits_out, (size_t)last.n_out * 4, out, (size_t)last.ld_out * 4, (size_t)last.n_out * 4,
                              (size_t)N, cudaMemcpyDeviceToHost, st));
  if (pred_out) PD_CUDA(cudaMemcpyAsync(pred_out, d_pred, (size_t)N * 4, cudaMemcpyDeviceToHost, st));
  unsigned long long h_counts[4];
  PD_CUDA(cudaMemcpyAsync(h_counts, d_counts, sizeof(h_counts), cudaMemcpyDeviceToHost, st));
  PD_CUDA(cudaStreamSynchronize(st));
  if (counts_out)
    for (int i = 0; i < 4; ++i) counts_out[i] = (int64_t)h_counts[i];
  int h_err = 0;
  PD_CUDA(cudaMemcpy(&h_err, c->d_flag + 1, 4, cudaMemcpyDeviceToHost));
  if (h_err) return fail(PDADMM_ETIMEOUT, "a bounded wait inside a tensor-core product expired");
  return PDADMM_OK;
}

extern "C" int pdadmm_residuals(pdadmm_ctx *c, double *per_layer_sq, int n) {
  if (!c) return fail(PDADMM_EINVAL, "context is null");
  if (n != c->L - 1 || (n > 0 && !per_layer_sq)) return fail(PDADMM_EINVAL, "n must be L-1 = %d", c->L - 1);
  PD_CUDA(cudaSetDevice(c->device));
  PD_TRY(ensure_residual(c));
  for (int l = 0; l + 1 < c->L; ++l) {
    Layer &ly = c->layers[l];
    const size_t nn = (size_t)c->N * ly.ld_out;
    const int grid = std::min(ew_grid(nn), 512);
    objective_layer_kernel<<<grid, EW_THREADS, 0, c->scr.st>>>(ly.r, ly.z, ly.q, ly.u, c->layers[l + 1].p, nn,
                                                              c->slope, c->scr.slots);
    double h[4];
    PD_TRY(read_slots(c, grid, 4, 4, h));
    per_layer_sq[l] = h[3];
  }
  PD_CUDA(cudaGetLastError());
  if (c->reduce != nullptr && n > 0) {
    if ((size_t)n > 8 + (size_t)c->layers[0].ld_out) return fail(PDADMM_EINVAL, "too many layers for the reduction buffer");
    PD_CUDA(cudaMemcpyAsync(c->scr.red, per_layer_sq, (size_t)n * 8, cudaMemcpyHostToDevice, c->scr.st));
    PD_TRY(shard_sum(c, c->scr.st, c->scr.red, (size_t)n, 1));
    PD_CUDA(cudaMemcpyAsync(per_layer_sq, c->scr.red, (size_t)n * 8, cudaMemcpyDeviceToHost, c->scr.st));
    PD_CUDA(cudaStreamSynchronize(c->scr.st));
  }
  return PDADMM_OK;
}

// ---- tensors in and out -------------------------------------------------------------------------------------
struct TensorRef { void *ptr; size_t rows, width, ld, elem; bool settable; };

static int locate(pdadmm_ctx *c, int kind, int layer, TensorRef *t) {
  const int L = c->L;
  auto need = [&](int lo, int hi) {
    return (layer >= lo && layer <= hi) ? PDADMM_OK
                                        : fail(PDADMM_EINVAL, "layer %d is outside [%d, %d] for tensor kind %d", layer, lo, hi, kind);
  };
  const size_t N = (size_t)c->N;
  switch (kind) {
    case PDADMM_T_X: { Layer &y = c->layers[0]; *t = {y.p, N, (size_t)y.n_in, (size_t)y.ld_in, 4, true}; return PDADMM_OK; }
    case PDADMM_T_P: { PD_TRY(need(1, L)); Layer &y = c->layers[layer - 1]; *t = {y.p, N, (size_t)y.n_in, (size_t)y.ld_in, 4, true}; return PDADMM_OK; }
    case PDADMM_T_W: { PD_TRY(need(1, L)); Layer &y = c->layers[layer - 1]; *t = {y.W, (size_t)y.n_out, (size_t)y.n_in, (size_t)y.ld_in, 4, true}; return PDADMM_OK; }
    case PDADMM_T_B: { PD_TRY(need(1, L)); Layer &y = c->layers[layer - 1]; *t = {y.b, 1, (size_t)y.n_out, (size_t)y.ld_out, 4, true}; return PDADMM_OK; }
    case PDADMM_T_Z: { PD_TRY(need(1, L)); Layer &y = c->layers[layer - 1]; *t = {y.z, N, (size_t)y.n_out, (size_t)y.ld_out, 4, true}; return PDADMM_OK; }
    case PDADMM_T_Q: { PD_TRY(need(1, L - 1)); Layer &y = c->layers[layer - 1]; *t = {y.q, N, (size_t)y.n_out, (size_t)y.ld_out, 4, true}; return PDADMM_OK; }
    case PDADMM_T_U: { PD_TRY(need(1, L - 1)); Layer &y = c->layers[layer - 1]; *t = {y.u, N, (size_t)y.n_out, (size_t)y.ld_out, 4, true}; return PDADMM_OK; }
    case PDADMM_T_CODES: {
      if (!c->levels) return fail(PDADMM_EINVAL, "codes exist only in quantised mode");
      PD_TRY(need(2, L)); Layer &y = c->layers[layer - 1];
      *t = {y.codes, N, (size_t)y.n_in, (size_t)y.ld_in, (size_t)c->code_bytes, false}; return PDADMM_OK;
    }
    case PDADMM_T_TAU: { PD_TRY(need(2, L)); *t = {&c->layers[layer - 1].sc->tau, 1, 1, 1, 8, false}; return PDADMM_OK; }
    case PDADMM_T_THETA: { PD_TRY(need(1, L)); *t = {&c->layers[layer - 1].sc->theta, 1, 1, 1, 8, false}; return PDADMM_OK; }
    case PDADMM_T_TRIALS: { PD_TRY(need(2, L)); *t = {&c->layers[layer - 1].sc->trials, 1, 1, 1, 4, false}; return PDADMM_OK; }
    case PDADMM_T_CSR_ROWPTR: *t = {c->row_ptr, 1, (size_t)c->N_total + 1, (size_t)c->N_total + 1, 4, false}; return PDADMM_OK;
    case PDADMM_T_CSR_COLIDX: *t = {c->col_idx, 1, (size_t)c->nnz, (size_t)c->nnz, 4, false}; return PDADMM_OK;
    case PDADMM_T_CSR_VAL: *t = {c->csr_val, 1, (size_t)c->nnz, (size_t)c->nnz, 4, false}; return PDADMM_OK;
    default: return fail(PDADMM_EINVAL, "unknown tensor kind %d", kind);
  }
}

extern "C" int pdadmm_get_tensor(pdadmm_ctx *c, int kind, int layer, void *host_dst, size_t bytes) {
  if (!c || !host_dst) return fail(PDADMM_EINVAL, "null argument");
  PD_CUDA(cudaSetDevice(c->device));
  if (kind == PDADMM_T_QSCALE) {
    if (layer < 2 || layer > c->L || bytes != 4) return fail(PDADMM_EINVAL, "QSCALE: layer in [2, L], 4 bytes");
    memcpy(host_dst, &c->layers[layer - 1].scale, 4);
    return PDADMM_OK;
  }
  TensorRef t;
  PD_TRY(locate(c, kind, layer, &t));
  if (bytes != t.rows * t.width * t.elem)
    return fail(PDADMM_EINVAL, "tensor kind %d layer %d has %zu bytes, caller passed %zu", kind, layer,
                t.rows * t.width * t.elem, bytes);
  PD_CUDA(cudaMemcpy2DAsync(host_dst, t.width * t.elem, t.ptr, t.ld * t.elem, t.width * t.elem, t.rows,
                            cudaMemcpyDeviceToHost, c->scr.st));
  PD_CUDA(cudaStreamSynchronize(c->scr.st));
  return PDADMM_OK;
}

// pdADMM-G-Q: the kernels read p_l (l >= 2, paper numbering) as its codes, so the two must always agree: the codes
// are taken from p_l and p_l becomes the levels of those codes (the same bits if it was on the level set already).
static int project_p_on_its_levels(pdadmm_ctx *c, int layer) {
  Layer &y = c->layers[layer - 1];
  const size_t n = (size_t)c->N * y.ld_in;
  quantize_kernel<<<ew_grid(n), EW_THREADS, 0, c->scr.st>>>(y.p, n, y.scale, y.lo, c->levels, y.p, y.codes, c->code_bytes == 2);
  if (c->int_operands) codes_to_plane_kernel<<<ew_grid(n / 4), EW_THREADS, 0, c->scr.st>>>(y.codes, c->code_bytes == 2, n / 4, y.p_plane);
  PD_CUDA(cudaGetLastError());
  PD_CUDA(cudaStreamSynchronize(c->scr.st));
  c->r_valid = false;
  c->amax_p_valid = false;
  c->t_valid = false;
  return PDADMM_OK;
}

extern "C" int pdadmm_set_tensor(pdadmm_ctx *c, int kind, int layer, const void *host_src, size_t bytes) {
  if (!c || !host_src) return fail(PDADMM_EINVAL, "null argument");
  PD_CUDA(cudaSetDevice(c->device));
  if (kind == PDADMM_T_QSCALE) {
    if (layer < 2 || layer > c->L || bytes != 4) return fail(PDADMM_EINVAL, "QSCALE: layer in [2, L], 4 bytes");
    float v;
    memcpy(&v, host_src, 4);
    if (!(v > 0.f)) return fail(PDADMM_EINVAL, "QSCALE must be positive");
    c->layers[layer - 1].scale = v;
    c->layers[layer - 1].lo = -(float)c->neg_levels * v;
    if (c->levels) PD_TRY(project_p_on_its_levels(c, layer));       // p_l moves to the new level set
    return PDADMM_OK;
  }
  TensorRef t;
  PD_TRY(locate(c, kind, layer, &t));
  if (!t.settable) return fail(PDADMM_EINVAL, "tensor kind %d is read-only", kind);
  if (bytes != t.rows * t.width * t.elem)
    return fail(PDADMM_EINVAL, "tensor kind %d layer %d has %zu bytes, caller passed %zu", kind, layer,
                t.rows * t.width * t.elem, bytes);
  PD_CUDA(cudaMemcpy2DAsync(t.ptr, t.ld * t.elem, host_src, t.width * t.elem, t.width * t.elem, t.rows,
                            cudaMemcpyHostToDevice, c->scr.st));
  PD_CUDA(cudaStreamSynchronize(c->scr.st));
  if (kind == PDADMM_T_X || kind == PDADMM_T_P || kind == PDADMM_T_W || kind == PDADMM_T_B || kind == PDADMM_T_Z)
    c->r_valid = false;
  if (kind == PDADMM_T_W) c->w_planes_valid = false;
  if (kind == PDADMM_T_X || kind == PDADMM_T_P) c->amax_p_valid = false;
  if (kind == PDADMM_T_X || (kind == PDADMM_T_P && layer == 1)) c->xT_valid = false;
  if (kind == PDADMM_T_P || kind == PDADMM_T_Q || kind == PDADMM_T_U) c->t_valid = false;
  if (kind == PDADMM_T_P && c->levels && layer >= 2) PD_TRY(project_p_on_its_levels(c, layer));
  return PDADMM_OK;
}

// ---- stand-alone entry points for single kernels ------------------------------------------------------------------
extern "C" int pdadmm_quantize(int device, const float *x, size_t n, float scale, float lo, int levels, void *codes_out,
                               float *p_out) {
  if (!x && n) return fail(PDADMM_EINVAL, "x is null");
  if (levels < 2 || levels > 65536 || !(scale > 0.f)) return fail(PDADMM_EINVAL, "levels in [2,65536], scale > 0");
  const size_t code_bytes = levels > 256 ? 2 : 1;
  if (n == 0) return PDADMM_OK;
  PD_CUDA(cudaSetDevice(device));
  float *dx = nullptr, *dp = nullptr;
  uint8_t *dc = nullptr;
  int rc = PDADMM_OK;
  auto body = [&]() -> int {
    PD_CUDA(cudaMalloc((void **)&dx, n * 4));
    PD_CUDA(cudaMalloc((void **)&dp, n * 4));
    PD_CUDA(cudaMalloc((void **)&dc, n * code_bytes));
    PD_CUDA(cudaMemcpy(dx, x, n * 4, cudaMemcpyHostToDevice));
    quantize_kernel<<<ew_grid(n), EW_THREADS>>>(dx, n, scale, lo, levels, dp, dc, code_bytes == 2);
    PD_CUDA(cudaGetLastError());
    PD_CUDA(cudaDeviceSynchronize());
    if (p_out) PD_CUDA(cudaMemcpy(p_out, dp, n * 4, cudaMemcpyDeviceToHost));
    if (codes_out) PD_CUDA(cudaMemcpy(codes_out, dc, n * code_bytes, cudaMemcpyDeviceToHost));
    return PDADMM_OK;
  };
  rc = body();
  cudaFree(dx); cudaFree(dp); cudaFree(dc);
  return rc;
}

extern "C" int pdadmm_spmm(int device, int64_t n_rows, const int32_t *row_ptr, const int32_t *col_idx, const float *val,
                           const float *x, int32_t width, float *y_out) {
  if (n_rows < 0 || width < 1 || !row_ptr || !y_out || !x) return fail(PDADMM_EINVAL, "bad argument");
  if (n_rows == 0) return PDADMM_OK;
  if (n_rows > INT32_MAX / 2) return fail(PDADMM_EINVAL, "too many rows");
  if (row_ptr[0] != 0) return fail(PDADMM_EINVAL, "row_ptr[0] must be 0");
  for (int64_t i = 0; i < n_rows; ++i)
    if (row_ptr[i + 1] < row_ptr[i]) return fail(PDADMM_EINVAL, "row_ptr decreases at row %lld", (long long)i);
  const int64_t nnz = row_ptr[n_rows];
  if (nnz > 0 && (!col_idx || !val)) return fail(PDADMM_EINVAL, "col_idx or val is null");
  for (int64_t e = 0; e < nnz; ++e)
    if (col_idx[e] < 0 || col_idx[e] >= n_rows) return fail(PDADMM_EINVAL, "column index %lld out of range", (long long)e);
  PD_CUDA(cudaSetDevice(device));
  int *drp = nullptr, *dci = nullptr;
  float *dv = nullptr, *dx = nullptr, *dy = nullptr;
  auto body = [&]() -> int {
    PD_CUDA(cudaMalloc((void **)&drp, (n_rows + 1) * 4));
    PD_CUDA(cudaMalloc((void **)&dci, std::max<int64_t>(nnz, 1) * 4));
    PD_CUDA(cudaMalloc((void **)&dv, std::max<int64_t>(nnz, 1) * 4));
    PD_CUDA(cudaMalloc((void **)&dx, (size_t)n_rows * width * 4));
    PD_CUDA(cudaMalloc((void **)&dy, (size_t)n_rows * width * 4));
    PD_CUDA(cudaMemcpy(drp, row_ptr, (n_rows + 1) * 4, cudaMemcpyHostToDevice));
    if (nnz) {
      PD_CUDA(cudaMemcpy(dci, col_idx, nnz * 4, cudaMemcpyHostToDevice));
      PD_CUDA(cudaMemcpy(dv, val, nnz * 4, cudaMemcpyHostToDevice));
    }
    PD_CUDA(cudaMemcpy(dx, x, (size_t)n_rows * width * 4, cudaMemcpyHostToDevice));
    launch_spmm(0, drp, dci, dv, (int)n_rows, dx, dy, width, width);
    PD_CUDA(cudaGetLastError());
    PD_CUDA(cudaDeviceSynchronize());
    PD_CUDA(cudaMemcpy(y_out, dy, (size_t)n_rows * width * 4, cudaMemcpyDeviceToHost));
    return PDADMM_OK;
  };
  const int rc = body();
  cudaFree(drp); cudaFree(dci); cudaFree(dv); cudaFree(dx); cudaFree(dy);
  return rc;
}

extern "C" int pdadmm_matmul(int device, int mode, int M, int N, int K, const float *A, const float *B, float *C,
                             double *sumsq, uint32_t flags) {
  if (mode < 0 || mode > 2 || M < 1 || N < 1 || K < 1 || !A || !B || !C) return fail(PDADMM_EINVAL, "bad argument");
  PD_CUDA(cudaSetDevice(device));
  pdadmm_ctx *c = new (std::nothrow) pdadmm_ctx();
  if (!c) return fail(PDADMM_ENOMEM, "out of host memory");
  c->device = device;
  c->use_tc = (flags & PDADMM_FLAG_SIMT_GEMM) == 0;
  auto body = [&]() -> int {
    PD_CUDA(cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, device));
    PD_CUDA(cudaStreamCreateWithFlags(&c->scr.st, cudaStreamNonBlocking));
    cudaStream_t st = c->scr.st;
    PD_TRY(dev_alloc(c, &c->d_flag, 4));
    if (c->use_tc) {
      PD_TRY(dev_alloc(c, &c->scr.tail_ws, (size_t)c->n_sms * TC_BM * TC_BN, false));
      PD_TRY(dev_alloc(c, &c->scr.tail_count, (size_t)c->n_sms * 8));
    }
    // operand shapes as stored: rows x cols
    const int a_rows = mode == 2 ? K : M, a_cols = mode == 2 ? M : K;
    const int b_rows = mode == 0 ? N : K, b_cols = mode == 0 ? K : N;
    const int lda = round_up(a_cols, mode == 2 ? 4 : 8), ldb = round_up(b_cols, 4), ldc = round_up(N, 4);
    float *dA, *dB, *dC, *part = nullptr;
    double *slots;
    Planes Bp;
    PD_TRY(dev_alloc(c, &dA, (size_t)a_rows * lda));
    PD_TRY(dev_alloc(c, &dB, (size_t)b_rows * ldb));
    PD_TRY(dev_alloc(c, &dC, (size_t)M * ldc));
    const int n_slots = 8 * (int)(ceil_div(M, 128) * ceil_div(N, 128)) + 2048;
    PD_TRY(dev_alloc(c, &slots, (size_t)n_slots));
    PD_TRY(upload_rows(st, dA, lda, A, a_cols, a_rows));
    PD_TRY(upload_rows(st, dB, ldb, B, b_cols, b_rows));
    if (c->use_tc) {
      PD_TRY(dev_alloc(c, &c->scr.amax_pool, (size_t)AMAX_POOL));
      // planes of B as [N][K]: B itself in mode 0, its transpose in mode 1
      if (mode != 2) PD_TRY(alloc_planes(c, b_rows, b_cols, mode == 1, mode == 0, &Bp));
      if (mode != 2) PD_TRY(split_planes(c, st, dB, b_rows, b_cols, ldb, Bp));
      if (mode != 2) PD_TRY(alloc_row_planes(c, c->scr, (size_t)a_rows * lda));     // used from four column tiles on
    }
    int np = 0;
    if (mode == 0) {
      EpiStoreSumsq epi{dC, ldc};
      PD_TRY(gemm_nodes<false>(c, KC_GEMM_WG, st, M, N, K, dA, lda, dB, ldb, PlaneRef{Bp.hi, Bp.lo, Bp.ldh, Bp.exp}, epi,
                               slots, &np, 0));
    } else if (mode == 1) {
      EpiStoreSumsq epi{dC, ldc};
      PD_TRY(gemm_nodes<true>(c, KC_GEMM_WG, st, M, N, K, dA, lda, dB, ldb, PlaneRef{Bp.hiT, Bp.loT, Bp.ldhT, Bp.exp}, epi,
                              slots, &np, 0));
    } else {
      const int split = (int)std::max<int64_t>(1, std::min<int64_t>(8, ceil_div(K, 64)));
      const int k_chunk = round_up((int)ceil_div(K, split), TC_BK);
      const int n_split = (int)ceil_div(K, k_chunk);
      PD_TRY(dev_alloc(c, &part, (size_t)n_split * M * ldc));
      if (!c->use_tc) {
        dim3 grid((unsigned)ceil_div(N, SG_BN), (unsigned)ceil_div(M, SG_BM), (unsigned)n_split);
        gemm_tn_kernel<<<grid, SG_THREADS, 0, st>>>(M, N, K, k_chunk, dA, lda, dB, ldb, part, ldc);
      } else {
        if (!planes_beforehand(M, N, false)) {
          PD_TRY(amax_reserve(c, st, 2));
          const uint32_t *wa = amax_of(c, st, dA, (size_t)K * lda / 4), *wb = amax_of(c, st, dB, (size_t)K * ldb / 4);
          PD_TRY(gemm_over_nodes_raw(c, KC_GEMM_GRADW, st, M, N, K, dA, lda, dB, ldb, part, ldc, k_chunk, n_split, wa, wb));
        } else {
        // transposed planes of both operands, then the contraction over their rows
        const int ldT = round_up(K, 8);
        __half *ah, *al, *bh, *bl;
        int *ea, *eb;
        PD_TRY(dev_alloc(c, &ah, (size_t)M * ldT)); PD_TRY(dev_alloc(c, &al, (size_t)M * ldT));
        PD_TRY(dev_alloc(c, &bh, (size_t)N * ldT)); PD_TRY(dev_alloc(c, &bl, (size_t)N * ldT));
        PD_TRY(dev_alloc(c, &ea, 1)); PD_TRY(dev_alloc(c, &eb, 1));
        PD_TRY(amax_reserve(c, st, 2));
        const uint32_t *wa = amax_of(c, st, dA, (size_t)K * lda / 4), *wb = amax_of(c, st, dB, (size_t)K * ldb / 4);
        transpose_planes(c, st, dA, K, M, lda, wa, ah, al, ldT, ea);
        transpose_planes(c, st, dB, K, N, ldb, wb, bh, bl, ldT, eb);
        PD_TRY(gemm_over_nodes_tc(c, KC_GEMM_GRADW, st, M, N, K, PlaneRef{ah, al, ldT, ea}, PlaneRef{bh, bl, ldT, eb}, part,
                                  ldc, k_chunk, n_split));
        }
      }
      const size_t n4 = (size_t)M * ldc / 4;
      np = ew_grid(n4);
      reduce_gradW_kernel<<<np, EW_THREADS, 0, st>>>(part, n_split, n4, 1.0f, dC, nullptr, slots);
    }
    double *res = slots + n_slots - 1;
    reduce_slots_kernel<<<1, 256, 0, st>>>(slots, np, 1, 1, res);
    double h = 0;
    PD_CUDA(cudaMemcpyAsync(&h, res, 8, cudaMemcpyDeviceToHost, st));
    PD_CUDA(cudaMemcpy2DAsync(C, (size_t)N * 4, dC, (size_t)ldc * 4, (size_t)N * 4, (size_t)M, cudaMemcpyDeviceToHost, st));
    int err = 0;
    PD_CUDA(cudaMemcpyAsync(&err, c->d_flag + 1, 4, cudaMemcpyDeviceToHost, st));
    PD_CUDA(cudaStreamSynchronize(st));
    PD_CUDA(cudaGetLastError());
    if (sumsq) *sumsq = h;
    if (err) return fail(PDADMM_ETIMEOUT, "a bounded wait inside a tensor-core product expired");
    return PDADMM_OK;
  };
  const int rc = body();
  destroy(c);
  return rc;
}

// ---- self-test of the bounded waits ------------------------------------------------------------------------------
namespace pd {
// One warp waits, with the products' own wait routine, on an mbarrier that nothing ever arrives at.  The wait gives up
// after `limit_cycles`, raises the block's abort flag, and the block reports through the same error word as the
// products and returns by itself.
__global__ void bounded_wait_selftest_kernel(long long limit_cycles, int *error, long long *waited) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  volatile int *abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    const bool ok = ptx::mbar_wait(&bar, 0, abort_flag, limit_cycles);
    *waited = clock64() - t0;
    if (!ok) atomicExch(error, 1);
  }
}
}  // namespace pd

extern "C" int pdadmm_selftest_bounded_wait(int device, long long limit_cycles, long long *waited_cycles) {
  if (limit_cycles < 1 || limit_cycles > 100000000ll) return fail(PDADMM_EINVAL, "limit_cycles must be in [1, 1e8]");
  PD_CUDA(cudaSetDevice(device));
  int *d_err = nullptr;
  auto body = [&]() -> int {
    PD_CUDA(cudaMalloc((void **)&d_err, 16));
    PD_CUDA(cudaMemset(d_err, 0, 16));
    bounded_wait_selftest_kernel<<<1, 32>>>(limit_cycles, d_err, reinterpret_cast<long long *>(d_err) + 1);
    PD_CUDA(cudaGetLastError());
    PD_CUDA(cudaDeviceSynchronize());
    long long h[2] = {0, 0};
    PD_CUDA(cudaMemcpy(h, d_err, 16, cudaMemcpyDeviceToHost));
    if (waited_cycles) *waited_cycles = h[1];
    if ((int)h[0] != 0) return fail(PDADMM_ETIMEOUT, "a bounded device-side wait expired after %lld cycles", h[1]);
    return PDADMM_OK;
  };
  const int rc = body();
  cudaFree(d_err);
  return rc;
}

// ---- timing ----------------------------------------------------------------------------------------------------
extern "C" int pdadmm_profile(pdadmm_ctx *c, int enable) {
  if (!c) return fail(PDADMM_EINVAL, "context is null");
  PD_CUDA(cudaSetDevice(c->device));
  PD_TRY(prof_collect(c));
  for (int k = 0; k < KC_COUNT; ++k) { c->prof_ms[k] = 0; c->prof_n[k] = 0; c->prof_bytes[k] = 0; c->prof_flops[k] = 0; }
  c->profiling = enable != 0;
  return PDADMM_OK;
}
extern "C" int pdadmm_profile_classes(void) { return KC_COUNT; }
extern "C" const char *pdadmm_profile_name(int k) { return (k >= 0 && k < KC_COUNT) ? kclass_names[k] : ""; }
extern "C" int pdadmm_profile_read(pdadmm_ctx *c, int k, double *ms, int64_t *launches, double *bytes, double *flops) {
  if (!c || k < 0 || k >= KC_COUNT) return fail(PDADMM_EINVAL, "bad argument");
  PD_TRY(prof_collect(c));
  if (ms) *ms = c->prof_ms[k];
  if (launches) *launches = c->prof_n[k];
  if (bytes) *bytes = c->prof_bytes[k];
  if (flops) *flops = c->prof_flops[k];
  return PDADMM_OK;
}
extern "C" int pdadmm_time_augmentation(pdadmm_ctx *c, int reps, double *ms_per_hop, double *bytes_per_hop) {
  if (!c || reps < 1 || reps > 1000 || !ms_per_hop) return fail(PDADMM_EINVAL, "bad argument");
  if (c->n_blocks < 2) return fail(PDADMM_EINVAL, "the input has a single block: no sparse product to time");
  if (c->N != c->N_total) return fail(PDADMM_EINVAL, "a sharded context keeps only its own rows of X");
  PD_CUDA(cudaSetDevice(c->device));
  Layer &l0 = c->layers[0];
  cudaStream_t st = c->scr.st;
  // the first hop again, block 0 -> block 1 of X: the same kernel on the same data writes the same bits
  launch_spmm(st, c->row_ptr, c->col_idx, c->csr_val, (int)c->N, l0.p, l0.p + c->d, c->d, l0.ld_in);
  PD_CUDA(cudaEventRecord(c->ev_begin, st));
  for (int i = 0; i < reps; ++i)
    launch_spmm(st, c->row_ptr, c->col_idx, c->csr_val, (int)c->N, l0.p, l0.p + c->d, c->d, l0.ld_in);
  PD_CUDA(cudaEventRecord(c->ev_end, st));
  PD_CUDA(cudaStreamSynchronize(st));
  PD_CUDA(cudaGetLastError());
  float ms = 0.f;
  PD_CUDA(cudaEventElapsedTime(&ms, c->ev_begin, c->ev_end));
  *ms_per_hop = ms / reps;
  if (bytes_per_hop) *bytes_per_hop = (double)c->nnz * (8.0 + 4.0 * c->d) + 8.0 * (double)c->N * c->d;
  return PDADMM_OK;
}
extern "C" int pdadmm_last_step_ms(pdadmm_ctx *c, double *ms) {
  if (!c || !ms) return fail(PDADMM_EINVAL, "null argument");
  *ms = c->last_step_ms;
  return PDADMM_OK;
}
extern "C" int pdadmm_launches(pdadmm_ctx *c, int64_t *count) {
  if (!c || !count) return fail(PDADMM_EINVAL, "null argument");
  *count = c->launches;
  return PDADMM_OK;
}

#include "no_alloc.cuh"
