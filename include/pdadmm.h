/*
 * pdadmm.h -- C ABI of the pdADMM-G / pdADMM-G-Q training iteration for graph-augmented MLPs
 * on one NVIDIA B200 (sm_100a).
 *
 * Notation follows the paper (Table "Important Notations"): |V| = N nodes, L layers,
 * W_l (n_l x n_{l-1}), b_l (n_l), p_l (input of layer l, p_1 = X), z_l, q_l, u_l, penalties nu, rho.
 * The paper stores one COLUMN per node (p_l is n_{l-1} x N); every host and device array of this
 * library is the same memory read node-major: row j holds node j, i.e. P_l is [N][n_{l-1}],
 * Z_l, Q_l, U_l are [N][n_l], row-major float32.  W_l is [n_l][n_{l-1}] row-major float32.
 * Layers are numbered 1..L as in the paper in every call.
 *
 * General rules
 *  - Every function returns PDADMM_OK (0) or a negative pdadmm_status; nothing aborts or throws
 *    across the boundary.  pdadmm_last_error() gives a thread-local text for the last failure.
 *  - All pointer arguments are HOST pointers unless a parameter is explicitly called a device
 *    pointer.  The caller owns every buffer it passes; the library copies what it needs during
 *    the call and never keeps a caller pointer.  Output buffers are written only after their
 *    size has been checked.
 *  - A context owns all of its device memory and streams; it is bound to one device and is not
 *    thread-safe.  There is no CPU fallback: without a usable CUDA device every call that needs
 *    one fails with PDADMM_ECUDA.
 */
#ifndef PDADMM_H
#define PDADMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pdadmm_ctx pdadmm_ctx;

typedef enum {
  PDADMM_OK = 0,
  PDADMM_EINVAL = -1,    /* bad argument (null pointer, size, range, unsorted or out-of-range index) */
  PDADMM_ENOMEM = -2,    /* host or device allocation failed                                         */
  PDADMM_ECUDA = -3,     /* a CUDA call failed, or no usable device                                  */
  PDADMM_ETIMEOUT = -4,  /* a bounded device-side wait expired                                       */
  PDADMM_ENUMERIC = -5,  /* a non-finite value was detected in the state                             */
  PDADMM_ENOTCONV = -6   /* the tau search of the quantised p-update hit its trial cap               */
} pdadmm_status;

/* Tensor kinds of pdadmm_get_tensor / pdadmm_set_tensor.  "layer" is the paper's l. */
typedef enum {
  PDADMM_T_X = 0,        /* float  [N][n_0]       augmented features = p_1 (layer ignored)             */
  PDADMM_T_P = 1,        /* float  [N][n_{l-1}]   l = 1..L (l = 1 is X)                                */
  PDADMM_T_W = 2,        /* float  [n_l][n_{l-1}] l = 1..L                                             */
  PDADMM_T_B = 3,        /* float  [n_l]          l = 1..L                                             */
  PDADMM_T_Z = 4,        /* float  [N][n_l]       l = 1..L                                             */
  PDADMM_T_Q = 5,        /* float  [N][n_l]       l = 1..L-1                                           */
  PDADMM_T_U = 6,        /* float  [N][n_l]       l = 1..L-1                                           */
  PDADMM_T_CODES = 7,    /* uint8 (uint16 above 256 levels) [N][n_{l-1}]  l = 2..L, pdADMM-G-Q only:
                            p_l = (code - quant_neg_levels) * QSCALE_l (get only)                      */
  PDADMM_T_TAU = 8,      /* double [1]            l = 2..L: tau_l of the last iteration (get only)     */
  PDADMM_T_THETA = 9,    /* double [1]            l = 1..L: theta_l of the last iteration (get only)   */
  PDADMM_T_QSCALE = 10,  /* float  [1]            l = 2..L: level spacing s_l of p_l                   */
  PDADMM_T_CSR_ROWPTR = 11, /* int32 [N+1]        renormalised adjacency, get only                     */
  PDADMM_T_CSR_COLIDX = 12, /* int32 [nnz]        columns ascending in each row, get only              */
  PDADMM_T_CSR_VAL = 13, /* float  [nnz]          get only                                             */
  PDADMM_T_TRIALS = 14   /* int32  [1]            l = 2..L: trials of the last quantised p-update      */
} pdadmm_tensor;

/* Bits of pdadmm_config.flags. */
#define PDADMM_FLAG_SIMT_GEMM 1u     /* run the dense products on CUDA cores (fp32 FMA) instead of tensor cores */
#define PDADMM_FLAG_QUANT_Q 2u       /* pdADMM-G-Q variant that keeps q_l on the level set of p_{l+1} as well   */
#define PDADMM_FLAG_NO_GRAPH 4u      /* launch every kernel of an iteration directly instead of replaying a CUDA graph */
#define PDADMM_FLAG_ONE_LANE 8u      /* queue all layers on one stream instead of spreading them over concurrent lanes */
#define PDADMM_FLAG_LEAST_SQUARES 16u /* R(z_L; y) = 1/2 sum over labelled nodes ||z_L - e_y||^2 instead of the cross-entropy
                                         (paper, "Problem Formulation": R is any convex, continuous risk); the z_L
                                         update then is the closed form z = (e_y + nu a)/(1 + nu)          */

/*
 * Problem statement (paper: Problem 2 / Problem 3, Algorithm 1 "Require", and the experimental
 * settings for the operator set Psi and the renormalised adjacency).
 */
typedef struct {
  int64_t n_nodes;               /* N = |V| >= 1                                                        */
  int64_t n_edges;               /* undirected edges, each listed once; self-loops/repeats are ignored  */
  const int32_t *edge_src;       /* [n_edges] node ids in [0, N)                                        */
  const int32_t *edge_dst;       /* [n_edges]                                                           */
  int32_t feat_dim;              /* d                                                                   */
  const float *features;         /* H, node-major [N][d]                                                */
  int32_t n_hops;                /* highest power of A~ used; the input has n_hops+1 blocks, n_0=(n_hops+1)d */
  int32_t n_classes;             /* C = n_L                                                             */
  const int32_t *labels;         /* [N] in [0, C)                                                       */
  const uint8_t *train_mask;     /* [N]; 1 = the node's cross-entropy is part of R(z_L; y)              */
  int32_t n_layers;              /* L >= 1                                                              */
  const int32_t *layer_widths;   /* [L]: n_1..n_L, n_L == n_classes                                     */
  float rho;                     /* > 0                                                                 */
  float nu;                      /* > 0                                                                 */
  int32_t quant_levels;          /* 0: pdADMM-G;  2..65536: pdADMM-G-Q with that many uniform levels (codes
                                    of one byte up to 256 levels, two bytes above)                      */
  int32_t quant_neg_levels;      /* levels below zero: Delta = {(c - quant_neg_levels) s, c = 0..m-1}; 0 = levels
                                    start at 0.  A value > 0 needs quant_step > 0.  ({-1..20}: m=22, 1, step 1) */
  float quant_step;              /* > 0: the same level spacing s for every layer; 0: s_l = max(p_l^0)/(m-1)  */
  float leaky_slope;             /* f_l of the hidden layers: 0 = ReLU; in (0, 1) = leaky ReLU, f(x) = slope x
                                    for x <= 0 (paper, "Convergence Analysis": both satisfy its assumptions) */
  int32_t activation;            /* f_l of the hidden layers: 0 = ReLU / leaky ReLU (leaky_slope); 1 = tanh; 2 = logistic
                                    sigmoid.  The smooth ones have no closed-form z-update: following the paper's remark
                                    after Eq. "update z" it is taken from a lookup table, the best of table_size candidates
                                    z_i = table_lo + i (table_hi - table_lo)/(table_size - 1) (single precision), i.e. z is
                                    resolved to the table step                                            */
  int32_t table_size;            /* 2..4096 candidates (activation 1, 2 only)                              */
  float table_lo, table_hi;      /* range of the candidates: should cover the values z takes              */
  const float *const *init_W;    /* [L] pointers: W_l^0 as [n_l][n_{l-1}] (required; the caller draws them) */
  int32_t device;                /* CUDA device ordinal                                                 */
  uint32_t flags;                /* PDADMM_FLAG_*                                                       */
} pdadmm_config;

/*
 * pdadmm_init -- build the problem on the device.
 * Computes the CSR form of A~ = (D+I)^{-1/2}(A+I)(D+I)^{-1/2} (paper, "Datasets and Settings"),
 * the augmented input X = [H; H A~; ...; H A~^{n_hops}] by sparse products (paper, "Problem
 * Formulation": X_k = H psi_k(A)), and the start of Algorithm 1: b = 0, a forward pass
 * z_l = W_l p_l, q_l = ReLU(z_l), p_{l+1} = q_l (pdADMM-G-Q: p_{l+1} = nearest level of q_l, with the
 * level spacing s_{l+1} = max(q_l)/(m-1)), u = 0.
 * On success *out receives a context that the caller must release with pdadmm_destroy.
 * Errors: EINVAL for inconsistent sizes / out-of-range indices / null pointers, ENOMEM, ECUDA.
 */
int pdadmm_init(const pdadmm_config *cfg, pdadmm_ctx **out);

/*
 * Node sharding (multi-GPU): after the augmentation every update of Algorithm 1 acts on one node's column at a time,
 * except for sums over nodes inside tau (Eq. "update p"), theta and nabla_W phi (Eq. "update W"), nabla_b phi (Eq.
 * "update b") and the acceptance test of Eq. "update p quantized".  A context may therefore own the nodes
 * [node_begin, node_begin + node_count) only -- p, z, q, u of those nodes, and full copies of W and b -- and hand every
 * such sum to the caller, who adds it over the contexts of all shards (one per GPU).  The paper distributes layers
 * over clients instead (Sec. "The pdADMM-G Algorithm"); sharding by nodes exchanges O(L h^2) bytes per iteration
 * instead of O(|V| h).
 *
 * pdadmm_allreduce_fn: reduce `count` elements (dtype 0: float, 1: double) at the DEVICE pointer `buf`, in place,
 * over all shards with op 0 (sum) or 1 (max), ordered after the work already queued on `stream` (a cudaStream_t of
 * the context) and before work queued on it later; return 0, anything else aborts the call with PDADMM_ECUDA.  The
 * buffer belongs to the context and lies in its own GPU's memory.  Every shard's context issues the same sequence of
 * calls, so a collective library can be called directly.  `user` is passed through.
 *
 * pdadmm_init_sharded: like pdadmm_init; cfg describes the WHOLE graph (all nodes, features, labels, mask: the graph
 * operator needs the neighbours of the shard's nodes) and the context keeps the shard.  Every shard must pass the same
 * cfg and init_W.  shard == NULL, or a null allreduce with the full node range, is pdadmm_init.  In a sharded context
 * tensors of node-sized kinds (X, P, Z, Q, U, CODES) are the shard's rows; pdadmm_objective and pdadmm_residuals
 * return the totals over all shards (they reduce, so all shards must call them together); pdadmm_predict counts the
 * shard's nodes.
 */
typedef int (*pdadmm_allreduce_fn)(void *user, void *buf, size_t count, int dtype, int op, void *stream);
typedef struct {
  int64_t node_begin;            /* first node of the shard                              */
  int64_t node_count;            /* >= 1, node_begin + node_count <= cfg->n_nodes       */
  pdadmm_allreduce_fn allreduce; /* adds over all shards; required unless the shard is the whole graph */
  void *user;
} pdadmm_shard;
int pdadmm_init_sharded(const pdadmm_config *cfg, const pdadmm_shard *shard, pdadmm_ctx **out);

/* Bytes handed to the reduction callback by pdadmm_step so far (the volume entering the all-reduces). */
int pdadmm_comm_bytes(pdadmm_ctx *ctx, int64_t *bytes);

/*
 * pdadmm_step -- run n_iters iterations of Algorithm 1: for every layer the p-update (Eq. "update
 * p"; pdADMM-G-Q: Eq. "update p quantized"), W-update (Eq. "update W"), b-update (Eq. "update b"),
 * z-update (Eq. "update z" with the ReLU closed form, Eq. "update zl" for the last layer), q-update
 * (Eq. "update q"), residual and dual update (Eq. "update u").  Returns after the device finished.
 * tau_l and theta_l are the smallest values that satisfy the paper's conditions
 * phi(p+) <= U_l(p+; tau) and phi(W+) <= V_l(W+; theta); the quantised update doubles tau from
 * that value until its condition holds (at most 30 trials, then ENOTCONV; the state stays valid).
 */
int pdadmm_step(pdadmm_ctx *ctx, int n_iters);

/*
 * pdadmm_last_step_ms -- device time of the last pdadmm_step call in milliseconds, measured with CUDA
 * events recorded on the context's own stream before the first and after the last kernel of the call.
 */
int pdadmm_last_step_ms(pdadmm_ctx *ctx, double *ms);

/*
 * pdadmm_objective -- the augmented Lagrangian L_rho (paper, Section "The pdADMM-G Algorithm") of the
 * current state: out = { R(z_L;y), (nu/2) sum_l ||z_l - W_l p_l - b_l||^2, (nu/2) sum_l ||q_l - ReLU(z_l)||^2,
 * sum_l <u_l, p_{l+1} - q_l>, (rho/2) sum_l ||p_{l+1} - q_l||^2, their sum }.  R is the sum of the
 * cross-entropies of the masked nodes.  Accumulated in double precision.
 */
int pdadmm_objective(pdadmm_ctx *ctx, double out[6]);

/*
 * pdadmm_residuals -- ||p_{l+1} - q_l||^2 for l = 1..L-1 (Algorithm 1, residual line) into
 * per_layer_sq[0..n-1]; n must be L-1 (n = 0 with a null pointer is accepted for L = 1).
 */
int pdadmm_residuals(pdadmm_ctx *ctx, double *per_layer_sq, int n);

/*
 * pdadmm_predict -- the trained model on every node (paper, Problem 1: p_1 = X, z_l = W_l p_l + b_l,
 * p_{l+1} = f_l(z_l) = ReLU(z_l); the class of a node is the largest entry of z_L, the quantity the
 * cross-entropy risk R(z_L; y) scores and the "Performance" section reports as accuracy).  A forward pass
 * with the current W and b, run with the same dense-product kernels as the iteration; the state of the
 * iteration (p, z, q, u) is neither read nor changed.
 *   logits_out : host [N][C] fp32, z_L of the forward pass                     (may be null)
 *   pred_out   : host [N] int32, argmax over the C classes, first one if equal (may be null)
 *   counts_out : host [4] int64: correct and total among nodes with train_mask = 1, correct and
 *                total among the other nodes                                   (may be null)
 * Returns 0, EINVAL, ECUDA or ETIMEOUT.
 */
int pdadmm_predict(pdadmm_ctx *ctx, float *logits_out, int32_t *pred_out, int64_t counts_out[4]);

/*
 * pdadmm_get_tensor / pdadmm_set_tensor -- copy one tensor of the state to / from a host buffer of
 * exactly `bytes` bytes (dense, without the device's row padding).  Together they are the
 * checkpoint / resume interface.  Setting P, W, B or Z invalidates the cached linear residual
 * W p + b - z, which the next step recomputes.  Setting P in pdADMM-G-Q mode expects values on the
 * level set: CODES are recomputed from them and P becomes the levels of those codes (the same bits for
 * values on the level set; the kernels read p_l through its codes).  Setting QSCALE of a layer moves its
 * p_l to the new level set in the same way, so set QSCALE before P.  EINVAL for a bad kind/layer/size or a
 * get-only kind.
 */
int pdadmm_get_tensor(pdadmm_ctx *ctx, int kind, int layer, void *host_dst, size_t bytes);
int pdadmm_set_tensor(pdadmm_ctx *ctx, int kind, int layer, const void *host_src, size_t bytes);

/*
 * pdadmm_start_layers_from -- the start of Algorithm 1 for layers first_layer..L from the current p_{first_layer}:
 * b_l = 0, z_l = W_l p_l, q_l = f_l(z_l), p_{l+1} = q_l (pdADMM-G-Q: its nearest level, the spacing taken from max(q_l)),
 * u_l = 0; the layers below keep their state.  It is the building block of the greedy layer-wise strategy (paper, end
 * of Section "The pdADMM-G Algorithm"; "Performance": two layers first, then five, then all ten): a deeper context is
 * created, the trained layers' tensors are copied in with pdadmm_set_tensor, and the added layers are started here from
 * the forward pass of the model trained so far.  first_layer = 1 restores the initial state for the current W.
 */
int pdadmm_start_layers_from(pdadmm_ctx *ctx, int first_layer);

/*
 * pdadmm_quantize -- the projection used by Eq. "update p quantized" on its own: for n host floats x,
 * code = clamp(floor((x - lo)/scale + 1/2), 0, levels-1) as uint8 and p = lo + code * scale (one rounded
 * single-precision multiply, one rounded add), computed by the same device function as inside
 * pdadmm_step.  lo is the smallest level (0 for levels that start at zero, -1 with scale 1 and 22 levels
 * for the set {-1..20} of the paper's experiments).  levels in [2, 65536]; codes are uint8 for up to 256
 * levels and uint16 above (the 8- and 16-bit cases of the paper's "Communication Overheads" experiment).
 * codes_out and p_out are host buffers of n elements (either may be null).
 */
int pdadmm_quantize(int device, const float *x, size_t n, float scale, float lo, int levels,
                    void *codes_out, float *p_out);

/*
 * pdadmm_spmm -- Y = A~ X for a caller-supplied CSR matrix (host arrays, columns in [0, n_rows))
 * and a node-major [n_rows][width] host matrix, by the same kernel that builds the augmented input
 * (paper, "Problem Formulation": X_{k+1} = X_k A~ with A~ symmetric).  y_out is [n_rows][width].
 */
int pdadmm_spmm(int device, int64_t n_rows, const int32_t *row_ptr, const int32_t *col_idx,
                const float *val, const float *x, int32_t width, float *y_out);

/*
 * pdadmm_matmul -- one dense product by the kernels that pdadmm_step uses for the W p, W^T r and r p^T
 * terms (paper, Section "The pdADMM-G Algorithm": the products inside nabla_p phi and nabla_W phi), on
 * host matrices, row-major float32 without padding:
 *   mode 0: C[M][N] = A[M][K] * B[N][K]^T      mode 1: C[M][N] = A[M][K] * B[K][N]
 *   mode 2: C[M][N] = A[K][M]^T * B[K][N]      (contraction over the leading index, split over node slices)
 * flags: PDADMM_FLAG_SIMT_GEMM selects the CUDA-core kernels, 0 the tensor-core kernels.
 * sumsq (may be null) receives sum(C^2) accumulated by the fused epilogue (modes 0 and 1); the tensor-core
 * kernels square in single precision, so it is meaningful for 1e-19 < |C| < 1e19 (C itself has no such limit:
 * every operand is scaled by a power of two taken from its largest magnitude before it is split into fp16 planes).
 */
int pdadmm_matmul(int device, int mode, int M, int N, int K, const float *A, const float *B, float *C,
                  double *sumsq, uint32_t flags);

/*
 * pdadmm_matmul_tn_static -- (no counterpart in the paper: an interface for callers that cannot allocate.)
 * C[M][ldc] = A[K][lda]^T * B[K][ldb] on DEVICE buffers of the caller, fp32 on the CUDA cores, ldc = N rounded
 * up to a multiple of 4 (rows of C are padded to that width and the padding is written as zero).  This is
 * the contraction over the node index that the W-gradient needs; like pdadmm_matmul mode 2 it cuts the nodes
 * into slices and adds the slices' partial tiles in slice order, but the partial tiles live in a fixed 4 MiB
 * array inside the library image, so the call performs no cudaMalloc, cudaFree or other allocation.  Meant
 * for callers that must not allocate: code running inside a stream capture, a latency-critical loop that may
 * not take the allocator lock or cause an implicit device synchronisation, or a layer that was given all of
 * its buffers up front.
 *  - dA, dB, dC: device pointers on `device`, 16-byte aligned; lda >= M, ldb >= N, both multiples of 4.
 *    The operands are read in groups of four columns: columns M..lda-1 of dA and N..ldb-1 of dB must be readable
 *    but may hold anything (NaN included); they reach neither the valid block nor the padding of C.
 *  - Limit: M * ldc <= 1048576 floats (one partial tile must fit the built-in array); larger outputs are
 *    rejected with PDADMM_EINVAL and a message that names both sizes.  Every GPU that loads the library holds
 *    the 4 MiB until the process exits.
 *  - The two kernels are enqueued on `stream` (a cudaStream_t, or null for the default stream) and the call
 *    returns without waiting for them.
 *  - The first call on each device looks up the device address of the built-in array (once per device); make
 *    that first call before beginning any stream capture.
 *  - All calls share the array and it keeps the contents of the last call.  Nothing in it has to start at
 *    zero: every element that a call reads was written earlier in the same call.  Two calls whose kernels
 *    overlap on the GPU (different streams, or different host threads) race on the array: serialise them.
 */
int pdadmm_matmul_tn_static(int device, int M, int N, int K, const float *dA, int lda, const float *dB, int ldb,
                            float *dC, void *stream);

/*
 * pdadmm_selftest_bounded_wait -- exercises the error path of PDADMM_ETIMEOUT without any faulty input: one warp
 * waits, with the wait routine of the tensor-core products, on a barrier that nothing arrives at; the wait gives up
 * after about limit_cycles SM cycles (1 .. 1e8), the kernel raises the products' error word and returns by itself.
 * Always returns PDADMM_ETIMEOUT when the device is usable (PDADMM_OK would mean the wait was satisfied, which cannot
 * happen); *waited_cycles (may be null) receives the cycles the wait lasted.  The context of the process stays usable:
 * a product launched afterwards runs normally.
 */
int pdadmm_selftest_bounded_wait(int device, long long limit_cycles, long long *waited_cycles);

/*
 * Per-kernel timing.  pdadmm_profile(ctx, 1) makes every later kernel launch of pdadmm_step be
 * bracketed by CUDA events on its own stream (the layers then run one after another);
 * pdadmm_profile(ctx, 0) turns it off; either call clears the counters.
 * pdadmm_profile_read returns, for kernel class k in [0, pdadmm_profile_classes()), the summed
 * device time in ms, the number of launches, and the algorithmic bytes and flops of those launches.
 * pdadmm_launches gives the number of kernels launched by pdadmm_step since the context was made.
 */
int pdadmm_profile(pdadmm_ctx *ctx, int enable);
int pdadmm_profile_classes(void);
const char *pdadmm_profile_name(int k);
int pdadmm_profile_read(pdadmm_ctx *ctx, int k, double *ms, int64_t *launches, double *bytes, double *flops);
int pdadmm_launches(pdadmm_ctx *ctx, int64_t *count);

/*
 * pdadmm_time_augmentation -- device time of one hop of the feature augmentation X_{k+1} = X_k A~ (paper, "Problem
 * Formulation"; the sparse products run once inside pdadmm_init, where they cannot be timed apart from the copies):
 * repeats the first hop `reps` times (1..1000) on the context's own CSR matrix and input block, writing the block of
 * X it already holds (same kernel, same data, same bits), between CUDA events on the context's stream.
 * *ms_per_hop receives the mean; *bytes_per_hop (may be null) the algorithmic bytes of a hop,
 * nnz (8 + 4 d) + 8 N d.  EINVAL if the input has a single block.
 */
int pdadmm_time_augmentation(pdadmm_ctx *ctx, int reps, double *ms_per_hop, double *bytes_per_hop);

/* Release the context and all of its device memory.  Null is accepted. */
int pdadmm_destroy(pdadmm_ctx *ctx);

/* Text of the calling thread's last failure ("" if none).  The pointer stays valid until the next failing call. */
const char *pdadmm_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PDADMM_H */
