/*
 * muon.h - C ABI of the B200 (sm_100a) Muon optimizer-step library.
 *
 * The library performs, for every 2-D parameter matrix it is given, the
 * per-matrix Muon step of "Muon is Scalable for LLM Training":
 *
 *   M <- mu*M + G                                   (Sec. 2.1, update rule)
 *   U  = mu*M + G  (Nesterov-style) or  U = M       (Sec. 2.1, footnote 1)
 *   X0 = U / (||U||_F + eps)                        (Sec. 2.1, Newton-Schulz paragraph)
 *   repeat ns_steps:  A = X X^T;  B = b*A + c*A^2;  X = a*X + B X      (Eq. 2)
 *   W <- W - lr*(rms_scale*sqrt(max(rows,cols))*X + wd*W)
 *                                                   (Sec. 2.2, Eq. 3 and the
 *                                                    "Matching update RMS" equation)
 *
 * Newton-Schulz runs in bf16 with fp32 accumulation on the matrix in its
 * short-side-first orientation (transposed when rows > cols); everything
 * element-wise is fp32.  Every step runs in hand-written CUDA kernels; there is
 * no CPU fallback.  All pointers in param-group descriptors are DEVICE pointers
 * unless a comment says "host".  All entry points return 0 on success and a
 * negative MUON_ERR_* code on failure; on a host-side failure nothing has been
 * launched.  muon_last_error() gives a thread-local message for the last
 * failure.
 *
 * Which parameters: 2-D weight matrices only.  Embeddings, the LM head and
 * norm gains stay with AdamW (Sec. 2.2 "Matching update RMS of AdamW"); the
 * caller also decides matrix granularity (Sec. 2.2 warns that splitting e.g.
 * each KV head into its own matrix makes max(rows, cols) too small).
 */
#ifndef MUON_H_
#define MUON_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MUON_OK = 0,
  MUON_ERR_INVALID_ARG = -1,  /* null pointer, non-positive size, bad enum */
  MUON_ERR_UNSUPPORTED = -2,  /* dtype / size the kernels do not handle */
  MUON_ERR_ALIGNMENT = -3,    /* pointer or leading dimension not aligned as required */
  MUON_ERR_WORKSPACE = -4,    /* workspace too small or misaligned */
  MUON_ERR_CUDA = -5,         /* a CUDA runtime / driver call failed */
  MUON_ERR_TIMEOUT = -6,      /* a bounded device-side wait expired (device status) */
  MUON_ERR_NONFINITE = -7     /* a matrix had a NaN/Inf Newton-Schulz input (device status) */
};

enum { MUON_DTYPE_BF16 = 0, MUON_DTYPE_FP32 = 1 };

/*
 * One group = `count` matrices of one shape [rows, cols] and one dtype pair.
 * Groups of equal (min(rows,cols), max(rows,cols), dtypes) are merged into one
 * shape bucket and processed by batched launches, whatever their orientation.
 *
 *   w, g, m : HOST arrays of `count` DEVICE pointers (weight, gradient,
 *             momentum).  Row-major, `rows` rows of `cols` elements, row
 *             stride ld_* elements.  The pointer arrays are copied at init;
 *             the matrices themselves stay owned by the caller and must stay
 *             allocated until muon_destroy.  W, G and M must not alias.
 *   w_dtype : dtype of W (bf16 or fp32).  g_dtype: dtype of G.  M is always
 *             fp32 and must be zero before the first step (M_0 = 0, Sec. 2.1).
 *   w_shadow: optional (NULL = none) HOST array of `count` DEVICE pointers to
 *             bf16 copies of fp32 weights (row stride ld_shadow): training
 *             set-ups that keep fp32 master weights (Sec. 2.3 counts an fp32
 *             parameter gather) and compute with a bf16 copy get both written
 *             by the step.  Only with w_dtype = fp32.
 *   Alignment: every pointer aligned to its element size; ld_w, ld_g, ld_m >=
 *             cols.  The fast vector paths need 16-byte aligned pointers and
 *             ld_* that are multiples of 8; anything else takes a slower
 *             scalar path with the same results.
 *   Magnitudes: the sum of squares behind ||U||_F and the first Gram product
 *             (formed from the un-normalised bf16(U) and scaled by 1/||U||_F^2
 *             in its epilogue) are fp32, so ||U||_F must stay within fp32's
 *             comfortable range: between about 1e-15 and 1e+18.  Above it the
 *             sums overflow and a finite input is reported as
 *             MUON_ERR_NONFINITE; far below it they underflow, the norm reads
 *             0 and the step only decays W.  Gradients of any loss scale used
 *             in practice are many orders of magnitude inside these limits.
 */
typedef struct muon_group {
  int32_t rows;
  int32_t cols;
  int32_t count;
  int32_t w_dtype;
  int32_t g_dtype;
  int32_t reserved;
  void* const* w;
  const void* const* g;
  float* const* m;
  int64_t ld_w;
  int64_t ld_g;
  int64_t ld_m;
  void* const* w_shadow;
  int64_t ld_shadow;
} muon_group;

/*
 * Hyper-parameters of one step (passed per call, nothing is cached).
 *   lr, wd    : eta and lambda of Eq. 3 (shared with AdamW, Sec. 2.2).
 *   mu        : momentum, 0.95 in the paper.
 *   nesterov  : non-zero selects the Nesterov-style input of footnote 1.
 *   ns_steps  : N of Eq. 2 (5 in the paper; 0 skips the iteration, O = X0).
 *   a, b, c   : quintic coefficients (3.4445, -4.7750, 2.0315).
 *   eps       : added to the Frobenius norm (the paper has none; 1e-7 keeps a
 *               zero input finite).
 *   rms_scale : the 0.2 of Sec. 2.2.
 *   scale_mode: how the update is scaled (Sec. 3.1 "Consistent Update RMS"):
 *               MUON_SCALE_ADJUSTED_LR  rms_scale * sqrt(max(rows, cols)) * O  (the method
 *                                       the paper adopts, Sec. 2.2; the default, 0),
 *               MUON_SCALE_FIXED_DIM    rms_scale * sqrt(scale_dim) * O  ("Baseline":
 *                                       scale_dim = the model's hidden size H),
 *               MUON_SCALE_UPDATE_NORM  rms_scale * O / RMS(O)  ("Update Norm").
 *   scale_dim : H for MUON_SCALE_FIXED_DIM, ignored otherwise.
 *   coeffs    : NULL, or a HOST array of 3 * ns_steps floats (a_1, b_1, c_1, a_2, ...)
 *               giving every iteration its own quintic; then a, b, c are ignored.
 *               (The paper uses one triple for all iterations.)
 *   protect_momentum: non-zero adds a pass over the gradients before the
 *               momentum update (2 or 4 more bytes read per element) that finds
 *               the matrices holding an Inf or a NaN; such a matrix keeps its M
 *               as well as its W, so that training can go on after a bad batch
 *               without repairing anything (the paper is silent on non-finite
 *               gradients).  0 (default): no such pass, see muon_status.
 */
enum { MUON_SCALE_ADJUSTED_LR = 0, MUON_SCALE_FIXED_DIM = 1, MUON_SCALE_UPDATE_NORM = 2 };
typedef struct muon_hparams {
  float lr;
  float wd;
  float mu;
  int32_t nesterov;
  int32_t ns_steps;
  float a;
  float b;
  float c;
  float eps;
  float rms_scale;
  int32_t scale_mode;
  float scale_dim;
  const float* coeffs;
  int32_t protect_momentum;
} muon_hparams;

typedef struct muon_ctx muon_ctx;

/*
 * Bytes of device workspace muon_init needs for these groups (pure host
 * computation; only rows/cols/count/dtypes are read).  The workspace holds the
 * bf16 Newton-Schulz operands of one bucket chunk (two X buffers, A and B, and
 * two more symmetric buffers where iterations are taken in pairs), pointer tables,
 * per-matrix scalars and the status word.  Large buckets are processed in
 * chunks so that the workspace stays bounded.
 */
int muon_workspace_bytes(const muon_group* groups, int n_groups, size_t* out_bytes);

/*
 * Owner-computes partition for data-parallel training (Sec. 2.3, Distributed
 * Muon: Newton-Schulz needs the whole gradient matrix, so each matrix is given
 * to ONE rank, which keeps its momentum, runs the step on it and shares the
 * updated weights afterwards; whole matrices are the unit, so nothing has to
 * be gathered inside the iteration).  Pure host computation on shapes and
 * counts: owner_out[i] (HOST, one int per matrix, groups in order) is the rank
 * in [0, world) that owns matrix i, balanced by the Newton-Schulz work
 * 3 m^2 n + m^3 with a deterministic longest-first greedy rule, so every rank
 * derives the same table.  load_out (HOST, world doubles, may be NULL) gets
 * the per-rank work.
 */
int muon_partition(const muon_group* groups, int n_groups, int world, int* owner_out, double* load_out);

/*
 * The same ownership question answered for storage that can be gathered in
 * place.  Every shape bucket (numbering of muon_plan_buckets) is cut into
 * `world` slots of share_out[bucket] = ceil(count / world) matrices; rank r owns
 * the matrices of slot r, which fill it from the front (a slot may hold one
 * matrix fewer than its capacity, or none when the bucket has fewer matrices
 * than ranks).  If a bucket's weights are stored slot after slot - matrix i at
 * index owner_out[i] * share + pos_out[i] of a [world * share] array of
 * matrices - the all-gather of the updated weights (Algorithm 1, last exchange)
 * writes every rank's slot where it already lives, and a reduce-scatter of
 * gradients stored the same way (Algorithm 1, first line) leaves every owner
 * with the reduced gradients of exactly its matrices; neither needs a staging
 * copy.  Within a bucket the matrices go to the ranks in consecutive runs,
 * groups in order; which ranks get the longer runs is decided by the
 * Newton-Schulz work (3 m^2 n + m^3 per matrix) accumulated over the earlier
 * buckets, so that the load stays balanced to within one matrix per bucket.
 * Pure host computation; owner_out, pos_out: one int per matrix (HOST);
 * share_out: one int per bucket (HOST); load_out: world doubles or NULL.
 */
int muon_partition_slots(const muon_group* groups, int n_groups, int world, int* owner_out, int* pos_out,
                         int* share_out, double* load_out);

/*
 * Build a context: validate the descriptors, form shape buckets, carve the
 * caller's workspace (DEVICE memory, 1024-byte aligned, at least
 * muon_workspace_bytes() long, owned by the caller, alive until destroy),
 * upload pointer tables and encode the TMA descriptors.  `device` is the CUDA
 * device ordinal all pointers live on.  This call and every other call on the
 * context switch to that device for their duration and restore the caller's
 * current device before returning.  Allocates no device memory itself.
 */
int muon_init(muon_ctx** out_ctx, const muon_group* groups, int n_groups, void* workspace,
              size_t workspace_bytes, int device);

/*
 * Enqueue one Muon step for every matrix of the context on `stream` (a
 * cudaStream_t passed as void*; NULL = legacy default stream).  Reads G,
 * updates W and M in place.  Asynchronous: returns after the launches are
 * enqueued, performs no allocation and no host synchronisation.  Device-side
 * problems (expired wait, non-finite input) are reported by muon_status.
 * Calls on one context must be stream-ordered with respect to each other.
 * Because the call only enqueues kernels, it may be recorded into a CUDA graph
 * by stream capture; the hyper-parameters are then those of the capture.
 */
int muon_step(muon_ctx* ctx, const muon_hparams* hp, void* stream);

/*
 * The shape buckets the planner forms from these groups (pure host
 * computation, like muon_workspace_bytes): bucket_out[i] (HOST, one int per
 * matrix, groups in order) is the bucket of matrix i, n_buckets_out the number
 * of buckets.  A bucket holds every matrix with the same short side, long
 * side and dtypes, whichever way round it is stored, and is the unit
 * muon_step_bucket works on.  A context built from the same groups uses the
 * same numbering.
 */
int muon_plan_buckets(const muon_group* groups, int n_groups, int* bucket_out, int* n_buckets_out);

/*
 * Newton-Schulz FLOPs of one step over these groups (pure host computation):
 * *algorithmic_out is Eq. 2 counted with the symmetric products halved,
 * ns_steps * (3 m^2 n + m^3) per matrix; *planned_out is what the planner's
 * launch sequence asks of the tensor cores, which is less where it takes
 * iterations two at a time (3 m^2 n + 5 m^3 per pair; see
 * muon_debug_set_pair_fold).  Neither counts tile padding.
 */
int muon_plan_flops(const muon_group* groups, int n_groups, int ns_steps, double* algorithmic_out,
                    double* planned_out);

/*
 * The same per kernel kind (arrays of MUON_KERNEL_KINDS doubles, indexed by
 * MUON_KERNEL_*; pure host computation).  planned_by_kind: the FLOPs the launch
 * sequence asks for, without padding (Gram m^2 n, every symmetric m x m x m
 * product m^3, combine 2 m^2 n; their sum is muon_plan_flops' planned figure).
 * executed_by_kind: the FLOPs the tensor cores execute, tile by tile - every
 * tile is 256 rows by 128 or 256 columns by the contraction length in whole
 * 64-element stages - so padding at ragged edges and the blocks that are
 * computed and dropped (below the diagonal of a symmetric result, the cross
 * terms of a tile shared by two matrices) are included: the figure to hold
 * against a tensor-pipe utilisation counter.
 */
int muon_plan_work(const muon_group* groups, int n_groups, int ns_steps, double* planned_by_kind,
                   double* executed_by_kind);

/*
 * muon_step for the matrices of ONE bucket (numbering of muon_plan_buckets).
 * Stepping every bucket once, in any order, is one muon_step.  Exists so that
 * a data-parallel caller can start sharing a bucket's updated weights while the
 * next bucket is still in its Newton-Schulz iteration (Sec. 2.3 asks for the
 * gather and the computation to overlap).  Same stream ordering, error
 * behaviour and asynchrony as muon_step; buckets share the workspace, so the
 * calls of one context stay on one stream.
 */
int muon_step_bucket(muon_ctx* ctx, const muon_hparams* hp, int bucket, void* stream);

/*
 * Same step with HOST gradients and HOST weight read-back, for callers whose
 * gradients arrive in (pinned) host memory: for every matrix i of every group
 * j, g_host[j][i] (host, dense rows*cols of the group's g_dtype) is copied
 * into the device G buffer, the step runs, and if w_host is non-NULL the
 * updated W is copied to w_host[j][i] (host, dense rows*cols of w_dtype).
 * The call does not synchronise; work enqueued on `stream` after it starts
 * only when the last copy has finished.  Uploads, kernels and downloads of
 * successive slices of a bucket overlap: the copies run on two streams the
 * context creates on first use (asynchronous copies need pinned host memory to
 * overlap).  A matrix's update RMS, norms and the status word are read as
 * after muon_step.
 */
int muon_step_host(muon_ctx* ctx, const muon_hparams* hp, const void* const* const* g_host,
                   void* const* const* w_host, void* stream);

/*
 * Synchronise `stream` and read the device status word.  *device_status is 0,
 * MUON_ERR_TIMEOUT or MUON_ERR_NONFINITE; *matrix_index (may be NULL) is the
 * global index (groups in order, matrices in order) of the first matrix that
 * reported it, or -1.  The status word is cleared.  A matrix with a non-finite
 * Newton-Schulz input keeps its W; its M has been updated by the first line of
 * the rule and now holds the non-finite values (the momentum pass runs before
 * the norm is known).  Before the next step the caller must repair that
 * matrix's M - zero it, or restore it from a copy - or every later step of the
 * matrix reports MUON_ERR_NONFINITE again and leaves its W unchanged; the
 * other matrices of the context are not affected.  With
 * muon_hparams.protect_momentum the matrix is reported in the same way but its
 * M is left as it was, and nothing needs repair.
 */
int muon_status(muon_ctx* ctx, void* stream, int* device_status, int* matrix_index);

/*
 * Per-matrix Frobenius norms ||U||_F of the last step's Newton-Schulz inputs:
 * copies `n` floats (global matrix order) to the HOST array `out` after
 * synchronising `stream`.
 */
int muon_get_norms(muon_ctx* ctx, void* stream, float* out, int n);

/*
 * Per-matrix update RMS of the last step, the value Algorithm 1 returns for
 * logging: sqrt(mean(u^2)) with u the scaled update before the learning rate
 * (rms_scale * sqrt(max(rows, cols)) * O in the default scale mode; it sits
 * near 0.2 by Sec. 2.2's design, and is rms_scale exactly with
 * MUON_SCALE_UPDATE_NORM).  Copies `n` floats (global matrix order) to the HOST array `out`
 * after synchronising `stream`.  A matrix whose input was non-finite reports
 * an unspecified value.
 */
int muon_get_update_rms(muon_ctx* ctx, void* stream, float* out, int n);

/* Free the host-side context.  Never touches caller memory. */
int muon_destroy(muon_ctx* ctx);

/* Message for the last failure on this thread ("" if none). */
const char* muon_last_error(void);

/* Number of kernels the last muon_step on this context enqueued. */
int muon_last_launch_count(const muon_ctx* ctx);

/*
 * Measurement mode.  While enabled, muon_step records a CUDA event pair around
 * every kernel it enqueues (on the step's stream).  muon_profile_read
 * synchronises the device, sums the elapsed milliseconds and the launch counts
 * per kernel kind since the last read (arrays of MUON_KERNEL_KINDS entries,
 * indexed by MUON_KERNEL_*) and resets the record.  Events are created on
 * demand; this mode is for benchmarks, not for training loops.
 */
enum {
  MUON_KERNEL_MOMENTUM = 0, /* momentum + Nesterov + sum of squares + bf16 cast */
  MUON_KERNEL_NORM = 1,     /* small helpers: norm and RMS finalisation, diagonal-block symmetrise */
  MUON_KERNEL_GRAM = 2,     /* A = X X^T */
  MUON_KERNEL_POLY = 3,     /* B = b A + c A A and the other symmetric m x m x m products */
  MUON_KERNEL_COMB = 4,     /* X' = a X + B X (last iteration: fused weight update) */
  MUON_KERNEL_UPDATE = 5,   /* separate weight update (ns_steps == 0, unaligned W, normalised update) */
  MUON_KERNEL_KINDS = 6
};
int muon_profile_enable(muon_ctx* ctx, int enable);
int muon_profile_read(muon_ctx* ctx, double* ms_by_kernel, int* launches_by_kernel);

/*
 * Test taps.  muon_debug_keep(ctx, 1) makes the last Newton-Schulz iteration
 * store its X (= O) in the workspace; the weights are then updated by the
 * separate update kernel instead of the last epilogue.  muon_debug_read copies one stage
 * of one matrix to a HOST buffer as dense bf16, short side first (m x n with
 * m = min(rows, cols); m x m for A and B): `which` is MUON_TAP_X0 (bf16(U),
 * NOT yet divided by the norm; valid while ns_steps <= 1), MUON_TAP_A,
 * MUON_TAP_B (last iteration; the kernels keep only the 128x128 blocks on or
 * above the diagonal of these symmetric matrices, the tap fills in the rest by
 * symmetry; when min(rows, cols) >= 16 the stored matrix is B + a*I, B of Eq.
 * 2's factorisation with the coefficient a added on the diagonal, so that
 * a*X + B X is the single product (B + a*I) X) or MUON_TAP_X (last iteration's X).  Only valid for a context with
 * a single shape bucket that fits one chunk (buckets share the chunk buffers).
 * Synchronises the device.
 */
enum { MUON_TAP_X0 = 0, MUON_TAP_A = 1, MUON_TAP_B = 2, MUON_TAP_X = 3 };
int muon_debug_keep(muon_ctx* ctx, int keep);
int muon_debug_read(muon_ctx* ctx, int matrix_index, int which, void* dst_host, size_t dst_bytes);

/*
 * Test probe for the device-side failure path.  Every wait in the kernels is
 * bounded: when one expires the kernel records MUON_ERR_TIMEOUT in the status
 * word, drains and returns instead of hanging.  This call enqueues a one-thread
 * kernel that waits, for at most limit_ms (1..1000) milliseconds, on a barrier
 * nothing arrives on, and reports the expiry the same way, naming
 * `matrix_index`.  muon_status then returns MUON_ERR_TIMEOUT and the context
 * remains usable.  Nothing faults or hangs.
 */
int muon_debug_wait_expiry(muon_ctx* ctx, void* stream, int matrix_index, unsigned limit_ms);

/*
 * Test knob: upper bound, in bytes, on the Newton-Schulz operands (X, A, B) of
 * one bucket chunk; a bucket that needs more is processed in several chunks
 * that reuse the workspace.  Process-wide, read by muon_workspace_bytes and
 * muon_init (a context keeps the plan it was created with).  0 restores the
 * default of 8 GiB.  Returns the previous value.  Tests lower it to run the
 * chunked path on small buckets.
 */
size_t muon_debug_set_chunk_bytes(size_t bytes);

/*
 * Knob: how tiles are cut where row blocks of 128 do not pair up.  Bit 0: a row
 * block without a partner (an odd number of row blocks in the combine) is a
 * half-height tile - UMMA M = 128, 64 rows per CTA, half a full tile's time -
 * instead of a full tile whose second CTA works on rows beyond the matrix.
 * Bit 1: the diagonal blocks of a symmetric product that no full tile can hold
 * without waste are half-height, half-width tiles, instead of sharing a
 * full-width tile with the neighbour matrix's (cross blocks dropped).  Bit 2
 * switches off the finer cut (every row block on its own at half height, or
 * block by block) that the symmetric products of a bucket take when full tiles
 * would be fewer than the CTA pairs of the GPU.  Default 1 (bit 1 computes
 * nothing in vain but measured slower).  Process-wide, read where muon_debug_set_pair_fold is.  Returns the
 * previous mode; a value outside 0..7 only queries.  The modes agree to
 * rounding, not bit for bit (instructions of different heights round their
 * sums differently); within one mode results are reproducible bit for bit.
 */
int muon_debug_set_tile_mode(int mode);

/*
 * Knob: where the planner takes two iterations per pass over X (Eq. 2 gives
 * X_{k+1} = P_k X_k with P_k = a*I + b*A_k + c*A_k^2, so A_{k+1} = P_k^2 A_k and
 * X_{k+2} = P_{k+1} P_k X_k need no Gram product and no combine for the second
 * iteration of a pair).  0 (default): the first two iterations, for matrices
 * of at least 256 rows whose long side is at least 1.25 x the short side (as
 * accurate as the plain sequence in bf16, and fewer FLOPs); 1: never; 2: the
 * first two iterations whenever the short side is at least 16; 3: as 0, and
 * every further pair too when the long side is at least twice the short side
 * (faster, up to twice the plain sequence's rounding error); 4: every pair
 * whenever the short side is at least 16.  Process-wide, read by
 * muon_workspace_bytes, muon_plan_flops and muon_init (a context keeps the
 * plan it was created with).  Returns the previous mode; a value outside 0..4
 * only queries.
 */
int muon_debug_set_pair_fold(int mode);

/*
 * Test tap (pure host computation): the tile table the Newton-Schulz products
 * of a bucket of `count` rows x cols matrices use (the count matters because a
 * bucket whose launches would leave SMs idle is cut into finer tiles).  which = 0: products with a symmetric result,
 * table of one unit of *unit_mats matrices; 1: the same for a last matrix
 * without a partner (empty when units are single matrices); 2: the combine;
 * 3: the combine formed transposed.  Every tile is ten int16 in `out` (room
 * for cap_tiles tiles; NULL only queries the count): row block of CTA 0 and of
 * CTA 1, column block of the first and of the second 128 accumulator columns,
 * width in column blocks (1 or 2), matrix of CTA 0 and of CTA 1 within the unit,
 * per CTA a mask of the column halves whose 128 x 128 block is stored, and 1 for
 * a half-height tile (one row block, 64 rows per CTA; its mask is the first).
 */
int muon_debug_tile_table(int rows, int cols, int count, int which, int16_t* out, int cap_tiles, int* n_tiles,
                          int* unit_mats);

/*
 * Test tap: the TMEM base address each CTA of the last Newton-Schulz GEMM launch
 * obtained (indexed by CTA; 0xFFFFFFFF where no CTA ran).  Copies `n` (at most
 * 1024) values to the HOST array.  Synchronises the device.
 */
int muon_debug_tmem_bases(muon_ctx* ctx, unsigned* out_host, int n);

/*
 * AdamW step for the parameters Muon does not handle: RMSNorm gains, the LM
 * head and embeddings (Sec. 2.2 "Matching update RMS of AdamW": they share lr
 * and wd with the Muon-updated matrices; the appendix notes that weight decay
 * on the RMSNorm gains matters).  Adam with bias correction and decoupled
 * weight decay, one fused streaming kernel over all tensors:
 *
 *   m <- beta1 m + (1-beta1) g;   v <- beta2 v + (1-beta2) g^2
 *   p <- p - lr * ( (m/(1-beta1^step)) / (sqrt(v/(1-beta2^step)) + eps) + wd p )
 *
 * `tensors` is a HOST array of descriptors with DEVICE pointers: p (bf16 or
 * fp32) and fp32 m, v are updated in place, g (bf16 or fp32) is read; numel
 * elements each, any shape, contiguous.  `step` counts from 1.  Asynchronous on
 * `stream`; needs no context, no workspace and allocates nothing.  16-byte
 * aligned tensors take the vector path; others a scalar path with the same
 * results.
 */
typedef struct muon_adamw_tensor {
  void* p;
  const void* g;
  float* m;
  float* v;
  int64_t numel;
  int32_t p_dtype;
  int32_t g_dtype;
} muon_adamw_tensor;

typedef struct muon_adamw_hparams {
  float lr;
  float wd;
  float beta1;
  float beta2;
  float eps;
  int32_t step;
} muon_adamw_hparams;

int muon_adamw_step(const muon_adamw_tensor* tensors, int n_tensors, const muon_adamw_hparams* hp,
                    int device, void* stream);

/*
 * Momentum update and Frobenius norm of ONE matrix with no workspace and no
 * allocation of any kind (the paper has no counterpart; this is a library
 * convenience, not a step of its method):
 *
 *   M <- mu*M + G;   U = mu*M + G if nesterov else M;   *norm_out = ||U||_F
 *
 * Who needs it: code that wants this reduction but cannot obtain device
 * memory for a workspace - for instance a monitoring hook in a process whose
 * framework has already reserved the whole GPU for its own pool, so a raw
 * cudaMalloc would fail, or a caller running where an allocation's implicit
 * device-wide synchronisation is not acceptable.  The per-tile partial sums
 * that muon_step keeps in the caller's workspace live here in a fixed array
 * inside the library image: MUON_STATIC_MAX_TILES floats (256 KiB), held by
 * every GPU that loads the library until the process exits.
 *
 *   g        : DEVICE, rows x cols, row stride ld_g elements, dtype g_dtype.
 *   m        : DEVICE, fp32, rows x cols, row stride ld_m; updated in place.
 *   norm_out : DEVICE, one float, written by the call (stream-ordered).
 *   device   : ordinal the pointers live on; it becomes the calling thread's
 *              current device.
 *   stream   : cudaStream_t as void* (NULL = legacy default stream).
 *
 * Limit: ceil(rows/64) * ceil(cols/128) must not exceed MUON_STATIC_MAX_TILES
 * (e.g. 16384 x 32768); larger matrices get MUON_ERR_UNSUPPORTED and nothing
 * is launched - use muon_step with a workspace for those.
 *
 * The first call for a device looks up the device address of the built-in
 * array (cudaGetSymbolAddress) and caches it; make that first call before
 * starting any stream capture.  Later calls only enqueue two kernels.  The call
 * never invokes cudaMalloc, cudaFree or any allocating routine and does not
 * synchronise.
 *
 * All calls on one GPU share the one array, and it keeps whatever the last
 * call left in it.  Nothing in it needs clearing (each call overwrites the
 * entries it later reads), but two calls that can overlap on the GPU - different
 * streams, or different host threads without stream ordering between them -
 * race on it and may return wrong norms.  Keep the calls of one GPU on one
 * stream, or order them with events.
 */
#define MUON_STATIC_MAX_TILES 65536
int muon_momentum_norm_static(const void* g, float* m, int rows, int cols, int64_t ld_g, int64_t ld_m,
                              int g_dtype, float mu, int nesterov, float* norm_out, int device,
                              void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MUON_H_ */
