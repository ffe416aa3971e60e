/* bsp.h — C ABI of the block-structured-pruning library for NVIDIA B200 (sm_100a).
 *
 * The library implements, on one GPU, the computations of
 *   Li, Kong et al., "Efficient Transformer-based Large Scale Language Representations using
 *   Hardware-friendly Block Structured Pruning", EMNLP-Findings 2020:
 * per-group l2 norms with the reweighted group-Lasso penalty and its gamma update (Section 3.2,
 * Eq. 2 and Eq. 3), threshold pruning of the groups (Algorithm 1) into a compressed
 * block-structured storage (Section 3.1), and the linear layer Y = act(X W^T + b) evaluated on
 * the pruned weight (the computation the pruning is meant to speed up, Sections 3.1 and 4.4).
 *
 * Conventions shared by every call
 * --------------------------------
 *  - W is one linear layer's weight, [rows = N_out, cols = K_in], row-major bf16 with leading
 *    dimension ldw (elements).  X is [tokens, K_in] bf16 row-major (ldx), Y is [tokens, N_out]
 *    bf16 row-major (ldy).
 *  - Orientation BSP_ORIENT_C (Eq. 3): W is cut into rows/block row-blocks of `block`
 *    consecutive rows; a group is one column of one row-block.  Per-group arrays are
 *    [rows/block, cols] row-major.  A "block" owns `cols` groups.
 *    Orientation BSP_ORIENT_R (Algorithm 1 as printed, Eq. 2): W is cut into cols/block vertical
 *    strips of `block` consecutive columns; a group is one row of one strip.  Per-group arrays
 *    are [rows, cols/block] row-major.  A "block" (strip) owns `rows` groups.
 *  - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns every
 *    buffer; the library allocates no device memory.  `stream` is a cudaStream_t passed as
 *    void* (NULL = the legacy default stream).  Calls enqueue work on `stream` and return
 *    without synchronising; outputs are valid once the stream has reached that point.
 *  - Every function returns BSP_OK (0) or a negative bsp_status.  Argument and shape errors are
 *    detected on the host before anything is launched.  Nothing aborts or throws.
 *  - Inputs must be finite (no NaN/Inf weights).
 */
#ifndef BSP_H_
#define BSP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BSP_OK = 0,
  BSP_ERR_ARG = -1,         /* null pointer, negative size, unknown enum value, misaligned buffer */
  BSP_ERR_SHAPE = -2,       /* block does not divide rows (C) / cols (R); leading dimension too small */
  BSP_ERR_WORKSPACE = -3,   /* workspace smaller than the matching *_bound / *_bytes query says   */
  BSP_ERR_CUDA = -4,        /* a CUDA runtime or driver call failed (see bsp_last_cuda_error)     */
  BSP_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (reported by bsp_linear_status) */
  BSP_ERR_UNSUPPORTED = -6  /* size beyond a documented limit                                     */
} bsp_status;

typedef enum { BSP_ORIENT_C = 0, BSP_ORIENT_R = 1 } bsp_orient;
typedef enum { BSP_PEN_L2 = 0, BSP_PEN_L2SQ = 1 } bsp_penalty;
typedef enum { BSP_ACT_NONE = 0, BSP_ACT_GELU = 1 } bsp_act;

/* Human-readable name of a status code (static string, host). */
const char* bsp_status_string(int status);
/* Last CUDA error code seen by the calling thread inside this library (0 if none); host. */
int bsp_last_cuda_error(void);

/* ---------------------------------------------------------------------------------------------
 * bsp_group_norms — Section 3.2: the square-rooted sums of Eq. 2 / Eq. 3 (the `l2_norms(i,j)` of
 * Algorithm 1), the gamma update printed under each equation, and the regulariser's value.
 *
 *   S_g  = sum of squares of group g (float32, elements added in increasing index order)
 *   n_g  = sqrt(S_g)                                      -> norms      (if non-NULL)
 *   BSP_PEN_L2   (the paper's form):
 *       gamma_g = 1 / (n_g + eps)                         -> gamma_out  (if non-NULL)
 *       penalty = sum_g gamma'_g * n_g                    -> *penalty   (if non-NULL)
 *   BSP_PEN_L2SQ (squared-norm variant of the same update):
 *       alpha_g = 1 / (S_g + eps)                         -> gamma_out
 *       penalty = sum_g alpha'_g * S_g                    -> *penalty
 *   gamma' (alpha') is gamma_in if it is non-NULL (weights kept from an earlier milestone of
 *   Algorithm 2), else the value just computed from this W.  Pass gamma_in = NULL and read
 *   sum n_g/(n_g+eps); for the plain group-Lasso term (gamma == 1) pass a gamma_in of ones.
 *   The factor lambda of Eq. 2 / Eq. 3 is left to the caller.
 *
 * norms, gamma_in, gamma_out: float32 per-group arrays (shape by orientation, see above).
 * penalty: one float64 device scalar; it is overwritten, not accumulated.  It is summed with
 * float64 atomics, so its last bits may differ between runs.
 * Errors: BSP_ERR_ARG (W NULL, all outputs NULL, bad enum, eps < 0), BSP_ERR_SHAPE.
 */
int bsp_group_norms(const void* W, int rows, int cols, int ldw, int block, int orient,
                    float eps, int pen,
                    float* norms, const float* gamma_in, float* gamma_out, double* penalty,
                    void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_penalty_grad — the regulariser's gradient with respect to W with the penalty weights held
 * fixed, which is what Algorithm 2's inner loop needs between two gamma updates (its Adam step
 * minimises the task loss plus the reweighted l1 term):
 *   BSP_PEN_L2   (Eq. 2 / Eq. 3):  G_e = scale * gamma_g * W_e / ||W_g||_2   (0 for an all-zero group)
 *   BSP_PEN_L2SQ (squared norms):  G_e = scale * 2 * alpha_g * W_e
 * gamma: float32 per-group array (shape by orientation) from an earlier bsp_group_norms call;
 * scale: the factor lambda; grad: float32 [rows, cols] with leading dimension ldg, overwritten,
 * or added to if accumulate != 0 (so that it can be summed onto the task gradient).
 * Errors: BSP_ERR_ARG, BSP_ERR_SHAPE.
 */
int bsp_penalty_grad(const void* W, int rows, int cols, int ldw, int block, int orient, int pen,
                     const float* gamma, float scale, float* grad, int ldg, int accumulate,
                     void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_pack_bound — host-only size query for bsp_prune_pack (worst case: nothing pruned).
 *   *idx_elems = number of int32 index entries, *val_elems = number of bf16 values,
 *   *ws_bytes  = workspace bytes bsp_prune_pack / bsp_percentile_threshold need for this shape.
 * Any of the three output pointers may be NULL.
 */
int bsp_pack_bound(int rows, int cols, int block, int orient,
                   size_t* idx_elems, size_t* val_elems, size_t* ws_bytes);
/* bsp_pack_scratch_bytes — host-only: the part of that workspace bsp_prune_pack itself touches
 * (per-block counts and one flag byte per group, about 1 byte per group; the float32 region that
 * makes up the rest of bsp_pack_bound's figure belongs to bsp_percentile_threshold).  A workspace
 * of this size is enough for bsp_prune_pack alone. */
int bsp_pack_scratch_bytes(int rows, int cols, int block, int orient, size_t* bytes);

/* ---------------------------------------------------------------------------------------------
 * bsp_prune_pack — Algorithm 1 followed by the compressed storage of Section 3.1 (one index per
 * kept row or column of a block, not one per weight).
 *
 * Decision (Algorithm 1 prunes a group iff its l2 norm <= t_b): group g is KEPT iff
 *   S_g > t_b * t_b, both sides float32, S_g as defined for bsp_group_norms; a negative t_b
 *   keeps everything.  t_b = 0 keeps exactly the groups holding a non-zero weight, i.e. the
 *   group-level form of Algorithm 2's Mask = (W != 0).
 *   t_b is `threshold`, or the device scalar *threshold_dev if that pointer is non-NULL (so
 *   that bsp_percentile_threshold can feed it without a host round trip).
 *   If keep_per_block >= 0 the threshold is ignored and exactly keep_per_block groups are kept
 *   in every block: the largest S_g, ties broken towards the lower group index (needs at most
 *   BSP_TOPK_MAX_GROUPS groups per block, else BSP_ERR_UNSUPPORTED).
 *
 * Outputs (canonical packed form; nb = number of blocks, kc_b = kept groups of block b):
 *   keep        uint8 per-group flags (1 = kept), per-group array shape; may be NULL
 *   blk_ptr     int32 [nb + 1], blk_ptr[b] = number of kept groups in blocks before b
 *   idx         int32 [blk_ptr[nb]]: for each block its kept group indices (column indices for
 *               C, row indices for R), strictly ascending
 *   vals        bf16: for each block in order one dense tile copied bit for bit from W, at
 *               element offset block * blk_ptr[b]:  C: [block, kc_b] row-major (row r of the
 *               row-block, kept columns in order);  R: [kc_b, block] row-major
 *   kept_weights int64 device scalar = block * blk_ptr[nb]; compression rate = rows*cols / it.
 *               May be NULL.
 * idx and vals must have room for bsp_pack_bound's counts.  ws/ws_bytes: scratch of at least
 * bsp_pack_scratch_bytes (bsp_pack_bound's *ws_bytes also serves), 256-byte aligned; contents are
 * undefined afterwards.
 * Errors: BSP_ERR_ARG, BSP_ERR_SHAPE, BSP_ERR_WORKSPACE, BSP_ERR_UNSUPPORTED.
 */
#define BSP_TOPK_MAX_GROUPS 8192
int bsp_prune_pack(const void* W, int rows, int cols, int ldw, int block, int orient,
                   float threshold, const float* threshold_dev, int keep_per_block,
                   uint8_t* keep, int32_t* blk_ptr, int32_t* idx, void* vals,
                   int64_t* kept_weights, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_prune_pack_static — bsp_prune_pack for callers that cannot provide a workspace.
 * (Library convenience; the paper has no counterpart to this call.)
 *
 * Some hosts of this library may not allocate device memory at the point where they prune: a
 * serving process whose framework reserved the whole GPU for its own pool at start-up (a later
 * cudaMalloc simply fails), a latency-critical thread that must avoid cudaMalloc/cudaFree because
 * they can synchronise the device, or a plug-in that is handed input and output buffers and
 * nothing else.  For them this variant keeps bsp_prune_pack's scratch (per-block counts and
 * per-group flags) in a fixed array of BSP_STATIC_SCRATCH_BYTES inside the library's device
 * image.  Each GPU on which the library is loaded holds that array until the process ends.
 *
 * Arguments, outputs, semantics and results are exactly those of bsp_prune_pack without
 * ws/ws_bytes; inputs and outputs are still the caller's buffers.  The call itself allocates
 * and frees nothing.
 *  - Limit: shapes whose bsp_pack_scratch_bytes exceeds BSP_STATIC_SCRATCH_BYTES (just under
 *    4.2 million groups; 8192 x 8192 at block 32 fits, at block 16 it does not) are refused with BSP_ERR_UNSUPPORTED before
 *    anything is launched.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array.  It needs no clearing between calls (each call
 *    writes every scratch byte before reading it), but two calls that can overlap on the GPU —
 *    different streams, or different host threads without ordering — race on it: serialise them.
 */
#define BSP_STATIC_SCRATCH_BYTES (4u << 20)
int bsp_prune_pack_static(const void* W, int rows, int cols, int ldw, int block, int orient,
                          float threshold, const float* threshold_dev, int keep_per_block,
                          uint8_t* keep, int32_t* blk_ptr, int32_t* idx, void* vals,
                          int64_t* kept_weights, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_percentile_threshold — Section 3.1 lets the threshold be given or follow from a
 * percentile.  Per-matrix threshold for a target compression rate c = total/kept:
 * with G groups, r = floor(G * (1 - 1/c)) groups are to be removed; *threshold_out (device
 * float) receives t_b = the float32 square root of the r-th smallest S_g, raised by single ulps
 * until t_b * t_b >= that S_g, so that Algorithm 1's `<=` removes that group and its ties.
 * r = 0 gives -1 (prune nothing).  ws as for bsp_prune_pack.
 * Errors: BSP_ERR_ARG (rate < 1), BSP_ERR_SHAPE, BSP_ERR_WORKSPACE.
 */
int bsp_percentile_threshold(const void* W, int rows, int cols, int ldw, int block, int orient,
                             double rate, float* threshold_out,
                             void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_apply_mask — Algorithm 2's retraining step W = W * Mask, with the mask given per group:
 * every element of a group whose keep flag is 0 is set to +0, in place.
 */
int bsp_apply_mask(void* W, int rows, int cols, int ldw, int block, int orient,
                   const uint8_t* keep, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_masked_adam_step — one iteration of Algorithm 2's retraining loop on one weight matrix:
 * the Adam update of W, then W = W * Mask, in one pass.  Adam as published (Kingma & Ba 2015,
 * bias-corrected; the paper names no hyper-parameters beyond the learning rate, so all are the
 * caller's):
 *   m = beta1 m + (1 - beta1) g,   v = beta2 v + (1 - beta2) g^2,
 *   W = W - lr ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay W ),
 *   then every weight of a group whose keep flag is 0 is set to +0 (the moments are updated for
 *   every weight, pruned or not, as the algorithm's order implies).
 * W, m, v: float32 [rows, cols] with leading dimension ldw, updated in place (the optimiser's
 * weights are float32: a bf16 weight cannot absorb steps of the paper's size); grad float32 with
 * leading dimension ldg (task gradient, plus bsp_penalty_grad's term during reweighted training).
 * keep: per-group flags as written by bsp_prune_pack for (block, orient), or NULL = no mask (the
 * reweighted-training loop's plain update; block and orient are then ignored).  step >= 1.
 * W_bf16: nullable bf16 [rows, cols] (ldb) output, the updated masked weights rounded to nearest
 * even: with ldb = cols it is the execution layout that bsp_linear_planned reads.
 * Needs cols and the leading dimensions multiples of 4 and 16-byte aligned float arrays (else
 * BSP_ERR_UNSUPPORTED).  Errors: BSP_ERR_ARG (NULL, step < 1, beta outside [0, 1), eps < 0),
 * BSP_ERR_SHAPE.
 *
 * bsp_repack_values — the packed values of an UPDATED W under fixed kept sets (orientation C):
 * Algorithm 2 fixes the mask before retraining, so Section 3.1's storage keeps blk_ptr and idx
 * and only vals changes: tile of block b = rows of the block restricted to its kept columns.
 * W: bf16 [rows, cols] (ldw); blk_ptr / idx as written by bsp_prune_pack; vals is overwritten.
 */
/* bsp_dense_mask — Algorithm 2's mask loop, element by element: mask[i, j] = 0 if W[i, j] == 0 else 1
 * (either sign of zero counts as zero).  W bf16 [rows, cols] (ldw), mask uint8 [rows, cols] (ldm).
 * The per-group keep flags of bsp_prune_pack are this mask reduced over each group; the calls of
 * this library take the flags, the dense mask is for callers that want Algorithm 2's own object. */
int bsp_dense_mask(const void* W, int rows, int cols, int ldw, uint8_t* mask, int ldm, void* stream);
int bsp_masked_adam_step(float* W, const float* grad, float* m, float* v, int rows, int cols, int ldw, int ldg,
                         const uint8_t* keep, int block, int orient,
                         float lr, float beta1, float beta2, float eps, float weight_decay, int step,
                         void* W_bf16, int ldb, void* stream);
int bsp_repack_values(const void* W, int rows, int cols, int ldw, int block,
                      const int32_t* blk_ptr, const int32_t* idx, void* vals, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_prepare_batched — the weight-side steps of the path for several matrices at once
 * (orientation C): the norms / gamma / penalty of Section 3.2, Algorithm 1's keep decision, the
 * packed storage of Section 3.1 and, optionally, bsp_linear's execution layout, in two launches
 * per 96 matrices (a small clearing kernel and one kernel that reads every weight exactly once)
 * instead of four or more per matrix.  Results are those of
 * bsp_group_norms + bsp_prune_pack (threshold mode) + bsp_linear_plan called per matrix, bit
 * for bit; the penalty is summed in a fixed order here and is reproducible run to run.
 * The kernel's bounded waits report through bsp_linear_status (BSP_ERR_TIMEOUT).
 *
 * In-place mode: a job whose `plan` pointer equals its `W` pointer gets no separate execution
 * layout.  Instead the weights of the pruned groups are overwritten with +0 inside W (Algorithm
 * 2's W = W * Mask) and nothing else of W is written; W, which must then be writable, is
 * afterwards its own execution layout (pass it to bsp_linear_planned as `plan`; that call wants
 * ldw == cols).  When W already holds zeros in every pruned group (threshold 0 on a pruned
 * matrix) this writes nothing at all.
 *
 * jobs: HOST array of n_jobs descriptors; the pointers inside are device pointers with the
 * meaning they have in the single-matrix calls.  norms, gamma_in, gamma_out, penalty, keep,
 * kept_weights, plan may be NULL (that output is skipped).  ws/ws_bytes as bsp_prune_pack.
 * block, eps and pen apply to every job.
 * Needs, for every job: cols and ldw multiples of 8, W and the float arrays 16-byte aligned,
 * cols <= 4096, rows/block <= 1024 (else BSP_ERR_UNSUPPORTED, and nothing is launched: use the
 * per-matrix calls).  Other errors as the per-matrix calls; all jobs are validated before the first launch.
 */
typedef struct bsp_layer_job {
  const void* W; int rows, cols, ldw;
  float threshold; const float* threshold_dev;
  float* norms; const float* gamma_in; float* gamma_out; double* penalty;
  uint8_t* keep; int32_t* blk_ptr; int32_t* idx; void* vals; int64_t* kept_weights;
  void* plan; size_t plan_bytes;
  void* ws; size_t ws_bytes;
} bsp_layer_job;
int bsp_prepare_batched(const bsp_layer_job* jobs, int n_jobs, int block, float eps, int pen, void* stream);
/* bsp_percentile_threshold_batched — bsp_percentile_threshold (Section 3.1's percentile) for the
 * matrices of a job array in two launches (orientation C): job i's threshold for the target rate
 * rates[i] (HOST array of n_jobs doubles, each >= 1) is written to the device float that the job
 * names as threshold_dev, where a following bsp_prepare_batched on the same array reads it.
 * Uses each job's ws (as bsp_percentile_threshold does); only W, rows, cols, ldw, threshold_dev,
 * ws and ws_bytes of a job are read.  Results are those of the single-matrix call, bit for bit.
 * Errors: BSP_ERR_ARG (NULL threshold_dev or ws, rate < 1), BSP_ERR_SHAPE, BSP_ERR_WORKSPACE. */
int bsp_percentile_threshold_batched(const bsp_layer_job* jobs, int n_jobs, int block, const double* rates,
                                     void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_linear — the pruned linear layer (orientation C packed form):
 *   Y[t, b*block + r] = act( sum_{j < kc_b} X[t, idx_b[j]] * vals_b[r, j] + bias[b*block + r] )
 * which equals act(X (W * Mask)^T + bias), the layer Algorithm 2 retrains (W = W * Mask) and
 * Sections 3.1 / 4.4 deploy.  Products are bf16 x bf16 accumulated in float32 on the tensor
 * cores; bias (bf16 [n_out], may be NULL) is added in float32; act is BSP_ACT_NONE or
 * BSP_ACT_GELU (0.5 x (1 + erf(x / sqrt 2)), evaluated in float32); the result is rounded to
 * bf16 (nearest even).
 *
 * bsp_linear_plan_bytes (host): bytes of the private execution layout for a packed matrix.
 * bsp_linear_plan: builds that layout in `plan` (device, 256-byte aligned) from the canonical
 *   packed form; do it once per packed matrix, reuse for any number of bsp_linear_planned calls.
 *   Needs k_in to be a multiple of 8 and at most 12288 (else BSP_ERR_UNSUPPORTED).
 * bsp_linear_planned: runs the layer from a plan.
 * bsp_linear: plan + run in one call, the plan living in ws (>= bsp_linear_plan_bytes).
 *
 * Alignment for the tensor-core path: X, Y and plan 16-byte aligned, k_in, ldx and ldy multiples
 * of 8 elements.  Other cases run on a slower CUDA-core kernel with identical semantics.
 * Device-side waits in the tensor-core kernel are bounded (bsp_set_wait_limit_ms); if one expires
 * the kernel stops early and records it: bsp_linear_status (host; synchronises the stream) then returns
 * BSP_ERR_TIMEOUT and Y is undefined.  It returns BSP_OK otherwise.
 * Errors: BSP_ERR_ARG, BSP_ERR_SHAPE (block does not divide n_out), BSP_ERR_WORKSPACE, BSP_ERR_CUDA.
 */
int bsp_linear_plan_bytes(int n_out, int k_in, int block, size_t* bytes);
int bsp_linear_plan(const int32_t* blk_ptr, const int32_t* idx, const void* vals,
                    int n_out, int k_in, int block, void* plan, size_t plan_bytes, void* stream);
/* bsp_linear_plan_r — the execution layout from the orientation-R packed form (Algorithm 1's own
 * geometry: strips of `block` columns, kept row segments; idx holds row indices, tiles are
 * [kc, block]).  n_out = rows of W, k_in = cols; plan_bytes >= n_out * k_in * 2 rounded up to 256.
 * The resulting plan feeds bsp_linear_planned / bsp_linear_chain like any other (their `block`
 * argument is then only checked to divide n_out: pass 1).
 * Errors: BSP_ERR_ARG, BSP_ERR_SHAPE (block does not divide k_in), BSP_ERR_WORKSPACE. */
int bsp_linear_plan_r(const int32_t* blk_ptr, const int32_t* row_idx, const void* vals,
                      int n_out, int k_in, int block, void* plan, size_t plan_bytes, void* stream);
/* bsp_linear_plan_t — the TRANSPOSED execution layout PT[k, n] = (W * Mask)[n, k] from the
 * orientation-C packed form.  It is the operand of the backward product with respect to the
 * activations of the masked layer that Algorithm 2 retrains (W = W * Mask):
 *   dX = dY (W * Mask)  =  bsp_linear_planned(plan_t, n_out := k_in, k_in := n_out, block := 1,
 *                                             X := dY [tokens, n_out], bias := NULL, act := none, Y := dX).
 * plan_bytes as bsp_linear_plan_bytes(n_out, k_in, block).  Errors as bsp_linear_plan. */
int bsp_linear_plan_t(const int32_t* blk_ptr, const int32_t* idx, const void* vals,
                      int n_out, int k_in, int block, void* plan_t, size_t plan_bytes, void* stream);
/* bsp_linear_backward_weight — the weight gradient of the masked layer that Algorithm 2 retrains
 * (W = W * Mask after every step):  dW = (dY^T X) * Mask, with dY [tokens, n_out] (ldy) and
 * X [tokens, k_in] (ldx) bf16, float32 accumulation over the tokens on the tensor cores, dW
 * [n_out, k_in] (lddw) rounded to bf16.  keep: per-group flags [n_out/block, k_in] as written by
 * bsp_prune_pack (orientation C); groups with flag 0 are written as +0; NULL = no mask.
 * Needs 16-byte aligned pointers and n_out, k_in and the leading dimensions multiples of 8
 * (else BSP_ERR_UNSUPPORTED).  Bounded waits as bsp_linear_planned: check bsp_linear_status. */
int bsp_linear_backward_weight(const void* dY, int ldy, const void* X, int ldx, int tokens, int n_out, int k_in,
                               int block, const uint8_t* keep, void* dW, int lddw, void* stream);
int bsp_linear_planned(const void* plan, int n_out, int k_in, int block,
                       const void* X, int tokens, int ldx, const void* bias, int act,
                       void* Y, int ldy, void* stream);
/* bsp_linear_planned with the kernel variant chosen by the caller: BSP_LINEAR_AUTO (what
 * bsp_linear_planned does), BSP_LINEAR_ONE_CTA (128 x BN tiles, one CTA each) or
 * BSP_LINEAR_CTA_PAIR (256 x 256 tiles shared by a cluster of two CTAs, one third less operand
 * traffic from L2).  Results are identical up to float32 summation order (the same in both). */
typedef enum { BSP_LINEAR_AUTO = 0, BSP_LINEAR_ONE_CTA = 1, BSP_LINEAR_CTA_PAIR = 2 } bsp_linear_algo;
/* May be OR-ed into `algo`: the caller vouches that the plan was complete before the work that
 * immediately precedes this call in the stream was launched (the usual case in a chain of layers:
 * the weights are old, only X is fresh).  The one-CTA kernel then starts fetching weight tiles
 * while that work is still finishing.  Never set it when the preceding kernel writes the plan. */
#define BSP_LINEAR_PLAN_STABLE 0x100
/* May be OR-ed into `algo`: write the output TRANSPOSED, Y := YT [n_out, tokens] row-major with
 * leading dimension ldy >= tokens (a multiple of 8), bit for bit the transpose of what the call
 * writes otherwise.  It is the form bsp_linear_gathered reads its activations in, so a chain of
 * layers can hand them on without a separate transposing pass.  One-CTA kernel only
 * (BSP_LINEAR_CTA_PAIR with this flag is BSP_ERR_UNSUPPORTED). */
#define BSP_LINEAR_OUT_TRANSPOSED 0x200
int bsp_linear_planned_ex(const void* plan, int n_out, int k_in, int block,
                          const void* X, int tokens, int ldx, const void* bias, int act,
                          void* Y, int ldy, int algo, void* stream);
int bsp_linear(const int32_t* blk_ptr, const int32_t* idx, const void* vals,
               int n_out, int k_in, int block,
               const void* X, int tokens, int ldx, const void* bias, int act,
               void* Y, int ldy, void* ws, size_t ws_bytes, void* stream);
int bsp_linear_status(void* stream);
/* bsp_set_wait_limit_ms — how long one device-side wait of the tensor-core and batched weight-side
 * kernels may last before the kernel gives up (default 2000; 1 <= ms <= 600000), for kernels
 * launched afterwards on the current device.  Host call; synchronises the device first, so kernels
 * already in flight keep the limit they started with.  Errors: BSP_ERR_ARG, BSP_ERR_CUDA.
 *
 * bsp_wait_selftest — runs the bail-out path once, without any fault: a single CTA sets up an
 * mbarrier and tensor memory as the tensor-core kernels do, then waits through the same bounded-wait
 * helpers on a barrier and on a counter that nothing ever signals.  Both waits run out at the
 * configured limit; the CTA records it, sits out a fixed millisecond for operations in flight, frees
 * its tensor memory and returns by itself.  Afterwards bsp_linear_status returns BSP_ERR_TIMEOUT once
 * and BSP_OK again from then on.  *expired (host, may be NULL) receives the number of waits that ran
 * out (2), *waited_ns (host, may be NULL) how long the mbarrier wait lasted.  Synchronises the stream;
 * takes about the wait limit, so lower the limit first. */
int bsp_set_wait_limit_ms(int ms);
int bsp_wait_selftest(int* expired, long long* waited_ns, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_linear_chain — several pruned linear layers, each reading the chain input or an earlier
 * layer's output, in one persistent launch (the paper's deployment target, Sections 3.1 / 4.4, is
 * the whole encoder; this runs an encoder layer's linears QKV -> attention output -> FFN-up ->
 * FFN-down back to back).  Every op computes what bsp_linear_planned computes:
 *   Y_i = act_i( S_i (W_i * Mask_i)^T + b_i ),  S_i = columns [src_col, src_col + k_in) of X
 *   (src = -1) or of Y_src (0 <= src < i).
 * Row-tile m of an op needs only row-tile m of its source, so no grid-wide barrier separates the
 * layers: the CTAs take output tiles of all ops from one list through a ticket counter, and a tile
 * waits (bounded) until the source rows it reads have been stored; see csrc/bsp_linear_chain.cu.
 * Outputs are bit-identical to calling bsp_linear_planned op by op.
 *
 * ops: HOST array of n_ops (1..8) descriptors; plan / bias / Y are device pointers as in
 * bsp_linear_planned (plan from bsp_linear_plan or bsp_prepare_batched).  ws: device scratch of
 * bsp_linear_chain_ws_bytes bytes, 256-byte aligned (per-row-tile completion counters and the
 * ticket counter; cleared by the call).  Needs the alignment of the tensor-core path for every op
 * and for src_col (multiple of 8), else BSP_ERR_UNSUPPORTED; one persistent CTA per SM.
 * Bounded waits as bsp_linear_planned: check bsp_linear_status.
 */
typedef struct bsp_chain_op {
  const void* plan; int n_out, k_in, block;
  const void* bias; int act;
  void* Y; int ldy;
  int src;       /* -1: the chain input X; i >= 0: the output of op i (must be an earlier op) */
  int src_col;   /* first column of the source that this op reads */
} bsp_chain_op;
int bsp_linear_chain_ws_bytes(int n_ops, int tokens, size_t* bytes);
int bsp_linear_chain(const bsp_chain_op* ops, int n_ops, const void* X, int tokens, int ldx,
                     void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_linear_gathered — the same layer, Y = act(X (W * Mask)^T + b), with the pruned work skipped:
 * for each row-block only the kept columns of X are fetched and multiplied (Section 3.1: only the
 * non-zero columns of a block take part in the product; Section 4.4: the compact storage is what
 * saves computation).  Flops executed = 2 * tokens * kept weights (rounded up to 16 kept columns
 * per block), against 2 * tokens * n_out * k_in for bsp_linear_planned.  Every gathered element
 * feeds only `block` multiply-adds per token, so this pays off for tall blocks and high
 * compression; bsp_linear_planned is the better choice for block 16 at 3x.
 *
 * XT: the activations TRANSPOSED, bf16 [k_in, tokens] row-major with leading dimension ldxt
 * (a kept column of X is then a contiguous row); make it with bsp_transpose, or have the producer
 * of X write it that way.  Y [tokens, n_out] row-major as elsewhere.
 * gplan: the gather plan, private scratch derived from the packed form by bsp_linear_gather_plan
 * (per 64 kept columns of a row-block: the weight tile in tensor-core layout, the column numbers,
 * a stage descriptor), bsp_linear_gather_plan_bytes bytes (worst case: nothing pruned), 256-byte
 * aligned; built once per pruned matrix and reused for every batch.
 * Needs block in {16, 32, 64, 128}, k_in < 32768, tokens / ldxt / ldy multiples of 8, 16-byte
 * aligned XT, Y and bias (else BSP_ERR_UNSUPPORTED).  Bounded waits as bsp_linear_planned: check
 * bsp_linear_status.  Errors: BSP_ERR_ARG, BSP_ERR_SHAPE, BSP_ERR_WORKSPACE, BSP_ERR_CUDA.
 *
 * bsp_transpose — XT[c, r] = X[r, c] for a row-major bf16 matrix [rows, cols] (rows, cols and
 * both leading dimensions multiples of 8, 16-byte aligned pointers, else BSP_ERR_UNSUPPORTED).
 */
int bsp_linear_gather_plan_bytes(int n_out, int k_in, int block, size_t* bytes);   /* host-only */
int bsp_linear_gather_plan(const int32_t* blk_ptr, const int32_t* idx, const void* vals,
                           int n_out, int k_in, int block, void* gplan, size_t gplan_bytes, void* stream);
int bsp_transpose(const void* X, int rows, int cols, int ldx, void* XT, int ldxt, void* stream);
int bsp_linear_gathered(const void* gplan, int n_out, int k_in, int block,
                        const void* XT, int tokens, int ldxt, const void* bias, int act,
                        void* Y, int ldy, void* stream);
/* bsp_linear_gathered_ex — the same; with out_transposed != 0 the output is written as
 * YT [n_out, tokens] row-major (ldy >= tokens, a multiple of 8), bit for bit the transpose of the
 * other form: the next gathered layer of a chain reads it as its XT. */
int bsp_linear_gathered_ex(const void* gplan, int n_out, int k_in, int block,
                           const void* XT, int tokens, int ldxt, const void* bias, int act,
                           void* Y, int ldy, int out_transposed, void* stream);

/* ---------------------------------------------------------------------------------------------
 * bsp_linear_route / bsp_linear_run / bsp_linear_tune — one call for the pruned linear layer
 * (Sections 3.1 / 4.4) over both routes: the zero-expanded one (bsp_linear_planned_ex) and the
 * gathering one (bsp_linear_gathered_ex).  The caller states what it has in a bsp_linear_call:
 *   plan / gplan      the weights' execution layouts (either may be NULL);
 *   kept_weights      host copy of the packed matrix's kept-weight count, or -1 (unknown: the
 *                     estimate then assumes nothing was pruned);
 *   X, ldx / XT, ldxt the activations, row-major [tokens, k_in] and/or transposed [k_in, tokens];
 *   Y, ldy / YT, ldyt where the output goes: exactly one of the two (YT = [n_out, tokens]);
 *   plan_stable       as BSP_LINEAR_PLAN_STABLE.
 * A route is possible when its weight layout and its activation layout are both given (zero-expanded:
 * plan and X; gathering: gplan and XT, block in {16, 32, 64, 128}).
 *   bsp_linear_route  host-only: the route BSP_ROUTE_AUTO would take.  With both possible it compares
 *                     estimates fitted to measurements on B200 (dense product at the zero-expanded
 *                     kernel's rate, against 0.62 us per 64 kept columns and 0.45 us per row-block per
 *                     128-token tile on every SM), which are good to about 10 %.
 *   bsp_linear_run    runs `route` (or the automatic choice) and reports it in *route_taken (may be NULL).
 *   bsp_linear_tune   times every possible route on the caller's own buffers (one untimed launch, then
 *                     `reps` timed ones per route; the outputs are written) and returns the faster one and
 *                     both times in milliseconds (-1 for a route that is not possible).  Synchronises the
 *                     stream; not for use during stream capture.
 * Errors: BSP_ERR_ARG (no possible route, both or neither output, bad route), BSP_ERR_SHAPE, and
 * whatever the chosen route's own call returns. */
typedef enum { BSP_ROUTE_AUTO = 0, BSP_ROUTE_ZERO_EXPANDED = 1, BSP_ROUTE_GATHERED = 2 } bsp_route;
typedef struct bsp_linear_call {
  const void* plan; const void* gplan; long long kept_weights;
  int n_out, k_in, block;
  const void* X; int ldx;
  const void* XT; int ldxt;
  int tokens;
  const void* bias; int act;
  void* Y; int ldy;
  void* YT; int ldyt;
  int plan_stable;
} bsp_linear_call;
int bsp_linear_route(const bsp_linear_call* call, int* route);
int bsp_linear_run(const bsp_linear_call* call, int route, int* route_taken, void* stream);
int bsp_linear_tune(const bsp_linear_call* call, int reps, int* best_route, float* ms_zero_expanded,
                    float* ms_gathered, void* stream);

/* bsp_linear_cuda_core — the same layer computed straight from the packed form by a plain
 * CUDA-core kernel (one thread per output, float32 accumulation in index order).  It is what
 * bsp_linear falls back to when the alignment rules above do not hold, and is exported so the
 * two paths can be compared.  No workspace. */
int bsp_linear_cuda_core(const int32_t* blk_ptr, const int32_t* idx, const void* vals,
                         int n_out, int k_in, int block,
                         const void* X, int tokens, int ldx, const void* bias, int act,
                         void* Y, int ldy, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BSP_H_ */
