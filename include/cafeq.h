/*
 * cafeq.h - C ABI of the CafeQ per-matrix optimisation path on one NVIDIA B200 (sm_100a).
 *
 * CafeQ (arXiv 2511.19705) quantises a weight matrix W after applying a learned invertible
 * transform M, chosen without calibration data by minimising a proxy of the quantisation error:
 *   single matrix  (Section 4, Eq. 3):   || M^-1 Q(M W) - W ||_F ,  M block-diagonal (Section 4.1)
 *   coupled pair   (Section 4.2, Eq. 5): || Q(W1 M) Q(M^-1 W2) - W1 W2 ||_F  (PQE)
 * trained through differentiable surrogates (Eq. 4; the LogSumExp of channel maxima, Section 4.2)
 * and, for pairs, followed by the alternating adaptive rounding of Algorithm 1 (Section 5).
 *
 * Conventions of this library
 *   - A weight is row-major [d_out, d_in] bf16 with `ld` elements between rows.  Quantisation
 *     groups are `group` consecutive entries along d_in (0 = one group per row); one fp32 scale
 *     per (row, group): s = absmax / qmax, qmax = 2^(bits-1) - 1, code = clamp(rne(u / s)).
 *   - A block-diagonal operator is fp32 T[nbT][k][k] (row-major blocks).  On CAFEQ_AXIS_IN it acts
 *     on the d_in index:  U[o, B*k+i] = sum_j T[B/replicas][i][j] W[o, B*k+j];  on CAFEQ_AXIS_OUT
 *     on the d_out index: U[B*k+i, c] = sum_j T[B/replicas][i][j] W[B*k+j, c].  `replicas`
 *     consecutive blocks of the matrix share one operator block (grouped-query heads).
 *     CAFEQ_APPLY_TT applies the transpose of every block instead.
 *   - Every operand of a transform product is rounded to bf16 first (the tensor-core operand
 *     type); products accumulate in fp32.  The transform that is deployed is therefore bf16(M).
 *   - All pointers are DEVICE pointers unless the comment says "host".  Every call only enqueues
 *     work on `stream` (a cudaStream_t passed as void*; NULL = default stream) and returns; results
 *     are valid after the caller synchronises that stream.  No call allocates or frees device
 *     memory: scratch comes from the caller's workspace `ws` (size from cafeq_workspace_size,
 *     256-byte aligned).  Calls that share a workspace must be ordered on one stream.
 *   - Return value: a cafeq_status.  Argument errors are found on the host before anything is
 *     launched and leave all outputs untouched.  Conditions found on the device (a singular block,
 *     a non-finite value) are written to the int32 `status` word (first error wins; the caller
 *     zeroes it) and later kernels of the same call skip their work.
 */
#ifndef CAFEQ_H_
#define CAFEQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CAFEQ_OK = 0,
  CAFEQ_ERR_INVALID_ARG = 1,
  CAFEQ_ERR_UNSUPPORTED = 2, /* shape / bits / group combination not covered */
  CAFEQ_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  CAFEQ_ERR_CUDA = 4,        /* a launch failed; cudaGetLastError has the detail */
  CAFEQ_ERR_SINGULAR = 5,    /* device: a transform block has no usable pivot */
  CAFEQ_ERR_NONFINITE = 6,   /* device: NaN or Inf met in a transformed weight */
  CAFEQ_ERR_TIMEOUT = 7,     /* device: a bounded wait inside a kernel ran out */
  CAFEQ_ERR_TOO_LARGE = 8    /* problem needs more scratch than the built-in buffer of cafeq_rtn_noalloc holds */
} cafeq_status;

enum { CAFEQ_AXIS_IN = 0, CAFEQ_AXIS_OUT = 1 };
enum { CAFEQ_APPLY_T = 0, CAFEQ_APPLY_TT = 1 };
enum { CAFEQ_PREC_BF16 = 0 };
/* loss kinds: what the backward pass differentiates */
enum {
  CAFEQ_LOSS_SURROGATE = 0, /* single: Eq. 4 */
  CAFEQ_LOSS_L2_STE = 1,    /* single: Eq. 3 with a straight-through rounding derivative */
  CAFEQ_LOSS_LSE = 2,       /* pair: LogSumExp of group maxima (+ orthonormality penalty) */
  CAFEQ_LOSS_PQE_STE = 3,   /* pair: Eq. 5 squared, straight-through */
  CAFEQ_LOSS_SUMSQ = 4,     /* pair, Appendix D.1: mean of the squared group maxima of U + the same of V */
  CAFEQ_LOSS_SUMSQ_WEIGHTED = 5 /* pair, Appendix D.1: ||V||_F mean(sq. maxima of U) + ||U||_F mean(sq. maxima of V) */
};
/* CAFEQ_OPT_CAYLEY (pairs only, Appendix D.2's strictly orthonormal baseline): momentum V <- beta1 V + grad,
 * A = V M^T - M V^T, M <- (I + lr/2 A)^-1 (I - lr/2 A) M per block (solved by five fixed-point rounds: choose lr so
 * that lr ||A|| stays well below 1); a rotation stays a rotation.  The momentum lives in the optimiser state's
 * first-moment slot. */
enum { CAFEQ_OPT_GD = 0, CAFEQ_OPT_ADAM = 1, CAFEQ_OPT_CAYLEY = 2 };
#define CAFEQ_OPT_STATE_HEADER 4 /* floats before the moment arrays of an optimiser state */
/* flags for the forward/backward calls */
enum {
  CAFEQ_FLAG_EXACT_LOSS = 1, /* also evaluate the quantised loss (l2 proxy / PQE) */
  CAFEQ_FLAG_NO_GRAD = 2,    /* forward only */
  CAFEQ_FLAG_GENERIC = 4,    /* force the shape-agnostic kernels (debugging aid) */
  CAFEQ_FLAG_WARM_MINV = 8   /* Minv holds an approximate inverse (e.g. the previous step's) to refine */
};
enum { CAFEQ_ROUND_ALG1 = 0, CAFEQ_ROUND_LEARNED_OFFSETS = 1 };
enum { CAFEQ_OFFSETS_NONE = 0, CAFEQ_OFFSETS_HARD_U8 = 1, CAFEQ_OFFSETS_SOFT_F32 = 2 };

/* One weight matrix and how it is transformed and quantised. */
typedef struct {
  uint32_t struct_size; /* sizeof(cafeq_matrix_desc), for versioning */
  int32_t d_out, d_in;  /* W is [d_out, d_in] row-major bf16 */
  int64_t ld;           /* elements between rows, >= d_in */
  int32_t bits;         /* 2..8 */
  int32_t group;        /* along d_in; 0 => per-channel */
  int32_t tblock;       /* transform block size k; 0 => no transform */
  int32_t taxis;        /* CAFEQ_AXIS_IN | CAFEQ_AXIS_OUT */
  int32_t trole;        /* CAFEQ_APPLY_T | CAFEQ_APPLY_TT (how cafeq_rtn uses the operator it is given) */
  int32_t replicas;     /* consecutive matrix blocks sharing one operator block, >= 1 */
  int32_t compute_prec; /* CAFEQ_PREC_BF16 */
} cafeq_matrix_desc;

/* Optimiser and loss settings (Section 4.1: gradient descent; Appendix D: Adam, t, lambda_orth). */
typedef struct {
  uint32_t struct_size;
  int32_t loss_kind;  /* CAFEQ_LOSS_* */
  int32_t optimizer;  /* CAFEQ_OPT_* */
  float lr, beta1, beta2, eps;
  float lambda_orth;  /* weight of ||M M^T - I||_F / sqrt(h) (pairs) */
  float lse_t;        /* LogSumExp temperature t (pairs) */
  float kappa;        /* constant of Eq. 4; <= 0 selects 1/(2^bits - 1)^2 */
  int32_t steps;
  int32_t eval_every; /* evaluate the quantised loss every n steps (0 = never) */
  int32_t resume;     /* non-zero: opt_state comes from an earlier call on the same problem (its stored
                         inverse is refined instead of inverting from scratch) */
} cafeq_opt_cfg;

/* Scratch bytes needed by the calls on d1 (and d2 for pair calls; NULL otherwise).  `bytes` is a host pointer.
 * cfg = NULL: the size that serves every entry point and every mode for these descriptors (matrix-sized fp32 and
 * bf16 buffers: about 30 bytes per weight).
 * cfg given: the size cafeq_optimize_single / cafeq_optimize_pair need for exactly that configuration.  For the
 * paper's objectives (CAFEQ_LOSS_SURROGATE / CAFEQ_LOSS_LSE) with eval_every = 0, block size 64 / 128 / 256 and a
 * shape the tensor-core pass covers, nothing matrix-sized is needed: the per-(row, group) records (16 bytes per
 * group) and the k x k scratch.  The size assumes 16-byte aligned weight rows; a call whose weights do not qualify
 * then returns CAFEQ_ERR_WORKSPACE. */
int cafeq_workspace_size(const cafeq_matrix_desc* d1, const cafeq_matrix_desc* d2, const cafeq_opt_cfg* cfg,
                         size_t* bytes);

/* Round-to-nearest quantisation of T o W (Eq. 1 in its symmetric absmax form, after the transform of
 * Section 4): codes int8 [d_out, d_in] (row stride d_in), scales fp32 [d_out, d_in/group].
 * T = NULL or tblock = 0 quantises W itself.  T is used as given (CAFEQ_APPLY_T) or transposed; no
 * inverse is taken here. */
int cafeq_rtn(const cafeq_matrix_desc* d, const void* W, const float* T, int8_t* codes, float* scales,
              void* ws, size_t ws_bytes, void* stream);

/* Scratch bytes cafeq_rtn takes from its workspace for this descriptor (host out), with (has_transform != 0) or
 * without an operator, for 16-byte aligned W and 8-byte aligned codes: 0 without a transform when the group is
 * 32 / 64 / 128 / 256 (one streaming kernel, ws may then be NULL); the per-group records when the tensor-core pass
 * covers the transformed call; matrix-sized buffers otherwise.  Never more than cafeq_workspace_size(d, NULL, NULL). */
int cafeq_rtn_workspace_size(const cafeq_matrix_desc* d, int has_transform, size_t* bytes);

/* cafeq_rtn for callers that cannot allocate device memory and therefore have no workspace to hand
 * over: code running inside a memory-pool or allocator callback, between the driver calls of another
 * library that forbids allocation, in a process whose memory budget is already fixed, or anywhere a
 * cudaMalloc (which synchronises the whole device) would stall other streams.  (The paper has no
 * counterpart; the arithmetic and the outputs are exactly those of cafeq_rtn.)
 *   - Scratch is a buffer of CAFEQ_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU
 *     that loads the library holds it from then until the process exits.  Inputs and outputs are still
 *     the caller's.  Neither this call nor anything under it calls cudaMalloc, cudaFree or an
 *     allocating library routine.
 *   - A call whose scratch need (cafeq_rtn_workspace_size) exceeds CAFEQ_NOALLOC_SCRATCH_BYTES is refused with
 *     CAFEQ_ERR_TOO_LARGE before anything is launched (use cafeq_rtn with your own workspace then).
 *   - The first call on each device looks up the buffer's device address (with that device current);
 *     make that first call outside any stream capture.  Later calls only enqueue kernels.
 *   - All calls in the process share the one buffer per device, and it keeps whatever the last call
 *     left there.  Nothing in this path reads scratch before writing it, so nothing needs clearing, but
 *     two calls that can overlap on the GPU (different streams, no dependency) race on it: order them. */
#define CAFEQ_NOALLOC_SCRATCH_BYTES (16u << 20)
int cafeq_rtn_noalloc(const cafeq_matrix_desc* d, const void* W, const float* T, int8_t* codes, float* scales,
                      void* stream);

/* One forward+backward evaluation for a single matrix (Section 4.1).
 *   M       [nb,k,k] fp32 transform parameters; the transform applied is bf16(M).
 *   Minv    optional out [nb,k,k]: inverse of bf16(M) as computed on the device; with
 *           CAFEQ_FLAG_WARM_MINV also an input, a nearby inverse that Newton-Schulz steps refine (block sizes
 *           64/128/256; the result is checked on the device and recomputed by elimination if it did not converge).
 *   offsets optional rounding offsets [d_out,d_in] (row stride d_in): uint8 {0,1} or fp32 in [0,1]
 *           (offsets_kind); code = clamp(floor(u/s) + offset) instead of round-to-nearest.
 *   losses  out fp32[4]: {surrogate (Eq. 4), ||M^-1 Q(MW) - W||_F^2 (Eq. 3), ||W||_F^2, 0};
 *           entries 1,2 only with CAFEQ_FLAG_EXACT_LOSS or loss_kind = CAFEQ_LOSS_L2_STE.
 *   gradM   out [nb,k,k] fp32 gradient of the chosen loss (ignored with CAFEQ_FLAG_NO_GRAD).
 *   grad_offsets optional out fp32 [d_out,d_in] (row stride d_in): d loss / d offset for soft offsets, only with
 *           offsets_kind = CAFEQ_OFFSETS_SOFT_F32 and loss_kind = CAFEQ_LOSS_L2_STE (else CAFEQ_ERR_INVALID_ARG).
 *           With the scales kept at their round-to-nearest values Uhat = s (floor(u/s) + offset), so the gradient is
 *           s * dL/dUhat = s * 2 M^-T (M^-1 (Uhat - U)).  The paper has no learned offsets (its adaptive rounding
 *           is Algorithm 1); a caller learns them by a projected step offset <- clip(offset - lr * grad, 0, 1) and
 *           hardens them at 1/2.
 * With offsets (either kind) an entry that attains its group's absmax is always coded +-qmax (its quotient is
 * exactly +-qmax, where floor is discontinuous) and its offset has no effect and no gradient.
 * The operator is M on d->taxis (trole is ignored: the parameter itself is applied). */
int cafeq_proxy_loss_fwd_bwd(const cafeq_matrix_desc* d, const void* W, const float* M, float* Minv,
                             const void* offsets, int offsets_kind, int loss_kind, float kappa, int flags,
                             float* losses, float* gradM, float* grad_offsets, int32_t* status, void* ws,
                             size_t ws_bytes, void* stream);

/* `cfg->steps` optimisation steps on a single matrix (Section 4.1: gradient descent on Eq. 4 from the
 * caller's initial M; Adam selectable).  M is updated in place (fp32 master parameters).
 * opt_state: fp32 [CAFEQ_OPT_STATE_HEADER + 3*nb*k*k] = {step count, 3 reserved floats, Adam first moments, Adam
 * second moments, inverse of the last step's transform}, 16-byte aligned (so that each array is: the kernels move
 * them 16 bytes at a time); required for Adam, optional for gradient descent.  Carrying it over between calls with
 * cfg->resume = 1 resumes a run; the caller zeroes it before the first call.  loss_history: out fp32 [steps, 2] =
 * {surrogate, quantised loss or NaN when not evaluated at that step}. */
int cafeq_optimize_single(const cafeq_matrix_desc* d, const void* W, float* M, float* opt_state,
                          const cafeq_opt_cfg* cfg, float* loss_history, int32_t* status, void* ws,
                          size_t ws_bytes, void* stream);

/* P = W1 W2 of Section 4.2 in stored layout: W1 is stored [h, d1] (= W1^T), W2 is stored [d3, r*h]
 * (= W2^T), r = d2->replicas; P[x, y] = sum_j W1[(B/r)*k + j', x] W2[y, B*k + j'] over all blocks B of W2.
 * P is fp32 [d1, d3] row-major.  With a workspace (cafeq_workspace_size(d1, d2)) and every dimension a multiple
 * of 64 the product runs on the tensor cores; otherwise (ws may be NULL) on a plain fp32 kernel. */
int cafeq_pair_product(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                       const void* W2, float* P, void* ws, size_t ws_bytes, void* stream);

/* One forward+backward evaluation for a coupled pair (Section 4.2).  d1 describes W1 (stored [h, d1],
 * transformed on CAFEQ_AXIS_OUT by M^T, i.e. U = W1 M), d2 describes W2 (stored [d3, r*h], transformed
 * on CAFEQ_AXIS_IN by bf16(inv(bf16(M))), i.e. V = M^-1 W2).  d1->tblock == d2->tblock == k,
 * M is [h/k, k, k].
 *   P       optional fp32 [d1, d3] from cafeq_pair_product; needed for PQE.
 *   losses  out fp32[4]: {LSE + lambda*orth, LSE, orth penalty, PQE^2 (Eq. 5 squared) or 0}.
 *   gradM   out [h/k, k, k].
 * loss_kind CAFEQ_LOSS_LSE is the surrogate of Section 4.2 / App. D; CAFEQ_LOSS_SUMSQ and CAFEQ_LOSS_SUMSQ_WEIGHTED are the
 * alternatives of App. D.1 over the same group maxima (losses[1] then holds their value instead of the LogSumExp).
 * CAFEQ_LOSS_PQE_STE differentiates Eq. 5 squared itself with
 * the quantiser passed straight through (only the scale's dependence on its group's arg-max entry is kept): P is
 * required, losses[0] = losses[3] = PQE^2, lambda_orth is ignored (losses[2] = 0), and every dimension must be
 * a multiple of 64 with k a multiple of 32 (CAFEQ_ERR_UNSUPPORTED otherwise); its products run on the tensor cores. */
int cafeq_pair_loss_fwd_bwd(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                            const void* W2, const float* M, const float* P, int loss_kind, float lse_t,
                            float lambda_orth, int flags, float* losses, float* gradM, int32_t* status,
                            void* ws, size_t ws_bytes, void* stream);

/* `cfg->steps` optimisation steps on a pair (Appendix D: Adam on the LogSumExp surrogate with the
 * orthonormality penalty).  loss_history: out fp32 [steps, 2] = {loss, PQE^2 or NaN}.  P as above
 * (NULL => PQE never evaluated). */
int cafeq_optimize_pair(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                        const void* W2, float* M, float* opt_state, const float* P, const cafeq_opt_cfg* cfg,
                        float* loss_history, int32_t* status, void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1 (Section 5) on the transformed pair U = W1 M, V = M^-1 W2 with Q = the group quantiser of
 * each descriptor: codes1/scales1 for U (stored [h, d1]), codes2/scales2 for V (stored [d3, r*h]);
 * pqe_history: out fp32 [2*iters + 1], the product error (Eq. 5, un-squared) after independent rounding and
 * after every half-iteration.  M = NULL rounds the untransformed pair.  iters <= 15.
 * The pseudo-inverses are computed by Newton-Schulz iteration on the tensor cores (three-term bf16 splits, fp32
 * accumulate), not by an SVD.  With r replicas the second factor's update is expand(pinv(Uhat^T) P) / r (which
 * equals the printed update when Uhat^T has full column rank) and the first factor's least-squares target is
 * P pinv(fold(Vhat^T)); both reduce to the printed lines for r = 1.
 * Every dimension (h, d1, d3) must be a multiple of 64 and the block size a multiple of 32, else
 * CAFEQ_ERR_UNSUPPORTED.
 *
 * mode = CAFEQ_ROUND_LEARNED_OFFSETS (the paper has no counterpart; it is this library's definition of the learned
 * rounding offsets the workload statement names): scales stay at their round-to-nearest values and the codes are
 * floor(x) + rho with soft offsets rho in [0, 1] started at the fractional parts (zero error).  Each of the `iters`
 * iterations (1..30) moves the first factor's offsets along d = (dL/dUhat) / (s * H), H = 2 * squared norm of the
 * other factor's matching row, L = Eq. 5 squared, with an exact line search (L is quadratic in one factor's offsets)
 * and projects to [0, 1]; does the same for the second factor at the updated first; then pushes both by
 * lambda_t (2 rho - 1), lambda_t = 0.5 t / iters, towards the nearer of {0, 1}.  At the end rho is hardened at 1/2.  pqe_history: fp32 [iters + 2] = {independent round-to-nearest, the soft iterate entering each
 * iteration, the hardened result}.  Any shape (the products run on the plain fp32 kernel). */
int cafeq_adaptive_round(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                         const void* W2, const float* M, int iters, int mode, int8_t* codes1, float* scales1,
                         int8_t* codes2, float* scales2, float* pqe_history, int32_t* status, void* ws,
                         size_t ws_bytes, void* stream);

/* Pack int8 codes [d_out, d_in] (row stride d_in) into `bits`-bit fields: u = q + qmax, little-endian bit
 * stream along d_in per row, row stride d_in*bits/8 bytes (4-bit: low nibble first; 3-bit: code i at
 * bits 3i..3i+2).  The paper fixes no layout (Section 5 only asks for fast dequantisation); this is the
 * library's.  d_in*bits must be a multiple of 8. */
int cafeq_pack(const cafeq_matrix_desc* d, const int8_t* codes, uint8_t* packed, void* stream);

/* ---- inference side (Section 4.1's cost argument and its table of extra FLOPs / wall-clock time) -------------
 * A matrix quantised as Q(W o T) on its input axis is used as  y = W x = (W o T) (T^-T x): the activations are
 * multiplied by the block-diagonal inverse before the (dequantised) matrix product.  cafeq_apply_transform does that
 * multiplication on a bf16 activation matrix X [d_out = tokens, d_in] (row pitch d->ld):
 *     Y[o, B k + i] = sum_j P[B][i][j] X[o, B k + j],   P = T (d->trole = CAFEQ_APPLY_T) or T^T (CAFEQ_APPLY_TT),
 * (CAFEQ_AXIS_OUT: the operator acts on the row index instead), with the operator rounded to bf16, fp32
 * accumulation, and Y written as bf16 [d_out, d_in], dense (row pitch d_in).  T: fp32 [d_in / k, k, k] on the device.
 * d->group and d->bits are not used.  Shapes the tensor-core pass covers (k in {64, 128, 256}, d_in a multiple of
 * 256, 16-byte aligned rows) run in one kernel; all others on the shape-agnostic kernels with an fp32 copy of Y in
 * the workspace.  Workspace: cafeq_apply_workspace_size bytes (sized for 16-byte aligned rows; CAFEQ_ERR_WORKSPACE
 * otherwise).  Device status word as elsewhere (may be NULL). */
int cafeq_apply_workspace_size(const cafeq_matrix_desc* d, size_t* bytes);
int cafeq_apply_transform(const cafeq_matrix_desc* d, const void* X, const float* T, void* Y, int32_t* status, void* ws,
                          size_t ws_bytes, void* stream);

/* Unpack the bit stream written by cafeq_pack and dequantise: What[o, c] = bf16(scales[o, c / group] * q[o, c]),
 * What bf16 [d_out, d_in] with row pitch ldo >= d_in (elements).  d_in must be a multiple of 8. */
int cafeq_dequant(const cafeq_matrix_desc* d, const uint8_t* packed, const float* scales, void* What, long long ldo,
                  void* stream);

/* ---- one decoder layer at a time --------------------------------------------------------------------------
 * Section 6 quantises a model layer by layer; within a layer every matrix (block-diagonal transform, Section 4.1)
 * and every coupled pair (Section 4.2) is an independent optimisation problem.  The calls below advance all
 * problems of a layer together.  Each step computes exactly what cafeq_optimize_single (loss CAFEQ_LOSS_SURROGATE,
 * Eq. 4) and cafeq_optimize_pair (loss CAFEQ_LOSS_LSE, Appendix D) compute for that problem; only the launch
 * structure differs: the k x k algebra runs once over the operator blocks of all problems, and the transform pass
 * and the backward take all matrices of a form in one launch each.
 *
 * One problem.  pair = 0: d1 / W1 describe the matrix, d2 / W2 are ignored.  pair = 1: d1 / W1 and d2 / W2 as in
 * cafeq_optimize_pair.  M [nb,k,k] is updated in place; opt_state as in the per-problem calls (required for Adam;
 * its stored-inverse slot is not used here); loss_history fp32 [steps, 2] = {loss, NaN}.  cfg: loss_kind must be
 * CAFEQ_LOSS_SURROGATE (single) or CAFEQ_LOSS_LSE (pair), eval_every 0 (the quantised losses are evaluated by the
 * per-problem calls); cfg.steps and cfg.resume are ignored.
 * Limits: at most 8 problems; one block size (128 or 256) and one group size (64 or 128) for the whole layer;
 * every matrix must be a shape the tensor-core pass covers (d_in a multiple of 256 on the input axis; d_out a
 * multiple of k and d_in of 128 on the output axis; 16-byte aligned rows).  Otherwise CAFEQ_ERR_UNSUPPORTED and the
 * per-problem calls apply.  M and opt_state must be 16-byte aligned. */
typedef struct {
  uint32_t struct_size; /* sizeof(cafeq_layer_problem) */
  int32_t pair;
  cafeq_matrix_desc d1, d2;
  const void* W1;
  const void* W2;
  float* M;
  float* opt_state;
  float* loss_history;
  cafeq_opt_cfg cfg;
} cafeq_layer_problem;

/* Scratch bytes for the layer calls on these problems (`probs` and `bytes` are host pointers; the device pointers
 * inside the problems are not read).  Includes an fp16 copy of every weight (2 bytes per weight). */
int cafeq_layer_workspace_size(const cafeq_layer_problem* probs, int n, size_t* bytes);

/* Once per layer, before the first cafeq_optimize_layer on `ws`: makes the fp16 copies of the weights that the
 * backward reads (scaled by a power of two per matrix; exact for every bf16 value within 2^-38 of the matrix
 * maximum) and inverts the initial transforms.  The workspace then carries that state (copies, last inverse)
 * between cafeq_optimize_layer calls: pass the same problems and the same `ws`, and let nothing else write it. */
int cafeq_layer_prepare(const cafeq_layer_problem* probs, int n, int32_t* status, void* ws, size_t ws_bytes, void* stream);

/* `steps` optimisation steps of every problem (forward, backward, parameter update), enqueued on `stream`.
 * Step i writes row i of every loss_history.  Every step refines the inverse of the previous step's transforms
 * (Newton-Schulz, checked on the device, recomputed by elimination when it did not converge). */
int cafeq_optimize_layer(const cafeq_layer_problem* probs, int n, int steps, int32_t* status, void* ws, size_t ws_bytes,
                         void* stream);

/* Benchmark aid (host out, synchronises the device): how many operator blocks, summed over all steps since
 * cafeq_layer_prepare on this workspace, were re-inverted by elimination because the iterative refinement of the
 * previous step's inverse had not converged (a step that changed a transform by more than about half its norm). */
int cafeq_layer_debug_fallbacks(const cafeq_layer_problem* probs, int n, void* ws, size_t ws_bytes, int* count);

/* Tuning knob of the layer step, process-wide (the paper has no counterpart; results do not depend on it).
 * dual = 1 (default): when a layer has matrices on both axes, their transform passes share one persistent launch and
 * their sparse backwards another; dual = 0: one launch per axis.  pass_out_pct / bwd_out_pct (> 0, default 130 / 80):
 * cost of an output-axis tile in percent of an input-axis tile of the same bytes, which sets how the 148 CTAs of a
 * shared launch are divided between the two lists; <= 0 keeps the current value.  Returns CAFEQ_ERR_INVALID_ARG
 * unless dual is 0 or 1 and the percentages are at most 1000. */
int cafeq_debug_set_layer_launch(int dual, int pass_out_pct, int bwd_out_pct);

const char* cafeq_status_string(int status);
int cafeq_version(void);
/* Tuning knob, process-wide (the paper has no counterpart).  overlapped = 0 (default): one problem runs alone:
 * narrow product tiles (about one CTA per SM) and every SM on every pass, for the lowest latency of a single chain
 * of kernels.  overlapped = 1: the caller runs several problems concurrently in different streams (the matrices
 * and pairs of a layer are independent), so a kernel should cost few SM-microseconds rather than finish early:
 * the k x k products of the block algebra take the widest output tile (fewest CTAs), and the transform pass and
 * the sparse backward give a small matrix fewer CTAs (at least 14 tiles each).  Results do not depend on it.
 * Returns CAFEQ_ERR_INVALID_ARG unless 0 or 1. */
int cafeq_set_overlap_mode(int overlapped);

/* Number of kernels this library has launched in the calling process so far (host counter, for
 * benchmarks that must state how many of the library's kernels ran inside a timed region). */
long long cafeq_debug_launch_count(void);
/* Benchmark aid: time selected kernels of later calls with CUDA events recorded on the launching stream.
 * begin() creates `capacity` event pairs (host objects, no device memory); read() waits for the recorded
 * events, writes up to `capacity` durations in milliseconds and kernel kinds (1 transform pass on the
 * shape-agnostic kernels, 2 sparse backward, 3 block inverse, 4 dense pair product, 5 fused tensor-core
 * transform pass) to HOST arrays, sets *count and releases the events.
 * Not thread-safe; launches beyond the capacity are simply not timed. */
int cafeq_debug_timer_begin(int capacity);
int cafeq_debug_timer_read(float* ms, int* kinds, int* count);

/* Self-test of the kernels' bounded waits (the paper has no counterpart).  Every wait inside the kernels of this
 * library is limited (2 s); when one runs out the kernel raises CAFEQ_ERR_TIMEOUT in the status word, its roles
 * leave their loops and it returns.  This call runs that wait helper in a one-thread kernel on a barrier that nothing
 * completes, with the limit given here (nanoseconds), then lets the thread complete the barrier itself and wait
 * again.  Device outputs: `status` receives CAFEQ_ERR_TIMEOUT (if it was 0), result[0] = 1 when the first wait gave
 * up, result[1] = 1 when the second succeeded.  Nothing in it can hang: no other thread is waited for. */
int cafeq_debug_wait_probe(unsigned long long limit_ns, int32_t* status, int* result, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CAFEQ_H_ */
