/*
 * lsgd.h -- C ABI of the Leader SGD step for a population of P workers in G groups that all live
 * on ONE CUDA device (sm_100a).
 *
 * Method: "Leader Stochastic Gradient Descent for Distributed Training of Deep Learning Models:
 * Extension" (Teng, Gao, Chalus, Choromanska, Goldfarb, Weller).  One synchronous step is
 *   1. every worker's stochastic gradient g_i at x_i                   (Section 2.2, Eq. (1))
 *   2. every worker's election loss        (Section 2.2; estimated losses: Section 3.1.3)
 *   3. local leaders (argmin inside each group) and the global leader (argmin over all workers)
 *                                              (Section 2.2, definitions below the multi-leader objective)
 *   4. the fused update                                                 (Eq. (1), eta-scaled as in
 *      x_i <- x_i - eta g_i - eta lambda_l (x_i - x_ll(i)) - eta lambda_g (x_i - x_gl)   Section 3.1.1)
 *      on steps t = 0, tau, 2 tau, ... and the plain step x_i <- x_i - eta g_i in between
 *      (communication period: Section 3.1.2).
 * The paper's leader broadcast is an on-device read: leaders are kept as row indices.
 *
 * General conventions
 *   - Every pointer is documented as HOST or DEVICE.  DEVICE buffers are owned by the caller, must
 *     stay alive and unmodified by others until the stream has drained, and are never freed here.
 *   - Worker parameters are a row-major float matrix x[P][ld]; row i is worker i; ld >= d is the
 *     row stride in floats and a multiple of 32; columns d..ld-1 are padding that callers keep 0.
 *   - All work is enqueued on the stream given at creation; grad / elect / step never synchronise.
 *   - Functions return an lsgd_status; nothing throws, aborts or prints.  Argument errors are
 *     detected on the host before anything is launched.
 *   - A handle is not thread-safe; distinct handles are independent.
 */
#ifndef LSGD_H_
#define LSGD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define LSGD_API __attribute__((visibility("default")))
#else
#define LSGD_API
#endif

typedef struct lsgd_ctx* lsgd_handle;

typedef enum {
  LSGD_OK = 0,
  LSGD_ERR_INVALID_ARG = 1,  /* NULL where not allowed, P < 1, tau < 1, non-finite eta, ld < d ...  */
  LSGD_ERR_BAD_GROUPS = 2,   /* G < 1, G > P, group id out of range, or an empty group               */
  LSGD_ERR_ALIGNMENT = 3,    /* a DEVICE pointer is not 16-byte aligned, or ld is not a multiple of 32 */
  LSGD_ERR_STATE = 4,        /* call order: pull step before any election, step without a gradient;
                                or grad / elect / step called while another device is current        */
  LSGD_ERR_CUDA = 5,         /* a CUDA runtime call or launch failed (no usable device included)     */
  LSGD_ERR_UNSUPPORTED = 6,  /* combination not implemented (documented at the argument)             */
  LSGD_ERR_DEVICE_FLAG = 7,  /* a kernel recorded a bounded-wait / bounds failure in its status word */
  LSGD_ERR_TOO_LARGE = 8     /* the problem exceeds a fixed capacity stated at the entry point       */
} lsgd_status;

typedef enum {
  LSGD_OBJ_EXTERNAL = 0,     /* caller writes g and supplies the loss vector                         */
  LSGD_OBJ_QUADRATIC = 1,    /* f(x) = 1/2 sum_k a_k (x_k - b_k)^2                                    */
  LSGD_OBJ_MATCOMP = 2,      /* factorised matrix completion on observed entries                     */
  LSGD_OBJ_MLP = 3,          /* population of ReLU MLP classifiers, bf16 GEMMs, fp32 accumulate      */
  LSGD_OBJ_PSD_COMPLETION = 4 /* F(X) = 1/4 ||M - X X^T||_F^2, the paper's own completion experiment  */
} lsgd_objective;

/* How the per-element formulas (update, quadratic gradient) are evaluated.  Storage is always fp32. */
typedef enum {
  LSGD_ARITH_FP64 = 0,       /* default: fp64, one IEEE operation per printed operation, one final
                                rounding to fp32 (what a double-precision restatement of Eq. (1) gives) */
  LSGD_ARITH_FP64_FMA = 1,   /* fp64 with fused multiply-adds                                        */
  LSGD_ARITH_FP32 = 2        /* fp32 fused multiply-adds                                             */
} lsgd_arithmetic;

/* Diagonal quadratic (the positive-definite quadratic model of Section 3.3 with diagonal Hessian):
 * g_i = a (x_i - b) + sigma * noise_i,  election loss f(x_i).                                      */
typedef struct {
  const float* a;            /* DEVICE float[ld], a_k > 0                                            */
  const float* b;            /* DEVICE float[ld]                                                     */
  float sigma;               /* weight of the per-step noise array given to lsgd_grad                */
} lsgd_quadratic_desc;

/* Matrix completion with factors: row i of x is [X (n_rows x rank) | Y (n_cols x rank)], row-major.
 * Minibatch loss (1/(2B)) sum (<X_r, Y_c> - v)^2 over B observed entries per worker per step, given
 * to lsgd_grad as positions into the observed list; election loss = mean squared residual over the
 * fixed held-out positions.  (Low-rank completion is the paper's motivating example, Section 2.1.)
 * batch <= 32768 (LSGD_ERR_UNSUPPORTED beyond): duplicates are summed exactly in a 2^-44 fixed-point
 * accumulator whose range also needs every contribution |e * y / B| < 2^4 (see LSGD_DEVFLAG_OVERFLOW). */
typedef struct {
  int32_t n_rows, n_cols, rank;
  int32_t n_obs;
  const int32_t* obs_r;      /* DEVICE int32[n_obs] row of each observed entry                       */
  const int32_t* obs_c;      /* DEVICE int32[n_obs] column                                           */
  const float* obs_v;        /* DEVICE float[n_obs] value                                            */
  int32_t batch;             /* B, entries per worker per step                                       */
  int32_t n_heldout;
  const int32_t* heldout_pos;/* DEVICE int32[n_heldout] positions into the observed list             */
  void* scratch;             /* DEVICE, 256-byte aligned, lsgd_matcomp_scratch_bytes(P, ld) bytes: the exact
                                fixed-point gradient accumulator (8 bytes per worker-parameter), owned by the
                                caller and cleared by lsgd_create.  NULL: the library allocates it itself     */
  uint64_t scratch_bytes;
} lsgd_matcomp_desc;

/* Positive semi-definite low-rank completion, the paper's motivating example (Section 2.1; settings in
 * the supplement's "Low-Rank Matrix Completion Experiments"): row i of x is X_i (n x r, row-major),
 * F(X) = 1/4 ||M - X X^T||_F^2, exact gradient (X X^T - M) X (batch LGD, no sampling; lsgd_grad ignores
 * its batch argument), election loss F(X_i).  d must equal n * r; r <= 128.                         */
typedef struct {
  int32_t n, r;
  const float* M;            /* DEVICE float[n*n], row-major, symmetric; shared by all workers       */
  void* scratch;             /* DEVICE, 256-byte aligned, lsgd_psd_scratch_bytes(r, P, ld) bytes (0 above rank 32):
                                the fp64 partial gradients of the two CTAs that share a row block at small
                                rank, owned by the caller.  NULL: the library allocates them itself          */
  uint64_t scratch_bytes;
} lsgd_psd_desc;

/* MLP population: row i of x is [W1 | b1 | W2 | b2 | W3 | b3]; W_l is [n_out][n_in] row-major
 * (input index contiguous); each segment starts at a multiple of 32 floats (see
 * lsgd_mlp_param_offsets).  Loss: mean softmax cross-entropy.  Matrix products take bf16 operands
 * (weights, inputs, stored activations and back-propagated deltas are rounded to bf16, ties to
 * even) and accumulate in fp32.                                                                   */
#define LSGD_MLP_MAX_LAYERS 3
typedef struct {
  int32_t dims[LSGD_MLP_MAX_LAYERS + 1]; /* n_in, hidden, hidden, n_classes                          */
  int32_t batch;             /* training samples per worker per step (multiple of 8, at most 1024)   */
  int32_t pool;              /* number of rows of pool_x                                             */
  const float* pool_x;       /* DEVICE float[pool][dims[0]] training samples                         */
  const int32_t* pool_y;     /* DEVICE int32[pool] labels                                            */
  int32_t n_heldout;         /* election batch (multiple of 128)                                     */
  const float* held_x;       /* DEVICE float[n_heldout][dims[0]]                                     */
  const int32_t* held_y;     /* DEVICE int32[n_heldout]                                              */
  void* scratch;             /* DEVICE, lsgd_mlp_scratch_bytes() bytes, 1024-byte aligned            */
  uint64_t scratch_bytes;
  int32_t loss_window;       /* 0: lsgd_elect(h, NULL) evaluates the held-out loss.  K in 1..64: it elects
                                on the mean of each worker's minibatch losses over the last K lsgd_grad
                                calls, the estimator of the paper's deep-network runs (Section 4.1: the
                                last 10 / 64 batches); fewer than K are averaged until K have been seen */
} lsgd_mlp_desc;

typedef struct {
  uint32_t struct_size;      /* = sizeof(lsgd_config)                                                */
  int32_t P;                 /* workers (the paper's n * l)                                          */
  int32_t G;                 /* groups  (the paper's n)                                              */
  const int32_t* group_of;   /* HOST int32[P], values in [0, G), every group non-empty; copied       */
  int64_t d;                 /* parameters per worker                                                */
  int64_t ld;                /* row stride in floats, ld >= d, ld % 32 == 0                          */
  float eta;                 /* learning rate eta                                                    */
  float lambda_l;            /* pull strength towards the local leader  (the paper's lambda)         */
  float lambda_g;            /* pull strength towards the global leader (the paper's lambda_G)       */
  int32_t tau;               /* communication period tau >= 1                                        */
  int32_t objective;         /* lsgd_objective                                                       */
  const void* objective_desc;/* HOST pointer to the matching *_desc (copied), NULL for EXTERNAL      */
  float* x;                  /* DEVICE float[P*ld], 16-byte aligned, updated in place                */
  float* g;                  /* DEVICE float[P*ld] gradients.  May be NULL only for QUADRATIC, whose
                                gradient is then evaluated inside the update kernel (no g traffic)  */
  void* stream;              /* cudaStream_t; NULL = the legacy default stream                       */
  int32_t arithmetic;        /* lsgd_arithmetic                                                      */
  uint32_t flags;            /* bit set of LSGD_FLAG_*; 0 = defaults                                 */
  /* --- only read with LSGD_FLAG_ALGORITHM1 (see below); leader_copies also with LSGD_FLAG_EAGD --- */
  float gamma_l;             /* searching scope gamma: every step pulls with strength eta gamma / tau  */
  float gamma_g;             /* gamma_G: every step pulls with strength eta gamma_G / tau_G           */
  int32_t tau_g;             /* global communication period tau_G >= 1                               */
  float* leader_copies;      /* DEVICE float[(G+1)*ld], 16-byte aligned: the leaders' parameters as of
                                their last election (rows 0..G-1 local, row G global); library-written */
  /* --- the optimiser of the paper's deep-network runs (Section 4.1); only read when v != NULL --- */
  float* v;                  /* DEVICE float[P*ld] momentum buffers, 16-byte aligned, caller-owned and
                                caller-initialised (zeros for a fresh run), updated in place by lsgd_step.
                                NULL: the step of Eq. (1), momentum and weight_decay are ignored.
                                Non-NULL: with d = g + weight_decay x,  v <- momentum v + d,
                                x <- x - eta (d + momentum v) - [the two pulls of Eq. (1) on a pull step]:
                                Nesterov momentum with the decay inside the gradient; the pulls stay
                                outside the buffer (the paper does not say how they combine), so that
                                momentum = weight_decay = 0 gives Eq. (1) again.  Needs cfg.g; not
                                combined with LSGD_FLAG_MLP_FUSED_STEP or LSGD_FLAG_ALGORITHM1
                                (LSGD_ERR_UNSUPPORTED).                                              */
  float momentum;            /* Nesterov momentum mu, finite (the paper uses 0.9)                    */
  float weight_decay;        /* L2 decay coefficient, finite (the paper uses 1e-4)                   */
} lsgd_config;

/* MLP objective: on steps that are not pull steps, let lsgd_grad apply x <- x - eta g itself: for W1 and
 * W2 inside the epilogue of the weight-gradient products (g is then not written for those two blocks), for
 * the biases and W3 in the kernel that sums their gradients over the batch.  Same arithmetic as the update
 * kernel, bit-identical result; lsgd_step then only advances the step counter.  With this flag, lsgd_grad
 * may be called once per step and lsgd_elect(h, NULL) must not be called between lsgd_grad and lsgd_step on
 * a non-pull step (LSGD_ERR_STATE): the parameters are already advanced.  Off by default.            */
#define LSGD_FLAG_MLP_FUSED_STEP 1u

/* MATCOMP objective: on steps that are not pull steps, lsgd_grad leaves the gradient as exact fixed-point
 * sums in the library's accumulator and does not write g; lsgd_step takes x <- x - eta g straight from those
 * sums, touching only the entries the minibatch reached (same arithmetic, bit-identical x).  lsgd_grad may
 * then be called once per step (a second call before lsgd_step: LSGD_ERR_STATE).  Ignored with a momentum
 * buffer or LSGD_FLAG_ALGORITHM1.  Off by default.                                                  */
#define LSGD_FLAG_MATCOMP_FUSED_STEP 4u

/* The schedule of the paper's Algorithm 1, run synchronously, instead of the fused Eq. (1) step:
 *   lsgd_elect at t = 0          initialisation: both elections, leader parameters copied, no pull;
 *   lsgd_grad, lsgd_step         x_i <- x_i - eta g_i - eta (gamma/tau)(x_i - x~^j) - eta (gamma_G/tau_G)(x_i - x~)
 *                                where x~^j, x~ are the COPIES in leader_copies (stale between
 *                                communications, as in the paper), then t <- t + 1;
 *   lsgd_elect when tau | t or tau_G | t (t after the step; LSGD_ERR_STATE otherwise):
 *                                if tau | t:   local leaders re-elected, x_i <- x_i - eta lambda (x_i - x~^j), copies refreshed;
 *                                if tau_G | t: global leader re-elected, x_i <- x_i - eta lambda_G (x_i - x~), copy refreshed.
 * All pulls are scaled by eta (Section 3.1.1; pass coefficient / eta for the unscaled form the listing
 * prints).  When both periods are due and loss == NULL, the order of the listing is kept: the objective's
 * loss is evaluated, the local leaders are elected and the local pull applied, then the loss is evaluated
 * AGAIN on the pulled parameters and the global leader elected from that second vector (lsgd_get_loss then
 * returns the second vector).  A loss vector given by the caller serves both elections of a communication.
 * LSGD_FLAG_MLP_FUSED_STEP is ignored in this mode.                                                   */
#define LSGD_FLAG_ALGORITHM1 2u

/* Elastic averaging (EAGD / EASGD), the method the paper compares LGD with (supplement, "Low-Rank Matrix
 * Completion Experiments"): instead of a leader, every worker is pulled towards a center variable X~,
 *   x_i <- x_i - eta g_i - eta lambda (x_i - X~),   X~ <- (1 - P eta lambda) X~ + P eta lambda (1/P) sum_i x_i,
 * both from the values at time t, on the steps t = 0, tau, 2 tau, ...; plain steps in between.  lambda is
 * lambda_l; lambda_g must be 0 (LSGD_ERR_INVALID_ARG).  leader_copies (DEVICE float[(G+1)*ld], as above) is
 * required: row G holds X~ (readable by the caller once the stream has drained), row 0 is scratch for the new
 * center; the library clears the buffer at creation and starts X~ at the workers' mean on the first step (the
 * paper does not say where it starts).  No election takes place: lsgd_elect is not needed, and the groups
 * play no role.  Not combined with LSGD_FLAG_ALGORITHM1, the fused-step flags or a momentum buffer
 * (LSGD_ERR_UNSUPPORTED).  A comparison line: it reuses the pull kernels and is not tuned.               */
#define LSGD_FLAG_EAGD 8u

/* Validates the configuration on the host, copies the group map, builds the group tables and
 * allocates O(P + G) words of device state plus reduction scratch for the objective's election
 * loss.  Large scratch is the caller's: the MLP's in lsgd_mlp_desc.scratch, MATCOMP's gradient accumulator
 * (8 bytes per worker-parameter) and PSD_COMPLETION's partial gradients (16 bytes per worker-parameter at ranks
 * up to 32) in the scratch field of their descriptors; only when that field is NULL does the library allocate
 * the buffer itself, here.  Nothing is allocated after this call.  Returns LSGD_ERR_CUDA if no CUDA device is
 * usable.  *out is NULL on failure.                                                              */
LSGD_API lsgd_status lsgd_create(const lsgd_config* cfg, lsgd_handle* out);

/* Step 1: stochastic gradients of all workers at the current x (Eq. (1): g_t^{j,i}).
 * batch is objective-specific, a DEVICE pointer valid until the stream has drained:
 *   EXTERNAL  ignored (the caller has written g);
 *   QUADRATIC const float noise[P*ld] (standard normal draws) or NULL for the exact gradient;
 *             with cfg.g == NULL nothing is launched: the gradient is evaluated in lsgd_step;
 *   MATCOMP   const int32_t pos[P*batch], positions into the observed list (duplicates add up);
 *   MLP       const int32_t idx[P*batch], rows of pool_x.                                          */
LSGD_API lsgd_status lsgd_grad(lsgd_handle h, const void* batch);

/* Steps 2+3: election.  loss is a DEVICE float[P] of election losses, or NULL to evaluate the
 * objective's own election loss at the current x first (not available for EXTERNAL).  Writes the
 * local leaders and the global leader to device state.  Order on losses: -inf < finite < +inf <
 * NaN, -0 == +0; ties go to the lowest worker index.  Callers normally call it on the steps with
 * t % tau == 0 only; electing more often is legal (the analysis allows any guiding point).        */
LSGD_API lsgd_status lsgd_elect(lsgd_handle h, const float* loss);

/* Step 4: the fused update, pull form iff t % tau == 0 (t = number of lsgd_step calls so far),
 * then t <- t + 1.  On a pull step every right-hand side is x at time t, although x is updated in
 * place.  LSGD_ERR_STATE if a pull step comes before any election, or if no gradient was
 * provided since the previous step (EXTERNAL is exempt: g is the caller's).                      */
LSGD_API lsgd_status lsgd_step(lsgd_handle h);

/* Frees the device state.  The caller's buffers are untouched.  NULL is accepted.                */
LSGD_API lsgd_status lsgd_destroy(lsgd_handle h);

/* Accessors.  They synchronise the stream and are not part of the step.                          */
LSGD_API lsgd_status lsgd_get_leaders(lsgd_handle h, int32_t* local_leaders /* HOST int32[G] */,
                             int32_t* global_leader /* HOST int32[1] */);
/* Overrides the elected leaders (enqueued on the stream; the next pull step uses them).  local_leaders: HOST
 * int32[G] with local_leaders[j] a member of group j, or NULL to keep the elected ones; global_leader: a worker
 * index, or -1 to keep the elected one.  The global leader need not be one of the local leaders.  Uses: a
 * population whose groups live on several devices (Section 2.2 maps a group to a node: the global leader may
 * then be a row received from another device, see paper_1905_10395_b200/sharded.py), re-running a step with
 * the leaders of a reference run when two losses are within rounding of each other, restoring a checkpoint.
 * Counts as an election for the step protocol; the leader statistics are not changed.
 * LSGD_ERR_BAD_GROUPS if an index is out of range or not in its group.                              */
LSGD_API lsgd_status lsgd_set_leaders(lsgd_handle h, const int32_t* local_leaders, int32_t global_leader);
/* A population whose groups live on several devices (Section 2.2 maps a group to a node; see
 * paper_1905_10395_b200/sharded.py): the global election across devices, in two device-side halves around ONE
 * exchange of 8 bytes per device.  A handle then holds its device's own workers first (n_own rows, in global
 * order) followed by a guest row that receives the global leader's parameters when another device owns it.
 *
 * lsgd_shard_best_key  after lsgd_elect: packs the best of the first n_own workers' election losses with that
 *   worker's GLOBAL index (global_index: DEVICE int32[n_own]) into *key_out (DEVICE int64[1], enqueued on the
 *   stream): (orderable loss << 32) | global index, an unsigned key whose minimum over all devices is the
 *   global leader under the rule of lsgd_elect (ties to the lowest global index).
 * lsgd_shard_pick_global  given every device's key (keys: DEVICE int64[world], e.g. from an all-gather), takes
 *   the minimum, points this handle's global leader at its own best worker (if my_rank won) or at guest_row, and
 *   returns result (HOST int32[3]) = {winning rank, the winner's global worker index, this device's best own
 *   worker (its row is what the winning device sends)}.  Synchronises the stream once.
 * The caller then broadcasts the winner's row into the other devices' guest rows and calls lsgd_step; the update
 * kernels read local memory only.  LSGD_ERR_STATE before any election.                                  */
LSGD_API lsgd_status lsgd_shard_best_key(lsgd_handle h, int32_t n_own, const int32_t* global_index, int64_t* key_out);
LSGD_API lsgd_status lsgd_shard_pick_global(lsgd_handle h, const int64_t* keys, int32_t world, int32_t my_rank,
                                            int32_t guest_row, int32_t* result);
LSGD_API lsgd_status lsgd_get_loss(lsgd_handle h, float* loss /* HOST float[P]: losses of the last election */);
LSGD_API lsgd_status lsgd_get_step(lsgd_handle h, int64_t* t);
/* Mean minibatch loss of every worker from the last lsgd_grad (MLP objective only; LSGD_ERR_UNSUPPORTED
 * otherwise).  The paper's deep-network runs elect on a running mean of such training losses
 * (Section 4.1); here it is reported for monitoring and parity checks.                             */
LSGD_API lsgd_status lsgd_get_train_loss(lsgd_handle h, float* loss /* HOST float[P] */);
/* The hidden activations the last lsgd_grad stored for its backward pass (MLP objective only), as bf16 bit
 * patterns: h1 HOST uint16[P][batch][dims[1]], h2 HOST uint16[P][batch][dims[2]] (either may be NULL).  They
 * hold every ReLU decision of that step, so a parity check can verify them against its own pre-activations
 * and then follow the same decisions where a pre-activation is within rounding of zero.  Synchronises.   */
LSGD_API lsgd_status lsgd_mlp_get_activations(lsgd_handle h, uint16_t* h1, uint16_t* h2);
/* Times each worker has been global / local leader so far (the leader statistics of Section 4.2). */
LSGD_API lsgd_status lsgd_get_leader_counts(lsgd_handle h, int32_t* global_counts /* HOST int32[P] */,
                                   int32_t* local_counts /* HOST int32[P] */);
/* Reads and clears the device status word; LSGD_ERR_DEVICE_FLAG if any kernel has set it.  Bits:
 *   LSGD_DEVFLAG_BAD_LEADER   a leader index outside [0, P) reached an update kernel (the pull was skipped);
 *   LSGD_DEVFLAG_WAIT_TIMEOUT a bounded wait on a copy / tensor-core barrier ran out (about one second): the
 *                             kernel left its loops and returned, its output is incomplete;
 *   LSGD_DEVFLAG_BAD_INDEX    a batch position, sample index or observed row / column out of range: that
 *                             entry was skipped before anything was dereferenced;
 *   LSGD_DEVFLAG_OVERFLOW     MATCOMP: a gradient contribution e * y / B was not finite or reached 2^4 in
 *                             magnitude, the range of the fixed-point accumulator (2^-44 resolution, at most
 *                             2^15 contributions per entry: batch <= 32768, LSGD_ERR_UNSUPPORTED beyond);
 *                             the contribution was not added -- a diverging worker is reported instead of
 *                             being turned into finite garbage.                                          */
#define LSGD_DEVFLAG_BAD_LEADER 1u
#define LSGD_DEVFLAG_WAIT_TIMEOUT 2u
#define LSGD_DEVFLAG_BAD_INDEX 4u
#define LSGD_DEVFLAG_OVERFLOW 8u
LSGD_API lsgd_status lsgd_check_device(lsgd_handle h, uint32_t* flag_out /* HOST, may be NULL */);
/* Self-test of the bounded device waits (test support; the paper has no counterpart).  Every wait of the
 * copy pipelines in the update kernels and of the copy / tensor-core pipelines in the product kernels is limited
 * by a clock budget after which the kernel records LSGD_DEVFLAG_WAIT_TIMEOUT and returns instead of hanging.
 * This call runs that same wait routine (which = 0: the update kernels', 1: the product kernels') in a one-warp
 * kernel on a barrier that nothing completes (no copy is in flight), with a budget of budget_cycles clock cycles
 * (1 .. 10^8, LSGD_ERR_INVALID_ARG otherwise), synchronises the stream and stores 1 in *gave_up (HOST) if the
 * wait ran out.  The status word keeps the bit until lsgd_check_device reads it; the context stays usable.  */
LSGD_API lsgd_status lsgd_selftest_wait_timeout(lsgd_handle h, int32_t which, int64_t budget_cycles, int32_t* gave_up);
/* The "center variable" the paper reports at test time for LSGD (Section 4.1): the average of the
 * parameters of all workers, center[k] = (1/P) sum_i x[i][k], summed in worker order in fp64 and rounded
 * once.  center: DEVICE float[ld] (columns d..ld-1 are written as the mean of the padding).  Enqueued
 * on the stream.                                                                                     */
LSGD_API lsgd_status lsgd_center(lsgd_handle h, float* center);
/* Call after overwriting x from outside (restoring a checkpoint, re-seeding a worker): re-derives
 * the library's internal copies of the parameters (the bf16 weight copy of the MLP objective) on the
 * stream.  The step counter and the leaders are kept.                                               */
LSGD_API lsgd_status lsgd_sync_parameters(lsgd_handle h);
/* CUDA-graph support.  grad / elect / step only enqueue kernels, so a sequence of whole steps can be
 * captured from the stream (after at least one un-captured step has run, so that one-time kernel
 * attributes are set) and replayed.  The pull / plain decision of every captured step is frozen into the
 * graph, so capture a whole number of communication periods starting at t % tau == 0 (and t % tau_G == 0
 * with LSGD_FLAG_ALGORITHM1) and replay from such a t.  The library counts steps on the host when they are
 * enqueued, not when a graph replays them: after each replay call lsgd_advance_step with the number of
 * steps the graph contains.                                                                        */
LSGD_API lsgd_status lsgd_advance_step(lsgd_handle h, int64_t n_steps);
/* Replaces eta (learning-rate schedules are the caller's, Section 4).                            */
LSGD_API lsgd_status lsgd_set_eta(lsgd_handle h, float eta);

LSGD_API const char* lsgd_status_string(lsgd_status s);

/* Allocation-free election loss of the diagonal quadratic.  (The paper has no counterpart: this is a
 * packaging variant of the loss evaluation, not a step of the method.)
 *
 * For callers that are not allowed to allocate device memory: code inside a framework-managed region
 * where every byte belongs to a memory pool, loops with a "no allocation after start-up" rule, or
 * guests in another component's CUDA context with a fixed memory budget.  lsgd_create is closed to
 * them because it calls cudaMalloc; this function calls no cudaMalloc / cudaFree and no allocating
 * library routine.
 *
 * Computes loss[i] = 1/2 sum_k a[k] (x[i][k] - b[k])^2 for i < P, bit-identical to what
 * lsgd_elect(h, NULL) stores for the QUADRATIC objective (same chunking, same fp64 summation order).
 *   x     DEVICE float[P*ld], 16-byte aligned; a, b DEVICE float[ld], 16-byte aligned
 *   loss  DEVICE float[P], written on `stream` (cudaStream_t; NULL = legacy default stream)
 *   d, ld as in lsgd_config (ld >= d, ld % 32 == 0).
 * Scratch: the per-chunk partial sums, P * ceil(d / 8192) doubles, live in a fixed 512 KiB array that
 * is part of the library image on every GPU that loads it (held until the process exits).  Capacity:
 * P * ceil(d / 8192) <= 65536, otherwise LSGD_ERR_TOO_LARGE and nothing is launched.
 * The first call on each device looks up the array's device address (with that device current); make
 * that first call before starting any stream capture.
 * All calls share the one array, which keeps the previous call's contents; every entry this call reads
 * is first overwritten by this call, so nothing needs clearing.  Two calls that overlap on the GPU
 * (different streams, or different host threads without ordering) race on the array: serialise them. */
LSGD_API lsgd_status lsgd_quadratic_loss_noalloc(const float* x, const float* a, const float* b, int32_t P,
                                                 int64_t d, int64_t ld, float* loss, void* stream);

/* MLP helpers (host only).  Offsets in floats of W_l and b_l inside a parameter row, and the row
 * length d.  n_layers = 3.                                                                        */
LSGD_API lsgd_status lsgd_mlp_param_offsets(const int32_t* dims /* HOST int32[4] */, int64_t* w_off /* [3] */,
                                   int64_t* b_off /* [3] */, int64_t* d_out);
LSGD_API uint64_t lsgd_mlp_scratch_bytes(const int32_t* dims, int32_t P, int32_t batch, int32_t n_heldout);
/* Sizes of the caller-owned scratch of the MATCOMP and PSD_COMPLETION descriptors (host only).             */
LSGD_API uint64_t lsgd_matcomp_scratch_bytes(int32_t P, int64_t ld);
LSGD_API uint64_t lsgd_psd_scratch_bytes(int32_t r, int32_t P, int64_t ld);

/* Batched bf16 x bf16 -> fp32-accumulate matrix product on the tensor cores: C[z] = A[z] . B[z] for
 * z < batch, C is M x N, contraction length K.  This is the product the MLP objective is built from
 * (its forward, back-propagation and weight-gradient products), exposed so that it can be checked
 * against a library matmul on its own.  All pointers DEVICE.
 *   a_mn_major = 0: A is stored [M][lda] (K contiguous);  1: A is stored [K][lda] (M contiguous).
 *   b_mn_major = 0: B is stored [N][ldb] (K contiguous);  1: B is stored [K][ldb] (N contiguous).
 *   lda, ldb, ldc: row pitch in elements; lda, ldb and the pitch of a bf16 C / mask multiples of 8, the
 *   pitch of an fp32 C a multiple of 4.  stride_*: elements between batch entries (stride_a / stride_b
 *   = 0 shares the operand across the batch; multiples of 8 otherwise).  a, b, c, mask 16-byte aligned.  epilogue: 0 C fp32 = acc; 1 C bf16 = relu(acc + bias[z][n]);
 *   2 C bf16 = (mask[z][m][n] > 0 ? acc : 0), mask bf16; 3 C bf16 = acc.
 * Enqueues on `stream` and returns.  LSGD_ERR_ALIGNMENT if an operand breaks the rules above.      */
typedef struct {
  const void* a;
  const void* b;
  void* c;
  int32_t M, N, K, batch;
  int32_t a_mn_major, b_mn_major;
  int64_t lda, ldb, ldc;
  int64_t stride_a, stride_b, stride_c;
  int32_t epilogue;
  const float* bias;
  int64_t stride_bias;
  const void* mask;
  int64_t ld_mask, stride_mask;
} lsgd_bgemm_desc;
LSGD_API lsgd_status lsgd_bgemm_bf16(const lsgd_bgemm_desc* desc, void* stream);
/* Synchronises the current device, then reads and clears the status word of lsgd_bgemm_bf16 on it (the
 * product's bounded waits record LSGD_DEVFLAG_WAIT_TIMEOUT there): LSGD_ERR_DEVICE_FLAG if it was set.  */
LSGD_API lsgd_status lsgd_bgemm_check_device(uint32_t* flag_out /* HOST, may be NULL */);

#ifdef __cplusplus
}
#endif
#endif /* LSGD_H_ */
