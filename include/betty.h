/* betty.h - C ABI of the B200 hypergradient library.
 *
 * The library evaluates the hot path of gradient-based multilevel optimisation (MLO) as the
 * Betty paper states it (arXiv 2207.02849): a program of problems P_1..P_n, each with own
 * parameters theta_k, a cost C_k(theta_k, U_k, L_k; D_k) and constraining parameters from upper
 * (U_k, non-optimal) and lower (L_k, optimal) problems (Sec. 2, Def. 1).  The gradient of an
 * upper cost is the direct gradient plus best-response Jacobians times direct gradients (Eq. 1),
 * a best-response Jacobian along a path being a product of per-edge Jacobians that is evaluated
 * right to left as repeated (Jacobian x vector) products (Eq. 2 and Sec. 3.2).  The per-edge
 * product  (d x* / d c)^T v = -M^T H^{-1} v  (x own parameters of the lower problem, c the
 * constraining block, H = d2C/dx2, M = d(dC/dx)/dc) is approximated by implicit differentiation
 * with a Neumann series, with conjugate gradient, or with a finite difference (Sec. 3.2), at
 * lower parameters obtained by a few unrolled gradient steps (Sec. 3.2).
 *
 * Conventions
 *  - Everything crossing this boundary is plain C: PODs, pointers, sizes.  Level descriptors and
 *    the `widths`/`constraints`/`path`/`per_edge` arrays are HOST memory and are only read during
 *    the call.  Every other pointer (params, X, y, aux, vectors, ws) is DEVICE memory on the
 *    current CUDA device, owned by the caller; the library never allocates, frees or keeps a
 *    pointer after a call returns.
 *  - Parameter blocks and every flat vector argument (u, q, v_in, out) are fp32.  An MLP block is
 *    [W_1, b_1, W_2, b_2, ...] with W_l of shape [widths[l+1], widths[l]] row-major and b_l of
 *    length widths[l+1].  A weight-net block (1-100-1 net of the data-reweighting experiment) is
 *    [a1(100), b1(100), a2(100), b2(1)].  fp32 vectors must be 16-byte aligned, X 16-byte aligned.
 *  - `ws` is scratch of at least betty_workspace_size() bytes, 256-byte aligned.  Its first 256
 *    bytes hold a device status block written by kernels (see betty_poll_status); contents do not
 *    need to be preserved between calls, but calls sharing one `ws` must not overlap in time.
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *    synchronising.  The MLP families also use one stream of the library's own (made once per host
 *    thread and device, never destroyed, no device memory): independent pieces of a call (the
 *    weight-gradient products and bias sums beside a reverse sweep's chain, one of the two
 *    perturbed passes of a finite difference, a lower level's base pass beside the upper level's
 *    gradients) run there, forked from and joined back into `stream` with events inside the call,
 *    so the caller sees ordinary stream order and a stream capture of a call records the same
 *    dependencies.  The first MLP-family call of a
 *    thread should not be made under a capture (it then runs without the second stream).  Argument errors are returned immediately and nothing is enqueued.
 *    Conditions found on the device (non-finite values, CG breakdown, an expired bounded wait)
 *    are recorded in the status block and reported by betty_poll_status.
 *  - One GPU (compute capability 10.0).  There is no CPU fallback.
 */
#ifndef BETTY_H_
#define BETTY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BETTY_OK = 0,
  BETTY_ERR_INVALID_ARG = 1,  /* null pointer, negative size, unknown enum, bad path */
  BETTY_ERR_SHAPE = 2,        /* sizes of participants do not fit the cost family */
  BETTY_ERR_DTYPE = 3,
  BETTY_ERR_ALIGNMENT = 4,
  BETTY_ERR_WORKSPACE = 5,    /* ws too small or misaligned */
  BETTY_ERR_CUDA = 6,         /* a CUDA runtime call failed (launch error, wrong device) */
  BETTY_ERR_NONFINITE = 7,    /* device: a reduction met Inf/NaN */
  BETTY_ERR_BREAKDOWN = 8,    /* device: CG met a direction with p^T H p <= 0 */
  BETTY_ERR_TIMEOUT = 9,      /* device: a bounded wait (mbarrier) expired */
  BETTY_ERR_UNSUPPORTED = 10, /* combination not implemented */
  BETTY_ERR_CAPACITY = 11     /* size exceeds the fixed built-in scratch of an allocation-free call */
} betty_status;

/* Cost families C_k.  "own" = the level's own parameter block. */
typedef enum {
  /* App. D.1 lower problem: own w[d]; constraint VECTOR lambda[d].
   * C = (1/n) sum_i softplus(-y_i x_i.w) + 1/2 sum_j lambda_j w_j^2.  X fp32 [n,d], y fp32 +-1. */
  BETTY_LOSS_LOGREG_WD = 0,
  /* App. D.1 upper problem: C = (1/n) sum_i softplus(-y_i x_i.w), w = the first VECTOR constraint. */
  BETTY_LOSS_LOGREG = 1,
  /* C = 1/2 |X w - y|^2 + 1/2 sum_j lambda_j w_j^2 (closed-form best response; used to test
   * solvers, and the indefinite case of CG).  own w[d]; constraint VECTOR lambda[d]; y fp32 [n]. */
  BETTY_LOSS_QUADRATIC_WD = 2,
  /* C = 1/2 |X w - y|^2 of the first VECTOR constraint w. */
  BETTY_LOSS_QUADRATIC = 3,
  /* App. A "Classifier" (data reweighting): own MLP; optional constraints WEIGHTNET theta and
   * LOGWD lambda.  C = (1/B) sum_i r_i l_i + 1/2 sum_l exp(lambda_l) |W_l|_F^2, l_i = softmax
   * cross-entropy of sample i, r_i = sigmoid(weightnet(l_i; theta)) with l_i detached: derivatives
   * w.r.t. the MLP treat r_i as constants, derivatives w.r.t. theta treat l_i as data.
   * r_i = 1 without a WEIGHTNET constraint; no decay term without a LOGWD constraint.
   * With a CORRECTNET constraint alpha (the extended bilevel program of Sec. 5.1) l_i is the cross-entropy against
   * the corrected soft label  new_i = rho_i onehot(y_i) + (1 - rho_i) s_i,  s_i = softmax(A h_i + a0),
   * rho_i = sigmoid(a2 . relu(A1 h_i + b1) + b2),  h_i the last hidden activation (width H >= 1 hidden layer needed);
   * the label is not detached from the classifier.  Gradients (all participants), lower steps and the finite-
   * difference hypergradient are offered; Hessian-vector and mixed products return BETTY_ERR_UNSUPPORTED (the paper
   * pairs this program with AID-FD).  Limits: at most 1024 classes, H <= 8192, no loss scaling.
   * X bf16 [n,d], y int32 class ids. */
  BETTY_LOSS_MLP_CE_REWEIGHT = 4,
  /* App. A "Reweight": C = (1/B) sum_i l_i of the first MLP constraint on this level's batch. */
  BETTY_LOSS_MLP_CE = 5,
  /* C = (1/B) sum_j (sigmoid(weightnet(l_j(w); theta)) - aux_j)^2 + mu/2 |theta|^2 with theta the
   * WEIGHTNET participant and w the MLP participant (own block or constraints); l_j is NOT
   * detached.  aux fp32 [n] in {0,1} (1 = label is clean).  X bf16 [n,d], y int32. */
  BETTY_LOSS_WEIGHTNET_DETECT = 6,
  /* App. A "Correct" (Sec. 5.1, correcting and reweighting corrupted labels): own block CORRECTNET alpha, constraint
   * MLP w.  C = (1/B) sum_j l_j(w) + (1/B) sum_j CE(softmax(A h_j + a0), y_j) on this level's (clean) batch, h_j the
   * classifier's last hidden activation: the classifier's cross-entropy plus that of the correction net's own soft
   * labels.  X in the classifier's operand type [n,d], y int32. */
  BETTY_LOSS_MLP_CE_CORRECT = 7
} betty_loss;

typedef enum {
  BETTY_PARAM_VECTOR = 0,    /* plain vector (logistic/quadratic w, per-feature weight decay) */
  BETTY_PARAM_MLP = 1,       /* classifier weights, layout above */
  BETTY_PARAM_WEIGHTNET = 2, /* 301 parameters of the 1-100-1 weight net */
  BETTY_PARAM_LOGWD = 3,     /* per-layer log weight decay, one per MLP layer */
  BETTY_PARAM_CORRECTNET = 4 /* label-correction net on a classifier with last hidden width H and C classes:
                              * [A (C x H), a0 (C), A1 (100 x H), b1 (100), a2 (100), b2], C*H + C + 100*H + 201 floats */
} betty_param_kind;

typedef enum { BETTY_NEUMANN = 0, BETTY_CG = 1, BETTY_FD = 2 } betty_method;
typedef enum { BETTY_ACT_RELU = 0, BETTY_ACT_GELU = 1 } betty_activation; /* GELU: erf form */
typedef enum { BETTY_F32 = 0, BETTY_BF16 = 1, BETTY_I32 = 2, BETTY_F16 = 3 } betty_dtype;

/* How a problem's gradient step is taken (the paper lets each problem bring its own optimiser: SGD with
 * momentum and weight decay for the classifiers, Adam for the weight net, App. C).
 *  GD      : x -= lr * g
 *  MOMENTUM: g' = g + weight_decay * x;  buf = momentum * buf + g';  x -= lr * buf      (buf starts at 0)
 *  ADAM    : g' = g + weight_decay * x;  m = b1 m + (1-b1) g';  v = b2 v + (1-b2) g'^2;  t += 1;
 *            x -= lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)
 * State lives in opt_state (device fp32, caller-owned, zero-initialised by the caller): MOMENTUM needs
 * n_params floats, ADAM 2 * n_params + 1 (the last one counts steps). */
typedef enum { BETTY_OPT_GD = 0, BETTY_OPT_MOMENTUM = 1, BETTY_OPT_ADAM = 2 } betty_optimizer;

/* Step size as a function of the number t of steps the problem has already taken (App. C trains the
 * classifiers with a step size "decayed by a factor of 10" at two given iterations, or "decayed with the
 * cosine annealing schedule" to a minimum by the end of training).
 *  CONSTANT : lr
 *  MULTISTEP: lr * lr_gamma^(number of lr_milestones[i] > 0 with lr_milestones[i] <= t)
 *  COSINE   : lr_min + (lr - lr_min) * (1 + cos(pi * min(t, lr_t_max) / lr_t_max)) / 2
 * t = lr_step0 + the steps taken so far inside the call (betty_lower_step, betty_hypergrad_itd,
 * betty_engine_run); the caller advances lr_step0 between calls.  The value is worked out on the host. */
typedef enum { BETTY_LR_CONSTANT = 0, BETTY_LR_MULTISTEP = 1, BETTY_LR_COSINE = 2 } betty_lr_schedule;

/* Approximation of one best-response Jacobian (Sec. 3.2).
 *  NEUMANN: q = alpha * sum_{j=0..K} (I - alpha H)^j v   (K Hessian-vector products)
 *  CG     : K iterations of conjugate gradient on H q = v from q = 0; stops early once
 *           |r| <= tol*|v|; p^T H p <= 0 stops it and records BETTY_ERR_BREAKDOWN
 *  FD     : eps = eps0/|v|_2;  -alpha * [dC/dc(x + eps v) - dC/dc(x - eps v)] / (2 eps) */
typedef struct {
  int32_t method; /* betty_method */
  int32_t K;
  float alpha;
  float eps0;
  float tol;
} betty_method_cfg;

/* Data-parallel evaluation (Sec. 4 lists data-parallel training among the systems features; App. E reports
 * its memory on 2 GPUs).  The rows of a problem's batch are partitioned over the ranks of a job, one GPU
 * and one process per rank; parameters and all solver state are replicated.  Every cost here is a mean
 * over the rows plus terms that do not depend on the data, so with row_weight_r = n_r / n (they sum to 1)
 *     C = sum_r row_weight_r * C_r ,   C_r = the same cost evaluated on rank r's rows,
 * and the same holds for every derivative of C.  A level whose `comm` is set is one rank's share of its
 * problem: whenever the library has formed a gradient, a Hessian-vector product, a mixed product or the
 * finite difference of gradients of that level's cost on the local rows, it multiplies the vector by
 * row_weight and calls `allreduce`, which must replace the count floats at buf (DEVICE memory on the
 * current device) by their sum over all ranks, ordered after the work already enqueued on `stream` and
 * before work enqueued later (enqueue it on that stream, or synchronise around it), and return 0 on success
 * (anything else makes the library call return BETTY_ERR_CUDA).  All ranks then hold the same bits and take
 * the same solver steps.  The library never touches another GPU's memory: the exchange is entirely the
 * caller's (torch.distributed / NCCL in the Python binding).  With `comm` set the fused forms (update in
 * the reduction kernel or in a matrix product's epilogue, whole loops on chip) are replaced by their
 * unfused equivalents; betty_hypergrad_itd and betty_engine_run return BETTY_ERR_UNSUPPORTED. */
typedef int32_t (*betty_allreduce_fn)(void* user, float* buf, int64_t count, void* stream);
typedef struct {
  betty_allreduce_fn allreduce;
  void* user;          /* passed back to allreduce */
  float row_weight;    /* this rank's rows / all rows of the problem's batch */
} betty_comm;

/* One problem P_k. */
typedef struct betty_level {
  int32_t loss;         /* betty_loss */
  int32_t param_kind;   /* betty_param_kind of the own block */
  float* params;        /* device fp32 [n_params]; updated in place by betty_lower_step */
  int64_t n_params;
  const void* X;        /* device, row-major [n, d]; dtype x_dtype */
  int32_t x_dtype;      /* betty_dtype */
  int64_t n, d;
  const void* y;        /* device [n]: fp32 (logistic +-1, quadratic targets) or int32 class ids */
  const float* aux;     /* device [n] fp32, WEIGHTNET_DETECT only, else NULL */
  int32_t n_layers;     /* MLP own block: number of weight matrices; else 0 */
  const int64_t* widths;/* host [n_layers+1]: input width, hidden widths, classes */
  int32_t activation;   /* betty_activation (hidden layers) */
  float lr;             /* step size of betty_lower_step */
  float mu;             /* WEIGHTNET_DETECT ridge term */
  int32_t optimizer;    /* betty_optimizer used by betty_lower_step and betty_engine_run */
  float momentum;       /* MOMENTUM */
  float beta1, beta2, adam_eps; /* ADAM */
  float weight_decay;   /* MOMENTUM / ADAM: L2 term added to the gradient */
  float* opt_state;     /* device fp32 state, see betty_optimizer; NULL for GD */
  int32_t n_constraints;
  const struct betty_level* const* constraints; /* host array: U_k and L_k providers */
  int32_t lr_schedule;  /* betty_lr_schedule; the fields below are read only when it is not CONSTANT */
  int32_t lr_step0;     /* steps this problem had taken before this call */
  int32_t lr_t_max;     /* COSINE: length of the schedule in steps (> 0) */
  int32_t lr_milestones[4]; /* MULTISTEP: step counts at which the step size drops; unused entries 0 */
  float lr_gamma;       /* MULTISTEP: factor per milestone passed */
  float lr_min;         /* COSINE: step size reached at lr_t_max */
  int32_t grad_accum;   /* gradient accumulation (Sec. 4, systems support): a step of a problem without lower
                         * problems takes its batch as grad_accum equal micro-batches of n / grad_accum rows, one
                         * after the other, and averages their gradients before the optimiser step: the
                         * activations of one micro-batch are alive at a time.  0 or 1: off.  n must be a
                         * multiple of it (else BETTY_ERR_SHAPE).  Used by betty_lower_step and betty_engine_run. */
  const betty_comm* comm; /* host; NULL: the level holds its problem's whole batch (see betty_comm) */
  int32_t precision;    /* MLP own block: operand type of its matrix products (Sec. 4, mixed precision): BETTY_BF16
                         * (0 means the same) or BETTY_F16, fp32 accumulation and fp32 master parameters either way.
                         * Every cost the block takes part in must bring its batch X in that type (x_dtype). */
  float* loss_scale;    /* device fp32[4], caller-owned, or NULL: loss scaling for the steps betty_lower_step takes on
                         * a BETTY_F16 block (the paper's fp16 option; a half-precision backward pass loses small
                         * gradients to underflow unless the loss is scaled up).  [0] scale S > 0, [1] steps taken in a
                         * row without overflow, [2] growth interval G (0: the scale is static), [3] steps skipped so far.
                         * Each step: the top-layer deltas are multiplied by S, the gradient divided by S; if it holds a
                         * non-finite value (a 16-bit delta overflowed) the update is skipped, S is halved, [1] returns
                         * to 0 and [3] counts up; otherwise the optimiser step is taken, [1] counts up, and when it
                         * reaches G > 0 the scale doubles and [1] returns to 0.  All of it stays on the device.
                         * Other calls on the block run unscaled.  Not offered by betty_engine_run. */
} betty_level;

/* Scratch bytes sufficient for any call below on these levels (Sec. 2: the whole program). */
betty_status betty_workspace_size(const betty_level* const* levels, int32_t n_levels,
                                  size_t* bytes);

/* Zero the status block at the head of ws (enqueued on stream).  Call once before first use. */
betty_status betty_reset_status(void* ws, size_t ws_bytes, void* stream);

/* Synchronises `stream`, reads the status block and returns the first device-side condition
 * recorded since the last reset (BETTY_OK if none).  cg_iters (host, may be NULL) receives the
 * iteration count of the most recent CG solve. */
betty_status betty_poll_status(const void* ws, void* stream, int32_t* cg_iters);

/* Sec. 3.2 (approximating w* by unrolled gradient steps): n_steps times
 * params <- params - lr_t * dC/d(params) on the level's batch (lr_t: betty_lr_schedule).  MLP blocks: the gradient is taken
 * at the bf16-rounded copy of the fp32 master, re-derived every step. */
betty_status betty_lower_step(const betty_level* L, int32_t n_steps, void* ws, size_t ws_bytes,
                              void* stream);

/* Eq. 1 "direct gradient": out[wrt->n_params] = dC_L / d(params of wrt), wrt being L itself or
 * one of its constraints (zeros when C_L does not depend on it). */
betty_status betty_grad(const betty_level* L, const betty_level* wrt, float* out, void* ws,
                        size_t ws_bytes, void* stream);

/* Hessian-vector product of Sec. 3.2's implicit methods: Hu = (d2 C_L / d own^2) u. */
betty_status betty_hvp(const betty_level* L, const float* u, float* Hu, void* ws, size_t ws_bytes,
                       void* stream);

/* Mixed second-derivative product (the upper-to-lower / lower-to-upper factor of Eq. 2 before the
 * solve): out[wrt->n_params] = M^T q = d/dc <dC_L/d own, q>, c = params of constraint `wrt`. */
betty_status betty_mixed_vjp(const betty_level* L, const betty_level* wrt, const float* q,
                             float* out, void* ws, size_t ws_bytes, void* stream);

/* Eq. 1 for one lower problem:  out[wrt->n_params] = dC_upper/d(wrt) + (d lower^opt / d wrt)^T
 * dC_upper/d(lower), the Jacobian product by the named approximation.  `wrt` must be a
 * constraint of `lower` (normally `upper` itself). */
betty_status betty_hypergrad_neumann(const betty_level* lower, const betty_level* upper,
                                     const betty_level* wrt, int32_t K, float alpha, float* out,
                                     void* ws, size_t ws_bytes, void* stream);
betty_status betty_hypergrad_cg(const betty_level* lower, const betty_level* upper,
                                const betty_level* wrt, int32_t K, float tol, float* out,
                                void* ws, size_t ws_bytes, void* stream);
betty_status betty_hypergrad_fd(const betty_level* lower, const betty_level* upper,
                                const betty_level* wrt, float eps0, float alpha, float* out,
                                void* ws, size_t ws_bytes, void* stream);

/* Iterative differentiation with reverse-mode autodiff (ITD-RMAD, Sec. 3.2; the method of the original
 * Meta-Weight-Net in Sec. 5.1): takes n_steps unrolled lower steps from the current lower parameters
 * (they are left at the last iterate; the earlier ones are kept in ws, or on chip where a small
 * logistic / least-squares problem and its iterates fit there), then differentiates the
 * upper cost through those steps in reverse:  a = dC_upper/d(lower) at the last iterate; for
 * t = T-1..0: out -= lr * M_t^T a, a -= lr * H_t a.  out[wrt->n_params] also receives the direct
 * gradient.  ws must hold n_steps parameter vectors in addition to betty_workspace_size(). */
betty_status betty_hypergrad_itd(const betty_level* lower, const betty_level* upper,
                                 const betty_level* wrt, int32_t n_steps, float* out, void* ws,
                                 size_t ws_bytes, void* stream);

/* One path term of Eq. 2, evaluated right to left (Sec. 3.2).  path = [k, q(1), ..., q(m)] indexes
 * `levels`; q(1) is reached from k by the upper-to-lower edge, q(i+1) from q(i) by lower-to-upper
 * edges; per_edge[i] configures the edge into q(i+1) (per_edge[0]: the upper-to-lower edge).
 * Start vector: v_in[levels[q(m)]->n_params], or dC_k/d theta_{q(m)} when v_in is NULL.
 * out[levels[k]->n_params] receives the product (accumulate != 0: is added to out).  The direct
 * gradient of Eq. 2 is not added.  path_len = m + 1 >= 2. */
betty_status betty_chain_levels(const betty_level* const* levels, int32_t n_levels,
                                const int32_t* path, int32_t path_len,
                                const betty_method_cfg* per_edge, const float* v_in, float* out,
                                int32_t accumulate, void* ws, size_t ws_bytes, void* stream);

/* (No counterpart in the paper: a deployment aid.)  Hessian-vector product of the logistic
 * weight-decay cost, Hu = (1/n) X^T (sigmoid(z) sigmoid(-z) . X u) + lam . u with z = X w, for callers
 * that have no device memory to give as workspace and may not allocate any: a host whose GPU memory
 * is fully reserved by another allocator or pool, or code that must not risk the device-wide
 * synchronisation an allocation or a free can cause.  The scratch (per-CTA column sums and a status
 * word) is a fixed array inside the library image, about 4.6 MiB, held by every GPU that loads the
 * library until the process exits.  This call allocates and frees nothing.
 *   X fp32 [n, d] row-major, w / lam / u / Hu fp32 [d], all DEVICE pointers, 16-byte aligned;
 *   d a multiple of 4 and at most 4096: a larger d returns BETTY_ERR_CAPACITY, nothing is enqueued;
 *   status_dev: DEVICE int32 owned by the caller, or NULL; receives 0 or the betty_status of a
 *   condition met on the device (BETTY_ERR_TIMEOUT).
 * Same kernels, launch shape and summation order as betty_hvp on a LOGREG_WD level.  The first call
 * on each device looks up the array's device address (with that device current); make that first
 * call outside any stream capture.  All calls on one device share the array, which keeps the previous
 * call's contents (the call clears the part that must start at zero): two calls whose kernels can
 * overlap on the GPU, e.g. on different streams, race on it, so serialise them. */
betty_status betty_hvp_logreg_static(const float* X, int64_t n, int64_t d, const float* w,
                                     const float* lam, const float* u, float* Hu,
                                     int32_t* status_dev, void* stream);

/* Building block of the MLP families' forward, backward and R-operator passes (the matrix products
 * behind the Hessian-vector products of Sec. 3.2), exposed so that it can be checked on its own:
 *   C[M,N] (fp32, leading dimension ldc) = sum_{i < n_pairs} alpha_i * op(A_i) op(B_i) + beta * C
 * with bf16 operands and fp32 accumulation, n_pairs in {1, 2}.  Logical A is [M,K]: stored row-major
 * [M,K] (a_transposed = 0) or [K,M] (a_transposed = 1); logical B is [K,N]: stored [K,N]
 * (b_transposed = 0) or [N,K] (b_transposed = 1); lda/ldb are leading dimensions in elements.
 * path: 0 = library's choice, 1 = CUDA-core kernel, 2 = tensor-core (tcgen05) kernel, 3 = its two-SM
 * (cta_group::2) form, both holding C transposed in tensor memory so that the epilogue's accesses
 * coalesce; 4 and 5 = the same two kernels with one accumulator row per thread; the tensor-core kernels need 16-byte aligned operands, lda/ldb multiples of 8 and alpha = +-1 (else BETTY_ERR_UNSUPPORTED).
 * All pointers are device pointers; `pairs` is host memory. */
typedef struct {
  const void* A; int64_t lda; int32_t a_transposed;
  const void* B; int64_t ldb; int32_t b_transposed;
  int32_t K;
  float alpha;
} betty_gemm_operands;
betty_status betty_gemm_bf16(int32_t M, int32_t N, int32_t n_pairs, const betty_gemm_operands* pairs,
                             float* C, int64_t ldc, float beta, int32_t path, void* ws, size_t ws_bytes,
                             void* stream);

/* The dataflow graph of Sec. 3.1: directed edges between problem indices.  An upper-to-lower edge
 * (from > to in the paper's ordering) says that theta_from constrains problem `to`; a lower-to-upper
 * edge says that theta*_from constrains problem `to`. */
typedef struct { int32_t from, to; } betty_edge;

/* Sec. 3.1 path finding (the paper's modified depth-first search): every valid path from theta_k to
 * the optimal parameters of a target problem starts with one upper-to-lower edge and continues over
 * lower-to-upper edges only.  Host-only; touches no device.  `targets` (host) lists L_k.  Paths are
 * written to `paths` (host, `capacity` ints) as records [len, k, q(1), ..., q(len-1)] in discovery
 * order, ready for betty_chain_levels; n_paths / n_ints (nullable) receive the totals even when the
 * buffer is too small (then BETTY_ERR_WORKSPACE is returned; paths == NULL only counts). */
betty_status betty_find_paths(int32_t n_levels, const betty_edge* u2l, int32_t n_u2l, const betty_edge* l2u,
                              int32_t n_l2u, int32_t k, const int32_t* targets, int32_t n_targets,
                              int32_t* paths, int32_t capacity, int32_t* n_paths, int32_t* n_ints);

/* Eq. 2 for problem k over the whole dataflow graph: out[levels[k]->n_params] = direct gradient + the
 * sum over all lower problems l in L_k (sources of lower-to-upper edges into k) and all valid paths from
 * theta_k to theta*_l of the path's Jacobian chain times dC_k/d theta*_l.  Paths that share a suffix are
 * merged at their common node (exact by linearity), so each edge's Jacobian product is taken once.
 * per_level[q] configures every best-response Jacobian of problem q.  Edge arrays are host memory. */
betty_status betty_hypergrad_graph(const betty_level* const* levels, int32_t n_levels, const betty_edge* u2l,
                                   int32_t n_u2l, const betty_edge* l2u, int32_t n_l2u, int32_t k,
                                   const betty_method_cfg* per_level, float* out, void* ws, size_t ws_bytes,
                                   void* stream);

/* Execution of the whole program (Sec. 3.3).  n_iterations times, every lowermost problem (one that no
 * lower-to-upper edge enters) takes one gradient step; a problem that has taken unroll_steps[j] steps
 * since its last call-out calls every problem it constrains through a lower-to-upper edge, and a called
 * problem takes its own step once all problems of its L set have called.  A step of problem j is
 * params_j -= lr_j * dC_j/d theta_j with the gradient of Eq. 2 (betty_hypergrad_graph); problems without
 * lower problems use the fused betty_lower_step.  step_log (host, nullable, log_capacity ints) receives the
 * indices of the problems in the order they stepped; n_steps_taken (nullable) the total count.
 * Everything is enqueued on `stream`; parameters are updated in place. */
betty_status betty_engine_run(const betty_level* const* levels, int32_t n_levels, const betty_edge* u2l, int32_t n_u2l,
                              const betty_edge* l2u, int32_t n_l2u, const betty_method_cfg* per_level,
                              const int32_t* unroll_steps, int32_t n_iterations, int32_t* step_log,
                              int32_t log_capacity, int32_t* n_steps_taken, void* ws, size_t ws_bytes, void* stream);

/* Self test of the failure path: enqueues a one-warp kernel whose bounded mbarrier wait can never be
 * satisfied.  The wait gives up after its poll limit (a fraction of a second), the kernel records
 * BETTY_ERR_TIMEOUT in the status block of ws and returns; the context stays usable.  betty_poll_status
 * then reports the condition.  Every wait in the library's kernels uses the same bounded form. */
betty_status betty_selftest_wait_timeout(void* ws, size_t ws_bytes, void* stream);

/* Self test of a piece of host logic; touches no device.  Kernels that need more than the default
 * dynamic shared memory have their limit raised once per kernel and per device ordinal (the setting
 * belongs to a device, and one process may drive several).  This call drives one private instance of
 * that bookkeeping: reset != 0 forgets everything first; the return value is 1 when a launch that
 * needs `bytes` on device ordinal `device` would have to set the limit, 0 when an earlier call already
 * covered it on that device.  Ordinals outside the table (negative or >= 64) always return 1. */
int32_t betty_selftest_smem_limit(int32_t reset, int32_t device, uint64_t bytes);

const char* betty_status_string(betty_status s);

/* Number of CUDA kernels this library has launched in the calling process since it was loaded
 * (host-side counter; used by benchmarks to report their launch count). */
uint64_t betty_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* BETTY_H_ */
