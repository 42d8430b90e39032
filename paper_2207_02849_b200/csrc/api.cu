// C ABI entry points: argument validation, dispatch on the cost family, and the host-side
// drivers of Sec. 3.2's approximations (Neumann series, conjugate gradient, finite difference),
// Eq. 1 and the right-to-left product along one path of Eq. 2.  Drivers only enqueue kernels;
// every scalar of the iterations stays on the device.
#include "ops.cuh"

namespace betty {

std::atomic<unsigned long long> g_kernel_launches{0};

// ------------------------------------------------------------------ MLP families: one per 16-bit operand type
// The classifier block that takes part in a cost decides which build of the family serves the call.
static inline bool mlp_f16(const betty_level* L) {
  const betty_level* M = find_participant(L, BETTY_PARAM_MLP);
  return M && M->precision == BETTY_F16;
}
#define BETTY_MLP_DISPATCH(L, call) (mlp_f16(L) ? fam_f16::call : fam_bf16::call)
static betty_status mlpfam_validate(const betty_level* L) { return BETTY_MLP_DISPATCH(L, mlpfam_validate(L)); }
static size_t mlpfam_workspace(const betty_level* L) { return BETTY_MLP_DISPATCH(L, mlpfam_workspace(L)); }
static betty_status mlpfam_grad(Ctx& c, const betty_level* L, const betty_level* wrt, float* out) {
  return BETTY_MLP_DISPATCH(L, mlpfam_grad(c, L, wrt, out));
}
static betty_status mlpfam_share_weights(Ctx& c, const betty_level* M) {
  return (M && M->precision == BETTY_F16) ? fam_f16::mlpfam_share_weights(c, M) : fam_bf16::mlpfam_share_weights(c, M);
}
static void mlpfam_unshare_weights(Ctx& c) { c.shared.master = nullptr; }
static betty_status mlpfam_hvp_begin(Ctx& c, const betty_level* L, MlpHvpCache** cache) {
  return BETTY_MLP_DISPATCH(L, mlpfam_hvp_begin(c, L, cache));
}
static betty_status mlpfam_hvp_keep_direction(Ctx& c, const betty_level* L, MlpHvpCache* cache) {
  return BETTY_MLP_DISPATCH(L, mlpfam_hvp_keep_direction(c, cache));
}
static betty_status mlpfam_hvp(Ctx& c, const betty_level* L, MlpHvpCache* cache, const float* u, float* Hu) {
  return BETTY_MLP_DISPATCH(L, mlpfam_hvp(c, L, cache, u, Hu));
}
static betty_status mlpfam_hvp_series(Ctx& c, const betty_level* L, MlpHvpCache* cache, const float* sv, const float* v,
                                      float alpha, float* s_out) {
  return BETTY_MLP_DISPATCH(L, mlpfam_hvp_series(c, L, cache, sv, v, alpha, s_out));
}
static betty_status mlpfam_mixed(Ctx& c, const betty_level* L, MlpHvpCache* cache, const betty_level* wrt, const float* q,
                                 float* out) {
  return BETTY_MLP_DISPATCH(L, mlpfam_mixed(c, L, cache, wrt, q, out));
}
static betty_status mlpfam_lower_step(Ctx& c, const betty_level* L, int n_steps, int first_step = 0) {
  return BETTY_MLP_DISPATCH(L, mlpfam_lower_step(c, L, n_steps, first_step));
}
static betty_status mlpfam_fd(Ctx& c, const betty_level* L, const betty_level* wrt, const float* v, const float* vnorm2,
                              float eps0, float alpha, float* out, bool accumulate, MlpHvpCache* pre) {
  return BETTY_MLP_DISPATCH(L, mlpfam_fd(c, L, wrt, v, vnorm2, eps0, alpha, out, accumulate, pre));
}
static betty_status mlpfam_fd_begin(Ctx& c, const betty_level* L, MlpHvpCache** cache) {
  return BETTY_MLP_DISPATCH(L, mlpfam_fd_begin(c, L, cache));
}

std::mutex& smem_limit_mutex() {
  static std::mutex m;
  return m;
}

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return -1; }
  return (dev >= 0 && dev < MAX_DEVICES) ? dev : -1;
}
int current_sm_count() {
  static std::atomic<int> cached[MAX_DEVICES];          // 0: not asked yet
  const int dev = current_device();
  if (dev < 0) return DEFAULT_SM_COUNT;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return DEFAULT_SM_COUNT;
  }
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

SideLane* side_lane(cudaStream_t main) {
  static thread_local SideLane lanes[MAX_DEVICES];
  static thread_local unsigned char state[MAX_DEVICES];   // 0: not tried, 1: made, 2: could not be made
  const int dev = current_device();
  if (dev < 0) return nullptr;
  if (state[dev] == 1) return &lanes[dev];
  if (state[dev] == 2) return nullptr;
  // nothing is created while the caller's stream is being captured: that call runs in program order
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(main, &cap) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
  if (cap != cudaStreamCaptureStatusNone) return nullptr;
  SideLane& ln = lanes[dev];
  bool ok = cudaStreamCreateWithFlags(&ln.stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&ln.fork, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&ln.join, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) { (void)cudaGetLastError(); state[dev] = 2; return nullptr; }
  state[dev] = 1;
  return &ln;
}

// ------------------------------------------------------------------ small kernels
// out (+)= scale * x
__global__ void k_scale_into(float* out, const float* x, float scale, int accumulate, int64_t n) {
  pdl_enter();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = (accumulate ? out[i] : 0.f) + scale * x[i];
}
// weight-decay constraint: dC/d(lambda) = 1/2 w^2, so the central difference is evaluated as written,
// in double to keep the cancellation exact:  out (+)= -alpha*[(w+ev)^2 - (w-ev)^2]/(4e)
__global__ void k_fd_weight_decay(float* out, const float* w, const float* v, const float* vnorm2, float eps0,
                                  float alpha, int accumulate, int64_t n) {
  pdl_enter();
  const double nv = sqrt((double)*vnorm2);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    float base = accumulate ? out[i] : 0.f;
    if (nv > 0.0) {
      const double eps = (double)eps0 / nv;
      const double wp = (double)w[i] + eps * (double)v[i], wm = (double)w[i] - eps * (double)v[i];
      base += (float)(-(double)alpha * (0.5 * wp * wp - 0.5 * wm * wm) / (2.0 * eps));
    }
    out[i] = base;
  }
}
// optimiser steps (see betty_optimizer); the step counter of Adam is the float behind the two moments
// `skip` (nullable, device): a step whose gradient overflowed under loss scaling is not taken
__global__ void k_opt_momentum(float* x, const float* g, float* buf, float lr, float mom, float wd, int64_t n, const int* skip) {
  pdl_enter();
  if (skip && *skip) return;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float gg = g[i] + wd * x[i];
    const float b = mom * buf[i] + gg;
    buf[i] = b;
    x[i] -= lr * b;
  }
}
__global__ void k_opt_adam(float* x, const float* g, float* m, float* v, const float* tcount, float lr, float b1, float b2,
                           float eps, float wd, int64_t n, const int* skip) {
  pdl_enter();
  if (skip && *skip) return;
  const float t = *tcount + 1.f;                       // this step's index; the counter is advanced afterwards
  const float c1 = 1.f - powf(b1, t), c2 = 1.f - powf(b2, t);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float gg = g[i] + wd * x[i];
    const float mi = b1 * m[i] + (1.f - b1) * gg;
    const float vi = b2 * v[i] + (1.f - b2) * gg * gg;
    m[i] = mi; v[i] = vi;
    x[i] -= lr * (mi / c1) / (sqrtf(vi / c2) + eps);
  }
}
__global__ void k_opt_tick(float* tcount, const int* skip) {
  pdl_enter();
  if (skip && *skip) return;
  *tcount += 1.f;
}
__global__ void k_opt_gd(float* x, const float* g, float lr, int64_t n, const int* skip) {
  pdl_enter();
  if (skip && *skip) return;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    x[i] -= lr * g[i];
}
// Loss scaling (betty_level.loss_scale = [S, good steps, growth interval, skipped steps]).
// g <- g / S; *flag |= any element non-finite (the flag is zeroed by the caller before the launch)
__global__ void k_unscale_check(float* g, int64_t n, const float* state, int* flag) {
  pdl_enter();
  const float inv = 1.f / state[0];
  int bad = 0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = g[i] * inv;
    g[i] = v;
    if (!isfinite(v)) bad = 1;
  }
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(flag, 1);
}
// overflow: halve the scale, count the skipped step; else count the good step and double the scale every G of them
__global__ void k_loss_scale_update(float* state, const int* flag) {
  pdl_enter();
  if (*flag) { state[0] *= 0.5f; state[1] = 0.f; state[3] += 1.f; return; }
  state[1] += 1.f;
  if (state[2] > 0.f && state[1] >= state[2]) { state[0] *= 2.f; state[1] = 0.f; }
}
static inline int ew_grid(int64_t n) {
  int64_t b = (n + 1023) / 1024;
  return (int)(b < 1 ? 1 : (b > 2368 ? 2368 : b));
}

// ------------------------------------------------------------------ vector families
static const betty_level* vec_w_level(const betty_level* L) {
  if (L->loss == BETTY_LOSS_LOGREG_WD || L->loss == BETTY_LOSS_QUADRATIC_WD) return L;
  return find_constraint(L, BETTY_PARAM_VECTOR);
}
static inline int vec_family(const betty_level* L) {
  return (L->loss == BETTY_LOSS_LOGREG_WD || L->loss == BETTY_LOSS_LOGREG) ? 0 : 1;
}
static inline bool vec_has_wd(const betty_level* L) {
  return L->loss == BETTY_LOSS_LOGREG_WD || L->loss == BETTY_LOSS_QUADRATIC_WD;
}

betty_status vecfam_validate(const betty_level* L) {
  if (L->n < 0 || L->d <= 0) return BETTY_ERR_SHAPE;
  if (L->x_dtype != BETTY_F32) return BETTY_ERR_DTYPE;
  if ((L->n > 0 && (!L->X || !L->y))) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(L->X)) return BETTY_ERR_ALIGNMENT;
  const betty_level* wl = vec_w_level(L);
  if (!wl || !wl->params) return BETTY_ERR_INVALID_ARG;
  if (wl->n_params != L->d) return BETTY_ERR_SHAPE;
  if (!aligned16(wl->params)) return BETTY_ERR_ALIGNMENT;
  if (vec_has_wd(L)) {
    if (L->param_kind != BETTY_PARAM_VECTOR) return BETTY_ERR_INVALID_ARG;
    const betty_level* lam = find_constraint(L, BETTY_PARAM_VECTOR);
    if (!lam || !lam->params) return BETTY_ERR_INVALID_ARG;
    if (lam->n_params != L->d) return BETTY_ERR_SHAPE;
  }
  return BETTY_OK;
}

betty_status vecfam_grad(Ctx& c, const betty_level* L, const betty_level* wrt, float* out) {
  const betty_level* wl = vec_w_level(L);
  if (wrt == wl) {
    const float* lam = vec_has_wd(L) ? find_constraint(L, BETTY_PARAM_VECTOR)->params : nullptr;
    return logreg_pass(c, vec_family(L), (const float*)L->X, (const float*)L->y, L->n, L->d, wl->params, nullptr, lam,
                       out, nullptr, 0.f);
  }
  if (vec_has_wd(L) && wrt == find_constraint(L, BETTY_PARAM_VECTOR))
    return vec_mul(c, out, 0.5f, L->params, L->params, L->d);
  return vec_zero(c, out, wrt->n_params);
}

betty_status vecfam_hvp(Ctx& c, const betty_level* L, const float* u, float* Hu, VecHvpCache* cache, const LrTail* tail) {
  if (!vec_has_wd(L)) return BETTY_ERR_UNSUPPORTED;
  return logreg_pass(c, vec_family(L), (const float*)L->X, (const float*)L->y, L->n, L->d, L->params, u,
                     find_constraint(L, BETTY_PARAM_VECTOR)->params, Hu, nullptr, 0.f, cache ? cache->curv : nullptr,
                     cache ? &cache->valid : nullptr, tail);
}

betty_status vecfam_mixed(Ctx& c, const betty_level* L, const betty_level* wrt, const float* q, float* out) {
  if (!vec_has_wd(L) || wrt != find_constraint(L, BETTY_PARAM_VECTOR)) return BETTY_ERR_INVALID_ARG;
  return vec_mul(c, out, 1.0f, L->params, q, L->d);
}

betty_status vecfam_lower_step(Ctx& c, const betty_level* L, int n_steps, int first_step) {
  if (!vec_has_wd(L)) return BETTY_ERR_UNSUPPORTED;
  const float* lam = find_constraint(L, BETTY_PARAM_VECTOR)->params;
  // all steps in one launch, data resident on chip (one step size for the whole launch)
  if (n_steps > 1 && L->lr_schedule == BETTY_LR_CONSTANT && logreg_small_eligible(L->n, 0, L->d))
    return logreg_small_lower_step(c, vec_family(L), (const float*)L->X, (const float*)L->y, L->n, L->d, L->params, lam,
                                   n_steps, L->lr);
  for (int s = 0; s < n_steps; ++s)
    BETTY_TRY(logreg_pass(c, vec_family(L), (const float*)L->X, (const float*)L->y, L->n, L->d, L->params, nullptr, lam,
                          nullptr, L->params, lr_at(L, first_step + s)));
  return BETTY_OK;
}

betty_status vecfam_fd(Ctx& c, const betty_level* L, const betty_level* wrt, const float* v, const float* vnorm2,
                       float eps0, float alpha, float* out, bool accumulate) {
  if (!vec_has_wd(L) || wrt != find_constraint(L, BETTY_PARAM_VECTOR)) return BETTY_ERR_INVALID_ARG;
  launch_pdl(k_fd_weight_decay, dim3(ew_grid(L->d)), dim3(256), 0, c.stream, out, L->params, v, vnorm2, eps0, alpha, accumulate ? 1 : 0, L->d);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// params of L <- one optimiser step along gradient g
static betty_status apply_optimizer(Ctx& c, const betty_level* L, const float* g, int step_in_call, const int* skip = nullptr) {
  const float lr = lr_at(L, step_in_call);
  const int64_t n = L->n_params;
  if (n <= 0) return BETTY_OK;
  const int grid = (int)((n + 1023) / 1024 < 1 ? 1 : ((n + 1023) / 1024 > 2368 ? 2368 : (n + 1023) / 1024));
  if (L->optimizer == BETTY_OPT_GD) {
    launch_pdl(k_opt_gd, dim3(grid), dim3(256), 0, c.stream, L->params, g, lr, n, skip);
  } else if (L->optimizer == BETTY_OPT_MOMENTUM) {
    launch_pdl(k_opt_momentum, dim3(grid), dim3(256), 0, c.stream, L->params, g, L->opt_state, lr, L->momentum, L->weight_decay, n, skip);
  } else {
    float* m = L->opt_state; float* v = m + n; float* t = v + n;
    launch_pdl(k_opt_adam, dim3(grid), dim3(256), 0, c.stream, L->params, g, m, v, t, lr, L->beta1, L->beta2, L->adam_eps, L->weight_decay, n, skip);
    BETTY_LAUNCH_CHECK();
    launch_pdl(k_opt_tick, dim3(1), dim3(1), 0, c.stream, t, skip);
  }
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// ------------------------------------------------------------------ dispatch
static betty_status validate_level(const betty_level* L) {
  if (!L) return BETTY_ERR_INVALID_ARG;
  if (L->n_constraints < 0 || (L->n_constraints > 0 && !L->constraints)) return BETTY_ERR_INVALID_ARG;
  for (int i = 0; i < L->n_constraints; ++i)
    if (!L->constraints[i]) return BETTY_ERR_INVALID_ARG;
  if (L->n_params < 0 || (L->n_params > 0 && !L->params)) return BETTY_ERR_INVALID_ARG;
  if (L->param_kind < BETTY_PARAM_VECTOR || L->param_kind > BETTY_PARAM_CORRECTNET) return BETTY_ERR_INVALID_ARG;
  if (L->optimizer < BETTY_OPT_GD || L->optimizer > BETTY_OPT_ADAM) return BETTY_ERR_INVALID_ARG;
  if (L->optimizer != BETTY_OPT_GD && !L->opt_state) return BETTY_ERR_INVALID_ARG;
  if (L->precision != 0 && L->precision != BETTY_BF16 && L->precision != BETTY_F16) return BETTY_ERR_DTYPE;
  if (L->precision == BETTY_F16 && L->param_kind != BETTY_PARAM_MLP) return BETTY_ERR_DTYPE;
  if (L->loss_scale && !(L->precision == BETTY_F16 && L->param_kind == BETTY_PARAM_MLP)) return BETTY_ERR_INVALID_ARG;
  if (is_vector_family(L->loss)) return vecfam_validate(L);
  if (is_mlp_family(L->loss)) return mlpfam_validate(L);
  return BETTY_ERR_INVALID_ARG;
}

static bool is_participant(const betty_level* L, const betty_level* wrt) {
  if (wrt == L) return true;
  for (int i = 0; i < L->n_constraints; ++i)
    if (L->constraints[i] == wrt) return true;
  return false;
}

static betty_status check_ws(void* ws, size_t ws_bytes) {
  if (!ws || ws_bytes < sizeof(StatusBlock)) return BETTY_ERR_WORKSPACE;
  if (((uintptr_t)ws) & 255u) return BETTY_ERR_WORKSPACE;
  return BETTY_OK;
}

// Data-parallel levels (betty_comm): a vector formed from this rank's rows becomes the whole batch's by
// weighting it with the rank's share of the rows and summing over the ranks.  The exchange is the caller's.
static betty_status dp_reduce(Ctx& c, const betty_level* L, float* vec, int64_t n) {
  if (!L->comm || n <= 0) return BETTY_OK;
  if (!L->comm->allreduce) return BETTY_ERR_INVALID_ARG;
  launch_pdl(k_scale_into, dim3(ew_grid(n)), dim3(256), 0, c.stream, vec, (const float*)vec, L->comm->row_weight, 0, n);
  BETTY_LAUNCH_CHECK();
  return L->comm->allreduce(L->comm->user, vec, n, (void*)c.stream) == 0 ? BETTY_OK : BETTY_ERR_CUDA;
}

static betty_status level_grad(Ctx& c, const betty_level* L, const betty_level* wrt, float* out) {
  BETTY_TRY(is_vector_family(L->loss) ? vecfam_grad(c, L, wrt, out) : mlpfam_grad(c, L, wrt, out));
  return dp_reduce(c, L, out, wrt->n_params);
}

// Gradient of a step of a problem without lower problems: dC_L/d(own), taken over the whole batch at once
// or, with gradient accumulation, as the average over L->grad_accum equal micro-batches processed one
// after the other (each micro-batch's activations are released before the next one starts).
static betty_status step_grad(Ctx& c, const betty_level* L, float* out) {
  const int A = L->grad_accum;
  if (A <= 1) return level_grad(c, L, L, out);
  if (L->n <= 0 || L->n % A != 0) return BETTY_ERR_SHAPE;
  const int64_t nb = L->n / A;
  const size_t xsz = L->x_dtype == BETTY_BF16 ? 2 : 4;
  const size_t mark = c.arena.mark();
  BETTY_ALLOC(ga, float, c, (size_t)L->n_params);
  for (int a = 0; a < A; ++a) {
    betty_level Ls = *L;                 // the same problem on rows a*nb .. (a+1)*nb - 1 of its batch
    Ls.n = nb;
    Ls.X = (const char*)L->X + (size_t)a * nb * L->d * xsz;
    Ls.y = (const char*)L->y + (size_t)a * nb * 4;          // labels are fp32 or int32
    if (L->aux) Ls.aux = L->aux + (size_t)a * nb;
    BETTY_TRY(level_grad(c, &Ls, &Ls, ga));
    BETTY_TRY(vec_axpby(c, out, 1.f / (float)A, ga, a > 0 ? 1.f : 0.f, a > 0 ? out : nullptr, L->n_params));
  }
  c.arena.release(mark);
  return BETTY_OK;
}

// (d x*/d c)^T v by the configured approximation; out (+)= result.
// pre: the base pass of an MLP-family level (mlpfam_hvp_begin) made by the caller, or null
static betty_status brj(Ctx& c, const betty_level* L, const betty_level* wrt, const float* v,
                        const betty_method_cfg& cfg, float* out, bool accumulate, MlpHvpCache* pre = nullptr) {
  if (!is_participant(L, wrt) || wrt == L) return BETTY_ERR_INVALID_ARG;
  const int64_t n = L->n_params, nc = wrt->n_params;
  const bool vecfam = is_vector_family(L->loss);
  const size_t mark = c.arena.mark();
  BETTY_ALLOC(partials, float, c, (size_t)vec_dot_partials(n));
  BETTY_TRY(vec_reduce_init(c, partials));
  betty_status rc = BETTY_OK;
  if (cfg.method == BETTY_FD) {
    BETTY_ALLOC(st, SolveState, c, 1);
    BETTY_TRY(vec_dot(c, v, v, n, &st->vnorm2, partials));
    float* dst = out;
    if (L->comm) {           // local rows first, then the sum over ranks, then into out
      dst = c.arena.alloc<float>((size_t)nc);
      if (!dst) return BETTY_ERR_WORKSPACE;
    }
    const bool acc_local = accumulate && !L->comm;
    rc = vecfam ? vecfam_fd(c, L, wrt, v, &st->vnorm2, cfg.eps0, cfg.alpha, dst, acc_local)
                : mlpfam_fd(c, L, wrt, v, &st->vnorm2, cfg.eps0, cfg.alpha, dst, acc_local, pre);
    if (rc == BETTY_OK && L->comm) {
      BETTY_TRY(dp_reduce(c, L, dst, nc));
      launch_pdl(k_scale_into, dim3(ew_grid(nc)), dim3(256), 0, c.stream, out, (const float*)dst, 1.f, accumulate ? 1 : 0, nc);
      BETTY_LAUNCH_CHECK();
    }
    c.arena.release(mark);
    return rc;
  }
  if (cfg.method != BETTY_NEUMANN && cfg.method != BETTY_CG) return BETTY_ERR_INVALID_ARG;
  if (cfg.K < 0) return BETTY_ERR_INVALID_ARG;
  MlpHvpCache* cache = pre;
  if (!vecfam && !cache) BETTY_TRY(mlpfam_hvp_begin(c, L, &cache));
  // logistic levels: the per-row curvature at the (fixed) lower parameters is shared by the solve's HVPs
  VecHvpCache vcache = {nullptr, false};
  if (vecfam && L->n > 0 && cfg.K > 1) vcache.curv = c.arena.alloc<float>((size_t)L->n);
  if (c.arena.overflow) { c.arena.overflow = false; vcache.curv = nullptr; }
  BETTY_ALLOC(q, float, c, (size_t)n);
  BETTY_ALLOC(h, float, c, (size_t)n);
  BETTY_ALLOC(m, float, c, (size_t)nc);
  float qscale = 1.f;
  if (cfg.method == BETTY_NEUMANN) {
    if (cfg.K == 0) BETTY_TRY(vec_copy(c, q, v, n));
    if (vecfam) {
      // term / sum recurrence; t_0 = s_0 = v are read straight from v in the first iteration: no copies
      BETTY_ALLOC(t, float, c, (size_t)n);
      // the update t <- t - alpha H t, s <- s + t rides in the pass's reduction kernel (one rank: nothing
      // comes between the product and its use)
      for (int k = 0; k < cfg.K; ++k) {
        const float* t_in = k == 0 ? v : t;
        const float* s_in = k == 0 ? v : q;
        if (L->comm) {
          BETTY_TRY(vecfam_hvp(c, L, t_in, h, &vcache));
          BETTY_TRY(dp_reduce(c, L, h, n));
          BETTY_TRY(neumann_update(c, t_in, s_in, h, cfg.alpha, t, q, n));
          continue;
        }
        LrTail tail = {};
        tail.kind = LR_TAIL_NEUMANN; tail.s_in = s_in; tail.t_out = t; tail.s_out = q; tail.alpha = cfg.alpha;
        BETTY_TRY(vecfam_hvp(c, L, t_in, h, &vcache, &tail));
      }
    } else if (L->comm) {
      // data-parallel MLP level: plain products, summed over ranks, then the term / sum recurrence
      BETTY_ALLOC(t, float, c, (size_t)n);
      for (int k = 0; k < cfg.K; ++k) {
        const float* t_in = k == 0 ? v : t;
        const float* s_in = k == 0 ? v : q;
        BETTY_TRY(mlpfam_hvp(c, L, cache, t_in, h));
        BETTY_TRY(dp_reduce(c, L, h, n));
        BETTY_TRY(neumann_update(c, t_in, s_in, h, cfg.alpha, t, q, n));
      }
    } else {
      // the same sum by Horner's rule, q <- v + (I - alpha H) q from q = v, fused into the HVP's epilogues
      if (cfg.K > 0 && L->param_kind == BETTY_PARAM_MLP) BETTY_TRY(mlpfam_hvp_keep_direction(c, L, cache));
      for (int k = 0; k < cfg.K; ++k) BETTY_TRY(mlpfam_hvp_series(c, L, cache, k == 0 ? v : q, v, cfg.alpha, q));
    }
    qscale = cfg.alpha;   // q holds the plain sum; alpha is applied with the sign below
  } else {
    BETTY_ALLOC(st, SolveState, c, 1);
    BETTY_ALLOC(r, float, c, (size_t)n);
    BETTY_ALLOC(p, float, c, (size_t)n);
    BETTY_TRY(cg_init(c, st, v, q, r, p, cfg.tol, n, partials));
    // vector families of moderate width: the whole iteration after H p rides in the pass's reduction kernel
    const bool fused = vecfam && !L->comm && n <= logreg_tail_max_d();
    LrTail tail = {};
    tail.kind = LR_TAIL_CG; tail.st = st; tail.q = q; tail.r = r; tail.p = p;
    tail.partials = (double*)partials; tail.counter = (unsigned*)((double*)partials + 592) + 2;
    for (int k = 0; k < cfg.K; ++k) {
      if (fused) {
        BETTY_TRY(vecfam_hvp(c, L, p, h, &vcache, &tail));
        continue;
      }
      BETTY_TRY(vecfam ? vecfam_hvp(c, L, p, h, &vcache) : mlpfam_hvp(c, L, cache, p, h));
      BETTY_TRY(dp_reduce(c, L, h, n));
      BETTY_TRY(cg_step(c, st, q, r, p, h, n, partials));
    }
  }
  BETTY_TRY(vecfam ? vecfam_mixed(c, L, wrt, q, m) : mlpfam_mixed(c, L, cache, wrt, q, m));
  BETTY_TRY(dp_reduce(c, L, m, nc));
  launch_pdl(k_scale_into, dim3(ew_grid(nc)), dim3(256), 0, c.stream, out, m, -qscale, accumulate ? 1 : 0, nc);
  BETTY_LAUNCH_CHECK();
  c.arena.release(mark);
  return BETTY_OK;
}

static betty_status hypergrad(const betty_level* lower, const betty_level* upper, const betty_level* wrt,
                              const betty_method_cfg& cfg, float* out, void* ws, size_t ws_bytes, void* stream) {
  BETTY_TRY(validate_level(lower));
  BETTY_TRY(validate_level(upper));
  if (!wrt || !out) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(out)) return BETTY_ERR_ALIGNMENT;
  BETTY_TRY(check_ws(ws, ws_bytes));
  if (!is_participant(upper, lower) || !is_participant(upper, wrt) || !is_participant(lower, wrt) || wrt == lower)
    return BETTY_ERR_INVALID_ARG;
  Ctx c(ws, ws_bytes, stream);
  // Small logistic / least-squares bilevel pair: the whole hypergradient in one launch.
  if (vec_has_wd(lower) && (upper->loss == BETTY_LOSS_LOGREG || upper->loss == BETTY_LOSS_QUADRATIC) &&
      find_constraint(upper, BETTY_PARAM_VECTOR) == lower && wrt == find_constraint(lower, BETTY_PARAM_VECTOR) &&
      cfg.K >= 0 && !lower->comm && !upper->comm && logreg_small_eligible(lower->n, upper->n, lower->d))
    return logreg_small_hypergrad(c, vec_family(lower), (const float*)lower->X, (const float*)lower->y, lower->n,
                                  vec_family(upper), (const float*)upper->X, (const float*)upper->y, upper->n, lower->d,
                                  lower->params, wrt->params, cfg, out);
  BETTY_ALLOC(v, float, c, (size_t)lower->n_params);
  // the upper gradient and the Jacobian product both evaluate costs at the lower level's present parameters
  BETTY_TRY(mlpfam_share_weights(c, lower));
  // An MLP-family lower level's base pass (forward and delta chain on its own batch, what every HVP of the solve
  // starts from) does not depend on the upper level's gradients: it runs on the side stream beside them.  Its
  // buffers sit below everything the gradients allocate and release, and stay until the call returns.
  // (For a finite difference the base pass is the forward pass alone; with respect to a weight decay it needs none.)
  const bool series = (cfg.method == BETTY_NEUMANN || cfg.method == BETTY_CG) && cfg.K >= 0;
  const bool fd = cfg.method == BETTY_FD && lower->loss == BETTY_LOSS_MLP_CE_REWEIGHT && wrt->param_kind != BETTY_PARAM_LOGWD;
  const bool early = (series || fd) && is_mlp_family(lower->loss) && !lower->comm && !upper->comm;
  MlpHvpCache* pre = nullptr;
  betty_status rc = BETTY_OK;
  {
    SideWork side(c, early);
    if (early) {
      side.begin();
      rc = fd ? mlpfam_fd_begin(c, lower, &pre) : mlpfam_hvp_begin(c, lower, &pre);
      side.end();
    }
    if (rc == BETTY_OK) rc = level_grad(c, upper, lower, v);     // dC_u / d theta_lower
    if (rc == BETTY_OK) rc = level_grad(c, upper, wrt, out);     // direct gradient
    const betty_status rj = side.join();
    if (rc == BETTY_OK) rc = rj;
  }
  if (rc == BETTY_OK) rc = brj(c, lower, wrt, v, cfg, out, true, pre);
  mlpfam_unshare_weights(c);
  return rc;
}

// ITD-RMAD: n_steps unrolled lower steps with the iterates kept in the workspace, then the reverse
// sweep  a <- a - lr H_t a,  out <- out - lr M_t^T a  from t = T-1 down to 0.
static betty_status hypergrad_itd(const betty_level* lower, const betty_level* upper, const betty_level* wrt,
                                  int n_steps, float* out, void* ws, size_t ws_bytes, void* stream) {
  BETTY_TRY(validate_level(lower));
  BETTY_TRY(validate_level(upper));
  if (!wrt || !out || n_steps < 0) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(out)) return BETTY_ERR_ALIGNMENT;
  if (lower->optimizer != BETTY_OPT_GD) return BETTY_ERR_UNSUPPORTED;   // the reverse sweep differentiates plain GD steps
  if (lower->comm || upper->comm) return BETTY_ERR_UNSUPPORTED;          // not offered for data-parallel levels
  BETTY_TRY(check_ws(ws, ws_bytes));
  if (!is_participant(upper, lower) || !is_participant(upper, wrt) || !is_participant(lower, wrt) || wrt == lower)
    return BETTY_ERR_INVALID_ARG;
  Ctx c(ws, ws_bytes, stream);
  // Small logistic / least-squares bilevel pair with one step size: unrolled steps and reverse sweep in one launch.
  if (n_steps > 0 && vec_has_wd(lower) && lower->lr_schedule == BETTY_LR_CONSTANT &&
      (upper->loss == BETTY_LOSS_LOGREG || upper->loss == BETTY_LOSS_QUADRATIC) &&
      find_constraint(upper, BETTY_PARAM_VECTOR) == lower && wrt == find_constraint(lower, BETTY_PARAM_VECTOR) &&
      logreg_small_eligible(lower->n, upper->n, lower->d, n_steps))
    return logreg_small_itd(c, vec_family(lower), (const float*)lower->X, (const float*)lower->y, lower->n, vec_family(upper),
                            (const float*)upper->X, (const float*)upper->y, upper->n, lower->d, lower->params, wrt->params,
                            n_steps, lower->lr, out);
  const int64_t n = lower->n_params, nc = wrt->n_params;
  const bool vecfam = is_vector_family(lower->loss);
  const size_t stride = ((size_t)n + 63) & ~size_t(63);
  BETTY_ALLOC(iter, float, c, stride * (size_t)(n_steps > 0 ? n_steps : 1));
  BETTY_ALLOC(a, float, c, (size_t)n);
  BETTY_ALLOC(h, float, c, (size_t)n);
  BETTY_ALLOC(m, float, c, (size_t)nc);
  for (int t = 0; t < n_steps; ++t) {
    BETTY_TRY(vec_copy(c, iter + stride * t, lower->params, n));
    BETTY_TRY(vecfam ? vecfam_lower_step(c, lower, 1, t) : mlpfam_lower_step(c, lower, 1, t));
  }
  BETTY_TRY(level_grad(c, upper, lower, a));
  BETTY_TRY(level_grad(c, upper, wrt, out));
  betty_level at = *lower;            // the lower problem seen at a stored iterate
  for (int t = n_steps - 1; t >= 0; --t) {
    at.params = iter + stride * t;
    const size_t mark = c.arena.mark();
    if (vecfam) {
      BETTY_TRY(vecfam_mixed(c, &at, wrt, a, m));
      BETTY_TRY(vecfam_hvp(c, &at, a, h));
    } else {
      MlpHvpCache* cache = nullptr;
      BETTY_TRY(mlpfam_hvp_begin(c, &at, &cache));
      BETTY_TRY(mlpfam_mixed(c, &at, cache, wrt, a, m));
      BETTY_TRY(mlpfam_hvp(c, &at, cache, a, h));
    }
    const float lr_t = lr_at(lower, t);     // the step size step t was taken with
    launch_pdl(k_scale_into, dim3(ew_grid(nc)), dim3(256), 0, c.stream, out, m, -lr_t, 1, nc);
    BETTY_LAUNCH_CHECK();
    BETTY_TRY(vec_axpby(c, a, 1.f, a, -lr_t, h, n));
    c.arena.release(mark);
  }
  return BETTY_OK;
}

// ------------------------------------------------------------------ dataflow graph (Sec. 3.1)
struct Graph {
  int n;
  const betty_edge* u2l; int n_u2l;
  const betty_edge* l2u; int n_l2u;
};
static bool graph_ok(const Graph& g) {
  if (g.n <= 0 || g.n_u2l < 0 || g.n_l2u < 0 || (g.n_u2l > 0 && !g.u2l) || (g.n_l2u > 0 && !g.l2u)) return false;
  for (int i = 0; i < g.n_u2l; ++i)
    if (g.u2l[i].from < 0 || g.u2l[i].from >= g.n || g.u2l[i].to < 0 || g.u2l[i].to >= g.n) return false;
  for (int i = 0; i < g.n_l2u; ++i)
    if (g.l2u[i].from < 0 || g.l2u[i].from >= g.n || g.l2u[i].to < 0 || g.l2u[i].to >= g.n) return false;
  return true;
}

// Depth-first enumeration: the first edge is upper-to-lower, every later edge lower-to-upper; a path is
// reported each time it stands on a target.  Records are [len, k, q(1), ..., q(m)], len = m + 1.
struct PathSink { int32_t* buf; int capacity; int used; int count; bool overflow; };
static void emit_path(PathSink& s, int k, const int* stack, int depth) {
  const int need = depth + 2;
  if (s.buf && s.used + need <= s.capacity) {
    s.buf[s.used] = depth + 1;
    s.buf[s.used + 1] = k;
    for (int i = 0; i < depth; ++i) s.buf[s.used + 2 + i] = stack[i];
  } else if (s.buf) {
    s.overflow = true;
  }
  s.used += need;
  s.count += 1;
}
static void dfs_paths(const Graph& g, int k, const bool* is_target, int* stack, bool* on_path, int depth, PathSink& s) {
  const int c = stack[depth - 1];
  if (is_target[c]) emit_path(s, k, stack, depth);
  for (int i = 0; i < g.n_l2u; ++i) {
    if (g.l2u[i].from != c) continue;
    const int nx = g.l2u[i].to;
    if (nx == k || on_path[nx]) continue;
    stack[depth] = nx; on_path[nx] = true;
    dfs_paths(g, k, is_target, stack, on_path, depth + 1, s);
    on_path[nx] = false;
  }
}

// Merged right-to-left evaluation of Eq. 2 over the graph: u_c = [c in L_k] dC_k/d theta_c +
// sum over lower-to-upper edges c -> n of (d theta_n* / d theta_c*)^T u_n, each edge's Jacobian product
// taken once (exact by linearity); out = direct gradient + sum over k -> c of (d theta_c*/d theta_k)^T u_c.
struct GraphEval {
  Ctx* c; const betty_level* const* levels; const Graph* g; int k; const bool* is_target;
  const betty_method_cfg* cfg; float** u; int* state;   // state: 0 new, 1 in progress, 2 done (u may stay null: no target above)
  float** tgrad;           // dC_k / d theta_c of the target nodes, where already evaluated (else null)
  MlpHvpCache** pre;       // base passes of MLP-family nodes, where already made (else null)
};
// The nodes an evaluation from k will visit below child c0 (each once), in the order their Jacobian products run.
static void collect_nodes(const Graph& g, int k, int cnode, bool* seen, int* order, int& n) {
  if (seen[cnode]) return;
  seen[cnode] = true;
  for (int i = 0; i < g.n_l2u; ++i)
    if (g.l2u[i].from == cnode && g.l2u[i].to != k) collect_nodes(g, k, g.l2u[i].to, seen, order, n);
  order[n++] = cnode;
}
static betty_status eval_node(GraphEval& e, int cnode) {
  if (e.state[cnode] == 2) return BETTY_OK;
  if (e.state[cnode] == 1) return BETTY_ERR_INVALID_ARG;      // cycle among lower-to-upper edges
  e.state[cnode] = 1;
  float* acc = nullptr;
  const int64_t nc = e.levels[cnode]->n_params;
  if (e.is_target[cnode]) {
    acc = e.tgrad[cnode];
    if (!acc) {
      acc = e.c->arena.alloc<float>((size_t)nc);
      if (!acc) return BETTY_ERR_WORKSPACE;
      BETTY_TRY(level_grad(*e.c, e.levels[e.k], e.levels[cnode], acc));
    }
  }
  for (int i = 0; i < e.g->n_l2u; ++i) {
    if (e.g->l2u[i].from != cnode) continue;
    const int nx = e.g->l2u[i].to;
    if (nx == e.k) continue;
    BETTY_TRY(eval_node(e, nx));
    if (!e.u[nx]) continue;                                   // nothing of C_k reaches through nx
    bool accumulate = true;
    if (!acc) {
      acc = e.c->arena.alloc<float>((size_t)nc);
      if (!acc) return BETTY_ERR_WORKSPACE;
      accumulate = false;
    }
    BETTY_TRY(brj(*e.c, e.levels[nx], e.levels[cnode], e.u[nx], e.cfg[nx], acc, accumulate, e.pre[nx]));
  }
  e.u[cnode] = acc;
  e.state[cnode] = 2;
  return BETTY_OK;
}

static betty_status graph_hypergrad(Ctx& c, const betty_level* const* levels, const Graph& g, int k,
                                    const betty_method_cfg* per_level, float* out) {
  bool is_target[256] = {false};
  float* u[256] = {nullptr};
  int state[256] = {0};
  for (int i = 0; i < g.n_l2u; ++i)
    if (g.l2u[i].to == k) is_target[g.l2u[i].from] = true;     // L_k: the lower problems that call k
  float* tgrad[256] = {nullptr};
  MlpHvpCache* pre[256] = {nullptr};
  GraphEval e = {&c, levels, &g, k, is_target, per_level, u, state, tgrad, pre};
  // No parameter changes during this evaluation, and every pass through a classifier evaluates it at the
  // same matrices: the first MLP level's matrices are rounded to operand precision once, not once per pass.
  const betty_level* mlp = nullptr;
  for (int i = 0; i < g.n && !mlp; ++i)
    if (levels[i] && levels[i]->param_kind == BETTY_PARAM_MLP) mlp = levels[i];
  const bool share = mlp && !c.shared.master;
  if (share) BETTY_TRY(mlpfam_share_weights(c, mlp));
  // What does not depend on anything computed here runs first, on two streams: the base passes of the MLP-family
  // nodes whose Jacobian products use a series solve (side stream; at most as many as the per-thread cache slots),
  // beside the gradients of C_k with respect to k's own parameters and to the target nodes (caller's stream).
  // Everything the side stream touches is allocated before the gradients' scratch and stays until the call returns.
  int order[256], n_ord = 0;
  {
    bool seen[256] = {false};
    for (int i = 0; i < g.n_u2l; ++i)
      if (g.u2l[i].from == k && g.u2l[i].to != k) collect_nodes(g, k, g.u2l[i].to, seen, order, n_ord);
  }
  bool plain = !levels[k]->comm;
  for (int i = 0; i < n_ord; ++i) plain = plain && !levels[order[i]]->comm;
  betty_status rc = BETTY_OK;
  {
    SideWork side(c, plain && n_ord > 0);
    if (plain) {
      side.begin();
      int made = 0;
      for (int i = 0; i < n_ord && made < MLP_HVP_CACHE_SLOTS; ++i) {
        const betty_level* L = levels[order[i]];
        const betty_method_cfg& m = per_level[order[i]];
        if (!is_mlp_family(L->loss) || (m.method != BETTY_NEUMANN && m.method != BETTY_CG) || m.K < 0) continue;
        // a pass that cannot be made here is left to the Jacobian product, which reports why
        if (mlpfam_hvp_begin(c, L, &pre[order[i]]) != BETTY_OK) pre[order[i]] = nullptr;
        ++made;
      }
      side.end();
    }
    rc = level_grad(c, levels[k], levels[k], out);          // direct gradient
    for (int i = 0; i < n_ord && rc == BETTY_OK && plain; ++i) {
      const int t = order[i];
      if (!is_target[t]) continue;
      tgrad[t] = c.arena.alloc<float>((size_t)levels[t]->n_params);
      if (!tgrad[t]) { rc = BETTY_ERR_WORKSPACE; break; }
      rc = level_grad(c, levels[k], levels[t], tgrad[t]);
    }
    const betty_status rj = side.join();
    if (rc == BETTY_OK) rc = rj;
  }
  for (int i = 0; i < g.n_u2l && rc == BETTY_OK; ++i) {
    if (g.u2l[i].from != k) continue;
    const int c0 = g.u2l[i].to;
    if (c0 == k) continue;
    rc = eval_node(e, c0);
    if (rc != BETTY_OK || !u[c0]) continue;
    rc = brj(c, levels[c0], levels[k], u[c0], per_level[c0], out, true, pre[c0]);
  }
  if (share) mlpfam_unshare_weights(c);
  return rc;
}

// Execution of Sec. 3.3: a problem takes one gradient step when called; after every unroll_steps of
// its steps it calls the problems it constrains through lower-to-upper edges; a called problem steps
// once all problems of its L set have called.
struct Engine {
  Ctx* c; const betty_level* const* levels; const Graph* g; const betty_method_cfg* cfg; const int32_t* unroll;
  int32_t* log; int log_capacity; int n_logged;
  int n_lower[256]; bool has_child[256]; int count[256]; int ready[256];
};
static betty_status engine_step(Engine& e, int j, int depth) {
  if (depth > 256) return BETTY_ERR_INVALID_ARG;
  const betty_level* L = e.levels[j];
  if (e.log && e.n_logged < e.log_capacity) e.log[e.n_logged] = j;
  e.n_logged += 1;
  const size_t mark = e.c->arena.mark();
  const bool fused = L->optimizer == BETTY_OPT_GD && L->grad_accum <= 1 && !e.has_child[j] && (L->loss == BETTY_LOSS_LOGREG_WD || L->loss == BETTY_LOSS_QUADRATIC_WD ||
                                         L->loss == BETTY_LOSS_MLP_CE_REWEIGHT);
  if (fused) {
    BETTY_TRY(is_vector_family(L->loss) ? vecfam_lower_step(*e.c, L, 1, e.count[j]) : mlpfam_lower_step(*e.c, L, 1, e.count[j]));
  } else {
    float* gvec = e.c->arena.alloc<float>((size_t)L->n_params);
    if (!gvec) return BETTY_ERR_WORKSPACE;
    if (e.n_lower[j] == 0 && L->grad_accum > 1) BETTY_TRY(step_grad(*e.c, L, gvec));
    else BETTY_TRY(graph_hypergrad(*e.c, e.levels, *e.g, j, e.cfg, gvec));
    BETTY_TRY(apply_optimizer(*e.c, L, gvec, e.count[j]));
  }
  e.c->arena.release(mark);
  e.count[j] += 1;
  if (e.count[j] % e.unroll[j] == 0) {
    for (int i = 0; i < e.g->n_l2u; ++i) {
      if (e.g->l2u[i].from != j) continue;
      const int m = e.g->l2u[i].to;
      e.ready[m] += 1;
      if (e.ready[m] >= e.n_lower[m]) {
        e.ready[m] = 0;
        BETTY_TRY(engine_step(e, m, depth + 1));
      }
    }
  }
  return BETTY_OK;
}

}  // namespace betty

using namespace betty;

extern "C" {

betty_status betty_find_paths(int32_t n_levels, const betty_edge* u2l, int32_t n_u2l, const betty_edge* l2u,
                              int32_t n_l2u, int32_t k, const int32_t* targets, int32_t n_targets, int32_t* paths,
                              int32_t capacity, int32_t* n_paths, int32_t* n_ints) {
  Graph g = {n_levels, u2l, n_u2l, l2u, n_l2u};
  if (!graph_ok(g) || k < 0 || k >= n_levels || n_targets < 0 || (n_targets > 0 && !targets) || n_levels > 4096 ||
      capacity < 0 || !n_paths)
    return BETTY_ERR_INVALID_ARG;
  bool is_target[4096] = {false};
  bool on_path[4096] = {false};
  int stack[4096];
  for (int i = 0; i < n_targets; ++i) {
    if (targets[i] < 0 || targets[i] >= n_levels) return BETTY_ERR_INVALID_ARG;
    is_target[targets[i]] = true;
  }
  PathSink s = {paths, capacity, 0, 0, false};
  for (int i = 0; i < n_u2l; ++i) {
    if (u2l[i].from != k) continue;
    const int c0 = u2l[i].to;
    if (c0 == k) continue;
    stack[0] = c0; on_path[c0] = true;
    dfs_paths(g, k, is_target, stack, on_path, 1, s);
    on_path[c0] = false;
  }
  *n_paths = s.count;
  if (n_ints) *n_ints = s.used;
  return s.overflow ? BETTY_ERR_WORKSPACE : BETTY_OK;
}

betty_status betty_hypergrad_graph(const betty_level* const* levels, int32_t n_levels, const betty_edge* u2l,
                                   int32_t n_u2l, const betty_edge* l2u, int32_t n_l2u, int32_t k,
                                   const betty_method_cfg* per_level, float* out, void* ws, size_t ws_bytes,
                                   void* stream) {
  Graph g = {n_levels, u2l, n_u2l, l2u, n_l2u};
  if (!levels || !graph_ok(g) || k < 0 || k >= n_levels || !per_level || !out || n_levels > 256) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(out)) return BETTY_ERR_ALIGNMENT;
  for (int i = 0; i < n_levels; ++i) BETTY_TRY(validate_level(levels[i]));
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  return graph_hypergrad(c, levels, g, k, per_level, out);
}

betty_status betty_engine_run(const betty_level* const* levels, int32_t n_levels, const betty_edge* u2l, int32_t n_u2l,
                              const betty_edge* l2u, int32_t n_l2u, const betty_method_cfg* per_level,
                              const int32_t* unroll_steps, int32_t n_iterations, int32_t* step_log,
                              int32_t log_capacity, int32_t* n_steps_taken, void* ws, size_t ws_bytes, void* stream) {
  Graph g = {n_levels, u2l, n_u2l, l2u, n_l2u};
  if (!levels || !graph_ok(g) || !per_level || !unroll_steps || n_iterations < 0 || n_levels > 256 || log_capacity < 0)
    return BETTY_ERR_INVALID_ARG;
  for (int i = 0; i < n_levels; ++i) {
    BETTY_TRY(validate_level(levels[i]));
    if (unroll_steps[i] < 1) return BETTY_ERR_INVALID_ARG;
    if (levels[i]->comm || levels[i]->loss_scale) return BETTY_ERR_UNSUPPORTED;   // not offered for data-parallel or loss-scaled levels
  }
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  Engine e = {};
  e.c = &c; e.levels = levels; e.g = &g; e.cfg = per_level; e.unroll = unroll_steps;
  e.log = step_log; e.log_capacity = log_capacity;
  for (int i = 0; i < n_l2u; ++i) e.n_lower[l2u[i].to] += 1;
  for (int i = 0; i < n_u2l; ++i) e.has_child[u2l[i].from] = true;
  betty_status st = BETTY_OK;
  for (int it = 0; it < n_iterations && st == BETTY_OK; ++it)
    for (int j = 0; j < n_levels && st == BETTY_OK; ++j)
      if (e.n_lower[j] == 0) st = engine_step(e, j, 0);       // only the lowermost problems are called directly
  if (n_steps_taken) *n_steps_taken = e.n_logged;
  return st;
}

betty_status betty_hypergrad_itd(const betty_level* lower, const betty_level* upper, const betty_level* wrt,
                                 int32_t n_steps, float* out, void* ws, size_t ws_bytes, void* stream) {
  return hypergrad_itd(lower, upper, wrt, n_steps, out, ws, ws_bytes, stream);
}

const char* betty_status_string(betty_status s) {
  switch (s) {
    case BETTY_OK: return "ok";
    case BETTY_ERR_INVALID_ARG: return "invalid argument";
    case BETTY_ERR_SHAPE: return "shape mismatch";
    case BETTY_ERR_DTYPE: return "unsupported dtype";
    case BETTY_ERR_ALIGNMENT: return "misaligned pointer";
    case BETTY_ERR_WORKSPACE: return "workspace too small or misaligned";
    case BETTY_ERR_CUDA: return "CUDA runtime error";
    case BETTY_ERR_NONFINITE: return "non-finite value met on the device";
    case BETTY_ERR_BREAKDOWN: return "conjugate gradient breakdown (p^T H p <= 0)";
    case BETTY_ERR_TIMEOUT: return "bounded device wait expired";
    case BETTY_ERR_UNSUPPORTED: return "unsupported combination";
    case BETTY_ERR_CAPACITY: return "size exceeds the fixed built-in scratch of this allocation-free call";
  }
  return "unknown status";
}

uint64_t betty_kernel_launches(void) { return (uint64_t)g_kernel_launches.load(std::memory_order_relaxed); }

int32_t betty_selftest_smem_limit(int32_t reset, int32_t device, uint64_t bytes) {
  static SmemLimit lim = {};
  if (reset) lim = SmemLimit{};
  return lim.raise(device, (size_t)bytes) ? 1 : 0;
}

betty_status betty_workspace_size(const betty_level* const* levels, int32_t n_levels, size_t* bytes) {
  if (!levels || n_levels <= 0 || !bytes) return BETTY_ERR_INVALID_ARG;
  size_t total = 1 << 20;
  size_t maxp = 0;
  for (int i = 0; i < n_levels; ++i) {
    const betty_level* L = levels[i];
    if (!L) return BETTY_ERR_INVALID_ARG;
    if ((size_t)L->n_params > maxp) maxp = (size_t)L->n_params;
    if (is_vector_family(L->loss)) {
      // per-CTA column partials of the streaming pass (2 CTAs per SM) or the fallback's row scratch
      size_t d = (size_t)(L->d > 0 ? L->d : 1), n = (size_t)(L->n > 0 ? L->n : 1);
      // (+ n floats: the per-row curvature shared by the HVPs of one solve)
      size_t need = (size_t)(2 * current_sm_count() + 64) * d * sizeof(float) + 2 * n * sizeof(float) + 8192;
      if (need > total) total = need + (1 << 20);
    } else if (is_mlp_family(L->loss)) {
      total += mlpfam_workspace(L);
    } else {
      return BETTY_ERR_INVALID_ARG;
    }
  }
  // solver vectors: v, q, h, t/r, p, m plus chain intermediates, each padded
  total += 10 * (maxp * sizeof(float) + 256) + (1 << 16);
  *bytes = (total + 255) & ~size_t(255);
  return BETTY_OK;
}

betty_status betty_reset_status(void* ws, size_t ws_bytes, void* stream) {
  BETTY_TRY(check_ws(ws, ws_bytes));
  if (cudaMemsetAsync(ws, 0, sizeof(StatusBlock), (cudaStream_t)stream) != cudaSuccess) return BETTY_ERR_CUDA;
  return BETTY_OK;
}

betty_status betty_poll_status(const void* ws, void* stream, int32_t* cg_iters) {
  if (!ws) return BETTY_ERR_WORKSPACE;
  StatusBlock h;
  if (cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) return BETTY_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BETTY_ERR_CUDA;
  if (cg_iters) *cg_iters = h.cg_iters;
  if (h.code < 0 || h.code > BETTY_ERR_CAPACITY) return BETTY_ERR_CUDA;   // not a status this library writes
  return (betty_status)h.code;
}

betty_status betty_lower_step(const betty_level* L, int32_t n_steps, void* ws, size_t ws_bytes, void* stream) {
  BETTY_TRY(validate_level(L));
  if (n_steps < 0) return BETTY_ERR_INVALID_ARG;
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  if (L->optimizer != BETTY_OPT_GD || L->grad_accum > 1 || L->comm || L->loss_scale) {
    BETTY_ALLOC(g, float, c, (size_t)L->n_params);
    int* overflow = nullptr;
    if (L->loss_scale) {
      overflow = c.arena.alloc<int>(8);
      if (!overflow) return BETTY_ERR_WORKSPACE;
      c.loss_scale = L->loss_scale;       // the gradient pass multiplies its top deltas by the scale
    }
    for (int s = 0; s < n_steps; ++s) {
      BETTY_TRY(step_grad(c, L, g));
      if (overflow) {
        if (cudaMemsetAsync(overflow, 0, sizeof(int), c.stream) != cudaSuccess) return BETTY_ERR_CUDA;
        launch_pdl(k_unscale_check, dim3(ew_grid(L->n_params)), dim3(256), 0, c.stream, g, L->n_params, (const float*)L->loss_scale, overflow);
        BETTY_LAUNCH_CHECK();
      }
      BETTY_TRY(apply_optimizer(c, L, g, s, overflow));
      if (overflow) {
        launch_pdl(k_loss_scale_update, dim3(1), dim3(1), 0, c.stream, L->loss_scale, (const int*)overflow);
        BETTY_LAUNCH_CHECK();
      }
    }
    c.loss_scale = nullptr;
    return BETTY_OK;
  }
  if (is_vector_family(L->loss)) return vecfam_lower_step(c, L, n_steps);
  return mlpfam_lower_step(c, L, n_steps);
}

betty_status betty_grad(const betty_level* L, const betty_level* wrt, float* out, void* ws, size_t ws_bytes,
                        void* stream) {
  BETTY_TRY(validate_level(L));
  if (!wrt || !out || !is_participant(L, wrt)) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(out)) return BETTY_ERR_ALIGNMENT;
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  return level_grad(c, L, wrt, out);
}

betty_status betty_hvp(const betty_level* L, const float* u, float* Hu, void* ws, size_t ws_bytes, void* stream) {
  BETTY_TRY(validate_level(L));
  if (!u || !Hu) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(u) || !aligned16(Hu)) return BETTY_ERR_ALIGNMENT;
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  if (is_vector_family(L->loss)) {
    BETTY_TRY(vecfam_hvp(c, L, u, Hu));
  } else {
    MlpHvpCache* cache = nullptr;
    BETTY_TRY(mlpfam_hvp_begin(c, L, &cache));
    BETTY_TRY(mlpfam_hvp(c, L, cache, u, Hu));
  }
  return dp_reduce(c, L, Hu, L->n_params);
}

betty_status betty_mixed_vjp(const betty_level* L, const betty_level* wrt, const float* q, float* out, void* ws,
                             size_t ws_bytes, void* stream) {
  BETTY_TRY(validate_level(L));
  if (!wrt || !q || !out || !is_participant(L, wrt) || wrt == L) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return BETTY_ERR_ALIGNMENT;
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  if (is_vector_family(L->loss)) {
    BETTY_TRY(vecfam_mixed(c, L, wrt, q, out));
  } else {
    MlpHvpCache* cache = nullptr;
    BETTY_TRY(mlpfam_hvp_begin(c, L, &cache));
    BETTY_TRY(mlpfam_mixed(c, L, cache, wrt, q, out));
  }
  return dp_reduce(c, L, out, wrt->n_params);
}

betty_status betty_hypergrad_neumann(const betty_level* lower, const betty_level* upper, const betty_level* wrt,
                                     int32_t K, float alpha, float* out, void* ws, size_t ws_bytes, void* stream) {
  betty_method_cfg cfg = {BETTY_NEUMANN, K, alpha, 0.f, 0.f};
  return hypergrad(lower, upper, wrt, cfg, out, ws, ws_bytes, stream);
}

betty_status betty_hypergrad_cg(const betty_level* lower, const betty_level* upper, const betty_level* wrt, int32_t K,
                                float tol, float* out, void* ws, size_t ws_bytes, void* stream) {
  betty_method_cfg cfg = {BETTY_CG, K, 0.f, 0.f, tol};
  return hypergrad(lower, upper, wrt, cfg, out, ws, ws_bytes, stream);
}

betty_status betty_hypergrad_fd(const betty_level* lower, const betty_level* upper, const betty_level* wrt, float eps0,
                                float alpha, float* out, void* ws, size_t ws_bytes, void* stream) {
  if (!(eps0 > 0.f)) return BETTY_ERR_INVALID_ARG;
  betty_method_cfg cfg = {BETTY_FD, 0, alpha, eps0, 0.f};
  return hypergrad(lower, upper, wrt, cfg, out, ws, ws_bytes, stream);
}

betty_status betty_chain_levels(const betty_level* const* levels, int32_t n_levels, const int32_t* path,
                                int32_t path_len, const betty_method_cfg* per_edge, const float* v_in, float* out,
                                int32_t accumulate, void* ws, size_t ws_bytes, void* stream) {
  if (!levels || n_levels <= 0 || !path || path_len < 2 || !per_edge || !out) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(out) || !aligned16(v_in)) return BETTY_ERR_ALIGNMENT;     // a null v_in counts as aligned
  for (int i = 0; i < path_len; ++i)
    if (path[i] < 0 || path[i] >= n_levels || !levels[path[i]]) return BETTY_ERR_INVALID_ARG;
  for (int i = 0; i < path_len; ++i) BETTY_TRY(validate_level(levels[path[i]]));
  BETTY_TRY(check_ws(ws, ws_bytes));
  Ctx c(ws, ws_bytes, stream);
  const betty_level* K = levels[path[0]];
  const int m = path_len - 1;
  const betty_level* last = levels[path[m]];
  const float* v = v_in;
  if (!v) {
    if (!is_participant(K, last)) return BETTY_ERR_INVALID_ARG;
    BETTY_ALLOC(v0, float, c, (size_t)last->n_params);
    BETTY_TRY(level_grad(c, K, last, v0));
    v = v0;
  }
  for (int i = m; i >= 2; --i) {
    const betty_level* Li = levels[path[i]];
    const betty_level* Lprev = levels[path[i - 1]];
    BETTY_ALLOC(vn, float, c, (size_t)Lprev->n_params);
    BETTY_TRY(brj(c, Li, Lprev, v, per_edge[i - 1], vn, false));
    v = vn;
  }
  return brj(c, levels[path[1]], K, v, per_edge[0], out, accumulate != 0);
}

}  // extern "C"
