// Per-cost-family operations behind the C ABI.  Each function enqueues kernels on ctx.stream
// and allocates its scratch from ctx.arena.
#pragma once
#include <math.h>
#include "common.cuh"

namespace betty {

static inline const betty_level* find_constraint(const betty_level* L, int kind) {
  for (int i = 0; i < L->n_constraints; ++i)
    if (L->constraints[i] && L->constraints[i]->param_kind == kind) return L->constraints[i];
  return nullptr;
}
static inline const betty_level* find_participant(const betty_level* L, int kind) {
  if (L->param_kind == kind) return L;
  return find_constraint(L, kind);
}
static inline bool is_vector_family(int loss) {
  return loss == BETTY_LOSS_LOGREG_WD || loss == BETTY_LOSS_LOGREG || loss == BETTY_LOSS_QUADRATIC_WD ||
         loss == BETTY_LOSS_QUADRATIC;
}
static inline bool is_mlp_family(int loss) {
  return loss == BETTY_LOSS_MLP_CE_REWEIGHT || loss == BETTY_LOSS_MLP_CE || loss == BETTY_LOSS_WEIGHTNET_DETECT ||
         loss == BETTY_LOSS_MLP_CE_CORRECT;
}

// logreg.cu
// What the pass's reduction kernel does with the finished product h = H u besides storing it: the solver update
// that would otherwise be one to three more small kernels between two passes over the matrix.
enum { LR_TAIL_NONE = 0, LR_TAIL_NEUMANN = 1, LR_TAIL_CG = 2 };
struct LrTail {
  int kind;
  // LR_TAIL_NEUMANN (the pass's direction u is the current term t):  t_out = u - alpha*h,  s_out = s_in + t_out
  const float* s_in; float* t_out; float* s_out; float alpha;
  // LR_TAIL_CG (the pass's direction u is p): gamma = p.h; a = rho/gamma; q += a p; r -= a h; rho' = r.r;
  // p = r + (rho'/rho) p; the state advances as in cg_step.  partials holds one double per 32 columns,
  // counter is a zeroed ticket (both from the solve's reduction buffer).
  SolveState* st; float* q; float* r; float* p; double* partials; unsigned* counter;
};
// number of 32-column blocks the fused CG iteration can take (size of a reduction buffer)
int64_t logreg_tail_max_d();
// curv / curv_valid: the per-row curvature buffer of one solve and whether it holds the curvature at w.  A pass
// reads it only when *curv_valid is set and sets *curv_valid only when it has itself written the buffer (the
// single-pass kernel in its full HVP form); the two-pass fallback neither reads nor writes it.
betty_status logreg_pass(Ctx& c, int family, const float* X, const float* y, int64_t n, int64_t d, const float* w,
                         const float* u, const float* lam, float* out, float* w_update, float lr, float* curv = nullptr,
                         bool* curv_valid = nullptr, const LrTail* tail = nullptr);

// logreg_small.cu: whole-loop kernels for problems that fit a cluster's shared memory
bool logreg_small_eligible(int64_t n, int64_t nv, int64_t d, int64_t unrolled_steps = 0);
betty_status logreg_small_itd(Ctx& c, int family, const float* X, const float* y, int64_t n, int family_up, const float* Xv,
                              const float* yv, int64_t nv, int64_t d, float* w, const float* lam, int n_steps, float lr,
                              float* out);
betty_status logreg_small_lower_step(Ctx& c, int family, const float* X, const float* y, int64_t n, int64_t d, float* w,
                                     const float* lam, int n_steps, float lr);
betty_status logreg_small_hypergrad(Ctx& c, int family, const float* X, const float* y, int64_t n, int family_up,
                                    const float* Xv, const float* yv, int64_t nv, int64_t d, float* w, const float* lam,
                                    const betty_method_cfg& cfg, float* out);

// ---- vector families (api.cu) ----
betty_status vecfam_validate(const betty_level* L);
betty_status vecfam_grad(Ctx& c, const betty_level* L, const betty_level* wrt, float* out);
// Per-row curvature of a logistic level at its present parameters, shared by the HVPs of one solve: the first
// HVP fills it, the later ones read it (n floats in the caller's workspace; null: every HVP recomputes z = X w).
struct VecHvpCache { float* curv; bool valid; };
betty_status vecfam_hvp(Ctx& c, const betty_level* L, const float* u, float* Hu, VecHvpCache* cache = nullptr,
                        const LrTail* tail = nullptr);
betty_status vecfam_mixed(Ctx& c, const betty_level* L, const betty_level* wrt, const float* q, float* out);
betty_status vecfam_lower_step(Ctx& c, const betty_level* L, int n_steps, int first_step = 0);
// out (+)= -alpha*[dC/dc(x+eps v) - dC/dc(x-eps v)]/(2 eps), eps = eps0/sqrt(*vnorm2) on the device
betty_status vecfam_fd(Ctx& c, const betty_level* L, const betty_level* wrt, const float* v, const float* vnorm2,
                       float eps0, float alpha, float* out, bool accumulate);

// ---- MLP families (mlp.cu) ----
// Step size of problem L for its step number `step_in_call` of the present call (betty_lr_schedule)
static inline float lr_at(const betty_level* L, int step_in_call) {
  const long long t = (long long)L->lr_step0 + step_in_call;
  if (L->lr_schedule == BETTY_LR_MULTISTEP) {
    double lr = L->lr;
    for (int i = 0; i < 4; ++i)
      if (L->lr_milestones[i] > 0 && t >= L->lr_milestones[i]) lr *= (double)L->lr_gamma;
    return (float)lr;
  }
  if (L->lr_schedule == BETTY_LR_COSINE && L->lr_t_max > 0) {
    const double u = (double)(t < L->lr_t_max ? t : L->lr_t_max) / (double)L->lr_t_max;
    return (float)((double)L->lr_min + ((double)L->lr - (double)L->lr_min) * 0.5 * (1.0 + cos(3.14159265358979323846 * u)));
  }
  return L->lr;
}

struct MlpHvpCache;  // opaque handle: base forward/backward state shared by the HVPs of one solve
// base passes (mlpfam_hvp_begin) a host thread may hold at once: handles are slots of a per-thread ring, and the
// oldest is reused by the call after this many
static constexpr int MLP_HVP_CACHE_SLOTS = 8;

// The MLP families exist once per 16-bit operand type (see common.cuh): identical declarations in two namespaces.
#define BETTY_DECLARE_MLP_FAMILY(NS)                                                                                   \
  namespace NS {                                                                                                       \
  betty_status mlpfam_validate(const betty_level* L);                                                                  \
  size_t mlpfam_workspace(const betty_level* L);                                                                       \
  betty_status mlpfam_grad(Ctx& c, const betty_level* L, const betty_level* wrt, float* out);                          \
  betty_status mlpfam_share_weights(Ctx& c, const betty_level* M);                                                     \
  void mlpfam_unshare_weights(Ctx& c);                                                                                 \
  betty_status mlpfam_hvp_begin(Ctx& c, const betty_level* L, MlpHvpCache** cache);                                    \
  betty_status mlpfam_hvp_keep_direction(Ctx& c, MlpHvpCache* cache);                                                  \
  betty_status mlpfam_hvp(Ctx& c, const betty_level* L, MlpHvpCache* cache, const float* u, float* Hu);                \
  betty_status mlpfam_hvp_series(Ctx& c, const betty_level* L, MlpHvpCache* cache, const float* s, const float* v, float alpha, \
                                 float* s_out);                                                                        \
  betty_status mlpfam_mixed(Ctx& c, const betty_level* L, MlpHvpCache* cache, const betty_level* wrt, const float* q,  \
                            float* out);                                                                               \
  betty_status mlpfam_lower_step(Ctx& c, const betty_level* L, int n_steps, int first_step = 0);                       \
  betty_status mlpfam_fd_begin(Ctx& c, const betty_level* L, MlpHvpCache** cache);                                     \
  betty_status mlpfam_fd(Ctx& c, const betty_level* L, const betty_level* wrt, const float* v, const float* vnorm2,    \
                         float eps0, float alpha, float* out, bool accumulate, MlpHvpCache* pre);                      \
  }
BETTY_DECLARE_MLP_FAMILY(fam_bf16)
BETTY_DECLARE_MLP_FAMILY(fam_f16)

}  // namespace betty
