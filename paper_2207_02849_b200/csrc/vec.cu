// Vector kernels for the inverse-Hessian solves of Sec. 3.2 (Neumann series, conjugate gradient):
// deterministic dot products (warp shuffles + a fixed-order second phase), fused axpy updates,
// and the device-resident state machine of CG so that no host synchronisation is needed.
#include "common.cuh"

namespace betty {

static constexpr int VT = 256;        // threads per block
static constexpr int DOT_MAX_BLOCKS = 592;

static inline int ew_blocks(int64_t n, int per_thread = 4) {
  int64_t b = (n + (int64_t)VT * per_thread - 1) / ((int64_t)VT * per_thread);
  if (b < 1) b = 1;
  if (b > 148 * 16) b = 148 * 16;
  return (int)b;
}

__global__ void k_zero(float* x, int64_t n) {
  pdl_enter();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) x[i] = 0.f;
}
__global__ void k_copy(float* d, const float* s, int64_t n) {
  pdl_enter();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) d[i] = s[i];
}
__global__ void k_axpby(float* out, float a, const float* x, float b, const float* y, int64_t n) {
  pdl_enter();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = y ? a * x[i] + b * y[i] : a * x[i];
}
__global__ void k_mul(float* out, float a, const float* x, const float* y, int64_t n) {
  pdl_enter();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = a * x[i] * y[i];
}
__global__ void k_neumann(const float* t_in, const float* s_in, const float* Ht, float alpha, float* t_out, float* s_out,
                          int64_t n) {
  pdl_enter();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    float tn = t_in[i] - alpha * Ht[i];
    t_out[i] = tn;
    s_out[i] = s_in[i] + tn;
  }
}

betty_status vec_zero(Ctx& c, float* x, int64_t n) {
  if (n <= 0) return BETTY_OK;
  launch_pdl(k_zero, dim3(ew_blocks(n)), dim3(VT), 0, c.stream, x, n);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
betty_status vec_copy(Ctx& c, float* d, const float* s, int64_t n) {
  if (n <= 0) return BETTY_OK;
  launch_pdl(k_copy, dim3(ew_blocks(n)), dim3(VT), 0, c.stream, d, s, n);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
betty_status vec_axpby(Ctx& c, float* out, float a, const float* x, float b, const float* y, int64_t n) {
  if (n <= 0) return BETTY_OK;
  launch_pdl(k_axpby, dim3(ew_blocks(n)), dim3(VT), 0, c.stream, out, a, x, b, y, n);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
betty_status vec_mul(Ctx& c, float* out, float a, const float* x, const float* y, int64_t n) {
  if (n <= 0) return BETTY_OK;
  launch_pdl(k_mul, dim3(ew_blocks(n)), dim3(VT), 0, c.stream, out, a, x, y, n);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
betty_status neumann_update(Ctx& c, const float* t_in, const float* s_in, const float* Ht, float alpha, float* t_out,
                            float* s_out, int64_t n) {
  if (n <= 0) return BETTY_OK;
  launch_pdl(k_neumann, dim3(ew_blocks(n)), dim3(VT), 0, c.stream, t_in, s_in, Ht, alpha, t_out, s_out, n);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// ------------------------------------------------------------------ deterministic reductions
// Block-level sum in double: warp shuffles, then one value per warp through shared memory, summed
// by every thread in warp order.  The order of additions depends only on the launch shape.
__device__ __forceinline__ double block_sum(double v, double* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int w = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) sh[w] = v;
  __syncthreads();
  double t = 0.0;
  for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += sh[i];
  __syncthreads();
  return t;
}

// Second phase: the block that draws the last ticket sums the per-block partials in index order.
// Returns true (in every thread of that block) with the total in *total.
__device__ __forceinline__ bool last_block_total(double part, double* partials, unsigned* counter,
                                                 double* sh, double* total) {
  __shared__ bool is_last;
  if (threadIdx.x == 0) {
    partials[blockIdx.x] = part;
    __threadfence();
    unsigned t = atomicAdd(counter, 1u);
    is_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return false;
  __threadfence();
  double v = 0.0;
  for (unsigned i = threadIdx.x; i < gridDim.x; i += blockDim.x) v += ((volatile double*)partials)[i];
  *total = block_sum(v, sh);
  if (threadIdx.x == 0) *counter = 0u;
  return true;
}

// partial buffer: [DOT_MAX_BLOCKS doubles][1 unsigned counter (zeroed once per call)]
int64_t vec_dot_partials(int64_t) { return 2 * DOT_MAX_BLOCKS + 8; }  // in floats

static inline int dot_blocks(int64_t n) {
  int64_t b = (n + VT * 8 - 1) / (VT * 8);
  if (b < 1) b = 1;
  if (b > DOT_MAX_BLOCKS) b = DOT_MAX_BLOCKS;
  return (int)b;
}

__global__ void k_dot(const float* x, const float* y, int64_t n, float* result, double* partials,
                      unsigned* counter, StatusBlock* sb) {
  pdl_enter();
  __shared__ double sh[VT / 32];
  double acc = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    acc += (double)x[i] * (double)y[i];
  double part = block_sum(acc, sh), total;
  if (last_block_total(part, partials, counter, sh, &total) && threadIdx.x == 0) {
    *result = (float)total;
    if (!isfinite(total)) record_status(sb, BETTY_ERR_NONFINITE);
  }
}

betty_status vec_reduce_init(Ctx& c, float* partials) {
  unsigned* counter = (unsigned*)((double*)partials + DOT_MAX_BLOCKS);
  return vec_zero(c, (float*)counter, 8);     // a kernel, not a memset: keeps the programmatic launch chain unbroken
}

betty_status vec_dot(Ctx& c, const float* x, const float* y, int64_t n, float* result, float* partials) {
  double* pd = (double*)partials;
  unsigned* counter = (unsigned*)(pd + DOT_MAX_BLOCKS);
  launch_pdl(k_dot, dim3(dot_blocks(n)), dim3(VT), 0, c.stream, x, y, n, result, pd, counter, c.arena.status());
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// ------------------------------------------------------------------ conjugate gradient
// q <- 0, r <- v, p <- v, rho <- v.v, stop <- tol^2 * v.v
__global__ void k_cg_init(SolveState* st, const float* v, float* q, float* r, float* p, float tol, int64_t n,
                          double* partials, unsigned* counter, StatusBlock* sb) {
  pdl_enter();
  __shared__ double sh[VT / 32];
  double acc = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    float vi = v[i];
    q[i] = 0.f; r[i] = vi; p[i] = vi;
    acc += (double)vi * (double)vi;
  }
  double part = block_sum(acc, sh), total;
  if (last_block_total(part, partials, counter, sh, &total) && threadIdx.x == 0) {
    st->rho = (float)total;
    st->vnorm2 = (float)total;
    st->stop = tol * tol * (float)total;
    st->gamma = 0.f; st->rho_new = 0.f; st->iters = 0;
    st->active = ((float)total > st->stop) ? 1 : 0;
    sb->cg_iters = 0;
    if (!isfinite(total)) { record_status(sb, BETTY_ERR_NONFINITE); st->active = 0; }
  }
}

// gamma <- p.h
__global__ void k_cg_gamma(SolveState* st, const float* p, const float* h, int64_t n, double* partials,
                           unsigned* counter, StatusBlock* sb) {
  pdl_enter();
  __shared__ double sh[VT / 32];
  double acc = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    acc += (double)p[i] * (double)h[i];
  double part = block_sum(acc, sh), total;
  if (last_block_total(part, partials, counter, sh, &total) && threadIdx.x == 0) {
    st->gamma = (float)total;
    if (st->active) {
      if (!isfinite(total)) { record_status(sb, BETTY_ERR_NONFINITE); st->active = 0; }
      else if (!(total > 0.0)) { record_status(sb, BETTY_ERR_BREAKDOWN); st->active = 0; }
    }
  }
}

// a = rho/gamma; q += a p; r -= a h; rho_new <- r.r   (no-op when the solve has stopped)
__global__ void k_cg_update(SolveState* st, float* q, float* r, const float* p, const float* h, int64_t n,
                            double* partials, unsigned* counter) {
  pdl_enter();
  __shared__ double sh[VT / 32];
  if (!st->active) return;
  const float a = st->rho / st->gamma;
  double acc = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    q[i] += a * p[i];
    float ri = r[i] - a * h[i];
    r[i] = ri;
    acc += (double)ri * (double)ri;
  }
  double part = block_sum(acc, sh), total;
  if (last_block_total(part, partials, counter, sh, &total) && threadIdx.x == 0) st->rho_new = (float)total;
}

// p <- r + (rho_new/rho) p ; then the last block advances the state: rho <- rho_new, iters++,
// and deactivates the solve once rho <= stop.
__global__ void k_cg_direction(SolveState* st, float* p, const float* r, int64_t n, unsigned* counter,
                               StatusBlock* sb) {
  pdl_enter();
  if (!st->active) return;
  const float beta = st->rho_new / st->rho;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    p[i] = r[i] + beta * p[i];
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    unsigned t = atomicAdd(counter, 1u);
    if (t == gridDim.x - 1) {
      *counter = 0u;
      st->rho = st->rho_new;
      st->iters += 1;
      sb->cg_iters = st->iters;
      if (!isfinite(st->rho_new)) { record_status(sb, BETTY_ERR_NONFINITE); st->active = 0; }
      else if (st->rho_new <= st->stop) st->active = 0;
    }
  }
}

betty_status cg_init(Ctx& c, SolveState* st, const float* v, float* q, float* r, float* p, float tol, int64_t n,
                     float* partials) {
  double* pd = (double*)partials;
  unsigned* counter = (unsigned*)(pd + DOT_MAX_BLOCKS);
  launch_pdl(k_cg_init, dim3(dot_blocks(n)), dim3(VT), 0, c.stream, st, v, q, r, p, tol, n, pd, counter, c.arena.status());
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

betty_status cg_step(Ctx& c, SolveState* st, float* q, float* r, float* p, const float* h, int64_t n,
                     float* partials) {
  double* pd = (double*)partials;
  unsigned* counter = (unsigned*)(pd + DOT_MAX_BLOCKS);
  const int nb = dot_blocks(n);
  launch_pdl(k_cg_gamma, dim3(nb), dim3(VT), 0, c.stream, st, p, h, n, pd, counter, c.arena.status());
  BETTY_LAUNCH_CHECK();
  launch_pdl(k_cg_update, dim3(nb), dim3(VT), 0, c.stream, st, q, r, p, h, n, pd, counter);
  BETTY_LAUNCH_CHECK();
  launch_pdl(k_cg_direction, dim3(nb), dim3(VT), 0, c.stream, st, p, r, n, counter + 1, c.arena.status());
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

}  // namespace betty
