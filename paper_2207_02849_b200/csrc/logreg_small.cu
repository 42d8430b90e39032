// Small-problem variant of the logistic / least-squares family (App. D.1 problem at a size where the
// whole data set fits on chip): one launch runs a complete loop -- all unrolled lower-level gradient
// steps, or a complete hypergradient (validation gradient, Neumann / CG / finite-difference solve,
// mixed product).  A cluster of 8 CTAs keeps the rows of X (and of the validation matrix) resident
// for the whole launch -- in registers where the shape allows (pass_reg), else in shared memory (pass).
// In every pass each CTA sends its column sums to all eight CTAs through distributed shared memory with
// stores that are counted on the receiver's barrier, waits for the sums addressed to it, and then repeats
// the same O(d) vector arithmetic on its own copy of the solver state, in the same order, so all copies
// stay bit-identical.  At this size the path is bound by the latency of ~100 dependent passes, not by
// bandwidth: the point of the kernel is to pay one launch instead of hundreds.
#include "ops.cuh"

namespace betty {

static constexpr int SM_CL = 8;          // CTAs per cluster
static constexpr int SM_T = 1024;        // threads per CTA: the passes are latency chains, many warps hide them
static constexpr int SM_MAXD = 256;
static constexpr int SM_PS = SM_MAXD + 4;   // row stride of the per-group partial sums
static constexpr int SM_NVEC = 10;       // vectors of length d kept per CTA

struct SmallArgs {
  const float* X; const float* y; int64_t n;       // lower problem data
  const float* Xv; const float* yv; int64_t nv;    // upper problem data (hypergradient mode)
  int d;
  int family, family_up;                            // 0 logistic, 1 least squares
  float* w;                                         // lower parameters (updated in lower-step mode)
  const float* lam;
  int mode;                                         // 0: lower steps; 1: hypergradient; 2: ITD-RMAD hypergradient over n_steps unrolled steps
  int n_steps; float lr;
  int method, K; float alpha, eps0, tol;            // betty_method and its parameters
  float* out;                                       // hypergradient [d] (added to nothing: direct gradient is zero)
  int rows_per_cta, rows_per_cta_v;
  int in_regs;                                      // rows live in registers (see pass_reg); else in shared memory
  StatusBlock* sb;
};

__device__ __forceinline__ uint32_t sm_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// One column sum sent to CTA `rank` of the cluster; its arrival is counted (4 bytes) on that CTA's barrier.
__device__ __forceinline__ void st_remote_counted(float* local_ptr, uint64_t* local_bar, uint32_t rank, float v) {
  uint32_t a, b;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(sm_u32(local_ptr)), "r"(rank));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(b) : "r"(sm_u32(local_bar)), "r"(rank));
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(a), "f"(v), "r"(b) : "memory");
}
static constexpr uint32_t SM_WAIT_POLLS = 1u << 20;   // bound on every wait for the neighbours' column sums

// Fold the per-group partial column sums of this CTA, send them to slot `rank` of every CTA of the cluster
// (each send counted on the receiver's barrier), wait until all SM_CL x d sums addressed to this CTA have
// landed, and add them up in rank order -- the same order everywhere, so every CTA holds the
// same bits and hands each sum to `post(j, sum)`.  No cluster-wide barrier: a CTA waits only for data, one way.  The two halves of cpart
// alternate between passes; a neighbour can be at most one pass ahead (it needs this CTA's sums of the
// pass before), so what it sends lands in the half this CTA is not reading.  Returns false when the wait
// ran out (uniform over the CTA).
template <class Post>
__device__ __forceinline__ bool exchange_cols(const float* part, int groups, int d, float* cpart, uint64_t* bar, uint32_t parity,
                                              Post post, uint32_t rank) {
  const int tid = threadIdx.x;
  if (tid == 0)
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_u32(bar)), "r"((uint32_t)(SM_CL * d * 4)) : "memory");
  for (int j = tid; j < d; j += SM_T) {
    float acc = 0.f;
    for (int g2 = 0; g2 < groups; ++g2) acc += part[g2 * SM_PS + j];   // unrolled where `groups` is a constant: independent loads
#pragma unroll
    for (uint32_t r = 0; r < SM_CL; ++r) st_remote_counted(cpart + rank * SM_MAXD + j, bar, r, acc);
  }
  // only the warps that read the sums poll the barrier; the others go on to the block barrier below
  uint32_t done = (tid & ~31) < d ? 0u : 1u, polls = 0;
  while (!done && polls < SM_WAIT_POLLS) {
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(sm_u32(bar)), "r"(parity) : "memory");
    ++polls;
  }
  if (done)
    for (int j = tid; j < d; j += SM_T) {
      float acc = 0.f;
#pragma unroll
      for (int r = 0; r < SM_CL; ++r) acc += cpart[r * SM_MAXD + j];
      post(j, acc);     // what the caller does with column j's sum (it owns index j of every vector until the barrier)
    }
  return __syncthreads_or(!done) == 0;
}

__device__ __forceinline__ float sigm(float t) { return 1.f / (1.f + expf(-t)); }

// Sum over j < d <= SM_MAXD of one term per thread (thread j holds term j), the same value in every thread
// (fixed order): only the first ceil(d / 32) warps hold terms, so only their partial sums are formed and added
__device__ __forceinline__ float vsum(float term, int d, float* sh) {
  const int tid = threadIdx.x, nw = (d + 31) >> 5;
  if ((tid >> 5) < nw) {
    float v = tid < d ? term : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((tid & 31) == 0) sh[tid >> 5] = v;
  }
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += sh[i];
  __syncthreads();
  return t;
}
__device__ __forceinline__ float vdot(const float* a, const float* b, int d, float* sh) {
  return vsum(threadIdx.x < d ? a[threadIdx.x] * b[threadIdx.x] : 0.f, d, sh);
}

// One pass over this CTA's resident rows: coef_i from the row dot products, then the column sums
// sum_i coef_i x_ij, reduced over the cluster into res[0..d) (identical in every CTA).
//   kind 0: gradient coefficients at `wv`;  kind 1: HVP coefficients curv_i * (x_i . dir);
//   kind 2: HVP coefficients with the curvature taken at `wv` on the fly (a stored iterate of the unrolled loop)
template <class Post>
__device__ __forceinline__ bool pass(const float* Xs, const float* ys, const float* curv, int rows, int d, int family, float inv_n,
                                     int kind, const float* wv, const float* dir, float* coef, float* part, float* cpart,
                                     uint64_t* bar, uint32_t parity, Post post, uint32_t rank) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // A: one warp per row, four rows in flight per warp so that the shuffle chains overlap
  const float* vv = kind == 0 ? wv : dir;
  for (int i0 = warp * 4; i0 < rows; i0 += (SM_T / 32) * 4) {
    float s[4] = {0.f, 0.f, 0.f, 0.f}, z[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u;
      if (i < rows) {
        const float* xr = Xs + (size_t)i * d;
        for (int j = lane; j < d; j += 32) s[u] += xr[j] * vv[j];
        if (kind == 2)
          for (int j = lane; j < d; j += 32) z[u] += xr[j] * wv[j];
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int u = 0; u < 4; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
    }
    if (kind == 2) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int u = 0; u < 4; ++u) z[u] += __shfl_xor_sync(0xffffffffu, z[u], o);
      }
    }
    if (lane < 4 && i0 + lane < rows) {
      const int i = i0 + lane;
      const float sv = lane == 0 ? s[0] : (lane == 1 ? s[1] : (lane == 2 ? s[2] : s[3]));
      const float zv = lane == 0 ? z[0] : (lane == 1 ? z[1] : (lane == 2 ? z[2] : z[3]));
      float cf;
      if (kind == 0) cf = family == 0 ? -ys[i] * sigm(-ys[i] * sv) * inv_n : (sv - ys[i]);
      else if (kind == 1) cf = curv[i] * sv;
      else { const float sg = sigm(zv); cf = (family == 0 ? sg * (1.f - sg) * inv_n : 1.f) * sv; }
      coef[i] = cf;
    }
  }
  __syncthreads();
  // B: thread per column (x row groups), then fold the row groups
  const int ct = d <= 32 ? 32 : (d <= 64 ? 64 : (d <= 128 ? 128 : 256));   // SM_T / ct row groups, at most 32
  const int groups = SM_T / ct, c0 = tid % ct, rg = tid / ct;
  for (int j = c0; j < d; j += ct) {
    float a = 0.f;
    for (int i = rg; i < rows; i += groups) a += coef[i] * Xs[(size_t)i * d + j];
    part[rg * SM_PS + j] = a;
  }
  __syncthreads();
  return exchange_cols(part, groups, d, cpart, bar, parity, post, rank);
}

// Column sums over the rows of one warp (TPR threads per row, so 32 / TPR rows; lane bits >= TPR select the
// row).  A butterfly that halves what a lane keeps at every round -- the lane with the round's bit clear keeps
// the lower half of its values and receives the partner's contribution to them, the other lane the upper
// half -- costs 4 + 2 + 1 shuffles for eight values where a plain butterfly costs 8 per round; shuffle issue
// (one warp-wide shuffle per clock per SM, 32 warps) is what the pass spends most of its time on.
// On return col[0 .. NF) are the sums of columns 8 c8 + off + i; `writer` is false in lanes holding duplicates.
template <int O, int N, int NV = 8>
struct WarpColumnSum {
  static __device__ __forceinline__ void run(float (&col)[NV], int lane, int& off, bool& writer) {
    if constexpr (O < 32) {
      const bool up = (lane & O) != 0;
      if constexpr (N > 1) {
        constexpr int H = N / 2;
#pragma unroll
        for (int i = 0; i < H; ++i) {
          const float send = up ? col[i] : col[i + H];
          const float keep = up ? col[i + H] : col[i];
          col[i] = keep + __shfl_xor_sync(0xffffffffu, send, O);
        }
        if (up) off += H;
        WarpColumnSum<O * 2, H, NV>::run(col, lane, off, writer);
      } else {
        col[0] += __shfl_xor_sync(0xffffffffu, col[0], O);
        if (up) writer = false;
        WarpColumnSum<O * 2, 1, NV>::run(col, lane, off, writer);
      }
    }
  }
};
template <int TPR> struct RowsPerWarp { static constexpr int value = 32 / TPR; };
template <int TPR> struct ColsLeft { static constexpr int value = 8 / RowsPerWarp<TPR>::value > 0 ? 8 / RowsPerWarp<TPR>::value : 1; };

// The same pass with the CTA's rows held in registers for the whole launch: TPR = d / 8 adjacent threads own
// one row, eight columns each (d a power of two between 8 and 256, at most SM_T / TPR rows per CTA: the
// 1024 x 64 problem gives every CTA 128 rows of 8 threads).  A pass is then 8 multiply-adds, a shuffle
// reduction over the row's threads, the coefficient, 8 more multiplies and the column sums over the warp's
// rows; shared memory is touched only for the 32 per-warp column sums.
//   x8: this thread's eight columns of its row; yv: the row's label (kind 0) or curvature (kind 1); has: row exists;
//   wt: the iterate the curvature is taken at (kind 2)
template <int TPR, class Post>
__device__ __forceinline__ bool pass_reg(const float (&x8)[8], float yv, bool has, int family, float inv_n, int kind,
                                         const float* vv, const float* wt, float* part, float* cpart, uint64_t* bar,
                                         uint32_t parity, Post post, uint32_t rank) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int d = 8 * TPR;
  const int c8 = tid & (TPR - 1);
  const float4 v0 = *(const float4*)(vv + 8 * c8), v1 = *(const float4*)(vv + 8 * c8 + 4);
  float sdot = x8[0] * v0.x + x8[1] * v0.y + x8[2] * v0.z + x8[3] * v0.w + x8[4] * v1.x + x8[5] * v1.y + x8[6] * v1.z + x8[7] * v1.w;
  float zdot = 0.f;
  if (kind == 2) {
    const float4 w0 = *(const float4*)(wt + 8 * c8), w1 = *(const float4*)(wt + 8 * c8 + 4);
    zdot = x8[0] * w0.x + x8[1] * w0.y + x8[2] * w0.z + x8[3] * w0.w + x8[4] * w1.x + x8[5] * w1.y + x8[6] * w1.z + x8[7] * w1.w;
  }
#pragma unroll
  for (int o = TPR >> 1; o > 0; o >>= 1) {
    sdot += __shfl_xor_sync(0xffffffffu, sdot, o);
    if (kind == 2) zdot += __shfl_xor_sync(0xffffffffu, zdot, o);
  }
  float cf = 0.f;
  if (has) {
    if (kind == 0) cf = family == 0 ? -yv * sigm(-yv * sdot) * inv_n : (sdot - yv);
    else if (kind == 1) cf = yv * sdot;
    else { const float sg = sigm(zdot); cf = (family == 0 ? sg * (1.f - sg) * inv_n : 1.f) * sdot; }
  }
  float col[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) col[k] = cf * x8[k];
  int off = 0;
  bool writer = true;
  WarpColumnSum<TPR, 8>::run(col, lane, off, writer);
  if (writer) {
#pragma unroll
    for (int i = 0; i < ColsLeft<TPR>::value; ++i) part[warp * SM_PS + 8 * c8 + off + i] = col[i];
  }
  __syncthreads();
  return exchange_cols(part, SM_T / 32, d, cpart, bar, parity, post, rank);
}
// dispatch on the threads per row
template <class Post>
__device__ __forceinline__ bool pass_reg_any(int tpr, const float (&x8)[8], float yv, bool has, int family, float inv_n, int kind,
                                             const float* vv, const float* wt, float* part, float* cpart, uint64_t* bar,
                                             uint32_t parity, Post post, uint32_t rank) {
  switch (tpr) {
    case 1: return pass_reg<1>(x8, yv, has, family, inv_n, kind, vv, wt, part, cpart, bar, parity, post, rank);
    case 2: return pass_reg<2>(x8, yv, has, family, inv_n, kind, vv, wt, part, cpart, bar, parity, post, rank);
    case 4: return pass_reg<4>(x8, yv, has, family, inv_n, kind, vv, wt, part, cpart, bar, parity, post, rank);
    case 8: return pass_reg<8>(x8, yv, has, family, inv_n, kind, vv, wt, part, cpart, bar, parity, post, rank);
    case 16: return pass_reg<16>(x8, yv, has, family, inv_n, kind, vv, wt, part, cpart, bar, parity, post, rank);
    default: return pass_reg<32>(x8, yv, has, family, inv_n, kind, vv, wt, part, cpart, bar, parity, post, rank);
  }
}

__global__ void __cluster_dims__(SM_CL, 1, 1) __launch_bounds__(SM_T, 1) k_logreg_small(SmallArgs a) {
  extern __shared__ __align__(16) float sm[];
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int d = a.d, tid = threadIdx.x;
  const int R = a.rows_per_cta, Rv = a.rows_per_cta_v;
  float* Xs = sm;                                  // [R, d]
  float* Xvs = Xs + (size_t)R * d;                 // [Rv, d]
  float* ys = Xvs + (size_t)Rv * d;                // [R]
  float* yvs = ys + R;                             // [Rv]
  float* curv = yvs + Rv;                          // [R]  sigmoid(z) sigmoid(-z) / n at the current w
  float* coef = curv + R;                          // [max(R, Rv)]
  float* vec = coef + (R > Rv ? R : Rv);           // SM_NVEC vectors of SM_MAXD, 16-byte aligned for float4 access
  vec += (4 - ((vec - sm) & 3)) & 3;
  float* part = vec + SM_NVEC * SM_MAXD;           // [32][SM_PS] row-group partials
  float* cpart = part + 32 * SM_PS;               // [2][SM_CL][SM_MAXD] column sums of every CTA (double-buffered)
  float* red = cpart + 2 * SM_CL * SM_MAXD;                // [32] block reduction scratch
  float* traj = red + 32;                                  // [n_steps][d] stored iterates (ITD-RMAD), 16-byte aligned
  traj += (4 - ((traj - sm) & 3)) & 3;
  float *w = vec, *lam = vec + SM_MAXD, *g = vec + 2 * SM_MAXD, *v = vec + 3 * SM_MAXD, *q = vec + 4 * SM_MAXD,
        *r = vec + 5 * SM_MAXD, *p = vec + 6 * SM_MAXD, *h = vec + 7 * SM_MAXD, *t = vec + 8 * SM_MAXD;

  // resident rows of this CTA
  const int64_t r0 = (int64_t)rank * R, r0v = (int64_t)rank * Rv;
  int rows = (int)(a.n - r0 < R ? a.n - r0 : R); if (rows < 0) rows = 0;
  int rowsv = (int)(a.nv - r0v < Rv ? a.nv - r0v : Rv); if (rowsv < 0) rowsv = 0;
  // register form: thread tid owns columns [8 c8, 8 c8 + 8) of row tid / (d / 8) of each matrix
  const bool regs = a.in_regs != 0;
  float x8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, xv8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  float yreg = 0.f, yvreg = 0.f, curvreg = 0.f;
  bool has = false, hasv = false;
  if (regs) {
    const int tpr = d >> 3, row = tid / tpr, c8 = tid & (tpr - 1);
    has = row < rows; hasv = a.mode != 0 && row < rowsv;
    if (has) {
      const float4 lo = *(const float4*)(a.X + (r0 + row) * d + 8 * c8), hi = *(const float4*)(a.X + (r0 + row) * d + 8 * c8 + 4);
      x8[0] = lo.x; x8[1] = lo.y; x8[2] = lo.z; x8[3] = lo.w; x8[4] = hi.x; x8[5] = hi.y; x8[6] = hi.z; x8[7] = hi.w;
      yreg = a.y[r0 + row];
    }
    if (hasv) {
      const float4 lo = *(const float4*)(a.Xv + (r0v + row) * d + 8 * c8), hi = *(const float4*)(a.Xv + (r0v + row) * d + 8 * c8 + 4);
      xv8[0] = lo.x; xv8[1] = lo.y; xv8[2] = lo.z; xv8[3] = lo.w; xv8[4] = hi.x; xv8[5] = hi.y; xv8[6] = hi.z; xv8[7] = hi.w;
      yvreg = a.yv[r0v + row];
    }
  } else {
    for (int64_t i = tid; i < (int64_t)rows * d; i += SM_T) Xs[i] = a.X[r0 * d + i];
    for (int i = tid; i < rows; i += SM_T) ys[i] = a.y[r0 + i];
    if (a.mode != 0) {
      for (int64_t i = tid; i < (int64_t)rowsv * d; i += SM_T) Xvs[i] = a.Xv[r0v * d + i];
      for (int i = tid; i < rowsv; i += SM_T) yvs[i] = a.yv[r0v + i];
    }
  }
  for (int j = tid; j < d; j += SM_T) { w[j] = a.w[j]; lam[j] = a.lam[j]; }
  __shared__ __align__(8) uint64_t xbar[2];   // one per half of cpart: counts the bytes of column sums that have landed
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(&xbar[0])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(&xbar[1])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster_barrier();    // every CTA of the cluster is running, its barriers set up, before anyone sends to it
  const float inv_n = a.n > 0 ? 1.f / (float)a.n : 0.f, inv_nv = a.nv > 0 ? 1.f / (float)a.nv : 0.f;
  int pb = 0;   // which half of cpart this pass writes
  // one pass over the training rows (kind 0: gradient at vv; kind 1: curvature-weighted product with vv)
  // or over the validation rows (gradient of the upper loss at vv)
  uint32_t ph = 0;   // bit b: parity of the phase half b waits for next
  bool alive = true; // false once a wait for the neighbours ran out: the loops stop and the status is recorded
  // `post(j, sum)` receives column j's sum in the thread that owns index j of every vector until the pass's last barrier
  auto train_pass = [&](int kind, const float* vv, const float* wt, auto post) {
    float* cp = cpart + pb * SM_CL * SM_MAXD;
    const uint32_t par = (ph >> pb) & 1u;
    bool ok;
    if (regs) ok = pass_reg_any(d >> 3, x8, kind == 0 ? yreg : curvreg, has, a.family, inv_n, kind, vv, wt, part, cp, &xbar[pb], par, post, rank);
    else ok = pass(Xs, ys, curv, rows, d, a.family, inv_n, kind, kind == 2 ? wt : vv, vv, coef, part, cp, &xbar[pb], par, post, rank);
    alive = alive && ok; ph ^= 1u << pb; pb ^= 1;
  };
  auto valid_pass = [&](const float* vv, float* res) {
    float* cp = cpart + pb * SM_CL * SM_MAXD;
    const uint32_t par = (ph >> pb) & 1u;
    auto post = [res](int j, float sum) { res[j] = sum; };
    bool ok;
    if (regs) ok = pass_reg_any(d >> 3, xv8, yvreg, hasv, a.family_up, inv_nv, 0, vv, nullptr, part, cp, &xbar[pb], par, post, rank);
    else ok = pass(Xvs, yvs, nullptr, rowsv, d, a.family_up, inv_nv, 0, vv, nullptr, coef, part, cp, &xbar[pb], par, post, rank);
    alive = alive && ok; ph ^= 1u << pb; pb ^= 1;
  };

  if (a.mode == 0) {
    const float lr = a.lr;
    for (int s = 0; s < a.n_steps && alive; ++s)
      train_pass(0, w, nullptr, [=](int j, float gsum) { w[j] -= lr * (gsum + lam[j] * w[j]); });
    if (rank == 0)
      for (int j = tid; j < d; j += SM_T) a.w[j] = w[j];
  } else if (a.mode == 2) {
    // ITD-RMAD (Sec. 3.2, iterative differentiation): the unrolled steps with every iterate kept on chip,
    // then the reverse sweep  out <- out - lr w_t .* a,  a <- a - lr (H(w_t) a + lam .* a)  for t = T-1 ... 0,
    // one pass per reverse step (both row dot products, x.w_t for the curvature and x.a, in the same pass)
    const float lr = a.lr;
    for (int s = 0; s < a.n_steps && alive; ++s) {
      float* ws = traj + (size_t)s * d;
      train_pass(0, w, nullptr, [=](int j, float gsum) { const float wj = w[j]; ws[j] = wj; w[j] = wj - lr * (gsum + lam[j] * wj); });
    }
    valid_pass(w, v);                                  // a = dC_upper/dw at w_T
    for (int j = tid; j < d; j += SM_T) q[j] = 0.f;    // the upper cost has no direct dependence on lam
    __syncthreads();
    for (int s = a.n_steps - 1; s >= 0 && alive; --s) {
      const float* wt = traj + (size_t)s * d;
      train_pass(2, v, wt, [=](int j, float hsum) {
        const float aj = v[j];
        q[j] -= lr * (wt[j] * aj);
        v[j] = aj - lr * (hsum + lam[j] * aj);
      });
    }
    if (rank == 0)
      for (int j = tid; j < d; j += SM_T) { a.out[j] = q[j]; a.w[j] = w[j]; }
  } else {
    // v = dC_upper/dw on the validation rows
    valid_pass(w, v);
    if (a.method == BETTY_FD) {
      // dC/d(lambda) = 1/2 w^2: the central difference at w +- eps v, evaluated as written
      const float nv2 = vdot(v, v, d, red);
      for (int j = tid; j < d; j += SM_T) {
        float o = 0.f;
        if (nv2 > 0.f) {
          const double eps = (double)a.eps0 / sqrt((double)nv2);
          const double wp = (double)w[j] + eps * (double)v[j], wm = (double)w[j] - eps * (double)v[j];
          o = (float)(-(double)a.alpha * (0.5 * wp * wp - 0.5 * wm * wm) / (2.0 * eps));
        }
        if (rank == 0) a.out[j] = o;
      }
    } else {
      // curvature weights at the current w (constant over the solve)
      if (regs) {
        const int tpr = d >> 3, c8 = tid & (tpr - 1);
        const float4 w0 = *(const float4*)(w + 8 * c8), w1 = *(const float4*)(w + 8 * c8 + 4);
        float s = x8[0] * w0.x + x8[1] * w0.y + x8[2] * w0.z + x8[3] * w0.w + x8[4] * w1.x + x8[5] * w1.y + x8[6] * w1.z + x8[7] * w1.w;
        for (int o = tpr >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float sg = sigm(s);
        curvreg = a.family == 0 ? sg * (1.f - sg) * inv_n : 1.f;
      } else {
        for (int i = tid >> 5; i < rows; i += SM_T / 32) {
          const float* xr = Xs + (size_t)i * d;
          float s = 0.f;
          for (int j = tid & 31; j < d; j += 32) s += xr[j] * w[j];
  #pragma unroll
          for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          if ((tid & 31) == 0) { const float sg = sigm(s); curv[i] = a.family == 0 ? sg * (1.f - sg) * inv_n : 1.f; }
        }
      }
      __syncthreads();
      float qscale = 1.f;
      if (a.method == BETTY_NEUMANN) {
        for (int j = tid; j < d; j += SM_T) { t[j] = v[j]; q[j] = v[j]; }
        __syncthreads();
        for (int k = 0; k < a.K && alive; ++k) {
          const float alpha = a.alpha;
          train_pass(1, t, nullptr, [=](int j, float hsum) {
            const float tn = t[j] - alpha * (hsum + lam[j] * t[j]);
            t[j] = tn; q[j] += tn;
          });
        }
        qscale = a.alpha;
      } else {
        // conjugate gradient on H q = v, same recurrences and stopping rules as the large-problem path
        for (int j = tid; j < d; j += SM_T) { q[j] = 0.f; r[j] = v[j]; p[j] = v[j]; }
        __syncthreads();
        float rho = vdot(r, r, d, red);
        const float stop = a.tol * a.tol * rho;
        int iters = 0, status = 0;
        bool active = rho > stop;
        if (!isfinite(rho)) { status = BETTY_ERR_NONFINITE; active = false; }
        for (int k = 0; k < a.K && active; ++k) {
          train_pass(1, p, nullptr, [=](int j, float hsum) { h[j] = hsum + lam[j] * p[j]; });
          if (!alive) break;
          const float gamma = vdot(p, h, d, red);
          if (!isfinite(gamma)) { status = BETTY_ERR_NONFINITE; break; }
          if (!(gamma > 0.f)) { status = BETTY_ERR_BREAKDOWN; break; }
          const float al = rho / gamma;
          float rr = 0.f;
          if (tid < d) {
            q[tid] += al * p[tid];
            const float rn = r[tid] - al * h[tid];
            r[tid] = rn; rr = rn * rn;
          }
          const float rho_new = vsum(rr, d, red);
          const float beta = rho_new / rho;
          for (int j = tid; j < d; j += SM_T) p[j] = r[j] + beta * p[j];
          __syncthreads();
          rho = rho_new;
          ++iters;
          if (!isfinite(rho)) { status = BETTY_ERR_NONFINITE; break; }
          if (rho <= stop) break;
        }
        if (rank == 0 && tid == 0) {
          a.sb->cg_iters = iters;
          if (status) record_status(a.sb, status);
        }
      }
      // out = -(w .* q) * qscale   (mixed second derivative of the weight-decay term)
      if (rank == 0)
        for (int j = tid; j < d; j += SM_T) a.out[j] = -qscale * w[j] * q[j];
    }
  }
  if (!alive && tid == 0) record_status(a.sb, BETTY_ERR_TIMEOUT);
  // no CTA may leave while a neighbour can still send to it
  cluster_barrier();
}

// The unrolled lower steps alone, rows in registers with CPT = 16, 32 or 64 columns per thread: TPR = d / CPT
// threads per row on 8192 / CPT threads (the 1024 x 64 problem: one thread per row, 128 threads per CTA).
// Against the 1024-thread, 8-column form above this leaves 4, 2 or 1 warps per scheduler instead of 8 and
// 60% to half of the warp instructions per pass, which is what a pass is bound by (1.235 -> 0.943 -> 0.785 ->
// 0.749 us per pass on that problem); the other modes keep the 8-column form (they hold the validation rows
// as well).  The block must have at least d threads: the fold and the gather take one column per thread.
template <int TPR, int CPT>
__global__ void __cluster_dims__(SM_CL, 1, 1) __launch_bounds__(8192 / CPT, 1) k_logreg_small_steps(SmallArgs a) {
  constexpr int SW_T = 8192 / CPT;   // 512 threads at 16 columns per thread, 256 at 32
  __shared__ __align__(16) float w[SM_MAXD];
  __shared__ __align__(16) float lam[SM_MAXD];
  __shared__ __align__(16) float part[(SW_T / 32) * SM_PS];
  __shared__ float cpart[2 * SM_CL * SM_MAXD];
  __shared__ __align__(8) uint64_t xbar[2];
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  constexpr int d = CPT * TPR;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int R = a.rows_per_cta, row = tid / TPR, c16 = tid & (TPR - 1);
  const int64_t r0 = (int64_t)rank * R;
  int rows = (int)(a.n - r0 < R ? a.n - r0 : R); if (rows < 0) rows = 0;
  const bool has = row < rows;
  float x[CPT];
#pragma unroll
  for (int k = 0; k < CPT; ++k) x[k] = 0.f;
  float yv = 0.f;
  if (has) {
    const float4* src = (const float4*)(a.X + (r0 + row) * d + CPT * c16);
#pragma unroll
    for (int k = 0; k < CPT / 4; ++k) { const float4 t = src[k]; x[4 * k] = t.x; x[4 * k + 1] = t.y; x[4 * k + 2] = t.z; x[4 * k + 3] = t.w; }
    yv = a.y[r0 + row];
  }
  for (int j = tid; j < d; j += SW_T) { w[j] = a.w[j]; lam[j] = a.lam[j]; }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(&xbar[0])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(&xbar[1])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster_barrier();    // every CTA of the cluster is running, its barriers set up, before anyone sends to it
  const float inv_n = a.n > 0 ? 1.f / (float)a.n : 0.f, lr = a.lr;
  const int family = a.family;
  float* wp = w; float* lp = lam;
  int pb = 0; uint32_t ph = 0; bool alive = true;
  for (int s = 0; s < a.n_steps && alive; ++s) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int k = 0; k < CPT / 4; ++k) {
      const float4 v = *(const float4*)(w + CPT * c16 + 4 * k);
      s0 += x[4 * k] * v.x + x[4 * k + 1] * v.y;
      s1 += x[4 * k + 2] * v.z + x[4 * k + 3] * v.w;
    }
    float sdot = s0 + s1;
#pragma unroll
    for (int o = TPR >> 1; o > 0; o >>= 1) sdot += __shfl_xor_sync(0xffffffffu, sdot, o);
    float cf = 0.f;
    if (has) cf = family == 0 ? -yv * sigm(-yv * sdot) * inv_n : (sdot - yv);
    float col[CPT];
#pragma unroll
    for (int k = 0; k < CPT; ++k) col[k] = cf * x[k];
    int off = 0;
    bool writer = true;
    WarpColumnSum<TPR, CPT, CPT>::run(col, lane, off, writer);
    constexpr int NF = CPT / (32 / TPR) > 0 ? CPT / (32 / TPR) : 1;
    if (writer) {
#pragma unroll
      for (int i = 0; i < NF; ++i) part[warp * SM_PS + CPT * c16 + off + i] = col[i];
    }
    __syncthreads();
    const bool ok = exchange_cols(part, SW_T / 32, d, cpart + pb * SM_CL * SM_MAXD, &xbar[pb], (ph >> pb) & 1u,
                                  [=](int j, float gsum) { wp[j] -= lr * (gsum + lp[j] * wp[j]); }, rank);
    alive = alive && ok; ph ^= 1u << pb; pb ^= 1;
  }
  if (rank == 0)
    for (int j = tid; j < d; j += SW_T) a.w[j] = w[j];
  if (!alive && tid == 0) record_status(a.sb, BETTY_ERR_TIMEOUT);
  cluster_barrier();    // no CTA may leave while a neighbour can still send to it
}

// The hypergradient (mode 1) and ITD-RMAD (mode 2) loops in the same wide-row form: CPT columns of a row per
// thread on 8192 / CPT threads.  One register array serves both matrices: it holds the training rows during
// the training passes and is refilled from global memory (256 KB at most, L2-resident) around the single pass
// over the validation rows, so a thread never keeps two row slices alive.  Same passes, same exchange, same
// solver arithmetic in the same order as k_logreg_small; only the number of threads that share a row differs.
template <int TPR, int CPT, class Post>
__device__ __forceinline__ bool wide_pass(const float (&x)[CPT], float yv, bool has, int family, float inv_n, int kind,
                                          const float* vv, const float* wt, float* part, float* cpart, uint64_t* bar,
                                          uint32_t parity, Post post, uint32_t rank) {
  constexpr int SW_T = 8192 / CPT, d = CPT * TPR;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cb = CPT * (tid & (TPR - 1));
  float s0 = 0.f, s1 = 0.f, z0 = 0.f, z1 = 0.f;
#pragma unroll
  for (int k = 0; k < CPT / 4; ++k) {
    const float4 v = *(const float4*)(vv + cb + 4 * k);
    s0 += x[4 * k] * v.x + x[4 * k + 1] * v.y;
    s1 += x[4 * k + 2] * v.z + x[4 * k + 3] * v.w;
    if (kind == 2) {
      const float4 u = *(const float4*)(wt + cb + 4 * k);
      z0 += x[4 * k] * u.x + x[4 * k + 1] * u.y;
      z1 += x[4 * k + 2] * u.z + x[4 * k + 3] * u.w;
    }
  }
  float sdot = s0 + s1, zdot = z0 + z1;
#pragma unroll
  for (int o = TPR >> 1; o > 0; o >>= 1) {
    sdot += __shfl_xor_sync(0xffffffffu, sdot, o);
    if (kind == 2) zdot += __shfl_xor_sync(0xffffffffu, zdot, o);
  }
  float cf = 0.f;
  if (has) {
    if (kind == 0) cf = family == 0 ? -yv * sigm(-yv * sdot) * inv_n : (sdot - yv);
    else if (kind == 1) cf = yv * sdot;
    else { const float sg = sigm(zdot); cf = (family == 0 ? sg * (1.f - sg) * inv_n : 1.f) * sdot; }
  }
  float col[CPT];
#pragma unroll
  for (int k = 0; k < CPT; ++k) col[k] = cf * x[k];
  int off = 0;
  bool writer = true;
  WarpColumnSum<TPR, CPT, CPT>::run(col, lane, off, writer);
  constexpr int NF = CPT / (32 / TPR) > 0 ? CPT / (32 / TPR) : 1;
  if (writer) {
#pragma unroll
    for (int i = 0; i < NF; ++i) part[warp * SM_PS + cb + off + i] = col[i];
  }
  __syncthreads();
  return exchange_cols(part, SW_T / 32, d, cpart, bar, parity, post, rank);
}

template <int TPR, int CPT>
__global__ void __cluster_dims__(SM_CL, 1, 1) __launch_bounds__(8192 / CPT, 1) k_logreg_small_wide(SmallArgs a) {
  constexpr int SW_T = 8192 / CPT, d = CPT * TPR;
  __shared__ __align__(16) float vec[SM_NVEC * SM_MAXD];
  __shared__ __align__(16) float part[(SW_T / 32) * SM_PS];
  __shared__ float cpart[2 * SM_CL * SM_MAXD];
  __shared__ float red[32];
  __shared__ __align__(8) uint64_t xbar[2];
  extern __shared__ __align__(16) float traj[];     // [n_steps][d] stored iterates (ITD-RMAD)
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int tid = threadIdx.x;
  float *w = vec, *lam = vec + SM_MAXD, *v = vec + 3 * SM_MAXD, *q = vec + 4 * SM_MAXD, *r = vec + 5 * SM_MAXD,
        *p = vec + 6 * SM_MAXD, *h = vec + 7 * SM_MAXD, *t = vec + 8 * SM_MAXD;
  const int R = a.rows_per_cta, Rv = a.rows_per_cta_v, row = tid / TPR, cb = CPT * (tid & (TPR - 1));
  const int64_t r0 = (int64_t)rank * R, r0v = (int64_t)rank * Rv;
  int rows = (int)(a.n - r0 < R ? a.n - r0 : R); if (rows < 0) rows = 0;
  int rowsv = (int)(a.nv - r0v < Rv ? a.nv - r0v : Rv); if (rowsv < 0) rowsv = 0;
  const bool has = row < rows, hasv = row < rowsv;
  float x[CPT];
  float yreg = 0.f, curvreg = 0.f;
  // this thread's CPT columns of its row of the training (which = 0) or validation (which = 1) matrix
  auto load_row = [&](int which) {
    const bool present = which == 0 ? has : hasv;
#pragma unroll
    for (int k = 0; k < CPT; ++k) x[k] = 0.f;
    yreg = 0.f;
    if (present) {
      const float* base = which == 0 ? a.X + (r0 + row) * d : a.Xv + (r0v + row) * d;
      const float4* src = (const float4*)(base + cb);
#pragma unroll
      for (int k = 0; k < CPT / 4; ++k) { const float4 u = src[k]; x[4 * k] = u.x; x[4 * k + 1] = u.y; x[4 * k + 2] = u.z; x[4 * k + 3] = u.w; }
      yreg = which == 0 ? a.y[r0 + row] : a.yv[r0v + row];
    }
  };
  for (int j = tid; j < d; j += SW_T) { w[j] = a.w[j]; lam[j] = a.lam[j]; }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(&xbar[0])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(&xbar[1])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster_barrier();    // every CTA of the cluster is running, its barriers set up, before anyone sends to it
  const float inv_n = a.n > 0 ? 1.f / (float)a.n : 0.f, inv_nv = a.nv > 0 ? 1.f / (float)a.nv : 0.f;
  int pb = 0; uint32_t ph = 0; bool alive = true;
  auto train_pass = [&](int kind, const float* vv, const float* wt, auto post) {
    const bool ok = wide_pass<TPR, CPT>(x, kind == 0 ? yreg : curvreg, has, a.family, inv_n, kind, vv, wt, part,
                                        cpart + pb * SM_CL * SM_MAXD, &xbar[pb], (ph >> pb) & 1u, post, rank);
    alive = alive && ok; ph ^= 1u << pb; pb ^= 1;
  };
  // gradient of the upper cost at vv over the validation rows: the row registers are lent to them for one pass
  auto valid_pass = [&](const float* vv, float* res) {
    load_row(1);
    const bool ok = wide_pass<TPR, CPT>(x, yreg, hasv, a.family_up, inv_nv, 0, vv, nullptr, part,
                                        cpart + pb * SM_CL * SM_MAXD, &xbar[pb], (ph >> pb) & 1u,
                                        [res](int j, float sum) { res[j] = sum; }, rank);
    alive = alive && ok; ph ^= 1u << pb; pb ^= 1;
    load_row(0);
  };

  if (a.mode == 2) {
    // ITD-RMAD: unrolled steps with every iterate kept on chip, then the reverse sweep (see k_logreg_small)
    const float lr = a.lr;
    load_row(0);
    for (int s = 0; s < a.n_steps && alive; ++s) {
      float* ws = traj + (size_t)s * d;
      train_pass(0, w, nullptr, [=](int j, float gsum) { const float wj = w[j]; ws[j] = wj; w[j] = wj - lr * (gsum + lam[j] * wj); });
    }
    valid_pass(w, v);
    for (int j = tid; j < d; j += SW_T) q[j] = 0.f;
    __syncthreads();
    for (int s = a.n_steps - 1; s >= 0 && alive; --s) {
      const float* wt = traj + (size_t)s * d;
      train_pass(2, v, wt, [=](int j, float hsum) {
        const float aj = v[j];
        q[j] -= lr * (wt[j] * aj);
        v[j] = aj - lr * (hsum + lam[j] * aj);
      });
    }
    if (rank == 0)
      for (int j = tid; j < d; j += SW_T) { a.out[j] = q[j]; a.w[j] = w[j]; }
  } else {
    valid_pass(w, v);          // leaves the training rows in the registers
    if (a.method == BETTY_FD) {
      const float nv2 = vdot(v, v, d, red);
      for (int j = tid; j < d; j += SW_T) {
        float o = 0.f;
        if (nv2 > 0.f) {
          const double eps = (double)a.eps0 / sqrt((double)nv2);
          const double wp = (double)w[j] + eps * (double)v[j], wm = (double)w[j] - eps * (double)v[j];
          o = (float)(-(double)a.alpha * (0.5 * wp * wp - 0.5 * wm * wm) / (2.0 * eps));
        }
        if (rank == 0) a.out[j] = o;
      }
    } else {
      {   // curvature weight of this thread's row at the current w (constant over the solve)
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < CPT / 4; ++k) {
          const float4 u = *(const float4*)(w + cb + 4 * k);
          s += x[4 * k] * u.x + x[4 * k + 1] * u.y + x[4 * k + 2] * u.z + x[4 * k + 3] * u.w;
        }
#pragma unroll
        for (int o = TPR >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float sg = sigm(s);
        curvreg = a.family == 0 ? sg * (1.f - sg) * inv_n : 1.f;
      }
      float qscale = 1.f;
      if (a.method == BETTY_NEUMANN) {
        for (int j = tid; j < d; j += SW_T) { t[j] = v[j]; q[j] = v[j]; }
        __syncthreads();
        for (int k = 0; k < a.K && alive; ++k) {
          const float alpha = a.alpha;
          train_pass(1, t, nullptr, [=](int j, float hsum) {
            const float tn = t[j] - alpha * (hsum + lam[j] * t[j]);
            t[j] = tn; q[j] += tn;
          });
        }
        qscale = a.alpha;
      } else {
        for (int j = tid; j < d; j += SW_T) { q[j] = 0.f; r[j] = v[j]; p[j] = v[j]; }
        __syncthreads();
        float rho = vdot(r, r, d, red);
        const float stop = a.tol * a.tol * rho;
        int iters = 0, status = 0;
        bool active = rho > stop;
        if (!isfinite(rho)) { status = BETTY_ERR_NONFINITE; active = false; }
        for (int k = 0; k < a.K && active; ++k) {
          train_pass(1, p, nullptr, [=](int j, float hsum) { h[j] = hsum + lam[j] * p[j]; });
          if (!alive) break;
          const float gamma = vdot(p, h, d, red);
          if (!isfinite(gamma)) { status = BETTY_ERR_NONFINITE; break; }
          if (!(gamma > 0.f)) { status = BETTY_ERR_BREAKDOWN; break; }
          const float al = rho / gamma;
          float rr = 0.f;
          if (tid < d) {
            q[tid] += al * p[tid];
            const float rn = r[tid] - al * h[tid];
            r[tid] = rn; rr = rn * rn;
          }
          const float rho_new = vsum(rr, d, red);
          const float beta = rho_new / rho;
          for (int j = tid; j < d; j += SW_T) p[j] = r[j] + beta * p[j];
          __syncthreads();
          rho = rho_new;
          ++iters;
          if (!isfinite(rho)) { status = BETTY_ERR_NONFINITE; break; }
          if (rho <= stop) break;
        }
        if (rank == 0 && tid == 0) {
          a.sb->cg_iters = iters;
          if (status) record_status(a.sb, status);
        }
      }
      if (rank == 0)
        for (int j = tid; j < d; j += SW_T) a.out[j] = -qscale * w[j] * q[j];
    }
  }
  if (!alive && tid == 0) record_status(a.sb, BETTY_ERR_TIMEOUT);
  cluster_barrier();    // no CTA may leave while a neighbour can still send to it
}

template <int TPR, int CPT>
static betty_status launch_wide(Ctx& c, const SmallArgs& a, size_t traj_bytes) {
  static SmemLimit limit = {};      // per form and per device
  if (traj_bytes > 0) BETTY_TRY(ensure_dynamic_smem(k_logreg_small_wide<TPR, CPT>, limit, traj_bytes));
  k_logreg_small_wide<TPR, CPT><<<SM_CL, 8192 / CPT, traj_bytes, c.stream>>>(a);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

static size_t small_smem_bytes(int R, int Rv, int d, int64_t traj_floats) {
  size_t floats = (size_t)R * d + (size_t)Rv * d + R + Rv + R + (R > Rv ? R : Rv) + (size_t)SM_NVEC * SM_MAXD + 32 * SM_PS +
                  2 * SM_CL * SM_MAXD + 32 + (size_t)traj_floats;
  return floats * sizeof(float) + 32;
}

// True when the whole problem (and `unrolled_steps` stored iterates, for ITD-RMAD) fits the cluster's shared memory.
bool logreg_small_eligible(int64_t n, int64_t nv, int64_t d, int64_t unrolled_steps) {
  if (d <= 0 || d > SM_MAXD || n <= 0 || n > (1 << 20) || nv < 0 || nv > (1 << 20) || unrolled_steps < 0 || unrolled_steps > (1 << 16))
    return false;
  const int R = (int)((n + SM_CL - 1) / SM_CL), Rv = (int)((nv + SM_CL - 1) / SM_CL);
  return small_smem_bytes(R, Rv, (int)d, unrolled_steps * d) <= 225 * 1024;
}

static betty_status launch_small(Ctx& c, SmallArgs& a) {
  a.rows_per_cta = (int)((a.n + SM_CL - 1) / SM_CL);
  a.rows_per_cta_v = a.mode != 0 ? (int)((a.nv + SM_CL - 1) / SM_CL) : 0;
  a.sb = c.arena.status();
  {
    const int d = a.d, tpr = d >> 3;
    const bool pow2 = d >= 8 && d <= SM_MAXD && (d & (d - 1)) == 0;
    a.in_regs = pow2 && a.rows_per_cta <= SM_T / tpr && a.rows_per_cta_v <= SM_T / tpr &&
                (reinterpret_cast<uintptr_t>(a.X) & 15) == 0 && (a.mode == 0 || (reinterpret_cast<uintptr_t>(a.Xv) & 15) == 0);
  }
  if (a.mode == 0 && a.in_regs && a.d >= 16) {
    // the widest form whose threads still cover the d columns in the fold and the gather (in_regs: at most
    // 8192 / d rows per CTA, which is the row capacity of every form)
    switch (a.d) {
      case 16: k_logreg_small_steps<1, 16><<<SM_CL, 512, 0, c.stream>>>(a); break;
      case 32: k_logreg_small_steps<1, 32><<<SM_CL, 256, 0, c.stream>>>(a); break;
      case 64: k_logreg_small_steps<1, 64><<<SM_CL, 128, 0, c.stream>>>(a); break;
      case 128: k_logreg_small_steps<2, 64><<<SM_CL, 128, 0, c.stream>>>(a); break;
      default: k_logreg_small_steps<8, 32><<<SM_CL, 256, 0, c.stream>>>(a); break;   // d = 256
    }
    BETTY_LAUNCH_CHECK();
    return BETTY_OK;
  }
  // hypergradient and ITD-RMAD modes: the wide-row form under the same conditions (power-of-two width of at
  // least 16, at most 8192 / d rows of either matrix per CTA), as long as the stored iterates fit beside its
  // 43 KB of static shared memory
  const size_t traj_bytes = a.mode == 2 ? (size_t)a.n_steps * a.d * sizeof(float) : 0;
  if (a.mode != 0 && a.in_regs && a.d >= 16 && traj_bytes <= 160 * 1024) {
    switch (a.d) {
      case 16: return launch_wide<1, 16>(c, a, traj_bytes);
      case 32: return launch_wide<1, 32>(c, a, traj_bytes);
      case 64: return launch_wide<1, 64>(c, a, traj_bytes);
      case 128: return launch_wide<2, 64>(c, a, traj_bytes);
      default: return launch_wide<8, 32>(c, a, traj_bytes);   // d = 256
    }
  }
  const size_t smem = small_smem_bytes(a.rows_per_cta, a.rows_per_cta_v, a.d, a.mode == 2 ? (int64_t)a.n_steps * a.d : 0);
  static SmemLimit limit = {};      // per device
  BETTY_TRY(ensure_dynamic_smem(k_logreg_small, limit, smem));
  k_logreg_small<<<SM_CL, SM_T, smem, c.stream>>>(a);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

betty_status logreg_small_lower_step(Ctx& c, int family, const float* X, const float* y, int64_t n, int64_t d, float* w,
                                     const float* lam, int n_steps, float lr) {
  SmallArgs a = {};
  a.X = X; a.y = y; a.n = n; a.d = (int)d; a.family = family; a.w = w; a.lam = lam; a.mode = 0; a.n_steps = n_steps; a.lr = lr;
  return launch_small(c, a);
}

betty_status logreg_small_hypergrad(Ctx& c, int family, const float* X, const float* y, int64_t n, int family_up,
                                    const float* Xv, const float* yv, int64_t nv, int64_t d, float* w, const float* lam,
                                    const betty_method_cfg& cfg, float* out) {
  SmallArgs a = {};
  a.X = X; a.y = y; a.n = n; a.Xv = Xv; a.yv = yv; a.nv = nv; a.d = (int)d; a.family = family; a.family_up = family_up;
  a.w = w; a.lam = lam; a.mode = 1; a.method = cfg.method; a.K = cfg.K; a.alpha = cfg.alpha; a.eps0 = cfg.eps0; a.tol = cfg.tol;
  a.out = out;
  return launch_small(c, a);
}

betty_status logreg_small_itd(Ctx& c, int family, const float* X, const float* y, int64_t n, int family_up, const float* Xv,
                              const float* yv, int64_t nv, int64_t d, float* w, const float* lam, int n_steps, float lr,
                              float* out) {
  SmallArgs a = {};
  a.X = X; a.y = y; a.n = n; a.Xv = Xv; a.yv = yv; a.nv = nv; a.d = (int)d; a.family = family; a.family_up = family_up;
  a.w = w; a.lam = lam; a.mode = 2; a.n_steps = n_steps; a.lr = lr; a.out = out;
  return launch_small(c, a);
}

}  // namespace betty
