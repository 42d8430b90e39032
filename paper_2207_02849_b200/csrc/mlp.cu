// MLP cost families: the reweighted cross-entropy classifier of the data-reweighting experiment
// (App. A listing), its plain cross-entropy upper cost, and the clean-label detector cost of the
// three-level configuration.  Gradients are hand-written reverse sweeps; Hessian-vector products
// are R-operator (forward-over-reverse) passes that reuse a cached base forward/backward pass;
// mixed second derivatives are a directional forward pass followed by the weight net's reverse
// sweep.  Matrices are op16 (rounded copies of the fp32 master), accumulation is fp32.
#include "ops.cuh"
#include "gemm.cuh"

namespace betty {
namespace BETTY_FAM {

static constexpr int MAXL = 16;
// Reverse sweeps of nets with fewer layers stay on one stream: with a single chain product there is nothing to run
// the weight products beside, and a join across streams costs more than a programmatic edge (two-layer
// classifier, batch 512: 0.685 ms per Neumann step with the fork, 0.660 without).
static constexpr int SIDE_MIN_LAYERS = 3;
static constexpr int WN_H = 100;
static constexpr int WN_P = 3 * WN_H + 1;

static inline int64_t ld8(int64_t n) { return (n + 7) & ~int64_t(7); }
static inline int grid_for(int64_t n, int per_block = 256) {
  int64_t b = (n + per_block - 1) / per_block;
  return (int)(b < 1 ? 1 : (b > 148 * 32 ? 148 * 32 : b));
}

// ------------------------------------------------------------------ helpers
__device__ __forceinline__ float fd_eps(const float* vnorm2, float eps0) {
  const float nv2 = *vnorm2;
  return nv2 > 0.f ? eps0 / sqrtf(nv2) : 0.f;
}

// ------------------------------------------------------------------ elementwise / row kernels
// dst[r, c] = op16(scale * src[r, c]); scale = eps0/|v| when vnorm2 is given, else 1.  Pad columns are zeroed.
__global__ void k_cast_rows(const float* src, op16* dst, int64_t rows, int64_t cols, int64_t ld, const float* vnorm2,
                            float eps0) {
  pdl_enter();
  const float s = vnorm2 ? fd_eps(vnorm2, eps0) : 1.f;
  const int64_t total = rows * ld;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / ld, c = i - r * ld;
    dst[i] = to_op16(c < cols ? s * src[r * cols + c] : 0.f);
  }
}
// a += bias; h = act(a) as op16 (hidden layers)
__global__ void k_bias_act(float* a, const float* bias, op16* h, int64_t rows, int64_t N, int64_t ldh, int act) {
  pdl_enter();
  const int64_t total = rows * N;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / N, n = i - r * N;
    const float v = a[i] + bias[n];
    a[i] = v;
    if (h) h[r * ldh + n] = to_op16(act_f(act, v));
  }
}
// one warp per row: p = softmax(z), ell = -log p[y].  Rows of up to 1024 classes are held in registers
// (32 values per lane, every load issued before the first use); longer rows are read three times.
__global__ void k_softmax_ce(const float* z, const int32_t* y, float* p, float* ell, int64_t B, int64_t C) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  if (row >= B) return;
  const float* zr = z + row * C;
  float mx = -INFINITY, s = 0.f, ls;
  if (C <= 1024) {
    float v[32];
    const int nk = (int)((C + 31) >> 5);      // uniform: rounds of 32 classes this row has
#pragma unroll
    for (int k = 0; k < 32; ++k) { const int64_t c = lane + 32 * k; v[k] = (k < nk && c < C) ? zr[c] : -INFINITY; }
#pragma unroll
    for (int k = 0; k < 32; ++k) if (k < nk) mx = fmaxf(mx, v[k]);
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
#pragma unroll
    for (int k = 0; k < 32; ++k) if (k < nk && lane + 32 * k < C) s += expf(v[k] - mx);     // same order as the loop below
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    ls = logf(s);
#pragma unroll
    for (int k = 0; k < 32; ++k) { const int64_t c = lane + 32 * k; if (k < nk && c < C) p[row * C + c] = expf(v[k] - mx - ls); }
  } else {
    for (int64_t c = lane; c < C; c += 32) mx = fmaxf(mx, zr[c]);
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    for (int64_t c = lane; c < C; c += 32) s += expf(zr[c] - mx);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    ls = logf(s);
    for (int64_t c = lane; c < C; c += 32) p[row * C + c] = expf(zr[c] - mx - ls);
  }
  if (lane == 0) {
    int32_t yy = y[row];
    yy = yy < 0 ? 0 : (yy >= C ? (int32_t)C - 1 : yy);     // class ids are validated on the host side of a dataset; clamp
    ell[row] = -(zr[yy] - mx - ls);
  }
}
// delta = coef_i * (p - onehot(y))
// lscale (nullable): device loss scale multiplied into every delta (betty_level.loss_scale)
__global__ void k_delta_top(const float* p, const int32_t* y, const float* coef, float scale, op16* delta, int64_t B,
                            int64_t C, int64_t ld, const float* lscale) {
  pdl_enter();
  const float S = lscale ? *lscale : 1.f;
  const int64_t total = B * ld;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / ld, c = i - r * ld;
    float v = 0.f;
    if (c < C) v = S * ((coef ? coef[r] : scale) * (p[r * C + c] - (c == y[r] ? 1.f : 0.f)));
    delta[i] = to_op16(v);
  }
}
// Column sums sum_i d[i, n] (bias gradients), with the consumer fused in.  Block = 32 columns (16 lanes x 2
// adjacent columns; ld is even, so a column pair is one 4-byte load) x 64 row groups; a thread's loads are
// issued 16 at a time (the kernel is bound by latency, not by bytes); fixed summation order.
//   mode 0: out[n] = sum            mode 1: out[n] -= step * sum   (gradient step on a bias)
//   mode 2: out[n] = s_in[n] + t_in[n] - step * sum   (one Horner step of the Neumann series; out may alias t_in)
struct ColsumSink { int mode; float step; float* out; const float* t_in; const float* s_in; };
static constexpr int CS_COLS = 32, CS_GROUPS = 64;
__device__ __forceinline__ void colsum_block(const op16* d, int64_t B, int64_t N, int64_t ld, const ColsumSink& k,
                                             int64_t block, float (*sh)[CS_COLS + 1]) {
  const int cx = threadIdx.x & 15, rg = threadIdx.x >> 4;
  const int64_t n = block * CS_COLS + 2 * cx;
  float a0 = 0.f, a1 = 0.f;
  if (n < N) {
    constexpr int U = 16;
    for (int64_t i0 = rg; i0 < B; i0 += CS_GROUPS * U) {
      op16x2 v[U];
#pragma unroll
      for (int k2 = 0; k2 < U; ++k2) {
        const int64_t i = i0 + CS_GROUPS * k2;
        v[k2] = i < B ? *(const op16x2*)(d + i * ld + n) : to_op16x2(0.f, 0.f);
      }
#pragma unroll
      for (int k2 = 0; k2 < U; ++k2) {   // same order as a plain loop over the rows
        const float2 f = from_op16x2(v[k2]);
        a0 += f.x; a1 += f.y;
      }
    }
  }
  sh[rg][2 * cx] = a0; sh[rg][2 * cx + 1] = a1;
  __syncthreads();
  if (threadIdx.x < CS_COLS) {
    const int64_t nn = block * CS_COLS + threadIdx.x;
    if (nn < N) {
      float t = 0.f;
#pragma unroll
      for (int r = 0; r < CS_GROUPS; ++r) t += sh[r][threadIdx.x];
      if (k.mode == 0) k.out[nn] = t;
      else if (k.mode == 1) k.out[nn] -= k.step * t;
      else k.out[nn] = k.s_in[nn] + (k.t_in[nn] - k.step * t);
    }
  }
}
__global__ void __launch_bounds__(1024) k_colsum_bf16(const op16* d, int64_t B, int64_t N, int64_t ld, ColsumSink k) {
  pdl_enter();
  __shared__ float sh[CS_GROUPS][CS_COLS + 1];
  colsum_block(d, B, N, ld, k, blockIdx.x, sh);
}
// The column sums of several layers in one launch (a reverse sweep that runs on one stream takes them together
// after its last product): block b belongs to the job whose block range contains it.
struct ColsumJob { const op16* d; int64_t B, N, ld; ColsumSink k; int first_block; };
struct ColsumJobs { int n; ColsumJob j[MAXL]; };
__global__ void __launch_bounds__(1024) k_colsum_multi(const __grid_constant__ ColsumJobs jobs) {
  pdl_enter();
  __shared__ float sh[CS_GROUPS][CS_COLS + 1];
  int i = jobs.n - 1;
  while (i > 0 && (int)blockIdx.x < jobs.j[i].first_block) --i;
  const ColsumJob& job = jobs.j[i];
  colsum_block(job.d, job.B, job.N, job.ld, job.k, (int64_t)blockIdx.x - job.first_block, sh);
}
// collects a sweep's column sums; launch() takes them all in one kernel
struct ColsumBatch {
  ColsumJobs jobs; int blocks;
  ColsumBatch() : blocks(0) { jobs.n = 0; }
  void add(const op16* d, int64_t B, int64_t N, int64_t ld, const ColsumSink& k) {
    ColsumJob& j = jobs.j[jobs.n++];
    j.d = d; j.B = B; j.N = N; j.ld = ld; j.k = k; j.first_block = blocks;
    blocks += (int)((N + CS_COLS - 1) / CS_COLS);
  }
  betty_status launch(Ctx& c) {
    if (jobs.n == 0) return BETTY_OK;
    launch_pdl(k_colsum_multi, dim3((unsigned)blocks), dim3(1024), 0, c.stream, jobs);
    BETTY_LAUNCH_CHECK();
    return BETTY_OK;
  }
};
// delta_prev = dh * act'(a)
__global__ void k_act_backward(const float* dh, const float* a, op16* dprev, int64_t B, int64_t N, int64_t ld, int act) {
  pdl_enter();
  const int64_t total = B * ld;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / ld, n = i - r * ld;
    dprev[i] = to_op16(n < N ? dh[r * N + n] * act_d1(act, a[r * N + n]) : 0.f);
  }
}
// Ra += c ; Rh = act'(a) * Ra
__global__ void k_r_act_forward(float* Ra, const float* cdir, const float* a, op16* Rh, int64_t B, int64_t N,
                                int64_t ldh, int act) {
  pdl_enter();
  const int64_t total = B * N;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / N, n = i - r * N;
    const float v = Ra[i] + cdir[n];
    Ra[i] = v;
    if (Rh) Rh[r * ldh + n] = to_op16(act_d1(act, a[i]) * v);
  }
}
// one warp per row: Rdelta = coef_i * (p.*Ra - p * (p . Ra))
__global__ void k_r_delta_top(const float* p, const float* Ra, const float* coef, float scale, op16* Rd, int64_t B,
                              int64_t C, int64_t ld) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  if (row >= B) return;
  float s = 0.f;
  for (int64_t c = lane; c < C; c += 32) s += p[row * C + c] * Ra[row * C + c];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float k = coef ? coef[row] : scale;
  for (int64_t c = lane; c < ld; c += 32) {
    float v = 0.f;
    if (c < C) { const float pc = p[row * C + c]; v = k * (pc * Ra[row * C + c] - pc * s); }
    Rd[row * ld + c] = to_op16(v);
  }
}
// Rdelta_prev = Rdh * act'(a) + dh * act''(a) * Ra
__global__ void k_r_act_backward(const float* Rdh, const float* dh, const float* a, const float* Ra, op16* Rdprev,
                                 int64_t B, int64_t N, int64_t ld, int act) {
  pdl_enter();
  const int64_t total = B * ld;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / ld, n = i - r * ld;
    float v = 0.f;
    if (n < N) {
      const int64_t j = r * N + n;
      v = Rdh[j] * act_d1(act, a[j]);
      if (act != BETTY_ACT_RELU) v += dh[j] * act_d2(act, a[j]) * Ra[j];
    }
    Rdprev[i] = to_op16(v);
  }
}
// one warp per row: d_i = sum_c (p - onehot) * Ra
__global__ void k_jvp_rows(const float* p, const int32_t* y, const float* Ra, float* d, int64_t B, int64_t C) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  if (row >= B) return;
  float s = 0.f;
  for (int64_t c = lane; c < C; c += 32) s += (p[row * C + c] - (c == y[row] ? 1.f : 0.f)) * Ra[row * C + c];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) d[row] = s;
}
// out[r, c] += exp(lam) * W[r, c]   (out contiguous [rows, cols]; W op16 with leading dimension ldw)
__global__ void k_wd_add_bf16(float* out, const op16* W, int64_t rows, int64_t cols, int64_t ldw, const float* lam,
                              const float* lscale) {
  pdl_enter();
  const float k = expf(*lam) * (lscale ? *lscale : 1.f);     // a scaled gradient takes a scaled decay term
  const int64_t total = rows * cols;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / cols, c = i - r * cols;
    out[i] += k * from_op16(W[r * ldw + c]);
  }
}
__global__ void k_wd_add_f32(float* out, const float* u, int64_t n, const float* lam) {
  pdl_enter();
  const float k = expf(*lam);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] += k * u[i];
}
// out (+)= scale * exp(lam) * <W, q>  (q == nullptr: <W, W>).  Each block sums a slice in fp64; the block
// that draws the last ticket adds the per-block sums in a fixed order (one warp: strided partial sums, then a
// shuffle tree), so the result does not depend on scheduling.
static constexpr int LD_MAX_BLOCKS = 128;
// block `blk` of `nblk` blocks working on one matrix
__device__ __forceinline__ void layer_dot_block(const op16* W, int64_t rows, int64_t cols, int64_t ldw, const float* q, const float* lam,
                                                float scale, float* out, int accumulate, double* partial, unsigned* counter,
                                                unsigned blk, unsigned nblk) {
  __shared__ double sh[32];
  __shared__ bool is_last;
  double acc = 0.0;
  const int64_t total = rows * cols;
  for (int64_t i = blk * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)nblk * blockDim.x) {
    const int64_t r = i / cols, c = i - r * cols;
    const float w = from_op16(W[r * ldw + c]);
    acc += (double)w * (double)(q ? q[i] : w);
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += sh[i];
    partial[blk] = t;
    __threadfence();
    is_last = atomicAdd(counter, 1u) == nblk - 1;
  }
  __syncthreads();
  if (is_last && threadIdx.x < 32) {
    // second phase by one warp: lane l adds blocks l, l+32, ... in order, then a fixed shuffle tree
    __threadfence();
    double tot = 0.0;
    for (unsigned bb = threadIdx.x; bb < nblk; bb += 32) tot += ((volatile double*)partial)[bb];
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
    if (threadIdx.x == 0) {
      const float v = scale * expf(*lam) * (float)tot;
      *out = (accumulate ? *out : 0.f) + v;
      *counter = 0u;
    }
  }
}
// All layers of a net in one launch: block b belongs to the job whose block range contains it; every job has partial
// sums, a ticket counter and an output of its own.
struct LayerDotJob { const op16* W; int64_t rows, cols, ldw; const float* q; const float* lam; float* out; double* partial; unsigned* counter; int first_block, n_blocks; };
struct LayerDotJobs { int n; float scale; int accumulate; LayerDotJob j[MAXL]; };
__global__ void k_layer_dot_multi(const __grid_constant__ LayerDotJobs jobs) {
  pdl_enter();
  int i = jobs.n - 1;
  while (i > 0 && (int)blockIdx.x < jobs.j[i].first_block) --i;
  const LayerDotJob& t = jobs.j[i];
  layer_dot_block(t.W, t.rows, t.cols, t.ldw, t.q, t.lam, jobs.scale, t.out, jobs.accumulate, t.partial, t.counter,
                  blockIdx.x - (unsigned)t.first_block, (unsigned)t.n_blocks);
}
// ------------------------------------------------------------------ weight net 1-100-1
enum WnMode { WN_REWEIGHT_COEF = 0, WN_REWEIGHT_TGRAD, WN_REWEIGHT_TMIXED, WN_DETECT_TGRAD, WN_DETECT_WGRAD,
              WN_DETECT_THVP, WN_DETECT_WMIXED };

// One thread per sample: s = a2 . relu(a1*l + b1) + b2, r = sigmoid(s), and the per-sample scalar the
// caller's reverse sweep needs (see WnMode).  dir: a direction in theta space (modes *_THVP, *_WMIXED).
__global__ void k_wn_sample(int mode, const float* theta, const float* dir, const float* ell, const float* aux,
                            const float* din, int64_t B, float invB, float* out1, float* out2) {
  pdl_enter();
  __shared__ float th[WN_P], dr[WN_P];
  for (int i = threadIdx.x; i < WN_P; i += blockDim.x) { th[i] = theta[i]; dr[i] = dir ? dir[i] : 0.f; }
  __syncthreads();
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= B) return;
  const float l = ell[i];
  float s = th[3 * WN_H], dsdl = 0.f, Jd = dr[3 * WN_H], dJd = 0.f;
  for (int k = 0; k < WN_H; ++k) {
    const float a1 = th[k], b1 = th[WN_H + k], a2 = th[2 * WN_H + k];
    const float pre = a1 * l + b1;
    if (pre > 0.f) {
      s += a2 * pre;
      dsdl += a1 * a2;
      Jd += a2 * l * dr[k] + a2 * dr[WN_H + k] + pre * dr[2 * WN_H + k];
      dJd += a2 * dr[k] + a1 * dr[2 * WN_H + k];
    }
  }
  const float r = 1.f / (1.f + expf(-s));
  const float rp = r * (1.f - r);
  const float c = aux ? aux[i] : 0.f;
  const float fp = 2.f * (r - c) * rp;
  const float fpp = 2.f * rp * rp + 2.f * (r - c) * rp * (1.f - 2.f * r);
  switch (mode) {
    case WN_REWEIGHT_COEF: out1[i] = r * invB; break;
    case WN_REWEIGHT_TGRAD: out1[i] = l * rp * invB; break;
    case WN_REWEIGHT_TMIXED: out1[i] = din[i] * rp * invB; break;
    case WN_DETECT_TGRAD: out1[i] = fp * invB; break;
    case WN_DETECT_WGRAD: out1[i] = fp * dsdl * invB; break;
    case WN_DETECT_THVP: out1[i] = fpp * Jd * invB; out2[i] = fp * invB; break;
    case WN_DETECT_WMIXED: out1[i] = (fpp * dsdl * Jd + fp * dJd) * invB; break;
  }
}
// out = sum_i cA_i * ds_i/dtheta + cB_i * (d2s_i/dtheta2 . dir) + mu*muvec.  Thread k owns hidden unit k;
// block b sums its slice of the samples (fp64), the block that draws the last ticket adds the per-block
// partial sums in block order: the result does not depend on scheduling.
static constexpr int WN_MAX_BLOCKS = 64;
static constexpr int WN_STRIDE = 304;    // doubles per block in the partial buffer
__global__ void k_wn_backward(const float* theta, const float* dir, const float* ell, const float* cA, const float* cB,
                              int64_t B, float mu, const float* muvec, float* out, int accumulate, float out_scale,
                              double* partial, unsigned* counter) {
  pdl_enter();
  const int k = threadIdx.x;
  const int64_t per = (B + gridDim.x - 1) / gridDim.x;
  const int64_t i0 = blockIdx.x * per, i1 = (i0 + per < B) ? i0 + per : B;
  double ga1 = 0.0, gb1 = 0.0, ga2 = 0.0, gb2 = 0.0;
  const bool unit = k < WN_H;
  const float a1 = unit ? theta[k] : 0.f, b1 = unit ? theta[WN_H + k] : 0.f, a2 = unit ? theta[2 * WN_H + k] : 0.f;
  const float da1 = (unit && dir) ? dir[k] : 0.f, db1 = (unit && dir) ? dir[WN_H + k] : 0.f, da2 = (unit && dir) ? dir[2 * WN_H + k] : 0.f;
  // the block's samples pass through shared memory 128 at a time (one coalesced load per array instead of one
  // broadcast load per sample and thread); every thread still adds its samples in index order
  __shared__ float s_l[128], s_a[128], s_b[128];
  for (int64_t c0 = i0; c0 < i1; c0 += 128) {
    const int cnt = (int)((i1 - c0 < 128) ? i1 - c0 : 128);
    __syncthreads();
    if (k < cnt) { s_l[k] = ell[c0 + k]; s_a[k] = cA[c0 + k]; s_b[k] = cB ? cB[c0 + k] : 0.f; }
    __syncthreads();
    if (unit) {
      for (int i = 0; i < cnt; ++i) {
        const float l = s_l[i], ca = s_a[i], cb = s_b[i];
        const float pre = a1 * l + b1;
        if (pre > 0.f) {
          const float t = ca * a2 + cb * da2;
          ga1 += (double)(l * t);
          gb1 += (double)t;
          ga2 += (double)(ca * pre + cb * (l * da1 + db1));
        }
      }
    } else if (k == WN_H) {
      for (int i = 0; i < cnt; ++i) gb2 += (double)s_a[i];
    }
  }
  double* mine = partial + (size_t)blockIdx.x * WN_STRIDE;
  if (k < WN_H) { mine[k] = ga1; mine[WN_H + k] = gb1; mine[2 * WN_H + k] = ga2; }
  else if (k == WN_H) mine[3 * WN_H] = gb2;
  __shared__ bool is_last;
  __threadfence();
  __syncthreads();
  if (k == 0) is_last = atomicAdd(counter, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // block order, eight loads in flight at a time (L2 loads: the partial sums were written by other SMs)
  auto total = [&](int idx) {
    double t = 0.0;
    for (unsigned b0 = 0; b0 < gridDim.x; b0 += 8) {
      double v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = b0 + u < gridDim.x ? __ldcg(partial + (size_t)(b0 + u) * WN_STRIDE + idx) : 0.0;
#pragma unroll
      for (int u = 0; u < 8; ++u) if (b0 + u < gridDim.x) t += v[u];
    }
    return t;
  };
  auto put = [&](int idx) {
    float v = out_scale * ((float)total(idx) + (muvec ? mu * muvec[idx] : 0.f));
    out[idx] = (accumulate ? out[idx] : 0.f) + v;
  };
  if (k < WN_H) { put(k); put(WN_H + k); put(2 * WN_H + k); }
  else if (k == WN_H) put(3 * WN_H);
  if (k == 0) *counter = 0u;
}

// ------------------------------------------------------------------ finite-difference pieces
// da_tot = da + sign*eps*c.  Hidden layer: hp = act(a + da_tot) -> op16, dh = hp - act(a) -> op16.
// Output layer: z = a + da_tot (fp32).
// hp32 (nullable, [B, N]): the perturbed activation in fp32, i.e. the rounded base value plus the displacement
// (what a consumer that is not a matrix product, the label-correction net, evaluates at).
__global__ void k_fd_act(const float* a, const float* da, const float* cdir, const float* vnorm2, float eps0, float sign,
                         op16* hpm, op16* dhd, float* zpm, int64_t B, int64_t N, int64_t ldh, int act, float* hp32) {
  pdl_enter();
  const float e = sign * fd_eps(vnorm2, eps0);
  const int64_t total = B * N;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / N, n = i - r * N;
    const float d = da[i] + e * cdir[n];
    if (zpm) { zpm[i] = a[i] + d; continue; }
    const float h0 = act_f(act, a[i]), hp = act_f(act, a[i] + d);
    hpm[r * ldh + n] = to_op16(hp);
    dhd[r * ldh + n] = to_op16(hp - h0);
    if (hp32) hp32[i] = from_op16(to_op16(h0)) + (hp - h0);
  }
}
__global__ void k_fd_combine(float* out, const float* gp, const float* gm, const float* vnorm2, float eps0, float alpha,
                             int accumulate, int64_t n) {
  pdl_enter();
  const float e = fd_eps(vnorm2, eps0);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float base = accumulate ? out[i] : 0.f;
    out[i] = e > 0.f ? base - alpha * (gp[i] - gm[i]) / (2.f * e) : base;
  }
}


// ------------------------------------------------------------------ label-correction net
// (Sec. 5.1 "Correcting & reweighting corrupted labels", its App. A listing and the App. C description.)  With h
// the classifier's last hidden activation (width H, as the matrix products see it) and y the given label:
//     s = softmax(A h + a0),   rho = sigmoid(a2 . relu(A1 h + b1) + b2),   new = rho onehot(y) + (1 - rho) s,
// alpha = [A (C x H), a0 (C), A1 (100 x H), b1 (100), a2 (100), b2].  The classifier's per-sample loss becomes
// l_i = -sum_c new_ic log p_ic, and the label is not detached from h.  The net is small (C + 100 outputs per sample):
// it runs on CUDA cores in fp32, one block per sample, every reduction in a fixed order.
static constexpr int CN_T = 128;          // threads per sample
static constexpr int CN_MAX_C = 1024;
static constexpr int CN_MAX_H = 8192;
struct CnOff { int64_t A, a0, A1, b1, a2, b2, total; };
__host__ __device__ static inline CnOff cn_offsets(int64_t H, int64_t C) {
  CnOff o; o.A = 0; o.a0 = C * H; o.A1 = o.a0 + C; o.b1 = o.A1 + WN_H * H; o.a2 = o.b1 + WN_H; o.b2 = o.a2 + WN_H; o.total = o.b2 + 1;
  return o;
}
// sum over the block, same value in every thread; fixed order (warp trees, then the warps in index order)
__device__ __forceinline__ float cn_block_sum(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < CN_T / 32; ++i) t += sh[i];
  __syncthreads();
  return t;
}
__device__ __forceinline__ float cn_block_max(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = -INFINITY;
  for (int i = 0; i < CN_T / 32; ++i) t = fmaxf(t, sh[i]);
  __syncthreads();
  return t;
}
// One block per sample.  h16 (operand type, leading dimension ldh) or h32 ([B, H]) is the last hidden activation;
// z the logits.  Writes hl32 (fp32 copy of h, unless it is h32 itself), logp, s, hid, rho, the new labels and the
// soft-label loss ell.  Dynamic shared memory: H + 2 C + 100 floats.
__global__ void __launch_bounds__(CN_T) k_cn_forward(const float* alpha, const op16* h16, int64_t ldh, const float* h32,
                                                     const float* z, const int32_t* y, int64_t H, int64_t C, float* hl32,
                                                     float* logp, float* s, float* hid, float* rho, float* newlab, float* ell) {
  pdl_enter();
  extern __shared__ float cn_sm[];
  __shared__ float red[CN_T / 32];
  float* hrow = cn_sm; float* tb = hrow + H; float* lp = tb + C; float* hd = lp + C;
  const int64_t row = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const CnOff o = cn_offsets(H, C);
  for (int64_t j = tid; j < H; j += CN_T) {
    const float v = h32 ? h32[row * H + j] : from_op16(h16[row * ldh + j]);
    hrow[j] = v;
    if (hl32 && !h32) hl32[row * H + j] = v;
  }
  // log-softmax of the logits
  const float* zr = z + row * C;
  float mx = -INFINITY;
  for (int64_t c = tid; c < C; c += CN_T) mx = fmaxf(mx, zr[c]);
  mx = cn_block_max(mx, red);          // also orders the writes of hrow before the reads below
  float se = 0.f;
  for (int64_t c = tid; c < C; c += CN_T) se += expf(zr[c] - mx);
  const float lse = logf(cn_block_sum(se, red));
  for (int64_t c = tid; c < C; c += CN_T) { const float v = zr[c] - mx - lse; lp[c] = v; logp[row * C + c] = v; }
  // the C + 100 outputs of the two linear maps: one warp per output, lanes along H
  for (int64_t e = warp; e < C + WN_H; e += CN_T / 32) {
    const float* wrow = e < C ? alpha + o.A + e * H : alpha + o.A1 + (e - C) * H;
    float acc = 0.f;
    for (int64_t j = lane; j < H; j += 32) acc += wrow[j] * hrow[j];
#pragma unroll
    for (int sh = 16; sh > 0; sh >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sh);
    if (lane == 0) {
      if (e < C) tb[e] = acc + alpha[o.a0 + e];
      else hd[e - C] = fmaxf(acc + alpha[o.b1 + (e - C)], 0.f);
    }
  }
  __syncthreads();
  float tm = -INFINITY;
  for (int64_t c = tid; c < C; c += CN_T) tm = fmaxf(tm, tb[c]);
  tm = cn_block_max(tm, red);
  float ts = 0.f;
  for (int64_t c = tid; c < C; c += CN_T) ts += expf(tb[c] - tm);
  ts = cn_block_sum(ts, red);
  const float m = cn_block_sum(tid < WN_H ? alpha[o.a2 + tid] * hd[tid] : 0.f, red) + alpha[o.b2];
  const float r = 1.f / (1.f + expf(-m));
  int32_t yy = y[row];
  yy = yy < 0 ? 0 : (yy >= C ? (int32_t)C - 1 : yy);
  float le = 0.f;
  for (int64_t c = tid; c < C; c += CN_T) {
    const float sc = expf(tb[c] - tm) / ts;
    const float nw = (c == yy ? r : 0.f) + (1.f - r) * sc;
    s[row * C + c] = sc;
    newlab[row * C + c] = nw;
    le -= nw * lp[c];
  }
  le = cn_block_sum(le, red);
  if (tid < WN_H) hid[row * WN_H + tid] = hd[tid];
  if (tid == 0) { rho[row] = r; ell[row] = le; }
}
// Per-sample derivatives of the loss with respect to the net's two pre-activations, times coef_i (or `scale`
// when coef is null).  mode 0: the classifier's soft-label loss (dt = s (g - <s, g>), g = -(1 - rho) log p;
// dm = (-log p_y + <s, log p>) rho (1 - rho); dpre = relu' a2 dm).  mode 1: the correction problem's own term,
// the mean cross-entropy of the soft label against y (dt = s - onehot; nothing through the interpolation net).
// G32 [B, C + 101] = [dt, dpre, dm]; G16 [B, ldg] = [dt, dpre] in the operand type (pad columns zero).
__global__ void __launch_bounds__(CN_T) k_cn_sample_grad(int mode, const float* alpha, const float* logp, const float* s,
                                                         const float* hid, const float* rho, const int32_t* y,
                                                         const float* coef, float scale, int64_t H, int64_t C, float* G32,
                                                         op16* G16, int64_t ldg) {
  pdl_enter();
  __shared__ float red[CN_T / 32];
  const int64_t row = blockIdx.x;
  const int tid = threadIdx.x;
  const CnOff o = cn_offsets(H, C);
  const float cf = coef ? coef[row] : scale;
  const float r = rho[row];
  int32_t yy = y[row];
  yy = yy < 0 ? 0 : (yy >= C ? (int32_t)C - 1 : yy);
  const int64_t W = C + WN_H + 1;
  float sg = 0.f, sl = 0.f;
  if (mode == 0) {
    for (int64_t c = tid; c < C; c += CN_T) {
      const float sc = s[row * C + c], l = logp[row * C + c];
      sg += sc * (-(1.f - r) * l);
      sl += sc * l;
    }
    sg = cn_block_sum(sg, red);
    sl = cn_block_sum(sl, red);
  }
  const float dm = mode == 0 ? (-logp[row * C + yy] + sl) * r * (1.f - r) : 0.f;
  for (int64_t c = tid; c < C; c += CN_T) {
    const float sc = s[row * C + c];
    const float dt = mode == 0 ? sc * (-(1.f - r) * logp[row * C + c] - sg) : sc - (c == yy ? 1.f : 0.f);
    G32[row * W + c] = cf * dt;
    G16[row * ldg + c] = to_op16(cf * dt);
  }
  for (int64_t k = tid; k < ldg - C; k += CN_T) {
    float v = 0.f;
    if (k < WN_H && mode == 0) v = cf * ((hid[row * WN_H + k] > 0.f ? alpha[o.a2 + k] : 0.f) * dm);
    if (k < WN_H) G32[row * W + C + k] = v;
    G16[row * ldg + C + k] = to_op16(v);
  }
  if (tid == 0) G32[row * W + C + WN_H] = cf * dm;
}
// out[e] = sum_i (derivative pieces of sample i) for every parameter e of the net, samples in index order, fp64.
__global__ void k_cn_param_grad(const float* G32, const float* hl32, const float* hid, int64_t B, int64_t H, int64_t C, float* out) {
  pdl_enter();
  const CnOff o = cn_offsets(H, C);
  const int64_t W = C + WN_H + 1;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < o.total; e += (int64_t)gridDim.x * blockDim.x) {
    int64_t gcol; const float* other; int64_t ostride, ocol;      // out[e] = sum_i G32[i, gcol] * other[i * ostride + ocol]
    if (e < o.a0) { gcol = e / H; other = hl32; ostride = H; ocol = e - gcol * H; }
    else if (e < o.A1) { gcol = e - o.a0; other = nullptr; ostride = 0; ocol = 0; }
    else if (e < o.b1) { const int64_t k = (e - o.A1) / H; gcol = C + k; other = hl32; ostride = H; ocol = (e - o.A1) - k * H; }
    else if (e < o.a2) { gcol = C + (e - o.b1); other = nullptr; ostride = 0; ocol = 0; }
    else if (e < o.b2) { gcol = C + WN_H; other = hid; ostride = WN_H; ocol = e - o.a2; }
    else { gcol = C + WN_H; other = nullptr; ostride = 0; ocol = 0; }
    double acc = 0.0;
    for (int64_t i = 0; i < B; ++i) acc += (double)G32[i * W + gcol] * (other ? (double)other[i * ostride + ocol] : 1.0);
    out[e] = (float)acc;
  }
}
// M16 [(C + 100), ldm] = [A; A1] in the operand type: the second operand of the term the label's dependence on h
// adds to the last hidden layer's delta (a matrix product like the others)
__global__ void k_cn_cast_maps(const float* alpha, int64_t H, int64_t C, op16* M16, int64_t ldm) {
  pdl_enter();
  const CnOff o = cn_offsets(H, C);
  const int64_t total = (C + WN_H) * ldm;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / ldm, j = i - r * ldm;
    float v = 0.f;
    if (j < H) v = r < C ? alpha[o.A + r * H + j] : alpha[o.A1 + (r - C) * H + j];
    M16[i] = to_op16(v);
  }
}
// delta = S * coef_i * (p - new label)
__global__ void k_delta_top_soft(const float* p, const float* newlab, const float* coef, float scale, op16* delta, int64_t B,
                                 int64_t C, int64_t ld, const float* lscale) {
  pdl_enter();
  const float S = lscale ? *lscale : 1.f;
  const int64_t total = B * ld;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / ld, c = i - r * ld;
    float v = 0.f;
    if (c < C) v = S * ((coef ? coef[r] : scale) * (p[r * C + c] - newlab[r * C + c]));
    delta[i] = to_op16(v);
  }
}

// ------------------------------------------------------------------ host-side state
struct Net {
  int L;
  int act;
  int64_t w[MAXL + 1];
  int64_t woff[MAXL], boff[MAXL], ldw[MAXL];
  const float* master;
  op16* W[MAXL];
};
struct Pass {
  int64_t B;
  const int32_t* y;
  const op16* h[MAXL];   // h[l]: input of layer l
  int64_t ldh[MAXL];
  float* a[MAXL];        // pre-activations [B, w[l+1]]
  float* p;              // softmax [B, C]
  float* ell;            // per-sample cross-entropy
  op16* delta[MAXL];     // dC/da_l, leading dimension ld8(w[l+1])
  float* dh[MAXL];       // dC/dh_l (input side of layer l), l >= 1, fp32 [B, w[l]]
};
struct HvpCache {
  Net net;
  Pass pass;
  const float* coef;     // per-sample top coefficient (r_i/B) or null (1/B)
  const float* lam;      // device per-layer log weight decay or null
  const betty_level* theta;
  // op16 copies of a direction's matrices that outlive one HVP (series solves): the weight-HVP epilogues
  // of iteration k leave the rounded next term here, so that iteration k+1 starts without a cast pass
  op16* dir16[MAXL];     // null: every R-forward pass rounds its direction into scratch of its own
  const float* dir16_of; // the fp32 vector that dir16 currently mirrors, or null
};

// Label-correction state of one pass (see the kernels above) and what a reverse sweep needs from it.
struct CorrPass {
  const betty_level* G;     // the correction net's level
  int64_t H, C;
  float *hl32, *logp, *s, *hid, *rho, *newlab;
};
struct CorrBack {
  const float* newlab;      // soft labels for the top delta (null: the given labels)
  const op16* G16; int64_t ldg;    // coef_i [dt_i, dpre_i], operand type
  const op16* M16; int64_t ldm;    // [A; A1], operand type
  int64_t Kc;               // C + 100
};

// out[l] (+)= scale * exp(lam[l]) * <W_l, q_l> for every layer (q == nullptr: <W_l, W_l>): one zeroing kernel for all
// ticket counters and one launch for all layers.
static betty_status layer_dots(Ctx& c, const Net& n, const float* q, const float* lam, float scale, float* out, bool accumulate) {
  const size_t mark = c.arena.mark();
  LayerDotJobs jobs;
  jobs.n = n.L; jobs.scale = scale; jobs.accumulate = accumulate ? 1 : 0;
  BETTY_ALLOC(counters, unsigned, c, (size_t)(8 * n.L));
  int blocks = 0;
  for (int l = 0; l < n.L; ++l) {
    const int64_t rows = n.w[l + 1], cols = n.w[l];
    int64_t nb = (rows * cols + 256 * 16 - 1) / (256 * 16);
    nb = nb < 1 ? 1 : (nb > LD_MAX_BLOCKS ? LD_MAX_BLOCKS : nb);
    BETTY_ALLOC(partial, double, c, (size_t)nb);
    LayerDotJob& t = jobs.j[l];
    t.W = n.W[l]; t.rows = rows; t.cols = cols; t.ldw = n.ldw[l];
    t.q = q ? q + n.woff[l] : nullptr; t.lam = lam + l; t.out = out + l;
    t.partial = partial; t.counter = counters + 8 * l; t.first_block = blocks; t.n_blocks = (int)nb;
    blocks += (int)nb;
  }
  BETTY_TRY(vec_zero(c, (float*)counters, 8 * n.L));
  launch_pdl(k_layer_dot_multi, dim3((unsigned)blocks), dim3(256), 0, c.stream, jobs);
  BETTY_LAUNCH_CHECK();
  c.arena.release(mark);
  return BETTY_OK;
}

static betty_status net_layout(const betty_level* M, Net& n) {
  if (M->param_kind != BETTY_PARAM_MLP || M->n_layers < 1 || M->n_layers > MAXL || !M->widths) return BETTY_ERR_INVALID_ARG;
  n.L = M->n_layers;
  n.act = M->activation;
  if (n.act != BETTY_ACT_RELU && n.act != BETTY_ACT_GELU) return BETTY_ERR_INVALID_ARG;
  int64_t off = 0;
  for (int l = 0; l <= n.L; ++l) {
    n.w[l] = M->widths[l];
    if (n.w[l] <= 0) return BETTY_ERR_SHAPE;
  }
  for (int l = 0; l < n.L; ++l) {
    n.woff[l] = off; off += n.w[l + 1] * n.w[l];
    n.boff[l] = off; off += n.w[l + 1];
    n.ldw[l] = ld8(n.w[l]);
  }
  if (off != M->n_params) return BETTY_ERR_SHAPE;
  n.master = M->params;
  return BETTY_OK;
}

// contiguous case (ld == cols, cols % 8 == 0): 8 elements per thread, 2 x float4 in, 1 x 16 bytes out
__global__ void k_cast_dense8(const float* src, op16* dst, int64_t n8, const float* vnorm2, float eps0) {
  pdl_enter();
  const float s = vnorm2 ? fd_eps(vnorm2, eps0) : 1.f;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    const float4 a = ((const float4*)src)[2 * i], b = ((const float4*)src)[2 * i + 1];
    op16x2 o[4];
    o[0] = to_op16x2(s * a.x, s * a.y); o[1] = to_op16x2(s * a.z, s * a.w);
    o[2] = to_op16x2(s * b.x, s * b.y); o[3] = to_op16x2(s * b.z, s * b.w);
    ((uint4*)dst)[i] = *(uint4*)o;
  }
}

static betty_status cast_matrix(Ctx& c, const float* src, op16* dst, int64_t rows, int64_t cols, int64_t ld,
                                const float* vnorm2 = nullptr, float eps0 = 0.f) {
  if (ld == cols && (cols & 7) == 0 && ((((uintptr_t)src) & 15) == 0)) {
    const int64_t n8 = rows * cols / 8;
    launch_pdl(k_cast_dense8, dim3(grid_for(n8)), dim3(256), 0, c.stream, src, dst, n8, vnorm2, eps0);
  } else {
    launch_pdl(k_cast_rows, dim3(grid_for(rows * ld)), dim3(256), 0, c.stream, src, dst, rows, cols, ld, vnorm2, eps0);
  }
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// op16 compute copy of the classifier's matrices (the single quantisation point)
static betty_status net_setup(Ctx& c, const betty_level* M, Net& n) {
  BETTY_TRY(net_layout(M, n));
  if (c.shared.master == M->params) {
    for (int l = 0; l < n.L; ++l) n.W[l] = (op16*)c.shared.W[l];
    return BETTY_OK;
  }
  for (int l = 0; l < n.L; ++l) {
    BETTY_ALLOC(Wl, op16, c, (size_t)(n.w[l + 1] * n.ldw[l]));
    n.W[l] = Wl;
    BETTY_TRY(cast_matrix(c, n.master + n.woff[l], Wl, n.w[l + 1], n.w[l], n.ldw[l]));
  }
  return BETTY_OK;
}

// Rounds the matrices of MLP level M once, at the arena's current top, for every pass of this call that
// evaluates a cost at M's present parameters.  The caller guarantees that the parameters do not change
// and that the arena is not released below this point while the copies are shared, and ends the sharing
// with mlpfam_unshare_weights.
betty_status mlpfam_share_weights(Ctx& c, const betty_level* M) {
  c.shared.master = nullptr;
  if (!M || M->param_kind != BETTY_PARAM_MLP) return BETTY_OK;
  Net n;
  BETTY_TRY(net_setup(c, M, n));
  for (int l = 0; l < n.L; ++l) c.shared.W[l] = n.W[l];
  c.shared.master = M->params;
  return BETTY_OK;
}
void mlpfam_unshare_weights(Ctx& c) { c.shared.master = nullptr; }

static betty_status forward(Ctx& c, const Net& n, const betty_level* D, Pass& ps) {
  ps.B = D->n;
  ps.y = (const int32_t*)D->y;
  const int64_t B = ps.B;
  ps.h[0] = (const op16*)D->X;
  ps.ldh[0] = D->d;
  for (int l = 0; l < n.L; ++l) {
    const int64_t N = n.w[l + 1];
    BETTY_ALLOC(al, float, c, (size_t)(B * N));
    ps.a[l] = al;
    op16* hn = nullptr;
    if (l < n.L - 1) {
      ps.ldh[l + 1] = ld8(N);
      hn = c.arena.alloc<op16>((size_t)(B * ps.ldh[l + 1]));
      if (!hn) return BETTY_ERR_WORKSPACE;
      if (ps.ldh[l + 1] != N) BETTY_TRY(vec_zero(c, (float*)hn, (int64_t)((size_t)(B * ps.ldh[l + 1])) / 2));
      ps.h[l + 1] = hn;
    }
    // a_l = h_l W_l^T + b_l (kept in fp32 for the derivative passes), h_{l+1} = act(a_l) in op16: one kernel
    GemmDesc g = {}; g.M = (int)B; g.N = (int)N; g.npairs = 1; g.C = al; g.ldc = N; g.beta = 0.f;
    g.p[0] = gemm_pair(ps.h[l], ps.ldh[l], false, n.W[l], n.ldw[l], true, (int)n.w[l]);
    g.epi.mode = EPI_BIAS_ACT; g.epi.act = n.act; g.epi.bias = n.master + n.boff[l];
    g.epi.out16 = hn; g.epi.ld16 = hn ? ps.ldh[l + 1] : 0;
    BETTY_TRY(gemm(c, g));
  }
  const int64_t C = n.w[n.L];
  BETTY_ALLOC(p, float, c, (size_t)(B * C));
  BETTY_ALLOC(ell, float, c, (size_t)B);
  ps.p = p; ps.ell = ell;
  launch_pdl(k_softmax_ce, dim3(grid_for(B * 32)), dim3(256), 0, c.stream, ps.a[n.L - 1], ps.y, p, ell, B, C);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// Where the parameter gradient of a reverse sweep goes.
struct GradSink {
  float* gflat;            // plain gradient [gW_l, gb_l] (null: no parameter gradient wanted)
  const float* lam;        // device per-layer log weight decay: adds exp(lam_l) W_l (null: none)
  bool sgd;                // instead of storing the gradient, take the step  master -= lr * grad  in the epilogue
  float lr;
  float* master;           // sgd: parameters to update in place
  op16* const* Wnext;      // sgd: per-layer op16 copies of the updated matrices (for the next step), or null
  const float* lscale;     // device loss scale: every delta, and with it the whole gradient, is multiplied by it (null: 1)
};

// Reverse sweep from delta_top = coef_i (p - onehot).  Always leaves delta[l] (and dh[l] for smooth
// activations) in `ps` for an R-operator pass.
static betty_status backward(Ctx& c, const Net& n, Pass& ps, const float* coef, const GradSink& sink, bool keep_dh = false,
                             const CorrBack* cb = nullptr) {
  const int64_t B = ps.B;
  const int64_t C = n.w[n.L];
  {
    const int64_t ld = ld8(C);
    BETTY_ALLOC(dt, op16, c, (size_t)(B * ld));
    ps.delta[n.L - 1] = dt;
    if (cb && cb->newlab)
      launch_pdl(k_delta_top_soft, dim3(grid_for(B * ld)), dim3(256), 0, c.stream, ps.p, cb->newlab, coef, B > 0 ? 1.f / (float)B : 0.f, dt, B, C, ld, sink.lscale);
    else
      launch_pdl(k_delta_top, dim3(grid_for(B * ld)), dim3(256), 0, c.stream, ps.p, ps.y, coef, B > 0 ? 1.f / (float)B : 0.f, dt, B, C, ld, sink.lscale);
    BETTY_LAUNCH_CHECK();
  }
  // The chain is delta_L -> delta_{L-1} -> ... ; each layer's parameter gradient hangs off it and goes to the
  // side stream.  (A gradient step there writes the master matrix and the *other* op16 copy, never the copy
  // the chain's product for the same layer reads.)
  SideWork side(c, n.L >= SIDE_MIN_LAYERS);
  const bool one_stream = !side.forks();
  ColsumBatch colsums;
  for (int l = n.L - 1; l >= 0; --l) {
    const int64_t N = n.w[l + 1], K = n.w[l], ldd = ld8(N);
    if (sink.gflat || sink.sgd) {
      side.begin();
      GemmDesc g = {}; g.M = (int)N; g.N = (int)K; g.npairs = 1; g.ldc = K; g.beta = 0.f;
      g.p[0] = gemm_pair(ps.delta[l], ldd, true, ps.h[l], ps.ldh[l], false, (int)B);
      ColsumSink cs = {};
      if (sink.sgd) {
        g.C = sink.master + n.woff[l];
        g.epi.mode = EPI_SGD; g.epi.lam = sink.lam ? sink.lam + l : nullptr; g.epi.w16 = n.W[l]; g.epi.ldw16 = n.ldw[l];
        g.epi.step = sink.lr; g.epi.out16 = sink.Wnext ? sink.Wnext[l] : nullptr; g.epi.ld16 = n.ldw[l];
        cs.mode = 1; cs.step = sink.lr; cs.out = sink.master + n.boff[l];
      } else {
        g.C = sink.gflat + n.woff[l];
        cs.mode = 0; cs.out = sink.gflat + n.boff[l];
      }
      BETTY_TRY(gemm(c, g));
      if (!sink.sgd && sink.lam) {
        launch_pdl(k_wd_add_bf16, dim3(grid_for(N * K)), dim3(256), 0, c.stream, sink.gflat + n.woff[l], n.W[l], N, K, n.ldw[l], sink.lam + l, sink.lscale);
        BETTY_LAUNCH_CHECK();
      }
      if (one_stream) {
        colsums.add(ps.delta[l], B, N, ldd, cs);      // taken together after the last product
      } else {
        launch_pdl(k_colsum_bf16, dim3((unsigned)((N + CS_COLS - 1) / CS_COLS)), dim3(1024), 0, c.stream, ps.delta[l], B, N, ldd, cs);
        BETTY_LAUNCH_CHECK();
      }
      side.end();
    }
    if (l > 0) {
      // dh = delta_l W_l ; delta_{l-1} = dh * act'(a_{l-1}) in op16: one kernel.  dh itself is kept
      // only for an R-operator pass over an activation with a second derivative.
      float* dh = nullptr;
      if (keep_dh && n.act != BETTY_ACT_RELU) {
        dh = c.arena.alloc<float>((size_t)(B * K));
        if (!dh) return BETTY_ERR_WORKSPACE;
      }
      ps.dh[l] = dh;
      const int64_t ldp = ld8(K);
      BETTY_ALLOC(dp, op16, c, (size_t)(B * ldp));
      if (ldp != K) BETTY_TRY(vec_zero(c, (float*)dp, (int64_t)((size_t)(B * ldp)) / 2));
      ps.delta[l - 1] = dp;
      GemmDesc g = {}; g.M = (int)B; g.N = (int)K; g.npairs = 1; g.C = dh; g.ldc = K; g.beta = 0.f;
      g.p[0] = gemm_pair(ps.delta[l], ldd, false, n.W[l], n.ldw[l], false, (int)N);
      // corrected labels move with the last hidden activation: one more product into the same accumulator
      if (cb && cb->G16 && l == n.L - 1) g.p[g.npairs++] = gemm_pair(cb->G16, cb->ldg, false, cb->M16, cb->ldm, false, (int)cb->Kc);
      g.epi.mode = EPI_ACT_BWD; g.epi.act = n.act; g.epi.a = ps.a[l - 1]; g.epi.out16 = dp; g.epi.ld16 = ldp;
      BETTY_TRY(gemm(c, g));
    }
  }
  BETTY_TRY(colsums.launch(c));
  return side.join();
}
static inline GradSink grad_into(float* gflat, const float* lam) {
  GradSink s = {}; s.gflat = gflat; s.lam = lam; return s;
}

// Directional derivative of the forward pass along `dir` (flat, same layout as the parameters).
struct RPass {
  op16* U[MAXL];
  float* Ra[MAXL];
  const op16* Rh[MAXL];   // Rh[0] == nullptr (inputs do not move)
};
static betty_status rforward(Ctx& c, const Net& n, const Pass& ps, const float* dir, RPass& rp, HvpCache* keep) {
  const int64_t B = ps.B;
  rp.Rh[0] = nullptr;
  const bool kept = keep && keep->dir16[0];
  const bool fresh = kept && keep->dir16_of == dir;      // the kept copies already mirror this direction
  for (int l = 0; l < n.L; ++l) {
    const int64_t N = n.w[l + 1], K = n.w[l];
    op16* Ul = kept ? keep->dir16[l] : c.arena.alloc<op16>((size_t)(N * n.ldw[l]));
    if (!Ul) return BETTY_ERR_WORKSPACE;
    rp.U[l] = Ul;
    if (!fresh) BETTY_TRY(cast_matrix(c, dir + n.woff[l], Ul, N, K, n.ldw[l]));
    BETTY_ALLOC(Ra, float, c, (size_t)(B * N));
    rp.Ra[l] = Ra;
    op16* Rhn = nullptr;
    if (l < n.L - 1) {
      Rhn = c.arena.alloc<op16>((size_t)(B * ps.ldh[l + 1]));
      if (!Rhn) return BETTY_ERR_WORKSPACE;
      if (ps.ldh[l + 1] != N) BETTY_TRY(vec_zero(c, (float*)Rhn, (int64_t)((size_t)(B * ps.ldh[l + 1])) / 2));
      rp.Rh[l + 1] = Rhn;
    }
    // Ra_l = h_l U_l^T + Rh_l W_l^T + c_l ; Rh_{l+1} = act'(a_l) * Ra_l: one kernel
    GemmDesc g = {}; g.M = (int)B; g.N = (int)N; g.C = Ra; g.ldc = N; g.beta = 0.f;
    g.npairs = 0;
    g.p[g.npairs++] = gemm_pair(ps.h[l], ps.ldh[l], false, Ul, n.ldw[l], true, (int)K);
    if (l > 0) g.p[g.npairs++] = gemm_pair(rp.Rh[l], ps.ldh[l], false, n.W[l], n.ldw[l], true, (int)K);
    g.epi.mode = EPI_R_FWD; g.epi.act = n.act; g.epi.bias = dir + n.boff[l]; g.epi.a = ps.a[l];
    g.epi.out16 = Rhn; g.epi.ld16 = Rhn ? ps.ldh[l + 1] : 0;
    BETTY_TRY(gemm(c, g));
  }
  if (kept) keep->dir16_of = dir;
  return BETTY_OK;
}

// ------------------------------------------------------------------ participants
struct Parts {
  const betty_level* mlp;
  const betty_level* theta;   // weight net or null
  const betty_level* lam;     // log weight decay or null
  const betty_level* corr;    // label-correction net or null
};
static Parts parts_of(const betty_level* L) {
  Parts p;
  p.mlp = find_participant(L, BETTY_PARAM_MLP);
  p.corr = nullptr;
  if (L->loss == BETTY_LOSS_MLP_CE_REWEIGHT) p.corr = find_constraint(L, BETTY_PARAM_CORRECTNET);
  if (L->loss == BETTY_LOSS_MLP_CE_CORRECT) p.corr = find_participant(L, BETTY_PARAM_CORRECTNET);
  if (L->loss == BETTY_LOSS_WEIGHTNET_DETECT) {
    p.theta = find_participant(L, BETTY_PARAM_WEIGHTNET);
    p.lam = nullptr;
  } else if (L->loss == BETTY_LOSS_MLP_CE_REWEIGHT) {
    p.theta = find_constraint(L, BETTY_PARAM_WEIGHTNET);
    p.lam = find_constraint(L, BETTY_PARAM_LOGWD);
  } else {
    p.theta = nullptr; p.lam = nullptr;
  }
  return p;
}

betty_status mlpfam_validate(const betty_level* L) {
  const Parts P = parts_of(L);
  if (!P.mlp || !P.mlp->params) return BETTY_ERR_INVALID_ARG;
  if (L->loss == BETTY_LOSS_MLP_CE_REWEIGHT && L->param_kind != BETTY_PARAM_MLP) return BETTY_ERR_INVALID_ARG;
  Net n;
  BETTY_TRY(net_layout(P.mlp, n));
  if (L->n < 0 || L->d != n.w[0]) return BETTY_ERR_SHAPE;
#ifdef BETTY_FP16_OPERANDS
  if (L->x_dtype != BETTY_F16) return BETTY_ERR_DTYPE;
#else
  if (L->x_dtype != BETTY_BF16) return BETTY_ERR_DTYPE;
#endif
  if (L->n > 0 && (!L->X || !L->y)) return BETTY_ERR_INVALID_ARG;
  if (!aligned16(L->X) || !aligned16(P.mlp->params)) return BETTY_ERR_ALIGNMENT;
  if (L->d % 8 != 0) return BETTY_ERR_ALIGNMENT;     // op16 rows must start on 16-byte boundaries
  if (L->loss == BETTY_LOSS_MLP_CE_CORRECT && !P.corr) return BETTY_ERR_INVALID_ARG;
  if (P.corr) {
    if (n.L < 2) return BETTY_ERR_SHAPE;                       // the net reads a hidden activation
    const int64_t H = n.w[n.L - 1], C = n.w[n.L];
    if (C > CN_MAX_C || H > CN_MAX_H) return BETTY_ERR_UNSUPPORTED;
    if (!P.corr->params || P.corr->n_params != cn_offsets(H, C).total) return BETTY_ERR_SHAPE;
    if (P.mlp->loss_scale) return BETTY_ERR_UNSUPPORTED;        // loss scaling is not offered together with label correction
  }
  if (P.theta && (P.theta->n_params != WN_P || !P.theta->params)) return BETTY_ERR_SHAPE;
  if (P.lam && (P.lam->n_params != n.L || !P.lam->params)) return BETTY_ERR_SHAPE;
  if (L->loss == BETTY_LOSS_WEIGHTNET_DETECT) {
    if (!P.theta) return BETTY_ERR_INVALID_ARG;
    if (L->n > 0 && !L->aux) return BETTY_ERR_INVALID_ARG;
  }
  return BETTY_OK;
}

size_t mlpfam_workspace(const betty_level* L) {
  const Parts P = parts_of(L);
  if (!P.mlp || !P.mlp->widths) return 0;
  size_t S = 0;
  for (int l = 0; l <= P.mlp->n_layers; ++l) S += (size_t)ld8(P.mlp->widths[l]) + 8;
  const size_t B = (size_t)(L->n > 0 ? L->n : 1);
  size_t extra = 0;
  if (P.corr && P.mlp->n_layers >= 2) {
    const size_t H = (size_t)P.mlp->widths[P.mlp->n_layers - 1], C = (size_t)P.mlp->widths[P.mlp->n_layers];
    extra = 16 * (size_t)P.corr->n_params + 64 * B * (H + 2 * C + 256) + (1 << 16);
  }
  return 24 * (size_t)P.mlp->n_params + 96 * B * S + 64 * 256 * (size_t)(P.mlp->n_layers + 4) + (1 << 20) + extra;
}

// per-sample scalar through the weight net
static betty_status wn_sample(Ctx& c, int mode, const betty_level* theta, const float* dir, const Pass& ps,
                              const float* aux, const float* din, float* out1, float* out2) {
  const int64_t B = ps.B;
  launch_pdl(k_wn_sample, dim3(grid_for(B, 128)), dim3(128), 0, c.stream, mode, theta->params, dir, ps.ell, aux, din, B,
                                                      B > 0 ? 1.f / (float)B : 0.f, out1, out2);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
// keep_scratch: the partial-sum scratch stays allocated (for a caller that runs this on the side stream and
// releases the arena only after the join)
static betty_status wn_backward(Ctx& c, const betty_level* theta, const float* dir, const Pass& ps, const float* cA,
                                const float* cB, float mu, const float* muvec, float* out, bool accumulate = false,
                                float out_scale = 1.f, bool keep_scratch = false) {
  // 64 samples per block: the block that comes last reads every block's 301 partial sums, so few blocks
  // keep that second phase short (batch 1024: 16 blocks)
  int nb = (int)((ps.B + 63) / 64);
  nb = nb < 1 ? 1 : (nb > WN_MAX_BLOCKS ? WN_MAX_BLOCKS : nb);
  const size_t mark = c.arena.mark();
  BETTY_ALLOC(partial, double, c, (size_t)nb * WN_STRIDE);
  BETTY_ALLOC(counter, unsigned, c, 8);
  BETTY_TRY(vec_zero(c, (float*)counter, 8));     // a kernel, not a memset: keeps the programmatic launch chain unbroken
  launch_pdl(k_wn_backward, dim3(nb), dim3(128), 0, c.stream, theta->params, dir, ps.ell, cA, cB, ps.B, mu, muvec, out, accumulate ? 1 : 0,
                                          out_scale, partial, counter);
  BETTY_LAUNCH_CHECK();
  if (!keep_scratch) c.arena.release(mark);
  return BETTY_OK;
}

// top coefficient of the classifier's own cost: r_i/B with a weight net attached, else 1/B (null)
static betty_status reweight_coef(Ctx& c, const Parts& P, const Pass& ps, const float** coef) {
  *coef = nullptr;
  if (!P.theta) return BETTY_OK;
  BETTY_ALLOC(cf, float, c, (size_t)(ps.B > 0 ? ps.B : 1));
  BETTY_TRY(wn_sample(c, WN_REWEIGHT_COEF, P.theta, nullptr, ps, nullptr, nullptr, cf, nullptr));
  *coef = cf;
  return BETTY_OK;
}

// ---- label-correction net: host side
// Runs the net on the pass's last hidden activation (or on h32, a perturbed copy) and logits (or z), and replaces
// the pass's per-sample losses by the soft-label losses.
static betty_status corr_forward(Ctx& c, const Net& n, Pass& ps, const betty_level* G, CorrPass& cp, const float* h32 = nullptr,
                                 const float* z = nullptr) {
  const int64_t B = ps.B, H = n.w[n.L - 1], C = n.w[n.L];
  cp.G = G; cp.H = H; cp.C = C;
  const size_t nb = (size_t)(B > 0 ? B : 1);
  cp.hl32 = h32 ? const_cast<float*>(h32) : c.arena.alloc<float>(nb * H);
  cp.logp = c.arena.alloc<float>(nb * C);
  cp.s = c.arena.alloc<float>(nb * C);
  cp.hid = c.arena.alloc<float>(nb * WN_H);
  cp.rho = c.arena.alloc<float>(nb);
  cp.newlab = c.arena.alloc<float>(nb * C);
  if (!cp.hl32 || !cp.logp || !cp.s || !cp.hid || !cp.rho || !cp.newlab) return BETTY_ERR_WORKSPACE;
  if (B <= 0) return BETTY_OK;
  const size_t smem = (size_t)(H + 2 * C + WN_H) * sizeof(float);
  launch_pdl(k_cn_forward, dim3((unsigned)B), dim3(CN_T), smem, c.stream, (const float*)G->params, ps.h[n.L - 1], ps.ldh[n.L - 1], h32,
             z ? z : (const float*)ps.a[n.L - 1], ps.y, H, C, cp.hl32, cp.logp, cp.s, cp.hid, cp.rho, cp.newlab, ps.ell);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
// coef_i times the per-sample derivatives (mode: see k_cn_sample_grad); G32 for the parameter gradient, G16 for the
// reverse sweep's extra product
static betty_status corr_sample_grad(Ctx& c, int mode, const CorrPass& cp, const Pass& ps, const float* coef, float** G32,
                                     op16** G16, int64_t* ldg) {
  const int64_t B = ps.B, W = cp.C + WN_H + 1;
  *ldg = ld8(cp.C + WN_H);
  const size_t nb = (size_t)(B > 0 ? B : 1);
  *G32 = c.arena.alloc<float>(nb * W);
  *G16 = c.arena.alloc<op16>(nb * (size_t)*ldg);
  if (!*G32 || !*G16) return BETTY_ERR_WORKSPACE;
  if (B <= 0) return BETTY_OK;
  launch_pdl(k_cn_sample_grad, dim3((unsigned)B), dim3(CN_T), 0, c.stream, mode, (const float*)cp.G->params, (const float*)cp.logp,
             (const float*)cp.s, (const float*)cp.hid, (const float*)cp.rho, ps.y, coef, B > 0 ? 1.f / (float)B : 0.f, cp.H, cp.C, *G32,
             *G16, *ldg);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
static betty_status corr_param_grad(Ctx& c, const CorrPass& cp, const Pass& ps, const float* G32, float* out) {
  const int64_t total = cn_offsets(cp.H, cp.C).total;
  launch_pdl(k_cn_param_grad, dim3(grid_for(total)), dim3(256), 0, c.stream, G32, (const float*)cp.hl32, (const float*)cp.hid, ps.B, cp.H, cp.C, out);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}
static betty_status corr_maps(Ctx& c, const betty_level* G, int64_t H, int64_t C, op16** M16, int64_t* ldm) {
  *ldm = ld8(H);
  *M16 = c.arena.alloc<op16>((size_t)((C + WN_H) * *ldm));
  if (!*M16) return BETTY_ERR_WORKSPACE;
  launch_pdl(k_cn_cast_maps, dim3(grid_for((C + WN_H) * *ldm)), dim3(256), 0, c.stream, (const float*)G->params, H, C, *M16, *ldm);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

betty_status mlpfam_grad(Ctx& c, const betty_level* L, const betty_level* wrt, float* out) {
  const Parts P = parts_of(L);
  const size_t mark = c.arena.mark();
  const bool touches = (wrt == P.mlp) || (P.theta && wrt == P.theta) || (P.lam && wrt == P.lam) || (P.corr && wrt == P.corr);
  if (!touches) return vec_zero(c, out, wrt->n_params);
  Net n; Pass ps;
  BETTY_TRY(net_setup(c, P.mlp, n));
  if (P.lam && wrt == P.lam) {
    BETTY_TRY(layer_dots(c, n, nullptr, P.lam->params, 0.5f, out, false));
    c.arena.release(mark);
    return BETTY_OK;
  }
  BETTY_TRY(forward(c, n, L, ps));
  BETTY_ALLOC(s1, float, c, (size_t)(ps.B > 0 ? ps.B : 1));
  CorrPass cp;
  if (P.corr) BETTY_TRY(corr_forward(c, n, ps, P.corr, cp));      // ps.ell now holds the soft-label losses
  if (L->loss == BETTY_LOSS_MLP_CE) {
    BETTY_TRY(backward(c, n, ps, nullptr, grad_into(out, nullptr)));
  } else if (L->loss == BETTY_LOSS_MLP_CE_CORRECT) {
    // mean CE of the classifier + mean CE of the correction net's own soft labels, both against the given labels
    float* G32; op16* G16; int64_t ldg;
    BETTY_TRY(corr_sample_grad(c, 1, cp, ps, nullptr, &G32, &G16, &ldg));
    if (wrt == P.corr) {
      BETTY_TRY(corr_param_grad(c, cp, ps, G32, out));
    } else {
      CorrBack cb = {};
      cb.G16 = G16; cb.ldg = ldg; cb.Kc = cp.C + WN_H;
      op16* M16;
      BETTY_TRY(corr_maps(c, P.corr, cp.H, cp.C, &M16, &cb.ldm));
      cb.M16 = M16;
      BETTY_TRY(backward(c, n, ps, nullptr, grad_into(out, nullptr), false, &cb));
    }
  } else if (L->loss == BETTY_LOSS_MLP_CE_REWEIGHT) {
    if (wrt == P.mlp || (P.corr && wrt == P.corr)) {
      const float* coef;
      BETTY_TRY(reweight_coef(c, P, ps, &coef));
      CorrBack cb = {};
      float* G32 = nullptr;
      if (P.corr) {
        op16* G16;
        BETTY_TRY(corr_sample_grad(c, 0, cp, ps, coef, &G32, &G16, &cb.ldg));
        cb.newlab = cp.newlab; cb.G16 = G16; cb.Kc = cp.C + WN_H;
      }
      if (P.corr && wrt == P.corr) {
        BETTY_TRY(corr_param_grad(c, cp, ps, G32, out));
      } else {
        if (P.corr) {
          op16* M16;
          BETTY_TRY(corr_maps(c, P.corr, cp.H, cp.C, &M16, &cb.ldm));
          cb.M16 = M16;
        }
        GradSink sink = grad_into(out, P.lam ? P.lam->params : nullptr);
        sink.lscale = c.loss_scale;       // set by a loss-scaled lower step only
        BETTY_TRY(backward(c, n, ps, coef, sink, false, P.corr ? &cb : nullptr));
      }
    } else {
      BETTY_TRY(wn_sample(c, WN_REWEIGHT_TGRAD, P.theta, nullptr, ps, nullptr, nullptr, s1, nullptr));
      BETTY_TRY(wn_backward(c, P.theta, nullptr, ps, s1, nullptr, 0.f, nullptr, out));
    }
  } else {  // WEIGHTNET_DETECT
    if (wrt == P.theta) {
      BETTY_TRY(wn_sample(c, WN_DETECT_TGRAD, P.theta, nullptr, ps, L->aux, nullptr, s1, nullptr));
      BETTY_TRY(wn_backward(c, P.theta, nullptr, ps, s1, nullptr, L->mu, P.theta->params, out));
    } else {
      BETTY_TRY(wn_sample(c, WN_DETECT_WGRAD, P.theta, nullptr, ps, L->aux, nullptr, s1, nullptr));
      BETTY_TRY(backward(c, n, ps, s1, grad_into(out, nullptr)));
    }
  }
  c.arena.release(mark);
  return BETTY_OK;
}

static HvpCache& next_cache_slot() {
  static thread_local HvpCache store[MLP_HVP_CACHE_SLOTS];   // host-side bookkeeping only; device state lives in the workspace
  static thread_local unsigned next_slot = 0;
  return store[next_slot++ % MLP_HVP_CACHE_SLOTS];
}
betty_status mlpfam_hvp_begin(Ctx& c, const betty_level* L, MlpHvpCache** cache) {
  HvpCache& h = next_cache_slot();
  const Parts P = parts_of(L);
  if (P.corr) return BETTY_ERR_UNSUPPORTED;     // second derivatives are not offered with label correction (the paper pairs it with AID-FD)
  h.theta = P.theta;
  h.lam = P.lam ? P.lam->params : nullptr;
  h.coef = nullptr;
  for (int l = 0; l < MAXL; ++l) h.dir16[l] = nullptr;
  h.dir16_of = nullptr;
  BETTY_TRY(net_setup(c, P.mlp, h.net));
  BETTY_TRY(forward(c, h.net, L, h.pass));
  if (L->loss == BETTY_LOSS_MLP_CE_REWEIGHT) {
    BETTY_TRY(reweight_coef(c, P, h.pass, &h.coef));
    BETTY_TRY(backward(c, h.net, h.pass, h.coef, grad_into(nullptr, nullptr), true));
  } else if (!(L->loss == BETTY_LOSS_WEIGHTNET_DETECT && L->param_kind == BETTY_PARAM_WEIGHTNET)) {
    return BETTY_ERR_UNSUPPORTED;
  }
  *cache = (MlpHvpCache*)&h;     // handed out as an opaque handle
  return BETTY_OK;
}

// Neumann-series consumer of an HVP.  The truncated series alpha * sum_{j<=K} (I - alpha H)^j v is
// evaluated by Horner's rule, s <- v + (I - alpha H) s starting from s = v: per step one vector is read
// as the HVP direction, v is read and the new partial sum written (the term/sum recurrence reads and
// writes two vectors per step; at 138M parameters that is 1.1 GB less traffic per step).
struct SeriesSink { const float* v; float alpha; float* out; };

// H u.  Without a sink the product is written to Hu; with one, u is the partial sum so far and the
// Horner step is applied inside the weight-gradient products and bias column sums (Hu is not used).
static betty_status hvp_impl(Ctx& c, const betty_level* L, HvpCache* h, const float* u, float* Hu,
                             const SeriesSink* sink) {
  const size_t mark = c.arena.mark();
  const Net& n = h->net;
  Pass& ps = h->pass;
  const int64_t B = ps.B;
  if (L->loss == BETTY_LOSS_WEIGHTNET_DETECT) {
    BETTY_ALLOC(cA, float, c, (size_t)(B > 0 ? B : 1));
    BETTY_ALLOC(cB, float, c, (size_t)(B > 0 ? B : 1));
    BETTY_TRY(wn_sample(c, WN_DETECT_THVP, L, u, ps, L->aux, nullptr, cA, cB));
    float* dst = Hu;
    if (sink) { dst = c.arena.alloc<float>(512); if (!dst) return BETTY_ERR_WORKSPACE; }
    BETTY_TRY(wn_backward(c, L, u, ps, cA, cB, L->mu, u, dst));
    if (sink) {   // out = v + (u - alpha H u)
      BETTY_ALLOC(tmp, float, c, 512);
      BETTY_TRY(neumann_update(c, u, sink->v, dst, sink->alpha, tmp, sink->out, WN_P));
    }
    c.arena.release(mark);
    return BETTY_OK;
  }
  RPass rp;
  BETTY_TRY(rforward(c, n, ps, u, rp, h));
  const int64_t C = n.w[n.L];
  op16* Rd;
  {
    const int64_t ld = ld8(C);
    Rd = c.arena.alloc<op16>((size_t)(B * ld));
    if (!Rd) return BETTY_ERR_WORKSPACE;
    launch_pdl(k_r_delta_top, dim3(grid_for(B * 32)), dim3(256), 0, c.stream, ps.p, rp.Ra[n.L - 1], h->coef, B > 0 ? 1.f / (float)B : 0.f, Rd,
                                                         B, C, ld);
    BETTY_LAUNCH_CHECK();
  }
  const bool leave16 = sink && h->dir16[0];     // the weight-HVP epilogues also leave the op16 copy of the new partial sum in dir16
  // The chain is Rdelta_L -> Rdelta_{L-1} -> ... ; each layer's weight product goes to the side stream once the
  // chain's product of the same layer has been launched (it reads the U_l that the weight product may overwrite).
  SideWork side(c, n.L >= SIDE_MIN_LAYERS);
  const bool one_stream = !side.forks();
  ColsumBatch colsums;
  for (int l = n.L - 1; l >= 0; --l) {
    const int64_t N = n.w[l + 1], K = n.w[l], ldd = ld8(N);
    op16* Rdp = nullptr;
    if (l > 0) {  // R dh = Rdelta W_l + delta_l U_l ; Rdelta_{l-1} = Rdh*act' + dh*act''*Ra
      // (before this layer's weight product, whose epilogue may overwrite U_l with the next term)
      const int64_t ldp = ld8(K);
      Rdp = c.arena.alloc<op16>((size_t)(B * ldp));
      if (!Rdp) return BETTY_ERR_WORKSPACE;
      if (ldp != K) BETTY_TRY(vec_zero(c, (float*)Rdp, (int64_t)((size_t)(B * ldp)) / 2));
      GemmDesc g = {}; g.M = (int)B; g.N = (int)K; g.C = nullptr; g.ldc = K; g.beta = 0.f; g.npairs = 2;
      g.p[0] = gemm_pair(Rd, ldd, false, n.W[l], n.ldw[l], false, (int)N);
      g.p[1] = gemm_pair(ps.delta[l], ldd, false, rp.U[l], n.ldw[l], false, (int)N);
      g.epi.mode = EPI_R_BWD; g.epi.act = n.act; g.epi.a = ps.a[l - 1]; g.epi.dh = ps.dh[l]; g.epi.Ra = rp.Ra[l - 1];
      g.epi.out16 = Rdp; g.epi.ld16 = ldp;
      BETTY_TRY(gemm(c, g));
    }
    {  // R gW_l = Rdelta^T h_l + delta_l^T Rh_l + exp(lam_l) U_l
      side.begin();
      GemmDesc g = {}; g.M = (int)N; g.N = (int)K; g.ldc = K; g.beta = 0.f; g.npairs = 0;
      g.p[g.npairs++] = gemm_pair(Rd, ldd, true, ps.h[l], ps.ldh[l], false, (int)B);
      if (l > 0) g.p[g.npairs++] = gemm_pair(ps.delta[l], ldd, true, rp.Rh[l], ps.ldh[l], false, (int)B);
      ColsumSink cs = {};
      if (sink) {
        g.C = sink->out + n.woff[l];
        g.epi.mode = EPI_NEUMANN; g.epi.lam = h->lam ? h->lam + l : nullptr; g.epi.step = sink->alpha;
        g.epi.t_in = u + n.woff[l]; g.epi.s_in = sink->v + n.woff[l];
        if (leave16) { g.epi.out16 = h->dir16[l]; g.epi.ld16 = n.ldw[l]; }
        cs.mode = 2; cs.step = sink->alpha; cs.out = sink->out + n.boff[l]; cs.t_in = u + n.boff[l];
        cs.s_in = sink->v + n.boff[l];
      } else {
        g.C = Hu + n.woff[l];
        cs.mode = 0; cs.out = Hu + n.boff[l];
      }
      BETTY_TRY(gemm(c, g));
      if (!sink && h->lam) {
        launch_pdl(k_wd_add_f32, dim3(grid_for(N * K)), dim3(256), 0, c.stream, Hu + n.woff[l], u + n.woff[l], N * K, h->lam + l);
        BETTY_LAUNCH_CHECK();
      }
      if (one_stream) {
        colsums.add(Rd, B, N, ldd, cs);
      } else {
        launch_pdl(k_colsum_bf16, dim3((unsigned)((N + CS_COLS - 1) / CS_COLS)), dim3(1024), 0, c.stream, Rd, B, N, ldd, cs);
        BETTY_LAUNCH_CHECK();
      }
      side.end();
    }
    if (l > 0) Rd = Rdp;
  }
  BETTY_TRY(colsums.launch(c));
  BETTY_TRY(side.join());
  if (leave16) h->dir16_of = sink->out;
  c.arena.release(mark);
  return BETTY_OK;
}

// Gives the HVPs of a series solve persistent storage for the op16 copy of the current term (allocated
// at the arena's current top: call it after mlpfam_hvp_begin and before the first HVP of the solve).
betty_status mlpfam_hvp_keep_direction(Ctx& c, MlpHvpCache* handle) {
  HvpCache* h = (HvpCache*)handle;
  if (!h || h->dir16[0]) return BETTY_OK;
  const Net& n = h->net;
  for (int l = 0; l < n.L; ++l) {
    h->dir16[l] = c.arena.alloc<op16>((size_t)(n.w[l + 1] * n.ldw[l]));
    if (!h->dir16[l]) { h->dir16[0] = nullptr; return BETTY_ERR_WORKSPACE; }
  }
  h->dir16_of = nullptr;
  return BETTY_OK;
}

betty_status mlpfam_hvp(Ctx& c, const betty_level* L, MlpHvpCache* h, const float* u, float* Hu) {
  return hvp_impl(c, L, (HvpCache*)h, u, Hu, nullptr);
}

betty_status mlpfam_hvp_series(Ctx& c, const betty_level* L, MlpHvpCache* h, const float* s, const float* v, float alpha,
                               float* s_out) {
  SeriesSink sink = {v, alpha, s_out};
  return hvp_impl(c, L, (HvpCache*)h, s, nullptr, &sink);
}

betty_status mlpfam_mixed(Ctx& c, const betty_level* L, MlpHvpCache* handle, const betty_level* wrt, const float* q,
                          float* out) {
  HvpCache* h = (HvpCache*)handle;
  const size_t mark = c.arena.mark();
  const Parts P = parts_of(L);
  const Net& n = h->net;
  Pass& ps = h->pass;
  const int64_t B = ps.B;
  if (L->loss == BETTY_LOSS_MLP_CE_REWEIGHT) {
    if (P.lam && wrt == P.lam) {
      BETTY_TRY(layer_dots(c, n, q, P.lam->params, 1.f, out, false));
    } else if (P.theta && wrt == P.theta) {
      RPass rp;
      BETTY_TRY(rforward(c, n, ps, q, rp, h));
      BETTY_ALLOC(d, float, c, (size_t)(B > 0 ? B : 1));
      BETTY_ALLOC(s1, float, c, (size_t)(B > 0 ? B : 1));
      launch_pdl(k_jvp_rows, dim3(grid_for(B * 32)), dim3(256), 0, c.stream, ps.p, ps.y, rp.Ra[n.L - 1], d, B, n.w[n.L]);
      BETTY_LAUNCH_CHECK();
      BETTY_TRY(wn_sample(c, WN_REWEIGHT_TMIXED, P.theta, nullptr, ps, nullptr, d, s1, nullptr));
      BETTY_TRY(wn_backward(c, P.theta, nullptr, ps, s1, nullptr, 0.f, nullptr, out));
    } else {
      return BETTY_ERR_INVALID_ARG;
    }
  } else if (L->loss == BETTY_LOSS_WEIGHTNET_DETECT && L->param_kind == BETTY_PARAM_WEIGHTNET && wrt == P.mlp) {
    BETTY_ALLOC(s1, float, c, (size_t)(B > 0 ? B : 1));
    BETTY_TRY(wn_sample(c, WN_DETECT_WMIXED, L, q, ps, L->aux, nullptr, s1, nullptr));
    BETTY_TRY(backward(c, n, ps, s1, grad_into(out, nullptr)));
  } else {
    return BETTY_ERR_INVALID_ARG;
  }
  c.arena.release(mark);
  return BETTY_OK;
}

betty_status mlpfam_lower_step(Ctx& c, const betty_level* L, int n_steps, int first_step) {
  if (L->loss != BETTY_LOSS_MLP_CE_REWEIGHT) return BETTY_ERR_UNSUPPORTED;
  if (n_steps <= 0) return BETTY_OK;
  const size_t mark = c.arena.mark();
  const Parts P = parts_of(L);
  // The gradient step is taken inside the weight-gradient products' epilogues, which also write the
  // op16 copy of the updated matrices for the next step: one cast at the start, none afterwards.
  Net n;
  BETTY_TRY(net_setup(c, P.mlp, n));
  CorrBack cb = {};
  if (P.corr) {       // the correction net does not move during the classifier's steps: its maps are cast once
    op16* M16;
    BETTY_TRY(corr_maps(c, P.corr, n.w[n.L - 1], n.w[n.L], &M16, &cb.ldm));
    cb.M16 = M16; cb.Kc = n.w[n.L] + WN_H;
  }
  op16* alt[MAXL];
  for (int l = 0; l < n.L; ++l) {
    const size_t cnt = (size_t)(n.w[l + 1] * n.ldw[l]);
    alt[l] = c.arena.alloc<op16>(cnt);
    if (!alt[l]) return BETTY_ERR_WORKSPACE;
    if (n.ldw[l] != n.w[l]) BETTY_TRY(vec_zero(c, (float*)alt[l], (int64_t)(cnt) / 2));
  }
  for (int s = 0; s < n_steps; ++s) {
    const size_t m2 = c.arena.mark();
    Pass ps;
    BETTY_TRY(forward(c, n, L, ps));
    CorrPass cp;
    if (P.corr) BETTY_TRY(corr_forward(c, n, ps, P.corr, cp));
    const float* coef;
    BETTY_TRY(reweight_coef(c, P, ps, &coef));
    if (P.corr) {
      float* G32; op16* G16;
      BETTY_TRY(corr_sample_grad(c, 0, cp, ps, coef, &G32, &G16, &cb.ldg));
      cb.newlab = cp.newlab; cb.G16 = G16;
    }
    GradSink sink = {};
    sink.lam = P.lam ? P.lam->params : nullptr;
    sink.sgd = true; sink.lr = lr_at(L, first_step + s); sink.master = L->params; sink.Wnext = alt;
    BETTY_TRY(backward(c, n, ps, coef, sink, false, P.corr ? &cb : nullptr));
    for (int l = 0; l < n.L; ++l) { op16* t = n.W[l]; n.W[l] = alt[l]; alt[l] = t; }
    c.arena.release(m2);
  }
  c.arena.release(mark);
  return BETTY_OK;
}

// Finite difference of dC/dc at x +- eps v.  For the weight-net constraint the two perturbed forward
// passes carry the perturbation separately from the base activations (base + delta operands), so that
// an eps*v far below op16 resolution of the weights survives the op16 matrix products.
// The part of mlpfam_fd that does not depend on the direction: the classifier's forward pass at the unperturbed
// parameters.  Its buffers stay allocated (the handle is a slot of the per-thread ring of base passes).
betty_status mlpfam_fd_begin(Ctx& c, const betty_level* L, MlpHvpCache** cache) {
  if (L->loss != BETTY_LOSS_MLP_CE_REWEIGHT) return BETTY_ERR_UNSUPPORTED;
  HvpCache& h = next_cache_slot();
  const Parts P = parts_of(L);
  BETTY_TRY(net_setup(c, P.mlp, h.net));
  BETTY_TRY(forward(c, h.net, L, h.pass));
  *cache = (MlpHvpCache*)&h;
  return BETTY_OK;
}

// pre: the forward pass made by mlpfam_fd_begin, or null
betty_status mlpfam_fd(Ctx& c, const betty_level* L, const betty_level* wrt, const float* v, const float* vnorm2,
                       float eps0, float alpha, float* out, bool accumulate, MlpHvpCache* pre) {
  if (L->loss != BETTY_LOSS_MLP_CE_REWEIGHT) return BETTY_ERR_UNSUPPORTED;
  const Parts P = parts_of(L);
  const size_t mark = c.arena.mark();
  Net n; Pass ps;
  if (pre) n = ((HvpCache*)pre)->net;
  else BETTY_TRY(net_setup(c, P.mlp, n));
  if (P.lam && wrt == P.lam) {
    // dC/d(lam_l) = 1/2 exp(lam_l)|W_l|^2 is quadratic in W: its central difference is exactly
    // exp(lam_l) <W_l, V_l> for every eps, which is what is evaluated.
    BETTY_TRY(layer_dots(c, n, v, P.lam->params, -alpha, out, accumulate));
    c.arena.release(mark);
    return BETTY_OK;
  }
  const bool wrt_theta = P.theta && wrt == P.theta, wrt_corr = P.corr && wrt == P.corr;
  if (!wrt_theta && !wrt_corr) return BETTY_ERR_INVALID_ARG;
  if (pre) ps = ((HvpCache*)pre)->pass;
  else BETTY_TRY(forward(c, n, L, ps));
  const int64_t B = ps.B, C = n.w[n.L];
  // The two perturbed passes (x + eps v and x - eps v) share nothing but read-only inputs: each gets buffers of
  // its own, the second runs on the side stream beside the first, and nothing is released before the join.
  const int64_t n_out = wrt->n_params, gstride = (n_out + 63) & ~int64_t(63);
  op16* E[MAXL];
  for (int l = 0; l < n.L; ++l) {
    E[l] = c.arena.alloc<op16>((size_t)(n.w[l + 1] * n.ldw[l]));
    if (!E[l]) return BETTY_ERR_WORKSPACE;
    BETTY_TRY(cast_matrix(c, v + n.woff[l], E[l], n.w[l + 1], n.w[l], n.ldw[l], vnorm2, eps0));
  }
  BETTY_ALLOC(G, float, c, (size_t)(2 * gstride));
  SideWork side(c);
  for (int pass = 0; pass < 2; ++pass) {
    // the side stream's pass is launched first: it starts after what is on the caller's stream at that moment
    const int sgn = 1 - pass;
    const float sign = sgn == 0 ? 1.f : -1.f;
    if (sgn == 1) side.begin();
    // the label-correction net is evaluated at the perturbed last hidden activation, in fp32
    float* hlast_p = nullptr;
    if (P.corr) {
      hlast_p = c.arena.alloc<float>((size_t)((B > 0 ? B : 1) * n.w[n.L - 1]));
      if (!hlast_p) return BETTY_ERR_WORKSPACE;
    }
    BETTY_ALLOC(zpm, float, c, (size_t)(B * C));
    BETTY_ALLOC(s1, float, c, (size_t)(B > 0 ? B : 1));
    Pass pp = ps;   // perturbed pass: reuses y/B, gets its own p/ell
    BETTY_ALLOC(p2, float, c, (size_t)(B * C));
    BETTY_ALLOC(ell2, float, c, (size_t)(B > 0 ? B : 1));
    pp.p = p2; pp.ell = ell2;
    const op16* hp = ps.h[0];      // perturbed input of the layer (layer 0: the data itself)
    const op16* dh = nullptr;      // its difference from the base input
    for (int l = 0; l < n.L; ++l) {
      const int64_t N = n.w[l + 1], K = n.w[l];
      BETTY_ALLOC(da, float, c, (size_t)(B * N));
      GemmDesc g = {}; g.M = (int)B; g.N = (int)N; g.C = da; g.ldc = N; g.beta = 0.f; g.npairs = 0;
      g.p[g.npairs++] = gemm_pair(hp, ps.ldh[l], false, E[l], n.ldw[l], true, (int)K, sign);
      if (l > 0) g.p[g.npairs++] = gemm_pair(dh, ps.ldh[l], false, n.W[l], n.ldw[l], true, (int)K);
      BETTY_TRY(gemm(c, g));
      if (l < n.L - 1) {
        const size_t cnt = (size_t)(B * ps.ldh[l + 1]);
        BETTY_ALLOC(hn, op16, c, cnt);
        BETTY_ALLOC(dn, op16, c, cnt);
        if (ps.ldh[l + 1] != N) {
          BETTY_TRY(vec_zero(c, (float*)hn, (int64_t)(cnt) / 2));
          BETTY_TRY(vec_zero(c, (float*)dn, (int64_t)(cnt) / 2));
        }
        launch_pdl(k_fd_act, dim3(grid_for(B * N)), dim3(256), 0, c.stream, ps.a[l], da, v + n.boff[l], vnorm2, eps0, sign, hn, dn, nullptr, B, N,
                                                       ps.ldh[l + 1], n.act, (P.corr && l == n.L - 2) ? hlast_p : (float*)nullptr);
        BETTY_LAUNCH_CHECK();
        hp = hn; dh = dn;
      } else {
        launch_pdl(k_fd_act, dim3(grid_for(B * N)), dim3(256), 0, c.stream, ps.a[l], da, v + n.boff[l], vnorm2, eps0, sign, nullptr, nullptr, zpm,
                                                       B, N, 0, n.act, (float*)nullptr);
        BETTY_LAUNCH_CHECK();
      }
    }
    launch_pdl(k_softmax_ce, dim3(grid_for(B * 32)), dim3(256), 0, c.stream, zpm, ps.y, pp.p, pp.ell, B, C);
    BETTY_LAUNCH_CHECK();
    CorrPass cpp;
    if (P.corr) BETTY_TRY(corr_forward(c, n, pp, P.corr, cpp, hlast_p, zpm));     // pp.ell: soft-label losses at x +- eps v
    if (wrt_theta) {
      BETTY_TRY(wn_sample(c, WN_REWEIGHT_TGRAD, P.theta, nullptr, pp, nullptr, nullptr, s1, nullptr));
      BETTY_TRY(wn_backward(c, P.theta, nullptr, pp, s1, nullptr, 0.f, nullptr, G + gstride * sgn, false, 1.f, true));
    } else {
      const float* coefp;
      BETTY_TRY(reweight_coef(c, P, pp, &coefp));
      float* G32; op16* G16; int64_t ldg;
      BETTY_TRY(corr_sample_grad(c, 0, cpp, pp, coefp, &G32, &G16, &ldg));
      BETTY_TRY(corr_param_grad(c, cpp, pp, G32, G + gstride * sgn));
    }
    if (sgn == 1) side.end();
  }
  BETTY_TRY(side.join());
  launch_pdl(k_fd_combine, dim3(grid_for(n_out)), dim3(256), 0, c.stream, out, G, G + gstride, vnorm2, eps0, alpha, accumulate ? 1 : 0, n_out);
  BETTY_LAUNCH_CHECK();
  c.arena.release(mark);
  return BETTY_OK;
}

}  // namespace BETTY_FAM
}  // namespace betty
