// Fused row-streaming pass for the logistic / least-squares cost families (App. D.1 problem):
//   gradient   g  = X^T c(z)        with z = X w,  c_i = -y_i sigmoid(-y_i z_i)/n   (logistic)
//   HVP        Hu = X^T (s(z) . Xu) with s_i = sigmoid(z_i) sigmoid(-z_i)/n         (logistic)
// and the analogous forms for 1/2|Xw-y|^2 (c_i = z_i - y_i, s_i = 1).  X is read from HBM exactly
// once per pass: a tile of rows is brought into shared memory by a bulk asynchronous copy (TMA,
// mbarrier completion), each thread keeps its columns of the tile in registers between the row dot
// products and the scaled accumulation, and per-CTA column sums are reduced in a fixed order by a
// small second kernel that also applies the weight-decay term and, for a lower-level step, the
// gradient-descent update.
#include "ops.cuh"

namespace betty {

static constexpr int LR_THREADS = 256;
static constexpr int LR_R = 2;       // rows per tile
static constexpr int LR_S = 3;       // pipeline stages
static constexpr int LR_WARPS = LR_THREADS / 32;
static constexpr uint32_t SPIN_LIMIT = 1u << 22;

struct LrArgs {
  const float* X; const float* y; int64_t n; int64_t d;
  const float* w; const float* u;
  float* partials;       // [gridDim.x][d]
  float* curv;           // [n] per-row curvature s_i = sigmoid(z_i) sigmoid(-z_i) / n at w: written by an HVP pass
                         // of form LR_HVP (if non-null), read by one of form LR_HVP_CACHED
  int family;            // 0 logistic, 1 least squares
  float inv_n;
  StatusBlock* sb;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within SPIN_LIMIT polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = SPIN_LIMIT) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ float sigmoidf_(float t) { return 1.f / (1.f + __expf(-t)); }

// Forms of the pass.  During one inverse-Hessian solve w does not move, so z = X w and with it the per-row
// curvature are the same in every HVP: the first HVP of a solve leaves the curvature in `curv`, the others read
// it and take one dot product per row instead of two (the cost of a gradient pass).
enum { LR_GRAD = 0, LR_HVP = 1, LR_HVP_CACHED = 2 };

// coefficient multiplying row i in the accumulation
template <bool HVP>
__device__ __forceinline__ float row_coef(int family, float z, float t, float y, float inv_n) {
  if (family == 0) {
    if (HVP) { float s = sigmoidf_(z); return (s * (1.f - s) * inv_n) * t; }     // curvature first: see LR_HVP_CACHED
    return -y * sigmoidf_(-y * z) * inv_n;
  }
  return HVP ? t : (z - y);
}

// NCH: float4 column chunks per thread (d <= 1024*NCH, d % 4 == 0)
template <int NCH, int FORM>
__global__ void __launch_bounds__(LR_THREADS, 2) k_logreg_stream(LrArgs a) {
  constexpr bool HVP = FORM != LR_GRAD;            // a direction u is read
  constexpr bool NEEDZ = FORM != LR_HVP_CACHED;    // z = x . w is formed
  extern __shared__ __align__(128) unsigned char smem[];
  const int64_t d = a.d;
  const int d4 = (int)(d >> 2);
  const size_t tile_floats = (size_t)LR_R * d;
  float* tiles = (float*)smem;
  uint64_t* full = (uint64_t*)(smem + LR_S * tile_floats * sizeof(float));
  float* red = (float*)(full + LR_S);     // [2][LR_WARPS][2*LR_R]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  const int64_t ntiles = (a.n + LR_R - 1) / LR_R;
  if (tid == 0) {
    for (int s = 0; s < LR_S; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // the barriers exist; everything below reads or writes global memory, which the previous kernel of the
  // stream (the reduction that produced w or u) must have finished with
  pdl_enter();

  // w and u were written by an earlier kernel of the same stream: plain (coherent) loads, not the read-only path
  float4 wv[NCH], uv[NCH], acc[NCH];
#pragma unroll
  for (int k = 0; k < NCH; ++k) {
    int c4 = tid + k * LR_THREADS;
    wv[k] = (NEEDZ && c4 < d4) ? *((const float4*)a.w + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
    uv[k] = (HVP && c4 < d4) ? *((const float4*)a.u + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
    acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  }

  auto issue = [&](int s, int64_t t) {
    int64_t rows = a.n - t * LR_R; if (rows > LR_R) rows = LR_R;
    uint32_t bytes = (uint32_t)(rows * d * sizeof(float));
    mbar_expect_tx(&full[s], bytes);
    bulk_load(tiles + (size_t)s * tile_floats, a.X + (size_t)t * LR_R * d, bytes, &full[s]);
  };
  if (tid == 0) {
    for (int s = 0; s < LR_S; ++s) {
      int64_t t = blockIdx.x + (int64_t)s * gridDim.x;
      if (t < ntiles) issue(s, t);
    }
  }

  int buf = 0;
  bool timed_out = false;
  int64_t i = 0;
  for (;; ++i) {
    const int64_t t = blockIdx.x + i * gridDim.x;
    if (t >= ntiles) break;
    const int s = (int)(i % LR_S);
    const uint32_t parity = (uint32_t)((i / LR_S) & 1);
    const bool landed = mbar_wait_bounded(&full[s], parity);
    int rows = (int)((a.n - t * LR_R) < LR_R ? (a.n - t * LR_R) : LR_R);
    const float4* tile4 = (const float4*)(tiles + (size_t)s * tile_floats);
    float4 x[LR_R][NCH];
    float pz[LR_R], pt[LR_R];
#pragma unroll
    for (int r = 0; r < LR_R; ++r) {
      pz[r] = 0.f; pt[r] = 0.f;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        int c4 = tid + k * LR_THREADS;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c4 < d4 && r < rows) v = tile4[(size_t)r * d4 + c4];
        x[r][k] = v;
        if (NEEDZ) pz[r] += v.x * wv[k].x + v.y * wv[k].y + v.z * wv[k].z + v.w * wv[k].w;
        if (HVP) pt[r] += v.x * uv[k].x + v.y * uv[k].y + v.z * uv[k].z + v.w * uv[k].w;
      }
    }
    float* rb = red + buf * (LR_WARPS * 2 * LR_R);
    static_assert(LR_R == 2, "the halving butterfly below is written for two rows per tile");
    // Sums over the warp by a butterfly that halves what a lane keeps at every round where it still holds more than
    // one value: 6 shuffles for the four sums of the full HVP form (20 with one full butterfly per sum), 5 for two.
    if (NEEDZ && HVP) {
      const bool up1 = (lane & 16) != 0, up2 = (lane & 8) != 0;
      // first halving: lanes with bit 4 clear keep row 0's sums, the others row 1's
      float k0 = up1 ? pz[1] : pz[0], k1 = up1 ? pt[1] : pt[0];
      const float s0 = up1 ? pz[0] : pz[1], s1 = up1 ? pt[0] : pt[1];
      k0 += __shfl_xor_sync(0xffffffffu, s0, 16);
      k1 += __shfl_xor_sync(0xffffffffu, s1, 16);
      // second halving: lanes with bit 3 clear keep the x.w sum, the others the x.u sum
      float v = up2 ? k1 : k0;
      v += __shfl_xor_sync(0xffffffffu, up2 ? k0 : k1, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      if ((lane & 7) == 0) rb[warp * 2 * LR_R + 2 * (lane >> 4) + ((lane >> 3) & 1)] = v;
    } else {
      const bool up1 = (lane & 16) != 0;
      const float a0 = NEEDZ ? pz[0] : pt[0], a1 = NEEDZ ? pz[1] : pt[1];
      float v = up1 ? a1 : a0;
      v += __shfl_xor_sync(0xffffffffu, up1 ? a0 : a1, 16);
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      if ((lane & 15) == 0) {
        rb[warp * 2 * LR_R + 2 * (lane >> 4) + (NEEDZ ? 0 : 1)] = v;
        rb[warp * 2 * LR_R + 2 * (lane >> 4) + (NEEDZ ? 1 : 0)] = 0.f;
      }
    }

    // every thread has copied its part of stage s into registers; the same barrier makes the
    // decision about an expired wait uniform across the CTA
    if (__syncthreads_or(!landed)) { timed_out = true; break; }
    if (tid == 0) {
      const int64_t tn = t + (int64_t)LR_S * gridDim.x;
      if (tn < ntiles) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(s, tn);
      }
    }
#pragma unroll
    for (int r = 0; r < LR_R; ++r) {
      float z = 0.f, tt = 0.f;
#pragma unroll
      for (int wi = 0; wi < LR_WARPS; ++wi) { z += rb[wi * 2 * LR_R + 2 * r]; tt += rb[wi * 2 * LR_R + 2 * r + 1]; }
      float c = 0.f;
      if (r < rows) {
        if (FORM == LR_HVP_CACHED) {
          c = (a.family == 0 ? __ldg(a.curv + t * LR_R + r) : 1.f) * tt;
        } else {
          c = row_coef<HVP>(a.family, z, tt, a.family == 0 && HVP ? 0.f : __ldg(a.y + t * LR_R + r), a.inv_n);
          if (FORM == LR_HVP && a.curv && a.family == 0 && tid == r) {
            const float sg = sigmoidf_(z);
            a.curv[t * LR_R + r] = sg * (1.f - sg) * a.inv_n;
          }
        }
      }
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        acc[k].x += c * x[r][k].x; acc[k].y += c * x[r][k].y; acc[k].z += c * x[r][k].z; acc[k].w += c * x[r][k].w;
      }
    }
    buf ^= 1;
  }
  if (timed_out) {
    if (tid == 0) {
      record_status(a.sb, BETTY_ERR_TIMEOUT);
      // give copies that are still in flight a bounded chance to land before the CTA exits
      for (int64_t j = i; j < i + LR_S; ++j) {
        if (blockIdx.x + j * gridDim.x >= ntiles) break;
        (void)mbar_wait_bounded(&full[j % LR_S], (uint32_t)((j / LR_S) & 1));
      }
    }
    __syncthreads();
  }
  float4* out4 = (float4*)(a.partials + (size_t)blockIdx.x * d);
#pragma unroll
  for (int k = 0; k < NCH; ++k) {
    int c4 = tid + k * LR_THREADS;
    if (c4 < d4) out4[c4] = acc[k];
  }
}

// ---- fallback for any d (odd widths, d > 4096): two passes over X with plain loads ----
template <bool HVP>
__global__ void k_rowcoef(LrArgs a, float* coef) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t i = warp; i < a.n; i += nwarps) {
    const float* xr = a.X + (size_t)i * a.d;
    float z = 0.f, t = 0.f;
    for (int64_t j = lane; j < a.d; j += 32) {
      float xv = xr[j];
      z += xv * a.w[j];
      if (HVP) t += xv * a.u[j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      z += __shfl_xor_sync(0xffffffffu, z, o);
      if (HVP) t += __shfl_xor_sync(0xffffffffu, t, o);
    }
    if (lane == 0) coef[i] = row_coef<HVP>(a.family, z, t, a.family == 0 && HVP ? 0.f : a.y[i], a.inv_n);
  }
}
__global__ void k_colacc(LrArgs a, const float* coef) {
  const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const int64_t rows_per = (a.n + gridDim.y - 1) / gridDim.y;
  const int64_t r0 = blockIdx.y * rows_per;
  int64_t r1 = r0 + rows_per; if (r1 > a.n) r1 = a.n;
  if (j >= a.d) return;
  float acc = 0.f;
  for (int64_t i = r0; i < r1; ++i) acc += coef[i] * a.X[(size_t)i * a.d + j];
  a.partials[(size_t)blockIdx.y * a.d + j] = acc;
}

// out_j = sum_c partials[c][j] + lam_j * vec_j ; optionally w_j <- w_j - lr * (that).
// TAIL selects what else happens to the finished vector h (see LrTail): nothing; one term/sum update of the
// Neumann series, elementwise, by the thread that owns the column; or one whole conjugate-gradient iteration,
// done by the block that draws the last ticket once every block has stored its part of h.  The iteration's
// arithmetic and its order of additions depend only on d, so results repeat bit for bit.
template <int TAIL>
__global__ void k_logreg_finalize(const float* partials, int nparts, int64_t d, const float* lam, const float* vec,
                                  float* out, float* w_update, float lr, LrTail tl, StatusBlock* sb) {
  pdl_enter();
  __shared__ float sh[8][32];
  __shared__ double shd[8];
  __shared__ int last_block;
  const int cx = threadIdx.x & 31, sl = threadIdx.x >> 5;
  const int64_t j = blockIdx.x * 32 + cx;
  float acc = 0.f;
  if (j < d) {
    const int per = (nparts + 7) / 8;
    const int c0 = sl * per, c1 = min(nparts, c0 + per);
    // same order of additions as a plain loop; eight loads are in flight at a time (the kernel is latency-bound)
    for (int c = c0; c < c1; c += 8) {
      float v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = c + k < c1 ? __ldcg(partials + (size_t)(c + k) * d + j) : 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) acc += v[k];
    }
  }
  sh[sl][cx] = acc;
  __syncthreads();
  double ph = 0.0;          // CG: this column's term of p . h
  if (sl == 0 && j < d) {
    float g = 0.f;
#pragma unroll
    for (int s = 0; s < 8; ++s) g += sh[s][cx];
    const float vj = (lam || TAIL != LR_TAIL_NONE) ? vec[j] : 0.f;
    if (lam) g += lam[j] * vj;
    if (out) out[j] = g;
    if (w_update) w_update[j] = w_update[j] - lr * g;
    if (TAIL == LR_TAIL_NEUMANN) {
      const float tn = vj - tl.alpha * g;
      const float sn = tl.s_in[j] + tn;
      tl.t_out[j] = tn;
      tl.s_out[j] = sn;
    }
    if (TAIL == LR_TAIL_CG) ph = (double)vj * (double)g;
  }
  if (TAIL != LR_TAIL_CG) return;
  // ---- conjugate gradient: gamma = p . h in fixed order, then the update by the last block
  if (sl == 0) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ph += __shfl_xor_sync(0xffffffffu, ph, o);
    if (cx == 0) {
      tl.partials[blockIdx.x] = ph;
      __threadfence();
      last_block = atomicAdd(tl.counter, 1u) == gridDim.x - 1 ? 1 : 0;
    }
  }
  __syncthreads();
  if (!last_block) return;
  __threadfence();
  SolveState* st = tl.st;
  __shared__ int s_active;
  __shared__ float s_rho;
  if (threadIdx.x == 0) { *tl.counter = 0u; s_active = st->active; s_rho = st->rho; }
  __syncthreads();
  if (!s_active) return;                         // the solve has stopped: h was stored, nothing else moves
  // gamma: the per-block terms, a few per thread in index order, then a fixed tree (warp shuffles, warps in order):
  // the order depends on the grid alone, and every thread ends with the same value
  double gsum = 0.0;
  for (unsigned i = threadIdx.x; i < gridDim.x; i += blockDim.x) gsum += __ldcg(tl.partials + i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gsum += __shfl_xor_sync(0xffffffffu, gsum, o);
  if (cx == 0) shd[sl] = gsum;
  __syncthreads();
  gsum = 0.0;
  for (int i = 0; i < 8; ++i) gsum += shd[i];
  __syncthreads();
  const float gamma = (float)gsum;
  if (!isfinite(gsum) || !(gsum > 0.0)) {
    if (threadIdx.x == 0) {
      st->gamma = gamma;
      record_status(sb, !isfinite(gsum) ? BETTY_ERR_NONFINITE : BETTY_ERR_BREAKDOWN);
      st->active = 0;
    }
    return;
  }
  const float rho = s_rho;
  const float a = rho / gamma;
  const float* h = out;
  double rr = 0.0;
  // one block walks the whole vector: eight elements per thread at a time, every load of a batch issued before its
  // first use (the loop is bound by load latency, not by bytes)
  constexpr int TB = 8;
  for (int64_t base = 0; base < d; base += (int64_t)blockDim.x * TB) {
    float pv[TB], qv[TB], rv[TB], hv[TB];
#pragma unroll
    for (int k = 0; k < TB; ++k) {
      const int64_t i = base + threadIdx.x + (int64_t)k * blockDim.x;
      const bool in = i < d;
      pv[k] = in ? tl.p[i] : 0.f; qv[k] = in ? tl.q[i] : 0.f; rv[k] = in ? tl.r[i] : 0.f; hv[k] = in ? __ldcg(h + i) : 0.f;
    }
#pragma unroll
    for (int k = 0; k < TB; ++k) {
      const int64_t i = base + threadIdx.x + (int64_t)k * blockDim.x;
      if (i < d) {
        tl.q[i] = qv[k] + a * pv[k];
        const float ri = rv[k] - a * hv[k];
        tl.r[i] = ri;
        rr += (double)ri * (double)ri;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) rr += __shfl_xor_sync(0xffffffffu, rr, o);
  if (cx == 0) shd[sl] = rr;
  __syncthreads();
  double rsum = 0.0;
  for (int i = 0; i < 8; ++i) rsum += shd[i];
  const float rho_new = (float)rsum;
  const float beta = rho_new / rho;
  for (int64_t base = 0; base < d; base += (int64_t)blockDim.x * TB) {
    float pv[TB], rv[TB];
#pragma unroll
    for (int k = 0; k < TB; ++k) {
      const int64_t i = base + threadIdx.x + (int64_t)k * blockDim.x;
      pv[k] = i < d ? tl.p[i] : 0.f; rv[k] = i < d ? tl.r[i] : 0.f;      // r: this thread's own stores of the loop above
    }
#pragma unroll
    for (int k = 0; k < TB; ++k) {
      const int64_t i = base + threadIdx.x + (int64_t)k * blockDim.x;
      if (i < d) tl.p[i] = rv[k] + beta * pv[k];
    }
  }
  if (threadIdx.x == 0) {
    st->gamma = gamma;
    st->rho_new = rho_new;
    st->rho = rho_new;
    st->iters += 1;
    sb->cg_iters = st->iters;
    if (!isfinite(rho_new)) { record_status(sb, BETTY_ERR_NONFINITE); st->active = 0; }
    else if (rho_new <= st->stop) st->active = 0;
  }
}

int64_t logreg_tail_max_d() { return 32 * 592; }     // one double per 32 columns in a 592-entry reduction buffer

static betty_status launch_finalize(Ctx& c, const float* partials, int nparts, int64_t d, const float* lam, const float* vec,
                                    float* out, float* w_update, float lr, const LrTail* tail) {
  LrTail tl = {};
  if (tail) tl = *tail;
  const dim3 grid((unsigned)((d + 31) / 32)), block(256);
  StatusBlock* sb = c.arena.status();
  if (tl.kind == LR_TAIL_CG) launch_pdl(k_logreg_finalize<LR_TAIL_CG>, grid, block, 0, c.stream, partials, nparts, d, lam, vec, out, w_update, lr, tl, sb);
  else if (tl.kind == LR_TAIL_NEUMANN) launch_pdl(k_logreg_finalize<LR_TAIL_NEUMANN>, grid, block, 0, c.stream, partials, nparts, d, lam, vec, out, w_update, lr, tl, sb);
  else launch_pdl(k_logreg_finalize<LR_TAIL_NONE>, grid, block, 0, c.stream, partials, nparts, d, lam, vec, out, w_update, lr, tl, sb);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

template <int NCH, int FORM>
static betty_status launch_stream(Ctx& c, const LrArgs& a, int grid) {
  size_t smem = (size_t)LR_S * LR_R * a.d * sizeof(float) + LR_S * sizeof(uint64_t) + 2 * LR_WARPS * 2 * LR_R * sizeof(float);
  auto kern = k_logreg_stream<NCH, FORM>;
  static SmemLimit limit = {};      // per instantiation and per device; raised again if a wider problem comes
  BETTY_TRY(ensure_dynamic_smem(kern, limit, smem));
  launch_pdl(kern, dim3(grid), dim3(LR_THREADS), smem, c.stream, a);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// One streaming pass.  u == nullptr: gradient form, else HVP form.  lam (nullable) adds lam.*w
// (gradient) or lam.*u (HVP).  out (nullable) receives the vector; w_update (nullable) is
// decremented by lr times it.
betty_status logreg_pass(Ctx& c, int family, const float* X, const float* y, int64_t n, int64_t d, const float* w,
                         const float* u, const float* lam, float* out, float* w_update, float lr, float* curv,
                         bool* curv_valid, const LrTail* tail) {
  if (d <= 0) return BETTY_OK;
  LrArgs a;
  a.X = X; a.y = y; a.n = n; a.d = d; a.w = w; a.u = u; a.family = family;
  a.inv_n = n > 0 ? 1.0f / (float)n : 0.f;
  a.sb = c.arena.status();
  a.curv = (u && curv_valid) ? curv : nullptr;
  const size_t mark = c.arena.mark();
  int nparts;
  const bool fast = (d % 4 == 0) && d <= 4096 && aligned16(X) && aligned16(w) && (!u || aligned16(u));
  if (fast) {
    const int64_t ntiles = (n + LR_R - 1) / LR_R;
    int grid = 2 * c.sm_count;
    if (ntiles < grid) grid = ntiles > 0 ? (int)ntiles : 1;
    nparts = grid;
    BETTY_ALLOC(partials, float, c, (size_t)grid * d);
    a.partials = partials;
    betty_status s;
    const int form = !u ? LR_GRAD : (a.curv && *curv_valid) ? LR_HVP_CACHED : LR_HVP;
    if (d <= 1024) s = form == LR_GRAD ? launch_stream<1, LR_GRAD>(c, a, grid) : form == LR_HVP ? launch_stream<1, LR_HVP>(c, a, grid) : launch_stream<1, LR_HVP_CACHED>(c, a, grid);
    else if (d <= 2048) s = form == LR_GRAD ? launch_stream<2, LR_GRAD>(c, a, grid) : form == LR_HVP ? launch_stream<2, LR_HVP>(c, a, grid) : launch_stream<2, LR_HVP_CACHED>(c, a, grid);
    else s = form == LR_GRAD ? launch_stream<4, LR_GRAD>(c, a, grid) : form == LR_HVP ? launch_stream<4, LR_HVP>(c, a, grid) : launch_stream<4, LR_HVP_CACHED>(c, a, grid);
    BETTY_TRY(s);
    if (form == LR_HVP && a.curv && family == 0) *curv_valid = true;     // this launch wrote the curvature
  } else {
    int64_t want = (n + 255) / 256; if (want < 1) want = 1; if (want > 64) want = 64;
    nparts = (int)want;
    BETTY_ALLOC(partials, float, c, (size_t)nparts * d);
    BETTY_ALLOC(coef, float, c, (size_t)(n > 0 ? n : 1));
    a.partials = partials;
    int rb = (int)((n + 7) / 8); if (rb < 1) rb = 1; if (rb > 148 * 8) rb = 148 * 8;
    if (u) k_rowcoef<true><<<rb, 256, 0, c.stream>>>(a, coef); else k_rowcoef<false><<<rb, 256, 0, c.stream>>>(a, coef);
    BETTY_LAUNCH_CHECK();
    dim3 g((unsigned)((d + 255) / 256), (unsigned)nparts);
    k_colacc<<<g, 256, 0, c.stream>>>(a, coef);
    BETTY_LAUNCH_CHECK();
  }
  if (tail && tail->kind != LR_TAIL_NONE && (!u || !out)) return BETTY_ERR_INVALID_ARG;   // tails act on an HVP's result
  BETTY_TRY(launch_finalize(c, a.partials, nparts, d, lam, u ? u : w, out, w_update, lr, tail));
  c.arena.release(mark);
  return BETTY_OK;
}

}  // namespace betty

// ------------------------------------------------------------------ bounded-wait self test
// A wait that nothing will ever satisfy: the same bounded mbarrier wait the streaming kernel uses must
// give up, record BETTY_ERR_TIMEOUT in the status block and let the kernel return normally.
namespace betty {
__global__ void k_wait_that_expires(StatusBlock* sb) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_bounded(&bar, 0, 1u << 15)) record_status(sb, BETTY_ERR_TIMEOUT);   // short limit: well under a second
  }
}
}  // namespace betty

extern "C" betty_status betty_selftest_wait_timeout(void* ws, size_t ws_bytes, void* stream) {
  using namespace betty;
  if (!ws || ws_bytes < sizeof(StatusBlock) || (((uintptr_t)ws) & 255u)) return BETTY_ERR_WORKSPACE;
  k_wait_that_expires<<<1, 32, 0, (cudaStream_t)stream>>>((StatusBlock*)ws);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

// ------------------------------------------------------------------ allocation-free HVP
// Scratch that belongs to the library image itself: every GPU that loads the library holds
// these bytes until the process exits.  Layout: [StatusBlock (256 B)][per-CTA column sums].
namespace betty {
static constexpr int NOALLOC_MAX_D = 4096;
static constexpr int NOALLOC_MAX_CTAS = 2 * 148;
static constexpr size_t NOALLOC_FLOATS = sizeof(StatusBlock) / sizeof(float) + (size_t)NOALLOC_MAX_CTAS * NOALLOC_MAX_D;
static __device__ __align__(256) float g_noalloc_scratch[NOALLOC_FLOATS];
static constexpr int NOALLOC_MAX_DEVICES = 64;
static float* g_noalloc_ptr[NOALLOC_MAX_DEVICES];   // device address of the array, per device ordinal

__global__ void k_noalloc_report(const StatusBlock* sb, int32_t* status_dev) {
  if (threadIdx.x == 0 && blockIdx.x == 0) *status_dev = sb->code;
}
}  // namespace betty

extern "C" betty_status betty_hvp_logreg_static(const float* X, int64_t n, int64_t d, const float* w,
                                                const float* lam, const float* u, float* Hu,
                                                int32_t* status_dev, void* stream) {
  using namespace betty;
  if (n < 0 || d <= 0) return BETTY_ERR_SHAPE;
  if (!w || !lam || !u || !Hu || (n > 0 && !X)) return BETTY_ERR_INVALID_ARG;
  if (d > NOALLOC_MAX_D) return BETTY_ERR_CAPACITY;          // beyond the fixed scratch
  if (d % 4 != 0) return BETTY_ERR_UNSUPPORTED;               // only the single-pass kernel is offered here
  if (!aligned16(X) || !aligned16(w) || !aligned16(u) || !aligned16(Hu)) return BETTY_ERR_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return BETTY_ERR_CUDA;
  if (!g_noalloc_ptr[dev]) {
    // In host code the array's name is only a handle; the device address has to be asked for,
    // once per device, with that device current.
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return BETTY_ERR_CUDA;
    }
    g_noalloc_ptr[dev] = p;
  }
  float* base = g_noalloc_ptr[dev];
  cudaStream_t s = (cudaStream_t)stream;
  // the status block is the only part that must start at zero: every per-CTA row that the
  // reduction reads is rewritten by this call's streaming kernel
  if (cudaMemsetAsync(base, 0, sizeof(StatusBlock), s) != cudaSuccess) return BETTY_ERR_CUDA;
  Ctx c(base, NOALLOC_FLOATS * sizeof(float), stream);
  LrArgs a;
  a.X = X; a.y = nullptr; a.n = n; a.d = d; a.w = w; a.u = u; a.family = 0;
  a.inv_n = n > 0 ? 1.0f / (float)n : 0.f;
  a.sb = c.arena.status();
  a.partials = base + sizeof(StatusBlock) / sizeof(float);
  const int64_t ntiles = (n + LR_R - 1) / LR_R;
  int grid = 2 * c.sm_count;
  if (grid > NOALLOC_MAX_CTAS) grid = NOALLOC_MAX_CTAS;
  if (ntiles < grid) grid = ntiles > 0 ? (int)ntiles : 1;
  betty_status st;
  a.curv = nullptr;
  if (d <= 1024) st = launch_stream<1, LR_HVP>(c, a, grid);
  else if (d <= 2048) st = launch_stream<2, LR_HVP>(c, a, grid);
  else st = launch_stream<4, LR_HVP>(c, a, grid);
  if (st != BETTY_OK) return st;
  if ((st = launch_finalize(c, a.partials, grid, d, lam, u, Hu, nullptr, 0.f, nullptr)) != BETTY_OK) return st;
  if (status_dev) {
    k_noalloc_report<<<1, 32, 0, s>>>(a.sb, status_dev);
    BETTY_LAUNCH_CHECK();
  }
  return BETTY_OK;
}
