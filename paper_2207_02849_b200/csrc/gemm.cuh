// op16 x op16 -> fp32 matrix products used by the MLP families (forward, backward and
// R-operator passes).  One call computes  C = sum_p alpha_p * op(A_p) op(B_p) + beta * C  over
// one or two operand pairs: the R-operator needs sums such as Rh W^T + h U^T in one accumulator.
#pragma once
#include "common.cuh"

namespace betty {
namespace BETTY_FAM {

struct GemmPair {
  const op16* A; int64_t lda; bool ta;   // logical A is [M,K]; ta: stored [K,M] (M contiguous)
  const op16* B; int64_t ldb; bool tb;   // logical B is [K,N]; tb: stored [N,K] (K contiguous)
  int K;
  float alpha;
};
// What happens to an accumulator element acc[m,n] on its way out.
enum GemmEpiMode {
  EPI_STORE = 0,     // C = acc + beta*C
  EPI_BIAS_ACT = 1,  // v = acc + bias[n];  C = v;  out16 = act(v)                       (forward layer)
  EPI_ACT_BWD = 2,   // C = acc (if C);     out16 = acc * act'(a[m,n])                   (backward through an activation)
  EPI_R_FWD = 3,     // v = acc + bias[n];  C = v;  out16 = act'(a[m,n]) * v             (R-operator forward)
  EPI_R_BWD = 4,     // out16 = acc * act'(a) + dh * act''(a) * Ra                       (R-operator backward)
  EPI_SGD = 5,       // g = acc + exp(lam) * w16;  C = C - lr * g;  out16 = op16(new C)  (weight gradient -> gradient step; w16 == op16(C))
  EPI_NEUMANN = 6    // Hu = acc + exp(lam) * t_in;  C = s_in + t_in - alpha * Hu;  out16 = op16(C) if given   (weight HVP -> one Horner step of the Neumann series)
};
struct GemmEpilogue {
  int mode;
  int act;                 // betty_activation
  const float* bias;       // [N]
  const float* a;          // [M,N] pre-activations, leading dimension N
  const float* dh;         // [M,N]
  const float* Ra;         // [M,N]
  op16* out16;             // [M, ld16] or null
  int64_t ld16;
  // EPI_SGD / EPI_NEUMANN (all [M,N] with the leading dimension of C unless noted)
  const float* lam;        // device scalar: log weight decay of this layer, or null
  const op16* w16;         // EPI_SGD: op16 weights the gradient was taken at, leading dimension ldw16
  int64_t ldw16;
  float step;              // EPI_SGD: learning rate; EPI_NEUMANN: alpha
  const float* t_in;       // EPI_NEUMANN: the HVP direction = the partial sum so far (may alias C)
  const float* s_in;       // EPI_NEUMANN: the series' constant term v
};
struct GemmDesc {
  int M, N;
  int npairs;
  GemmPair p[2];
  float* C; int64_t ldc;   // may be null for EPI_ACT_BWD / EPI_R_BWD
  float beta;
  GemmEpilogue epi;        // zero-initialise for a plain store
};

// ---- activation functions shared by the matrix-product epilogues and the row kernels ----
// Standard normal density and distribution function.  The distribution function uses the rational
// approximation 7.1.26 of Abramowitz & Stegun for erf (|error| <= 1.5e-7, far below the op16 rounding of
// every quantity it feeds): no branches, one reciprocal and one exponential, and exp(-x^2) with
// x = a / sqrt(2) is the density's own exponential, so a kernel that needs both evaluates it once.
__device__ __forceinline__ float norm_pdf(float a) { return 0.3989422804014327f * __expf(-0.5f * a * a); }
__device__ __forceinline__ float norm_cdf(float a) {
  const float x = a * 0.7071067811865476f;
  const float t = __fdividef(1.f, fmaf(0.3275911f, fabsf(x), 1.f));
  float p = fmaf(1.061405429f, t, -1.453152027f);
  p = fmaf(p, t, 1.421413741f);
  p = fmaf(p, t, -0.284496736f);
  p = fmaf(p, t, 0.254829592f);
  const float tail = p * t * __expf(-0.5f * a * a);        // 1 - erf(|x|)
  return a >= 0.f ? 1.f - 0.5f * tail : 0.5f * tail;
}
__device__ __forceinline__ float act_f(int act, float a) { return act == BETTY_ACT_RELU ? fmaxf(a, 0.f) : a * norm_cdf(a); }
__device__ __forceinline__ float act_d1(int act, float a) {
  return act == BETTY_ACT_RELU ? (a > 0.f ? 1.f : 0.f) : norm_cdf(a) + a * norm_pdf(a);
}
__device__ __forceinline__ float act_d2(int act, float a) {
  return act == BETTY_ACT_RELU ? 0.f : norm_pdf(a) * (2.f - a * a);
}

// One output element.  Used as is by the CUDA-core kernel; the tensor-core kernel applies the same
// formulas to 32 consecutive columns of a row at a time.
__device__ __forceinline__ void gemm_epilogue_store(const GemmEpilogue& e, float* C, int64_t ldc, float beta, int N,
                                                    int m, int n, float acc) {
  const int64_t j = (int64_t)m * N + n;
  float* cp = C ? C + (int64_t)m * ldc + n : nullptr;
  switch (e.mode) {
    case EPI_STORE:
      *cp = acc + (beta != 0.f ? beta * *cp : 0.f);
      break;
    case EPI_BIAS_ACT: {
      const float v = acc + e.bias[n];
      *cp = v;
      if (e.out16) e.out16[(int64_t)m * e.ld16 + n] = to_op16(act_f(e.act, v));
      break;
    }
    case EPI_ACT_BWD:
      if (cp) *cp = acc;
      e.out16[(int64_t)m * e.ld16 + n] = to_op16(acc * act_d1(e.act, e.a[j]));
      break;
    case EPI_R_FWD: {
      const float v = acc + e.bias[n];
      *cp = v;
      if (e.out16) e.out16[(int64_t)m * e.ld16 + n] = to_op16(act_d1(e.act, e.a[j]) * v);
      break;
    }
    case EPI_R_BWD: {
      float v = acc * act_d1(e.act, e.a[j]);
      if (e.act != BETTY_ACT_RELU) v += e.dh[j] * act_d2(e.act, e.a[j]) * e.Ra[j];
      e.out16[(int64_t)m * e.ld16 + n] = to_op16(v);
      break;
    }
    case EPI_SGD: {
      float gval = acc;
      if (e.lam) gval += expf(*e.lam) * from_op16(e.w16[(int64_t)m * e.ldw16 + n]);
      const float w = *cp - e.step * gval;
      *cp = w;
      if (e.out16) e.out16[(int64_t)m * e.ld16 + n] = to_op16(w);
      break;
    }
    case EPI_NEUMANN: {
      const int64_t jc = (int64_t)m * ldc + n;
      const float ti = e.t_in[jc];
      float hu = acc;
      if (e.lam) hu += expf(*e.lam) * ti;
      const float tn = e.s_in[jc] + (ti - e.step * hu);
      *cp = tn;
      if (e.out16) e.out16[(int64_t)m * e.ld16 + n] = to_op16(tn);
      break;
    }
  }
}

betty_status gemm(Ctx& c, const GemmDesc& g);
// tcgen05 / tensor-memory path (gemm_tc.cu): needs 16-byte aligned operands, leading dimensions that
// are multiples of 8 elements and alpha = +-1
bool gemm_tc_eligible(const GemmDesc& g);
// tr: keep C transposed in tensor memory (operand roles exchanged) so that the epilogue's global accesses
// coalesce; false: one accumulator row per thread.
betty_status gemm_tc(Ctx& c, const GemmDesc& g, bool tr = true);
betty_status gemm_tc_pair(Ctx& c, const GemmDesc& g, bool tr = true);   // two-SM (cta_group::2) kernel, 256 x 256 tiles
// CUDA-core reference path (any shape, any stride); also the fallback for shapes the tensor-core
// path does not take.
betty_status gemm_simt(Ctx& c, const GemmDesc& g);

static inline GemmPair gemm_pair(const op16* A, int64_t lda, bool ta, const op16* B, int64_t ldb, bool tb, int K,
                                 float alpha = 1.f) {
  GemmPair p; p.A = A; p.lda = lda; p.ta = ta; p.B = B; p.ldb = ldb; p.tb = tb; p.K = K; p.alpha = alpha;
  return p;
}

}  // namespace BETTY_FAM
}  // namespace betty
