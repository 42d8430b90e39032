// bf16 x bf16 -> fp32 matrix products used by the MLP families (forward, backward and
// R-operator passes).  One call computes  C = sum_p alpha_p * op(A_p) op(B_p) + beta * C  over
// one or two operand pairs: the R-operator needs sums such as Rh W^T + h U^T in one accumulator.
#pragma once
#include "common.cuh"

namespace betty {

struct GemmPair {
  const bf16* A; int64_t lda; bool ta;   // logical A is [M,K]; ta: stored [K,M] (M contiguous)
  const bf16* B; int64_t ldb; bool tb;   // logical B is [K,N]; tb: stored [N,K] (K contiguous)
  int K;
  float alpha;
};
struct GemmDesc {
  int M, N;
  int npairs;
  GemmPair p[2];
  float* C; int64_t ldc;
  float beta;
};

betty_status gemm(Ctx& c, const GemmDesc& g);
// tcgen05 / tensor-memory path (gemm_tc.cu): needs 16-byte aligned operands, leading dimensions that
// are multiples of 8 elements and alpha = +-1
bool gemm_tc_eligible(const GemmDesc& g);
betty_status gemm_tc(Ctx& c, const GemmDesc& g);
// CUDA-core reference path (any shape, any stride); also the fallback for shapes the tensor-core
// path does not take.
betty_status gemm_simt(Ctx& c, const GemmDesc& g);

static inline GemmPair gemm_pair(const bf16* A, int64_t lda, bool ta, const bf16* B, int64_t ldb, bool tb, int K,
                                 float alpha = 1.f) {
  GemmPair p; p.A = A; p.lda = lda; p.ta = ta; p.B = B; p.ldb = ldb; p.tb = tb; p.K = K; p.alpha = alpha;
  return p;
}

}  // namespace betty
