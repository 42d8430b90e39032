// Matrix products for the MLP families: dispatcher and the CUDA-core path.
#include "gemm.cuh"

namespace betty {
namespace BETTY_FAM {

static constexpr int GT = 64;   // C tile edge
static constexpr int GK = 16;   // K slab

__global__ void __launch_bounds__(256) k_gemm_simt(GemmDesc g) {
  pdl_enter();
  __shared__ float As[GK][GT + 1];
  __shared__ float Bs[GK][GT + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * GT, n0 = blockIdx.x * GT;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int pi = 0; pi < g.npairs; ++pi) {
    const GemmPair p = g.p[pi];
    for (int k0 = 0; k0 < p.K; k0 += GK) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m, k;
        if (!p.ta) { int idx = tid * 4 + j; m = idx >> 4; k = idx & 15; }
        else { int idx = tid + j * 256; m = idx & 63; k = idx >> 6; }
        float v = 0.f;
        if (m0 + m < g.M && k0 + k < p.K)
          v = from_op16(p.ta ? p.A[(int64_t)(k0 + k) * p.lda + m0 + m] : p.A[(int64_t)(m0 + m) * p.lda + k0 + k]);
        As[k][m] = v * p.alpha;
        int n;
        if (p.tb) { int idx = tid * 4 + j; n = idx >> 4; k = idx & 15; }
        else { int idx = tid + j * 256; n = idx & 63; k = idx >> 6; }
        v = 0.f;
        if (n0 + n < g.N && k0 + k < p.K)
          v = from_op16(p.tb ? p.B[(int64_t)(n0 + n) * p.ldb + k0 + k] : p.B[(int64_t)(k0 + k) * p.ldb + n0 + n]);
        Bs[k][n] = v;
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < GK; ++k) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; b[i] = Bs[k][tx * 4 + i]; }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
      }
      __syncthreads();
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      gemm_epilogue_store(g.epi, g.C, g.ldc, g.beta, g.N, m, n, acc[i][j]);
    }
  }
}

betty_status gemm_simt(Ctx& c, const GemmDesc& g) {
  if (g.M <= 0 || g.N <= 0) return BETTY_OK;
  dim3 grid((unsigned)((g.N + GT - 1) / GT), (unsigned)((g.M + GT - 1) / GT));
  launch_pdl(k_gemm_simt, dim3(grid), dim3(256), 0, c.stream, g);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

int g_gemm_path = 0;   // 0: tensor cores when the operands allow it; 1: CUDA cores always

betty_status gemm(Ctx& c, const GemmDesc& g) {
  if (g_gemm_path == 0 && gemm_tc_eligible(g)) return gemm_tc(c, g);
  return gemm_simt(c, g);
}

}  // namespace BETTY_FAM
}  // namespace betty

#ifndef BETTY_FP16_OPERANDS      // the kernel-level check is offered for the default operand type
using namespace betty;
using namespace betty::BETTY_FAM;

extern "C" betty_status betty_gemm_bf16(int32_t M, int32_t N, int32_t n_pairs, const betty_gemm_operands* pairs,
                                        float* C, int64_t ldc, float beta, int32_t path, void* ws, size_t ws_bytes,
                                        void* stream) {
  if (M < 0 || N < 0 || n_pairs < 1 || n_pairs > 2 || !pairs || (!C && M > 0 && N > 0)) return BETTY_ERR_INVALID_ARG;
  if (!ws || ws_bytes < sizeof(StatusBlock) || (((uintptr_t)ws) & 255u)) return BETTY_ERR_WORKSPACE;
  Ctx c(ws, ws_bytes, stream);
  GemmDesc g = {};
  g.M = M; g.N = N; g.npairs = n_pairs; g.C = C; g.ldc = ldc; g.beta = beta;
  for (int i = 0; i < n_pairs; ++i) {
    const betty_gemm_operands& o = pairs[i];
    if (!o.A || !o.B || o.K < 0) return BETTY_ERR_INVALID_ARG;
    g.p[i] = gemm_pair((const op16*)o.A, o.lda, o.a_transposed != 0, (const op16*)o.B, o.ldb, o.b_transposed != 0, o.K,
                       o.alpha);
  }
  if (path == 1) return gemm_simt(c, g);
  if (path == 2) return gemm_tc_eligible(g) ? gemm_tc(c, g) : BETTY_ERR_UNSUPPORTED;
  if (path == 3) return gemm_tc_eligible(g) ? gemm_tc_pair(c, g) : BETTY_ERR_UNSUPPORTED;
  if (path == 4) return gemm_tc_eligible(g) ? gemm_tc(c, g, false) : BETTY_ERR_UNSUPPORTED;
  if (path == 5) return gemm_tc_eligible(g) ? gemm_tc_pair(c, g, false) : BETTY_ERR_UNSUPPORTED;
  return gemm(c, g);
}
#endif
