// Matrix products for the MLP families: dispatcher and the CUDA-core path.
#include "gemm.cuh"

namespace betty {

static constexpr int GT = 64;   // C tile edge
static constexpr int GK = 16;   // K slab

__global__ void __launch_bounds__(256) k_gemm_simt(GemmDesc g) {
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
          v = __bfloat162float(p.ta ? p.A[(int64_t)(k0 + k) * p.lda + m0 + m] : p.A[(int64_t)(m0 + m) * p.lda + k0 + k]);
        As[k][m] = v * p.alpha;
        int n;
        if (p.tb) { int idx = tid * 4 + j; n = idx >> 4; k = idx & 15; }
        else { int idx = tid + j * 256; n = idx & 63; k = idx >> 6; }
        v = 0.f;
        if (n0 + n < g.N && k0 + k < p.K)
          v = __bfloat162float(p.tb ? p.B[(int64_t)(n0 + n) * p.ldb + k0 + k] : p.B[(int64_t)(k0 + k) * p.ldb + n0 + n]);
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
      float* cp = g.C + (int64_t)m * g.ldc + n;
      *cp = acc[i][j] + (g.beta != 0.f ? g.beta * *cp : 0.f);
    }
  }
}

betty_status gemm_simt(Ctx& c, const GemmDesc& g) {
  if (g.M <= 0 || g.N <= 0) return BETTY_OK;
  dim3 grid((unsigned)((g.N + GT - 1) / GT), (unsigned)((g.M + GT - 1) / GT));
  k_gemm_simt<<<grid, 256, 0, c.stream>>>(g);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

betty_status gemm(Ctx& c, const GemmDesc& g) { return gemm_simt(c, g); }

}  // namespace betty
