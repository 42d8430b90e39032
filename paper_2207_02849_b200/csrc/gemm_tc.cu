// Tensor-core matrix products for sm_100a: tcgen05.mma with the accumulator in tensor memory,
// operands staged in shared memory by TMA (cp.async.bulk.tensor, 128-byte swizzle), an mbarrier
// pipeline between one producer thread, one MMA-issuing thread and four epilogue warps.
//
//   C[M,N] (fp32) = sum over 1..2 operand pairs of (+/-) op(A) op(B)  (+ beta * C)
//
// Each operand may be K-major (K contiguous in memory) or MN-major (M or N contiguous): forward
// passes are K-major x K-major, backward-data passes K-major x N-major, weight-gradient passes
// M-major x N-major.  Ragged M, N and K are handled by TMA's zero fill and predicated stores.
// Every CTA issues plain TMA loads for its own operand slabs.
#include <cuda.h>
#include "gemm.cuh"

namespace betty {
namespace BETTY_FAM {

static constexpr int TC_BM = 128;
static constexpr int TC_BK = 64;            // 64 op16 = one 128-byte swizzle row
static constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;
static constexpr uint32_t TC_SPIN = 1u << 24;
static constexpr int TC_THREADS = 320;      // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
static constexpr int TC_EPI_WARPS = 8;      // two warps per accumulator lane quarter, each takes half of the columns
template <int BN> struct TcCfg {
  static constexpr int B_BYTES = BN * TC_BK * 2;
  static constexpr int STAGE_BYTES = TC_A_BYTES + B_BYTES;
  static constexpr int STAGES = BN == 256 ? 4 : (BN == 128 ? 6 : 8);     // 192 KB of stages in every case
  static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
  static constexpr int TMEM_COLS = 2 * BN;  // two accumulators: the epilogue of one tile overlaps the next tile's MMAs
};

struct TcPair { int K; int a_mn; int b_mn; int neg; };
struct TcArgs {
  int M, N, npairs;
  TcPair p[2];
  float* C; int64_t ldc; float beta;
  GemmEpilogue epi;
  int vec_ok;            // every pointer the epilogue touches is 16-byte aligned and N, ldc, ld16 allow vector access
  int tr;                // the accumulator holds C transposed: lane = column of C, accumulator column = row of C
  int pf_ok;             // transposed mode: the epilogue's fp32 inputs are pulled into L2 one tile ahead
  StatusBlock* sb;
};

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void tc_mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool tc_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(s_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Gives up early when another role has already raised the abort flag.
__device__ __forceinline__ bool tc_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < TC_SPIN; ++i) {
    if (tc_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(s_u32(dst)), "l"(tm), "r"(x), "r"(y), "r"(s_u32(bar)) : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte
// offsets in 16-byte units, descriptor version 1 (bits 46-47), layout type 2 (bits 61-63).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor for kind::f16: fp32 accumulator, op16 operands, majors, optional negation of A.
__device__ __forceinline__ uint32_t instr_desc(int a_mn, int b_mn, int neg_a, int n, int m) {
  uint32_t d = 0;
  d |= 1u << 4;                 // D format: F32
#ifndef BETTY_FP16_OPERANDS
  d |= 1u << 7;                 // A format: BF16 (0: F16)
  d |= 1u << 10;                // B format: BF16 (0: F16)
#endif
  d |= (uint32_t)(neg_a & 1) << 13;
  d |= (uint32_t)(a_mn & 1) << 15;
  d |= (uint32_t)(b_mn & 1) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(m >> 4) << 24;
  return d;
}

__device__ __forceinline__ void tc_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_u32(bar)) : "memory");
}

// 32 consecutive accumulator columns of this thread's lane
__device__ __forceinline__ void tmem_load32(uint32_t (&r)[32], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Epilogue of row m, columns nb .. nb+31 (accumulator bits in r)
__device__ __forceinline__ void epilogue_row32(const TcArgs& g, int m, int nb, const uint32_t (&r)[32]) {
  const GemmEpilogue& e = g.epi;
  if (g.vec_ok && nb + 32 <= g.N) {
    float* crow = g.C ? g.C + (int64_t)m * g.ldc + nb : nullptr;
    const int64_t jb = (int64_t)m * g.N + nb;
    op16* orow = e.out16 ? e.out16 + (int64_t)m * e.ld16 + nb : nullptr;
#pragma unroll
    for (int j8 = 0; j8 < 32; j8 += 8) {
      float v[8], o[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) { v[k] = __uint_as_float(r[j8 + k]); o[k] = 0.f; }
      if (e.mode == EPI_STORE) {
        if (g.beta != 0.f) {
          const float4 c0 = *(const float4*)(crow + j8), c1 = *(const float4*)(crow + j8 + 4);
          v[0] += g.beta * c0.x; v[1] += g.beta * c0.y; v[2] += g.beta * c0.z; v[3] += g.beta * c0.w;
          v[4] += g.beta * c1.x; v[5] += g.beta * c1.y; v[6] += g.beta * c1.z; v[7] += g.beta * c1.w;
        }
      } else if (e.mode == EPI_BIAS_ACT || e.mode == EPI_R_FWD) {
        const float4 b0 = *(const float4*)(e.bias + nb + j8), b1 = *(const float4*)(e.bias + nb + j8 + 4);
        v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
        v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
        if (orow) {
          if (e.mode == EPI_BIAS_ACT) {
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = act_f(e.act, v[k]);
          } else {
            const float4 a0 = *(const float4*)(e.a + jb + j8), a1 = *(const float4*)(e.a + jb + j8 + 4);
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = act_d1(e.act, av[k]) * v[k];
          }
        }
      } else if (e.mode == EPI_SGD) {
        const float kap = e.lam ? expf(*e.lam) : 0.f;
        const float4 c0 = *(const float4*)(crow + j8), c1 = *(const float4*)(crow + j8 + 4);
        const float cv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        float wv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (e.lam) {
          const uint4 wq = *(const uint4*)(e.w16 + (int64_t)m * e.ldw16 + nb + j8);
          const op16x2* wp = (const op16x2*)&wq;
#pragma unroll
          for (int k = 0; k < 4; ++k) { const float2 f = from_op16x2(wp[k]); wv[2 * k] = f.x; wv[2 * k + 1] = f.y; }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) { v[k] = cv[k] - e.step * (v[k] + kap * wv[k]); o[k] = v[k]; }
      } else if (e.mode == EPI_NEUMANN) {
        const float kap = e.lam ? expf(*e.lam) : 0.f;
        const int64_t jc = (int64_t)m * g.ldc + nb + j8;
        const float4 t0 = *(const float4*)(e.t_in + jc), t1 = *(const float4*)(e.t_in + jc + 4);
        const float4 s0 = *(const float4*)(e.s_in + jc), s1 = *(const float4*)(e.s_in + jc + 4);
        const float tv[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
        const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
        for (int k = 0; k < 8; ++k) { v[k] = sv[k] + (tv[k] - e.step * (v[k] + kap * tv[k])); o[k] = v[k]; }
      } else {   // EPI_ACT_BWD, EPI_R_BWD
        const float4 a0 = *(const float4*)(e.a + jb + j8), a1 = *(const float4*)(e.a + jb + j8 + 4);
        const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] = v[k] * act_d1(e.act, av[k]);
        if (e.mode == EPI_R_BWD && e.act != BETTY_ACT_RELU) {
          const float4 d0 = *(const float4*)(e.dh + jb + j8), d1 = *(const float4*)(e.dh + jb + j8 + 4);
          const float4 q0 = *(const float4*)(e.Ra + jb + j8), q1 = *(const float4*)(e.Ra + jb + j8 + 4);
          const float dv[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
          const float qv[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
          for (int k = 0; k < 8; ++k) o[k] += dv[k] * act_d2(e.act, av[k]) * qv[k];
        }
      }
      if (crow && e.mode != EPI_R_BWD) {
        *(float4*)(crow + j8) = make_float4(v[0], v[1], v[2], v[3]);
        *(float4*)(crow + j8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
      }
      if (orow && e.mode != EPI_STORE) {
        op16x2 ob[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) ob[k] = to_op16x2(o[2 * k], o[2 * k + 1]);
        *(uint4*)(orow + j8) = *(uint4*)ob;
      }
    }
  } else {
#pragma unroll   // constant indices keep r in registers
    for (int jj = 0; jj < 32; ++jj)
      if (nb + jj < g.N) gemm_epilogue_store(e, g.C, g.ldc, g.beta, g.N, m, nb + jj, __uint_as_float(r[jj]));
  }
}

// Transposed accumulator (tr): the host swapped the operand roles, so this thread's accumulator lane is
// column n of C and r holds rows mb .. mb+31 of that column.  For a fixed row the 32 lanes of a warp
// touch 32 consecutive elements of C and of every epilogue input: each access is one full 128-byte
// line per warp (64 bytes for the op16 outputs) instead of 32 separate lines.
// C is [MC, NC] = [g.N, g.M] here.  Every load of a batch of rows is issued before the first use: the
// epilogue is bound by bytes in flight per SM (eight warps), so a batch is as deep as the registers
// allow (all 32 rows; 16 when three inputs are read).  Mode and activation are compile-time
// parameters: one compact loop per case.
template <int MODE, int ACT, bool FULL>
__device__ __forceinline__ void epilogue_t32_rows(const TcArgs& g, int n, int mb, const uint32_t (&r)[32]) {
  const GemmEpilogue& e = g.epi;
  const int MC = g.N, NC = g.M;
  constexpr int U = (MODE == EPI_R_BWD && ACT != BETTY_ACT_RELU) ? 16 : 32;
  const float bias = (MODE == EPI_BIAS_ACT || MODE == EPI_R_FWD) ? e.bias[n] : 0.f;
  const float kap = ((MODE == EPI_SGD || MODE == EPI_NEUMANN) && e.lam) ? expf(*e.lam) : 0.f;
  float* cp = g.C ? g.C + (int64_t)mb * g.ldc + n : nullptr;
  const float* ap = e.a ? e.a + (int64_t)mb * NC + n : nullptr;
  const float* dp = e.dh ? e.dh + (int64_t)mb * NC + n : nullptr;
  const float* qp = e.Ra ? e.Ra + (int64_t)mb * NC + n : nullptr;
  const float* tp = e.t_in ? e.t_in + (int64_t)mb * g.ldc + n : nullptr;
  const float* sp = e.s_in ? e.s_in + (int64_t)mb * g.ldc + n : nullptr;
  op16* op = e.out16 ? e.out16 + (int64_t)mb * e.ld16 + n : nullptr;
  const int rows = MC - mb;     // > 0; FULL: >= 32, and no per-row guards, so that the rows' dependency chains interleave
  const bool second = MODE == EPI_R_BWD && ACT != BETTY_ACT_RELU;
#pragma unroll
  for (int j0 = 0; j0 < 32; j0 += U) {
    float x0[U], x1[U], x2[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
      const int j = j0 + k;
      x0[k] = 0.f; x1[k] = 0.f; x2[k] = 0.f;
      if (FULL || j < rows) {
        if (MODE == EPI_STORE) { if (g.beta != 0.f) x0[k] = cp[(int64_t)j * g.ldc]; }
        if (MODE == EPI_R_FWD) { if (op) x0[k] = ap[(int64_t)j * NC]; }
        if (MODE == EPI_ACT_BWD || MODE == EPI_R_BWD) x0[k] = ap[(int64_t)j * NC];
        if (second) { x1[k] = dp[(int64_t)j * NC]; x2[k] = qp[(int64_t)j * NC]; }
        if (MODE == EPI_SGD) x0[k] = cp[(int64_t)j * g.ldc];
        if (MODE == EPI_NEUMANN) { x0[k] = tp[(int64_t)j * g.ldc]; x1[k] = sp[(int64_t)j * g.ldc]; }
      }
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
      const int j = j0 + k;
      if (FULL || j < rows) {
        const float acc = __uint_as_float(r[j]);
        float* c1 = cp + (int64_t)j * g.ldc;
        op16* o1 = op + (int64_t)j * e.ld16;
        if (MODE == EPI_STORE) *c1 = acc + g.beta * x0[k];
        if (MODE == EPI_BIAS_ACT) {
          const float v = acc + bias;
          *c1 = v;
          if (op) *o1 = to_op16(act_f(ACT, v));
        }
        if (MODE == EPI_R_FWD) {
          const float v = acc + bias;
          *c1 = v;
          if (op) *o1 = to_op16(act_d1(ACT, x0[k]) * v);
        }
        if (MODE == EPI_ACT_BWD) {
          if (cp) *c1 = acc;
          *o1 = to_op16(acc * act_d1(ACT, x0[k]));
        }
        if (MODE == EPI_R_BWD) {
          float v = acc * act_d1(ACT, x0[k]);
          if (second) v += x1[k] * act_d2(ACT, x0[k]) * x2[k];
          *o1 = to_op16(v);
        }
        if (MODE == EPI_SGD) {
          // the op16 weights the gradient was taken at (w16) are the rounded master weights: no second read
          const float wq = from_op16(to_op16(x0[k]));
          const float w = x0[k] - e.step * (acc + kap * wq);
          *c1 = w;
          if (op) *o1 = to_op16(w);
        }
        if (MODE == EPI_NEUMANN) {
          const float tn = x1[k] + (x0[k] - e.step * (acc + kap * x0[k]));
          *c1 = tn;
          if (op) *o1 = to_op16(tn);
        }
      }
    }
  }
}
template <int MODE, int ACT>
__device__ __forceinline__ void epilogue_t32_impl(const TcArgs& g, int n, int mb, const uint32_t (&r)[32]) {
  if (g.N - mb >= 32) epilogue_t32_rows<MODE, ACT, true>(g, n, mb, r);
  else epilogue_t32_rows<MODE, ACT, false>(g, n, mb, r);
}
template <int MODE>
__device__ __forceinline__ void epilogue_t32_act(const TcArgs& g, int n, int mb, const uint32_t (&r)[32]) {
  if (g.epi.act == BETTY_ACT_RELU) epilogue_t32_impl<MODE, BETTY_ACT_RELU>(g, n, mb, r);
  else epilogue_t32_impl<MODE, BETTY_ACT_GELU>(g, n, mb, r);
}
__device__ __forceinline__ void epilogue_t32(const TcArgs& g, int n, int mb, const uint32_t (&r)[32]) {
  switch (g.epi.mode) {
    case EPI_STORE: epilogue_t32_impl<EPI_STORE, BETTY_ACT_RELU>(g, n, mb, r); break;
    case EPI_BIAS_ACT: epilogue_t32_act<EPI_BIAS_ACT>(g, n, mb, r); break;
    case EPI_ACT_BWD: epilogue_t32_act<EPI_ACT_BWD>(g, n, mb, r); break;
    case EPI_R_FWD: epilogue_t32_act<EPI_R_FWD>(g, n, mb, r); break;
    case EPI_R_BWD: epilogue_t32_act<EPI_R_BWD>(g, n, mb, r); break;
    case EPI_SGD: epilogue_t32_impl<EPI_SGD, BETTY_ACT_RELU>(g, n, mb, r); break;
    case EPI_NEUMANN: epilogue_t32_impl<EPI_NEUMANN, BETTY_ACT_RELU>(g, n, mb, r); break;
  }
}

// What the MMA-issuing thread needs per operand pair, worked out once per kernel: the issuing thread is a
// single lane, and every instruction it spends between two MMAs is paid in full (measured: with the
// descriptors rebuilt per k-step and the ring position taken by division, one 64-wide slab cost the
// issuer ~800 clocks against the 512 its four MMAs run for).
struct IssuePlan {
  uint64_t a0, b0;            // shared-memory descriptors of stage 0, k-step 0
  uint32_t a_step, b_step;    // descriptor increment per 16-element k-step, in 16-byte units
  uint32_t idesc;
};
__device__ __forceinline__ IssuePlan issue_plan(const TcPair& p, uint32_t sa0, uint32_t sb0, int n, int m) {
  IssuePlan q;
  // K-major: 16 elements = 32 bytes further along the swizzled row; groups of 8 rows 1024 B apart.
  // MN-major: 16 k-rows = 2048 bytes further; 64-element blocks along M/N 8192 B apart.
  q.a0 = p.a_mn ? smem_desc(sa0, 8192, 1024) : smem_desc(sa0, 16, 1024);
  q.b0 = p.b_mn ? smem_desc(sb0, 8192, 1024) : smem_desc(sb0, 16, 1024);
  q.a_step = p.a_mn ? (2048u >> 4) : (32u >> 4);
  q.b_step = p.b_mn ? (2048u >> 4) : (32u >> 4);
  q.idesc = instr_desc(p.a_mn, p.b_mn, p.neg, n, m);
  return q;
}
// Position in the stage ring: stage, how many times the ring has wrapped, and the stage's offset in
// 16-byte units (what is added to a stage-0 descriptor; the address field holds 14 bits and shared
// memory ends below 2^18 bytes, so the sum never carries out of the field).
struct RingPos {
  int s; uint32_t round; uint32_t off16;
  __device__ __forceinline__ void advance(int S, uint32_t stage16) {
    if (++s == S) { s = 0; ++round; off16 = 0; } else off16 += stage16;
  }
};
template <int CG>
__device__ __forceinline__ void mma_f16(uint32_t tmem_acc, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  if (CG == 1)
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_acc), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_acc), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}

// Warms L2 with the fp32 arrays that the epilogue of the tile at kernel coordinates (m0, n0) will read
// (transposed mode: rows n0 .. n0+BN-1 of C, up to 128 columns from m0).  Issued by the 256 epilogue
// threads (e = 0 .. 255, one row each) a whole tile ahead, so that the epilogue's loads find their
// lines in L2 instead of waiting on HBM.  Plain loads of one word per 256 bytes with the 256-byte L2
// prefetch size: measured on this part, prefetch instructions proper (prefetch.global.L2 and the bulk L2
// prefetch) left most later loads at HBM latency, loads with the size hint did not.
__device__ __forceinline__ void l2_touch(const float* p) {
  float v;
  asm volatile("ld.global.L2::256B.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
  (void)v;
}
__device__ __forceinline__ void prefetch_epilogue_inputs(const TcArgs& g, int m0, int n0, int BN, int e) {
  if (!g.pf_ok || m0 >= g.M) return;
  const GemmEpilogue& ep = g.epi;
  const float* pc[2] = {nullptr, nullptr};   // arrays with the leading dimension of C
  const float* pa[3] = {nullptr, nullptr, nullptr};   // arrays stored [MC, NC] densely
  switch (ep.mode) {
    case EPI_STORE: if (g.beta != 0.f) pc[0] = g.C; break;
    case EPI_SGD: pc[0] = g.C; break;
    case EPI_NEUMANN: pc[0] = ep.t_in; pc[1] = ep.s_in; break;
    case EPI_R_FWD: if (ep.out16) pa[0] = ep.a; break;
    case EPI_ACT_BWD: pa[0] = ep.a; break;
    case EPI_R_BWD: pa[0] = ep.a; if (ep.act != BETTY_ACT_RELU) { pa[1] = ep.dh; pa[2] = ep.Ra; } break;
    default: break;
  }
  const int R = n0 + e;
  if (e >= BN || R >= g.N) return;
  const bool two = g.M - m0 > 64;       // the row segment spans a second 256-byte block
#pragma unroll
  for (int i = 0; i < 2; ++i)
    if (pc[i]) {
      const float* p = pc[i] + (int64_t)R * g.ldc + m0;
      l2_touch(p);
      if (two) l2_touch(p + 64);
    }
#pragma unroll
  for (int i = 0; i < 3; ++i)
    if (pa[i]) {
      const float* p = pa[i] + (int64_t)R * g.M + m0;
      l2_touch(p);
      if (two) l2_touch(p + 64);
    }
}

// Persistent kernel: CTA b works on output tiles b, b + gridDim.x, ...
template <int BN>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
          const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1, TcArgs g) {
  using Cfg = TcCfg<BN>;
  constexpr int S = Cfg::STAGES;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + S * Cfg::STAGE_BYTES);
  uint64_t* empty = full + S;
  uint64_t* acc_full = empty + S;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int iters[2] = {0, 0};
  for (int p = 0; p < g.npairs; ++p) iters[p] = (g.p[p].K + TC_BK - 1) / TC_BK;
  const int T = iters[0] + iters[1];
  const int tiles_n = (g.N + BN - 1) / BN;
  const int tiles = tiles_n * ((g.M + TC_BM - 1) / TC_BM);

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { tc_mbar_init(&full[s], 1); tc_mbar_init(&empty[s], 1); }
    for (int s = 0; s < 2; ++s) { tc_mbar_init(&acc_full[s], 1); tc_mbar_init(&acc_empty[s], TC_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {   // one warp allocates the accumulator columns in tensor memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(Cfg::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touched only this CTA's shared and tensor memory and may overlap the previous
  // kernel's tail; global memory (operands, epilogue inputs and outputs) is touched from here on.
  pdl_enter();

  if (warp == 0 && lane == 0 && T > 0) {
    // ---------------- producer: TMA loads into the stage ring
    RingPos r = {0, 0u, 0u};
    long long armed = 0;
    for (int t = blockIdx.x; t < tiles && !*abort_flag; t += gridDim.x) {
      const int m0 = (t / tiles_n) * TC_BM, n0 = (t % tiles_n) * BN;
      int p = 0, k0 = 0;
      const CUtensorMap* ta = &tmA0;
      const CUtensorMap* tb = &tmB0;
      bool a_mn = g.p[0].a_mn, b_mn = g.p[0].b_mn;
      bool ok = true;
      for (int it = 0; it < T; ++it, k0 += TC_BK) {
        if (p == 0 && it == iters[0]) { p = 1; k0 = 0; ta = &tmA1; tb = &tmB1; a_mn = g.p[1].a_mn; b_mn = g.p[1].b_mn; }
        if (r.round && !tc_wait(&empty[r.s], (r.round - 1) & 1u, abort_flag)) { ok = false; break; }
        unsigned char* sa = smem + r.s * Cfg::STAGE_BYTES;
        unsigned char* sb = sa + TC_A_BYTES;
        tc_expect_tx(&full[r.s], Cfg::STAGE_BYTES);
        if (!a_mn) {
          tma_load_2d(sa, ta, k0, m0, &full[r.s]);                                  // box 64(K) x 128(M)
        } else {
          for (int j = 0; j < TC_BM / 64; ++j) tma_load_2d(sa + j * 8192, ta, m0 + 64 * j, k0, &full[r.s]);   // box 64(M) x 64(K)
        }
        if (!b_mn) {
          tma_load_2d(sb, tb, k0, n0, &full[r.s]);                                  // box 64(K) x BN(N)
        } else {
          for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * 8192, tb, n0 + 64 * j, k0, &full[r.s]);      // box 64(N) x 64(K)
        }
        ++armed;
        r.advance(S, Cfg::STAGE_BYTES >> 4);
      }
      if (!ok) break;
    }
    if (*abort_flag) {
      // let copies that were already issued land before the CTA's shared memory goes away
      for (long long i2 = (armed > S ? armed - S : 0); i2 < armed; ++i2)
        for (uint32_t i = 0; i < (1u << 16); ++i)
          if (tc_try_wait(&full[i2 % S], (uint32_t)((i2 / S) & 1))) break;
    }
  } else if (warp == 1 && lane == 0 && T > 0) {
    // ---------------- MMA issuer
    const uint32_t sa0 = s_u32(smem), sb0 = sa0 + TC_A_BYTES;
    const IssuePlan plan0 = issue_plan(g.p[0], sa0, sb0, BN, TC_BM);
    const IssuePlan plan1 = issue_plan(g.p[1], sa0, sb0, BN, TC_BM);
    RingPos r = {0, 0u, 0u};
    int j = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++j) {
      const int as = j & 1;
      if (j >= 2 && !tc_wait(&acc_empty[as], (uint32_t)(((j >> 1) - 1) & 1), abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tmem_acc = tmem_base + (uint32_t)(as * BN);
      for (int it = 0; it < T; ++it) {
        if (!tc_wait(&full[r.s], r.round & 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const IssuePlan& pl = it < iters[0] ? plan0 : plan1;
        uint64_t da = pl.a0 + r.off16, db = pl.b0 + r.off16;
        mma_f16<1>(tmem_acc, da, db, pl.idesc, it > 0 ? 1u : 0u);
#pragma unroll
        for (int kk = 1; kk < TC_BK / 16; ++kk) {
          da += pl.a_step; db += pl.b_step;
          mma_f16<1>(tmem_acc, da, db, pl.idesc, 1u);
        }
        // the stage may be refilled once these MMAs have read it
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s_u32(&empty[r.s])) : "memory");
        r.advance(S, Cfg::STAGE_BYTES >> 4);
      }
      if (ok) asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s_u32(&acc_full[as])) : "memory");
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: warp w may touch accumulator lanes 32*(w%4) .. 32*(w%4)+31
    const int q = warp & 3;
    int j = 0;
    if ((int)blockIdx.x < tiles)
      prefetch_epilogue_inputs(g, ((int)blockIdx.x / tiles_n) * TC_BM, ((int)blockIdx.x % tiles_n) * BN, BN, tid - 64);
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++j) {
      const int m0 = (t / tiles_n) * TC_BM, n0 = (t % tiles_n) * BN;
      const int as = j & 1;
      const int m = m0 + q * 32 + lane;
      if (T > 0) {
        const int tn = t + (int)gridDim.x;    // this CTA's next tile: ask for its inputs one epilogue ahead
        if (tn < tiles) prefetch_epilogue_inputs(g, (tn / tiles_n) * TC_BM, (tn % tiles_n) * BN, BN, tid - 64);
        bool have = tc_wait(&acc_full[as], (uint32_t)((j >> 1) & 1), abort_flag);
        have = __all_sync(0xffffffffu, have);
        if (!have) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int half = (warp - 2) >> 2;           // which half of the tile's columns this warp drains
#pragma unroll 1
        for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
          if (n0 + c * 32 >= g.N) break;            // uniform: nothing to store from these columns
          uint32_t r[32];
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN + c * 32);
          tmem_load32(r, taddr);
          if (m < g.M) {
            if (g.tr) epilogue_t32(g, m, n0 + c * 32, r);
            else epilogue_row32(g, m, n0 + c * 32, r);
          }
        }
        // this warp has drained its quarter of the accumulator: the MMA warp may reuse it
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) tc_arrive(&acc_empty[as]);
      } else if (m < g.M) {
        // no products: the accumulator is zero
        for (int n = n0; n < n0 + BN && n < g.N; ++n) {
          if (g.tr) gemm_epilogue_store(g.epi, g.C, g.ldc, g.beta, g.M, n, m, 0.f);
          else gemm_epilogue_store(g.epi, g.C, g.ldc, g.beta, g.N, m, n, 0.f);
        }
      }
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*abort_flag && tid == 0) record_status(g.sb, BETTY_ERR_TIMEOUT);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------ two-SM variant
// A pair of CTAs (a cluster of two, on the two SMs of one TPC) works on one 256 x 256 output tile
// with tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of A and 128 of the 256 columns
// of B, so every byte of B fetched from L2 feeds twice as many MMA rows as in the one-SM kernel.
// The even CTA of the pair issues the MMAs; each CTA holds the accumulator rows of its own half in
// its tensor memory and runs its own epilogue.  Each CTA loads its own slabs with plain TMA loads.
static constexpr int TC2_BN = 256;           // tile width; each CTA stages half of it
static constexpr int TC2_STAGE_BYTES = TC_A_BYTES + (TC2_BN / 2) * TC_BK * 2;   // 32 KB per CTA
static constexpr int TC2_STAGES = 6;
static constexpr int TC2_SMEM = TC2_STAGES * TC2_STAGE_BYTES + 1024 + 256;

__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* tm, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(s_u32(dst)), "l"(tm), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
// Arrival, once the MMAs issued so far have completed, on the barrier at this shared-memory offset in
// both CTAs of the pair (multicast over the cluster; the mask names CTA ranks 0 and 1).
__device__ __forceinline__ void commit_both(uint32_t bar_local_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar_local_addr), "h"((uint16_t)3) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
k_gemm_tc2(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
           const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1, TcArgs g) {
  constexpr int S = TC2_STAGES;
  constexpr int BN = TC2_BN, HB = TC2_BN / 2;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + S * TC2_STAGE_BYTES);
  uint64_t* empty = full + S;
  uint64_t* acc_full = empty + S;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  int iters[2] = {0, 0};
  for (int p = 0; p < g.npairs; ++p) iters[p] = (g.p[p].K + TC_BK - 1) / TC_BK;
  const int T = iters[0] + iters[1];
  const int tiles_n = (g.N + BN - 1) / BN;
  const int tiles = tiles_n * ((g.M + 2 * TC_BM - 1) / (2 * TC_BM));

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { tc_mbar_init(&full[s], 1); tc_mbar_init(&empty[s], 1); }
    for (int s = 0; s < 2; ++s) { tc_mbar_init(&acc_full[s], 1); tc_mbar_init(&acc_empty[s], 2 * TC_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {   // the same warp of both CTAs allocates the pair's accumulator columns
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(2 * BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();     // the peer's barriers exist before anything is signalled across the pair
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  pdl_enter();            // set-up done; global memory is touched from here on

  if (warp == 0 && lane == 0 && T > 0) {
    // ---------------- producer (both CTAs): own half of A and of B; completion counted on the leader's barrier
    RingPos r = {0, 0u, 0u};
    const uint32_t full0 = map_to_cta(s_u32(&full[0]), 0);      // the leader's full[0]; barriers are 8 bytes apart
    for (int t = cluster_id; t < tiles && !*abort_flag; t += n_clusters) {
      const int m0 = (t / tiles_n) * (2 * TC_BM) + (int)rank * TC_BM, n0 = (t % tiles_n) * BN + (int)rank * HB;
      int p = 0, k0 = 0;
      const CUtensorMap* ta = &tmA0;
      const CUtensorMap* tb = &tmB0;
      bool a_mn = g.p[0].a_mn, b_mn = g.p[0].b_mn;
      bool ok = true;
      for (int it = 0; it < T; ++it, k0 += TC_BK) {
        if (p == 0 && it == iters[0]) { p = 1; k0 = 0; ta = &tmA1; tb = &tmB1; a_mn = g.p[1].a_mn; b_mn = g.p[1].b_mn; }
        if (r.round && !tc_wait(&empty[r.s], (r.round - 1) & 1u, abort_flag)) { ok = false; break; }
        unsigned char* sa = smem + r.s * TC2_STAGE_BYTES;
        unsigned char* sb = sa + TC_A_BYTES;
        const uint32_t bar = full0 + 8u * (uint32_t)r.s;
        if (leader) tc_expect_tx(&full[r.s], 2 * TC2_STAGE_BYTES);
        if (!a_mn) {
          tma_load_2d_pair(sa, ta, k0, m0, bar);
        } else {
          for (int j = 0; j < TC_BM / 64; ++j) tma_load_2d_pair(sa + j * 8192, ta, m0 + 64 * j, k0, bar);
        }
        if (!b_mn) {
          tma_load_2d_pair(sb, tb, k0, n0, bar);
        } else {
          for (int j = 0; j < HB / 64; ++j) tma_load_2d_pair(sb + j * 8192, tb, n0 + 64 * j, k0, bar);
        }
        r.advance(S, TC2_STAGE_BYTES >> 4);
      }
      if (!ok) break;
    }
  } else if (warp == 1 && lane == 0 && T > 0 && leader) {
    // ---------------- MMA issuer (even CTA of the pair only)
    const uint32_t sa0 = s_u32(smem), sb0 = sa0 + TC_A_BYTES;
    const IssuePlan plan0 = issue_plan(g.p[0], sa0, sb0, BN, 2 * TC_BM);
    const IssuePlan plan1 = issue_plan(g.p[1], sa0, sb0, BN, 2 * TC_BM);
    RingPos r = {0, 0u, 0u};
    int j = 0;
    bool ok = true;
    for (int t = cluster_id; t < tiles && ok; t += n_clusters, ++j) {
      const int as = j & 1;
      if (j >= 2 && !tc_wait(&acc_empty[as], (uint32_t)(((j >> 1) - 1) & 1), abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tmem_acc = tmem_base + (uint32_t)(as * BN);
      for (int it = 0; it < T; ++it) {
        if (!tc_wait(&full[r.s], r.round & 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const IssuePlan& pl = it < iters[0] ? plan0 : plan1;
        uint64_t da = pl.a0 + r.off16, db = pl.b0 + r.off16;
        mma_f16<2>(tmem_acc, da, db, pl.idesc, it > 0 ? 1u : 0u);
#pragma unroll
        for (int kk = 1; kk < TC_BK / 16; ++kk) {
          da += pl.a_step; db += pl.b_step;
          mma_f16<2>(tmem_acc, da, db, pl.idesc, 1u);
        }
        // both CTAs may refill the stage once these MMAs have read it: one arrival on empty[s] of each CTA
        commit_both(s_u32(&empty[r.s]));
        r.advance(S, TC2_STAGE_BYTES >> 4);
      }
      if (ok) commit_both(s_u32(&acc_full[as]));
    }
  } else if (warp >= 2) {
    // ---------------- epilogue (both CTAs): own 128 rows of the pair's tile
    const int q = warp & 3;
    int j = 0;
    if (cluster_id < tiles)
      prefetch_epilogue_inputs(g, (cluster_id / tiles_n) * (2 * TC_BM) + (int)rank * TC_BM, (cluster_id % tiles_n) * BN, BN, tid - 64);
    for (int t = cluster_id; t < tiles; t += n_clusters, ++j) {
      const int m0 = (t / tiles_n) * (2 * TC_BM) + (int)rank * TC_BM, n0 = (t % tiles_n) * BN;
      const int as = j & 1;
      const int m = m0 + q * 32 + lane;
      if (T > 0) {
        const int tn = t + n_clusters;
        if (tn < tiles)
          prefetch_epilogue_inputs(g, (tn / tiles_n) * (2 * TC_BM) + (int)rank * TC_BM, (tn % tiles_n) * BN, BN, tid - 64);
        bool have = tc_wait(&acc_full[as], (uint32_t)((j >> 1) & 1), abort_flag);
        have = __all_sync(0xffffffffu, have);
        if (!have) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int half = (warp - 2) >> 2;
#pragma unroll 1
        for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
          if (n0 + c * 32 >= g.N) break;
          uint32_t r[32];
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN + c * 32);
          tmem_load32(r, taddr);
          if (m < g.M) {
            if (g.tr) epilogue_t32(g, m, n0 + c * 32, r);
            else epilogue_row32(g, m, n0 + c * 32, r);
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          const uint32_t bar = map_to_cta(s_u32(&acc_empty[as]), 0);
          asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
        }
      } else if (m < g.M) {
        for (int n = n0; n < n0 + BN && n < g.N; ++n) {
          if (g.tr) gemm_epilogue_store(g.epi, g.C, g.ldc, g.beta, g.M, n, m, 0.f);
          else gemm_epilogue_store(g.epi, g.C, g.ldc, g.beta, g.N, m, n, 0.f);
        }
      }
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();     // neither CTA leaves while the other may still signal its barriers
  if (*abort_flag && tid == 0) record_status(g.sb, BETTY_ERR_TIMEOUT);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn lookup_encode_fn() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return (EncodeTiledFn)p;
  (void)cudaGetLastError();
  return nullptr;
}
static EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = lookup_encode_fn();     // looked up once; the initialisation is thread-safe
  return fn;
}

// 2-D op16 tensor map over a row-major matrix [outer, inner] with leading dimension ld (elements)
static bool make_map(CUtensorMap* tm, const op16* base, int64_t inner, int64_t outer, int64_t ld, int box_inner,
                     int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(op16)};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
#ifdef BETTY_FP16_OPERANDS
  const CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
#else
  const CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
#endif
  return fn(tm, dtype, 2, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool gemm_tc_eligible(const GemmDesc& g) {
  if (g.M <= 0 || g.N <= 0 || g.npairs < 1 || g.npairs > 2) return false;
  for (int i = 0; i < g.npairs; ++i) {
    const GemmPair& p = g.p[i];
    if (p.K <= 0) return false;
    if (p.alpha != 1.f && p.alpha != -1.f) return false;
    if ((((uintptr_t)p.A) & 15) || (((uintptr_t)p.B) & 15)) return false;
    if ((p.lda & 7) || (p.ldb & 7)) return false;
  }
  return encode_fn() != nullptr;
}

static void fill_args(Ctx& c, const GemmDesc& g, TcArgs& a, bool tr);

// C^T = B^T A^T: the same products with the operand roles exchanged.  The kernels then hold C transposed
// in tensor memory (lane = column of C), which is what the coalesced epilogue wants.
static GemmDesc swapped(const GemmDesc& g) {
  GemmDesc s = g;
  s.M = g.N; s.N = g.M;
  for (int i = 0; i < g.npairs; ++i) {
    const GemmPair& p = g.p[i];
    s.p[i] = gemm_pair(p.B, p.ldb, !p.tb, p.A, p.lda, !p.ta, p.K, p.alpha);
  }
  return s;
}

template <int BN>
static betty_status launch_tc(Ctx& c, const GemmDesc& g0, bool tr) {
  using Cfg = TcCfg<BN>;
  const GemmDesc g = tr ? swapped(g0) : g0;
  static SmemLimit limit = {};      // per tile width and per device
  BETTY_TRY(ensure_dynamic_smem(k_gemm_tc<BN>, limit, (size_t)Cfg::SMEM));
  CUtensorMap tm[4];
  TcArgs a;
  fill_args(c, g, a, tr);
  for (int i = 0; i < 2; ++i) {
    const GemmPair& p = g.p[i < g.npairs ? i : 0];
    // A: K-major = stored [M,K]; M-major = stored [K,M]
    bool ok = p.ta ? make_map(&tm[2 * i], p.A, g.M, p.K, p.lda, 64, 64) : make_map(&tm[2 * i], p.A, p.K, g.M, p.lda, TC_BK, TC_BM);
    if (!ok) return BETTY_ERR_CUDA;
    // B: K-major = stored [N,K]; N-major = stored [K,N]
    ok = p.tb ? make_map(&tm[2 * i + 1], p.B, p.K, g.N, p.ldb, TC_BK, BN) : make_map(&tm[2 * i + 1], p.B, g.N, p.K, p.ldb, 64, 64);
    if (!ok) return BETTY_ERR_CUDA;
  }
  const int tiles = ((g.N + BN - 1) / BN) * ((g.M + TC_BM - 1) / TC_BM);
  const int grid = tiles < c.sm_count ? tiles : c.sm_count;
  launch_pdl(k_gemm_tc<BN>, dim3(grid), dim3(TC_THREADS), Cfg::SMEM, c.stream, tm[0], tm[1], tm[2], tm[3], a);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

static void fill_args(Ctx& c, const GemmDesc& g, TcArgs& a, bool tr) {
  a.tr = tr ? 1 : 0;
  a.M = g.M; a.N = g.N; a.npairs = g.npairs; a.C = g.C; a.ldc = g.ldc; a.beta = g.beta; a.sb = c.arena.status();
  a.epi = g.epi;
  auto al16 = [](const void* p) { return (((uintptr_t)p) & 15) == 0; };
  const GemmEpilogue& e = g.epi;
  const bool ok = (g.N % 4 == 0) && al16(g.C) && (g.ldc % 4 == 0) && al16(e.bias) && al16(e.a) && al16(e.dh) && al16(e.Ra) &&
                  al16(e.out16) && (e.ld16 % 8 == 0) && al16(e.w16) && (e.ldw16 % 8 == 0) && al16(e.t_in) && al16(e.s_in);
  a.vec_ok = ok ? 1 : 0;
  a.pf_ok = tr ? 1 : 0;
  for (int i = 0; i < 2; ++i) {
    const GemmPair& p = g.p[i < g.npairs ? i : 0];
    a.p[i].K = i < g.npairs ? p.K : 0;
    a.p[i].a_mn = p.ta ? 1 : 0;
    a.p[i].b_mn = p.tb ? 0 : 1;
    a.p[i].neg = p.alpha < 0.f ? 1 : 0;
  }
}

static betty_status launch_tc2(Ctx& c, const GemmDesc& g0, bool tr) {
  const GemmDesc g = tr ? swapped(g0) : g0;
  static SmemLimit limit = {};      // per device
  BETTY_TRY(ensure_dynamic_smem(k_gemm_tc2, limit, (size_t)TC2_SMEM));
  CUtensorMap tm[4];
  TcArgs a;
  fill_args(c, g, a, tr);
  for (int i = 0; i < 2; ++i) {
    const GemmPair& p = g.p[i < g.npairs ? i : 0];
    bool ok = p.ta ? make_map(&tm[2 * i], p.A, g.M, p.K, p.lda, 64, 64) : make_map(&tm[2 * i], p.A, p.K, g.M, p.lda, TC_BK, TC_BM);
    if (!ok) return BETTY_ERR_CUDA;
    ok = p.tb ? make_map(&tm[2 * i + 1], p.B, p.K, g.N, p.ldb, TC_BK, TC2_BN / 2) : make_map(&tm[2 * i + 1], p.B, g.N, p.K, p.ldb, 64, 64);
    if (!ok) return BETTY_ERR_CUDA;
  }
  const int tiles = ((g.N + TC2_BN - 1) / TC2_BN) * ((g.M + 2 * TC_BM - 1) / (2 * TC_BM));
  const int max_pairs = c.sm_count / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  launch_pdl(k_gemm_tc2, dim3(2 * pairs), dim3(TC_THREADS), TC2_SMEM, c.stream, tm[0], tm[1], tm[2], tm[3], a);
  BETTY_LAUNCH_CHECK();
  return BETTY_OK;
}

betty_status gemm_tc_pair(Ctx& c, const GemmDesc& g, bool tr) { return launch_tc2(c, g, tr); }

betty_status gemm_tc(Ctx& c, const GemmDesc& g0, bool tr) {
  const GemmDesc g = tr ? swapped(g0) : g0;    // tile counts are taken in the kernel's own orientation
  // many tiles per SM (weight-gradient shapes): the two-SM kernel halves the B traffic per SM and measured faster
  const int pair_tiles = ((g.N + TC2_BN - 1) / TC2_BN) * ((g.M + 2 * TC_BM - 1) / (2 * TC_BM));
  if (pair_tiles >= 2 * (c.sm_count / 2)) return launch_tc2(c, g0, tr);
  // wide tiles unless the problem is narrow or would leave most SMs without a tile
  const int tiles256 = ((g.N + 255) / 256) * ((g.M + TC_BM - 1) / TC_BM);
  if (g.N > 128 && tiles256 >= 96) return launch_tc<256>(c, g0, tr);
  // 128-wide tiles would fill under half of the SMs: halve the tile width again (twice the CTAs, each
  // staging and reading a quarter less per k-slab)
  const int tiles128 = ((g.N + 127) / 128) * ((g.M + TC_BM - 1) / TC_BM);
  if (g.N > 64 && tiles128 * 2 <= c.sm_count) return launch_tc<64>(c, g0, tr);
  return launch_tc<128>(c, g0, tr);
}

}  // namespace BETTY_FAM
}  // namespace betty
