// Shared host/device helpers of the library: workspace arena, status block, launch checks.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>
#include <atomic>
#include <mutex>
#include "betty.h"

namespace betty {

// 16-bit operand type of the MLP families' matrix products.  The family sources (mlp.cu, gemm.cu, gemm_tc.cu)
// are compiled twice into two namespaces: with bfloat16 operands (fam_bf16, the default) and, with
// BETTY_FP16_OPERANDS defined, with IEEE binary16 operands (fam_f16; Sec. 4 lists mixed precision, and the
// paper's listings switch it on with an fp16 flag).  Accumulation is fp32 in both.
#ifdef BETTY_FP16_OPERANDS
#define BETTY_FAM fam_f16
typedef __half op16;
typedef __half2 op16x2;
__device__ __forceinline__ op16 to_op16(float v) { return __float2half_rn(v); }
__device__ __forceinline__ float from_op16(op16 v) { return __half2float(v); }
__device__ __forceinline__ op16x2 to_op16x2(float a, float b) { return __floats2half2_rn(a, b); }
__device__ __forceinline__ float2 from_op16x2(op16x2 v) { return __half22float2(v); }
#else
#define BETTY_FAM fam_bf16
typedef __nv_bfloat16 op16;
typedef __nv_bfloat162 op16x2;
__device__ __forceinline__ op16 to_op16(float v) { return __float2bfloat16_rn(v); }
__device__ __forceinline__ float from_op16(op16 v) { return __bfloat162float(v); }
__device__ __forceinline__ op16x2 to_op16x2(float a, float b) { return __floats2bfloat162_rn(a, b); }
__device__ __forceinline__ float2 from_op16x2(op16x2 v) { return __bfloat1622float2(v); }
#endif

// Device status block: the first 256 bytes of the caller's workspace.
struct StatusBlock {
  int32_t code;      // first device-side condition (betty_status), 0 if none
  int32_t cg_iters;  // iterations done by the most recent CG solve
  int32_t pad[62];
};
static_assert(sizeof(StatusBlock) == 256, "status block is 256 bytes");

// State of one inverse-Hessian solve, kept on the device so that no host sync is needed.
struct SolveState {
  float rho;       // r.r
  float gamma;     // p.Hp
  float rho_new;
  float stop;      // tol^2 * v.v
  float vnorm2;    // v.v (FD: |v|^2)
  int32_t active;  // 1 while iterations still update the iterate
  int32_t iters;
  int32_t pad;
};

__device__ __forceinline__ void record_status(StatusBlock* sb, int32_t code) {
  atomicCAS(&sb->code, 0, code);
}

// Bump allocator over the caller's workspace.  Nothing is ever freed inside a call.
struct Arena {
  char* base;
  size_t size;
  size_t off;
  bool overflow;
  __host__ Arena(void* b, size_t s) : base((char*)b), size(s), off(sizeof(StatusBlock)), overflow(false) {}
  template <typename T>
  __host__ T* alloc(size_t count) {
    size_t bytes = (count * sizeof(T) + 255) & ~size_t(255);
    if (off + bytes > size) { overflow = true; return nullptr; }
    T* p = (T*)(base + off);
    off += bytes;
    return p;
  }
  __host__ size_t mark() const { return off; }
  __host__ void release(size_t m) { off = m; }
  __host__ StatusBlock* status() const { return (StatusBlock*)base; }
};

// bf16 copies of an MLP's matrices that several passes of one call share (see mlpfam_share_weights)
struct SharedWeights {
  const float* master;   // the fp32 parameters the copies were rounded from; null: none
  void* W[16];           // 16-bit copies, of the operand type of the family that made them
};

// ---- per-device facts and settings ----
// A process may drive several GPUs.  The SM count and every cudaFuncSetAttribute belong to one device, so both
// are remembered per device ordinal, never process-wide.
static constexpr int MAX_DEVICES = 64;
static constexpr int DEFAULT_SM_COUNT = 148;
// ordinal of the current device, or -1 (no device, or an ordinal beyond MAX_DEVICES)
int current_device();
// SM count of the current device, asked once per device; DEFAULT_SM_COUNT when it cannot be asked
int current_sm_count();
// Largest dynamic-shared-memory limit already set for one kernel, per device.  One instance per kernel
// instantiation (a function-local static).
struct SmemLimit {
  size_t bytes[MAX_DEVICES];
  // true when `want` bytes on device `dev` need the attribute to be (re)set; records the new limit
  bool raise(int dev, size_t want) {
    if (dev < 0 || dev >= MAX_DEVICES) return true;        // unknown device: set it every time
    if (want <= bytes[dev]) return false;
    bytes[dev] = want;
    return true;
  }
};
// Make `bytes` of dynamic shared memory launchable for `kernel` on the current device.
// Several host threads may call the library at once (each on its own stream and workspace): the check and the
// setting happen under one lock, so that no thread launches on the strength of a limit another thread has
// recorded but not yet set.
std::mutex& smem_limit_mutex();
template <typename K>
static inline betty_status ensure_dynamic_smem(K kernel, SmemLimit& lim, size_t bytes) {
  std::lock_guard<std::mutex> guard(smem_limit_mutex());
  if (!lim.raise(current_device(), bytes)) return BETTY_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
    (void)cudaGetLastError();
    return BETTY_ERR_CUDA;
  }
  return BETTY_OK;
}

struct Ctx {
  cudaStream_t stream;
  Arena arena;
  int sm_count;
  SharedWeights shared;
  const float* loss_scale;   // device loss scale of the lower step in progress (betty_level.loss_scale), else null
  bool on_side;              // launches currently go to the side stream (see SideWork)
  __host__ Ctx(void* ws, size_t ws_bytes, void* s)
      : stream((cudaStream_t)s), arena(ws, ws_bytes), sm_count(current_sm_count()), loss_scale(nullptr), on_side(false) {
    shared.master = nullptr;
  }
};

#define BETTY_TRY(expr)                       \
  do {                                        \
    betty_status _s = (expr);                 \
    if (_s != BETTY_OK) return _s;            \
  } while (0)

// Every kernel launch of the library passes through this check, which also counts it.
extern std::atomic<unsigned long long> g_kernel_launches;
#define BETTY_LAUNCH_CHECK()                                   \
  do {                                                         \
    betty::g_kernel_launches.fetch_add(1, std::memory_order_relaxed); \
    if (cudaPeekAtLastError() != cudaSuccess) {                \
      (void)cudaGetLastError();                                \
      return BETTY_ERR_CUDA;                                   \
    }                                                          \
  } while (0)

#define BETTY_ALLOC(var, T, ctx, count)                        \
  T* var = (ctx).arena.template alloc<T>(count);               \
  if (!(var)) return BETTY_ERR_WORKSPACE;

static inline bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

// ---- programmatic dependent launch ----
// Consecutive kernels of a call are launched with programmatic stream serialisation: the next grid
// may be scheduled while the current one is still running, and blocks in griddepcontrol.wait until
// the current grid has completed and its memory operations are visible.  What this hides is launch
// latency and per-kernel set-up (barrier initialisation, tensor-memory allocation).  The rules that
// keep it correct: every kernel launched through launch_pdl executes pdl_wait() before its first
// global-memory access (reads and writes: the predecessor may still be reading what this kernel
// overwrites), and no kernel depends on anything older than its stream predecessor without that
// predecessor having waited too (completion is transitive only because every kernel waits).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// wait for the predecessor, then let the successor start its own set-up
__device__ __forceinline__ void pdl_enter() { pdl_wait(); pdl_trigger(); }

template <typename... KArgs, typename... Args>
static inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // errors surface in BETTY_LAUNCH_CHECK
}

// ---- side stream ----
// A reverse sweep is a chain (the product that carries delta to the layer below) with work hanging off it
// that nothing in the chain waits for: each layer's weight-gradient product, its regulariser term and its
// bias column sums.  Launched on the caller's stream they lengthen the chain; launched on a second stream
// they run beside it and fill the SMs a one-wave product leaves idle.  The second stream and two events
// belong to the library (one set per host thread and device, made at the first call outside a stream
// capture and kept for the life of the process); they hold no device memory.  Dependencies are stated with
// event record / wait pairs, which a stream capture turns into graph edges, so that a captured call
// replays with the same concurrency.
struct SideLane { cudaStream_t stream; cudaEvent_t fork, join; };
// the calling thread's lane on the current device; null when there is none and none can be made now
// (no device, a failed creation, or `main` is being captured and the lane does not exist yet)
SideLane* side_lane(cudaStream_t main);

// Scope of one fork/join region.  begin() ... end() brackets launches that go to the side stream; they start
// after everything launched on the caller's stream before begin().  join() (also run by the destructor, so that
// an early error return leaves no work behind) makes the caller's stream wait for the side stream.  All memory
// the side work touches must stay allocated until the join.  Without a lane everything stays on the caller's
// stream, in program order.
class SideWork {
 public:
  // enable = false: a scope that forks nothing (everything in program order on the caller's stream)
  explicit SideWork(Ctx& c, bool enable = true)
      : c_(c), lane_((c.on_side || !enable) ? nullptr : side_lane(c.stream)), main_(c.stream), used_(false), ok_(true) {}
  ~SideWork() { (void)join(); }
  bool forks() const { return lane_ != nullptr; }   // false: everything stays on the caller's stream
  SideWork(const SideWork&) = delete;
  SideWork& operator=(const SideWork&) = delete;
  void begin() {
    if (!lane_) return;
    ok_ = ok_ && cudaEventRecord(lane_->fork, main_) == cudaSuccess &&
          cudaStreamWaitEvent(lane_->stream, lane_->fork, 0) == cudaSuccess;
    c_.stream = lane_->stream; c_.on_side = true; used_ = true;
  }
  void end() { c_.stream = main_; if (lane_) c_.on_side = false; }
  betty_status join() {
    end();
    if (used_) {
      ok_ = ok_ && cudaEventRecord(lane_->join, lane_->stream) == cudaSuccess &&
            cudaStreamWaitEvent(main_, lane_->join, 0) == cudaSuccess;
      used_ = false;
    }
    if (!ok_) { (void)cudaGetLastError(); return BETTY_ERR_CUDA; }
    return BETTY_OK;
  }
 private:
  Ctx& c_;
  SideLane* lane_;
  cudaStream_t main_;
  bool used_, ok_;
};

// ---- vector kernels (vec.cu); all vectors fp32, scalars stay on the device ----
betty_status vec_zero(Ctx& c, float* x, int64_t n);
betty_status vec_copy(Ctx& c, float* dst, const float* src, int64_t n);
// out = a*x + b*y (y may be null => a*x); in-place allowed
betty_status vec_axpby(Ctx& c, float* out, float a, const float* x, float b, const float* y, int64_t n);
// out = x * y (elementwise), scaled by a
betty_status vec_mul(Ctx& c, float* out, float a, const float* x, const float* y, int64_t n);
// *result = x.y, deterministic two-phase; records NONFINITE
betty_status vec_dot(Ctx& c, const float* x, const float* y, int64_t n, float* result, float* partials);
int64_t vec_dot_partials(int64_t n);
// Neumann: t_out = t_in - alpha*Ht ; s_out = s_in + t_out  (in-place allowed)
betty_status neumann_update(Ctx& c, const float* t_in, const float* s_in, const float* Ht, float alpha, float* t_out,
                            float* s_out, int64_t n);
// CG pieces driven by a SolveState on the device
betty_status cg_init(Ctx& c, SolveState* st, const float* v, float* q, float* r, float* p, float tol,
                     int64_t n, float* partials);
betty_status cg_step(Ctx& c, SolveState* st, float* q, float* r, float* p, const float* h, int64_t n,
                     float* partials);
// zero the ticket counters that live behind a partials buffer; once per buffer per call
betty_status vec_reduce_init(Ctx& c, float* partials);

}  // namespace betty
