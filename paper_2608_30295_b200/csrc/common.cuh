// Shared device helpers and host-side error plumbing for the CateKV kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <nvtx3/nvToolsExt.h>

#include "catekv.h"

namespace catekv {

constexpr int kD = CATEKV_HEAD_DIM;     // head dim
constexpr int kRowBytes = kD * 2;       // one bf16 row
constexpr int kMaxG = CATEKV_MAX_GROUP; // query heads per KV head, padded to 8 in the MMA N dimension

// ---- host: error bookkeeping -------------------------------------------------------------
void set_cuda_error(cudaError_t e);
#define CATEKV_CUDA_TRY(expr)                        \
  do {                                               \
    cudaError_t e__ = (expr);                        \
    if (e__ != cudaSuccess) {                        \
      ::catekv::set_cuda_error(e__);                 \
      return CATEKV_ERR_CUDA;                        \
    }                                                \
  } while (0)

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// SMs of the current device (looked up once per device; 148, the B200's count, when no device answers, so that
// the workspace-size functions still work on a host without a GPU).
int sm_count();

// ---- device status block (the first CATEKV_STATUS_BYTES of a workspace, or the checked build's own block) ---
enum KernelId { kKidScore = 1, kKidTopk = 2, kKidGather = 3, kKidAttention = 4, kKidMeta = 5 };
// Device address of the checked build's status block; null in an unchecked library.
int32_t* checked_status_ptr();

// Launch with programmatic stream serialization: the grid may be scheduled while the previous kernel of
// the stream is still draining; it must execute pdl_wait() before it touches anything that earlier work
// on the stream produced.  After a kernel that never signals, this is an ordinary in-order launch.
// Invariant the attention kernel relies on: it requests rows that were valid at plan time BEFORE its
// pdl_wait().  A kernel that rewrites cache rows a plan already covers (gather_kernel, regrow_kernel) must
// therefore never call pdl_launch_dependents(): as long as it does not, the dependent grid cannot start before
// that kernel has completed and flushed, and the early requests see the rewritten rows.  Kernels that only
// write rows behind every planned row (the appends) may signal early.
template <class... KArgs, class... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- host: an NVTX range per entry point (named after the function; costs nothing without a profiler attached)
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
  ApiRange(const ApiRange&) = delete;
  ApiRange& operator=(const ApiRange&) = delete;
};
#define CATEKV_API_RANGE() ::catekv::ApiRange catekv_api_range_(__func__)

// ---- device: record a failure in a status block {flags, kernel, segment, index}; the first reporter's details stay
__device__ __forceinline__ void raise_status(int32_t* st, int flag, int kernel, int seg, int index) {
  if (!st) return;
  if (atomicOr(st, flag) == 0) {
    st[1] = kernel;
    st[2] = seg;
    st[3] = index;
  }
}
#ifdef CATEKV_CHECKED
// Checked build: clamp a device-produced value into [lo, hi] and record a violation (never trap, never assert).
__device__ __forceinline__ int checked_clamp(int v, int lo, int hi, int32_t* st, int kernel, int seg) {
  if (v < lo || v > hi) {
    raise_status(st, CATEKV_STATUS_INDEX_RANGE, kernel, seg, v);
    v = v < lo ? lo : hi;
  }
  return v;
}
#endif

// ---- device: programmatic dependent launch ------------------------------------------------
// Let the next kernel of the stream be scheduled (it still waits, in pdl_wait, for this grid to finish).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::); }
// Block until every kernel launched before this one on the stream has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

// ---- device: asynchronous copies, ldmatrix, mma -------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte global->shared copy; src_bytes = 0 zero-fills and reads nothing.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n"
               : "=r"(r[0]), "=r"(r[1])
               : "r"(addr));
}
// 8x8 b16 transpose across the warp (fragment layout in, fragment layout out).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// pack two floats into bf16x2 (lo = first), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory tile of bf16 rows of 128 elements (256 B): the 16-byte chunk c of row r
// lives at chunk position c ^ (r & 7), so that the 8 rows touched by one ldmatrix phase
// fall in 8 different bank groups.
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return static_cast<uint32_t>(row * kRowBytes + ((chunk ^ (row & 7)) << 4));
}

}  // namespace catekv
