// Host-only entry points: version, error text, pool layout, head classification.
#include <algorithm>
#include <atomic>
#include <math.h>
#include <vector>

#include "common.cuh"

namespace catekv {
static thread_local int g_last_cuda_error = 0;
void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return 148;
  }
  int v = cached[dev].load(std::memory_order_relaxed);
  if (v > 0) return v;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
    cudaGetLastError();
    return 148;
  }
  cached[dev].store(v, std::memory_order_relaxed);
  return v;
}

#ifdef CATEKV_CHECKED
static __device__ __align__(16) int32_t g_checked_status[4];
int32_t* checked_status_ptr() {
  static std::atomic<int32_t*> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  int32_t* p = cached[dev].load(std::memory_order_relaxed);
  if (p) return p;
  void* q = nullptr;
  if (cudaGetSymbolAddress(&q, g_checked_status) != cudaSuccess) return nullptr;
  cached[dev].store((int32_t*)q, std::memory_order_relaxed);
  return (int32_t*)q;
}
#else
int32_t* checked_status_ptr() { return nullptr; }
#endif

// copy a status block to the host, synchronise, optionally clear it
static int read_status(int32_t* dev_block, catekv_status* out, int32_t clear, cudaStream_t st) {
  catekv_status h = {0, 0, 0, 0};
  CATEKV_CUDA_TRY(cudaMemcpyAsync(&h, dev_block, sizeof(h), cudaMemcpyDeviceToHost, st));
  if (clear) CATEKV_CUDA_TRY(cudaMemsetAsync(dev_block, 0, sizeof(h), st));
  CATEKV_CUDA_TRY(cudaStreamSynchronize(st));
  if (out) *out = h;
  return h.flags ? CATEKV_ERR_DEVICE : CATEKV_OK;
}
}  // namespace catekv

extern "C" int catekv_workspace_status(void* ws, catekv_status* out, int32_t clear, catekv_stream stream) {
  if (!ws) return CATEKV_ERR_INVALID_ARG;
  return catekv::read_status((int32_t*)ws, out, clear, (cudaStream_t)stream);
}

extern "C" int catekv_checked_build(void) {
#ifdef CATEKV_CHECKED
  return 1;
#else
  return 0;
#endif
}

extern "C" int catekv_checked_status(catekv_status* out, int32_t clear) {
  int32_t* p = catekv::checked_status_ptr();
  if (!p) return CATEKV_ERR_UNSUPPORTED;
  CATEKV_CUDA_TRY(cudaDeviceSynchronize());
  return catekv::read_status(p, out, clear, (cudaStream_t)0);
}

extern "C" int catekv_version(void) { return 2001; }

extern "C" int catekv_last_cuda_error(void) { return catekv::g_last_cuda_error; }

extern "C" const char* catekv_error_string(int code) {
  switch (code) {
    case CATEKV_OK: return "ok";
    case CATEKV_ERR_INVALID_ARG: return "invalid argument";
    case CATEKV_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case CATEKV_ERR_CAPACITY: return "segment capacity exceeded";
    case CATEKV_ERR_WORKSPACE: return "workspace or plan buffer too small";
    case CATEKV_ERR_CUDA: return "CUDA error";
    case CATEKV_ERR_DEVICE: return "a kernel reported a failure in its status block";
    default: return "unknown error code";
  }
}

extern "C" int catekv_cache_layout(int32_t B, int32_t Hkv, const int32_t* len0, int32_t max_new, int32_t* seg_off,
                                   int32_t* seg_cap, int64_t* total_rows) {
  if (B <= 0 || Hkv <= 0 || !len0 || max_new < 0 || !seg_off || !seg_cap || !total_rows) return CATEKV_ERR_INVALID_ARG;
  int64_t off = 0;
  const int n = B * Hkv;
  for (int s = 0; s < n; ++s) {
    if (len0[s] < 0) return CATEKV_ERR_INVALID_ARG;
    const int64_t cap = ((int64_t)len0[s] + max_new + CATEKV_SEG_ALIGN - 1) / CATEKV_SEG_ALIGN * CATEKV_SEG_ALIGN;
    if (off + cap > INT32_MAX) return CATEKV_ERR_UNSUPPORTED;
    seg_off[s] = (int32_t)off;
    seg_cap[s] = (int32_t)cap;
    off += cap;
  }
  *total_rows = off;
  return CATEKV_OK;
}

// Eq. 5 per sample, then the vote over the reference set.
extern "C" int catekv_classify_heads(const float* cv, int32_t n_samples, int32_t n_heads, float r, uint8_t* mask_out) {
  if (!cv || !mask_out || n_samples <= 0 || n_heads <= 0 || !(r >= 0.f && r <= 1.f)) return CATEKV_ERR_INVALID_ARG;
  const int kth = (int)floor((double)r * (n_heads - 1));
  std::vector<int> votes(n_heads, 0);
  std::vector<double> mean(n_heads, 0.0);
  std::vector<float> tmp(n_heads);
  for (int s = 0; s < n_samples; ++s) {
    const float* row = cv + (size_t)s * n_heads;
    std::copy(row, row + n_heads, tmp.begin());
    std::nth_element(tmp.begin(), tmp.begin() + kth, tmp.end());
    const float gamma = tmp[kth];
    for (int h = 0; h < n_heads; ++h) {
      if (row[h] > gamma) votes[h] += 1;
      mean[h] += row[h];
    }
  }
  std::vector<int> order(n_heads);
  for (int h = 0; h < n_heads; ++h) order[h] = h;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    if (votes[a] != votes[b]) return votes[a] > votes[b];
    if (mean[a] != mean[b]) return mean[a] > mean[b];
    return a < b;
  });
  const int n_consistent = n_heads - (kth + 1);
  for (int h = 0; h < n_heads; ++h) mask_out[h] = 0;
  for (int i = 0; i < n_consistent; ++i) mask_out[order[i]] = 1;
  return CATEKV_OK;
}
