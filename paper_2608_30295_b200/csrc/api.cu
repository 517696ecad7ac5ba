// Host-only entry points: version, error text, pool layout, head classification.
#include <algorithm>
#include <math.h>
#include <vector>

#include "common.cuh"

namespace catekv {
static thread_local int g_last_cuda_error = 0;
void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }
}  // namespace catekv

extern "C" int catekv_version(void) { return 1000; }

extern "C" int catekv_last_cuda_error(void) { return catekv::g_last_cuda_error; }

extern "C" const char* catekv_error_string(int code) {
  switch (code) {
    case CATEKV_OK: return "ok";
    case CATEKV_ERR_INVALID_ARG: return "invalid argument";
    case CATEKV_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case CATEKV_ERR_CAPACITY: return "segment capacity exceeded";
    case CATEKV_ERR_WORKSPACE: return "workspace or plan buffer too small";
    case CATEKV_ERR_CUDA: return "CUDA error";
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
