// Growth of the per-head lists: append, the host mirror, overflow pages, the copy into a larger cache; and the
// attention-recall diagnostic (Section 3.4).
#include <math.h>

#include "decode.cuh"

namespace catekv {

__global__ void __launch_bounds__(128) append_kernel(uint8_t* k_pool, uint8_t* v_pool, const int32_t* seg_off,
                                                     int32_t* seg_len, const uint8_t* k_new, const uint8_t* v_new,
                                                     int n_segs, const PageArgs pg) {
  const int seg = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_launch_dependents();
  pdl_wait();
  if (seg >= n_segs) return;
  const int len = seg_len[seg];
  int64_t row = (int64_t)seg_off[seg] + len;
  if (pg.table && len >= pg.seg_cap[seg]) {  // the row goes to an overflow page
    const int o = len - pg.seg_cap[seg];
    row = (int64_t)pg.table[(int64_t)seg * pg.max_pages + (o >> 6)] * 64 + (o & 63);
    k_pool = pg.k_ovf;
    v_pool = pg.v_ovf;
  }
  const int c = lane & 15;
  const uint8_t* src = (lane < 16 ? k_new : v_new) + (size_t)seg * kRowBytes + c * 16;
  uint8_t* dst = (lane < 16 ? k_pool : v_pool) + row * kRowBytes + c * 16;
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  __syncwarp();
  if (lane == 0) seg_len[seg] = len + 1;
}

}  // namespace catekv

using namespace catekv;

extern "C" int catekv_append(catekv_cache* cache, const void* k_new, const void* v_new, catekv_stream stream) {
  CATEKV_API_RANGE();
  int rc = check_cache(cache);
  if (rc) return rc;
  if (!k_new || !v_new) return CATEKV_ERR_INVALID_ARG;
  const int n = cache->B * cache->Hkv;
  for (int s = 0; s < n; ++s) {
    if (cache->seg_len[s] < 0) return CATEKV_ERR_INVALID_ARG;
    if (cache->seg_len[s] + 1 > seg_capacity(cache, s)) return CATEKV_ERR_CAPACITY;
  }
  CATEKV_CUDA_TRY(launch_pdl(append_kernel, dim3((n + 3) / 4), dim3(128), 0, (cudaStream_t)stream,
                             (uint8_t*)cache->k_pool, (uint8_t*)cache->v_pool, cache->seg_off_dev, cache->seg_len_dev,
                             (const uint8_t*)k_new, (const uint8_t*)v_new, n, page_args(cache)));
  for (int s = 0; s < n; ++s) cache->seg_len[s] += 1;
  return CATEKV_OK;
}

// recall = exp(lse_kept - lse_full): the share of the full attention mass that falls on the kept rows
__global__ void recall_kernel(const float* lse_kept, const float* lse_full, float* recall, int n) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) recall[i] = (lse_kept[i] == -INFINITY) ? 0.f : expf(lse_kept[i] - lse_full[i]);
}

extern "C" int catekv_attention_recall(const float* lse_kept, const float* lse_full, float* recall, int32_t n,
                                       catekv_stream stream) {
  CATEKV_API_RANGE();
  if (!lse_kept || !lse_full || !recall || n < 0) return CATEKV_ERR_INVALID_ARG;
  if (n == 0) return CATEKV_OK;
  CATEKV_CUDA_TRY(launch_pdl(recall_kernel, dim3((n + 255) / 256), dim3(256), 0, (cudaStream_t)stream, lse_kept, lse_full,
                             recall, (int)n));
  return CATEKV_OK;
}

extern "C" int catekv_cache_advance(catekv_cache* cache, int32_t n_tokens) {
  int rc = check_cache(cache);
  if (rc) return rc;
  if (n_tokens < 0) return CATEKV_ERR_INVALID_ARG;
  const int n = cache->B * cache->Hkv;
  for (int s = 0; s < n; ++s)
    if ((int64_t)cache->seg_len[s] + n_tokens > seg_capacity(cache, s)) return CATEKV_ERR_CAPACITY;
  for (int s = 0; s < n; ++s) cache->seg_len[s] += n_tokens;
  return CATEKV_OK;
}

extern "C" int catekv_cache_sync_lengths(catekv_cache* cache, catekv_stream stream) {
  int rc = check_cache(cache);
  if (rc) return rc;
  const int n = cache->B * cache->Hkv;
  CATEKV_CUDA_TRY(cudaMemcpyAsync(cache->seg_len, cache->seg_len_dev, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToHost,
                                  (cudaStream_t)stream));
  CATEKV_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  cache->reserved = 0;
  return CATEKV_OK;
}

// Growth: every segment's valid rows move to the same segment of a cache with larger capacities.  One warp per
// row (lanes 0-15 the K row, 16-31 the V row); block 0 of a segment records its length.  Like the gather, this
// kernel writes rows a decode plan of the destination may cover: plain launch, no early signal to dependents.
namespace catekv {
constexpr int kRegrowRowsPerBlock = 64;
__global__ void __launch_bounds__(256) regrow_kernel(const uint8_t* sk, const uint8_t* sv, const int32_t* s_off,
                                                     const int32_t* s_len, uint8_t* dk, uint8_t* dv, const int32_t* d_off,
                                                     int32_t* d_len, const PageArgs pg) {
  const int seg = blockIdx.y;
  const int len = s_len[seg];
  if (blockIdx.x == 0 && threadIdx.x == 0) d_len[seg] = len;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint8_t* src = (lane < 16 ? sk : sv) + (int64_t)s_off[seg] * kRowBytes + (lane & 15) * 16;
  const uint8_t* ovf = (lane < 16 ? pg.k_ovf : pg.v_ovf) + (lane & 15) * 16;
  const int cap = pg.table ? pg.seg_cap[seg] : 0x7fffffff;  // rows from here on come from the source's overflow pages
  uint8_t* dst = (lane < 16 ? dk : dv) + (int64_t)d_off[seg] * kRowBytes + (lane & 15) * 16;
  const int r0 = blockIdx.x * kRegrowRowsPerBlock;
#pragma unroll 4
  for (int i = warp; i < kRegrowRowsPerBlock; i += 8) {
    const int r = r0 + i;
    if (r >= len) break;
    const uint8_t* from = src + (int64_t)r * kRowBytes;
    if (r >= cap) {
      const int o = r - cap;
      from = ovf + ((int64_t)pg.table[(int64_t)seg * pg.max_pages + (o >> 6)] * 64 + (o & 63)) * kRowBytes;
    }
    *reinterpret_cast<uint4*>(dst + (int64_t)r * kRowBytes) = __ldg(reinterpret_cast<const uint4*>(from));
  }
}
}  // namespace catekv

extern "C" int catekv_pages_reserve(catekv_cache* cache, int32_t n_new, catekv_stream stream) {
  CATEKV_API_RANGE();
  int rc = check_cache(cache);
  if (rc) return rc;
  if (!cache->pages || n_new < 0) return CATEKV_ERR_INVALID_ARG;
  catekv_pages* p = cache->pages;
  const int n = cache->B * cache->Hkv;
  // first pass: what is needed, nothing changed yet
  int64_t extra = 0;
  for (int s = 0; s < n; ++s) {
    if (cache->seg_len[s] < 0 || cache->seg_len[s] > seg_capacity(cache, s)) return CATEKV_ERR_INVALID_ARG;
    const int64_t over = (int64_t)cache->seg_len[s] + n_new - cache->seg_cap[s];
    const int64_t want = over > 0 ? (over + CATEKV_PAGE_ROWS - 1) / CATEKV_PAGE_ROWS : 0;
    if (want > p->max_pages) return CATEKV_ERR_CAPACITY;
    if (want > p->seg_pages[s]) extra += want - p->seg_pages[s];
  }
  if (extra > (int64_t)p->n_pages - p->next_free) return CATEKV_ERR_CAPACITY;
  for (int s = 0; s < n; ++s) {
    const int64_t over = (int64_t)cache->seg_len[s] + n_new - cache->seg_cap[s];
    const int want = over > 0 ? (int)((over + CATEKV_PAGE_ROWS - 1) / CATEKV_PAGE_ROWS) : 0;
    const int have = p->seg_pages[s];
    if (want <= have) continue;
    int32_t* row = p->table + (size_t)s * p->max_pages;
    for (int q = have; q < want; ++q) row[q] = p->next_free++;
    p->seg_pages[s] = want;
    CATEKV_CUDA_TRY(cudaMemcpyAsync(p->table_dev + (size_t)s * p->max_pages + have, row + have,
                                    sizeof(int32_t) * (size_t)(want - have), cudaMemcpyHostToDevice, (cudaStream_t)stream));
  }
  return CATEKV_OK;
}

extern "C" int catekv_cache_regrow(const catekv_cache* src, catekv_cache* dst, catekv_stream stream) {
  CATEKV_API_RANGE();
  int rc = check_cache(src);
  if (rc) return rc;
  rc = check_cache(dst);
  if (rc) return rc;
  if (src->B != dst->B || src->Hkv != dst->Hkv) return CATEKV_ERR_INVALID_ARG;
  if (src->k_pool == dst->k_pool || src->v_pool == dst->v_pool) return CATEKV_ERR_INVALID_ARG;
  if (dst->pages) return CATEKV_ERR_UNSUPPORTED;  // the destination is one contiguous segment per (sequence, head)
  const int n = src->B * src->Hkv;
  int max_len = 0;
  for (int s = 0; s < n; ++s) {
    if (src->seg_len[s] < 0 || src->seg_len[s] > seg_capacity(src, s)) return CATEKV_ERR_INVALID_ARG;
    if (src->seg_len[s] > dst->seg_cap[s]) return CATEKV_ERR_CAPACITY;
    max_len = src->seg_len[s] > max_len ? src->seg_len[s] : max_len;
  }
  const int gx = max_len > 0 ? (max_len + kRegrowRowsPerBlock - 1) / kRegrowRowsPerBlock : 1;
  regrow_kernel<<<dim3(gx, n), 256, 0, (cudaStream_t)stream>>>((const uint8_t*)src->k_pool, (const uint8_t*)src->v_pool,
                                                               src->seg_off_dev, src->seg_len_dev, (uint8_t*)dst->k_pool,
                                                               (uint8_t*)dst->v_pool, dst->seg_off_dev, dst->seg_len_dev,
                                                               page_args(src));
  CATEKV_CUDA_TRY(cudaGetLastError());
  for (int s = 0; s < n; ++s) dst->seg_len[s] = src->seg_len[s];
  dst->reserved = src->reserved;  // upper-bound lengths stay upper bounds
  return CATEKV_OK;
}
