// Query-aware retrieval on adaptive heads (Algorithm 1, decoding stage: "Retrival(q, cache)", query-aware
// form; page criterion of Quest, which the paper combines with at chunk size 8).
//
//   metadata   per chunk of cs consecutive cached rows: element-wise maximum and minimum of the keys
//   score      bound(c) = max over the group's heads of sum_d max(q_d kmin_d, q_d kmax_d)
//                       = max_g ( max(q_g, 0) . kmax_c + min(q_g, 0) . kmin_c )
//   select     the chunks of the sink rows and of the most recent rows always; of the others the best
//              floor((budget - forced rows) / cs), ties to the lowest chunk (same top-k kernel as the
//              prefill-end selection)
//   gather     the selected rows, ascending, into the segment of a per-step cache on which
//              catekv_decode_attn then runs unchanged
#include <math.h>

#include <vector>

#include "select.cuh"

namespace catekv {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---- metadata ------------------------------------------------------------------------------
// One warp per chunk; a lane owns four consecutive d (8 bytes of a row).  meta: [chunk][2][128] bf16 (max, min).
__global__ void __launch_bounds__(256) meta_build_kernel(const uint8_t* k_pool, const int32_t* seg_off, const int32_t* seg_len,
                                                         uint8_t* meta, int cs) {
  const int seg = blockIdx.y;
  const int len = seg_len[seg];
  const int chunk = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int r0 = chunk * cs;
  if (r0 >= len) return;
  const int r1 = min(len, r0 + cs);
  const int64_t row_base = (int64_t)seg_off[seg] + r0;
  float mx[4], mn[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) mx[e] = -INFINITY, mn[e] = INFINITY;
  for (int r = 0; r < r1 - r0; ++r) {
    const uint2 w = *reinterpret_cast<const uint2*>(k_pool + (row_base + r) * kRowBytes + lane * 8);
    const float v[4] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y)};
#pragma unroll
    for (int e = 0; e < 4; ++e) mx[e] = fmaxf(mx[e], v[e]), mn[e] = fminf(mn[e], v[e]);
  }
  uint8_t* dst = meta + ((int64_t)seg_off[seg] / cs + chunk) * (2 * kRowBytes) + lane * 8;
  // the extremes are bf16 values: packing them is exact
  *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(mx[0], mx[1]), pack_bf16(mx[2], mx[3]));
  *reinterpret_cast<uint2*>(dst + kRowBytes) = make_uint2(pack_bf16(mn[0], mn[1]), pack_bf16(mn[2], mn[3]));
}

// After an append: fold the newest row (index len - 1) into its chunk.  One warp per segment.
__global__ void __launch_bounds__(128) meta_append_kernel(const int32_t* seg_off, const int32_t* seg_len, const uint8_t* k_new,
                                                          uint8_t* meta, int cs, int n_segs) {
  const int seg = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (seg >= n_segs) return;
  const int r = seg_len[seg] - 1;
  if (r < 0) return;
  const uint2 w = *reinterpret_cast<const uint2*>(k_new + (size_t)seg * kRowBytes + lane * 8);
  uint8_t* dst = meta + ((int64_t)seg_off[seg] / cs + r / cs) * (2 * kRowBytes) + lane * 8;
  if (r % cs == 0) {
    *reinterpret_cast<uint2*>(dst) = w;
    *reinterpret_cast<uint2*>(dst + kRowBytes) = w;
  } else {
    const uint2 a = *reinterpret_cast<const uint2*>(dst), b = *reinterpret_cast<const uint2*>(dst + kRowBytes);
    *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(fmaxf(bf16_lo(a.x), bf16_lo(w.x)), fmaxf(bf16_hi(a.x), bf16_hi(w.x))),
                                                pack_bf16(fmaxf(bf16_lo(a.y), bf16_lo(w.y)), fmaxf(bf16_hi(a.y), bf16_hi(w.y))));
    *reinterpret_cast<uint2*>(dst + kRowBytes) =
        make_uint2(pack_bf16(fminf(bf16_lo(b.x), bf16_lo(w.x)), fminf(bf16_hi(b.x), bf16_hi(w.x))),
                   pack_bf16(fminf(bf16_lo(b.y), bf16_lo(w.y)), fminf(bf16_hi(b.y), bf16_hi(w.y))));
  }
}

// ---- chunk scores ----------------------------------------------------------------------------
struct RetJob {
  int32_t b, h;        // sequence and KV head
  int32_t chunk0;      // global index of the first candidate chunk
  int32_t n_pool;      // candidate chunks
};

// One warp per candidate chunk; a lane owns four d of both extremes and of the G query rows.
__global__ void __launch_bounds__(256) retrieval_score_kernel(const RetJob* jobs, const uint8_t* meta, const uint16_t* q, int Hq,
                                                              int G, float* P, int64_t p_stride) {
  const RetJob job = jobs[blockIdx.y];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // q+ = max(q, 0), q- = min(q, 0) of the group's heads, this lane's four d
  float qp[kMaxG][4], qn[kMaxG][4];
#pragma unroll
  for (int g = 0; g < kMaxG; ++g) {
    uint2 w = make_uint2(0u, 0u);
    if (g < G) w = *reinterpret_cast<const uint2*>(q + ((int64_t)job.b * Hq + job.h * G + g) * kD + lane * 4);
    const float v[4] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y)};
#pragma unroll
    for (int e = 0; e < 4; ++e) qp[g][e] = fmaxf(v[e], 0.f), qn[g][e] = fminf(v[e], 0.f);
  }
  for (int c = blockIdx.x * 8 + warp; c < job.n_pool; c += gridDim.x * 8) {
    const uint8_t* src = meta + ((int64_t)job.chunk0 + c) * (2 * kRowBytes) + lane * 8;
    const uint2 a = *reinterpret_cast<const uint2*>(src), b = *reinterpret_cast<const uint2*>(src + kRowBytes);
    const float mx[4] = {bf16_lo(a.x), bf16_hi(a.x), bf16_lo(a.y), bf16_hi(a.y)};
    const float mn[4] = {bf16_lo(b.x), bf16_hi(b.x), bf16_lo(b.y), bf16_hi(b.y)};
    float best = -INFINITY;
#pragma unroll
    for (int g = 0; g < kMaxG; ++g) {
      if (g < G) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) s = fmaf(qp[g][e], mx[e], fmaf(qn[g][e], mn[e], s));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        best = fmaxf(best, s);
      }
    }
    if (lane == 0) P[(size_t)blockIdx.y * p_stride + c] = best;
  }
}

// Monotone map of arbitrary finite floats to non-negative floats whose bit patterns order the same way as the
// values (what the radix select of the top-k kernel needs): flip so that larger values get larger unsigned
// patterns, then clear the sign by halving the range.  Ties are preserved (it is injective on 31 bits after the
// least significant bit is dropped, so values one ulp apart may merge: within the parity tolerance band).
__global__ void monotone_key_kernel(float* P, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint32_t u = __float_as_uint(P[i]);
  const uint32_t k = (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // unsigned order == float order
  P[i] = __uint_as_float(k >> 1);                                 // non-negative finite float pattern
}

struct RetWs {
  size_t off_segs, off_jobs, off_srcoff, off_P, off_idx, bytes;
  int64_t p_stride, idx_stride;
};
static RetWs ret_ws_layout(int n_segs, int max_len) {
  RetWs w;
  w.p_stride = (int64_t)align_up((size_t)(max_len > 0 ? max_len : 1), 64);
  w.idx_stride = w.p_stride;
  size_t o = 0;
  w.off_segs = o; o = align_up(o + sizeof(SelSeg) * (size_t)n_segs, 256);
  w.off_jobs = o; o = align_up(o + sizeof(RetJob) * (size_t)n_segs, 256);
  w.off_srcoff = o; o = align_up(o + sizeof(int32_t) * (size_t)n_segs, 256);
  w.off_P = o; o = align_up(o + sizeof(float) * (size_t)n_segs * w.p_stride, 256);
  w.off_idx = o; o = align_up(o + sizeof(int32_t) * (size_t)n_segs * w.idx_stride, 256);
  w.bytes = o;
  return w;
}

static int check_cache_r(const catekv_cache* c) {
  if (!c) return CATEKV_ERR_INVALID_ARG;
  if (c->B <= 0 || c->Hkv <= 0) return CATEKV_ERR_INVALID_ARG;
  if (c->d != kD) return CATEKV_ERR_UNSUPPORTED;
  if (!c->k_pool || !c->v_pool || !c->seg_off_dev || !c->seg_len_dev || !c->seg_off || !c->seg_cap || !c->seg_len)
    return CATEKV_ERR_INVALID_ARG;
  return CATEKV_OK;
}
static bool chunk_size_ok(int cs) { return cs >= 1 && cs <= CATEKV_SEG_ALIGN && (CATEKV_SEG_ALIGN % cs) == 0; }

}  // namespace catekv

using namespace catekv;

extern "C" size_t catekv_retrieval_meta_bytes(const catekv_cache* cache, int32_t chunk_size) {
  if (check_cache_r(cache) || !chunk_size_ok(chunk_size)) return 0;
  return (size_t)(cache->total_rows / chunk_size) * 2 * kRowBytes;
}

extern "C" int catekv_retrieval_build(const catekv_cache* cache, int32_t chunk_size, void* meta, catekv_stream stream) {
  int rc = check_cache_r(cache);
  if (rc) return rc;
  if (!meta) return CATEKV_ERR_INVALID_ARG;
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = cache->B * cache->Hkv;
  int max_len = 0;
  for (int s = 0; s < n_segs; ++s) max_len = cache->seg_len[s] > max_len ? cache->seg_len[s] : max_len;
  if (max_len == 0) return CATEKV_OK;
  const int max_chunks = (max_len + chunk_size - 1) / chunk_size;
  meta_build_kernel<<<dim3((max_chunks + 7) / 8, n_segs), 256, 0, (cudaStream_t)stream>>>(
      (const uint8_t*)cache->k_pool, cache->seg_off_dev, cache->seg_len_dev, (uint8_t*)meta, chunk_size);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}

extern "C" int catekv_retrieval_append(const catekv_cache* cache, int32_t chunk_size, const void* k_new, void* meta,
                                       catekv_stream stream) {
  int rc = check_cache_r(cache);
  if (rc) return rc;
  if (!meta || !k_new) return CATEKV_ERR_INVALID_ARG;
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = cache->B * cache->Hkv;
  meta_append_kernel<<<(n_segs + 3) / 4, 128, 0, (cudaStream_t)stream>>>(cache->seg_off_dev, cache->seg_len_dev,
                                                                           (const uint8_t*)k_new, (uint8_t*)meta, chunk_size, n_segs);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}

extern "C" size_t catekv_retrieve_workspace_bytes(int32_t B, int32_t Hkv, int32_t max_len) {
  if (B <= 0 || Hkv <= 0 || max_len < 0) return 0;
  return ret_ws_layout(B * Hkv, max_len).bytes;
}

extern "C" int catekv_retrieve_compact(const catekv_cache* cache, const void* meta, int32_t chunk_size, const void* q,
                                       int32_t Hq, const uint8_t* retrieval_mask, int32_t budget, int32_t sink, int32_t local,
                                       catekv_cache* step_cache, int32_t* idx_out, int64_t idx_stride, void* ws,
                                       size_t ws_bytes, catekv_stream stream) {
  int rc = check_cache_r(cache);
  if (rc) return rc;
  rc = check_cache_r(step_cache);
  if (rc) return rc;
  if (!meta || !q || !retrieval_mask || !ws) return CATEKV_ERR_INVALID_ARG;
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  if (step_cache->B != cache->B || step_cache->Hkv != cache->Hkv) return CATEKV_ERR_INVALID_ARG;
  if (Hq <= 0 || Hq % cache->Hkv || budget < 0 || sink < 0 || local < 0) return CATEKV_ERR_INVALID_ARG;
  const int G = Hq / cache->Hkv;
  if (G > kMaxG) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = cache->B * cache->Hkv;
  const int cs = chunk_size;
  int max_len = 0;
  for (int s = 0; s < n_segs; ++s) {
    if (cache->seg_len[s] < 0 || cache->seg_len[s] > cache->seg_cap[s]) return CATEKV_ERR_INVALID_ARG;
    max_len = cache->seg_len[s] > max_len ? cache->seg_len[s] : max_len;
  }
  if (idx_out && idx_stride < max_len) return CATEKV_ERR_INVALID_ARG;
  const RetWs W = ret_ws_layout(n_segs, max_len);
  if (ws_bytes < W.bytes) return CATEKV_ERR_WORKSPACE;

  const int S2 = (sink + cs - 1) / cs * cs;  // sink rows rounded up to whole chunks
  std::vector<SelSeg> segs(n_segs);
  std::vector<RetJob> jobs;
  std::vector<int32_t> new_len(n_segs);
  int max_out = 0, max_pool = 0;
  for (int s = 0; s < n_segs; ++s) {
    const int n = cache->seg_len[s];
    SelSeg d = {};
    d.n = n;
    d.job = -1;
    d.keep_all = 1;
    d.len_ub = n;
    if (retrieval_mask[s] && budget < n) {
      const int cand_end = (n - local > 0 ? n - local : 0) / cs * cs;  // first row of the always-taken tail
      if (cand_end > S2) {
        const int forced = S2 + (n - cand_end);
        const int n_pool = (cand_end - S2) / cs;
        const int k_sel = budget - forced > 0 ? (budget - forced) / cs : 0;
        if (k_sel < n_pool) {
          d.keep_all = 0;
          d.cand_end = cand_end;
          d.n_pool = n_pool;
          d.k_sel = k_sel;
          d.len_ub = forced + k_sel * cs;
          if (k_sel > 0) {
            d.job = (int)jobs.size();
            jobs.push_back(RetJob{s / cache->Hkv, s % cache->Hkv, cache->seg_off[s] / cs + S2 / cs, n_pool});
            max_pool = n_pool > max_pool ? n_pool : max_pool;
          }
        }
      }
    }
    if (d.len_ub > step_cache->seg_cap[s]) return CATEKV_ERR_CAPACITY;
    max_out = d.len_ub > max_out ? d.len_ub : max_out;
    new_len[s] = d.len_ub;
    segs[s] = d;
  }

  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w8 = (uint8_t*)ws;
  SelSeg* d_segs = (SelSeg*)(w8 + W.off_segs);
  RetJob* d_jobs = (RetJob*)(w8 + W.off_jobs);
  float* P = (float*)(w8 + W.off_P);
  CATEKV_CUDA_TRY(cudaMemcpyAsync(d_segs, segs.data(), sizeof(SelSeg) * n_segs, cudaMemcpyHostToDevice, st));
  if (!jobs.empty()) {
    CATEKV_CUDA_TRY(cudaMemcpyAsync(d_jobs, jobs.data(), sizeof(RetJob) * jobs.size(), cudaMemcpyHostToDevice, st));
    int gx = (max_pool + 7) / 8;
    if (gx > 512) gx = 512;  // warps stride over the chunks
    retrieval_score_kernel<<<dim3(gx, (unsigned)jobs.size()), 256, 0, st>>>(d_jobs, (const uint8_t*)meta, (const uint16_t*)q, Hq, G,
                                                                            P, W.p_stride);
    CATEKV_CUDA_TRY(cudaGetLastError());
    const int64_t np = (int64_t)jobs.size() * W.p_stride;
    monotone_key_kernel<<<(unsigned)((np + 255) / 256), 256, 0, st>>>(P, np);
    CATEKV_CUDA_TRY(cudaGetLastError());
  }
  TopkArgs ta;
  ta.segs = d_segs;
  ta.C = P;
  ta.P = P;
  ta.c_stride = W.p_stride;
  ta.idx = (int32_t*)(w8 + W.off_idx);
  ta.idx_stride = W.idx_stride;
  ta.seg_len_dev = step_cache->seg_len_dev;
  ta.sink = S2;
  ta.L_obs = 0;
  ta.pool_mode = kPoolPrescored;
  ta.pool_param = cs;
  rc = launch_topk(ta, n_segs, st);
  if (rc) return rc;
  rc = launch_set_full_len(d_segs, step_cache->seg_len_dev, n_segs, st);
  if (rc) return rc;
  GatherArgs ga;
  ga.segs = d_segs;
  ga.idx = ta.idx;
  ga.idx_stride = W.idx_stride;
  ga.k = (const uint8_t*)cache->k_pool;
  ga.v = (const uint8_t*)cache->v_pool;
  ga.sb = 0;
  ga.sh = 0;
  ga.st = kRowBytes;
  ga.src_seg_off = cache->seg_off_dev;
  ga.k_pool = (uint8_t*)step_cache->k_pool;
  ga.v_pool = (uint8_t*)step_cache->v_pool;
  ga.seg_off = step_cache->seg_off_dev;
  ga.seg_len_dev = step_cache->seg_len_dev;
  ga.idx_out = idx_out;
  ga.idx_out_stride = idx_stride;
  ga.Hkv = cache->Hkv;
  rc = launch_gather(ga, max_out, n_segs, st);
  if (rc) return rc;
  for (int s = 0; s < n_segs; ++s) step_cache->seg_len[s] = new_len[s];
  return CATEKV_OK;
}
