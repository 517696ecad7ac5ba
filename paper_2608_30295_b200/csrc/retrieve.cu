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

#include <atomic>

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

// Fold row r of a segment (its key given as this lane's 8 bytes, w) into the metadata of its chunk.
__device__ __forceinline__ void meta_fold_row(uint8_t* meta, int64_t seg_row0, int r, int cs, int lane, uint2 w) {
  // (checked build: the callers clamp r to the segment's capacity before they get here)
  uint8_t* dst = meta + (seg_row0 / cs + r / cs) * (2 * kRowBytes) + lane * 8;
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

// After an append: fold the newest row (index len - 1) into its chunk.  One warp per segment.
__global__ void __launch_bounds__(128) meta_append_kernel(const int32_t* seg_off, const int32_t* seg_len, const uint8_t* k_new,
                                                          uint8_t* meta, int cs, int n_segs, const int32_t* seg_cap,
                                                          int32_t* chk) {
  const int seg = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_launch_dependents();
  pdl_wait();  // the length and k_new come from earlier kernels of the stream
  if (seg >= n_segs) return;
  int r = seg_len[seg] - 1;
  if (r < 0) return;
#ifdef CATEKV_CHECKED
  if (seg_cap) r = checked_clamp(r, 0, seg_cap[seg] - 1, chk, kKidMeta, seg);
#endif
  const uint2 w = *reinterpret_cast<const uint2*>(k_new + (size_t)seg * kRowBytes + lane * 8);
  meta_fold_row(meta, seg_off[seg], r, cs, lane, w);
}

// The append and the metadata update in one launch.  One warp per segment: lanes 0-15 store the K row, lanes
// 16-31 the V row (16 bytes each), all 32 fold the key into its chunk, lane 0 bumps the length.
__global__ void __launch_bounds__(128) append_meta_kernel(uint8_t* k_pool, uint8_t* v_pool, const int32_t* seg_off,
                                                          int32_t* seg_len, const uint8_t* k_new, const uint8_t* v_new,
                                                          uint8_t* meta, int cs, int n_segs, const int32_t* seg_cap,
                                                          int32_t* chk) {
  const int seg = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_launch_dependents();
  pdl_wait();
  if (seg >= n_segs) return;
  int len = seg_len[seg];
#ifdef CATEKV_CHECKED
  if (seg_cap) len = checked_clamp(len, 0, seg_cap[seg] - 1, chk, kKidMeta, seg);  // the row must fit the segment
#endif
  const int64_t row0 = seg_off[seg];
  const int c = lane & 15;
  const uint8_t* src = (lane < 16 ? k_new : v_new) + (size_t)seg * kRowBytes + c * 16;
  uint8_t* dst = (lane < 16 ? k_pool : v_pool) + (row0 + len) * kRowBytes + c * 16;
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  const uint2 w = *reinterpret_cast<const uint2*>(k_new + (size_t)seg * kRowBytes + lane * 8);
  meta_fold_row(meta, row0, len, cs, lane, w);
  __syncwarp();
  if (lane == 0) seg_len[seg] = len + 1;
}

// Per-segment decisions (what to keep, how many chunks to select) are taken on the device from its own lengths,
// by the scoring kernel itself: a step needs no host-to-device copy and can be captured in a CUDA graph.  The
// host makes the same decisions from its mirror for the capacity check.
struct RetParams {
  int32_t cs, budget, sink2 /* sink rounded up to whole chunks */, local, Hkv;
};
constexpr int kRetMaxSegs = 2048;
struct RetMask {  // which segments retrieve, one bit each; travels by value in the kernel arguments
  uint32_t w[kRetMaxSegs / 32];
};
__host__ __device__ inline SelSeg retrieval_decide(int n, bool enabled, const RetParams& p) {
  SelSeg d = {};
  d.n = n;
  d.job = -1;
  d.keep_all = 1;
  d.len_ub = n;
  if (enabled && p.budget < n) {
    const int cand_end = (n - p.local > 0 ? n - p.local : 0) / p.cs * p.cs;  // first row of the always-taken tail
    if (cand_end > p.sink2) {
      const int forced = p.sink2 + (n - cand_end);
      const int n_pool = (cand_end - p.sink2) / p.cs;
      const int k_sel = p.budget - forced > 0 ? (p.budget - forced) / p.cs : 0;
      if (k_sel < n_pool) {
        d.keep_all = 0;
        d.cand_end = cand_end;
        d.n_pool = n_pool;
        d.k_sel = k_sel;
        d.len_ub = forced + k_sel * p.cs;
      }
    }
  }
  return d;
}

// bound(c, g) = [kmax_c | kmin_c] . [max(q_g, 0) | min(q_g, 0)]: a [chunks x 256] x [256 x 8 heads] product, so the
// tensor cores take it (mma.m16n8k16, chunks are M, the group's heads N = 8).  The 64-chunk tiles (32 KB, contiguous)
// of all segments that retrieve, laid end to end, are cut into equal shares, one per CTA of a persistent grid: a CTA
// streams its tiles through a 3-stage cp.async pipeline into XOR-swizzled shared memory, across segment boundaries
// (it reloads the group's queries there); each of its 4 warps owns 16 chunks of a tile, takes the maximum over the
// heads and writes one score per chunk.  The cut is made over the tiles the segments' capacities allow, so that it
// does not move while the caches grow (a captured step stays valid); tiles past a segment's live end are skipped.
constexpr int kRsTile = 64, kRsThreads = 128, kRsStages = 3;
constexpr int kRsRowBytes = 2 * kRowBytes;                 // one chunk: 256 bf16
constexpr int kRsStageBytes = kRsTile * kRsRowBytes;
constexpr int kRsSmemFixed = kRsStages * kRsStageBytes;
static size_t rs_smem_bytes(int n_segs) { return (size_t)kRsSmemFixed + (size_t)n_segs * 4 + align_up((size_t)n_segs * 2, 16); }
__device__ __forceinline__ uint32_t rs_off(int row, int piece) {  // 16-byte piece (0..31) of a 512-byte row
  return (uint32_t)(row * kRsRowBytes + ((piece ^ (row & 7)) << 4));
}
// 64-chunk tiles that the candidate chunks of a segment of capacity cap can fill at most
__host__ __device__ inline int rs_tiles_cap(int cap, const RetParams& p) {
  const int pool = (cap - p.sink2) / p.cs;
  return pool > 0 ? (pool + kRsTile - 1) / kRsTile : 0;
}

struct RetScoreArgs {
  RetParams p;
  RetMask mask;
  const int32_t* seg_len;  // the source cache's lengths, offsets and capacities
  const int32_t* seg_off;
  const int32_t* seg_cap;
  const uint8_t* meta;
  const uint16_t* q;
  int32_t Hq, G, n_segs;
  float* P;
  int64_t p_stride;
  SelSeg* segs;  // out: the decision per segment, for the top-k and gather kernels that follow
};

__global__ void __launch_bounds__(kRsThreads, 2) retrieval_score_kernel(const RetScoreArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ int s_wsum[kRsThreads / 32];
  __shared__ int s_start[2];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_segs = a.n_segs;
  int32_t* s_npool = reinterpret_cast<int32_t*>(smem + kRsSmemFixed);             // live candidate chunks per segment
  uint16_t* s_tcap = reinterpret_cast<uint16_t*>(s_npool + n_segs);               // tiles by capacity per segment
  pdl_launch_dependents();
  // ---- this CTA's share of the tiles (from the capacities: nothing an earlier kernel of the stream writes)
  const int per = (n_segs + kRsThreads - 1) / kRsThreads;  // consecutive segments per thread
  int my_sum = 0;
  for (int k = 0; k < per; ++k) {
    const int sg = tid * per + k;
    if (sg < n_segs) {
      const int tc = ((a.mask.w[sg >> 5] >> (sg & 31)) & 1u) ? rs_tiles_cap(a.seg_cap[sg], a.p) : 0;
      s_tcap[sg] = (uint16_t)tc;
      my_sum += tc;
    }
  }
  int inc = my_sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) s_wsum[warp] = inc;
  if (tid == 0) s_start[0] = -1;
  __syncthreads();
  int total = 0;
#pragma unroll
  for (int w = 0; w < kRsThreads / 32; ++w) {
    if (w < warp) inc += s_wsum[w];
    total += s_wsum[w];
  }
  const int64_t g_lo = (int64_t)blockIdx.x * total / gridDim.x, g_hi = (int64_t)(blockIdx.x + 1) * total / gridDim.x;
  {
    int64_t off = inc - my_sum;  // tiles before this thread's segments
    if (off <= g_lo && g_lo < off + my_sum)
      for (int k = 0; k < per; ++k) {
        const int sg = tid * per + k;
        const int tc = s_tcap[sg];
        if (g_lo < off + tc) {
          s_start[0] = sg;
          s_start[1] = (int)(g_lo - off);
          break;
        }
        off += tc;
      }
  }
  pdl_wait();  // lengths, metadata and queries come from earlier kernels of the stream
  // ---- the decision of every segment (the CTAs share the writes), and its live candidate chunks
  for (int k = 0; k < per; ++k) {
    const int sg = tid * per + k;
    if (sg < n_segs) {
      SelSeg d = retrieval_decide(a.seg_len[sg], (a.mask.w[sg >> 5] >> (sg & 31)) & 1u, a.p);
      const bool scores = !d.keep_all && d.k_sel > 0;
      if (scores) d.job = sg;  // score row = segment index
      s_npool[sg] = scores ? d.n_pool : 0;
      if (sg % gridDim.x == blockIdx.x) a.segs[sg] = d;
    }
  }
  __syncthreads();
  if (g_lo >= g_hi || s_start[0] < 0) return;
  const int Hq = a.Hq, G = a.G, Hkv = a.p.Hkv, cs = a.p.cs;
  const int g = lane >> 2, t = lane & 3;
  const uint32_t s_stage = smem_u32(smem);
  const int n_tiles = (int)(g_hi - g_lo);
  struct Cursor {
    int seg, lt;         // segment and tile within it
    int n_pool;          // live candidate chunks of the segment
    const uint8_t* src;  // metadata of its first candidate chunk
  };
  auto enter = [&](Cursor& c) {
    c.n_pool = c.seg < n_segs ? s_npool[c.seg] : 0;
    c.src = a.meta + (int64_t)(c.seg < n_segs ? a.seg_off[c.seg] / cs + a.p.sink2 / cs : 0) * kRsRowBytes;
  };
  auto advance = [&](Cursor& c) {
    if (++c.lt >= (int)s_tcap[c.seg]) {
      do {
        ++c.seg;
      } while (c.seg < n_segs && s_tcap[c.seg] == 0);
      c.lt = 0;
      enter(c);
    }
  };
  Cursor ci = {s_start[0], s_start[1], 0, nullptr};  // the tile requested next
  enter(ci);
  Cursor cc = ci;  // the tile computed next
  int issued = 0;
  auto issue = [&]() {
    if (issued < n_tiles && ci.seg < n_segs) {
      const int n_pool = ci.n_pool;
      const int c0 = ci.lt * kRsTile;
      if (c0 < n_pool) {
        const uint8_t* src0 = ci.src;
        const uint32_t sb = s_stage + (issued % kRsStages) * kRsStageBytes;
#pragma unroll
        for (int i = 0; i < (kRsTile * 32) / kRsThreads; ++i) {
          const int id = tid + i * kRsThreads;
          const int r = id >> 5, pc = id & 31;
          const int ok = (c0 + r) < n_pool ? 16 : 0;
          cp_async16(sb + rs_off(r, pc), src0 + (int64_t)(ok ? c0 + r : 0) * kRsRowBytes + pc * 16, ok);
        }
      }
      advance(ci);
    }
    ++issued;
    cp_async_commit();
  };
  issue();
  issue();
  // B fragments of head g = lane / 4 of the group (zero from head G on): [max(q, 0) | min(q, 0)], the split by sign
  // being exact in bf16.  The words of the segment after the current one are requested ahead, so that a CTA whose
  // share crosses a segment boundary does not wait for them there.
  uint32_t qf[16][2], q_next[16];
  auto next_seg_of = [&](int sg) {
    do {
      ++sg;
    } while (sg < n_segs && s_tcap[sg] == 0);
    return sg;
  };
  auto load_q = [&](int sg, uint32_t (&raw)[16]) {
    const uint16_t* qp = a.q + ((int64_t)(sg / Hkv) * Hq + (sg % Hkv) * G + g) * kD;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      raw[2 * ks] = (g < G && sg < n_segs) ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 2 * t) : 0u;
      raw[2 * ks + 1] = (g < G && sg < n_segs) ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + 2 * t) : 0u;
    }
  };
  int q_seg = -1, q_next_seg = cc.seg;
  load_q(q_next_seg, q_next);
  for (int it = 0; it < n_tiles; ++it) {
    cp_async_wait<kRsStages - 2>();
    __syncthreads();
    issue();
    const int n_pool = cc.n_pool;
    const int c0 = cc.lt * kRsTile;
    if (c0 < n_pool) {
      if (cc.seg != q_seg) {
        q_seg = cc.seg;
        if (q_next_seg != q_seg) load_q(q_seg, q_next);  // a segment without live tiles lay in between
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint32_t w = q_next[2 * ks + j];
            const uint32_t pos = ((w & 0x8000u) ? 0u : (w & 0xffffu)) | ((w & 0x80000000u) ? 0u : (w & 0xffff0000u));
            qf[ks][j] = pos;
            qf[ks + 8][j] = w ^ pos;
          }
        q_next_seg = next_seg_of(q_seg);
        load_q(q_next_seg, q_next);
      }
      const uint32_t sb = s_stage + (it % kRsStages) * kRsStageBytes;
      const int row0 = warp * 16;
      float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb2[4] = {0.f, 0.f, 0.f, 0.f};
      const int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
      const int padd = lane >> 4;
#pragma unroll
      for (int ks = 0; ks < 16; ks += 2) {
        uint32_t af[4];
        ldmatrix_x4(af, sb + rs_off(r, ks * 2 + padd));
        mma_bf16_16816(sa, af, qf[ks][0], qf[ks][1]);
        ldmatrix_x4(af, sb + rs_off(r, ks * 2 + 2 + padd));
        mma_bf16_16816(sb2, af, qf[ks + 1][0], qf[ks + 1][1]);
      }
      // c0, c1: chunk row0 + g, heads 2t, 2t+1;  c2, c3: chunk row0 + g + 8
      float lo = fmaxf(2 * t < G ? sa[0] + sb2[0] : -INFINITY, 2 * t + 1 < G ? sa[1] + sb2[1] : -INFINITY);
      float hi = fmaxf(2 * t < G ? sa[2] + sb2[2] : -INFINITY, 2 * t + 1 < G ? sa[3] + sb2[3] : -INFINITY);
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {
        lo = fmaxf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
      }
      if (t == 0) {
        const int c = c0 + row0 + g;
        float* Prow = a.P + (size_t)cc.seg * a.p_stride;
        if (c < n_pool) Prow[c] = monotone_key(lo);
        if (c + 8 < n_pool) Prow[c + 8] = monotone_key(hi);
      }
    }
    if (cc.seg < n_segs) advance(cc);
  }
  cp_async_wait<0>();
}

struct RetWs {
  size_t off_status, off_segs, off_P, off_idx, bytes;
  int64_t p_stride, idx_stride;
};
static RetWs ret_ws_layout(int n_segs, int max_len) {
  RetWs w;
  w.p_stride = (int64_t)align_up((size_t)(max_len > 0 ? max_len : 1), 64);
  w.idx_stride = w.p_stride;
  size_t o = 0;
  w.off_status = o; o = CATEKV_STATUS_BYTES;
  w.off_segs = o; o = align_up(o + sizeof(SelSeg) * (size_t)n_segs, 256);
  w.off_P = o; o = align_up(o + sizeof(float) * (size_t)n_segs * w.p_stride, 256);
  w.off_idx = o; o = align_up(o + sizeof(int32_t) * (size_t)n_segs * w.idx_stride, 256);
  w.bytes = o;
  return w;
}

static int check_cache_r(const catekv_cache* c) {
  if (!c) return CATEKV_ERR_INVALID_ARG;
  if (c->B <= 0 || c->Hkv <= 0) return CATEKV_ERR_INVALID_ARG;
  if (c->d != kD || c->pages) return CATEKV_ERR_UNSUPPORTED;  // retrieval walks contiguous segments
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
  CATEKV_API_RANGE();
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
  CATEKV_API_RANGE();
  int rc = check_cache_r(cache);
  if (rc) return rc;
  if (!meta || !k_new) return CATEKV_ERR_INVALID_ARG;
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = cache->B * cache->Hkv;
  CATEKV_CUDA_TRY(launch_pdl(meta_append_kernel, dim3((n_segs + 3) / 4), dim3(128), 0, (cudaStream_t)stream,
                             cache->seg_off_dev, cache->seg_len_dev, (const uint8_t*)k_new, (uint8_t*)meta, chunk_size, n_segs,
                             cache->seg_cap_dev, checked_status_ptr()));
  return CATEKV_OK;
}

extern "C" int catekv_append_retrieval(catekv_cache* cache, const void* k_new, const void* v_new, int32_t chunk_size,
                                       void* meta, catekv_stream stream) {
  CATEKV_API_RANGE();
  int rc = check_cache_r(cache);
  if (rc) return rc;
  if (!meta || !k_new || !v_new) return CATEKV_ERR_INVALID_ARG;
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = cache->B * cache->Hkv;
  for (int s = 0; s < n_segs; ++s) {
    if (cache->seg_len[s] < 0) return CATEKV_ERR_INVALID_ARG;
    if (cache->seg_len[s] + 1 > cache->seg_cap[s]) return CATEKV_ERR_CAPACITY;
  }
  CATEKV_CUDA_TRY(launch_pdl(append_meta_kernel, dim3((n_segs + 3) / 4), dim3(128), 0, (cudaStream_t)stream,
                             (uint8_t*)cache->k_pool, (uint8_t*)cache->v_pool, cache->seg_off_dev, cache->seg_len_dev,
                             (const uint8_t*)k_new, (const uint8_t*)v_new, (uint8_t*)meta, chunk_size, n_segs,
                             cache->seg_cap_dev, checked_status_ptr()));
  for (int s = 0; s < n_segs; ++s) cache->seg_len[s] += 1;
  return CATEKV_OK;
}

extern "C" size_t catekv_retrieve_workspace_bytes(int32_t B, int32_t Hkv, int32_t max_len) {
  if (B <= 0 || Hkv <= 0 || max_len < 0) return 0;
  return ret_ws_layout(B * Hkv, max_len).bytes;
}

// Scoring and chunk selection, then either the gather into step_cache (catekv_retrieve_compact) or, with
// step_cache == NULL, just the index lists and kept lengths for catekv_decode_attn_indexed (catekv_retrieve_select).
static int retrieve_impl(const catekv_cache* cache, const void* meta, int32_t chunk_size, const void* q,
                         int32_t Hq, const uint8_t* retrieval_mask, int32_t budget, int32_t sink, int32_t local,
                         catekv_cache* step_cache, int32_t* idx_out, int64_t idx_stride, int32_t* sel_len, void* ws,
                         size_t ws_bytes, catekv_stream stream) {
  int rc = check_cache_r(cache);
  if (rc) return rc;
  if (step_cache) {
    rc = check_cache_r(step_cache);
    if (rc) return rc;
    if (step_cache->B != cache->B || step_cache->Hkv != cache->Hkv) return CATEKV_ERR_INVALID_ARG;
    if (!step_cache->seg_cap_dev) return CATEKV_ERR_INVALID_ARG;  // the gather clamps to it on the device
  } else if (!idx_out || !sel_len) {
    return CATEKV_ERR_INVALID_ARG;
  }
  if (!meta || !q || !retrieval_mask || !ws) return CATEKV_ERR_INVALID_ARG;
  if (!cache->seg_cap_dev) return CATEKV_ERR_INVALID_ARG;  // the scoring kernel shares out its tiles by the capacities
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  if (Hq <= 0 || Hq % cache->Hkv || budget < 0 || sink < 0 || local < 0) return CATEKV_ERR_INVALID_ARG;
  const int G = Hq / cache->Hkv;
  if (G > kMaxG) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = cache->B * cache->Hkv;
  const int cs = chunk_size;
  if (n_segs > kRetMaxSegs) return CATEKV_ERR_UNSUPPORTED;
  // Launch shapes and the scratch layout follow the capacities, not the current lengths: the same launches stay
  // valid while the caches grow, so a captured step can be replayed.
  int max_len = 0, max_cap = 0, max_step_cap = 0;
  for (int s = 0; s < n_segs; ++s) {
    if (cache->seg_len[s] < 0 || cache->seg_len[s] > cache->seg_cap[s]) return CATEKV_ERR_INVALID_ARG;
    max_len = cache->seg_len[s] > max_len ? cache->seg_len[s] : max_len;
    max_cap = cache->seg_cap[s] > max_cap ? cache->seg_cap[s] : max_cap;
    if (step_cache) max_step_cap = step_cache->seg_cap[s] > max_step_cap ? step_cache->seg_cap[s] : max_step_cap;
  }
  if (step_cache && idx_out && idx_stride < max_len) return CATEKV_ERR_INVALID_ARG;
  const RetWs W = ret_ws_layout(n_segs, max_cap);
  if (ws_bytes < W.bytes) return CATEKV_ERR_WORKSPACE;

  RetScoreArgs sa = {};
  RetParams& rp = sa.p;
  rp.cs = cs;
  rp.budget = budget;
  rp.sink2 = (sink + cs - 1) / cs * cs;  // sink rows rounded up to whole chunks
  rp.local = local;
  rp.Hkv = cache->Hkv;
  const int S2 = rp.sink2;
  for (int s = 0; s < n_segs; ++s) {
    const SelSeg d = retrieval_decide(cache->seg_len[s], retrieval_mask[s] != 0, rp);
    if (step_cache && d.len_ub > step_cache->seg_cap[s]) return CATEKV_ERR_CAPACITY;
    if (!step_cache && !d.keep_all && d.len_ub > idx_stride) return CATEKV_ERR_INVALID_ARG;  // its index list must fit
    if (retrieval_mask[s]) sa.mask.w[s >> 5] |= 1u << (s & 31);
  }
  const int max_pool = max_cap / cs;  // bound of the candidate chunks of a segment

  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w8 = (uint8_t*)ws;
  SelSeg* d_segs = (SelSeg*)(w8 + W.off_segs);
  float* P = (float*)(w8 + W.off_P);
  {
    // one wave of resident CTAs (2 per SM), never more CTAs than tiles
    int64_t tiles = 0;
    for (int s = 0; s < n_segs; ++s) {
      const int tc = retrieval_mask[s] ? rs_tiles_cap(cache->seg_cap[s], rp) : 0;
      if (tc > 65535) return CATEKV_ERR_UNSUPPORTED;  // the kernel keeps the tile counts as 16-bit numbers
      tiles += tc;
    }
    int64_t gx = 2 * sm_count();
    if (gx > tiles) gx = tiles;
    if (gx < 1) gx = 1;
    const size_t smem = rs_smem_bytes(n_segs);
    static std::atomic<bool> attr_set[64];
    int dev = 0;
    CATEKV_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
      CATEKV_CUDA_TRY(cudaFuncSetAttribute(retrieval_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)rs_smem_bytes(kRetMaxSegs)));
      if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
    sa.seg_len = cache->seg_len_dev;
    sa.seg_off = cache->seg_off_dev;
    sa.seg_cap = cache->seg_cap_dev;
    sa.meta = (const uint8_t*)meta;
    sa.q = (const uint16_t*)q;
    sa.Hq = Hq;
    sa.G = G;
    sa.n_segs = n_segs;
    sa.P = P;
    sa.p_stride = W.p_stride;
    sa.segs = d_segs;
    CATEKV_CUDA_TRY(launch_pdl(retrieval_score_kernel, dim3((unsigned)gx), dim3(kRsThreads), smem, st, sa));
  }
  TopkArgs ta = {};
  ta.segs = d_segs;
  ta.C = P;
  ta.P = P;
  ta.c_stride = W.p_stride;
  ta.idx = step_cache ? (int32_t*)(w8 + W.off_idx) : idx_out;
  ta.idx_stride = step_cache ? W.idx_stride : idx_stride;
  ta.seg_len_dev = step_cache ? step_cache->seg_len_dev : sel_len;
  ta.mark_keep_all = step_cache ? 0 : 1;  // select only: a segment that keeps all rows gets the length -1
  ta.sink = S2;
  ta.L_obs = 0;
  ta.pool_mode = kPoolPrescored;
  ta.pool_param = cs;
  ta.row_is_seg = 1;  // retrieval_score_kernel writes the scores of segment s to row s
  int n_masked = 0;
  for (int s = 0; s < n_segs; ++s) n_masked += retrieval_mask[s] != 0;
  rc = launch_topk(ta, n_segs, max_pool, n_masked, st);
  if (rc) return rc;
  if (!step_cache) return CATEKV_OK;
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
  ga.seg_cap = step_cache->seg_cap_dev;
  ga.status = (int32_t*)(w8 + W.off_status);
  rc = launch_gather(ga, max_step_cap, n_segs, st);
  if (rc) return rc;
  for (int s = 0; s < n_segs; ++s) step_cache->seg_len[s] = retrieval_decide(cache->seg_len[s], retrieval_mask[s] != 0, rp).len_ub;
  return CATEKV_OK;
}

extern "C" int catekv_retrieve_compact(const catekv_cache* cache, const void* meta, int32_t chunk_size, const void* q,
                                       int32_t Hq, const uint8_t* retrieval_mask, int32_t budget, int32_t sink, int32_t local,
                                       catekv_cache* step_cache, int32_t* idx_out, int64_t idx_stride, void* ws,
                                       size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  if (!step_cache) return CATEKV_ERR_INVALID_ARG;
  return retrieve_impl(cache, meta, chunk_size, q, Hq, retrieval_mask, budget, sink, local, step_cache, idx_out, idx_stride,
                       nullptr, ws, ws_bytes, stream);
}

extern "C" int catekv_retrieve_select(const catekv_cache* cache, const void* meta, int32_t chunk_size, const void* q,
                                      int32_t Hq, const uint8_t* retrieval_mask, int32_t budget, int32_t sink, int32_t local,
                                      int32_t* idx, int64_t idx_stride, int32_t* sel_len, void* ws, size_t ws_bytes,
                                      catekv_stream stream) {
  CATEKV_API_RANGE();
  return retrieve_impl(cache, meta, chunk_size, q, Hq, retrieval_mask, budget, sink, local, nullptr, idx, idx_stride, sel_len,
                       ws, ws_bytes, stream);
}

extern "C" int catekv_retrieve_lengths(const catekv_cache* cache, int32_t chunk_size, const uint8_t* retrieval_mask,
                                       int32_t budget, int32_t sink, int32_t local, int32_t* lens_out) {
  int rc = check_cache_r(cache);
  if (rc) return rc;
  if (!retrieval_mask || !lens_out || budget < 0 || sink < 0 || local < 0) return CATEKV_ERR_INVALID_ARG;
  if (!chunk_size_ok(chunk_size)) return CATEKV_ERR_UNSUPPORTED;
  RetParams rp;
  rp.cs = chunk_size;
  rp.budget = budget;
  rp.sink2 = (sink + chunk_size - 1) / chunk_size * chunk_size;
  rp.local = local;
  rp.Hkv = cache->Hkv;
  const int n_segs = cache->B * cache->Hkv;
  for (int s = 0; s < n_segs; ++s) lens_out[s] = retrieval_decide(cache->seg_len[s], retrieval_mask[s] != 0, rp).len_ub;
  return CATEKV_OK;
}
