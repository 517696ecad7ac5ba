// Head identification statistic (Section 3.2, Eq. 1-4): observation matrix, matrix-global
// percentile threshold, per-column counts, coefficient of variation.
#include <math.h>
#include <string.h>

#include <atomic>
#include <vector>

#include <cooperative_groups.h>

#include "radix.cuh"
#include "score.cuh"

namespace cg = cooperative_groups;

namespace catekv {

struct CvSeg {
  int32_t m;        // columns of A: n - L_init - L_rec
  int32_t need;     // the percentile element is the need-th largest of the L_obs * m entries
};

struct CvArgs {
  const CvSeg* segs;
  const float* A;  // [n_segs][L_obs * m], dense
  int64_t seg_stride;
  int32_t L_obs;
  float alpha;
  float* cv_out;
};

constexpr int kCvThreads = 1024;
constexpr int kCvCluster = 8;
#ifndef CATEKV_CV_UNROLL
#define CATEKV_CV_UNROLL 16
#endif
constexpr int kCvUnroll = CATEKV_CV_UNROLL;  // loads a thread keeps in flight in the sweeps over its share of the matrix
constexpr int kCvListCap = 16384;            // entries of the threshold bin a CTA can keep in shared memory
constexpr int kCvBins = 2048;                // == 256 * kHistCopies: the fast path reuses the copies' array
static_assert(kCvBins == 256 * kHistCopies && kCvBins == 2 * kCvThreads, "two bins per thread in the scan");

// One thread-block cluster of 8 CTAs per (sequence, KV head): Phi = alpha * percentile element (Eq. 2),
// C_j = #{i: A_ij >= Phi} (Eq. 3), cv = std_pop(C) / mean(C) (Eq. 4) from exact integer sums.
// The percentile element is found by a radix select on the bit patterns (entries are >= 0); every CTA owns a
// contiguous share of the flat matrix and the CTAs' histograms are summed through distributed shared memory.
// Fast path, two sweeps over the matrix: a 2048-bin histogram of the patterns' top bits (entries are below 2, so
// bits 30..19 fit: exponent and four mantissa bits) finds the bin of the percentile element; a second sweep copies
// that bin's entries into shared memory, where two more levels (bits 18..8, bits 7..0) resolve it.  If an entry
// is 2 or more, or a CTA's part of the bin does not fit its list, the general path takes over: extremes, then the
// bits below the highest one in which they differ, 8 per sweep.  For the counts every CTA owns a range of
// columns; the sums meet in CTA 0.
__global__ void __launch_bounds__(kCvThreads) cv_kernel(const CvArgs a) {
  cg::cluster_group cluster = cg::this_cluster();
  const int seg = blockIdx.x / kCvCluster;
  const int rank = (int)cluster.block_rank();
  const CvSeg s = a.segs[seg];
  __shared__ unsigned int hist[256];
  __shared__ unsigned int hcopies[256 * kHistCopies];
  __shared__ unsigned int hsum[256];
  __shared__ unsigned int s_pair[2];
  __shared__ unsigned int s_mm[2];
  __shared__ unsigned long long red[2][32];
  __shared__ unsigned long long s_sums[2];
  __shared__ unsigned int s_pick[2], s_big, s_nlist, s_wtot[32];
  extern __shared__ unsigned int s_list[];  // kCvListCap entries
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* A = a.A + (size_t)seg * a.seg_stride;
  const unsigned int* Ab = reinterpret_cast<const unsigned int*>(A);
  const int m = s.m;
  const int N = a.L_obs * m;
  const int per = ((N + kCvCluster - 1) / kCvCluster + 3) / 4 * 4;
  const int lo = min(N, rank * per), hi = min(N, lo + per);

  // ---- fast path
  bool have_thr = false;
  unsigned int thr_bits = 0u;
  {
    unsigned int* h2k = hcopies;
    // Sum of the CTAs' histograms, suffix scan (thread t owns bins 2047 - 2t and 2046 - 2t), and the bin that
    // holds the need-th largest entry with what is still needed inside it.  The caller ends with a cluster
    // barrier before anybody's histogram is written again.
    auto pick = [&](unsigned int need_in, unsigned int& bin, unsigned int& need_out) {
      cluster.sync();  // all histograms complete
      unsigned int c_hi = 0, c_lo = 0;
#pragma unroll
      for (int r = 0; r < kCvCluster; ++r) {
        const unsigned int* hp = cluster.map_shared_rank(h2k, r);
        c_hi += hp[kCvBins - 1 - 2 * tid];
        c_lo += hp[kCvBins - 2 - 2 * tid];
      }
      const unsigned int cnt = c_hi + c_lo;
      unsigned int inc = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
      }
      if (lane == 31) s_wtot[warp] = inc;
      __syncthreads();
      inc += __reduce_add_sync(0xffffffffu, lane < warp ? s_wtot[lane] : 0u);
      const unsigned int before = inc - cnt;
      if (before < need_in && need_in <= before + c_hi) {
        s_pick[0] = (unsigned int)(kCvBins - 1 - 2 * tid);
        s_pick[1] = need_in - before;
      } else if (before + c_hi < need_in && need_in <= inc) {
        s_pick[0] = (unsigned int)(kCvBins - 2 - 2 * tid);
        s_pick[1] = need_in - before - c_hi;
      }
      __syncthreads();
      bin = s_pick[0];
      need_out = s_pick[1];
    };
    for (int i = tid; i < kCvBins; i += kCvThreads) h2k[i] = 0u;
    if (tid == 0) {
      s_big = 0u;
      s_nlist = 0u;
      s_pick[0] = 0u;
      s_pick[1] = 1u;
    }
    __syncthreads();
    bool big = false;
    for (int c0 = lo; c0 < hi; c0 += kCvUnroll * kCvThreads) {  // whole warps stay in the loop: the vote needs them
      unsigned int v[kCvUnroll];
      bool in[kCvUnroll];
#pragma unroll
      for (int e = 0; e < kCvUnroll; ++e) {
        const int c = c0 + e * kCvThreads + tid;
        in[e] = c < hi;
        v[e] = in[e] ? Ab[c] : 0u;
      }
#pragma unroll
      for (int e = 0; e < kCvUnroll; ++e) {
        unsigned int dgt = v[e] >> 19;
        if (dgt >= (unsigned int)kCvBins) {
          big = true;
          dgt = kCvBins - 1;
        }
        if (!in[e]) dgt = 0xffffu;
        // a warp whose lanes all fall in one bin adds once; otherwise every entry adds for itself
        int same;
        __match_all_sync(0xffffffffu, dgt, &same);
        if (same) {
          if (in[e] && lane == 0) atomicAdd(&h2k[dgt], 32u);
        } else if (in[e]) {
          atomicAdd(&h2k[dgt], 1u);
        }
      }
    }
    if (big) s_big = 1u;
    unsigned int b1, need1;
    pick((unsigned int)s.need, b1, need1);
    unsigned int own_max = 0u, big_any = 0u;
#pragma unroll
    for (int r = 0; r < kCvCluster; ++r) {
      own_max = max(own_max, cluster.map_shared_rank(h2k, r)[b1]);
      big_any |= *cluster.map_shared_rank(&s_big, r);
    }
    cluster.sync();  // the peers have read this CTA's histogram and flag
    if (!big_any && own_max <= (unsigned int)kCvListCap) {  // the same decision in every CTA of the cluster
      // second sweep: this CTA's entries of bin b1 go to its list
      for (int c0 = lo; c0 < hi; c0 += kCvUnroll * kCvThreads) {
        unsigned int v[kCvUnroll];
#pragma unroll
        for (int e = 0; e < kCvUnroll; ++e) {
          const int c = c0 + e * kCvThreads + tid;
          v[e] = c < hi ? Ab[c] : 0xffffffffu;  // a pattern that is in no bin
        }
#pragma unroll
        for (int e = 0; e < kCvUnroll; ++e) {
          const bool hit = (v[e] >> 19) == b1;
          const unsigned int votes = __ballot_sync(0xffffffffu, hit);
          if (votes) {
            unsigned int base = 0;
            if (lane == 0) base = atomicAdd(&s_nlist, (unsigned int)__popc(votes));
            base = __shfl_sync(0xffffffffu, base, 0);
            if (hit) s_list[base + __popc(votes & ((1u << lane) - 1u))] = v[e];
          }
        }
      }
      for (int i = tid; i < kCvBins; i += kCvThreads) h2k[i] = 0u;
      __syncthreads();
      const int n_list = (int)s_nlist;
      for (int i = tid; i < n_list; i += kCvThreads) atomicAdd(&h2k[(s_list[i] >> 8) & 0x7ffu], 1u);
      unsigned int b2, need2;
      pick(need1, b2, need2);
      cluster.sync();
      for (int i = tid; i < kCvBins; i += kCvThreads) h2k[i] = 0u;
      __syncthreads();
      for (int i = tid; i < n_list; i += kCvThreads) {
        const unsigned int v = s_list[i];
        if (((v >> 8) & 0x7ffu) == b2) atomicAdd(&h2k[v & 0xffu], 1u);
      }
      unsigned int b3, need3;
      pick(need2, b3, need3);
      cluster.sync();
      thr_bits = (b1 << 19) | (b2 << 8) | b3;
      have_thr = true;
    }
  }
  if (!have_thr) {
  // ---- extremes of the bit patterns
  unsigned int vmin = 0xffffffffu, vmax = 0u;
  for (int c0 = lo + tid; c0 < hi; c0 += kCvUnroll * kCvThreads) {  // several loads in flight
    unsigned int v[kCvUnroll];
#pragma unroll
    for (int e = 0; e < kCvUnroll; ++e) v[e] = (c0 + e * kCvThreads < hi) ? Ab[c0 + e * kCvThreads] : 0u;
#pragma unroll
    for (int e = 0; e < kCvUnroll; ++e)
      if (c0 + e * kCvThreads < hi) {
        vmin = min(vmin, v[e]);
        vmax = max(vmax, v[e]);
      }
  }
  if (tid == 0) {
    s_mm[0] = 0xffffffffu;
    s_mm[1] = 0u;
  }
  __syncthreads();
  vmin = __reduce_min_sync(0xffffffffu, vmin);
  vmax = __reduce_max_sync(0xffffffffu, vmax);
  if (lane == 0) {
    atomicMin(&s_mm[0], vmin);
    atomicMax(&s_mm[1], vmax);
  }
  cluster.sync();
  unsigned int gmin = 0xffffffffu, gmax = 0u;
#pragma unroll
  for (int r = 0; r < kCvCluster; ++r) {
    gmin = min(gmin, *cluster.map_shared_rank(&s_mm[0], r));
    gmax = max(gmax, *cluster.map_shared_rank(&s_mm[1], r));
  }

  // ---- radix select of the need-th largest entry
  int nb = 32 - __clz(gmin ^ gmax);  // 0: all entries are equal
  unsigned int prefix = nb >= 32 ? 0u : (gmax >> nb) << nb, need = (unsigned int)s.need;
  while (nb > 0) {
    const int wbits = min(8, nb);
    const int shift = nb - wbits;
    const unsigned int dmask = (1u << wbits) - 1u;
    const unsigned int pmask = shift + wbits >= 32 ? 0u : (0xffffffffu << (shift + wbits));
    radix_hist_zero(hcopies);
    __syncthreads();
    for (int c0 = lo; c0 < hi; c0 += kCvUnroll * kCvThreads) {  // whole warps stay in the loop: the vote needs them
      unsigned int v[kCvUnroll];
      bool in[kCvUnroll];
#pragma unroll
      for (int e = 0; e < kCvUnroll; ++e) {
        const int c = c0 + e * kCvThreads + tid;
        in[e] = c < hi;
        v[e] = in[e] ? Ab[c] : 0u;
      }
#pragma unroll
      for (int e = 0; e < kCvUnroll; ++e) {
        const bool hit = in[e] && (v[e] & pmask) == prefix;
        // a warp whose lanes all fall in one bin adds once; otherwise every hit adds for itself
        const unsigned int dgt = hit ? ((v[e] >> shift) & dmask) : 0x100u;
        int same;
        __match_all_sync(0xffffffffu, dgt, &same);
        if (same) {
          if (hit && lane == 0) radix_hist_add(hcopies, dgt, 32u);
        } else if (hit) {
          radix_hist_add(hcopies, dgt, 1u);
        }
      }
    }
    __syncthreads();
    radix_hist_fold(hcopies, hist);
    cluster.sync();  // all histograms complete
    if (tid < 256) {
      unsigned int t = 0;
#pragma unroll
      for (int r = 0; r < kCvCluster; ++r) t += *cluster.map_shared_rank(&hist[tid], r);
      hsum[tid] = t;
    }
    __syncthreads();
    if (tid < 32) radix_pick_digit(hsum, need, prefix, shift, s_pair);
    cluster.sync();  // decision visible; the peers are done reading this CTA's histogram
    prefix = s_pair[0];
    need = s_pair[1];
    nb = shift;
  }
  thr_bits = prefix;
  }
  const float phi = __uint_as_float(thr_bits) * a.alpha;

  // ---- column counts over this CTA's columns
  const int cper = (m + kCvCluster - 1) / kCvCluster;
  const int j_lo = min(m, rank * cper), j_hi = min(m, j_lo + cper);
  unsigned long long sum = 0, sum2 = 0;
  for (int j = j_lo + tid; j < j_hi; j += kCvThreads) {
    unsigned int c = 0;
#pragma unroll 8
    for (int i = 0; i < a.L_obs; ++i) c += A[(size_t)i * m + j] >= phi ? 1u : 0u;
    sum += c;
    sum2 += (unsigned long long)c * c;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
    sum2 += __shfl_xor_sync(0xffffffffu, sum2, o);
  }
  if (lane == 0) { red[0][warp] = sum; red[1][warp] = sum2; }
  __syncthreads();
  if (tid == 0) {
    unsigned long long S1 = 0, S2 = 0;
    for (int w = 0; w < kCvThreads / 32; ++w) { S1 += red[0][w]; S2 += red[1][w]; }
    s_sums[0] = S1;
    s_sums[1] = S2;
  }
  cluster.sync();
  if (rank == 0 && tid == 0) {
    unsigned long long S1 = 0, S2 = 0;
    for (int r = 0; r < kCvCluster; ++r) {
      S1 += *cluster.map_shared_rank(&s_sums[0], r);
      S2 += *cluster.map_shared_rank(&s_sums[1], r);
    }
    // std_pop / mean = sqrt(m * sum(C^2) - (sum C)^2) / sum C
    double cv = 0.0;
    if (S1 > 0) {
      const double num = (double)m * (double)S2 - (double)S1 * (double)S1;
      cv = sqrt(num > 0.0 ? num : 0.0) / (double)S1;
    }
    a.cv_out[seg] = (float)cv;
  }
  cluster.sync();  // no CTA leaves while CTA 0 may still read its sums
}

struct CvWs {
  size_t off_status, off_segs, off_jobs, off_part, off_stats, off_A, bytes;
  int64_t row_stride;
};
static CvWs cv_ws_layout(int n_segs, int G, int m_max, int L_obs) {
  CvWs w;
  w.row_stride = (int64_t)align_up((size_t)m_max, 64);
  size_t o = 0;
  w.off_status = o; o = CATEKV_STATUS_BYTES;
  w.off_segs = o; o = align_up(o + sizeof(CvSeg) * (size_t)n_segs, 256);
  w.off_jobs = o; o = align_up(o + sizeof(ScoreJob) * (size_t)n_segs, 256);
  w.off_part = o; o = align_up(o + sizeof(float2) * (size_t)score_max_ctas(n_segs) * 2 * kScoreMaxRows, 256);
  w.off_stats = o; o = align_up(o + sizeof(float2) * (size_t)n_segs * kScoreMaxRows, 256);
  w.off_A = o; o = align_up(o + sizeof(float) * (size_t)n_segs * L_obs * w.row_stride, 256);
  w.bytes = o;
  return w;
}

}  // namespace catekv

using namespace catekv;

extern "C" size_t catekv_head_cv_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t n_max, int32_t L_obs,
                                                 int32_t L_init, int32_t L_rec) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || L_obs <= 0 || L_init < 0 || L_rec < 0) return 0;
  const int m = n_max - L_init - L_rec;
  if (m < 1) return 0;
  return cv_ws_layout(B * Hkv, Hq / Hkv, m, L_obs).bytes;
}

extern "C" int catekv_head_cv(const void* q_win, const void* k, int64_t k_stride_b, int64_t k_stride_h,
                              int64_t k_stride_t, const int32_t* seq_len, int32_t B, int32_t Hq, int32_t Hkv,
                              int32_t d, int32_t L_obs, int32_t L_init, int32_t L_rec, float quantile_k, float alpha,
                              int32_t causal, float* cv_out, void* ws, size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  if (!q_win || !k || !seq_len || !cv_out || !ws) return CATEKV_ERR_INVALID_ARG;
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv) return CATEKV_ERR_INVALID_ARG;
  if (d != kD) return CATEKV_ERR_UNSUPPORTED;
  const int G = Hq / Hkv;
  if (G > kMaxG) return CATEKV_ERR_UNSUPPORTED;
  if (L_obs < 1 || L_init < 0 || L_rec < 0) return CATEKV_ERR_INVALID_ARG;
  if (G * L_obs > kScoreMaxRows) return CATEKV_ERR_UNSUPPORTED;
  if (!(quantile_k >= 0.f && quantile_k <= 1.f) || !(alpha >= 0.f) || isinf(alpha)) return CATEKV_ERR_INVALID_ARG;
  const int n_segs = B * Hkv;
  int m_max = 0, n_max_tokens = 0;
  for (int b = 0; b < B; ++b) {
    n_max_tokens = seq_len[b] > n_max_tokens ? seq_len[b] : n_max_tokens;
    const int64_t m = (int64_t)seq_len[b] - L_init - L_rec;
    if (m < 1 || seq_len[b] < L_obs) return CATEKV_ERR_INVALID_ARG;
    if (m * L_obs > INT32_MAX) return CATEKV_ERR_UNSUPPORTED;
    m_max = (int)m > m_max ? (int)m : m_max;
  }
  const CvWs W = cv_ws_layout(n_segs, G, m_max, L_obs);
  if (ws_bytes < W.bytes) return CATEKV_ERR_WORKSPACE;

  std::vector<CvSeg> segs(n_segs);
  std::vector<ScoreJob> jobs(n_segs);
  for (int b = 0; b < B; ++b) {
    const int n = seq_len[b];
    const int m = n - L_init - L_rec;
    const int64_t N = (int64_t)L_obs * m;
    const int64_t q = (int64_t)floor((double)quantile_k * (double)(N - 1));  // ascending order statistic
    for (int h = 0; h < Hkv; ++h) {
      segs[b * Hkv + h] = CvSeg{m, (int32_t)(N - q)};
      jobs[b * Hkv + h] = ScoreJob{b, h, n, L_init, n - L_rec, 0};
    }
  }
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w8 = (uint8_t*)ws;
  {
    // one copy brings the cleared status block, the segment table and the job list (they are adjacent in the workspace)
    std::vector<uint8_t> head(W.off_jobs + sizeof(ScoreJob) * (size_t)n_segs, 0);
    memcpy(head.data() + W.off_segs, segs.data(), sizeof(CvSeg) * n_segs);
    memcpy(head.data() + W.off_jobs, jobs.data(), sizeof(ScoreJob) * n_segs);
    CATEKV_CUDA_TRY(cudaMemcpyAsync(w8, head.data(), head.size(), cudaMemcpyHostToDevice, st));
  }
  ScoreArgs sa = {};
  sa.q_win = (const uint16_t*)q_win;
  sa.k = (const uint16_t*)k;
  sa.sb = k_stride_b;
  sa.sh = k_stride_h;
  sa.st = k_stride_t;
  sa.jobs = (const ScoreJob*)(w8 + W.off_jobs);
  sa.n_jobs = n_segs;
  sa.Hq = Hq;
  sa.B = B;
  sa.Hkv = Hkv;
  sa.n_max = n_max_tokens;
  sa.G = G;
  sa.L_obs = L_obs;
  sa.causal = causal ? 1 : 0;
  sa.g_major = L_obs == 64 ? 1 : 0;  // the paper's window: head-major rows make the group mean a register sum
  sa.scale_log2 = 1.4426950408889634f / sqrtf((float)kD);
  sa.max_keys = m_max;
  sa.stats_part = (float2*)(w8 + W.off_part);
  sa.stats = (float2*)(w8 + W.off_stats);
  sa.status = (int32_t*)(w8 + W.off_status);
  sa.out = (float*)(w8 + W.off_A);
  sa.out_job_stride = (int64_t)L_obs * W.row_stride;
  int rc = score_launch(sa, kScoreMatrix, st);
  if (rc) return rc;
  CvArgs ca;
  ca.segs = (const CvSeg*)(w8 + W.off_segs);
  ca.A = sa.out;
  ca.seg_stride = sa.out_job_stride;
  ca.L_obs = L_obs;
  ca.alpha = alpha;
  ca.cv_out = cv_out;
  cudaLaunchConfig_t cfg = {};
  {
    static std::atomic<bool> attr_set[64];
    int dev = 0;
    CATEKV_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
      CATEKV_CUDA_TRY(cudaFuncSetAttribute(cv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCvListCap * 4));
      if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
  }
  cfg.gridDim = dim3(n_segs * kCvCluster);
  cfg.blockDim = dim3(kCvThreads);
  cfg.dynamicSmemBytes = kCvListCap * 4;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCvCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  CATEKV_CUDA_TRY(cudaLaunchKernelEx(&cfg, cv_kernel, ca));
  return CATEKV_OK;
}
