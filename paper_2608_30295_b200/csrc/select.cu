// Prefill-end selection (Algorithm 1, pre-filling stage): window scores -> pooling -> per-KV-head
// top-k with lowest-index tie-break -> ascending kept list -> gather of K/V rows into the
// head's segment of the pool.
#include <math.h>
#include <string.h>

#include <atomic>
#include <vector>

#include <cooperative_groups.h>

#include "radix.cuh"
#include "score.cuh"
#include "select.cuh"

namespace cg = cooperative_groups;

namespace catekv {

constexpr int kTopkThreads = 1024;


// Block-wide exclusive scan of a packed pair (lo 32 bits, hi 32 bits) over 1024 threads.
__device__ __forceinline__ unsigned long long block_excl_scan(unsigned long long v, unsigned long long* s_warp,
                                                              unsigned long long& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) s_warp[warp] = x;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = s_warp[lane], ws = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long y = __shfl_up_sync(0xffffffffu, ws, o);
      if (lane >= o) ws += y;
    }
    s_warp[lane] = ws - w;            // exclusive prefix of the warp totals
    if (lane == 31) s_warp[32] = ws;  // grand total
  }
  __syncthreads();
  const unsigned long long res = s_warp[warp] + x - v;
  total = s_warp[32];
  __syncthreads();  // s_warp is reused by the next call
  return res;
}

// Pooled entry c of segment seg is the rnk-th selected one: its tokens go to slot rnk of the kept list (cs tokens
// per slot; the last chunk of the range may be short).
__device__ __forceinline__ void topk_emit(const TopkArgs& a, const SelSeg& s, int seg, int32_t* idx, int cs, int c,
                                          unsigned int rnk) {
  const int S = a.sink;
#ifdef CATEKV_CHECKED
  // the rank must be one of the k_sel slots and the list position inside the segment's row of idx
  rnk = (unsigned int)checked_clamp((int)rnk, 0, s.k_sel - 1, a.chk, kKidTopk, seg);
  if ((int64_t)S + ((int64_t)rnk + 1) * cs > a.idx_stride) {
    raise_status(a.chk, CATEKV_STATUS_INDEX_RANGE, kKidTopk, seg, (int)rnk);
    return;
  }
#endif
  if (cs == 1) {
    idx[S + rnk] = S + c;
  } else {
    const int l2 = S + c * cs, h2 = min(l2 + cs, s.cand_end);
    int32_t* dst = idx + S + (size_t)rnk * cs;
    if ((cs & 3) == 0 && h2 - l2 == cs && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
      for (int u = 0; u < cs; u += 4) *reinterpret_cast<int4*>(dst + u) = make_int4(l2 + u, l2 + u + 1, l2 + u + 2, l2 + u + 3);
    } else {
      for (int u = l2; u < h2; ++u) dst[u - l2] = u;
    }
  }
}

// One thread-block cluster of CL CTAs (1 or 8) per segment that selects: pooling, radix select of the k-th largest
// pooled score, ordered compaction into the ascending kept list.  Every CTA owns a contiguous share of the pooled
// entries.  The CTAs meet only through distributed shared memory: the per-pass digit histograms and the per-CTA
// (greater, equal) totals are read from the peers' shared memory, every CTA derives the same decisions from them.
template <int CL>
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const TopkArgs a) {
  cg::cluster_group cluster = cg::this_cluster();
  const int seg = blockIdx.x / CL;
  const int rank = CL > 1 ? (int)cluster.block_rank() : 0;
  pdl_launch_dependents();
  pdl_wait();  // the decisions and the scores come from earlier kernels of the stream
  const SelSeg s = a.segs[seg];
  if (s.keep_all) {  // the whole cluster leaves
    if (a.mark_keep_all && rank == 0 && threadIdx.x == 0) a.seg_len_dev[seg] = -1;
    return;
  }
  __shared__ unsigned int hist[256];
  __shared__ unsigned int hsum[256];
  __shared__ unsigned long long s_warp[33];
  __shared__ unsigned int s_pair[2];
  __shared__ unsigned int s_mm[2];  // smallest and largest bit pattern of this CTA's share
  __shared__ unsigned long long s_tot;  // this CTA's (greater, equal) totals, read by its peers
  extern __shared__ unsigned int stage[];  // a.stage_entries words: this CTA's share of the pooled scores
  auto cluster_sync = [&]() {
    if (CL > 1) cluster.sync(); else __syncthreads();
  };
  const int tid = threadIdx.x;
  int32_t* idx = a.idx + (size_t)seg * a.idx_stride;
  const int S = a.sink;
  int n_sel_tokens = 0;

  if (s.k_sel > 0) {
    const float* C = a.C + (size_t)s.job * a.c_stride;
    float* P = a.P + (size_t)s.job * a.c_stride;
    const int n_sc = s.n - a.L_obs;
    // this CTA's share of the pooled entries (a multiple of 4 entries, so that 4-entry steps stay aligned)
    const int per = ((s.n_pool + CL - 1) / CL + 3) / 4 * 4;
    const int lo = min(s.n_pool, rank * per), hi = min(s.n_pool, lo + per);
    // ---- pooling (four entries per thread and step, so that several loads are in flight)
    const float* __restrict__ Cr = C;
    float* __restrict__ Pw = P;
    if (a.pool_mode == kPoolPrescored) {
      // P was filled by the caller's scoring kernel
    } else if (a.pool_mode == CATEKV_POOL_NONE) {
      for (int c0 = lo + tid; c0 < hi; c0 += 4 * kTopkThreads) {
        float vv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) vv[e] = (c0 + e * kTopkThreads < hi) ? Cr[S + c0 + e * kTopkThreads] : 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (c0 + e * kTopkThreads < hi) Pw[c0 + e * kTopkThreads] = vv[e];
      }
    } else if (a.pool_mode == CATEKV_POOL_SLIDING) {
      const int half = (a.pool_param - 1) / 2;
      for (int c0 = lo + tid; c0 < hi; c0 += 4 * kTopkThreads) {
        float mm[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = c0 + e * kTopkThreads;
          mm[e] = 0.f;
          if (c < hi) {
            const int j = S + c;
            const int l2 = max(0, j - half), h2 = min(n_sc - 1, j + half);
            float m = Cr[l2];
            for (int u = l2 + 1; u <= h2; ++u) m = fmaxf(m, Cr[u]);
            mm[e] = m;
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (c0 + e * kTopkThreads < hi) Pw[c0 + e * kTopkThreads] = mm[e];
      }
    } else {
      const int cs = a.pool_param;
      for (int c0 = lo + tid; c0 < hi; c0 += 4 * kTopkThreads) {
        float mm[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = c0 + e * kTopkThreads;
          mm[e] = 0.f;
          if (c < hi) {
            const int l2 = S + c * cs, h2 = min(l2 + cs, s.cand_end);
            float m = Cr[l2];
            for (int u = l2 + 1; u < h2; ++u) m = fmaxf(m, Cr[u]);
            mm[e] = m;
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (c0 + e * kTopkThreads < hi) Pw[c0 + e * kTopkThreads] = mm[e];
      }
    }
    __syncthreads();  // a CTA reads back only its own share of P
    // The share is read several more times (digit passes, counts, compaction): from shared memory if it fits the
    // staging area the launch provided (entry i of the share at word i + i / 32: the pad keeps both the strided
    // sweeps of the digit passes and the per-thread runs of the compaction free of bank conflicts), else from
    // global memory (L2).  The same sweep finds the smallest and largest bit pattern.
    const unsigned int* Pg = reinterpret_cast<const unsigned int*>(P);
    const int n_loc = hi - lo;
    const bool staged = n_loc <= a.stage_entries;
    auto sp = [](int i) { return i + (i >> 5); };
    unsigned int vmin = 0xffffffffu, vmax = 0u;
    for (int i0 = tid; i0 < n_loc; i0 += 4 * kTopkThreads) {  // four loads in flight
      unsigned int vv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) vv[e] = (i0 + e * kTopkThreads < n_loc) ? Pg[lo + i0 + e * kTopkThreads] : 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (i0 + e * kTopkThreads < n_loc) {
          if (staged) stage[sp(i0 + e * kTopkThreads)] = vv[e];
          vmin = min(vmin, vv[e]);
          vmax = max(vmax, vv[e]);
        }
    }
    if (tid == 0) {
      s_mm[0] = 0xffffffffu;
      s_mm[1] = 0u;
    }
    __syncthreads();
    vmin = __reduce_min_sync(0xffffffffu, vmin);
    vmax = __reduce_max_sync(0xffffffffu, vmax);
    if ((tid & 31) == 0) {
      atomicMin(&s_mm[0], vmin);
      atomicMax(&s_mm[1], vmax);
    }
    cluster_sync();  // staging complete; every CTA's extremes are in its shared memory
    unsigned int gmin = 0xffffffffu, gmax = 0u;
#pragma unroll
    for (int r = 0; r < CL; ++r) {
      gmin = min(gmin, CL > 1 ? *cluster.map_shared_rank(&s_mm[0], r) : s_mm[0]);
      gmax = max(gmax, CL > 1 ? *cluster.map_shared_rank(&s_mm[1], r) : s_mm[1]);
    }
    auto ldp = [&](int i) { return staged ? stage[sp(i)] : Pg[lo + i]; };  // entry i of this CTA's share
    // ---- radix select of the k_sel-th largest pooled score (scores are >= 0, so their bit patterns order as
    // integers).  The bits above the highest bit in which the extremes differ are common to all entries and become
    // the prefix; the nb bits below are resolved from the top, up to 8 per pass, with the CTAs' histograms summed
    // through distributed shared memory.  Scores within a factor of two of one another need three passes.
    int nb = 32 - __clz(gmin ^ gmax);  // 0: all entries are equal
    unsigned int prefix = nb >= 32 ? 0u : (gmax >> nb) << nb, need = (unsigned int)s.k_sel;
    int pass_no = 0;
    while (nb > 0) {
      const int wbits = min(8, nb);
      const int shift = nb - wbits;
      const unsigned int dmask = (1u << wbits) - 1u;
      const unsigned int pmask = shift + wbits >= 32 ? 0u : (0xffffffffu << (shift + wbits));
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      for (int i0 = 0; i0 < n_loc; i0 += 4 * kTopkThreads) {  // whole warps stay in the loop: the vote needs them
        unsigned int v[4];
        bool in[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = i0 + e * kTopkThreads + tid;
          in[e] = i < n_loc;
          v[e] = in[e] ? ldp(i) : 0u;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool hit = in[e] && (v[e] & pmask) == prefix;
          // a warp whose lanes all fall in one bin adds once; otherwise every hit adds for itself
          const unsigned int dgt = hit ? ((v[e] >> shift) & dmask) : 0x100u;
          int same;
          __match_all_sync(0xffffffffu, dgt, &same);
          if (same) {
            if (hit && (tid & 31) == 0) atomicAdd(&hist[dgt], 32u);
          } else if (hit) {
            atomicAdd(&hist[dgt], 1u);
          }
        }
      }
      cluster_sync();  // all histograms complete
      if (tid < 256) {
        unsigned int t = 0;
#pragma unroll
        for (int r = 0; r < CL; ++r) t += CL > 1 ? *cluster.map_shared_rank(&hist[tid], r) : hist[tid];
        hsum[tid] = t;
      }
      __syncthreads();
      if (tid < 32) radix_pick_digit(hsum, need, prefix, shift, s_pair);
      cluster_sync();  // decision visible; the peers are done reading this CTA's histogram
      prefix = s_pair[0];
      need = s_pair[1];
      nb = shift;
      ++pass_no;
    }
    const unsigned int thr = prefix, need_eq = need;  // threshold bits; ties taken (lowest index first)
    // ---- ordered compaction.  A thread owns a run of consecutive entries of the share (staged) or, per step of
    // 4096 entries, four consecutive ones (from global memory): it counts its entries above and at the threshold,
    // an exclusive scan over the block (plus the totals of the CTAs before this one) says where its selected
    // entries go, and it writes them in order.
    const int cs = (a.pool_mode == CATEKV_POOL_CHUNK || a.pool_mode == kPoolPrescored) ? a.pool_param : 1;
    auto emit = [&](int c, unsigned int rnk) { topk_emit(a, s, seg, idx, cs, c, rnk); };
    unsigned long long all = 0;  // packed: low = entries above the threshold, high = entries equal to it
    if (staged) {
      const int E = (n_loc + kTopkThreads - 1) / kTopkThreads;
      const int r0 = min(n_loc, tid * E), r1 = min(n_loc, r0 + E);
      unsigned long long mine = 0;
      for (int i = r0; i < r1; ++i) {
        const unsigned int v = stage[sp(i)];
        mine += (unsigned long long)(v > thr) | ((unsigned long long)(v == thr) << 32);
      }
      unsigned long long tot;
      unsigned long long ex = block_excl_scan(mine, s_warp, tot);
      if (tid == 0) s_tot = tot;
      cluster_sync();
#pragma unroll
      for (int r = 0; r < CL; ++r) {
        const unsigned long long t = CL > 1 ? *cluster.map_shared_rank(&s_tot, r) : s_tot;
        if (r < rank) ex += t;
        all += t;
      }
      for (int i = r0; i < r1; ++i) {
        const unsigned int v = stage[sp(i)];
        const bool gt = v > thr, eq = v == thr;
        const unsigned int gt_before = (unsigned int)(ex & 0xffffffffu), eq_before = (unsigned int)(ex >> 32);
        if (gt || (eq && eq_before < need_eq)) emit(lo + i, gt_before + min(eq_before, need_eq));
        ex += (unsigned long long)gt | ((unsigned long long)eq << 32);
      }
    } else {
      unsigned long long mine_tot = 0;
      for (int c = lo + tid; c < hi; c += kTopkThreads) {
        const unsigned int v = Pg[c];
        mine_tot += (unsigned long long)(v > thr) | ((unsigned long long)(v == thr) << 32);
      }
      {
        unsigned long long tot;
        block_excl_scan(mine_tot, s_warp, tot);
        if (tid == 0) s_tot = tot;
      }
      cluster_sync();
      unsigned long long run = 0;
#pragma unroll
      for (int r = 0; r < CL; ++r) {
        const unsigned long long t = CL > 1 ? *cluster.map_shared_rank(&s_tot, r) : s_tot;
        if (r < rank) run += t;
        all += t;
      }
      for (int base = lo; base < hi; base += 4 * kTopkThreads) {
        const int c4 = base + tid * 4;
        unsigned int v[4];
        bool gt[4], eq[4];
        unsigned long long mine = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          v[e] = (c4 + e < hi) ? Pg[c4 + e] : 0u;
          gt[e] = (c4 + e < hi) && v[e] > thr;
          eq[e] = (c4 + e < hi) && v[e] == thr;
          mine += (unsigned long long)gt[e] | ((unsigned long long)eq[e] << 32);
        }
        unsigned long long tot;
        unsigned long long ex = run + block_excl_scan(mine, s_warp, tot);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int gt_before = (unsigned int)(ex & 0xffffffffu), eq_before = (unsigned int)(ex >> 32);
          if (gt[e] || (eq[e] && eq_before < need_eq)) emit(c4 + e, gt_before + min(eq_before, need_eq));
          ex += (unsigned long long)gt[e] | ((unsigned long long)eq[e] << 32);
        }
        run += tot;
      }
    }
    // selected tokens: whole chunks, except that the last chunk of the range may be short
    n_sel_tokens = s.k_sel * cs;
    if (cs > 1) {
      const int last = s.n_pool - 1;
      const int last_sz = s.cand_end - (S + last * cs);
      const unsigned int vl = Pg[last];  // written by the last CTA before the cluster barriers above
      // the last chunk is taken iff it is above the threshold, or ties with it and is within the quota of ties
      const unsigned int eq_total = (unsigned int)(all >> 32);
      const bool last_taken = vl > thr || (vl == thr && eq_total <= need_eq);
      if (last_taken) n_sel_tokens -= cs - last_sz;
    }
    cluster_sync();  // no CTA leaves while a peer may still read its shared memory
  }
  if (rank == 0) {
    for (int i = tid; i < S; i += kTopkThreads) idx[i] = i;
    const int n_tail = s.n - s.cand_end;  // the always-kept most recent tokens
    for (int i = tid; i < n_tail; i += kTopkThreads) idx[S + n_sel_tokens + i] = s.cand_end + i;
    if (tid == 0) a.seg_len_dev[seg] = S + n_sel_tokens + n_tail;
  }
}

// ---- short prescored lists (the per-step retrieval: a few thousand chunk scores per segment) -------------------------
// One CTA per segment, the whole list in shared memory, thread t owning entries t, t + 1024, ...  The kernel runs
// once per segment on a cold instruction cache, so every loop over a thread's entries stays rolled: the steps are
//   1. a 1024-bin histogram over the scores mapped linearly between the extremes of the first 1024 entries (monotone
//      in the score, and spread over the bins where the scores are: their bit patterns crowd into a few exponents),
//      a suffix scan (thread t owns bin 1023 - t) finds the bin that holds the k-th largest entry;
//   2. that bin's entries (a few, as a rule) are ranked against one another by (score descending, index ascending):
//      the k-th entry's pattern is the threshold and the rank gives the number of ties to take;
//   3. more than kTsRank entries in the bin (many equal or nearly equal scores): histogram passes over their bit
//      patterns, 10 bits at a time between the extremes of what is left, until the bin is resolved or small;
//   4. ordered compaction: the warps' votes give one bitmap of the entries above the threshold and one of those at
//      it; thread t takes word t of both (32 consecutive entries), one scan over the counts, the writes.
// Per entry two flags live in registers: above the threshold for sure (gtm), still a candidate (cand).
constexpr int kTsPer = 32;     // entries a thread may own (one flag bit each in two 32-bit registers)
constexpr int kTsBins = 1024;  // == kTopkThreads: one bin per thread in the scan
constexpr int kTsRank = 256;   // candidates resolved by ranking
constexpr int kTopkSmallMax = kTsPer * kTopkThreads;
static_assert(kTopkSmallMax / 32 == kTopkThreads, "one bitmap word per thread");

__global__ void __launch_bounds__(kTopkThreads) topk_small_kernel(const TopkArgs a) {
  __shared__ unsigned int hist[kTsBins];
  __shared__ unsigned int s_gt[kTopkSmallMax / 32], s_eq[kTopkSmallMax / 32];
  __shared__ unsigned int s_tot[32];
  __shared__ unsigned int s_mm[2];
  __shared__ unsigned int s_sel[3];
  __shared__ unsigned int s_ncand;
  __shared__ unsigned int s_cv[kTsRank];
  __shared__ int s_ci[kTsRank];
  __shared__ unsigned int s_thr[2];
  __shared__ int s_last;
  extern __shared__ __align__(16) unsigned int sv[];  // the list (small_pool entries, rounded up to 4), then its digits
  unsigned short* sd = reinterpret_cast<unsigned short*>(sv + (a.small_pool + 3) / 4 * 4);
  const int seg = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  hist[tid] = 0;
  s_gt[tid] = 0u;  // kTopkSmallMax / 32 == kTopkThreads words each
  s_eq[tid] = 0u;
  if (tid == 0) {
    s_mm[0] = 0xffffffffu;
    s_mm[1] = 0u;
    s_ncand = 0u;
    s_last = 0;
    s_sel[0] = 0u, s_sel[1] = 1u, s_sel[2] = 1u;
  }
  pdl_wait();  // the decisions and the scores come from earlier kernels of the stream
  // The scores are requested before the decision has arrived: entries past the list's end are masked out below
  // (they lie inside the row, whose stride covers small_pool entries rounded up to 4).
  const unsigned int* Pg = reinterpret_cast<const unsigned int*>(a.P + (size_t)seg * a.c_stride);
  {
    const uint32_t sv_addr = smem_u32(sv);
#pragma unroll 1
    for (int i = tid * 4; i < a.small_pool; i += 4 * kTopkThreads) cp_async16(sv_addr + i * 4, Pg + i, 16);
    cp_async_commit();
  }
  SelSeg s = a.segs[seg];
  if (s.n_pool > a.small_pool) {  // cannot happen with decisions taken from lengths within the capacities
    raise_status(a.chk, CATEKV_STATUS_INDEX_RANGE, kKidTopk, seg, s.n_pool);  // (a.chk is null outside the checked build)
    s.n_pool = a.small_pool;
    s.k_sel = min(s.k_sel, s.n_pool);
  }
  if (s.keep_all) {
    cp_async_wait<0>();
    if (a.mark_keep_all && tid == 0) a.seg_len_dev[seg] = -1;
    return;
  }
  int32_t* idx = a.idx + (size_t)seg * a.idx_stride;
  const int S = a.sink, cs = a.pool_param;
  const int E = (s.n_pool + kTopkThreads - 1) / kTopkThreads;  // entries of the busiest thread (<= kTsPer)
  int n_sel_tokens = 0;
  cp_async_wait<0>();
  __syncthreads();  // the list is in shared memory; the histogram and the extremes are initialised
  if (s.k_sel > 0) {
    unsigned int cand = 0u, gtm = 0u, need = (unsigned int)s.k_sel;
    // The range of the first histogram comes from a sample, the first 1024 entries: scores outside it fall into
    // the first or the last bin, which keeps the digits monotone (a crowded bin is resolved like any other).
    unsigned int vmin = 0xffffffffu, vmax = 0u;
    if (tid < s.n_pool) vmin = vmax = sv[tid];
#pragma unroll 1
    for (int e = 0; e < E; ++e)
      if (e * kTopkThreads + tid < s.n_pool) cand |= 1u << e;
    vmin = __reduce_min_sync(0xffffffffu, vmin);
    vmax = __reduce_max_sync(0xffffffffu, vmax);
    if (lane == 0) {
      atomicMin(&s_mm[0], vmin);
      atomicMax(&s_mm[1], vmax);
    }
    __syncthreads();
    unsigned int base = s_mm[0];
    unsigned int range = s_mm[1] - base;
    {
      bool linear = true;
      const float xmin = key_to_score(base);
      const float scale = (float)(kTsBins - 1) / (key_to_score(s_mm[1]) - xmin);
      int shift = 0;
      auto digit = [&](unsigned int val) -> int {
        if (linear) {
          // monotone in val, also when the sample's range is empty (scale infinite): a product that is not a number
          // converts to 0, an infinite or negative one is clamped
          const int d = (int)((key_to_score(val) - xmin) * scale);
          return min(max(d, 0), kTsBins - 1);
        }
        return (int)((val - base) >> shift);
      };
      while (true) {
#pragma unroll 1
        for (int e = 0; e < E; ++e)
          if ((cand >> e) & 1u) {
            const int d = digit(sv[e * kTopkThreads + tid]);
            sd[e * kTopkThreads + tid] = (unsigned short)d;
            atomicAdd(&hist[d], 1u);
          }
        __syncthreads();
        // suffix scan over the bins, larger digits first; every thread clears the bin it read for the next pass
        const unsigned int cnt = hist[kTsBins - 1 - tid];
        hist[kTsBins - 1 - tid] = 0u;
        unsigned int inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned int y = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += y;
        }
        if (lane == 31) s_tot[warp] = inc;
        if (tid == 0) {
          s_mm[0] = 0xffffffffu;
          s_mm[1] = 0u;
        }
        __syncthreads();
        inc += __reduce_add_sync(0xffffffffu, lane < warp ? s_tot[lane] : 0u);
        if (inc - cnt < need && need <= inc) {  // this thread's bin holds the need-th largest candidate
          s_sel[0] = (unsigned int)(kTsBins - 1 - tid);
          s_sel[1] = need - (inc - cnt);
          s_sel[2] = cnt;
        }
        __syncthreads();
        const int b = (int)s_sel[0];
        need = s_sel[1];
        const unsigned int m = s_sel[2];
        const bool rank_it = m != need && !(!linear && shift == 0) && m <= (unsigned int)kTsRank;
#pragma unroll 1
        for (int e = 0; e < E; ++e)
          if ((cand >> e) & 1u) {
            const int d = sd[e * kTopkThreads + tid];
            if (d > b) gtm |= 1u << e;
            if (d != b) {
              cand &= ~(1u << e);
            } else if (rank_it) {  // the bin's entries are ranked against one another below
              const unsigned int pos = atomicAdd(&s_ncand, 1u);
              if (pos < (unsigned int)kTsRank) {
                s_cv[pos] = sv[e * kTopkThreads + tid];
                s_ci[pos] = e * kTopkThreads + tid;
              }
            }
          }
        if (m == need) break;              // the whole bin is taken
        if (!linear && shift == 0) break;  // the bin is one bit pattern: need of its entries, lowest indices first
        if (rank_it) {
          __syncthreads();
          if (tid < (int)m) {
            const unsigned int mv = s_cv[tid];
            const int mi = s_ci[tid];
            unsigned int rank = 0, ties_before = 0;
#pragma unroll 4
            for (int j = 0; j < (int)m; ++j) {
              const unsigned int vj = s_cv[j];
              const bool tie_before = vj == mv && s_ci[j] < mi;
              rank += (vj > mv) || tie_before;
              ties_before += tie_before;
            }
            if (rank == need - 1u) {
              s_thr[0] = mv;
              s_thr[1] = ties_before + 1u;
            }
          }
          __syncthreads();
          const unsigned int thr = s_thr[0];
          need = s_thr[1];
#pragma unroll 1
          for (int e = 0; e < E; ++e)
            if ((cand >> e) & 1u) {
              const unsigned int val = sv[e * kTopkThreads + tid];
              if (val > thr) gtm |= 1u << e;
              if (val != thr) cand &= ~(1u << e);
            }
          break;
        }
        // a crowded bin: go on with the bit patterns of what is left, between their extremes
        unsigned int cmin = 0xffffffffu, cmax = 0u;
#pragma unroll 1
        for (int e = 0; e < E; ++e)
          if ((cand >> e) & 1u) {
            const unsigned int val = sv[e * kTopkThreads + tid];
            cmin = min(cmin, val);
            cmax = max(cmax, val);
          }
        cmin = __reduce_min_sync(0xffffffffu, cmin);
        cmax = __reduce_max_sync(0xffffffffu, cmax);
        if (lane == 0 && cmin <= cmax) {
          atomicMin(&s_mm[0], cmin);
          atomicMax(&s_mm[1], cmax);
        }
        __syncthreads();
        base = s_mm[0];
        range = s_mm[1] - base;
        if (range == 0u) break;  // all that is left ties
        linear = false;
        shift = max(0, 32 - __clz(range) - 10);
      }
    }
    // ---- ordered compaction: entries above the threshold (gtm) and the first `need` of those at it (cand).
    // Warp w's entries of step e are the 32 consecutive entries of bitmap word e * 32 + w (the words were cleared
    // at the start; few entries have a flag set).
    for (unsigned int mk = gtm; mk; mk &= mk - 1u) atomicOr(&s_gt[(__ffs(mk) - 1) * 32 + warp], 1u << lane);
    for (unsigned int mk = cand; mk; mk &= mk - 1u) atomicOr(&s_eq[(__ffs(mk) - 1) * 32 + warp], 1u << lane);
    __syncthreads();
    const int n_words = (s.n_pool + 31) / 32;  // <= 1024: thread t < n_words takes word t
    const unsigned int g = tid < n_words ? s_gt[tid] : 0u, q = tid < n_words ? s_eq[tid] : 0u;
    const unsigned int mine = (unsigned int)__popc(g) | ((unsigned int)__popc(q) << 16);
    unsigned int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) s_tot[warp] = inc;
    __syncthreads();
    const unsigned int ex = inc - mine + __reduce_add_sync(0xffffffffu, lane < warp ? s_tot[lane] : 0u);
    const int last = s.n_pool - 1;
    const int last_sz = s.cand_end - (S + last * cs);
    {
      unsigned int eq_before = ex >> 16;
      unsigned int rnk = (ex & 0xffffu) + min(eq_before, need);  // slot of this thread's next selected entry
      unsigned int bits = g | q;
      while (bits) {
        const int e = __ffs(bits) - 1;
        bits &= bits - 1u;
        const bool gt = (g >> e) & 1u;
        if (gt || eq_before < need) {
          const int c = tid * 32 + e;
          if (rnk < (unsigned int)s.k_sel) topk_emit(a, s, seg, idx, cs, c, rnk);
          if (c == last) s_last = 1;
          ++rnk;
        }
        eq_before += gt ? 0u : 1u;
      }
    }
    // selected tokens: whole chunks, except that the last chunk of the range may be short
    n_sel_tokens = s.k_sel * cs;
    if (last_sz < cs) {
      __syncthreads();
      if (s_last) n_sel_tokens -= cs - last_sz;
    }
  }
  for (int i = tid; i < S; i += kTopkThreads) idx[i] = i;
  const int n_tail = s.n - s.cand_end;  // the always-kept most recent tokens
  for (int i = tid; i < n_tail; i += kTopkThreads) idx[S + n_sel_tokens + i] = s.cand_end + i;
  if (tid == 0) a.seg_len_dev[seg] = S + n_sel_tokens + n_tail;
}

// Row statistics from a given normaliser: stats[job][r] = (log-sum-exp of row r over the scored keys in the log2 domain,
// 1), so that the second scoring pass computes exp2(logit - lse) directly.  Row r = i * G + g.
__global__ void stats_from_lse_kernel(const ScoreJob* jobs, const float* lse, float2* stats, int R, int G, int L_obs, int Hq) {
  const ScoreJob job = jobs[blockIdx.x];
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const int i = r / G, g = r - i * G;
    const float v = lse[((size_t)job.b * Hq + job.h * G + g) * L_obs + i];
    stats[(size_t)blockIdx.x * kScoreMaxRows + r] = v > -INFINITY ? make_float2(v * 1.4426950408889634f, 1.f) : make_float2(-INFINITY, 0.f);
  }
}

constexpr int kGatherRowsPerBlock = 64;

// One warp per kept row: lanes 0-15 move the K row, lanes 16-31 the V row (16 bytes each).
// This kernel rewrites rows that a decode plan may already cover: it is launched without the programmatic-launch
// attribute and never signals its dependents early (see launch_pdl), so the attention kernel that follows cannot
// request those rows before they are written.
__global__ void __launch_bounds__(256) gather_kernel(const GatherArgs a) {
  const int seg = blockIdx.y;
  const SelSeg s = a.segs[seg];
  int len = s.keep_all ? s.n : a.seg_len_dev[seg];  // a straight copy keeps all n rows
  // Never write past the destination segment: a list that does not fit (a replayed retrieval step whose step
  // cache is too small for what the source has grown to) is cut at the capacity, the length says so, and the
  // status block records it.  Every block of the segment takes the same decision.
  const int cap = a.seg_cap ? a.seg_cap[seg] : 0x7fffffff;
  const bool cut = len > cap;
  if (cut) len = cap;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (s.keep_all || cut) a.seg_len_dev[seg] = len;
    if (cut) raise_status(a.status, CATEKV_STATUS_CAPACITY, kKidGather, seg, s.keep_all ? s.n : cap + 1);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = seg / a.Hkv, h = seg % a.Hkv;
  const int64_t off = a.seg_off[seg];
  const uint8_t* src_base = (lane < 16 ? a.k : a.v) + (lane & 15) * 16 +
                            (a.src_seg_off ? (int64_t)a.src_seg_off[seg] * a.st : b * a.sb + h * a.sh);
  uint8_t* dst_base = (lane < 16 ? a.k_pool : a.v_pool) + off * kRowBytes + (lane & 15) * 16;
  const int r0 = blockIdx.x * kGatherRowsPerBlock;
#pragma unroll 4
  for (int i = warp; i < kGatherRowsPerBlock; i += 8) {
    const int r = r0 + i;
    if (r >= len) break;
    int tok = s.keep_all ? r : a.idx[(size_t)seg * a.idx_stride + r];
#ifdef CATEKV_CHECKED
    tok = checked_clamp(tok, 0, s.n - 1, a.chk, kKidGather, seg);  // a kept index names a row of the source list
#endif
    const uint4 val = __ldg(reinterpret_cast<const uint4*>(src_base + (int64_t)tok * a.st));
    *reinterpret_cast<uint4*>(dst_base + (int64_t)r * kRowBytes) = val;
    if (a.idx_out && lane == 0) a.idx_out[(size_t)seg * a.idx_out_stride + r] = tok;
  }
}

constexpr int kTopkStageMax = 32768;  // pooled entries a CTA may stage in shared memory (132 KB with the padding)

template <int CL>
static int launch_topk_cluster(const TopkArgs& a, int n_segs, size_t smem, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_segs * CL);
  cfg.blockDim = dim3(kTopkThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  CATEKV_CUDA_TRY(cudaLaunchKernelEx(&cfg, topk_kernel<CL>, a));
  return CATEKV_OK;
}

int launch_topk(const TopkArgs& a0, int n_segs, int max_pool, int n_active, cudaStream_t stream) {
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  CATEKV_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
    const int bytes = (kTopkStageMax + kTopkStageMax / 32 + 1) * 4;
    CATEKV_CUDA_TRY(cudaFuncSetAttribute(topk_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    CATEKV_CUDA_TRY(cudaFuncSetAttribute(topk_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    CATEKV_CUDA_TRY(cudaFuncSetAttribute(topk_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    CATEKV_CUDA_TRY(cudaFuncSetAttribute(topk_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTopkSmallMax * 6));
    if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
  }
  TopkArgs a = a0;
  a.chk = checked_status_ptr();
  if (a.pool_mode == kPoolPrescored && a.row_is_seg && max_pool <= kTopkSmallMax && (max_pool + 3) / 4 * 4 <= a.c_stride) {
    // short prescored lists: one CTA per segment with the list in registers
    a.small_pool = max_pool;
    CATEKV_CUDA_TRY(launch_pdl(topk_small_kernel, dim3(n_segs), dim3(kTopkThreads), (size_t)((max_pool + 3) / 4 * 4) * 6, stream, a));
    return CATEKV_OK;
  }
  // CTAs per segment: one for short lists, a cluster of 8 for long ones.  The cluster's barriers and exchanges
  // have a fixed cost, one CTA's passes grow with the list: the cluster pays from about 12 K entries, provided the
  // clusters of the segments that select fit one wave of resident CTAs (two per SM); beyond 16 K entries a single
  // CTA is slower in any case.
  int CL = (max_pool > 16384 || (max_pool >= 12288 && n_active * 8 <= 2 * sm_count())) ? 8 : 1;
  // many long lists: clusters of 4 when those fit one wave and clusters of 8 would need two (a share of up to
  // kTopkStageMax entries is still staged in shared memory)
  if (CL == 8 && n_active * 8 > 2 * sm_count() && n_active * 4 <= 2 * sm_count() && (max_pool + 3) / 4 <= kTopkStageMax) CL = 4;
  const int share = ((max_pool + CL - 1) / CL + 3) / 4 * 4;
  a.stage_entries = share <= kTopkStageMax ? share : 0;  // longer shares are read from global memory
  const size_t smem = (size_t)(a.stage_entries + a.stage_entries / 32 + 1) * 4;
  if (CL == 8) return launch_topk_cluster<8>(a, n_segs, smem, stream);
  if (CL == 4) return launch_topk_cluster<4>(a, n_segs, smem, stream);
  CATEKV_CUDA_TRY(launch_pdl(topk_kernel<1>, dim3(n_segs), dim3(kTopkThreads), smem, stream, a));
  return CATEKV_OK;
}
int launch_gather(const GatherArgs& a0, int max_len, int n_segs, cudaStream_t stream) {
  GatherArgs a = a0;
  a.chk = checked_status_ptr();
  // at least one block per segment: block 0 also records the length of a straight copy
  const int gx = max_len > 0 ? (max_len + kGatherRowsPerBlock - 1) / kGatherRowsPerBlock : 1;
  gather_kernel<<<dim3(gx, n_segs), 256, 0, stream>>>(a);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}

struct SelWs {
  size_t off_status, off_segs, off_jobs, off_part, off_stats, off_C, off_P, off_idx, bytes;
  int64_t c_stride, idx_stride;
};
static SelWs sel_ws_layout(int n_segs, int G, int n_max, int L_obs) {
  SelWs w;
  const int n_sc = n_max > L_obs ? n_max - L_obs : 1;
  w.c_stride = (int64_t)align_up((size_t)n_sc, 64);
  w.idx_stride = (int64_t)align_up((size_t)n_max, 64);
  size_t o = 0;
  w.off_status = o; o = CATEKV_STATUS_BYTES;
  w.off_segs = o; o = align_up(o + sizeof(SelSeg) * (size_t)n_segs, 256);
  w.off_jobs = o; o = align_up(o + sizeof(ScoreJob) * (size_t)n_segs, 256);
  w.off_part = o; o = align_up(o + sizeof(float2) * (size_t)score_max_ctas(n_segs) * 2 * kScoreMaxRows, 256);
  w.off_stats = o; o = align_up(o + sizeof(float2) * (size_t)n_segs * kScoreMaxRows, 256);
  w.off_C = o; o = align_up(o + sizeof(float) * (size_t)n_segs * w.c_stride, 256);
  w.off_P = o; o = align_up(o + sizeof(float) * (size_t)n_segs * w.c_stride, 256);
  w.off_idx = o; o = align_up(o + sizeof(int32_t) * (size_t)n_segs * w.idx_stride, 256);
  w.bytes = o;
  return w;
}

}  // namespace catekv

using namespace catekv;

extern "C" size_t catekv_select_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t n_max, int32_t L_obs) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || n_max <= 0 || L_obs <= 0 || Hq % Hkv) return 0;
  return sel_ws_layout(B * Hkv, Hq / Hkv, n_max, L_obs).bytes;
}

extern "C" int catekv_select_compact(const catekv_select_params* p, catekv_cache* cache, int32_t* idx_out,
                                     int64_t idx_stride, void* ws, size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  if (!p || !cache || !ws) return CATEKV_ERR_INVALID_ARG;
  if (p->B <= 0 || p->Hq <= 0 || p->Hkv <= 0 || p->Hq % p->Hkv) return CATEKV_ERR_INVALID_ARG;
  if (p->d != kD) return CATEKV_ERR_UNSUPPORTED;
  const int G = p->Hq / p->Hkv;
  if (G > kMaxG) return CATEKV_ERR_UNSUPPORTED;
  if (p->L_obs < 1 || p->sink < 0 || p->local < p->L_obs || p->budget_consistent < 0) return CATEKV_ERR_INVALID_ARG;
  if (G * p->L_obs > kScoreMaxRows) return CATEKV_ERR_UNSUPPORTED;
  if (!(p->eta_adaptive >= 0.f)) return CATEKV_ERR_INVALID_ARG;
  if (p->pool_mode == CATEKV_POOL_CHUNK) {
    if (p->pool_param < 1) return CATEKV_ERR_INVALID_ARG;
  } else if (p->pool_mode == CATEKV_POOL_SLIDING) {
    if (p->pool_param < 1 || p->pool_param % 2 == 0) return CATEKV_ERR_INVALID_ARG;
  } else if (p->pool_mode != CATEKV_POOL_NONE) {
    return CATEKV_ERR_UNSUPPORTED;
  }
  if (!p->q_win || !p->k || !p->v || !p->seq_len || !p->head_mask) return CATEKV_ERR_INVALID_ARG;
  if (cache->B != p->B || cache->Hkv != p->Hkv || cache->d != kD) return CATEKV_ERR_INVALID_ARG;
  if (!cache->k_pool || !cache->v_pool || !cache->seg_off_dev || !cache->seg_len_dev || !cache->seg_off ||
      !cache->seg_cap || !cache->seg_len)
    return CATEKV_ERR_INVALID_ARG;
  const int n_segs = p->B * p->Hkv;
  int n_max = 0;
  for (int b = 0; b < p->B; ++b) {
    if (p->seq_len[b] < 1) return CATEKV_ERR_INVALID_ARG;
    n_max = p->seq_len[b] > n_max ? p->seq_len[b] : n_max;
  }
  if (idx_out && idx_stride < n_max) return CATEKV_ERR_INVALID_ARG;
  const SelWs W = sel_ws_layout(n_segs, G, n_max, p->L_obs);
  if (ws_bytes < W.bytes) return CATEKV_ERR_WORKSPACE;

  // ---- per-segment decisions, all on the host
  std::vector<SelSeg> segs(n_segs);
  std::vector<ScoreJob> jobs;
  std::vector<int32_t> new_len(n_segs);
  bool need_readback = false;  // CHUNK mode with a short last chunk: the kept length depends on the scores
  int max_len_ub = 0, n_sc_jobs_max = 0;
  const int S = p->sink, Lc = p->local;
  for (int b = 0; b < p->B; ++b) {
    const int n = p->seq_len[b];
    for (int h = 0; h < p->Hkv; ++h) {
      const int sgi = b * p->Hkv + h;
      SelSeg s = {};
      s.n = n;
      s.job = -1;
      int64_t T;
      if (p->head_mask[sgi] > 2) return CATEKV_ERR_INVALID_ARG;
      if (p->head_mask[sgi] == 2) T = (int64_t)S + Lc;  // streaming head: sinks and recent tokens only
      else if (p->head_mask[sgi] == 1) T = p->budget_consistent;
      else T = p->eta_adaptive >= 1.f ? n : (int64_t)floor((double)p->eta_adaptive * (double)n);
      if (T >= n || (int64_t)S + Lc >= n) {
        s.keep_all = 1;
        s.len_ub = n;
      } else {
        s.cand_end = n - Lc;
        const int ncand = s.cand_end - S;
        const int k_rest = (int)(T - S - Lc > 0 ? T - S - Lc : 0);
        int sel_tokens;
        if (p->pool_mode == CATEKV_POOL_CHUNK) {
          const int cs = p->pool_param;
          s.n_pool = (ncand + cs - 1) / cs;
          s.k_sel = k_rest / cs;
          sel_tokens = s.k_sel * cs;
          if (s.k_sel > 0 && ncand % cs != 0) need_readback = true;
        } else {
          s.n_pool = ncand;
          s.k_sel = k_rest;
          sel_tokens = k_rest;
        }
        s.len_ub = S + sel_tokens + Lc;
        if (s.k_sel > 0) {
          s.job = (int)jobs.size();
          jobs.push_back(ScoreJob{b, h, n, 0, n - p->L_obs, 0});
          n_sc_jobs_max = n - p->L_obs > n_sc_jobs_max ? n - p->L_obs : n_sc_jobs_max;
        }
      }
      if (s.len_ub > cache->seg_cap[sgi]) return CATEKV_ERR_CAPACITY;
      max_len_ub = s.len_ub > max_len_ub ? s.len_ub : max_len_ub;
      new_len[sgi] = s.len_ub;
      segs[sgi] = s;
    }
  }

  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w8 = (uint8_t*)ws;
  SelSeg* d_segs = (SelSeg*)(w8 + W.off_segs);
  ScoreJob* d_jobs = (ScoreJob*)(w8 + W.off_jobs);
  {
    // one copy brings the cleared status block, the segment table and the job list (they are adjacent in the workspace)
    std::vector<uint8_t> head(W.off_jobs + sizeof(ScoreJob) * jobs.size(), 0);
    memcpy(head.data() + W.off_segs, segs.data(), sizeof(SelSeg) * n_segs);
    if (!jobs.empty()) memcpy(head.data() + W.off_jobs, jobs.data(), sizeof(ScoreJob) * jobs.size());
    CATEKV_CUDA_TRY(cudaMemcpyAsync(w8, head.data(), head.size(), cudaMemcpyHostToDevice, st));
  }
  if (!jobs.empty()) {
    ScoreArgs sa = {};
    sa.q_win = (const uint16_t*)p->q_win;
    sa.k = (const uint16_t*)p->k;
    sa.sb = p->kv_stride_b;
    sa.sh = p->kv_stride_h;
    sa.st = p->kv_stride_t;
    sa.jobs = d_jobs;
    sa.n_jobs = (int)jobs.size();
    sa.Hq = p->Hq;
    sa.B = p->B;
    sa.Hkv = p->Hkv;
    sa.n_max = n_max;
    sa.G = G;
    sa.L_obs = p->L_obs;
    sa.causal = 0;  // every scored key precedes every window query
    sa.scale_log2 = 1.4426950408889634f / sqrtf((float)kD);
    sa.max_keys = n_sc_jobs_max;
    if (p->row_lse_scored) {
      // the prefill pass already knows every window row's normaliser over the scored keys: no first pass over K
      stats_from_lse_kernel<<<(unsigned)jobs.size(), 128, 0, st>>>(d_jobs, p->row_lse_scored, (float2*)(w8 + W.off_stats),
                                                                  G * p->L_obs, G, p->L_obs, p->Hq);
      CATEKV_CUDA_TRY(cudaGetLastError());
      sa.stats_given = 1;
    }
    sa.stats_part = (float2*)(w8 + W.off_part);
    sa.stats = (float2*)(w8 + W.off_stats);
    sa.status = (int32_t*)(w8 + W.off_status);
    sa.out = (float*)(w8 + W.off_C);
    sa.out_job_stride = W.c_stride;
    int rc = score_launch(sa, kScoreColsum, st);
    if (rc) return rc;
  }
  TopkArgs ta = {};
  ta.segs = d_segs;
  ta.C = (const float*)(w8 + W.off_C);
  ta.P = (float*)(w8 + W.off_P);
  ta.c_stride = W.c_stride;
  ta.idx = (int32_t*)(w8 + W.off_idx);
  ta.idx_stride = W.idx_stride;
  ta.seg_len_dev = cache->seg_len_dev;
  ta.sink = S;
  ta.L_obs = p->L_obs;
  ta.pool_mode = p->pool_mode;
  ta.pool_param = p->pool_param;
  {
    int max_pool = 0;
    for (const SelSeg& sg : segs) max_pool = sg.n_pool > max_pool ? sg.n_pool : max_pool;
    int n_active = 0;
    for (const SelSeg& sg : segs) n_active += (!sg.keep_all && sg.k_sel > 0) ? 1 : 0;
    int rc2 = launch_topk(ta, n_segs, max_pool, n_active, st);
    if (rc2) return rc2;
  }
  GatherArgs ga;
  ga.segs = d_segs;
  ga.idx = ta.idx;
  ga.idx_stride = W.idx_stride;
  ga.k = (const uint8_t*)p->k;
  ga.v = (const uint8_t*)p->v;
  ga.sb = p->kv_stride_b * 2;
  ga.sh = p->kv_stride_h * 2;
  ga.st = p->kv_stride_t * 2;
  ga.k_pool = (uint8_t*)cache->k_pool;
  ga.v_pool = (uint8_t*)cache->v_pool;
  ga.seg_off = cache->seg_off_dev;
  ga.seg_len_dev = cache->seg_len_dev;
  ga.idx_out = idx_out;
  ga.idx_out_stride = idx_stride;
  ga.Hkv = p->Hkv;
  ga.src_seg_off = nullptr;
  ga.seg_cap = cache->seg_cap_dev;  // the host check above is exact here; the clamp can only fire on a caller's error
  ga.status = (int32_t*)(w8 + W.off_status);
  {
    int rc2 = launch_gather(ga, max_len_ub, n_segs, st);
    if (rc2) return rc2;
  }

  // A short last chunk makes the kept length depend on the scores: the mirror then holds the upper bound (the
  // device's length is at most cs - 1 rows shorter) and the cache is marked; catekv_cache_sync_lengths fetches
  // the exact lengths when the caller wants them.
  for (int i = 0; i < n_segs; ++i) cache->seg_len[i] = new_len[i];
  cache->reserved = need_readback ? 1 : 0;
  return CATEKV_OK;
}
