// Observation-window scoring on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// A CTA scores `keys_per_cta` keys of one (sequence, KV head) against the R = G * L_obs window
// query rows of the group (row r = i * G + g: window row i of the group's g-th query head).
// Q stays in shared memory for the CTA's lifetime, 128-key tiles of K stream through two
// cp.async stages, both in the K-major SWIZZLE_128B layout the UMMA descriptors expect.
//
//   pass 1 (row statistics)   D[128 rows x 128 keys] = Q_rows . K_tile^T   (M = rows, N = keys)
//       every thread owns one query row (one TMEM lane): running max and sum of exp2 over the
//       keys are thread-local.  Partials per CTA, merged by a small kernel.
//   pass 2 (column sums / group-mean matrix)
//                             D[128 keys x R rows]   = K_tile . Q^T        (M = keys, N = rows)
//       the same two shared-memory tiles with the operand roles swapped: now every thread owns
//       one key, so C_j = sum_r exp2(x_rj - m_r) / l_r and A_ij = mean_g (...) are thread-local
//       sums over TMEM columns and the global writes are coalesced over keys.
//
// One elected thread issues tcgen05.mma (8 k-steps of 16 per 128-wide head dim) and commits to an
// mbarrier; accumulators are double- or quad-buffered in TMEM so that the MMAs of the next unit
// run under the exp2 epilogue of the current one.  Every mbarrier wait is bounded: on expiry the
// CTA records a status word, drains its copies, frees its TMEM and returns.
#include <math.h>

#include "score.cuh"

namespace catekv {

constexpr int kScThreads = 256;                    // 8 warps: two per TMEM lane quarter, each takes half the columns
constexpr int kKeyTile = 128;                       // keys per tile
constexpr int kKBlockBytes = kKeyTile * 128;        // one 64-element k-block of a K tile
constexpr int kKStageBytes = 2 * kKBlockBytes;      // K tile: 128 keys x 128 dims bf16
constexpr uint32_t kSpinLimit = 1u << 22;

struct ScoreShape {
  int R;         // query rows
  int MT;        // 128-row M tiles of pass 1
  int q_rows;    // rows of the Q region in shared memory (MT * 128)
  int NH, NW;    // pass 2: N halves and their width (multiple of 16)
  int nslot1, la1, cols1;  // pass 1: TMEM slots of 128 columns, issue look-ahead, allocated columns
  int slotw2, cols2;       // pass 2: 2 slots of slotw2 columns
};

static ScoreShape score_shape(int G, int L_obs) {
  ScoreShape s;
  s.R = G * L_obs;
  s.MT = (s.R + 127) / 128;
  s.q_rows = s.MT * 128;
  // pass 2 splits the R rows into NH halves of NW columns: a multiple of 16 (UMMA N) and of G (so that the
  // G heads of one window row never straddle two halves)
  int unit = 16;
  while (unit % G) unit += 16;
  s.NH = (s.R + unit - 1) / unit * unit <= 256 ? 1 : 2;
  s.NW = ((s.R + s.NH - 1) / s.NH + unit - 1) / unit * unit;
  if (s.NH * s.NW > s.q_rows) s.q_rows = (s.NH * s.NW + 7) / 8 * 8;
  s.nslot1 = s.MT >= 3 ? 4 : 2;
  s.la1 = s.MT >= 3 ? 2 : 1;
  s.cols1 = s.nslot1 * 128;
  s.slotw2 = (s.NW + 31) / 32 * 32;
  int c = 32;
  while (c < 2 * s.slotw2) c *= 2;
  s.cols2 = c;
  return s;
}

// ---- tcgen05 / mbarrier wrappers ----------------------------------------------------------
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  // K-major, SWIZZLE_128B: rows of 128 bytes, 8-row groups 1024 bytes apart
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;               // leading byte offset: unused for this layout
  d |= (uint64_t)(1024 >> 4) << 32;     // stride byte offset
  d |= (uint64_t)1 << 46;               // descriptor version
  d |= (uint64_t)2 << 61;               // SWIZZLE_128B
  return d;
}
__device__ __forceinline__ uint32_t umma_idesc_bf16(int M, int N) {
  // D = f32, A = B = bf16, both K-major
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
// bounded wait for a phase of an mbarrier; false if it never completed
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  uint32_t done = 0;
  for (uint32_t it = 0; it < kSpinLimit && !done; ++it)
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
  return done != 0;
}
// 32 consecutive TMEM columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// offset of the 16-byte chunk c (0..15) of row r inside a two-k-block SW128 region of `rows` rows
__device__ __forceinline__ uint32_t sw128_off(int r, int c, int rows) {
  return (uint32_t)((c >> 3) * rows * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int MODE>
__global__ void __launch_bounds__(kScThreads) score_tc_kernel(const ScoreArgs a, const ScoreShape sh) {
  extern __shared__ uint8_t smem_raw[];
  const ScoreJob job = a.jobs[blockIdx.y];
  const int j_lo = job.j_begin + blockIdx.x * a.keys_per_cta;
  if (j_lo >= job.j_end) return;
  const int j_hi = min(job.j_end, j_lo + a.keys_per_cta);
  const int n_tiles = (j_hi - j_lo + kKeyTile - 1) / kKeyTile;
  const int tid = threadIdx.x, warp = tid >> 5;

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle)
  const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (s_base - smem_u32(smem_raw));
  const uint32_t q_block = (uint32_t)sh.q_rows * 128;  // one k-block of Q
  const uint32_t s_q = s_base;
  const uint32_t s_k = s_q + 2 * q_block;
  float* s_f = reinterpret_cast<float*>(smem + 2 * q_block + 2 * kKStageBytes);  // pass 1: (m, l)[MT][128]; pass 2: m'[R]
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_f + 4 * kScoreMaxRows);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 4);

  constexpr bool kStats = MODE == kScoreStats;
  const int UPT = kStats ? sh.MT : sh.NH;          // MMA units per key tile
  const int NSLOT = kStats ? sh.nslot1 : 2;
  const int LA = kStats ? sh.la1 : 1;
  const int slot_w = kStats ? 128 : sh.slotw2;
  const int n_cols = kStats ? sh.cols1 : sh.cols2;
  const int U = n_tiles * UPT;

  // ---- stage Q (row r = i * G + g) and the first two K tiles
  for (int id = tid; id < sh.q_rows * 16; id += kScThreads) {
    const int r = id >> 4, c = id & 15;
    const int i = r / a.G, g = r - i * a.G;
    const int ok = r < sh.R ? 16 : 0;
    const uint16_t* src = a.q_win + (((int64_t)job.b * a.Hq + job.h * a.G + (ok ? g : 0)) * a.L_obs + (ok ? i : 0)) * kD + c * 8;
    cp_async16(s_q + sw128_off(r, c, sh.q_rows), src, ok);
  }
  const uint16_t* kbase = a.k + (int64_t)job.b * a.sb + (int64_t)job.h * a.sh;
  auto load_tile = [&](int tile) {
    if (tile < n_tiles) {
      const uint32_t sb = s_k + (tile & 1) * kKStageBytes;
      const int j0 = j_lo + tile * kKeyTile;
#pragma unroll 4
      for (int id = tid; id < kKeyTile * 16; id += kScThreads) {
        const int r = id >> 4, c = id & 15;
        const int ok = (j0 + r) < j_hi ? 16 : 0;
        cp_async16(sb + sw128_off(r, c, kKeyTile), kbase + (int64_t)(ok ? j0 + r : job.j_begin) * a.st + c * 8, ok);
      }
    }
    cp_async_commit();
  };
  load_tile(0);
  load_tile(1);
  if (kStats) {
    for (int i = tid; i < 2 * kScoreMaxRows; i += kScThreads) {
      s_f[2 * i] = -INFINITY;
      s_f[2 * i + 1] = 0.f;
    }
  } else {
    // m'_r = m_r + log2(l_r): exp2(x - m'_r) is the normalised probability; rows without mass get +inf (-> 0)
    const float2* st = a.stats + (size_t)blockIdx.y * kScoreMaxRows;
    for (int r = tid; r < sh.R; r += kScThreads) {
      const float2 v = st[r];
      s_f[r] = v.y > 0.f ? v.x + log2f(v.y) : INFINITY;
    }
  }
  if (tid == 0) {
    for (int i = 0; i < 4; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(s_bar + i)));
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(s_tmem)), "r"(n_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  cp_async_wait<0>();
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const uint32_t idesc = kStats ? umma_idesc_bf16(128, 128) : umma_idesc_bf16(128, sh.NW);
  auto issue_unit = [&](int v) {  // thread 0 only
    const int tile = v / UPT, sub = v - tile * UPT;
    const uint32_t sk = s_k + (tile & 1) * kKStageBytes;
    const uint32_t d = tmem + (uint32_t)((v % NSLOT) * slot_w);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const uint32_t koff = (kk & 3) * 32;
      const uint32_t aq = s_q + (kk >> 2) * q_block + koff;
      const uint32_t ak = sk + (kk >> 2) * kKBlockBytes + koff;
      if (kStats)  // D[rows x keys]: A = Q rows of this M tile, B = K tile
        umma_bf16(d, umma_desc_sw128(aq + sub * 128 * 128), umma_desc_sw128(ak), idesc, kk ? 1u : 0u);
      else         // D[keys x rows]: A = K tile, B = Q rows of this half
        umma_bf16(d, umma_desc_sw128(ak), umma_desc_sw128(aq + sub * sh.NW * 128), idesc, kk ? 1u : 0u);
    }
    umma_commit(smem_u32(s_bar + (v % NSLOT)));
  };
  if (tid == 0)
    for (int v = 0; v < LA && v < U; ++v) issue_unit(v);

  // warp w reads TMEM lanes 32 * (w % 4) ...; warps 0-3 take the first half of a unit's columns, warps 4-7 the second
  const int lane_row = (warp & 3) * 32 + (tid & 31);  // this thread's TMEM lane: a query row (pass 1) or a key (pass 2)
  const int half = warp >> 2;
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
  const float inv_g = 1.f / (float)a.G;
  float* s_col = s_f + kScoreMaxRows;  // pass 2: [2][128] per-half sums of a key
  float col_acc = 0.f;                 // pass 2, column sums: this key's sum over this thread's rows of the tile
  bool alive = true;

  for (int u = 0; u < U; ++u) {
    const int tile = u / UPT, sub = u - tile * UPT;
    const int v = u + LA;
    if (sub == 0 && tile >= 1) load_tile(tile + 1);  // into the stage of tile - 1, whose MMAs have been waited for
    if (v < U && v % UPT == 0) {                     // the tile of unit v must have landed before its MMAs are issued
      cp_async_wait<0>();
      fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0 && v < U) issue_unit(v);
    alive = __syncthreads_and(mbar_wait(smem_u32(s_bar + (u % NSLOT)), (uint32_t)((u / NSLOT) & 1)));
    if (!alive) break;
    tc_fence_after();
    const uint32_t tbase = tmem + lane_base + (uint32_t)((u % NSLOT) * slot_w);
    const int j0 = j_lo + tile * kKeyTile;

    if (kStats) {
      // this thread's query row, keys [64 * half, 64 * half + 64) of the tile
      const int r = sub * 128 + lane_row;
      const int i = r / a.G;
      const int lim = a.causal ? job.n - a.L_obs + i : 0x7fffffff;  // last key this window row sees
      const int jmax = min(j_hi - 1, lim);                          // keys j <= jmax are live
      float m = s_f[2 * (half * kScoreMaxRows + r)], l = s_f[2 * (half * kScoreMaxRows + r) + 1];
#pragma unroll 1
      for (int c0 = half * 64; c0 < half * 64 + 64; c0 += 32) {
        if (j0 + c0 >= j_hi) break;  // uniform: the rest of the tile is padding
        float x[32];
        tmem_ld32(tbase + c0, x);
        if (j0 + c0 + 31 > jmax) {  // tail of the key range or the causal edge: mask entry by entry
#pragma unroll
          for (int c = 0; c < 32; ++c) x[c] = (j0 + c0 + c <= jmax) ? x[c] : -INFINITY;
        }
        float mx = x[0];
#pragma unroll
        for (int c = 1; c < 32; ++c) mx = fmaxf(mx, x[c]);
        mx *= a.scale_log2;  // the scale is positive: the max commutes with it
        if (mx > m) {
          l *= fast_exp2(m - mx);
          m = mx;
        }
        if (m > -INFINITY) {
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
            s0 += fast_exp2(fmaf(x[c], a.scale_log2, -m));
            s1 += fast_exp2(fmaf(x[c + 1], a.scale_log2, -m));
            s2 += fast_exp2(fmaf(x[c + 2], a.scale_log2, -m));
            s3 += fast_exp2(fmaf(x[c + 3], a.scale_log2, -m));
          }
          l += (s0 + s1) + (s2 + s3);
        }
      }
      s_f[2 * (half * kScoreMaxRows + r)] = m;
      s_f[2 * (half * kScoreMaxRows + r) + 1] = l;
    } else {
      // this thread's key; the unit's rows [r_begin, r_end) are cut, at a multiple of G, between the two halves
      const int j = j0 + lane_row;
      const int r_begin = sub * sh.NW, r_end = min(sh.R, r_begin + sh.NW);
      // column sums cut at a multiple of 32 columns, the matrix at a multiple of G (whole window rows per thread)
      const int cut = MODE == kScoreColsum ? min(r_end, r_begin + ((r_end - r_begin) / 2 + 31) / 32 * 32)
                                           : r_begin + ((r_end - r_begin) / 2 / a.G) * a.G;
      const int r0 = half ? cut : r_begin, r1 = half ? r_end : cut;
      if (MODE == kScoreColsum) {
        if (sub == 0) col_acc = 0.f;
        float c0s = 0.f, c1s = 0.f, c2s = 0.f, c3s = 0.f;
#pragma unroll 1
        for (int rr = r0; rr < r1; rr += 32) {
          float x[32];
          tmem_ld32(tbase + (rr - r_begin), x);
          if (rr + 32 <= r1) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              const float4 mm = *reinterpret_cast<const float4*>(s_f + rr + c);  // rr is a multiple of 16
              c0s += fast_exp2(fmaf(x[c], a.scale_log2, -mm.x));
              c1s += fast_exp2(fmaf(x[c + 1], a.scale_log2, -mm.y));
              c2s += fast_exp2(fmaf(x[c + 2], a.scale_log2, -mm.z));
              c3s += fast_exp2(fmaf(x[c + 3], a.scale_log2, -mm.w));
            }
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (rr + c < r1) c0s += fast_exp2(fmaf(x[c], a.scale_log2, -s_f[rr + c]));
          }
        }
        col_acc += (c0s + c1s) + (c2s + c3s);
        if (sub == UPT - 1) {
          s_col[half * 128 + lane_row] = col_acc;
          __syncthreads();
          if (half == 0 && j < j_hi)
            a.out[(size_t)blockIdx.y * a.out_job_stride + (j - job.j_begin)] = (s_col[lane_row] + s_col[128 + lane_row]) * inv_g;
          // s_col is rewritten one tile later, after several barriers
        }
      } else {
        // group-mean matrix: rows come in runs of G heads per window row; r0 is a multiple of G
        float* A = a.out + (size_t)blockIdx.y * a.out_job_stride;
        int i = r0 / a.G, g = 0;
        float acc = 0.f;
#pragma unroll 1
        for (int rr = r0; rr < r1; rr += 32) {
          float x[32];
          tmem_ld32(tbase + (rr - r_begin), x);
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if (rr + c < r1) {
              const bool seen = !a.causal || j <= job.n - a.L_obs + i;
              acc += seen ? fast_exp2(fmaf(x[c], a.scale_log2, -s_f[rr + c])) : 0.f;
              if (++g == a.G) {
                if (j < j_hi) A[(size_t)i * a.out_row_stride + (j - job.j_begin)] = acc * inv_g;
                acc = 0.f;
                g = 0;
                ++i;
              }
            }
          }
        }
      }
    }
  }

  // ---- drain, release TMEM
  cp_async_wait<0>();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(n_cols) : "memory");
  if (!alive) {
    if (tid == 0) atomicExch(a.status, 1);
    return;
  }
  if (kStats) {
    // two partials per CTA and row: one per column half
    float2* outp = a.stats_part + ((size_t)blockIdx.y * a.n_chunks + blockIdx.x) * (2 * kScoreMaxRows);
    for (int r = tid; r < 2 * kScoreMaxRows; r += kScThreads)
      if ((r & (kScoreMaxRows - 1)) < sh.R) outp[r] = make_float2(s_f[2 * r], s_f[2 * r + 1]);
  }
}

// Merge the per-CTA row partials: stats[job][row] = (max, sum).  One warp per row.
__global__ void __launch_bounds__(256) score_stats_merge_kernel(const ScoreArgs a, int R) {
  const int jobi = blockIdx.y;
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= R) return;
  const ScoreJob job = a.jobs[jobi];
  const int used = (job.j_end - job.j_begin + a.keys_per_cta - 1) / a.keys_per_cta;
  float m = -INFINITY, l = 0.f;
  for (int c = lane; c < 2 * used; c += 32) {
    const float2 p = a.stats_part[((size_t)jobi * a.n_chunks + (c >> 1)) * (2 * kScoreMaxRows) + (c & 1) * kScoreMaxRows + r];
    if (p.x == -INFINITY) continue;
    const float mn = fmaxf(m, p.x);
    l = l * ((m == -INFINITY) ? 0.f : exp2f(m - mn)) + p.y * exp2f(p.x - mn);
    m = mn;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o), ol = __shfl_xor_sync(0xffffffffu, l, o);
    const float mn = fmaxf(m, om);
    l = l * ((m == -INFINITY) ? 0.f : exp2f(m - mn)) + ol * ((om == -INFINITY) ? 0.f : exp2f(om - mn));
    m = mn;
  }
  if (lane == 0) a.stats[(size_t)jobi * kScoreMaxRows + r] = make_float2(m, l);
}

static size_t score_smem_bytes(const ScoreShape& sh) {
  return 1024 + 2 * (size_t)sh.q_rows * 128 + 2 * kKStageBytes + 4 * kScoreMaxRows * sizeof(float) + 4 * sizeof(uint64_t) + 16;
}

template <int MODE>
static int launch_one(const ScoreArgs& a, const ScoreShape& sh, cudaStream_t stream) {
  const size_t smem = score_smem_bytes(sh);
  CATEKV_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  score_tc_kernel<MODE><<<dim3(a.n_chunks, a.n_jobs), kScThreads, smem, stream>>>(a, sh);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}

int score_launch(const ScoreArgs& a, ScoreMode out_mode, cudaStream_t stream) {
  if (a.n_jobs <= 0 || a.n_chunks <= 0) return CATEKV_OK;
  if (a.G * a.L_obs > kScoreMaxRows || a.keys_per_cta % kKeyTile || !a.status) return CATEKV_ERR_UNSUPPORTED;
  const ScoreShape sh = score_shape(a.G, a.L_obs);
  int rc = launch_one<kScoreStats>(a, sh, stream);
  if (rc) return rc;
  score_stats_merge_kernel<<<dim3((sh.R + 7) / 8, a.n_jobs), 256, 0, stream>>>(a, sh.R);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return out_mode == kScoreColsum ? launch_one<kScoreColsum>(a, sh, stream) : launch_one<kScoreMatrix>(a, sh, stream);
}

}  // namespace catekv
