// Observation-window scoring on the 5th-generation tensor cores (TMA + tcgen05 + TMEM).
//
// A CTA scores `keys_per_cta` keys of one (sequence, KV head) against the R = G * L_obs window
// query rows of the group (row r = i * G + g: window row i of the group's g-th query head).
// Q stays in shared memory for the CTA's lifetime; 128-key tiles of K are fetched by TMA
// (cp.async.bulk.tensor, two 64-column boxes per tile) straight into the K-major SWIZZLE_128B
// layout the UMMA descriptors expect, two stages deep.
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
// Warp roles: warp 9 (one elected lane) is the TMA producer: it refills a K stage as soon as the
// MMAs that read it have completed (a tcgen05.commit on the stage's "empty" barrier), however far
// the epilogue lags.  Warp 8 (one elected lane) waits for a K tile, issues the eight k-steps of
// tcgen05.mma per unit and commits them to the unit's "done" barrier; warps 0-7 are the epilogue
// (two groups of four, one warp per TMEM lane quarter): the groups take alternate units, so that
// one group's exponentials overlap the other group's wait, load and maximum; a group waits for its
// unit, reads the accumulators with tcgen05.ld into registers 64 columns at a time, hands the TMEM
// slot back right after its last load and then finishes the exp2 arithmetic.  (The head-major
// matrix mode keeps both groups on every unit, half the columns each.)  There is no CTA-wide
// barrier in the main loop.  Every mbarrier wait is bounded: on
// expiry the thread raises a CTA-wide abort flag (which ends all other waits early) and a status
// word in the workspace; the CTA then frees its TMEM and returns.
#include <cuda.h>
#include <math.h>

#include <atomic>

#include "score.cuh"
#include "tc.cuh"

namespace catekv {

constexpr int kEpiThreads = 256;                   // 8 epilogue warps: two per TMEM lane quarter, each takes half the columns
constexpr int kScThreads = kEpiThreads + 64;       // + the MMA warp (8) and the TMA warp (9)

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

template <int MODE>
__global__ void __launch_bounds__(kScThreads, 2) score_tc_kernel(const __grid_constant__ CUtensorMap k_map, const ScoreArgs a,
                                                              const ScoreShape sh) {
  extern __shared__ uint8_t smem_raw[];
  // Programmatic dependent launch: the next kernel of the chain (merge, second pass, top-k) may be scheduled while
  // this grid drains.  The first pass has nothing to wait for but its inputs, which a stream-ordered copy or a
  // kernel that never signals early produced; the second pass sets up (queries, barriers, tensor memory) and then
  // waits for the merged statistics.
  pdl_launch_dependents();
  if (MODE == kScoreStats) pdl_wait();
  const ScoreJob job = a.jobs[blockIdx.y];
  const int j_lo = job.j_begin + blockIdx.x * a.keys_per_cta;
  if (j_lo >= job.j_end) return;
  const int j_hi = min(job.j_end, j_lo + a.keys_per_cta);
  const int n_tiles = (j_hi - j_lo + kKeyTile - 1) / kKeyTile;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle)
  const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (s_base - smem_u32(smem_raw));
  const uint32_t q_block = (uint32_t)sh.q_rows * 128;  // one k-block of Q
  const uint32_t s_q = s_base;
  const uint32_t s_k = s_q + 2 * q_block;
  float* s_f = reinterpret_cast<float*>(smem + 2 * q_block + 2 * kKStageBytes);  // pass 1: (m, l)[2][512]; pass 2: m'[R]
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_f + 4 * kScoreMaxRows);         // full[2], done[4], free[4], empty[2]
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 12);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const uint32_t bar_full = smem_u32(s_bar), bar_done = smem_u32(s_bar + 2), bar_free = smem_u32(s_bar + 6);
  const uint32_t bar_empty = smem_u32(s_bar + 10);  // a K stage has been read by all the MMAs of its tile

  constexpr bool kStats = MODE == kScoreStats;
  constexpr bool kPingPong = MODE != kScoreMatrix;  // the two groups of four epilogue warps take alternate units
  const int UPT = kStats ? sh.MT : sh.NH;          // MMA units per key tile
  const int NSLOT = kStats ? sh.nslot1 : 2;
  const int slot_w = kStats ? 128 : sh.slotw2;
  const int n_cols = kStats ? sh.cols1 : sh.cols2;
  const int U = n_tiles * UPT;

  // ---- set-up: Q (row r = i * G + g, or g * L_obs + i) by cp.async from all threads, barriers, TMEM
  for (int id = tid; id < sh.q_rows * 16; id += kScThreads) {
    const int r = id >> 4, c = id & 15;
    int i, g;
    if (a.g_major) {
      g = r / a.L_obs;
      i = r - g * a.L_obs;
    } else {
      i = r / a.G;
      g = r - i * a.G;
    }
    const int ok = r < sh.R ? 16 : 0;
    const uint16_t* src = a.q_win + (((int64_t)job.b * a.Hq + job.h * a.G + (ok ? g : 0)) * a.L_obs + (ok ? i : 0)) * kD + c * 8;
    cp_async16(s_q + sw128_off(r, c, sh.q_rows), src, ok);
  }
  cp_async_commit();
  if (kStats) {
    for (int i = tid; i < 2 * kScoreMaxRows; i += kScThreads) {
      s_f[2 * i] = -INFINITY;
      s_f[2 * i + 1] = 0.f;
    }
  } else {
    // m'_r = m_r + log2(l_r): exp2(x - m'_r) is the normalised probability; rows without mass get +inf (-> 0)
    pdl_wait();  // the statistics are the preceding kernel's output
    const float2* st = a.stats + (size_t)blockIdx.y * kScoreMaxRows;
    for (int r = tid; r < sh.R; r += kScThreads) {
      const float2 v = st[r];
      s_f[r] = v.y > 0.f ? v.x + log2f(v.y) : INFINITY;
    }
  }
  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < 2; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(bar_full + 8 * i));
    for (int i = 0; i < 4; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(bar_done + 8 * i));
    // a slot is handed back by the epilogue warps that read it: the 4 warps of the group that owns the unit, or
    // (matrix mode) all 8, two per lane quarter with half the columns each
    for (int i = 0; i < 4; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar_free + 8 * i), "r"(kPingPong ? 4 : 8));
    for (int i = 0; i < 2; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(bar_empty + 8 * i));
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(s_tmem)), "r"(n_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  cp_async_wait<0>();
  fence_async_smem();  // Q was written through the generic proxy; the MMAs read it through the async proxy
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // K tile `tile` -> stage tile & 1: two boxes of 64 columns (one k-block each), 32 KB on the stage's barrier
  auto load_tile = [&](int tile) {
    const uint32_t sb = s_k + (tile & 1) * kKStageBytes;
    const uint32_t bar = bar_full + 8 * (tile & 1);
    mbar_expect_tx(bar, kKStageBytes);
    tma_load_box(sb, &k_map, 0, j_lo + tile * kKeyTile, job.h, job.b, bar);
    tma_load_box(sb + kKBlockBytes, &k_map, 64, j_lo + tile * kKeyTile, job.h, job.b, bar);
  };

  if (warp == 8) {
    // ================= TMA + MMA issue: one elected lane =================
    if (lane == 0 && !a.idle_producer) {
      const uint32_t idesc = kStats ? umma_idesc_bf16(128, 128) : umma_idesc_bf16(128, sh.NW);
      for (int v = 0; v < U; ++v) {
        const int tile = v / UPT, sub = v - tile * UPT;
        if (sub == 0 && !mbar_wait(bar_full + 8 * (tile & 1), (uint32_t)((tile >> 1) & 1), s_abort, a.spin_limit)) break;
        if (v >= NSLOT && !mbar_wait(bar_free + 8 * (v % NSLOT), (uint32_t)(((v / NSLOT) - 1) & 1), s_abort, a.spin_limit)) break;
        tc_fence_after();
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
        umma_commit(bar_done + 8 * (v % NSLOT));
        if (sub == UPT - 1) umma_commit(bar_empty + 8 * (tile & 1));  // the tile's stage may be refilled once these MMAs are done
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ================= TMA producer: one elected lane keeps both K stages in flight =================
    if (lane == 0 && !a.idle_producer) {
      for (int tile = 0; tile < n_tiles; ++tile) {
        if (tile >= 2 && !mbar_wait(bar_empty + 8 * (tile & 1), (uint32_t)(((tile >> 1) - 1) & 1), s_abort, a.spin_limit)) break;
        load_tile(tile);
      }
    }
    __syncwarp();
  } else {
    // ================= epilogue warps =================
    // warp w reads TMEM lanes 32 * (w % 4) ...; warps 0-3 take the first half of a unit's columns, warps 4-7 the second
    const int lane_row = (warp & 3) * 32 + lane;  // this thread's TMEM lane: a query row (pass 1) or a key (pass 2)
    const int half = warp >> 2;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float inv_g = 1.f / (float)a.G;
    float col_acc = 0.f;  // pass 2, column sums: this key's sum over this thread's rows of the tile
    float macc[32];       // pass 2, head-major matrix: this key's entries of this thread's 32 window rows

    // hand the TMEM slot of unit u back to the MMA warp: once per epilogue warp, after its last load of the unit
    auto release_slot = [&](int u) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_free + 8 * (u % NSLOT));
    };

    // Row statistics and column sums: the two groups of four warps take alternate units (a group reads all the
    // columns of its units), so that one group's exponentials overlap the other group's wait, load and maximum.
    // Matrix mode: both groups work on every unit, half the columns each.
    for (int u = kPingPong ? half : 0; u < U; u += kPingPong ? 2 : 1) {
      const int tile = u / UPT, sub = u - tile * UPT;
      if (!mbar_wait(bar_done + 8 * (u % NSLOT), (uint32_t)((u / NSLOT) & 1), s_abort, a.spin_limit)) break;
      tc_fence_after();
      const uint32_t tbase = tmem + lane_base + (uint32_t)((u % NSLOT) * slot_w);
      const int j0 = j_lo + tile * kKeyTile;

      if (kStats) {
        // this thread's query row against the tile's 128 keys, 64 columns at a time; after the second load the TMEM
        // slot goes straight back to the MMA warp (the arithmetic runs on registers)
        const int r = sub * 128 + lane_row;
        const int i = a.g_major ? r % a.L_obs : r / a.G;
        const int lim = a.causal ? job.n - a.L_obs + i : 0x7fffffff;  // last key this window row sees
        const int jmax = min(j_hi - 1, lim);                          // keys j <= jmax are live
        float m = s_f[2 * (half * kScoreMaxRows + r)], l = s_f[2 * (half * kScoreMaxRows + r) + 1];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int c0 = hh * 64;
          const bool any = j0 + c0 < j_hi;  // uniform: otherwise this half of the tile is padding
          float x[64];
          if (any) {
            tmem_ld64(tbase + c0, x);
            tmem_wait_ld64(x);
          }
          if (hh == 1) release_slot(u);
          if (any) {
            if (j0 + c0 + 63 > jmax) {  // tail of the key range or the causal edge: mask entry by entry
#pragma unroll
              for (int c = 0; c < 64; ++c) x[c] = (j0 + c0 + c <= jmax) ? x[c] : -INFINITY;
            }
            // four independent chains of three-input maxima
            float mx0 = fmax3(x[0], x[1], x[2]), mx1 = fmax3(x[3], x[4], x[5]);
            float mx2 = fmax3(x[6], x[7], x[8]), mx3 = fmax3(x[9], x[10], x[11]);
#pragma unroll
            for (int c = 12; c < 60; c += 8) {
              mx0 = fmax3(mx0, x[c], x[c + 1]);
              mx1 = fmax3(mx1, x[c + 2], x[c + 3]);
              mx2 = fmax3(mx2, x[c + 4], x[c + 5]);
              mx3 = fmax3(mx3, x[c + 6], x[c + 7]);
            }
            mx0 = fmax3(mx0, x[60], x[61]);
            mx1 = fmax3(mx1, x[62], x[63]);
            float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            mx *= a.scale_log2;  // the scale is positive: the max commutes with it
            if (mx > m) {
              l *= fast_exp2(m - mx);
              m = mx;
            }
            if (m > -INFINITY) {
              float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
              for (int c = 0; c < 64; c += 4) {
                s0 += fast_exp2(fmaf(x[c], a.scale_log2, -m));
                s1 += fast_exp2(fmaf(x[c + 1], a.scale_log2, -m));
                s2 += fast_exp2(fmaf(x[c + 2], a.scale_log2, -m));
                s3 += fast_exp2(fmaf(x[c + 3], a.scale_log2, -m));
              }
              l += (s0 + s1) + (s2 + s3);
            }
          }
        }
        s_f[2 * (half * kScoreMaxRows + r)] = m;
        s_f[2 * (half * kScoreMaxRows + r) + 1] = l;
      } else {
        // this thread's key against the unit's rows [r_begin, r_end)
        const int j = j0 + lane_row;
        const int r_begin = sub * sh.NW, r_end = min(sh.R, r_begin + sh.NW);
        // column sums: all of the unit's rows; matrix: the rows are cut between the halves at a multiple of G
        const int cut = r_begin + ((r_end - r_begin) / 2 / a.G) * a.G;
        const int r0 = MODE == kScoreColsum ? r_begin : (half ? cut : r_begin);
        const int r1 = MODE == kScoreColsum ? r_end : (half ? r_end : cut);
        if (MODE == kScoreColsum) {
          col_acc = 0.f;
          float c0s = 0.f, c1s = 0.f, c2s = 0.f, c3s = 0.f;
          // 64 rows per load where that many are left, else 32; the slot is handed back after the last load
#pragma unroll 1
          for (int rr = r0; rr < r1;) {
            const int left = r1 - rr;
            if (left > 32) {
              float x[64];
              tmem_ld64(tbase + (rr - r_begin), x);
              tmem_wait_ld64(x);
              if (rr + 64 >= r1) release_slot(u);
              if (left >= 64) {
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
                  const float4 mm = *reinterpret_cast<const float4*>(s_f + rr + c);  // rr is a multiple of 16
                  c0s += fast_exp2(fmaf(x[c], a.scale_log2, -mm.x));
                  c1s += fast_exp2(fmaf(x[c + 1], a.scale_log2, -mm.y));
                  c2s += fast_exp2(fmaf(x[c + 2], a.scale_log2, -mm.z));
                  c3s += fast_exp2(fmaf(x[c + 3], a.scale_log2, -mm.w));
                }
              } else {
#pragma unroll
                for (int c = 0; c < 64; ++c)
                  if (c < left) c0s += fast_exp2(fmaf(x[c], a.scale_log2, -s_f[rr + c]));
              }
              rr += 64;
            } else {
              float x[32];
              tmem_ld32(tbase + (rr - r_begin), x);
              tmem_wait_ld32(x);
              release_slot(u);  // at most 32 rows were left: this was the last load
              if (left == 32) {
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                  const float4 mm = *reinterpret_cast<const float4*>(s_f + rr + c);
                  c0s += fast_exp2(fmaf(x[c], a.scale_log2, -mm.x));
                  c1s += fast_exp2(fmaf(x[c + 1], a.scale_log2, -mm.y));
                  c2s += fast_exp2(fmaf(x[c + 2], a.scale_log2, -mm.z));
                  c3s += fast_exp2(fmaf(x[c + 3], a.scale_log2, -mm.w));
                }
              } else {
#pragma unroll
                for (int c = 0; c < 32; ++c)
                  if (c < left) c0s += fast_exp2(fmaf(x[c], a.scale_log2, -s_f[rr + c]));
              }
              rr += 32;
            }
          }
          if (r0 >= r1) release_slot(u);  // nothing to read for this thread's half
          col_acc += (c0s + c1s) + (c2s + c3s);
          // One unit per tile: this thread holds the key's whole sum.  Two units per tile (more than 256 rows):
          // they belong to different groups, whose threads add their shares to the zero-initialised output
          // (0 + x + y is the same in either order, so the result does not depend on timing).
          if (j < j_hi) {
            float* dst = a.out + (size_t)blockIdx.y * a.out_job_stride + (j - job.j_begin);
            if (UPT == 1) *dst = col_acc * inv_g;
            else atomicAdd(dst, col_acc * inv_g);
          }
        } else if (a.g_major) {
          // group-mean matrix with head-major rows and L_obs = 64: this thread owns the window rows 32 * half + c
          // (c = 0..31) of its key; head g's logits for them are the 32 TMEM columns from g * 64 + 32 * half on, so
          // the mean over the heads is a register accumulation without any bookkeeping
          float* A = a.out + (size_t)blockIdx.y * a.out_job_stride;
          const int m_cols = job.j_end - job.j_begin;
          if (sub == 0) {
#pragma unroll
            for (int c = 0; c < 32; ++c) macc[c] = 0.f;
          }
          const int i_min = j - (job.n - a.L_obs);  // causal: window row i sees key j iff i >= i_min
          const bool edge = a.causal && __any_sync(0xffffffffu, i_min > half * 32);
          // the heads whose 32 columns lie in this unit are consecutive; they are read 16 columns at a time, the
          // next load in flight while the current one's exponentials run, and the slot goes back to the MMA warp
          // after the last load.  Piece p: head p / 2, columns 16 * (p % 2) of this thread's 32.
          auto add_piece = [&](const float (&x)[16], int p) {
            const int col = (p >> 1) * 64 + half * 32 + (p & 1) * 16;
            const int cb = (p & 1) * 16;
#pragma unroll
            for (int c = 0; c < 16; c += 4) {
              const float4 mm = *reinterpret_cast<const float4*>(s_f + col + c);
              float e0 = fast_exp2(fmaf(x[c], a.scale_log2, -mm.x));
              float e1 = fast_exp2(fmaf(x[c + 1], a.scale_log2, -mm.y));
              float e2 = fast_exp2(fmaf(x[c + 2], a.scale_log2, -mm.z));
              float e3 = fast_exp2(fmaf(x[c + 3], a.scale_log2, -mm.w));
              if (edge) {
                const int i0 = half * 32 + cb + c;
                e0 = i0 >= i_min ? e0 : 0.f;
                e1 = i0 + 1 >= i_min ? e1 : 0.f;
                e2 = i0 + 2 >= i_min ? e2 : 0.f;
                e3 = i0 + 3 >= i_min ? e3 : 0.f;
              }
              if (p & 1) {
                macc[16 + c] += e0, macc[17 + c] += e1, macc[18 + c] += e2, macc[19 + c] += e3;
              } else {
                macc[c] += e0, macc[c + 1] += e1, macc[c + 2] += e2, macc[c + 3] += e3;
              }
            }
          };
          auto in_unit = [&](int gg) {
            const int col = gg * 64 + half * 32;
            return gg < a.G && col >= r_begin && col < r_end;
          };
          auto taddr_of = [&](int p) { return tbase + (uint32_t)((p >> 1) * 64 + half * 32 + (p & 1) * 16 - r_begin); };
          int g_first = 0;
          while (g_first < a.G && !in_unit(g_first)) ++g_first;
          int g_last = g_first;
          while (in_unit(g_last)) ++g_last;  // one past the unit's last head
          if (g_first < g_last) {
            float xa[16], xb[16];
            int p = 2 * g_first;
            const int p_end = 2 * g_last;  // an even number of pieces
            tmem_ld16(taddr_of(p), xa);
            tmem_wait_ld16(xa);
#pragma unroll 1
            for (; p < p_end; p += 2) {
              tmem_ld16(taddr_of(p + 1), xb);
              add_piece(xa, p);
              tmem_wait_ld16(xb);
              const bool more = p + 2 < p_end;
              if (more) tmem_ld16(taddr_of(p + 2), xa);
              else release_slot(u);
              add_piece(xb, p + 1);
              if (more) tmem_wait_ld16(xa);
            }
          } else {
            release_slot(u);
          }
          if (sub == UPT - 1 && j < j_hi) {
#pragma unroll
            for (int c = 0; c < 32; ++c) A[(size_t)(half * 32 + c) * m_cols + (j - job.j_begin)] = macc[c] * inv_g;
          }
        } else {
          // group-mean matrix, stored densely ([L_obs][m], m = the job's key range): rows come in runs of G heads per
          // window row; r0 is a multiple of G
          float* A = a.out + (size_t)blockIdx.y * a.out_job_stride;
          const int m_cols = job.j_end - job.j_begin;
          int i = r0 / a.G, g = 0;
          float acc = 0.f;
#pragma unroll 1
          for (int rr = r0; rr < r1; rr += 32) {
            float x[32];
            tmem_ld32(tbase + (rr - r_begin), x);
            tmem_wait_ld32(x);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              if (rr + c < r1) {
                const bool seen = !a.causal || j <= job.n - a.L_obs + i;
                acc += seen ? fast_exp2(fmaf(x[c], a.scale_log2, -s_f[rr + c])) : 0.f;
                if (++g == a.G) {
                  if (j < j_hi) A[(size_t)i * m_cols + (j - job.j_begin)] = acc * inv_g;
                  acc = 0.f;
                  g = 0;
                  ++i;
                }
              }
            }
          }
        }
      }
      if (MODE == kScoreMatrix && !a.g_major) release_slot(u);  // the others handed it back right after their last load
    }
  }

  // ---- release TMEM (after an abort: first give copies that may still be in flight time to land)
  if (*s_abort)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(n_cols) : "memory");
  if (*s_abort) {
    if (tid == 0) raise_status(a.status, CATEKV_STATUS_WAIT_EXPIRED, kKidScore, (int)blockIdx.y, (int)blockIdx.x);
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
  pdl_launch_dependents();
  pdl_wait();  // the partials are the preceding kernel's output
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
  return 1024 + 2 * (size_t)sh.q_rows * 128 + 2 * kKStageBytes + 4 * kScoreMaxRows * sizeof(float) + 12 * sizeof(uint64_t) + 16;
}

// Test hook (catekv_test_expire_score_waits): launches left that run with an idle producer lane.
static std::atomic<int> g_expire_launches{0};

// true if this launch is one of those the test hook asked to run with an idle producer lane
bool score_take_expire_launch() {
  int left = g_expire_launches.load(std::memory_order_relaxed);
  while (left > 0 && !g_expire_launches.compare_exchange_weak(left, left - 1)) {
  }
  return left > 0;
}

template <int MODE>
static int launch_one(const ScoreArgs& a0, const ScoreShape& sh, const CUtensorMap& map, cudaStream_t stream) {
  ScoreArgs a = a0;
  a.spin_limit = kSpinLimit;
  a.idle_producer = 0;
  if (score_take_expire_launch()) {
    a.spin_limit = 512;
    a.idle_producer = 1;
  }
  const size_t smem = score_smem_bytes(sh);
  CATEKV_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  CATEKV_CUDA_TRY(launch_pdl(score_tc_kernel<MODE>, dim3(a.n_chunks, a.n_jobs), dim3(kScThreads), smem, stream, map, a, sh));
  return CATEKV_OK;
}

int score_keys_per_cta(int n_jobs, int max_keys) {
  if (n_jobs < 1) n_jobs = 1;
  const int ctas = 2 * sm_count();                 // the kernel runs two CTAs per SM
  int chunks = (ctas + n_jobs / 2) / n_jobs;  // about one full wave in all
  if (chunks < 1) chunks = 1;
  int kp = ((max_keys + chunks - 1) / chunks + kKeyTile - 1) / kKeyTile * kKeyTile;
  if (kp < 4 * kKeyTile) kp = 4 * kKeyTile;  // at least a few tiles per CTA: the queries are staged once per CTA
  return kp;
}

int score_launch(const ScoreArgs& a0, ScoreMode out_mode, cudaStream_t stream) {
  if (a0.n_jobs <= 0 || a0.max_keys <= 0) return CATEKV_OK;
  if (a0.G * a0.L_obs > kScoreMaxRows || !a0.status) return CATEKV_ERR_UNSUPPORTED;
  if (a0.g_major && (a0.L_obs != 64 || out_mode != kScoreMatrix)) return CATEKV_ERR_UNSUPPORTED;
  const ScoreShape sh = score_shape(a0.G, a0.L_obs);
  CUtensorMap map;
  const KvTensor kt = {a0.k, a0.sb, a0.sh, a0.st, a0.B, a0.Hkv, a0.n_max};
  int rc = make_kv_map(kt, &map);
  if (rc) return rc;
  if (out_mode == kScoreColsum && sh.NH > 1)  // two units per tile add their shares into a zeroed vector
    CATEKV_CUDA_TRY(cudaMemsetAsync(a0.out, 0, sizeof(float) * (size_t)a0.n_jobs * a0.out_job_stride, stream));
  // (Scoring the jobs in groups whose keys fit the L2 together, both passes of a group back to back, was measured
  // and lost: the smaller grids and extra launches cost more than the second pass gains from L2 hits.)
  ScoreArgs a = a0;
  a.keys_per_cta = score_keys_per_cta(a.n_jobs_split > 0 ? a.n_jobs_split : a.n_jobs, a.max_keys);
  a.n_chunks = (a.max_keys + a.keys_per_cta - 1) / a.keys_per_cta;  // jobs * chunks <= score_max_ctas(jobs): fits the partials
  if (!a.stats_given) {
    rc = launch_one<kScoreStats>(a, sh, map, stream);
    if (rc) return rc;
    CATEKV_CUDA_TRY(launch_pdl(score_stats_merge_kernel, dim3((sh.R + 7) / 8, a.n_jobs), dim3(256), 0, stream, a, sh.R));
  }
  if (out_mode == kScoreStats) return CATEKV_OK;  // the caller wants the row statistics only
  return out_mode == kScoreColsum ? launch_one<kScoreColsum>(a, sh, map, stream) : launch_one<kScoreMatrix>(a, sh, map, stream);
}

}  // namespace catekv

extern "C" void catekv_test_expire_score_waits(int32_t n_launches) {
  catekv::g_expire_launches.store(n_launches > 0 ? n_launches : 0);
}
