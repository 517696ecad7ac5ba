// Attention of the observation window (Algorithm 1, pre-filling stage): the causal attention rows of the last L_obs
// prefill queries of every query head - what a prefill attention pass produces for those positions - together with
// their log-sum-exp and the log-sum-exp over the scored keys [0, n - L_obs) alone, which is the softmax normaliser
// of the token-criticality line.  catekv_select_compact takes the latter in place of its own first pass over K.
//
// One sweep over K and V.  window_pv_kernel: a CTA owns a range of keys of one (sequence, KV head) and 128 query
// rows, which it keeps in tensor memory.  Per 128-key tile: S = Q K^T (tcgen05.mma with Q as the A operand from
// TMEM, so that only the K tile is fetched from shared memory, into one of two TMEM slots); an epilogue thread owns a query row
// and 64 of the tile's keys: it finds their maximum, the row's threads agree on the row's reference value, and it
// turns its part of S into P = exp2(logit - ref), adds the row sums (all visible keys; scored keys only) and writes P
// back over the same TMEM columns as a bf16 hi + lo pair (hi in the first 16 of every 32 columns, lo in the last 16,
// two values per column).  P never touches shared memory: 16 more tcgen05.mma take it from TMEM as their A operand
// and add P_hi V and P_lo V (V as the MN-major B operand, straight from the TMA tile) to O in TMEM.  The reference
// only moves when a tile's maximum exceeds it by more than 2^8 (P stays below 256, far inside what bf16 hi + lo and
// the fp32 accumulator carry); then the row's O is read from TMEM, scaled and stored back before the tile's P V is
// issued.  The ranges' partial results (O, reference, sums) are merged in range order by window_reduce_kernel,
// which also writes the two log-sum-exps.
//
// Warp roles: warps 17 and 18 (one lane each) feed the three K stages and the three V stages by TMA; warp 16 (one
// lane) issues every MMA: S(0), S(1), then per tile P V(t) followed by S(t + 2) into the slot P V(t) has just read
// (the tensor pipe keeps issue order); warps 0-15 are the epilogue, two groups of eight (two warps per TMEM lane
// quarter: 64 keys each) that take alternate tiles in alternate slots, so that one group's exponentials overlap the
// other group's loads, maxima and hand-shakes.  Only the decision "does the reference move" is serial from tile to
// tile (a barrier between the groups; the reference sits in shared memory).  Every mbarrier wait is bounded: on
// expiry the CTA raises the abort flag, frees its tensor memory, records CATEKV_STATUS_WAIT_EXPIRED and returns.
#include <math.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "score.cuh"
#include "tc.cuh"

namespace catekv {

constexpr int kWaEpiWarps = 16;                     // two groups of eight: two warps per TMEM lane quarter and group
constexpr int kWaSub = 4;                           // epilogue threads per query row (2 groups x 2 halves)
constexpr int kWaThreads = (kWaEpiWarps + 3) * 32;  // + the MMA warp and the two TMA warps (K, V)
constexpr int kWaKStages = 3, kWaVStages = 3;
constexpr int kWaTmemCols = 512;         // S / P slots at columns 0 and 128, O at 256, Q (bf16, two per column) at 384
constexpr int kWaOCol = 256, kWaQCol = 384;
constexpr int kWaTileBytes = 128 * 256;  // a [128 x 128] bf16 tile: a K or V stage
constexpr int kWaStateWords = 1 + 2 * kWaSub;  // per row and key range: reference, the threads' sums (visible keys), (scored keys)
constexpr float kWaTau = 8.f;            // a row's reference follows a tile maximum that exceeds it by more than 2^kWaTau
constexpr int kWaBarriers = 36;
constexpr size_t kWaSmemBytes = 1024 + (size_t)(kWaKStages + kWaVStages) * kWaTileBytes + (4 * 128 + 256) * sizeof(float) +
                                kWaBarriers * sizeof(uint64_t) + 16;
static_assert(kWaSmemBytes <= 227 * 1024, "window_pv_kernel: one CTA's shared memory");

struct WinArgs {
  const uint16_t* q_win;  // [B, Hq, L_obs, d]
  const ScoreJob* jobs;   // [n_segs]: b, h, n (j_begin / j_end unused)
  int32_t G, L_obs, R, Hq;
  float scale_log2;
  int32_t keys_per_cta, n_chunks;
  float* part;            // [n_segs][MT][n_chunks][128 rows][128 d]: O relative to the range's reference
  float* part_s;          // [n_segs][MT][n_chunks][kWaStateWords][128 rows]: reference (log2 domain), the row's threads'
                          //                                       sums over the visible keys, over the scored keys
  int32_t* status;
  uint32_t spin_limit;
  int32_t idle_producer;  // test hook: the TMA and MMA lanes issue nothing, so every wait runs out
};

__device__ __forceinline__ float max32(const float (&x)[32]) {
  float m0 = fmax3(x[0], x[1], x[2]), m1 = fmax3(x[3], x[4], x[5]);
  float m2 = fmax3(x[6], x[7], x[8]), m3 = fmax3(x[9], x[10], x[11]);
#pragma unroll
  for (int c = 12; c < 28; c += 8) {
    m0 = fmax3(m0, x[c], x[c + 1]);
    m1 = fmax3(m1, x[c + 2], x[c + 3]);
    m2 = fmax3(m2, x[c + 4], x[c + 5]);
    m3 = fmax3(m3, x[c + 6], x[c + 7]);
  }
  m0 = fmax3(m0, x[28], x[29]);
  m1 = fmax3(m1, x[30], x[31]);
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

__global__ void __launch_bounds__(kWaThreads, 1) window_pv_kernel(const __grid_constant__ CUtensorMap k_map,
                                                                const __grid_constant__ CUtensorMap v_map, const WinArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const ScoreJob job = a.jobs[blockIdx.y];
  const int mt = blockIdx.z;
  const int n = job.n;
  const int j_lo = blockIdx.x * a.keys_per_cta;
  if (j_lo >= n) return;  // the reduction knows how many ranges a sequence of n keys has
  const int j_hi = min(n, j_lo + a.keys_per_cta);
  const int n_tiles = (j_hi - j_lo + kKeyTile - 1) / kKeyTile;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const uint32_t s_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (s_base - smem_u32(smem_raw));
  const uint32_t s_k = s_base;
  const uint32_t s_v = s_k + kWaKStages * kWaTileBytes;
  float* s_xch = reinterpret_cast<float*>(smem + (kWaKStages + kWaVStages) * kWaTileBytes);  // [group][half][row]: part-tile maxima
  float* s_ref = s_xch + 4 * 128;  // [tile parity][row]: the row's reference after the decision for a tile of that parity
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_ref + 256);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + kWaBarriers);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const uint32_t bar0 = smem_u32(s_bar);
  auto B = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  // barrier indices
  constexpr int kFullK = 0, kEmptyK = 3, kFullV = 6, kEmptyV = 9, kDoneS = 12, kPReady = 14, kPvDone = 16, kDoneO = 17, kDec = 18,
                kXw = 19, kXr = 27;  // kXw / kXr: [group][quarter]
  static_assert(kXr + 8 <= kWaBarriers, "barrier table");

  // ---- set-up: the row references, barriers, tensor memory; then this M tile's query rows (row r = i * G + g) go
  // into tensor memory, where the S MMAs take them as their A operand (lane = row, two bf16 per column)
  for (int row = tid; row < 256; row += kWaThreads) s_ref[row] = -INFINITY;
  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < kWaBarriers; ++i) {
      // arrivals: the 8 warps of an epilogue group (P ready, decision), the 2 warps of a group's lane quarter (maxima), else one
      const int count = (i == kPReady || i == kPReady + 1 || i == kDec) ? 8 : (i >= kXw ? 2 : 1);
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(B(i)), "r"(count));
    }
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == kWaEpiWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(s_tmem)), "r"(kWaTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  if (warp < kWaEpiWarps) {
    // four threads per row, 32 of its 128 values (16 columns) each
    const int row = (warp & 3) * 32 + lane, part = warp >> 2;
    const int r = mt * 128 + row;
    uint32_t w[16];
    if (r < a.R) {
      const int i = r / a.G, g = r - i * a.G;
      const uint4* src = reinterpret_cast<const uint4*>(a.q_win + (((int64_t)job.b * a.Hq + job.h * a.G + g) * a.L_obs + i) * kD + part * 32);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 v = __ldg(src + c);
        w[4 * c] = v.x, w[4 * c + 1] = v.y, w[4 * c + 2] = v.z, w[4 * c + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int c = 0; c < 16; ++c) w[c] = 0u;
    }
    tmem_st16u(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(kWaQCol + part * 16), w);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  if (warp == kWaEpiWarps + 1) {
    // ================= TMA producer, K: three stages, refilled as soon as the S that read one has completed
    if (lane == 0 && !a.idle_producer) {
      for (int t = 0; t < n_tiles; ++t) {
        const int st = t % kWaKStages, use = t / kWaKStages;
        if (use >= 1 && !mbar_wait(B(kEmptyK + st), (uint32_t)((use - 1) & 1), s_abort, a.spin_limit)) break;
        const int j0 = j_lo + t * kKeyTile;
        mbar_expect_tx(B(kFullK + st), kWaTileBytes);
        tma_load_box(s_k + st * kWaTileBytes, &k_map, 0, j0, job.h, job.b, B(kFullK + st));
        tma_load_box(s_k + st * kWaTileBytes + kKBlockBytes, &k_map, 64, j0, job.h, job.b, B(kFullK + st));
      }
    }
    __syncwarp();
  } else if (warp == kWaEpiWarps + 2) {
    // ================= TMA producer, V: three stages, refilled when the P V that read one has completed
    if (lane == 0 && !a.idle_producer) {
      for (int t = 0; t < n_tiles; ++t) {
        const int st = t % kWaVStages, use = t / kWaVStages;
        if (use >= 1 && !mbar_wait(B(kEmptyV + st), (uint32_t)((use - 1) & 1), s_abort, a.spin_limit)) break;
        const int j0 = j_lo + t * kKeyTile;
        mbar_expect_tx(B(kFullV + st), kWaTileBytes);
        tma_load_box(s_v + st * kWaTileBytes, &v_map, 0, j0, job.h, job.b, B(kFullV + st));
        tma_load_box(s_v + st * kWaTileBytes + kKBlockBytes, &v_map, 64, j0, job.h, job.b, B(kFullV + st));
      }
    }
    __syncwarp();
  } else if (warp == kWaEpiWarps) {
    // ================= MMA issue: S(0), S(1), then per tile P V(t) and S(t + 2) into the slot P V(t) has just read
    if (lane == 0 && !a.idle_producer) {
      const uint32_t idesc_s = umma_idesc_bf16(128, 128);      // S[rows x keys]: A = Q (in TMEM), B = K (K-major)
      const uint32_t idesc_o = umma_idesc_bf16_bmn(128, 128);  // O[rows x d]: A = P (in TMEM), B = V (MN-major)
      // B descriptors as (low, high) halves: high is constant, low = (address >> 4) + constants
      const uint64_t dk0 = umma_desc_sw128(s_k), dv0 = umma_desc_sw128_mn(s_v, kKBlockBytes);
      const uint32_t dk_hi = (uint32_t)(dk0 >> 32), dv_hi = (uint32_t)(dv0 >> 32);
      const uint32_t dk_lo0 = (uint32_t)dk0, dv_lo0 = (uint32_t)dv0;
      auto issue_s = [&](int t) -> bool {
        const int st = t % kWaKStages;
        if (!mbar_wait(B(kFullK + st), (uint32_t)((t / kWaKStages) & 1), s_abort, a.spin_limit)) return false;
        tc_fence_after();
        const uint32_t lo = dk_lo0 + (uint32_t)(st * (kWaTileBytes >> 4));
        const uint32_t d = tmem + (uint32_t)((t & 1) * 128);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)  // 16 of the 128 head dimensions per step: 8 columns of Q in TMEM, 32 bytes of every K row
          umma_bf16_ta_lohi(d, tmem + (uint32_t)(kWaQCol + kk * 8), lo + (uint32_t)((kk >> 2) * (kKBlockBytes >> 4) + (kk & 3) * 2),
                            dk_hi, idesc_s, kk ? 1u : 0u);
        umma_commit(B(kDoneS + (t & 1)));
        umma_commit(B(kEmptyK + st));
        return true;
      };
      bool ok = issue_s(0) && (n_tiles < 2 || issue_s(1));
      for (int t = 0; ok && t < n_tiles; ++t) {
        const int g = t & 1, sv_st = t % kWaVStages;
        if (!mbar_wait(B(kPReady + g), (uint32_t)((t >> 1) & 1), s_abort, a.spin_limit)) break;
        if (!mbar_wait(B(kFullV + sv_st), (uint32_t)((t / kWaVStages) & 1), s_abort, a.spin_limit)) break;
        tc_fence_after();
        const uint32_t lo = dv_lo0 + (uint32_t)(sv_st * (kWaTileBytes >> 4));
        const uint32_t slot = tmem + (uint32_t)(g * 128);
        const uint32_t first = t ? 1u : 0u;
        // P of the 32-key block b of the tile sits in the block's own 32 columns of the slot: hi in the first 16
        // (two bf16 per column), lo in the last 16; a k-step is 16 keys = 8 columns of P and 2 KB of the V tile
#pragma unroll
        for (int part = 0; part < 2; ++part) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_bf16_ta_lohi(tmem + kWaOCol, slot + (uint32_t)((kk >> 1) * 32 + part * 16 + (kk & 1) * 8), lo + (uint32_t)(kk * 128), dv_hi,
                              idesc_o, (part | kk) ? 1u : first);
        }
        umma_commit(B(kPvDone));
        umma_commit(B(kEmptyV + sv_st));
        if (t == n_tiles - 1) umma_commit(B(kDoneO));
        if (t + 2 < n_tiles && !issue_s(t + 2)) break;  // executes after P V(t): the tensor pipe keeps issue order
      }
    }
    __syncwarp();
  } else {
    // ================= epilogue: group g = warp / 8 takes the tiles t = g, g + 2, ... in slot g
    const int g = warp >> 3;
    const int quarter = warp & 3, half = (warp >> 2) & 1;  // TMEM lane quarter; keys [64 half, 64 half + 64) of the tile
    const int lane_row = quarter * 32 + lane;              // this thread's TMEM lane = its query row of the M tile
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int r = mt * 128 + lane_row;
    const bool row_ok = r < a.R;
    const int pos = n - a.L_obs + (row_ok ? r / a.G : 0);  // the row's own position: it sees keys j <= pos
    const int n_sc = n - a.L_obs;                           // keys below are scored keys
    const uint32_t s_slot = tmem + lane_base + (uint32_t)(g * 128 + half * 64);
    float* xch_mine = s_xch + (g * 2 + half) * 128 + lane_row;
    const float* xch_other = s_xch + (g * 2 + (half ^ 1)) * 128 + lane_row;
    // The four threads of a row (two groups x two halves) share one reference, kept in shared memory: the decision
    // for tile t (does the reference move?) follows the decision for tile t - 1 of the other group, but only the
    // short decision is serial: the exponentials of a tile run while the other group is at work on the next one.
    float my_ref = -INFINITY, l = 0.f, lsc = 0.f;  // this thread's sums and the reference they are relative to
    bool alive = true;
    for (int t = g; t < n_tiles; t += 2) {
      const int use = t >> 1;
      if (!mbar_wait(B(kDoneS + g), (uint32_t)(use & 1), s_abort, a.spin_limit)) { alive = false; break; }
      tc_fence_after();
      const int jb = j_lo + t * kKeyTile + half * 64;  // key of this thread's first column
      const bool edge = jb + 63 >= n_sc;               // uniform: the block reaches the window's own keys (or the end)
      // ---- pass 1: this thread's maximum over the keys its row sees, exchanged with the other half
      float mx = -INFINITY;
#pragma unroll
      for (int blk = 0; blk < 2; ++blk) {
        float x[32];
        tmem_ld32(s_slot + blk * 32, x);
        tmem_wait_ld32(x);
        if (edge) {
#pragma unroll
          for (int c = 0; c < 32; ++c) x[c] = (jb + blk * 32 + c <= pos) ? x[c] : -INFINITY;
        }
        mx = fmaxf(mx, max32(x));
      }
      if (use >= 1 && !mbar_wait(B(kXr + g * 4 + quarter), (uint32_t)((use - 1) & 1), s_abort, a.spin_limit)) { alive = false; break; }
      *xch_mine = mx;
      __syncwarp();
      if (lane == 0) mbar_arrive(B(kXw + g * 4 + quarter));
      if (!mbar_wait(B(kXw + g * 4 + quarter), (uint32_t)(use & 1), s_abort, a.spin_limit)) { alive = false; break; }
      mx = fmaxf(mx, *xch_other);
      __syncwarp();
      if (lane == 0) mbar_arrive(B(kXr + g * 4 + quarter));  // read: after both halves, the slots may be rewritten
      mx = row_ok ? mx * a.scale_log2 : -INFINITY;  // the scale is positive: the max commutes with it
      // ---- the decision, after the other group's for the tile before
      if (t >= 1 && !mbar_wait(B(kDec), (uint32_t)((t - 1) & 1), s_abort, a.spin_limit)) { alive = false; break; }
      // (two copies by tile parity: this tile reads the one the tile before wrote and writes the other, so the two
      // halves of a row never race on it)
      const float ref_old = s_ref[((t & 1) ^ 1) * 128 + lane_row];
      const bool grow = mx > ref_old + kWaTau;  // also the first tile with a visible key (reference -inf)
      const float ref = grow ? mx : ref_old;
      const bool rescale = grow && ref_old > -INFINITY;
      if (half == 0) s_ref[(t & 1) * 128 + lane_row] = ref;
      __syncwarp();
      if (lane == 0) mbar_arrive(B(kDec));
      if (__any_sync(0xffffffffu, rescale)) {
        // O moves to the new reference before this tile's P V is issued; the P V of the tile before must be done
        if (!mbar_wait(B(kPvDone), (uint32_t)((t - 1) & 1), s_abort, a.spin_limit)) { alive = false; break; }
        tc_fence_after();
        const float factor = rescale ? fast_exp2(ref_old - ref) : 1.f;
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 32) {
          float o[32];
          tmem_ld32(tmem + lane_base + (uint32_t)(kWaOCol + half * 64 + c0), o);
          tmem_wait_ld32(o);
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] *= factor;
          tmem_st32(tmem + lane_base + (uint32_t)(kWaOCol + half * 64 + c0), o);
        }
        tmem_wait_st();
      }
      if (ref > my_ref) {  // this thread's sums move to the reference in force
        const float f = my_ref > -INFINITY ? fast_exp2(my_ref - ref) : 0.f;
        l *= f;
        lsc *= f;
        my_ref = ref;
      }
      // ---- pass 2: P = exp2(logit - reference) per 32-key block, written over the block's own columns of S
      const float nref_neg = ref > -INFINITY ? -ref : -INFINITY;  // no reference yet: every P is exp2(-inf) = 0
#pragma unroll
      for (int blk = 0; blk < 2; ++blk) {
        float x[32];
        tmem_ld32(s_slot + blk * 32, x);
        tmem_wait_ld32(x);
        if (edge) {
#pragma unroll
          for (int c = 0; c < 32; ++c) x[c] = (jb + blk * 32 + c <= pos) ? x[c] : -INFINITY;
        }
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          x[c] = fast_exp2(fmaf(x[c], a.scale_log2, nref_neg));
          x[c + 1] = fast_exp2(fmaf(x[c + 1], a.scale_log2, nref_neg));
          x[c + 2] = fast_exp2(fmaf(x[c + 2], a.scale_log2, nref_neg));
          x[c + 3] = fast_exp2(fmaf(x[c + 3], a.scale_log2, nref_neg));
          s0 += x[c];
          s1 += x[c + 1];
          s2 += x[c + 2];
          s3 += x[c + 3];
        }
        const float sum = (s0 + s1) + (s2 + s3);
        float ssc = sum;
        if (edge) {  // a branch of its own (the condition is uniform), so that ordinary tiles do not carry this code
          ssc = 0.f;
#pragma unroll
          for (int c = 0; c < 32; ++c) ssc += (jb + blk * 32 + c < n_sc) ? x[c] : 0.f;
        }
        l += sum;
        lsc += ssc;
        uint32_t ph[16], pl[16];  // the block's probabilities as bf16 hi + lo pairs
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          // hi = the upper 16 bits (a byte permute, no conversion; p - hi is exact in fp32), lo = p - hi rounded to bf16:
          // hi + lo carries 16 significant bits of p
          const uint32_t b0 = __float_as_uint(x[c]), b1 = __float_as_uint(x[c + 1]);
          ph[c / 2] = __byte_perm(b0, b1, 0x7632);
          pl[c / 2] = pack_bf16(x[c] - __uint_as_float(b0 & 0xffff0000u), x[c + 1] - __uint_as_float(b1 & 0xffff0000u));
        }
        tmem_st16u(s_slot + blk * 32, ph);
        tmem_st16u(s_slot + blk * 32 + 16, pl);
      }
      tmem_wait_st();
      tc_fence_before();  // P (and a rescaled O) before the MMAs that read them
      __syncwarp();
      if (lane == 0) mbar_arrive(B(kPReady + g));  // the MMA warp may issue this tile's P V
    }
    // ---- the CTA's partial result: this thread's row, 32 of the 128 d, and its sums relative to the final reference
    if (alive && mbar_wait(B(kDec), (uint32_t)((n_tiles - 1) & 1), s_abort, a.spin_limit) &&
        mbar_wait(B(kDoneO), 0u, s_abort, a.spin_limit)) {
      tc_fence_after();
      const int sub = g * 2 + half;
      const float ref_end = s_ref[((n_tiles - 1) & 1) * 128 + lane_row];
      const float f = (my_ref > -INFINITY && ref_end > my_ref) ? fast_exp2(my_ref - ref_end) : 1.f;
      float o[32];
      tmem_ld32(tmem + lane_base + (uint32_t)(kWaOCol + sub * 32), o);
      tmem_wait_ld32(o);
      const size_t cta = ((size_t)blockIdx.y * gridDim.z + mt) * a.n_chunks + blockIdx.x;
      float* dst = a.part + (cta * 128 + lane_row) * 128 + sub * 32;
#pragma unroll
      for (int c = 0; c < 32; c += 4) *reinterpret_cast<float4*>(dst + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
      float* ds = a.part_s + cta * (kWaStateWords * 128);
      if (sub == 0) ds[lane_row] = ref_end;
      ds[(1 + sub) * 128 + lane_row] = l * f;
      ds[(1 + kWaSub + sub) * 128 + lane_row] = lsc * f;
    }
  }

  // ---- release tensor memory (after an abort: first give copies that may still be in flight time to land)
  if (*s_abort)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == kWaEpiWarps) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kWaTmemCols) : "memory");
  if (*s_abort && tid == 0) raise_status(a.status, CATEKV_STATUS_WAIT_EXPIRED, kKidScore, (int)blockIdx.y, (int)blockIdx.x);
}

// Merge the partial results of a (sequence, KV head)'s key ranges in range order: out = sum_c 2^(ref_c - M) O_c /
// sum_c 2^(ref_c - M) l_c with M the largest reference; the same weights give the two log-sum-exps.  One warp per
// query row; a lane owns four d.
__global__ void __launch_bounds__(128) window_reduce_kernel(const float* part, const float* part_s, const ScoreJob* jobs,
                                                            int keys_per_cta, int n_chunks, int MT, int R, int G, int L_obs, int Hq,
                                                            void* out, int out_fp32, float* lse_out, float* lse_scored_out) {
  const int seg = blockIdx.y;
  const int r = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= R) return;
  const ScoreJob job = jobs[seg];
  const int used = (job.n + keys_per_cta - 1) / keys_per_cta;
  const int mt = r >> 7, row = r & 127;
  const size_t cta0 = ((size_t)seg * MT + mt) * n_chunks;
  const float* ps = part_s + cta0 * (kWaStateWords * 128) + row;
  constexpr size_t kStep = (size_t)kWaStateWords * 128;  // words from one range's state to the next
  float M = -INFINITY;
  for (int c = 0; c < used; ++c) M = fmaxf(M, ps[c * kStep]);
  const float* p = part + (cta0 * 128 + row) * 128 + lane * 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float L = 0.f, Lsc = 0.f;
  for (int c = 0; c < used; ++c) {
    const float ref = ps[c * kStep];
    if (ref == -INFINITY) continue;  // the row saw none of this range's keys
    const float w = exp2f(ref - M);
    const float4 v = *reinterpret_cast<const float4*>(p + (size_t)c * 128 * 128);
    acc.x += w * v.x;
    acc.y += w * v.y;
    acc.z += w * v.z;
    acc.w += w * v.w;
    float lc = 0.f, lscc = 0.f;
#pragma unroll
    for (int k = 0; k < kWaSub; ++k) {
      lc += ps[c * kStep + (1 + k) * 128];
      lscc += ps[c * kStep + (1 + kWaSub + k) * 128];
    }
    L += w * lc;
    Lsc += w * lscc;
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
  acc.x *= inv;
  acc.y *= inv;
  acc.z *= inv;
  acc.w *= inv;
  const int i = r / G, g = r - i * G;
  const size_t orow = ((size_t)job.b * Hq + job.h * G + g) * L_obs + i;
  const size_t o = orow * kD + lane * 4;
  if (out_fp32) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + o) = acc;
  } else {
    uint2 pk;
    pk.x = pack_bf16(acc.x, acc.y);
    pk.y = pack_bf16(acc.z, acc.w);
    *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(out) + o) = pk;
  }
  if (lane == 0) {
    const float ln2 = 0.6931471805599453f;
    if (lse_out) lse_out[orow] = L > 0.f ? (M + log2f(L)) * ln2 : -INFINITY;
    if (lse_scored_out) lse_scored_out[orow] = Lsc > 0.f ? (M + log2f(Lsc)) * ln2 : -INFINITY;
  }
}


struct WaWs {
  size_t off_status, off_jobs, off_part, off_part_s, bytes;
  int keys_per_cta, n_chunks, MT;
};
static WaWs wa_ws_layout(int n_segs, int G, int n_max, int L_obs) {
  WaWs w;
  const int R = G * L_obs;
  w.MT = (R + 127) / 128;
  // key ranges: at most one CTA per SM over all (segment, M tile) pairs (the kernel runs one CTA per SM: a grid
  // just above the SM count would take two waves), in whole tiles, at least four tiles each
  int chunks = sm_count() / (n_segs * w.MT);
  if (chunks < 1) chunks = 1;
  int kp = ((n_max + chunks - 1) / chunks + kKeyTile - 1) / kKeyTile * kKeyTile;
  if (kp < 4 * kKeyTile) kp = 4 * kKeyTile;
  w.keys_per_cta = kp;
  w.n_chunks = (n_max + kp - 1) / kp;
  const size_t ctas = (size_t)n_segs * w.MT * w.n_chunks;
  size_t o = 0;
  w.off_status = o; o = CATEKV_STATUS_BYTES;
  w.off_jobs = o; o = align_up(o + sizeof(ScoreJob) * (size_t)n_segs, 256);
  w.off_part = o; o = align_up(o + sizeof(float) * ctas * 128 * 128, 256);
  w.off_part_s = o; o = align_up(o + sizeof(float) * ctas * kWaStateWords * 128, 256);
  w.bytes = o;
  return w;
}

}  // namespace catekv

using namespace catekv;

extern "C" size_t catekv_window_attn_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t n_max, int32_t L_obs) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || n_max <= 0 || L_obs <= 0 || Hq % Hkv) return 0;
  return wa_ws_layout(B * Hkv, Hq / Hkv, n_max, L_obs).bytes;
}

extern "C" int catekv_window_attn(const void* q_win, const void* k, const void* v, int64_t kv_stride_b, int64_t kv_stride_h,
                                  int64_t kv_stride_t, const int32_t* seq_len, int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                                  int32_t L_obs, void* out, int32_t out_dtype, float* lse_out, float* lse_scored_out, void* ws,
                                  size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  if (!q_win || !k || !v || !seq_len || !out || !ws) return CATEKV_ERR_INVALID_ARG;
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || L_obs < 1) return CATEKV_ERR_INVALID_ARG;
  if (d != kD) return CATEKV_ERR_UNSUPPORTED;
  const int G = Hq / Hkv;
  if (G > kMaxG || G * L_obs > kScoreMaxRows) return CATEKV_ERR_UNSUPPORTED;
  if (out_dtype != CATEKV_OUT_BF16 && out_dtype != CATEKV_OUT_FP32) return CATEKV_ERR_UNSUPPORTED;
  const int n_segs = B * Hkv;
  int n_max = 0;
  for (int b = 0; b < B; ++b) {
    if (seq_len[b] < L_obs) return CATEKV_ERR_INVALID_ARG;  // the window rows are the last L_obs tokens
    n_max = seq_len[b] > n_max ? seq_len[b] : n_max;
  }
  const WaWs W = wa_ws_layout(n_segs, G, n_max, L_obs);
  if (ws_bytes < W.bytes) return CATEKV_ERR_WORKSPACE;

  std::vector<ScoreJob> jobs(n_segs);
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < Hkv; ++h) jobs[b * Hkv + h] = ScoreJob{b, h, seq_len[b], 0, seq_len[b], 0};
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w8 = (uint8_t*)ws;
  {
    // one copy brings the cleared status block and the job list (they are adjacent in the workspace)
    std::vector<uint8_t> head(W.off_jobs + sizeof(ScoreJob) * jobs.size(), 0);
    memcpy(head.data() + W.off_jobs, jobs.data(), sizeof(ScoreJob) * jobs.size());
    CATEKV_CUDA_TRY(cudaMemcpyAsync(w8, head.data(), head.size(), cudaMemcpyHostToDevice, st));
  }
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)kD);
  const int R = G * L_obs;
  int rc;

  CUtensorMap k_map, v_map;
  const KvTensor kt = {(const uint16_t*)k, kv_stride_b, kv_stride_h, kv_stride_t, B, Hkv, n_max};
  const KvTensor vt = {(const uint16_t*)v, kv_stride_b, kv_stride_h, kv_stride_t, B, Hkv, n_max};
  rc = make_kv_map(kt, &k_map);
  if (rc) return rc;
  rc = make_kv_map(vt, &v_map);
  if (rc) return rc;
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  CATEKV_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
    CATEKV_CUDA_TRY(cudaFuncSetAttribute(window_pv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWaSmemBytes));
    if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
  }
  WinArgs wa = {};
  wa.q_win = (const uint16_t*)q_win;
  wa.jobs = (const ScoreJob*)(w8 + W.off_jobs);
  wa.G = G;
  wa.L_obs = L_obs;
  wa.R = R;
  wa.Hq = Hq;
  wa.scale_log2 = scale_log2;
  wa.keys_per_cta = W.keys_per_cta;
  wa.n_chunks = W.n_chunks;
  wa.part = (float*)(w8 + W.off_part);
  wa.part_s = (float*)(w8 + W.off_part_s);
  wa.status = (int32_t*)(w8 + W.off_status);
  wa.spin_limit = kSpinLimit;
  if (score_take_expire_launch()) {
    wa.spin_limit = 512;
    wa.idle_producer = 1;
  }
  window_pv_kernel<<<dim3(W.n_chunks, n_segs, W.MT), kWaThreads, kWaSmemBytes, st>>>(k_map, v_map, wa);
  CATEKV_CUDA_TRY(cudaGetLastError());
  window_reduce_kernel<<<dim3((R + 3) / 4, n_segs), 128, 0, st>>>(wa.part, wa.part_s, wa.jobs, W.keys_per_cta, W.n_chunks, W.MT, R,
                                                                  G, L_obs, Hq, out, out_dtype == CATEKV_OUT_FP32, lse_out,
                                                                  lse_scored_out);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}
