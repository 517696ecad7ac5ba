// Attention of the observation window (Algorithm 1, pre-filling stage): the causal attention rows of the last L_obs
// prefill queries of every query head - what a prefill attention pass produces for those positions - together with
// their log-sum-exp and the log-sum-exp over the scored keys [0, n - L_obs) alone, which is the softmax normaliser
// of the token-criticality line.  catekv_select_compact takes the latter in place of its own first pass over K.
//
//   1. row statistics (score_tc_kernel, statistics mode): two jobs per (sequence, KV head), the scored keys
//      [0, n - L_obs) and the window's own keys [n - L_obs, n) under the causal mask;
//   2. window_stats_kernel merges the two into the causal normaliser of every row and writes both log-sum-exps;
//   3. window_pv_kernel: O[rows x d] = sum over key tiles of P V with P = exp2(logit - normaliser) already final,
//      so the accumulator in tensor memory is never rescaled.  Per key tile: S = Q K^T (tcgen05.mma, accumulator
//      slot in TMEM), the epilogue warps turn S into P and write it to shared memory as a bf16 hi + lo pair in the
//      K-major SWIZZLE_128B operand layout, and two more chains of tcgen05.mma add P_hi V and P_lo V (V as the
//      MN-major B operand, straight from the TMA tile) to O in TMEM.  A CTA owns a range of keys of one
//      (sequence, KV head) and 128 query rows; the ranges' partial outputs are summed in a fixed order by
//   4. window_reduce_kernel, which also converts to the output type.
//
// Warp roles of window_pv_kernel: warp 9 (one lane) feeds the K and V stages by TMA; warp 8 (one lane) issues
// every MMA, the S of tile t + 1 before the P V of tile t; warps 0-7 are the epilogue (two per TMEM lane quarter,
// 64 keys each).  Every mbarrier wait is bounded: on expiry the CTA raises the abort flag, frees its tensor memory,
// records CATEKV_STATUS_WAIT_EXPIRED and returns.
#include <math.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "score.cuh"
#include "tc.cuh"

namespace catekv {

constexpr int kWaThreads = 320;
constexpr int kWaTmemCols = 512;       // S slots at columns 0 and 128, O at 256
constexpr int kWaOCol = 256;
constexpr int kWaTileBytes = 128 * 256;  // a [128 x 128] bf16 tile: Q rows, a K or V stage, P hi, P lo

struct WinArgs {
  const uint16_t* q_win;  // [B, Hq, L_obs, d]
  const ScoreJob* jobs;   // [n_segs]: b, h, n (j_begin / j_end unused)
  const float* mfull;     // [n_segs][kScoreMaxRows]: log2-domain causal normaliser of every row; +inf: the row has no mass
  int32_t G, L_obs, R, Hq;
  float scale_log2;
  int32_t keys_per_cta, n_chunks;
  float* part;            // [n_segs][MT][n_chunks][128 rows][128 d]
  int32_t* status;
  uint32_t spin_limit;
};

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
  const uint32_t s_q = s_base;
  const uint32_t s_k = s_q + kWaTileBytes;
  const uint32_t s_v = s_k + 2 * kWaTileBytes;
  const uint32_t s_ph = s_v + 2 * kWaTileBytes;
  const uint32_t s_pl = s_ph + kWaTileBytes;
  float* s_m = reinterpret_cast<float*>(smem + 7 * kWaTileBytes);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_m + 128);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 16);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const uint32_t bar0 = smem_u32(s_bar);
  const uint32_t bar_full_k = bar0, bar_empty_k = bar0 + 16, bar_full_v = bar0 + 32, bar_empty_v = bar0 + 48;
  const uint32_t bar_done_s = bar0 + 64, bar_free_s = bar0 + 80, bar_p_ready = bar0 + 96, bar_p_free = bar0 + 104;
  const uint32_t bar_done_o = bar0 + 112;

  // ---- set-up: this M tile's query rows (row r = i * G + g), their normalisers, barriers, tensor memory
  for (int id = tid; id < 128 * 16; id += kWaThreads) {
    const int row = id >> 4, c = id & 15;
    const int r = mt * 128 + row;
    const int ok = r < a.R ? 16 : 0;
    const int i = ok ? r / a.G : 0, g = ok ? r - i * a.G : 0;
    const uint16_t* src = a.q_win + (((int64_t)job.b * a.Hq + job.h * a.G + g) * a.L_obs + i) * kD + c * 8;
    cp_async16(s_q + sw128_off(row, c, 128), src, ok);
  }
  cp_async_commit();
  for (int row = tid; row < 128; row += kWaThreads) {
    const int r = mt * 128 + row;
    s_m[row] = r < a.R ? a.mfull[(size_t)blockIdx.y * kScoreMaxRows + r] : INFINITY;
  }
  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < 15; ++i) {
      const uint32_t bar = bar0 + 8 * i;
      const int count = (bar == bar_free_s || bar == bar_free_s + 8 || bar == bar_p_ready) ? 8 : 1;  // one arrival per epilogue warp
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
    }
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(s_tmem)), "r"(kWaTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  cp_async_wait<0>();
  fence_async_smem();  // Q was written through the generic proxy; the MMAs read it through the async proxy
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  if (warp == 9) {
    // ================= TMA producer =================
    if (lane == 0) {
      for (int tile = 0; tile < n_tiles; ++tile) {
        const int st = tile & 1;
        const uint32_t par = (uint32_t)(((tile >> 1) - 1) & 1);
        const int j0 = j_lo + tile * kKeyTile;
        if (tile >= 2 && !mbar_wait(bar_empty_k + 8 * st, par, s_abort, a.spin_limit)) break;
        mbar_expect_tx(bar_full_k + 8 * st, kWaTileBytes);
        tma_load_box(s_k + st * kWaTileBytes, &k_map, 0, j0, job.h, job.b, bar_full_k + 8 * st);
        tma_load_box(s_k + st * kWaTileBytes + kKBlockBytes, &k_map, 64, j0, job.h, job.b, bar_full_k + 8 * st);
        if (tile >= 2 && !mbar_wait(bar_empty_v + 8 * st, par, s_abort, a.spin_limit)) break;
        mbar_expect_tx(bar_full_v + 8 * st, kWaTileBytes);
        tma_load_box(s_v + st * kWaTileBytes, &v_map, 0, j0, job.h, job.b, bar_full_v + 8 * st);
        tma_load_box(s_v + st * kWaTileBytes + kKBlockBytes, &v_map, 64, j0, job.h, job.b, bar_full_v + 8 * st);
      }
    }
    __syncwarp();
  } else if (warp == 8) {
    // ================= MMA issue =================
    if (lane == 0) {
      const uint32_t idesc_s = umma_idesc_bf16(128, 128);      // S[rows x keys]: A = Q, B = K, both K-major
      const uint32_t idesc_o = umma_idesc_bf16_bmn(128, 128);  // O[rows x d]: A = P (K-major), B = V (MN-major)
      auto issue_s = [&](int t) -> bool {
        const int st = t & 1;
        if (!mbar_wait(bar_full_k + 8 * st, (uint32_t)((t >> 1) & 1), s_abort, a.spin_limit)) return false;
        if (t >= 2 && !mbar_wait(bar_free_s + 8 * st, (uint32_t)(((t >> 1) - 1) & 1), s_abort, a.spin_limit)) return false;
        tc_fence_after();
        const uint32_t sk = s_k + st * kWaTileBytes;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (kk >> 2) * kKBlockBytes + (kk & 3) * 32;
          umma_bf16(tmem + (uint32_t)(st * 128), umma_desc_sw128(s_q + off), umma_desc_sw128(sk + off), idesc_s, kk ? 1u : 0u);
        }
        umma_commit(bar_done_s + 8 * st);
        umma_commit(bar_empty_k + 8 * st);
        return true;
      };
      bool ok = issue_s(0);
      for (int t = 0; ok && t < n_tiles; ++t) {
        if (t + 1 < n_tiles && !issue_s(t + 1)) break;
        const int st = t & 1;
        if (!mbar_wait(bar_p_ready, (uint32_t)(t & 1), s_abort, a.spin_limit)) break;
        if (!mbar_wait(bar_full_v + 8 * st, (uint32_t)((t >> 1) & 1), s_abort, a.spin_limit)) break;
        tc_fence_after();
        const uint32_t sv = s_v + st * kWaTileBytes;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          const uint32_t sp = part ? s_pl : s_ph;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {  // 16 keys per step
            const uint32_t aoff = (kk >> 2) * kKBlockBytes + (kk & 3) * 32;
            umma_bf16(tmem + kWaOCol, umma_desc_sw128(sp + aoff), umma_desc_sw128_mn(sv + kk * 2048, kKBlockBytes), idesc_o,
                      (t | part | kk) ? 1u : 0u);
          }
        }
        umma_commit(bar_p_free);
        umma_commit(bar_empty_v + 8 * st);
        if (t == n_tiles - 1) umma_commit(bar_done_o);
      }
    }
    __syncwarp();
  } else {
    // ================= epilogue warps =================
    const int lane_row = (warp & 3) * 32 + lane;  // this thread's TMEM lane = its query row of the M tile
    const int half = warp >> 2;                   // keys [64 * half, 64 * half + 64) of every tile
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const int r = mt * 128 + lane_row;
    const int pos = n - a.L_obs + (r < a.R ? r / a.G : 0);  // the row's own position: it sees keys j <= pos
    const float mr = s_m[lane_row];
    bool alive = true;
    for (int t = 0; t < n_tiles; ++t) {
      const int st = t & 1;
      if (!mbar_wait(bar_done_s + 8 * st, (uint32_t)((t >> 1) & 1), s_abort, a.spin_limit)) { alive = false; break; }
      tc_fence_after();
      float x[64];
      tmem_ld64(tmem + lane_base + (uint32_t)(st * 128 + half * 64), x);
      tmem_wait_ld64(x);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_free_s + 8 * st);  // the S slot goes back to the MMA warp
      const int jb = j_lo + t * kKeyTile + half * 64;   // key of x[0]
      const bool edge = jb + 63 > n - a.L_obs;          // uniform: some key of the block may be masked for some row
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        float p = fast_exp2(fmaf(x[c], a.scale_log2, -mr));
        if (edge) p = (jb + c <= pos) ? p : 0.f;
        x[c] = p;
      }
      // P of the previous tile must have been consumed before this one overwrites it
      if (t >= 1 && !mbar_wait(bar_p_free, (uint32_t)((t - 1) & 1), s_abort, a.spin_limit)) { alive = false; break; }
#pragma unroll
      for (int c = 0; c < 64; c += 8) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float h0 = bf16_round(x[c + 2 * e]), h1 = bf16_round(x[c + 2 * e + 1]);
          hi[e] = pack_bf16(h0, h1);
          lo[e] = pack_bf16(x[c + 2 * e] - h0, x[c + 2 * e + 1] - h1);
        }
        const uint32_t off = sw128_off(lane_row, half * 8 + (c >> 3), 128);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};\n" ::"r"(s_ph + off), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};\n" ::"r"(s_pl + off), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
      }
      fence_async_smem();  // generic-proxy writes of P before the async-proxy reads of the MMAs
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p_ready);
    }
    // ---- the CTA's partial output: this thread's row, 64 of the 128 d
    if (alive && mbar_wait(bar_done_o, 0u, s_abort, a.spin_limit)) {
      tc_fence_after();
      float o[64];
      tmem_ld64(tmem + lane_base + (uint32_t)(kWaOCol + half * 64), o);
      tmem_wait_ld64(o);
      float* dst = a.part + ((((size_t)blockIdx.y * gridDim.z + mt) * a.n_chunks + blockIdx.x) * 128 + lane_row) * 128 + half * 64;
#pragma unroll
      for (int c = 0; c < 64; c += 4) *reinterpret_cast<float4*>(dst + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
    }
  }

  // ---- release tensor memory (after an abort: first give copies that may still be in flight time to land)
  if (*s_abort)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kWaTmemCols) : "memory");
  if (*s_abort && tid == 0) raise_status(a.status, CATEKV_STATUS_WAIT_EXPIRED, kKidScore, (int)blockIdx.y, (int)blockIdx.x);
}

// Merge the statistics of the scored keys (job s) and of the window's own keys (job n_segs + s) of every row.
__global__ void window_stats_kernel(const float2* stats, const ScoreJob* jobs, int R, int G, int L_obs, int Hq, float* mfull,
                                    float* lse_out, float* lse_scored_out) {
  const int seg = blockIdx.x;
  const ScoreJob job = jobs[seg];
  const float ln2 = 0.6931471805599453f;
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const float2 sa = stats[(size_t)seg * kScoreMaxRows + r], sb = stats[(size_t)(gridDim.x + seg) * kScoreMaxRows + r];
    const float m = fmaxf(sa.x, sb.x);
    float l = 0.f;
    if (sa.y > 0.f) l += sa.y * exp2f(sa.x - m);
    if (sb.y > 0.f) l += sb.y * exp2f(sb.x - m);
    const float full = l > 0.f ? m + log2f(l) : INFINITY;
    mfull[(size_t)seg * kScoreMaxRows + r] = full;
    const int i = r / G, g = r - i * G;
    const size_t o = ((size_t)job.b * Hq + job.h * G + g) * L_obs + i;
    if (lse_out) lse_out[o] = l > 0.f ? full * ln2 : -INFINITY;
    if (lse_scored_out) lse_scored_out[o] = sa.y > 0.f ? (sa.x + log2f(sa.y)) * ln2 : -INFINITY;
  }
}

// Sum the partial outputs of a (sequence, KV head)'s key ranges in range order; one warp per query row.
__global__ void __launch_bounds__(128) window_reduce_kernel(const float* part, const ScoreJob* jobs, int keys_per_cta, int n_chunks,
                                                            int MT, int R, int G, int L_obs, int Hq, void* out, int out_fp32) {
  const int seg = blockIdx.y;
  const int r = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= R) return;
  const ScoreJob job = jobs[seg];
  const int used = (job.n + keys_per_cta - 1) / keys_per_cta;
  const int mt = r >> 7, row = r & 127;
  const float* p = part + ((((size_t)seg * MT + mt) * n_chunks) * 128 + row) * 128 + lane * 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c = 0; c < used; ++c) {
    const float4 v = *reinterpret_cast<const float4*>(p + (size_t)c * 128 * 128);
    acc.x += v.x;
    acc.y += v.y;
    acc.z += v.z;
    acc.w += v.w;
  }
  const int i = r / G, g = r - i * G;
  const size_t o = (((size_t)job.b * Hq + job.h * G + g) * L_obs + i) * kD + lane * 4;
  if (out_fp32) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + o) = acc;
  } else {
    uint2 pk;
    pk.x = pack_bf16(acc.x, acc.y);
    pk.y = pack_bf16(acc.z, acc.w);
    *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(out) + o) = pk;
  }
}

constexpr size_t kWaSmemBytes = 1024 + 7 * (size_t)kWaTileBytes + 128 * sizeof(float) + 16 * sizeof(uint64_t) + 16;

struct WaWs {
  size_t off_status, off_jobs2, off_jobs, off_part_stats, off_stats, off_mfull, off_part, bytes;
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
  size_t o = 0;
  w.off_status = o; o = CATEKV_STATUS_BYTES;
  w.off_jobs2 = o; o = align_up(o + sizeof(ScoreJob) * (size_t)(2 * n_segs), 256);
  w.off_jobs = o; o = align_up(o + sizeof(ScoreJob) * (size_t)n_segs, 256);
  w.off_part_stats = o; o = align_up(o + sizeof(float2) * (size_t)score_max_ctas(2 * n_segs) * 2 * kScoreMaxRows, 256);
  w.off_stats = o; o = align_up(o + sizeof(float2) * (size_t)(2 * n_segs) * kScoreMaxRows, 256);
  w.off_mfull = o; o = align_up(o + sizeof(float) * (size_t)n_segs * kScoreMaxRows, 256);
  w.off_part = o; o = align_up(o + sizeof(float) * (size_t)n_segs * w.MT * w.n_chunks * 128 * 128, 256);
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

  std::vector<ScoreJob> jobs2(2 * n_segs), jobs(n_segs);
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < Hkv; ++h) {
      const int s = b * Hkv + h, n = seq_len[b];
      // the scored jobs first: their CTAs fill the machine in one wave, the one-tile window jobs follow
      jobs2[s] = ScoreJob{b, h, n, 0, n - L_obs, 0};           // the scored keys
      jobs2[n_segs + s] = ScoreJob{b, h, n, n - L_obs, n, 0};  // the window's own keys (causal)
      jobs[s] = ScoreJob{b, h, n, 0, n, 0};
    }
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w8 = (uint8_t*)ws;
  {
    // one copy brings the cleared status block and both job lists (they are adjacent in the workspace)
    std::vector<uint8_t> head(W.off_jobs + sizeof(ScoreJob) * jobs.size(), 0);
    memcpy(head.data() + W.off_jobs2, jobs2.data(), sizeof(ScoreJob) * jobs2.size());
    memcpy(head.data() + W.off_jobs, jobs.data(), sizeof(ScoreJob) * jobs.size());
    CATEKV_CUDA_TRY(cudaMemcpyAsync(w8, head.data(), head.size(), cudaMemcpyHostToDevice, st));
  }
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)kD);
  ScoreArgs sa = {};
  sa.q_win = (const uint16_t*)q_win;
  sa.k = (const uint16_t*)k;
  sa.sb = kv_stride_b;
  sa.sh = kv_stride_h;
  sa.st = kv_stride_t;
  sa.jobs = (const ScoreJob*)(w8 + W.off_jobs2);
  sa.n_jobs = 2 * n_segs;
  sa.n_jobs_split = n_segs;  // the window jobs are one CTA each: the key ranges are cut for the scored jobs alone
  sa.Hq = Hq;
  sa.B = B;
  sa.Hkv = Hkv;
  sa.n_max = n_max;
  sa.G = G;
  sa.L_obs = L_obs;
  sa.causal = 1;
  sa.scale_log2 = scale_log2;
  sa.max_keys = n_max > L_obs ? n_max - L_obs : L_obs;
  if (sa.max_keys < L_obs) sa.max_keys = L_obs;
  sa.stats_part = (float2*)(w8 + W.off_part_stats);
  sa.stats = (float2*)(w8 + W.off_stats);
  sa.status = (int32_t*)(w8 + W.off_status);
  int rc = score_launch(sa, kScoreStats, st);
  if (rc) return rc;
  const int R = G * L_obs;
  float* mfull = (float*)(w8 + W.off_mfull);
  window_stats_kernel<<<n_segs, 128, 0, st>>>(sa.stats, (const ScoreJob*)(w8 + W.off_jobs), R, G, L_obs, Hq, mfull, lse_out,
                                              lse_scored_out);
  CATEKV_CUDA_TRY(cudaGetLastError());

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
  wa.mfull = mfull;
  wa.G = G;
  wa.L_obs = L_obs;
  wa.R = R;
  wa.Hq = Hq;
  wa.scale_log2 = scale_log2;
  wa.keys_per_cta = W.keys_per_cta;
  wa.n_chunks = W.n_chunks;
  wa.part = (float*)(w8 + W.off_part);
  wa.status = (int32_t*)(w8 + W.off_status);
  wa.spin_limit = kSpinLimit;
  window_pv_kernel<<<dim3(W.n_chunks, n_segs, W.MT), kWaThreads, kWaSmemBytes, st>>>(k_map, v_map, wa);
  CATEKV_CUDA_TRY(cudaGetLastError());
  window_reduce_kernel<<<dim3((R + 3) / 4, n_segs), 128, 0, st>>>(wa.part, wa.jobs, W.keys_per_cta, W.n_chunks, W.MT, R, G, L_obs,
                                                                  Hq, out, out_dtype == CATEKV_OUT_FP32);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}
