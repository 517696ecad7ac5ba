// Observation-window scoring kernels (first version: mma.sync tensor-core tiles).
//
// A CTA scores `keys_per_cta` keys of one (sequence, KV head) against the L_obs window queries
// of all G query heads of the group.  The queries (G * L_obs rows) sit in swizzled shared
// memory for the CTA's lifetime; 64-key tiles of K stream through a two-stage cp.async
// pipeline.  Warp w owns one 16-row slice of the window (i-tile) and a group of key columns of
// the tile, and loops over the G heads, so that sums over heads and over window rows stay in
// registers.  Two passes over K: row max / row sum (online, merged over CTAs by a small
// kernel), then exp(s - max) / sum reduced to column sums (selection) or to the group-mean
// matrix (head identification).
#include <math.h>

#include "score.cuh"

namespace catekv {

constexpr int kScoreThreads = 256;
constexpr int kScoreWarps = 8;
constexpr int kKeyTile = 64;

int score_rows_pad(int G, int L_obs) { return G * (L_obs <= 32 ? 32 : 64); }
int score_key_groups(int L_obs) { return kScoreWarps / (L_obs <= 32 ? 2 : 4); }

template <int MODE, int N_IT>
__global__ void __launch_bounds__(kScoreThreads) score_kernel(const ScoreArgs a) {
  constexpr int ROWS_IT = N_IT * 16;          // padded window rows per head
  constexpr int KG = kScoreWarps / N_IT;      // key groups per tile
  constexpr int NP = 4 / KG;                  // 16-key pairs per warp per tile (N_IT=2 -> 1, N_IT=4 -> 2)
  extern __shared__ __align__(128) uint8_t smem[];
  const ScoreJob job = a.jobs[blockIdx.y];
  const int j_lo = job.j_begin + blockIdx.x * a.keys_per_cta;
  if (j_lo >= job.j_end) return;
  const int j_hi = min(job.j_end, j_lo + a.keys_per_cta);
  const int n_tiles = (j_hi - j_lo + kKeyTile - 1) / kKeyTile;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int it = warp % N_IT, kg = warp / N_IT;
  const int rows_pad = a.G * ROWS_IT;

  const uint32_t s_q = smem_u32(smem);
  const uint32_t s_k = s_q + rows_pad * kRowBytes;
  float2* s_stats = reinterpret_cast<float2*>(smem + rows_pad * kRowBytes + 2 * kKeyTile * kRowBytes);
  float* s_col = reinterpret_cast<float*>(s_stats + rows_pad);  // [N_IT][64] per-i-tile column sums of the tile

  // ---- stage the group's window queries (rows >= L_obs zero) and, for pass 2, the row stats
  for (int id = tid; id < rows_pad * 16; id += kScoreThreads) {
    const int r = id >> 4, c = id & 15;
    const int gh = r / ROWS_IT, i = r % ROWS_IT;
    const int ok = i < a.L_obs ? 16 : 0;
    const uint16_t* src = a.q_win + (((int64_t)job.b * a.Hq + job.h * a.G + gh) * a.L_obs + (ok ? i : 0)) * kD + c * 8;
    cp_async16(s_q + tile_off(r, c), src, ok);
  }
  if (MODE != kScoreStats) {
    const float2* st = a.stats + (size_t)blockIdx.y * rows_pad;
    for (int r = tid; r < rows_pad; r += kScoreThreads) s_stats[r] = st[r];
  }
  const uint16_t* kbase = a.k + (int64_t)job.b * a.sb + (int64_t)job.h * a.sh;
  auto issue = [&](int tile) {
    if (tile < n_tiles) {
      const uint32_t sb = s_k + (tile & 1) * (kKeyTile * kRowBytes);
      const int j0 = j_lo + tile * kKeyTile;
#pragma unroll
      for (int i = 0; i < (kKeyTile * 16) / kScoreThreads; ++i) {
        const int id = tid + i * kScoreThreads;
        const int r = id >> 4, c = id & 15;
        const int ok = (j0 + r) < j_hi ? 16 : 0;
        cp_async16(sb + tile_off(r, c), kbase + (int64_t)(ok ? j0 + r : job.j_begin) * a.st + c * 8, ok);
      }
    }
    cp_async_commit();
  };
  issue(0);

  // pass-1 state: running max / sum of the rows (it*16 + g) and (+8) of every head
  float rm[kMaxG][2], rl[kMaxG][2];
#pragma unroll
  for (int gh = 0; gh < kMaxG; ++gh) rm[gh][0] = rm[gh][1] = -INFINITY, rl[gh][0] = rl[gh][1] = 0.f;
  const int row_lo = it * 16 + g, row_hi = row_lo + 8;  // window rows of this thread
  const float inv_g = 1.f / (float)a.G;
  // causal: window row i sits at position n - L_obs + i and sees keys j <= that position
  const int lim_lo = a.causal ? job.n - a.L_obs + row_lo : 0x7fffffff;
  const int lim_hi = a.causal ? job.n - a.L_obs + row_hi : 0x7fffffff;

  for (int tile = 0; tile < n_tiles; ++tile) {
    cp_async_wait<0>();
    __syncthreads();
    issue(tile + 1);
    const uint32_t kb = s_k + (tile & 1) * (kKeyTile * kRowBytes);
    const int j0 = j_lo + tile * kKeyTile;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int key0 = (kg * NP + p) * 16;  // first key of the pair inside the tile
      if (j0 + key0 >= j_hi) continue;      // warp-uniform: padding columns
      uint32_t bf[8][4];
      {
        const int r = key0 + (lane & 7) + ((lane >> 4) & 1) * 8;
        const int cadd = (lane >> 3) & 1;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) ldmatrix_x4(bf[ks], kb + tile_off(r, ks * 2 + cadd));
      }
      // keys held by this thread: n-tile 0 -> key0 + 2t, +1 ; n-tile 1 -> key0 + 8 + 2t, +1
      const int jA = j0 + key0 + 2 * t, jB = jA + 8;
      float acc[2][4];  // pass 2: sum over heads of the probabilities, C-fragment layout per n-tile
#pragma unroll
      for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
#pragma unroll
      for (int gh = 0; gh < kMaxG; ++gh) {
        if (gh >= a.G) break;
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
          const int r = gh * ROWS_IT + it * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int cadd = lane >> 4;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t af[4];
            ldmatrix_x4(af, s_q + tile_off(r, ks * 2 + cadd));
            mma_bf16_16816(s0, af, bf[ks][0], bf[ks][1]);
            mma_bf16_16816(s1, af, bf[ks][2], bf[ks][3]);
          }
        }
        // logits in the log2 domain; masked entries are -inf
        float x[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const float* s = nt ? s1 : s0;
          const int j = nt ? jB : jA;
          x[nt][0] = (j < j_hi && j <= lim_lo) ? s[0] * a.scale_log2 : -INFINITY;
          x[nt][1] = (j + 1 < j_hi && j + 1 <= lim_lo) ? s[1] * a.scale_log2 : -INFINITY;
          x[nt][2] = (j < j_hi && j <= lim_hi) ? s[2] * a.scale_log2 : -INFINITY;
          x[nt][3] = (j + 1 < j_hi && j + 1 <= lim_hi) ? s[3] * a.scale_log2 : -INFINITY;
        }
        if (MODE == kScoreStats) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {  // row_lo, row_hi
            const float e0 = x[0][2 * half], e1 = x[0][2 * half + 1], e2 = x[1][2 * half], e3 = x[1][2 * half + 1];
            const float mx = fmaxf(fmaxf(e0, e1), fmaxf(e2, e3));
            if (mx > rm[gh][half]) {  // the running max rises only a few times per row
              rl[gh][half] *= fast_exp2(rm[gh][half] - mx);
              rm[gh][half] = mx;
            }
            if (rm[gh][half] > -INFINITY) {
              const float m = rm[gh][half];
              rl[gh][half] += fast_exp2(e0 - m) + fast_exp2(e1 - m) + fast_exp2(e2 - m) + fast_exp2(e3 - m);
            }
          }
        } else {
          const float2 st_lo = s_stats[gh * ROWS_IT + row_lo], st_hi = s_stats[gh * ROWS_IT + row_hi];
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            acc[nt][0] += fast_exp2(x[nt][0] - st_lo.x) * st_lo.y;
            acc[nt][1] += fast_exp2(x[nt][1] - st_lo.x) * st_lo.y;
            acc[nt][2] += fast_exp2(x[nt][2] - st_hi.x) * st_hi.y;
            acc[nt][3] += fast_exp2(x[nt][3] - st_hi.x) * st_hi.y;
          }
        }
      }
      if (MODE == kScoreColsum) {
        // sum over this warp's 16 window rows, then over warps through shared memory
        float c0 = acc[0][0] + acc[0][2], c1 = acc[0][1] + acc[0][3];
        float c2 = acc[1][0] + acc[1][2], c3 = acc[1][1] + acc[1][3];
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
          c0 += __shfl_xor_sync(0xffffffffu, c0, sh);
          c1 += __shfl_xor_sync(0xffffffffu, c1, sh);
          c2 += __shfl_xor_sync(0xffffffffu, c2, sh);
          c3 += __shfl_xor_sync(0xffffffffu, c3, sh);
        }
        if (g == 0) {  // each (i-tile, key) has one writer: the sum over i-tiles below runs in a fixed order
          float* sc = s_col + it * kKeyTile + key0;
          sc[2 * t] = c0;
          sc[2 * t + 1] = c1;
          sc[8 + 2 * t] = c2;
          sc[8 + 2 * t + 1] = c3;
        }
      } else if (MODE == kScoreMatrix) {
        float* A = a.out + (size_t)blockIdx.y * a.out_job_stride;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int j = nt ? jB : jA;
          if (row_lo < a.L_obs) {
            if (j < j_hi) A[(size_t)row_lo * a.out_row_stride + (j - job.j_begin)] = acc[nt][0] * inv_g;
            if (j + 1 < j_hi) A[(size_t)row_lo * a.out_row_stride + (j + 1 - job.j_begin)] = acc[nt][1] * inv_g;
          }
          if (row_hi < a.L_obs) {
            if (j < j_hi) A[(size_t)row_hi * a.out_row_stride + (j - job.j_begin)] = acc[nt][2] * inv_g;
            if (j + 1 < j_hi) A[(size_t)row_hi * a.out_row_stride + (j + 1 - job.j_begin)] = acc[nt][3] * inv_g;
          }
        }
      }
    }
    if (MODE == kScoreColsum) {
      __syncthreads();
      if (tid < kKeyTile) {
        const int j = j0 + tid;
        float c = 0.f;
#pragma unroll
        for (int i = 0; i < N_IT; ++i) c += s_col[i * kKeyTile + tid];
        if (j < j_hi) a.out[(size_t)blockIdx.y * a.out_job_stride + (j - job.j_begin)] = c * inv_g;
      }
      // the next tile's partial sums are written after the next iteration's barrier
    }
  }
  cp_async_wait<0>();

  if (MODE == kScoreStats) {
    // per-row partials of this warp: merge the four lanes of a quad, lane t == 0 writes
    float2* outp = a.stats_part + ((size_t)blockIdx.y * a.n_chunks * KG + (size_t)blockIdx.x * KG + kg) * rows_pad;
#pragma unroll
    for (int gh = 0; gh < kMaxG; ++gh) {
      if (gh >= a.G) break;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        float m = rm[gh][half], l = rl[gh][half];
#pragma unroll
        for (int sh = 1; sh <= 2; sh <<= 1) {
          const float om = __shfl_xor_sync(0xffffffffu, m, sh), ol = __shfl_xor_sync(0xffffffffu, l, sh);
          const float mn = fmaxf(m, om);
          const float sa = (m == -INFINITY) ? 0.f : fast_exp2(m - mn);
          const float sb2 = (om == -INFINITY) ? 0.f : fast_exp2(om - mn);
          l = l * sa + ol * sb2;
          m = mn;
        }
        if (t == 0) outp[gh * ROWS_IT + it * 16 + g + half * 8] = make_float2(m, l);
      }
    }
  }
}

// Merge the per-CTA row partials: stats[job][row] = (max, 1 / sum); padding rows get (0, 0).
// One warp per row: the lanes stride over the partials, then merge pairwise.
__global__ void __launch_bounds__(256) score_stats_merge_kernel(const ScoreArgs a, int rows_it, int kgroups) {
  const int jobi = blockIdx.y;
  const int rows_pad = a.G * rows_it;
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= rows_pad) return;
  const ScoreJob job = a.jobs[jobi];
  float m = -INFINITY, l = 0.f;
  if (r % rows_it < a.L_obs) {
    const int used = (job.j_end - job.j_begin + a.keys_per_cta - 1) / a.keys_per_cta;
    for (int c = lane; c < used * kgroups; c += 32) {
      const float2 p = a.stats_part[((size_t)jobi * a.n_chunks * kgroups + c) * rows_pad + r];
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
  }
  if (lane == 0) a.stats[(size_t)jobi * rows_pad + r] = (l > 0.f) ? make_float2(m, 1.f / l) : make_float2(0.f, 0.f);
}

template <int MODE, int N_IT>
static int launch_one(const ScoreArgs& a, cudaStream_t stream) {
  const int rows_pad = a.G * N_IT * 16;
  const size_t smem = (size_t)rows_pad * kRowBytes + 2 * kKeyTile * kRowBytes + rows_pad * sizeof(float2) +
                      N_IT * kKeyTile * sizeof(float);
  CATEKV_CUDA_TRY(cudaFuncSetAttribute(score_kernel<MODE, N_IT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  score_kernel<MODE, N_IT><<<dim3(a.n_chunks, a.n_jobs), kScoreThreads, smem, stream>>>(a);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}

int score_launch(const ScoreArgs& a, ScoreMode out_mode, cudaStream_t stream) {
  if (a.n_jobs <= 0 || a.n_chunks <= 0) return CATEKV_OK;
  const bool small = a.L_obs <= 32;
  int rc = small ? launch_one<kScoreStats, 2>(a, stream) : launch_one<kScoreStats, 4>(a, stream);
  if (rc) return rc;
  const int rows_it = small ? 32 : 64;
  const int rows_pad = a.G * rows_it;
  score_stats_merge_kernel<<<dim3((rows_pad + 7) / 8, a.n_jobs), 256, 0, stream>>>(a, rows_it, score_key_groups(a.L_obs));
  CATEKV_CUDA_TRY(cudaGetLastError());
  if (out_mode == kScoreColsum)
    return small ? launch_one<kScoreColsum, 2>(a, stream) : launch_one<kScoreColsum, 4>(a, stream);
  return small ? launch_one<kScoreMatrix, 2>(a, stream) : launch_one<kScoreMatrix, 4>(a, stream);
}

}  // namespace catekv
