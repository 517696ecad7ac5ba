// Head identification statistic (Section 3.2, Eq. 1-4): observation matrix, matrix-global
// percentile threshold, per-column counts, coefficient of variation.
#include <math.h>

#include <vector>

#include "radix.cuh"
#include "score.cuh"

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

// One CTA per (sequence, KV head): Phi = alpha * percentile element (Eq. 2), C_j = #{i: A_ij >= Phi}
// (Eq. 3), cv = std_pop(C) / mean(C) (Eq. 4) from exact integer sums.
__global__ void __launch_bounds__(kCvThreads) cv_kernel(const CvArgs a) {
  const int seg = blockIdx.x;
  const CvSeg s = a.segs[seg];
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_pair[2];
  __shared__ unsigned long long red[2][32];
  const float* A = a.A + (size_t)seg * a.seg_stride;
  const unsigned int* Ab = reinterpret_cast<const unsigned int*>(A);
  const int m = s.m;
  const int N = a.L_obs * m;
  unsigned int thr, need_eq;
  block_radix_select([&](int e) { return Ab[e]; }, N, (unsigned int)s.need, hist, s_pair, thr, need_eq);
  const float phi = __uint_as_float(thr) * a.alpha;
  unsigned long long sum = 0, sum2 = 0;
  for (int j = threadIdx.x; j < m; j += kCvThreads) {
    unsigned int c = 0;
#pragma unroll 8
    for (int i = 0; i < a.L_obs; ++i) c += A[(size_t)i * m + j] >= phi ? 1u : 0u;
    sum += c;
    sum2 += (unsigned long long)c * c;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
    sum2 += __shfl_xor_sync(0xffffffffu, sum2, o);
  }
  if (lane == 0) { red[0][warp] = sum; red[1][warp] = sum2; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long S1 = 0, S2 = 0;
    for (int w = 0; w < kCvThreads / 32; ++w) { S1 += red[0][w]; S2 += red[1][w]; }
    // std_pop / mean = sqrt(m * sum(C^2) - (sum C)^2) / sum C
    double cv = 0.0;
    if (S1 > 0) {
      const double num = (double)m * (double)S2 - (double)S1 * (double)S1;
      cv = sqrt(num > 0.0 ? num : 0.0) / (double)S1;
    }
    a.cv_out[seg] = (float)cv;
  }
}

struct CvWs {
  size_t off_status, off_segs, off_jobs, off_part, off_stats, off_A, bytes;
  int keys_per_cta, n_chunks;
  int64_t row_stride;
};
static CvWs cv_ws_layout(int n_segs, int G, int m_max, int L_obs) {
  CvWs w;
  int kp = 512;
  while ((long)n_segs * ((m_max + kp - 1) / kp) > 148 * 4 && kp < (1 << 30)) kp *= 2;
  w.keys_per_cta = kp;
  w.n_chunks = (m_max + kp - 1) / kp;
  w.row_stride = (int64_t)align_up((size_t)m_max, 64);
  size_t o = 0;
  w.off_status = o; o = 256;
  w.off_segs = o; o = align_up(o + sizeof(CvSeg) * (size_t)n_segs, 256);
  w.off_jobs = o; o = align_up(o + sizeof(ScoreJob) * (size_t)n_segs, 256);
  w.off_part = o; o = align_up(o + sizeof(float2) * (size_t)(n_segs + 148 * 4) * 2 * kScoreMaxRows, 256);
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
  CATEKV_CUDA_TRY(cudaMemsetAsync(w8 + W.off_status, 0, 256, st));
  CATEKV_CUDA_TRY(cudaMemcpyAsync(w8 + W.off_segs, segs.data(), sizeof(CvSeg) * n_segs, cudaMemcpyHostToDevice, st));
  CATEKV_CUDA_TRY(cudaMemcpyAsync(w8 + W.off_jobs, jobs.data(), sizeof(ScoreJob) * n_segs, cudaMemcpyHostToDevice, st));
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
  sa.scale_log2 = 1.4426950408889634f / sqrtf((float)kD);
  sa.keys_per_cta = score_keys_per_cta(n_segs, m_max);
  sa.n_chunks = (m_max + sa.keys_per_cta - 1) / sa.keys_per_cta;
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
  cv_kernel<<<n_segs, kCvThreads, 0, st>>>(ca);
  CATEKV_CUDA_TRY(cudaGetLastError());
  return CATEKV_OK;
}
