// Observation-window scoring shared by catekv_select_compact (Algorithm 1, token criticality)
// and catekv_head_cv (Eq. 1): softmax(Q_win K^T / sqrt(d)) over a key range, per query head
// of the group, reduced either to column sums (C_j) or to the group-mean matrix (A_ij).
#pragma once

#include "common.cuh"

namespace catekv {

// One (sequence, KV head) to score: keys [j_begin, j_end) of a sequence of n tokens.
struct ScoreJob {
  int32_t b, h, n, j_begin, j_end, reserved;
};

struct ScoreArgs {
  const uint16_t* q_win;  // [B, Hq, L_obs, d]
  const uint16_t* k;      // element strides sb, sh, st; d contiguous
  int64_t sb, sh, st;
  const ScoreJob* jobs;   // device
  int32_t n_jobs, Hq, G, L_obs, causal;
  int32_t g_major;        // row order of the window queries: 0: r = i * G + g; 1: r = g * L_obs + i (matrix mode, L_obs = 64)
  int32_t B, Hkv, n_max;  // extents of k (sequences, KV heads, tokens) for the TMA descriptor
  float scale_log2;       // log2(e) / sqrt(d)
  int32_t max_keys;       // longest key range of any job
  int32_t n_jobs_split;   // jobs the key ranges are cut for (0: n_jobs); smaller when some jobs are known to be tiny
  int32_t stats_given;    // 1: `stats` already holds every row's (max, sum): the first pass and its merge are skipped
  int32_t keys_per_cta;   // multiple of 128 (set by score_launch, per group of jobs)
  int32_t n_chunks;       // grid.x: ceil(max key range / keys_per_cta) (set by score_launch)
  float2* stats_part;     // [n_jobs][n_chunks][kScoreMaxRows]  per-CTA (row max in the log2 domain, row sum)
  float2* stats;          // [n_jobs][kScoreMaxRows]            merged (row max, row sum)
  int32_t* status;        // device status block: CATEKV_STATUS_WAIT_EXPIRED is raised if a tensor-core wait ever runs out
  uint32_t spin_limit;    // polls a wait may take (set by score_launch)
  int32_t idle_producer;  // test hook: the TMA / MMA lane issues nothing, so every wait runs out (set by score_launch)
  float* out;             // column sums C[job][j - j_begin], or the dense matrix A[job][i * m + (j - j_begin)], m = j_end - j_begin
  int64_t out_job_stride;
};

enum ScoreMode { kScoreStats = 0, kScoreColsum = 1, kScoreMatrix = 2 };

constexpr int kScoreMaxRows = 512;  // G * L_obs may not exceed this (8 heads x 64 window rows)
// Keys per CTA for n_jobs jobs of at most max_keys keys: a multiple of 128 chosen so that the grid is close to two
// CTAs per SM in whole waves (never more than score_max_ctas(n_jobs)).
int score_keys_per_cta(int n_jobs, int max_keys);
// Upper bound of n_jobs * n_chunks for keys_per_cta = score_keys_per_cta(n_jobs, .): the per-CTA row partials of
// pass 1 are sized by it.  (chunks = round(2 SMs / jobs), so jobs * chunks <= 2 SMs + jobs / 2.)
static inline int score_max_ctas(int n_jobs) { return n_jobs + 4 * sm_count(); }
// Test hook (catekv_test_expire_score_waits): true if the launch about to be made is to run with an idle producer
// lane and a short wait limit; consumes one of the requested launches.
bool score_take_expire_launch();
// Enqueue: pass 1 (row max / sum partials), their merge, and pass 2 (column sums or matrix).
int score_launch(const ScoreArgs& a, ScoreMode out_mode, cudaStream_t stream);

}  // namespace catekv
