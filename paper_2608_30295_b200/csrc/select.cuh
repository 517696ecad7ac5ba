// Structures and launchers shared by the prefill-end selection (catekv_select_compact) and the per-step
// query-aware retrieval (catekv_retrieve_compact): top-k over pooled scores and the row gather.
#pragma once

#include "common.cuh"

namespace catekv {

constexpr int kPoolPrescored = 3;  // internal pool mode: P already holds one score per chunk of pool_param tokens

struct SelSeg {
  int32_t n;         // tokens of the sequence
  int32_t keep_all;  // 1: straight copy of all n rows
  int32_t job;       // scoring job index, -1 if none (keep_all, or nothing to select)
  int32_t k_sel;     // candidates (tokens, or chunks in CHUNK mode) to select
  int32_t n_pool;    // pooled entries (candidate tokens, or chunks)
  int32_t cand_end;  // candidates are tokens [sink, cand_end)
  int32_t len_ub;    // upper bound of the kept length (exact except for a short last chunk)
  int32_t reserved;
};

struct TopkArgs {
  const SelSeg* segs;
  const float* C;       // [n_jobs][c_stride] criticality of tokens [0, n - L_obs)
  float* P;             // [n_jobs][c_stride] pooled scores (scratch)
  int64_t c_stride;
  int32_t* idx;         // [n_segs][idx_stride] kept indices (scratch)
  int64_t idx_stride;
  int32_t* seg_len_dev;
  int32_t sink, L_obs, pool_mode, pool_param;  // the always-kept tail of a segment is [cand_end, n)
  int32_t mark_keep_all;  // 1: a keep_all segment gets seg_len_dev = -1 ("the whole list") instead of being skipped
  int32_t stage_entries;  // set by launch_topk: pooled entries per CTA that the dynamic shared memory holds
  int32_t* chk;           // set by launch_topk: the checked build's status block, else null
  int32_t row_is_seg;     // 1 (prescored lists only): the score row of segment s is row s, whatever its job says
  int32_t small_pool;     // set by launch_topk for topk_small_kernel: bound of the pooled entries of a segment
};

// Monotone map of arbitrary finite floats to non-negative floats whose bit patterns order the same way as the
// values (what the radix select of the top-k kernels needs): flip so that larger values get larger unsigned
// patterns, then clear the sign by halving the range.  Values one ulp apart may merge into a tie: within the
// parity tolerance band.  key_to_score inverts it up to that last bit (still monotone).
__device__ __forceinline__ float monotone_key(float x) {
  const uint32_t u = __float_as_uint(x);
  const uint32_t k = (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // unsigned order == float order
  return __uint_as_float(k >> 1);                                 // non-negative pattern
}
__device__ __forceinline__ float key_to_score(uint32_t key) {
  const uint32_t k = key << 1;
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

struct GatherArgs {
  const SelSeg* segs;
  const int32_t* idx;
  int64_t idx_stride;
  const uint8_t* k;
  const uint8_t* v;
  int64_t sb, sh, st;  // byte strides
  const int32_t* src_seg_off;  // if set: the source row of token t of segment s is src_seg_off[s] + t (sb, sh unused)
  uint8_t* k_pool;
  uint8_t* v_pool;
  const int32_t* seg_off;
  int32_t* seg_len_dev;  // kept length per segment: read for selecting segments, written for keep_all ones
  int32_t* idx_out;
  int64_t idx_out_stride;
  int32_t Hkv;
  const int32_t* seg_cap;  // capacity of every destination segment (device), or null: the copy is cut there
  int32_t* status;         // status block of the caller's workspace: CATEKV_STATUS_CAPACITY when a copy was cut
  int32_t* chk;            // set by launch_gather: the checked build's status block, else null
};


// max_pool: longest pooled list; n_active: upper bound of the segments that select (the others leave at once)
int launch_topk(const TopkArgs& a, int n_segs, int max_pool, int n_active, cudaStream_t stream);
int launch_gather(const GatherArgs& a, int max_len, int n_segs, cudaStream_t stream);

}  // namespace catekv
