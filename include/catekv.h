/*
 * catekv.h - C ABI of the CateKV hot path on one NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel part of CateKV (hybrid-head KV-cache
 * attention for long-context decoding):
 *
 *   catekv_head_cv         Section 3.2, Eq. 1-4: per-head coefficient-of-variation score
 *   catekv_classify_heads  Section 3.2, Eq. 5 + "Reference-Based Static Identification"
 *   catekv_select_compact  Algorithm 1, pre-filling stage: window scores, pooling,
 *                          per-KV-head top-k, Cache()
 *   catekv_append          growth of every head's list by the decoded token
 *                          (the paper is silent; implied by autoregressive decoding)
 *   catekv_decode_attn     Algorithm 1, decoding stage: Attention(q, k, v) over the
 *                          per-head lists ("all" retrieval on adaptive heads)
 *
 * Conventions
 *   - Every function returns 0 (CATEKV_OK) or a negative error code.  Arguments
 *     are checked on the host before anything is launched; a failed check
 *     launches nothing and changes no buffer.
 *   - "device" pointers are CUDA device memory owned by the caller; "host"
 *     pointers are ordinary host memory owned by the caller.  The library
 *     allocates no device memory.  Between calls it keeps the last CUDA error
 *     code (thread-local) and, per device, a few values it looks up once (SM
 *     count, which kernels have had their shared-memory limit raised, the
 *     address of the fixed scratch array of catekv_decode_attn_noalloc); these
 *     caches are atomics and safe to fill from several host threads.
 *   - Kernels are enqueued on the caller's stream (a cudaStream_t passed as
 *     void*); calls do not synchronise unless stated.
 *   - bf16 values are raw 16-bit patterns.  The head dimension d is the
 *     contiguous inner dimension and must be 128.  Hq / Hkv = G <= 8; where an
 *     observation window is involved, G * L_obs <= 512.
 *   - A "segment" is the cached list of one (sequence b, KV head h), index
 *     b * Hkv + h.  All segments of a layer live in two pools, k_pool and
 *     v_pool, each [total_rows, d] bf16; segment s owns rows
 *     [seg_off[s], seg_off[s] + seg_cap[s]) of which the first seg_len[s] are
 *     valid, in ascending token order.
 */
#ifndef CATEKV_H_
#define CATEKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CATEKV_OK 0
#define CATEKV_ERR_INVALID_ARG (-1) /* null pointer, negative size, inconsistent shapes */
#define CATEKV_ERR_UNSUPPORTED (-2) /* d != 128, G > 8, unknown mode */
#define CATEKV_ERR_CAPACITY (-3)    /* a segment would outgrow its capacity */
#define CATEKV_ERR_WORKSPACE (-4)   /* workspace or plan buffer too small */
#define CATEKV_ERR_CUDA (-5)        /* a CUDA call failed: see catekv_last_cuda_error() */
#define CATEKV_ERR_DEVICE (-6)      /* a kernel reported a failure in a status block: see catekv_workspace_status() */

#define CATEKV_POOL_NONE 0    /* top-k on the raw criticality C */
#define CATEKV_POOL_CHUNK 1   /* BlockMax(C, cs) of Algorithm 1; whole chunks are selected */
#define CATEKV_POOL_SLIDING 2 /* stride-1 max pool of odd width w, -inf padding */

#define CATEKV_OUT_BF16 0
#define CATEKV_OUT_FP32 1

#define CATEKV_HEAD_DIM 128
#define CATEKV_MAX_GROUP 8
#define CATEKV_SEG_ALIGN 128 /* rows; segment offsets and capacities are multiples of it */

typedef void* catekv_stream; /* cudaStream_t */

#define CATEKV_PAGE_ROWS 64 /* rows of an overflow page */

/*
 * Overflow pages of a cache: room for segments to grow past the capacity they were laid out with, without moving
 * what they hold (the paper sizes its caches up front and has no counterpart).  Row r of segment s lives in the
 * cache's own pools while r < seg_cap[s]; beyond that, row seg_cap[s] + 64 p + i is row 64 table[s][p] + i of the
 * overflow pools.  Pages are handed out by catekv_pages_reserve (host bump allocator) and never move or return.
 * All arrays are allocated by the caller; table and table_dev start out filled with -1, seg_pages with 0.
 */
typedef struct catekv_pages {
  int32_t max_pages;   /* table entries per segment */
  int32_t n_pages;     /* pages of the overflow pools */
  int32_t next_free;   /* host: pages handed out so far (start at 0) */
  int32_t reserved;
  void* k_ovf;         /* device, bf16 [n_pages * 64, d] */
  void* v_ovf;         /* device, bf16 [n_pages * 64, d] */
  int32_t* table_dev;  /* device [B*Hkv, max_pages] */
  int32_t* table;      /* host   [B*Hkv, max_pages], mirror of table_dev */
  int32_t* seg_pages;  /* host   [B*Hkv], pages handed to each segment */
  const int32_t* seg_cap_dev; /* device [B*Hkv], copy of the cache's seg_cap */
} catekv_pages;

/* Hybrid per-head KV cache of one layer (Section 1; Section 3.2 last paragraph). */
typedef struct catekv_cache {
  int32_t B;              /* sequences */
  int32_t Hkv;            /* KV heads */
  int32_t d;              /* head dim, 128 */
  int32_t reserved;       /* 0; set to 1 by catekv_select_compact when seg_len (host) holds upper bounds */
  int64_t total_rows;     /* rows of each pool */
  void* k_pool;           /* device, bf16 [total_rows, d] */
  void* v_pool;           /* device, bf16 [total_rows, d] */
  const int32_t* seg_off_dev; /* device [B*Hkv], first row of each segment */
  int32_t* seg_len_dev;       /* device [B*Hkv], valid rows; written by select_compact and append */
  const int32_t* seg_off;     /* host   [B*Hkv] */
  const int32_t* seg_cap;     /* host   [B*Hkv] */
  int32_t* seg_len;           /* host   [B*Hkv], mirror of seg_len_dev kept by the library's calls */
  catekv_pages* pages;        /* overflow pages, or NULL.  With pages a segment may hold up to
                                 seg_cap + 64 * seg_pages rows; catekv_append, catekv_cache_advance,
                                 catekv_decode_plan, catekv_decode_attn / _partials / _combine / _noalloc,
                                 catekv_append_decode_attn and catekv_cache_regrow (as the source) follow them;
                                 every other call refuses such a cache with CATEKV_ERR_UNSUPPORTED */
  const int32_t* seg_cap_dev; /* device [B*Hkv], copy of seg_cap, or NULL.  Kernels that write rows whose number
                                 is decided on the device (the gather of catekv_retrieve_compact) clamp to it;
                                 catekv_retrieve_compact requires it on its step cache, and both retrieval calls
                                 on `cache` (the scoring kernel shares out its work by the capacities) */
} catekv_cache;

/*
 * Device status block.  The first CATEKV_STATUS_BYTES of every workspace handed to catekv_select_compact,
 * catekv_head_cv, catekv_retrieve_compact and catekv_retrieve_select belong to it.  Kernels never trap or assert:
 * a kernel that cannot do its work records why here and returns, and the context stays usable.
 *   CATEKV_STATUS_WAIT_EXPIRED  a bounded wait of the tensor-core scoring kernel ran out (the CTA freed its tensor
 *                               memory and left); scores, and everything derived from them, are invalid
 *   CATEKV_STATUS_CAPACITY      a gather was cut at the capacity of its destination segment (a replayed retrieval
 *                               step whose step cache is too small for what the source has grown to)
 *   CATEKV_STATUS_INDEX_RANGE   checked build only (catekv_checked_build): a device-produced row index, page or
 *                               list position was outside its segment; the access was clamped into range
 * kernel / segment / index describe the first failure recorded (kernel: 1 scoring, 2 top-k, 3 gather,
 * 4 attention, 5 retrieval metadata).
 * catekv_select_compact and catekv_head_cv clear the block when they start.  The retrieval calls never clear it
 * (a replayed CUDA graph accumulates): zero the first CATEKV_STATUS_BYTES of a retrieval workspace once after
 * allocating it, or read it with clear != 0.
 */
#define CATEKV_STATUS_BYTES 256
#define CATEKV_STATUS_WAIT_EXPIRED 1
#define CATEKV_STATUS_CAPACITY 2
#define CATEKV_STATUS_INDEX_RANGE 4
typedef struct catekv_status {
  int32_t flags;   /* OR of CATEKV_STATUS_*; 0 = healthy */
  int32_t kernel;
  int32_t segment;
  int32_t index;
} catekv_status;

/*
 * Read the status block of workspace `ws` (device): copies it to *out (host, may be NULL) on `stream`,
 * synchronises the stream, and with clear != 0 zeroes the block afterwards.  Returns CATEKV_OK if no flag is
 * set, CATEKV_ERR_DEVICE if one is (the outputs of the calls that used the workspace since the block was last
 * cleared are then not to be trusted), CATEKV_ERR_CUDA if the copy fails.
 */
int catekv_workspace_status(void* ws, catekv_status* out, int32_t clear, catekv_stream stream);

/*
 * Checked build (the stand-in for a memory checker on machines where none can be run): a library compiled with
 * -DCATEKV_CHECKED (python -m paper_2608_30295_b200.build --checked) clamps every device-produced index to its
 * segment before using it - the kept lists read by the gather, the row lists and page-table entries of the
 * attention kernel, the positions the top-k writes, the chunk a metadata update folds into - and records the
 * first violation in a status block of its own.  catekv_checked_build returns 1 for such a library, 0 otherwise.
 * catekv_checked_status reads that block like catekv_workspace_status (device-wide synchronisation);
 * CATEKV_ERR_UNSUPPORTED in an unchecked library.
 */
int catekv_checked_build(void);
int catekv_checked_status(catekv_status* out, int32_t clear);

/*
 * Test hook, host side: the next n_launches launches of the tensor-core kernels (window scoring, window
 * attention) run with their producer lanes idle
 * (no copy and no tensor-core instruction is issued) and a wait limit of 512 polls, so that every wait runs out
 * with nothing in flight and the CATEKV_STATUS_WAIT_EXPIRED path executes.  Process-wide counter; 0 switches
 * it off.  Nothing faults or hangs: the CTAs free their tensor memory and return.
 */
void catekv_test_expire_score_waits(int32_t n_launches);

/* Version of this ABI (major * 1000 + minor). */
int catekv_version(void);
/* Static text for an error code. */
const char* catekv_error_string(int code);
/* cudaError_t value of the last CUDA failure seen by this thread (0 if none). */
int catekv_last_cuda_error(void);

/*
 * Canonical pool layout.  Host only.
 * len0 [B*Hkv]: rows each segment starts with; max_new: rows it may still grow by.
 * Writes seg_cap[s] = round_up(len0[s] + max_new, 128), seg_off = exclusive prefix
 * sum of seg_cap, *total_rows = sum of seg_cap.  All arrays are host arrays.
 */
int catekv_cache_layout(int32_t B, int32_t Hkv, const int32_t* len0, int32_t max_new,
                        int32_t* seg_off, int32_t* seg_cap, int64_t* total_rows);

/* ---------------------------------------------------------------- head identification */

/*
 * CV score of every (sequence, KV head): Section 3.2, Eq. 1-4.
 *
 * For each group: A = mean over the group's G query heads of
 * softmax(Q[-L_obs:] K[L_init : n - L_rec]^T / sqrt(d)) (Eq. 1, row softmax over
 * the sliced keys; with `causal` != 0 window row i, at position n - L_obs + i,
 * does not see later keys and those entries of A are 0);
 * Phi = alpha * (the floor(k (N-1))-th ascending element of the whole matrix A),
 * N = L_obs * m, m = n - L_init - L_rec (Eq. 2); C_j = #{i : A_ij >= Phi}
 * (Eq. 3); cv = population std(C) / mean(C), 0 when the mean is 0 (Eq. 4).
 *
 *   q_win   device bf16 [B, Hq, L_obs, d], contiguous
 *   k       device bf16, element strides (k_stride_b, k_stride_h, k_stride_t), d contiguous
 *   seq_len host [B], n of each sequence (n - L_init - L_rec >= 1, n >= L_obs)
 *   cv_out  device float [B*Hkv]
 *   ws      device scratch of at least catekv_head_cv_workspace_bytes(...)
 */
size_t catekv_head_cv_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t n_max, int32_t L_obs,
                                      int32_t L_init, int32_t L_rec);
int catekv_head_cv(const void* q_win, const void* k, int64_t k_stride_b, int64_t k_stride_h,
                   int64_t k_stride_t, const int32_t* seq_len, int32_t B, int32_t Hq, int32_t Hkv,
                   int32_t d, int32_t L_obs, int32_t L_init, int32_t L_rec, float quantile_k, float alpha,
                   int32_t causal, float* cv_out, void* ws, size_t ws_bytes, catekv_stream stream);

/*
 * Eq. 5 per sample and the static vote over a reference set.  Host only.
 * cv [n_samples, n_heads] host (n_heads = all KV heads of the model, flattened);
 * r = share of adaptive heads.  Per sample, Gamma = the floor(r (H-1))-th ascending
 * score and a head is consistent iff its score > Gamma.  mask_out[h] = 1 for the
 * H - (floor(r (H-1)) + 1) heads ranked first by (times classified consistent
 * descending, mean score descending, index ascending), else 0.
 */
int catekv_classify_heads(const float* cv, int32_t n_samples, int32_t n_heads, float r, uint8_t* mask_out);

/* ---------------------------------------------------------------- prefill-end selection */

typedef struct catekv_select_params {
  int32_t B, Hq, Hkv, d;
  int32_t L_obs;             /* observation window: the last L_obs queries */
  int32_t sink;              /* S: first tokens always kept */
  int32_t local;             /* Lc: last tokens always kept; must be >= L_obs */
  int32_t budget_consistent; /* token budget T of a consistent head (sink and local included) */
  float eta_adaptive;        /* adaptive head keeps T = floor(eta * n) tokens; >= 1 keeps all */
  int32_t pool_mode;         /* CATEKV_POOL_* */
  int32_t pool_param;        /* chunk size cs, or odd window w */
  int32_t reserved;
  const void* q_win;         /* device bf16 [B, Hq, L_obs, d], contiguous */
  const void* k;             /* device bf16 prefill keys   */
  const void* v;             /* device bf16 prefill values */
  int64_t kv_stride_b, kv_stride_h, kv_stride_t; /* element strides of k and v; d contiguous */
  const int32_t* seq_len;    /* host [B]: n of each sequence */
  const uint8_t* head_mask;  /* host [B*Hkv]: 0 = adaptive, 1 = consistent, 2 = streaming (T = sink + local; Section 4.2.4) */
  const float* row_lse_scored; /* device float [B, Hq, L_obs] or NULL: natural-log sum of exp(q.k / sqrt(d)) of every
                                  window query over the scored keys [0, n - L_obs), as catekv_window_attn (or any
                                  prefill attention pass that tracks it) delivers it.  With it the call skips its
                                  own first pass over K (the row maxima and sums) */
} catekv_select_params;

/*
 * Algorithm 1, pre-filling stage, for every (sequence, KV head):
 *   C_j = mean over the group's heads of sum_i softmax(Q_win K[:n-L_obs]^T / sqrt(d))_ij;
 *   pooled scores over the candidates [S, n - Lc);
 *   the k_rest = max(0, T - S - Lc) best candidates (ties: lowest index; CHUNK mode:
 *   floor(k_rest / cs) whole chunks, chunk origin at S, last chunk may be short);
 *   kept = [0, S) + selected + [n - Lc, n), ascending; K and V rows gathered in that
 *   order into the segment; seg_len set (device and host).  T >= n or S + Lc >= n
 *   keeps every token.
 *
 *   idx_out  device int32 [B*Hkv, idx_stride] or NULL: the kept indices of each segment
 *   ws       device scratch; its first CATEKV_STATUS_BYTES are the status block (cleared by this call)
 *   The call enqueues and returns; it never synchronises.  The host mirror cache->seg_len is
 *   computed on the host and is exact on return, except in CHUNK mode when (n - Lc - S) is not
 *   a multiple of cs and the head selects: whether the short last chunk is taken depends on the
 *   scores, so the mirror then holds the upper bound (the device length is at most cs - 1 rows
 *   shorter) and cache->reserved is set to 1.  catekv_cache_sync_lengths makes the mirror exact.
 *   Everything that only needs an upper bound works on such a cache (capacity checks, decode
 *   plans, catekv_decode_attn: every work item clamps to the device's length);
 *   catekv_append_decode_attn needs exact lengths and refuses it (CATEKV_ERR_INVALID_ARG).
 *   Errors: CATEKV_ERR_CAPACITY if a kept list can exceed its segment capacity.
 */
size_t catekv_select_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t n_max, int32_t L_obs);
int catekv_select_compact(const catekv_select_params* p, catekv_cache* cache, int32_t* idx_out,
                          int64_t idx_stride, void* ws, size_t ws_bytes, catekv_stream stream);

/*
 * Algorithm 1, pre-filling stage, seen from the prefill side: the window queries Q[-L_obs:] are ordinary prefill
 * queries, so their attention rows and softmax normalisers exist before any scoring starts.  This call is the
 * library's stand-in for that part of a prefill attention pass: for the last L_obs queries of every query head,
 *   out        = softmax(q K[:pos+1]^T / sqrt(d)) V[:pos+1], the causal attention row at position pos = n - L_obs + i
 *   lse        = natural-log sum of exp(logits) over that causal prefix (what attention kernels return as LSE)
 *   lse_scored = the same sum over the scored keys [0, n - L_obs) alone: the normaliser of the softmax in the
 *                "token criticality" line; hand it to catekv_select_compact as row_lse_scored
 * bf16 inputs, fp32 accumulation; the probabilities enter the P V product as a bf16 hi + lo pair.
 *   q_win  device bf16 [B, Hq, L_obs, d] contiguous;  k, v  device bf16 with element strides, d contiguous
 *   seq_len host [B], n >= L_obs;  out device [B, Hq, L_obs, d] bf16 or float per out_dtype
 *   lse_out, lse_scored_out device float [B, Hq, L_obs] or NULL (-inf where a row has no key)
 *   ws device scratch of at least catekv_window_attn_workspace_bytes(...); its first CATEKV_STATUS_BYTES are the
 *   status block (cleared by this call).
 * One sweep: K and V are each read once.
 */
size_t catekv_window_attn_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t n_max, int32_t L_obs);
int catekv_window_attn(const void* q_win, const void* k, const void* v, int64_t kv_stride_b, int64_t kv_stride_h,
                       int64_t kv_stride_t, const int32_t* seq_len, int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                       int32_t L_obs, void* out, int32_t out_dtype, float* lse_out, float* lse_scored_out, void* ws,
                       size_t ws_bytes, catekv_stream stream);

/*
 * Copy the device's segment lengths into the host mirror cache->seg_len (on `stream`, which is synchronised)
 * and clear cache->reserved.  Needed only after a catekv_select_compact that left upper bounds (see there).
 */
int catekv_cache_sync_lengths(catekv_cache* cache, catekv_stream stream);

/* ---------------------------------------------------------------- decoding */

/*
 * Append the decoded token's key and value to every segment.
 * k_new, v_new: device bf16 [B, Hkv, d] contiguous.  Row seg_off + seg_len of each
 * segment is written and seg_len grows by one on the device and in the host
 * mirror.  CATEKV_ERR_CAPACITY (nothing launched) if any segment is full.
 */
int catekv_append(catekv_cache* cache, const void* k_new, const void* v_new, catekv_stream stream);

/*
 * Host mirror only: record that n_tokens appends have run (or are about to run) on the device without
 * the library's host code seeing them - the case of a caller who captured catekv_append in a CUDA
 * graph and replays it.  Call it before each replay: it checks every segment's capacity
 * (CATEKV_ERR_CAPACITY, nothing changed) and then adds n_tokens to cache->seg_len.  Launches nothing.
 */
int catekv_cache_advance(catekv_cache* cache, int32_t n_tokens);

/*
 * Paged growth.  Makes sure that every segment can take n_new more rows: segments whose capacity
 * (seg_cap + 64 * seg_pages) is short get further overflow pages, the new table entries are copied to the device
 * on `stream` (from cache->pages->table: leave it untouched until that copy has run).  Host bookkeeping only
 * besides that copy; nothing is launched.  CATEKV_ERR_CAPACITY (nothing changed) if the overflow pools or a
 * segment's table row run out; CATEKV_ERR_INVALID_ARG if the cache has no pages.  Decode plans built before
 * stay valid.  catekv_cache_regrow with such a cache as the source gathers base rows and pages into one
 * contiguous segment again.
 */
int catekv_pages_reserve(catekv_cache* cache, int32_t n_new, catekv_stream stream);

/*
 * Growth beyond the capacity a cache was laid out with (Section 4.4.3 keeps generating for as long as the
 * request runs; the paper sizes its caches up front and has no counterpart to this call).  The caller lays out
 * a second cache with larger capacities (catekv_cache_layout with a larger max_new), and this call copies the
 * seg_len valid rows of every segment of `src` to the start of the same segment of `dst` and sets dst's lengths
 * (device and host mirror).  src is left untouched; plans and retrieval metadata are per cache and must be
 * rebuilt for dst.  CATEKV_ERR_CAPACITY (nothing launched) if a segment of src does not fit its segment of dst;
 * CATEKV_ERR_INVALID_ARG if the two caches differ in B or Hkv or share a pool.
 */
int catekv_cache_regrow(const catekv_cache* src, catekv_cache* dst, catekv_stream stream);

/*
 * Work-balanced split-KV schedule for catekv_decode_attn.
 *
 * The rows of all segments, laid end to end, are cut into num_ctas near-equal
 * ranges; a range that crosses segment boundaries yields one work item per
 * segment it touches, so short (consistent) and long (adaptive) segments load
 * every CTA evenly.  The plan is built on the host from cache->seg_len, stored
 * in plan_host and copied to plan_dev (cudaMemcpyAsync on `stream`; plan_host
 * must stay untouched until that copy has run - use pinned memory to make it
 * asynchronous).  A plan stays valid while the segments' lengths change within
 * their capacities: every item reads the current length on the device, the last
 * item of a segment follows rows appended since (append), and rows behind a length
 * that has shrunk (a per-step cache refilled by catekv_retrieve_compact) are left
 * out; rebuild it now and then to restore balance.  catekv_append_decode_attn
 * alone needs lengths that are not below the plan's (ERR_INVALID_ARG otherwise).
 *
 * catekv_decode_num_ctas: SM count * resident CTAs per SM of the decode kernel
 * on the current device (a CUDA query); < 0 on error.
 */
int catekv_decode_num_ctas(void);
size_t catekv_decode_plan_bytes(int32_t B, int32_t Hkv, int32_t num_ctas);
size_t catekv_decode_workspace_bytes(int32_t B, int32_t Hkv, int32_t num_ctas);
int catekv_decode_plan(const catekv_cache* cache, int32_t num_ctas, void* plan_host, void* plan_dev,
                       size_t plan_bytes, catekv_stream stream);

/*
 * Attention(q, k, v) of Algorithm 1 for one decode step: for every query head hq
 * of every sequence, softmax(sm_scale * q . K^T) V over the current list of KV
 * head hq / G.  bf16 inputs, fp32 accumulation; the logit scale is applied in
 * fp32 after the dot product.
 *
 *   q        device bf16 [B, Hq, d] contiguous
 *   sm_scale 0 means 1/sqrt(d)
 *   out      device [B, Hq, d], bf16 or float per out_dtype; an empty list gives 0
 *   lse_out  device float [B, Hq] or NULL: natural-log sum of exp(logits); -inf if empty
 *   plan_host / plan_dev  the plan built by catekv_decode_plan for this cache
 *   ws       device scratch of at least catekv_decode_workspace_bytes(...)
 *
 * Ordering: the kernels use programmatic dependent launch.  They wait for all earlier work of the
 * stream before they read lengths, queries or appended rows, but they may request cache rows that
 * were valid when the plan was built while the previous kernel is still finishing.  Such rows must
 * therefore not be rewritten (by catekv_select_compact, say) between catekv_decode_plan and this call.
 */
int catekv_decode_attn(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                       int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                       size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream);

/*
 * The two phases of catekv_decode_attn as separate calls, with the same arguments: the split-KV
 * attention partials (every CTA range of the plan: online softmax over its rows; a segment that
 * fits one range is written to `out` directly) and the combine pass (log-sum-exp merge of the
 * partials of every segment that was cut).  catekv_decode_attn is exactly partials then combine
 * on one stream; the split exists so that a caller can time or overlap the phases.
 */
int catekv_decode_partials(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                           int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                           size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream);
int catekv_decode_combine(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                          int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                          size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream);

/* ---------------------------------------------------------------- query-aware retrieval */

/*
 * Algorithm 1, decoding stage: "k, v = Retrival(q, cache)" on adaptive heads in its query-aware form, with the
 * page criterion of Quest (the retrieval method the paper combines with, chunk size 8; Section 4.2.2 and
 * appendix B.2.2).  The full list of a retrieval head stays in `cache`; every step a subset of its rows is
 * gathered into the same segment of a second, small cache (`step_cache`, same B and Hkv) on which
 * catekv_decode_attn then runs unchanged.
 *
 *   metadata  per chunk of chunk_size consecutive cached rows (chunks start at row 0 of a segment) the
 *             element-wise maximum and minimum of the keys: device bf16 [total_rows / chunk_size][2][d].
 *             chunk_size must divide 128.  catekv_retrieval_build fills it for all current rows of all
 *             segments; catekv_retrieval_append folds in the row that the preceding catekv_append (or
 *             catekv_append_decode_attn) stored, k_new being that call's k_new.
 *   score     bound(c) = max over the group's G query heads of sum_d max(q_d kmin_d, q_d kmax_d), an upper
 *             bound of q.k over the chunk's rows (fp32).
 *   select    (segments with retrieval_mask[s] != 0 and more than `budget` rows) the chunks holding the first
 *             `sink` rows and every chunk from the one holding row len - local on are always taken; of the
 *             chunks in between the floor((budget - forced rows) / chunk_size) with the largest bound, ties to
 *             the lowest chunk.  Other segments are copied whole.
 *   gather    the taken rows, ascending, K and V; step_cache->seg_len (device and host) is set; the kept
 *             length depends only on the lengths and the parameters, never on the scores.
 *
 *   q         device bf16 [B, Hq, d], this step's queries
 *   idx_out   device int32 [B*Hkv, idx_stride] or NULL: the rows taken from each segment
 *   ws        device scratch of at least catekv_retrieve_workspace_bytes(B, Hkv, largest seg_cap of `cache`)
 * Errors: CATEKV_ERR_CAPACITY if a kept list does not fit its segment of step_cache (nothing launched);
 * CATEKV_ERR_INVALID_ARG if cache or step_cache has no seg_cap_dev;
 * CATEKV_ERR_UNSUPPORTED for more than 2048 segments (the mask travels in the kernel arguments).
 * The call copies nothing from the host and takes every per-segment decision on the device from the device's
 * lengths; launch shapes follow the capacities.  A step (append, metadata append, this call, attention over
 * step_cache with a plan built once) can therefore be captured in a CUDA graph and replayed while the caches
 * grow; step_cache->seg_len on the host is then the value of the captured call (an upper bound: the kept
 * length moves within one chunk as the source grows).  The capacity check above sees the lengths of the call
 * that was captured, not those of later replays: a step-cache segment that is copied whole (mask 0, or not
 * longer than the budget) has to be as large as its source segment may become, one that retrieves needs
 * budget + 2 * chunk_size rows.  On the device the gather never writes past seg_cap_dev of the step cache: a
 * list that does not fit is cut there, step_cache's device length is set to the rows written, and
 * CATEKV_STATUS_CAPACITY is raised in the status block at the start of `ws` (catekv_workspace_status).
 */
size_t catekv_retrieval_meta_bytes(const catekv_cache* cache, int32_t chunk_size);
int catekv_retrieval_build(const catekv_cache* cache, int32_t chunk_size, void* meta, catekv_stream stream);
int catekv_retrieval_append(const catekv_cache* cache, int32_t chunk_size, const void* k_new, void* meta,
                            catekv_stream stream);
/* catekv_append and catekv_retrieval_append in one launch (same checks and errors as catekv_append). */
int catekv_append_retrieval(catekv_cache* cache, const void* k_new, const void* v_new, int32_t chunk_size, void* meta,
                            catekv_stream stream);
size_t catekv_retrieve_workspace_bytes(int32_t B, int32_t Hkv, int32_t max_len);
int catekv_retrieve_compact(const catekv_cache* cache, const void* meta, int32_t chunk_size, const void* q, int32_t Hq,
                            const uint8_t* retrieval_mask, int32_t budget, int32_t sink, int32_t local,
                            catekv_cache* step_cache, int32_t* idx_out, int64_t idx_stride, void* ws, size_t ws_bytes,
                            catekv_stream stream);

/*
 * The same retrieval without the copy: catekv_retrieve_select stops after the chunk selection and leaves, per
 * segment, the ascending list of the rows to attend to; catekv_decode_attn_indexed then reads those rows in
 * place, straight from `cache` (the same split-KV kernel, each 256-byte row addressed through the list), and
 * the whole list of every segment that retrieves nothing.  No per-step cache, no gather traffic.
 *
 *   idx      device int32 [B*Hkv, idx_stride]: rows (relative to the segment) of the segments that retrieve;
 *            idx_stride must hold the longest kept list (catekv_retrieve_lengths)
 *   sel_len  device int32 [B*Hkv]: the kept length of a segment that retrieves, -1 for a segment that is
 *            attended to as a whole (mask 0, or not longer than the budget)
 *   catekv_retrieve_lengths: host only; lens_out[s] = rows segment s will be attended over for these
 *            parameters and the current host lengths.  A decode plan for catekv_decode_attn_indexed is built by
 *            catekv_decode_plan from a cache descriptor whose host seg_len array holds these lengths (same
 *            pools, offsets and capacities); like every plan it stays valid while the lengths move.
 *   The other arguments, the errors and the CUDA-graph property are those of catekv_retrieve_compact and
 *   catekv_decode_attn.  catekv_decode_attn_indexed requests no rows before the preceding kernel has finished
 *   (the lists are that kernel's output).
 */
int catekv_retrieve_select(const catekv_cache* cache, const void* meta, int32_t chunk_size, const void* q, int32_t Hq,
                           const uint8_t* retrieval_mask, int32_t budget, int32_t sink, int32_t local, int32_t* idx,
                           int64_t idx_stride, int32_t* sel_len, void* ws, size_t ws_bytes, catekv_stream stream);
int catekv_retrieve_lengths(const catekv_cache* cache, int32_t chunk_size, const uint8_t* retrieval_mask, int32_t budget,
                            int32_t sink, int32_t local, int32_t* lens_out);
int catekv_decode_attn_indexed(const catekv_cache* cache, const int32_t* idx, int64_t idx_stride, const int32_t* sel_len,
                               const void* q, int32_t Hq, float sm_scale, void* out, int32_t out_dtype, float* lse_out,
                               const void* plan_host, const void* plan_dev, size_t plan_bytes, void* ws, size_t ws_bytes,
                               catekv_stream stream);

/*
 * Attention recall of the kept rows (Section 3.4, the recall curves of the consistent / streaming / Quest /
 * top-k patterns): for each query head, the share of the full softmax mass that falls on the rows its hybrid
 * list keeps, recall = exp(lse_kept - lse_full), 0 for an empty list.  lse_kept is the lse_out of a
 * catekv_decode_attn call over the hybrid cache, lse_full that of a call with the same queries over a cache
 * that keeps every token.  All three arrays: device float [n].
 */
int catekv_attention_recall(const float* lse_kept, const float* lse_full, float* recall, int32_t n,
                            catekv_stream stream);

/*
 * catekv_append followed by catekv_decode_attn, as one call with one attention launch: the CTA that
 * owns the end of a segment takes the decoded token's row from k_new / v_new, attends to it and stores
 * it in the pool; seg_len grows by one (device and host mirror).  Same results as the two calls.
 * CATEKV_ERR_CAPACITY (nothing launched) if any segment is full.
 */
int catekv_append_decode_attn(catekv_cache* cache, const void* k_new, const void* v_new, const void* q, int32_t Hq,
                              float sm_scale, void* out, int32_t out_dtype, float* lse_out, const void* plan_host,
                              const void* plan_dev, size_t plan_bytes, void* ws, size_t ws_bytes,
                              catekv_stream stream);

/*
 * catekv_decode_attn for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, same arithmetic, same results.)
 *
 * Who needs it: hosts that take all of the GPU's memory for themselves at start-up and give a
 * plugin no allocator afterwards (an inference server with a pre-sized arena, a sandboxed
 * extension), and code on a request path where an allocation would stall the whole device
 * (cudaMalloc and cudaFree synchronise it) or fail because nothing is left.  Such callers still
 * own the inputs, the cache, the plan and `out`; what they lack is a place for the split-KV
 * partials.  Here those live in a fixed array of CATEKV_NOALLOC_SCRATCH_BYTES (4 MiB) that is
 * part of the library image: every GPU that loads the library carries it until the process
 * exits, whether or not this function is ever called.
 *
 * The call allocates and frees nothing, on the device or through any library.  Its arguments are
 * those of catekv_decode_attn minus ws / ws_bytes.  A plan whose partials do not fit
 * - (num_ctas + B*Hkv) * 4128 bytes > CATEKV_NOALLOC_SCRATCH_BYTES, i.e. more than 1016 slots -
 * is refused with CATEKV_ERR_WORKSPACE before anything is launched; build the plan with fewer
 * CTAs or use catekv_decode_attn.
 *
 * The first call on a device looks up the array's device address (with that device current) and
 * keeps it; make that first call outside any stream capture.  All calls of a process share the
 * one array per GPU: nothing in it has to start at zero and it keeps whatever the last call left,
 * but two calls whose kernels overlap on the same GPU (different streams, or different threads)
 * would overwrite each other's partials - keep them on one stream or otherwise ordered.
 */
#define CATEKV_NOALLOC_SCRATCH_BYTES (4u << 20)
int catekv_decode_attn_noalloc(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                               int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                               size_t plan_bytes, catekv_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* CATEKV_H_ */
