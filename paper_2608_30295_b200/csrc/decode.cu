// Decoding stage of Algorithm 1: the split-KV attention partials and the combine pass over per-(sequence, KV head)
// variable-length caches (the schedule is built in plan.cu, the lists grow in cache.cu).
//
// The attention kernel is a memory-bound stream over the K and V rows of the cache.  Each CTA
// owns a contiguous range of the rows of all segments laid end to end (so short consistent
// heads and long adaptive heads load the SMs evenly), stages 64-row K/V tiles through a
// multi-stage cp.async pipeline into XOR-swizzled shared memory, and uses the tensor cores
// only to keep the ALU work off the critical path: the G <= 8 query heads of the group are
// packed into the N = 8 dimension of mma.m16n8k16 (tokens are M), softmax runs online per
// warp in fp32, and P enters the P.V product as a bf16 hi + lo pair so that no precision of
// the fp32 probabilities is lost.
#include <math.h>

#include <atomic>

#include "decode.cuh"

namespace catekv {

// ------------------------------------------------------------------------------------------
// Attention partials
// ------------------------------------------------------------------------------------------
struct DecodeArgs {
  uint8_t* k_pool;
  uint8_t* v_pool;
  const int32_t* seg_off;
  int32_t* seg_len;
  const uint8_t* k_new;  // fused append: this step's [B*Hkv, d] rows, else null
  const uint8_t* v_new;
  // indexed variant only: segment s attends to the rows idx[s * idx_stride + 0 .. sel_len[s]) of its list (ascending
  // row numbers relative to the segment) if sel_len[s] >= 0, to its whole list if sel_len[s] < 0
  const int32_t* idx;
  int64_t idx_stride;
  const int32_t* sel_len;
  // paged variant only: row r >= cap of segment s is row 64 * page_table[s * max_pages + (r - cap) / 64] + (r - cap) % 64
  // of the overflow pools
  uint8_t* k_ovf;
  uint8_t* v_ovf;
  const int32_t* page_table;
  int32_t max_pages;
  const uint16_t* q;  // [B, Hq, d]
  int32_t Hq, Hkv, G;
  float scale_log2;  // sm_scale * log2(e)
  const CtaHeader* ctas;
  const WorkItem* items;
  float* part_o;    // [slots, 8, 128]
  float* part_lse;  // [slots, 8], log2 domain
  void* out;
  int32_t out_fp32;
  float* lse_out;
  int32_t n_pages;  // pages of the overflow pools (checked build: bound of a page-table entry)
  int32_t* chk;     // the checked build's status block, else null
};

constexpr int kStageBytes = 2 * kTile * kRowBytes;     // K tile + V tile
constexpr int kQSlotBytes = kMaxG * kRowBytes;         // 8 query rows
constexpr int kMergeRegs = 36;                         // 32 accumulators + m0, m1, l0, l1
constexpr int kMergeSlotBytes = kMergeRegs * 32 * 4;
constexpr int kDecodeSmem = kStages * (kStageBytes + kQSlotBytes) + 2 * kMergeSlotBytes;

// A piece is streamed as 64-row tiles of its rows [t0, live): live is t1 for an inner piece of a segment (or less,
// if the segment has shrunk) and the segment's current length for its last piece, which so also covers the rows
// appended since the plan was built - they continue the piece's last, partly filled plan-time tile.  The live
// length is loaded when the item is read but first used only after the tiles that hold nothing but plan-time rows
// (np of them: these may be requested before the dependency wait) have been issued, so the stream never waits
// for that load.
constexpr int kModePlain = 0, kModeIndexed = 1, kModePaged = 2;  // instantiations of the attention kernel
struct ItemCursor {
  int seg, t0, t1, slot, last;
  int np;            // leading tiles that hold only plan-time rows
  int live;          // rows to attend to: current segment length (plus the row being appended), if last
  int new_row;       // fused append: the segment-relative row that comes from k_new / v_new, else -1
  int indexed;       // indexed variant: the item's rows are taken through the index list
  int cap;           // paged variant: rows from here on live in overflow pages
  int64_t row_base;
};

// the part of a cursor that needs only the plan
__device__ __forceinline__ ItemCursor plan_cursor(const WorkItem& w) {
  ItemCursor c;
  c.seg = w.seg;
  c.t0 = w.t0;
  c.t1 = w.t1;
  c.slot = w.slot;
  c.last = w.last;
  c.row_base = w.row_base;
  // tiles of plan-time rows only; the last piece's partly filled tile is left to the live length
  c.np = w.last ? (w.t1 - w.t0) / kTile : (w.t1 - w.t0 + kTile - 1) / kTile;
  c.live = w.t1;
  c.new_row = -1;
  c.indexed = 0;
  c.cap = w.cap;
  return c;
}
// the part that depends on what earlier kernels wrote: the live length (with a fused append this kernel itself
// updates the length when it is done with the segment); len and sel are the loaded seg_len / sel_len entries
template <int kMode>
__device__ __forceinline__ void apply_live(const DecodeArgs& a, ItemCursor& c, int len, int sel) {
  constexpr bool kIndexed = kMode == kModeIndexed;
  if (kIndexed) {
    c.indexed = sel >= 0;
    if (sel >= 0) len = sel;
  }
  if (c.last) {
    c.new_row = (!kIndexed && a.k_new) ? len : -1;
    c.live = (!kIndexed && a.k_new) ? len + 1 : len;
  } else {
    c.live = min(c.t1, len);  // a segment that has shrunk since the plan was built: attend only to what it holds
  }
}
template <int kMode>
__device__ __forceinline__ void live_cursor(const DecodeArgs& a, ItemCursor& c) {
  const int len = *reinterpret_cast<const volatile int32_t*>(a.seg_len + c.seg);
  const int sel = kMode == kModeIndexed ? *reinterpret_cast<const volatile int32_t*>(a.sel_len + c.seg) : -1;
  apply_live<kMode>(a, c, len, sel);
}
// What the cursor of the next piece is made of, requested one piece ahead: a piece change then finds the values in
// registers instead of waiting for two dependent loads while no tile is being issued.
struct NextItem {
  int4 x, y;
  int len, sel;
};
__device__ __forceinline__ WorkItem unpack_item(const int4& x, const int4& y) {
  WorkItem w;
  w.seg = x.x; w.t0 = x.y; w.t1 = x.z; w.slot = x.w;
  w.row_base = (int64_t)(((uint64_t)(uint32_t)y.y << 32) | (uint32_t)y.x);
  w.last = y.z; w.cap = y.w;
  return w;
}
// item `it` belongs to segment `seg` (pieces after a CTA's first belong to consecutive segments)
template <int kMode>
__device__ __forceinline__ void fetch_next(const DecodeArgs& a, int it, int seg, NextItem& n) {
  const int4* p = reinterpret_cast<const int4*>(a.items + it);
  n.x = __ldg(p);
  n.y = __ldg(p + 1);
  n.len = *reinterpret_cast<const volatile int32_t*>(a.seg_len + seg);
  n.sel = kMode == kModeIndexed ? *reinterpret_cast<const volatile int32_t*>(a.sel_len + seg) : -1;
}
template <int kMode>
__device__ __forceinline__ ItemCursor make_cursor(const DecodeArgs& a, const NextItem& n) {
  ItemCursor c = plan_cursor(unpack_item(n.x, n.y));
  apply_live<kMode>(a, c, n.len, n.sel);
  return c;
}
// tiles of the item's live rows; at least one
__device__ __forceinline__ int item_tiles(const ItemCursor& c) {
  return max(1, (c.live - c.t0 + kTile - 1) / kTile);
}
// first row (relative to the segment) and number of valid rows of tile i (may exceed kTile, or be <= 0 for a tile
// that lies behind the live length)
__device__ __forceinline__ void tile_rows(const ItemCursor& c, int i, int& start, int& nvalid) {
  start = c.t0 + i * kTile;
  nvalid = c.live - start;
}

template <int kMode>
__global__ void __launch_bounds__(kDecodeThreads, 2) decode_partial_kernel(const DecodeArgs a) {
  constexpr bool kIndexed = kMode == kModeIndexed;
  constexpr bool kPaged = kMode == kModePaged;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ ItemCursor s_ring[4];  // cursors of the pieces the producer has started, for the consumer
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  pdl_launch_dependents();
  int item_begin, item_end;
  ItemCursor pc;
  {
    // the plan was uploaded by a copy that precedes the previous kernel: it may be read before the wait
    const int4* hp = reinterpret_cast<const int4*>(a.ctas + blockIdx.x);
    const int4 h0 = __ldg(hp), x = __ldg(hp + 1), y = __ldg(hp + 2);
    item_begin = h0.x;
    item_end = h0.y;
    if (item_begin >= item_end) return;
    pc = plan_cursor(unpack_item(x, y));
  }

  const uint32_t s_stage = smem_u32(smem);
  const uint32_t s_q = s_stage + kStages * kStageBytes;
  float* merge = reinterpret_cast<float*>(smem + kStages * (kStageBytes + kQSlotBytes));

  // ---- producer
  int p_item = item_begin, p_tile = 0, p_seq = 0;
  int ix[(kTile * 16) / kDecodeThreads];  // indexed variant: see load_idx
  auto issue_tile = [&]() {  // tile p_tile of the producer's item into stage p_seq % kStages
    const uint32_t sb = s_stage + (p_seq % kStages) * kStageBytes;
    int start, rows_left;
    tile_rows(pc, p_tile, start, rows_left);
    const int64_t row0 = pc.row_base + (start - pc.t0);
    const int new_r = pc.new_row - start;  // tile row that is being appended by this call, if in [0, kTile)
    // paged variant: a tile touches at most two overflow pages; their table entries are read once, together
    int pg0 = 0, page0 = 0, page1 = 0;
    if (kPaged && start + kTile > pc.cap && rows_left > 0) {
      pg0 = max(0, start - pc.cap) >> 6;
      const int32_t* row = a.page_table + (int64_t)pc.seg * a.max_pages;
      page0 = __ldg(row + min(pg0, a.max_pages - 1));
      page1 = __ldg(row + min(pg0 + 1, a.max_pages - 1));
#ifdef CATEKV_CHECKED
      // a page the tile's valid rows reach must have been handed out (an entry behind them may still be -1)
      if (start + rows_left > pc.cap + pg0 * 64) page0 = checked_clamp(page0, 0, a.n_pages - 1, a.chk, kKidAttention, pc.seg);
      if (start + rows_left > pc.cap + (pg0 + 1) * 64) page1 = checked_clamp(page1, 0, a.n_pages - 1, a.chk, kKidAttention, pc.seg);
#endif
    }
#pragma unroll
    for (int i = 0; i < (kTile * 16) / kDecodeThreads; ++i) {
      const int id = tid + i * kDecodeThreads;
      const int r = id >> 4, c = id & 15;
      const int ok = r < rows_left ? 16 : 0;
      int64_t grow = ok ? row0 + r : 0;  // padding rows read nothing
      uint8_t* kp = a.k_pool;
      uint8_t* vp = a.v_pool;
#ifdef CATEKV_CHECKED
      // a list entry names a row of its own segment
      if (kIndexed && pc.indexed && ok) ix[i] = checked_clamp(ix[i], 0, pc.cap - 1, a.chk, kKidAttention, pc.seg);
#endif
      if (kIndexed && pc.indexed && ok) grow = (pc.row_base - pc.t0) + ix[i];
      if (kPaged && ok && start + r >= pc.cap) {  // the row lives in an overflow page
        const int o = start + r - pc.cap;
        grow = (int64_t)((o >> 6) == pg0 ? page0 : page1) * 64 + (o & 63);
        kp = a.k_ovf;
        vp = a.v_ovf;
      }
      const int64_t goff = grow * kRowBytes + c * 16;
      const uint32_t so = tile_off(r, c);
      if (ok && r == new_r && pc.new_row >= 0) {  // only inside the tile's valid rows (never in one of the np tiles)
        // the decoded token's row: attend to it from k_new / v_new and store it in the pool
        const size_t noff = (size_t)pc.seg * kRowBytes + c * 16;
        cp_async16(sb + so, a.k_new + noff, 16);
        cp_async16(sb + kTile * kRowBytes + so, a.v_new + noff, 16);
        *reinterpret_cast<uint4*>(kp + goff) = *reinterpret_cast<const uint4*>(a.k_new + noff);
        *reinterpret_cast<uint4*>(vp + goff) = *reinterpret_cast<const uint4*>(a.v_new + noff);
      } else {
        cp_async16(sb + so, kp + goff, ok);
        cp_async16(sb + kTile * kRowBytes + so, vp + goff, ok);
      }
    }
  };
  // indexed variant: the list entries of this thread's 8 rows of the producer's next tile, fetched one tile
  // ahead (right after the previous tile was issued) so that their latency is off the issue path
  auto load_idx = [&]() {
    if (kIndexed && p_item < item_end && pc.indexed) {
      int start, rows_left;
      tile_rows(pc, p_tile, start, rows_left);
      const int32_t* src = a.idx + (int64_t)pc.seg * a.idx_stride + start;
#pragma unroll
      for (int i = 0; i < (kTile * 16) / kDecodeThreads; ++i) {
        const int r = (tid + i * kDecodeThreads) >> 4;
        ix[i] = r < rows_left ? __ldg(src + r) : 0;
      }
    }
  };
  auto issue_q = [&](int ordinal, int seg) {  // the group's G query rows; heads >= G are zero-filled
    const uint32_t qb = s_q + (ordinal % kStages) * kQSlotBytes;
    const int b = seg / a.Hkv, h = seg % a.Hkv;
    const int r = tid >> 4, c = tid & 15;  // 128 threads = 8 rows x 16 chunks
    const int ok = r < a.G ? 16 : 0;
    const uint16_t* src = a.q + ((int64_t)b * a.Hq + h * a.G + (ok ? r : 0)) * kD + c * 8;
    cp_async16(qb + r * kRowBytes + c * 16, src, ok);
  };
  // The producer moves on to the next piece: its cursor comes from the values requested one piece ahead, is handed
  // to the consumer through a small ring in shared memory (the consumer gets there at least one barrier later and
  // at most kStages - 1 tiles, hence pieces, behind), and the piece after it is requested.
  NextItem nxt;
  auto next_item = [&]() {
    p_tile = 0;
    if (++p_item < item_end) {
      pc = make_cursor<kMode>(a, nxt);
      if (tid == 0) s_ring[(p_item - item_begin) & 3] = pc;
      if (p_item + 1 < item_end) fetch_next<kMode>(a, p_item + 1, pc.seg + 1, nxt);
    }
  };
  auto advance = [&]() {  // after a tile was issued; the plan-time tiles need no look at the live length
    ++p_seq;
    if (++p_tile >= pc.np && p_tile >= item_tiles(pc)) next_item();
    load_idx();
  };
  auto issue = [&]() {  // one tile (with the item's queries if it is the item's first) = one commit group
    if (p_item < item_end) {
      issue_tile();
      if (p_tile == 0 && p_item != item_begin) issue_q(p_item - item_begin, pc.seg);
      advance();
    }
    cp_async_commit();
  };

  // Rows that were valid when the plan was built are older than anything the previous kernel of the stream
  // may still be writing (an append writes behind them): the first tiles are requested before the wait.
  // (not in the indexed variant: its rows are named by the index list, which the preceding kernel writes)
  const int pre = kIndexed ? 0 : min(kStages - 1, pc.np);
  for (int s = 0; s < pre; ++s) {
    issue_tile();
    ++p_seq;
    ++p_tile;
    cp_async_commit();
  }
  pdl_wait();  // from here on: lengths, queries and rows written by earlier kernels
  live_cursor<kMode>(a, pc);
  const ItemCursor first = pc;
  if (item_begin + 1 < item_end) fetch_next<kMode>(a, item_begin + 1, pc.seg + 1, nxt);
  issue_q(0, pc.seg);
  if (p_tile >= pc.np && p_tile >= item_tiles(pc)) next_item();
  load_idx();
  for (int s = pre; s < kStages - 1; ++s) issue();
  if (pre == kStages - 1) cp_async_commit();  // the queries of the first item form a group of their own

  int seq = 0;
  for (int c_item = item_begin; c_item < item_end; ++c_item) {
    const ItemCursor cc = c_item == item_begin ? first : s_ring[(c_item - item_begin) & 3];
    uint32_t qf[8][2];
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    for (int tile = 0; tile < cc.np || tile < item_tiles(cc); ++tile, ++seq) {
      if (seq == 0)
        cp_async_wait<0>();  // first tile and the first item's queries (whichever group they are in)
      else
        cp_async_wait<kStages - 2>();
      __syncthreads();
      issue();
      if (tile == 0) {
        const uint8_t* qs = smem + kStages * kStageBytes + ((c_item - item_begin) % kStages) * kQSlotBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          qf[ks][0] = *reinterpret_cast<const uint32_t*>(qs + g * kRowBytes + (ks * 16 + 2 * t) * 2);
          qf[ks][1] = *reinterpret_cast<const uint32_t*>(qs + g * kRowBytes + (ks * 16 + 8 + 2 * t) * 2);
        }
      }
      int tstart, nvalid;  // valid rows of this tile (may exceed kTile)
      tile_rows(cc, tile, tstart, nvalid);
      const int row0 = warp * 16;
      if (row0 >= nvalid) continue;  // warp-uniform: this warp's 16 rows are all padding
      const uint32_t kb = s_stage + (seq % kStages) * kStageBytes;
      const uint32_t vb = kb + kTile * kRowBytes;

      // ---- S[16 tokens x 8 heads] = K_tile . Q^T
      float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb2[4] = {0.f, 0.f, 0.f, 0.f};
      {
        const int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int cadd = lane >> 4;
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
          uint32_t af[4];
          ldmatrix_x4(af, kb + tile_off(r, ks * 2 + cadd));
          mma_bf16_16816(sa, af, qf[ks][0], qf[ks][1]);
          ldmatrix_x4(af, kb + tile_off(r, ks * 2 + 2 + cadd));
          mma_bf16_16816(sb2, af, qf[ks + 1][0], qf[ks + 1][1]);
        }
      }
      // x0: (token g, head 2t)  x1: (token g, head 2t+1)  x2: (token g+8, head 2t)  x3: (token g+8, head 2t+1)
      const bool v_lo = row0 + g < nvalid, v_hi = row0 + g + 8 < nvalid;
      const float x0 = v_lo ? (sa[0] + sb2[0]) * a.scale_log2 : -INFINITY;
      const float x1 = v_lo ? (sa[1] + sb2[1]) * a.scale_log2 : -INFINITY;
      const float x2 = v_hi ? (sa[2] + sb2[2]) * a.scale_log2 : -INFINITY;
      const float x3 = v_hi ? (sa[3] + sb2[3]) * a.scale_log2 : -INFINITY;
      float mx0 = fmaxf(x0, x2), mx1 = fmaxf(x1, x3);
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
      }
      // row 0 of the warp's block is valid here, so the new maxima are finite
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);  // exp2(-inf) = 0 on the first block
      m0 = mn0;
      m1 = mn1;
      const float p0 = fast_exp2(x0 - mn0), p1 = fast_exp2(x1 - mn1);
      const float p2 = fast_exp2(x2 - mn0), p3 = fast_exp2(x3 - mn1);
      l0 = l0 * al0 + p0 + p2;
      l1 = l1 * al1 + p1 + p3;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        o[i][0] *= al0;
        o[i][1] *= al1;
        o[i][2] *= al0;
        o[i][3] *= al1;
      }
      // P as bf16 hi + lo, transposed into the B-operand layout (k = token, n = head)
      const float h0 = bf16_round(p0), h1 = bf16_round(p1), h2 = bf16_round(p2), h3 = bf16_round(p3);
      const uint32_t bh0 = movmatrix_trans(pack_bf16(h0, h1));
      const uint32_t bh1 = movmatrix_trans(pack_bf16(h2, h3));
      const uint32_t bl0 = movmatrix_trans(pack_bf16(p0 - h0, p1 - h1));
      const uint32_t bl1 = movmatrix_trans(pack_bf16(p2 - h2, p3 - h3));
      // ---- O^T[128 d x 8 heads] += V_tile^T . P
      {
        const int r = row0 + (lane & 7) + ((lane >> 4) & 1) * 8;
        const int cadd = (lane >> 3) & 1;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          uint32_t af[4];
          ldmatrix_x4_trans(af, vb + tile_off(r, mt * 2 + cadd));
          mma_bf16_16816(o[mt], af, bh0, bh1);
          mma_bf16_16816(o[mt], af, bl0, bl1);
        }
      }
    }

    // ---- end of the piece: finish the row sums, merge the four warps, write the result
    if (cc.new_row >= 0 && tid == 0) a.seg_len[cc.seg] = cc.live;  // fused append: the segment has grown by one row
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
      l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
    }
#pragma unroll
    for (int lvl = 0; lvl < 2; ++lvl) {
      const int stride = 1 << lvl;                       // 1, then 2
      const bool writer = (warp & (2 * stride - 1)) == stride;  // level 0: warps 1,3; level 1: warp 2
      const bool reader = (warp & (2 * stride - 1)) == 0;       // level 0: warps 0,2; level 1: warp 0
      float* mb = merge + (warp >> (lvl + 1)) * (kMergeRegs * 32);
      if (writer) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) mb[(i * 4 + j) * 32 + lane] = o[i][j];
        mb[32 * 32 + lane] = m0;
        mb[33 * 32 + lane] = m1;
        mb[34 * 32 + lane] = l0;
        mb[35 * 32 + lane] = l1;
      }
      __syncthreads();
      if (reader) {
        const float om0 = mb[32 * 32 + lane], om1 = mb[33 * 32 + lane];
        const float ol0 = mb[34 * 32 + lane], ol1 = mb[35 * 32 + lane];
        const float mn0 = fmaxf(m0, om0), mn1 = fmaxf(m1, om1);
        const float a0 = (m0 == -INFINITY) ? 0.f : fast_exp2(m0 - mn0);
        const float b0 = (om0 == -INFINITY) ? 0.f : fast_exp2(om0 - mn0);
        const float a1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - mn1);
        const float b1 = (om1 == -INFINITY) ? 0.f : fast_exp2(om1 - mn1);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          o[i][0] = o[i][0] * a0 + mb[(i * 4 + 0) * 32 + lane] * b0;
          o[i][1] = o[i][1] * a1 + mb[(i * 4 + 1) * 32 + lane] * b1;
          o[i][2] = o[i][2] * a0 + mb[(i * 4 + 2) * 32 + lane] * b0;
          o[i][3] = o[i][3] * a1 + mb[(i * 4 + 3) * 32 + lane] * b1;
        }
        l0 = l0 * a0 + ol0 * b0;
        l1 = l1 * a1 + ol1 * b1;
        m0 = mn0;
        m1 = mn1;
      }
      if (lvl == 0) __syncthreads();  // slot 0 is rewritten by warp 2 at the next level
    }
    if (warp == 0) {
      // stage the normalised [8 heads x 128] block in shared memory, then write whole rows
      float* st = merge;  // slot 0: free again (its reader is this warp)
      const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        st[(2 * t) * kD + i * 16 + g] = o[i][0] * i0;
        st[(2 * t + 1) * kD + i * 16 + g] = o[i][1] * i1;
        st[(2 * t) * kD + i * 16 + g + 8] = o[i][2] * i0;
        st[(2 * t + 1) * kD + i * 16 + g + 8] = o[i][3] * i1;
      }
      __syncwarp();
      const float lse0 = l0 > 0.f ? m0 + log2f(l0) : -INFINITY;
      const float lse1 = l1 > 0.f ? m1 + log2f(l1) : -INFINITY;
      const int b = cc.seg / a.Hkv, h = cc.seg % a.Hkv;
      if (cc.slot >= 0) {
        float* po = a.part_o + (size_t)cc.slot * (kMaxG * kD);
        for (int hd = 0; hd < a.G; ++hd)
          reinterpret_cast<float4*>(po + hd * kD)[lane] = reinterpret_cast<const float4*>(st + hd * kD)[lane];
        if (g == 0) {
          if (2 * t < a.G) a.part_lse[(size_t)cc.slot * kMaxG + 2 * t] = lse0;
          if (2 * t + 1 < a.G) a.part_lse[(size_t)cc.slot * kMaxG + 2 * t + 1] = lse1;
        }
      } else {
        const size_t obase = ((size_t)b * a.Hq + (size_t)h * a.G) * kD;
        for (int hd = 0; hd < a.G; ++hd) {
          const float4 v = reinterpret_cast<const float4*>(st + hd * kD)[lane];
          if (a.out_fp32) {
            reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + obase + hd * kD)[lane] = v;
          } else {
            uint2 pk;
            pk.x = pack_bf16(v.x, v.y);
            pk.y = pack_bf16(v.z, v.w);
            reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.out) + obase + hd * kD)[lane] = pk;
          }
        }
        if (a.lse_out && g == 0) {
          const float ln2 = 0.6931471805599453f;
          if (2 * t < a.G) a.lse_out[(size_t)b * a.Hq + h * a.G + 2 * t] = lse0 * ln2;
          if (2 * t + 1 < a.G) a.lse_out[(size_t)b * a.Hq + h * a.G + 2 * t + 1] = lse1 * ln2;
        }
      }
    }
  }
  cp_async_wait<0>();
}

// ------------------------------------------------------------------------------------------
// Combine: merge the partials of every segment that was cut into several pieces
// ------------------------------------------------------------------------------------------
struct CombineArgs {
  const SegInfo* seg_info;
  const float* part_o;
  const float* part_lse;
  void* out;
  float* lse_out;
  int32_t Hq, Hkv, G, out_fp32;
};

// One CTA of 8 warps per (segment, query head of the group).  The kernel is a chain of dependent trips to
// memory, so it is arranged to have one: a warp loads the values and the LSEs of its eighth of the pieces at
// once (a lane owns four consecutive d, a piece is one 512-byte row per warp-load) and merges them under a
// running maximum of its own; the warps are then merged through shared memory in a fixed order.
constexpr int kCombineWarps = 8;
constexpr int kCombineUnroll = 16;
__global__ void __launch_bounds__(kCombineWarps * 32) decode_combine_kernel(const CombineArgs a) {
  const int seg = blockIdx.x, hd = blockIdx.y;
  pdl_launch_dependents();
  const SegInfo si = a.seg_info[seg];  // plan data: older than the previous kernel
  pdl_wait();
  if (si.n_pieces <= 1) return;  // written directly by the attention kernel
  __shared__ float4 s_acc[kCombineWarps][32];
  __shared__ float s_w[kCombineWarps];
  __shared__ float s_m[kCombineWarps];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = si.n_pieces;
  const float* lse = a.part_lse + (size_t)si.slot_begin * kMaxG + hd;
  // One trip to memory: a warp loads the values and the LSEs of its pieces together (16 pieces in flight: a single pass for up to 128 pieces) and merges
  // them with a running maximum of its own; the 8 warps are then merged through shared memory.
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float wsum = 0.f, mw = -INFINITY;
  {
    const float* po = a.part_o + ((size_t)si.slot_begin * kMaxG + hd) * kD + lane * 4;
    for (int p0 = warp; p0 < n; p0 += kCombineWarps * kCombineUnroll) {
      float4 v[kCombineUnroll];
      float w[kCombineUnroll];
#pragma unroll
      for (int u = 0; u < kCombineUnroll; ++u) {
        const int p = p0 + u * kCombineWarps;
        const bool ok = p < n;
        v[u] = ok ? *reinterpret_cast<const float4*>(po + (size_t)p * (kMaxG * kD)) : make_float4(0.f, 0.f, 0.f, 0.f);
        w[u] = ok ? lse[(size_t)p * kMaxG] : -INFINITY;
      }
      float mx = mw;
#pragma unroll
      for (int u = 0; u < kCombineUnroll; ++u) mx = fmaxf(mx, w[u]);
      if (mx > -INFINITY) {
        const float sc = exp2f(mw - mx);  // 0 on the first pass (mw = -inf)
        acc.x *= sc;
        acc.y *= sc;
        acc.z *= sc;
        acc.w *= sc;
        wsum *= sc;
        mw = mx;
#pragma unroll
        for (int u = 0; u < kCombineUnroll; ++u) {
          const float e = exp2f(w[u] - mx);  // an empty piece (LSE -inf) weighs 0
          acc.x += e * v[u].x;
          acc.y += e * v[u].y;
          acc.z += e * v[u].z;
          acc.w += e * v[u].w;
          wsum += e;
        }
      }
    }
  }
  s_acc[warp][lane] = acc;
  if (lane == 0) {
    s_w[warp] = wsum;
    s_m[warp] = mw;
  }
  __syncthreads();
  if (warp == 0) {
    float M = -INFINITY;
#pragma unroll
    for (int wv = 0; wv < kCombineWarps; ++wv) M = fmaxf(M, s_m[wv]);
    float W = 0.f;
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int wv = 0; wv < kCombineWarps; ++wv) {
      const float f = s_m[wv] > -INFINITY ? exp2f(s_m[wv] - M) : 0.f;
      W += f * s_w[wv];
      r.x += f * s_acc[wv][lane].x;
      r.y += f * s_acc[wv][lane].y;
      r.z += f * s_acc[wv][lane].z;
      r.w += f * s_acc[wv][lane].w;
    }
    const float inv = W > 0.f ? 1.f / W : 0.f;
    r.x *= inv;
    r.y *= inv;
    r.z *= inv;
    r.w *= inv;
    const int b = seg / a.Hkv, h = seg % a.Hkv;
    const size_t obase = ((size_t)b * a.Hq + (size_t)h * a.G + hd) * kD;
    if (a.out_fp32) {
      reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + obase)[lane] = r;
    } else {
      uint2 pk;
      pk.x = pack_bf16(r.x, r.y);
      pk.y = pack_bf16(r.z, r.w);
      reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.out) + obase)[lane] = pk;
    }
    if (a.lse_out && lane == 0)
      a.lse_out[(size_t)b * a.Hq + h * a.G + hd] = W > 0.f ? (M + log2f(W)) * 0.6931471805599453f : -INFINITY;
  }
}

}  // namespace catekv

using namespace catekv;

extern "C" int catekv_decode_num_ctas(void) {
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return CATEKV_ERR_CUDA;
  cudaError_t e = cudaFuncSetAttribute(decode_partial_kernel<kModePlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem);
  if (e != cudaSuccess) { set_cuda_error(e); return CATEKV_ERR_CUDA; }
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) { set_cuda_error(e); return CATEKV_ERR_CUDA; }
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_partial_kernel<kModePlain>, kDecodeThreads, kDecodeSmem);
  if (e != cudaSuccess) { set_cuda_error(e); return CATEKV_ERR_CUDA; }
  if (per_sm < 1) per_sm = 1;
  return sms * per_sm;
}

// phases: 1 = attention partials, 2 = combine, 3 = both
struct IndexList {  // indexed attention: see DecodeArgs
  const int32_t* idx;
  int64_t idx_stride;
  const int32_t* sel_len;
};

static int decode_launch(int phases, const catekv_cache* cache, const void* k_new, const void* v_new, const void* q,
                         int32_t Hq, float sm_scale, void* out,
                         int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                         size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream,
                         const IndexList* il = nullptr) {
  int rc = check_cache(cache);
  if (rc) return rc;
  if (!q || !out || !plan_host || !plan_dev || !ws) return CATEKV_ERR_INVALID_ARG;
  if (Hq <= 0 || Hq % cache->Hkv != 0) return CATEKV_ERR_INVALID_ARG;
  const int G = Hq / cache->Hkv;
  if (G > kMaxG) return CATEKV_ERR_UNSUPPORTED;
  if (out_dtype != CATEKV_OUT_BF16 && out_dtype != CATEKV_OUT_FP32) return CATEKV_ERR_UNSUPPORTED;
  if (!(sm_scale >= 0.f) || isinf(sm_scale)) return CATEKV_ERR_INVALID_ARG;
  const PlanHeader* hdr = (const PlanHeader*)plan_host;
  const int n_segs = cache->B * cache->Hkv;
  if (plan_bytes < sizeof(PlanHeader) || hdr->magic != kPlanMagic || hdr->n_segs != n_segs || hdr->num_ctas <= 0 ||
      hdr->tile != kTile)
    return CATEKV_ERR_INVALID_ARG;
  const PlanLayout L = plan_layout(n_segs, hdr->num_ctas);
  if (plan_bytes < L.bytes) return CATEKV_ERR_WORKSPACE;
  size_t off_lse = 0;
  if (ws_bytes < ws_layout(n_segs, hdr->num_ctas, &off_lse)) return CATEKV_ERR_WORKSPACE;

  const uint8_t* pd = (const uint8_t*)plan_dev;
  cudaStream_t st = (cudaStream_t)stream;
  float* part_o = (float*)ws;
  float* part_lse = (float*)((uint8_t*)ws + off_lse);
  const int out_fp32 = out_dtype == CATEKV_OUT_FP32;
  if ((phases & 1) && hdr->n_items > 0) {
    static std::atomic<bool> attr_set[64];
    int dev = 0;
    CATEKV_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
      CATEKV_CUDA_TRY(cudaFuncSetAttribute(decode_partial_kernel<kModePlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem));
      CATEKV_CUDA_TRY(cudaFuncSetAttribute(decode_partial_kernel<kModeIndexed>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem));
      CATEKV_CUDA_TRY(cudaFuncSetAttribute(decode_partial_kernel<kModePaged>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem));
      if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
    DecodeArgs a;
    a.k_pool = (uint8_t*)cache->k_pool;
    a.v_pool = (uint8_t*)cache->v_pool;
    a.k_new = (const uint8_t*)k_new;
    a.v_new = (const uint8_t*)v_new;
    a.seg_off = cache->seg_off_dev;
    a.seg_len = cache->seg_len_dev;
    a.q = (const uint16_t*)q;
    a.Hq = Hq;
    a.Hkv = cache->Hkv;
    a.G = G;
    a.scale_log2 = (sm_scale == 0.f ? 1.0f / sqrtf((float)kD) : sm_scale) * 1.4426950408889634f;
    a.ctas = (const CtaHeader*)(pd + L.off_cta);
    a.items = (const WorkItem*)(pd + L.off_items);
    a.part_o = part_o;
    a.part_lse = part_lse;
    a.out = out;
    a.out_fp32 = out_fp32;
    a.lse_out = lse_out;
    a.idx = il ? il->idx : nullptr;
    a.idx_stride = il ? il->idx_stride : 0;
    a.sel_len = il ? il->sel_len : nullptr;
    const PageArgs pg = page_args(cache);
    a.k_ovf = pg.k_ovf;
    a.v_ovf = pg.v_ovf;
    a.page_table = pg.table;
    a.max_pages = pg.max_pages;
    a.n_pages = cache->pages ? cache->pages->n_pages : 0;
    a.chk = checked_status_ptr();
    if (il)
      CATEKV_CUDA_TRY(launch_pdl(decode_partial_kernel<kModeIndexed>, dim3(hdr->num_ctas), dim3(kDecodeThreads), kDecodeSmem, st, a));
    else if (cache->pages)
      CATEKV_CUDA_TRY(launch_pdl(decode_partial_kernel<kModePaged>, dim3(hdr->num_ctas), dim3(kDecodeThreads), kDecodeSmem, st, a));
    else
      CATEKV_CUDA_TRY(launch_pdl(decode_partial_kernel<kModePlain>, dim3(hdr->num_ctas), dim3(kDecodeThreads), kDecodeSmem, st, a));
  }
  if ((phases & 2) && hdr->n_slots > 0) {
    CombineArgs ca;
    ca.seg_info = (const SegInfo*)(pd + L.off_seg);
    ca.part_o = part_o;
    ca.part_lse = part_lse;
    ca.out = out;
    ca.lse_out = lse_out;
    ca.Hq = Hq;
    ca.Hkv = cache->Hkv;
    ca.G = G;
    ca.out_fp32 = out_fp32;
    CATEKV_CUDA_TRY(launch_pdl(decode_combine_kernel, dim3(n_segs, G), dim3(kCombineWarps * 32), 0, st, ca));
  }
  return CATEKV_OK;
}

extern "C" int catekv_decode_attn(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                                  int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                                  size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  return decode_launch(3, cache, nullptr, nullptr, q, Hq, sm_scale, out, out_dtype, lse_out, plan_host, plan_dev, plan_bytes, ws,
                       ws_bytes, stream);
}

extern "C" int catekv_decode_attn_indexed(const catekv_cache* cache, const int32_t* idx, int64_t idx_stride,
                                          const int32_t* sel_len, const void* q, int32_t Hq, float sm_scale, void* out,
                                          int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                                          size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  if (!idx || !sel_len || idx_stride < 0) return CATEKV_ERR_INVALID_ARG;
  if (cache && cache->pages) return CATEKV_ERR_UNSUPPORTED;
  const IndexList il = {idx, idx_stride, sel_len};
  return decode_launch(3, cache, nullptr, nullptr, q, Hq, sm_scale, out, out_dtype, lse_out, plan_host, plan_dev, plan_bytes, ws,
                       ws_bytes, stream, &il);
}

extern "C" int catekv_decode_partials(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                                      int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                                      size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  return decode_launch(1, cache, nullptr, nullptr, q, Hq, sm_scale, out, out_dtype, lse_out, plan_host, plan_dev, plan_bytes, ws,
                       ws_bytes, stream);
}

extern "C" int catekv_decode_combine(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale, void* out,
                                     int32_t out_dtype, float* lse_out, const void* plan_host, const void* plan_dev,
                                     size_t plan_bytes, void* ws, size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  return decode_launch(2, cache, nullptr, nullptr, q, Hq, sm_scale, out, out_dtype, lse_out, plan_host, plan_dev, plan_bytes, ws,
                       ws_bytes, stream);
}

extern "C" int catekv_append_decode_attn(catekv_cache* cache, const void* k_new, const void* v_new, const void* q,
                                         int32_t Hq, float sm_scale, void* out, int32_t out_dtype, float* lse_out,
                                         const void* plan_host, const void* plan_dev, size_t plan_bytes, void* ws,
                                         size_t ws_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  int rc = check_cache(cache);
  if (rc) return rc;
  if (!k_new || !v_new) return CATEKV_ERR_INVALID_ARG;
  // the kernel places the appended row by the plan: the host lengths the plan was built from must be exact
  if (cache->reserved) return CATEKV_ERR_INVALID_ARG;
  const int n = cache->B * cache->Hkv;
  for (int s = 0; s < n; ++s) {
    if (cache->seg_len[s] < 0) return CATEKV_ERR_INVALID_ARG;
    if (cache->seg_len[s] + 1 > seg_capacity(cache, s)) return CATEKV_ERR_CAPACITY;
  }
  // The appended row must lie behind every row the plan knows: the kernel requests plan-time tiles before it
  // may look at the lengths.  (catekv_decode_attn, without the append, also takes segments that have shrunk.)
  if (plan_host && plan_bytes >= sizeof(PlanHeader)) {
    const PlanHeader* hdr = (const PlanHeader*)plan_host;
    if (hdr->magic == kPlanMagic && hdr->n_segs == n && hdr->num_ctas > 0) {
      const PlanLayout L = plan_layout(n, hdr->num_ctas);
      if (plan_bytes >= L.bytes) {
        const SegInfo* si = (const SegInfo*)((const uint8_t*)plan_host + L.off_seg);
        for (int s = 0; s < n; ++s)
          if (cache->seg_len[s] < si[s].plan_len) return CATEKV_ERR_INVALID_ARG;
      }
    }
  }
  rc = decode_launch(3, cache, k_new, v_new, q, Hq, sm_scale, out, out_dtype, lse_out, plan_host, plan_dev,
                     plan_bytes, ws, ws_bytes, stream);
  if (rc) return rc;
  for (int s = 0; s < n; ++s) cache->seg_len[s] += 1;
  return CATEKV_OK;
}

// ------------------------------------------------------------------------------------------
// Decode attention without caller-provided scratch
// ------------------------------------------------------------------------------------------
// The split-KV partials of this variant live in a fixed array inside the library image instead of
// a caller workspace.  In host code the array's name only stands for the symbol; the address the
// kernels need is looked up once per device.
static __device__ __align__(256) unsigned char g_decode_noalloc_scratch[CATEKV_NOALLOC_SCRATCH_BYTES];

extern "C" int catekv_decode_attn_noalloc(const catekv_cache* cache, const void* q, int32_t Hq, float sm_scale,
                                          void* out, int32_t out_dtype, float* lse_out, const void* plan_host,
                                          const void* plan_dev, size_t plan_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  static std::atomic<void*> scratch_of_device[64];
  int dev = 0;
  CATEKV_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return CATEKV_ERR_UNSUPPORTED;
  void* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // first call on this device (which is current): resolve the device address of the array
    CATEKV_CUDA_TRY(cudaGetSymbolAddress(&scratch, g_decode_noalloc_scratch));
    if (!scratch) return CATEKV_ERR_CUDA;
    scratch_of_device[dev].store(scratch, std::memory_order_release);
  }
  // decode_launch checks the plan and returns CATEKV_ERR_WORKSPACE when the partials of this plan
  // (num_ctas + B*Hkv slots) do not fit the fixed array
  return decode_launch(3, cache, nullptr, nullptr, q, Hq, sm_scale, out, out_dtype, lse_out, plan_host, plan_dev, plan_bytes,
                       scratch, (size_t)CATEKV_NOALLOC_SCRATCH_BYTES, stream);
}
