// Shared by the decode sources: the plan's layout in memory, cache checks, overflow pages.
#pragma once

#include <string.h>

#include "common.cuh"

namespace catekv {

// ------------------------------------------------------------------------------------------
// Plan (host)
// ------------------------------------------------------------------------------------------
constexpr uint32_t kPlanMagic = 0x43544B56u;  // "CTKV"
constexpr int kTile = 64;                     // rows per pipeline stage
constexpr int kDecodeWarps = kTile / 16;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kStages = 3;
constexpr int kSplitAlign = 16;               // CTA ranges are cut at multiples of this many rows
constexpr int kSegEndCharge = 256;            // rows charged to the CTA that owns a segment's end (see catekv_decode_plan)

struct PlanHeader {
  uint32_t magic;
  int32_t num_ctas;
  int32_t n_segs;
  int32_t n_items;
  int32_t n_slots;
  int32_t tile;
  int64_t total_rows;
  int32_t off_cta, off_items, off_seg;  // byte offsets of the three tables
  int32_t max_pieces;                   // most pieces any segment was cut into
};
static_assert(sizeof(PlanHeader) == 48, "plan header layout");

struct WorkItem {  // 32 bytes
  int32_t seg;
  int32_t t0;        // first row of the piece, relative to the segment
  int32_t t1;        // one past its last row at plan time
  int32_t slot;      // partial slot, or -1 when the piece is the whole segment (final output written directly)
  int64_t row_base;  // pool row of t0 (segment offset + t0)
  int32_t last;      // 1: last piece of its segment; it also covers rows [t1, current length)
  int32_t cap;       // capacity of the segment in the cache's own pools (rows from there on live in overflow pages)
};
static_assert(sizeof(WorkItem) == 32, "work item layout");
struct CtaHeader {  // 48 bytes: the CTA's item range and a copy of its first item (one load starts the stream)
  int32_t item_begin, item_end, reserved0, reserved1;
  WorkItem first;
};
static_assert(sizeof(CtaHeader) == 48, "cta header layout");
struct SegInfo {
  int32_t slot_begin;
  int32_t n_pieces;
  int32_t plan_len;  // rows the segment held when the plan was built
  int32_t reserved;
};

struct PlanLayout {
  size_t off_cta, off_items, off_seg, bytes;
  int n_items_cap;
};
static PlanLayout plan_layout(int n_segs, int num_ctas) {
  PlanLayout L;
  L.n_items_cap = num_ctas + n_segs;
  L.off_cta = sizeof(PlanHeader);
  L.off_items = align_up(L.off_cta + sizeof(CtaHeader) * (size_t)num_ctas, 32);
  L.off_seg = L.off_items + sizeof(WorkItem) * (size_t)L.n_items_cap;
  L.bytes = align_up(L.off_seg + sizeof(SegInfo) * (size_t)n_segs, 16);
  return L;
}

constexpr size_t kPartOBytes = (size_t)kMaxG * kD * sizeof(float);  // one partial: 8 heads x 128 floats
static size_t ws_layout(int n_segs, int num_ctas, size_t* off_lse) {
  size_t slots = (size_t)num_ctas + n_segs;
  size_t o = slots * kPartOBytes;
  if (off_lse) *off_lse = o;
  return o + slots * kMaxG * sizeof(float);
}

struct PageArgs {  // overflow pages of a cache (all null / 0 without pages)
  uint8_t* k_ovf;
  uint8_t* v_ovf;
  const int32_t* table;
  const int32_t* seg_cap;
  int32_t max_pages;
};
static PageArgs page_args(const catekv_cache* c) {
  PageArgs p = {nullptr, nullptr, nullptr, nullptr, 0};
  if (c->pages) {
    p.k_ovf = (uint8_t*)c->pages->k_ovf;
    p.v_ovf = (uint8_t*)c->pages->v_ovf;
    p.table = c->pages->table_dev;
    p.seg_cap = c->pages->seg_cap_dev;
    p.max_pages = c->pages->max_pages;
  }
  return p;
}

static int check_cache(const catekv_cache* c) {
  if (!c) return CATEKV_ERR_INVALID_ARG;
  if (c->B <= 0 || c->Hkv <= 0 || c->total_rows < 0) return CATEKV_ERR_INVALID_ARG;
  if (c->d != kD) return CATEKV_ERR_UNSUPPORTED;
  if (!c->k_pool || !c->v_pool || !c->seg_off_dev || !c->seg_len_dev || !c->seg_off || !c->seg_cap || !c->seg_len)
    return CATEKV_ERR_INVALID_ARG;
  if (c->pages) {
    const catekv_pages* p = c->pages;
    if (p->max_pages <= 0 || p->n_pages < 0 || p->next_free < 0 || p->next_free > p->n_pages) return CATEKV_ERR_INVALID_ARG;
    if (!p->k_ovf || !p->v_ovf || !p->table_dev || !p->table || !p->seg_pages || !p->seg_cap_dev) return CATEKV_ERR_INVALID_ARG;
  }
  return CATEKV_OK;
}
// rows segment s can hold: its own capacity plus the overflow pages it has been given
static inline int64_t seg_capacity(const catekv_cache* c, int s) {
  return (int64_t)c->seg_cap[s] + (c->pages ? (int64_t)c->pages->seg_pages[s] * CATEKV_PAGE_ROWS : 0);
}


}  // namespace catekv
