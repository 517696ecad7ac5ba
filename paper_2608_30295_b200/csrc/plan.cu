// Work-balanced split-KV schedule of the decode attention (host only).
#include "decode.cuh"

using namespace catekv;

extern "C" size_t catekv_decode_plan_bytes(int32_t B, int32_t Hkv, int32_t num_ctas) {
  if (B <= 0 || Hkv <= 0 || num_ctas <= 0) return 0;
  return plan_layout(B * Hkv, num_ctas).bytes;
}

extern "C" size_t catekv_decode_workspace_bytes(int32_t B, int32_t Hkv, int32_t num_ctas) {
  if (B <= 0 || Hkv <= 0 || num_ctas <= 0) return 0;
  return ws_layout(B * Hkv, num_ctas, nullptr);
}

extern "C" int catekv_decode_plan(const catekv_cache* cache, int32_t num_ctas, void* plan_host, void* plan_dev,
                                  size_t plan_bytes, catekv_stream stream) {
  CATEKV_API_RANGE();
  int rc = check_cache(cache);
  if (rc) return rc;
  if (num_ctas <= 0 || !plan_host) return CATEKV_ERR_INVALID_ARG;
  const int n_segs = cache->B * cache->Hkv;
  const PlanLayout L = plan_layout(n_segs, num_ctas);
  if (plan_bytes < L.bytes) return CATEKV_ERR_WORKSPACE;
  // The CTA that owns the end of a segment does more than stream rows: its last tile also takes the rows appended
  // since the plan was built, it stores the appended row, and it finishes one piece and starts the next (merge of
  // the warps, output, the next group's queries) while nothing new is issued.  Every non-empty segment's end is
  // therefore charged kSegEndCharge rows, so that those CTAs get fewer plan-time rows and do not finish last.
  int64_t total = 0, charged = 0;
  for (int s = 0; s < n_segs; ++s) {
    if (cache->seg_len[s] < 0 || cache->seg_len[s] > seg_capacity(cache, s)) return CATEKV_ERR_INVALID_ARG;
    total += cache->seg_len[s];
    charged += cache->seg_len[s] + (cache->seg_len[s] > 0 ? kSegEndCharge : 0);
  }
  uint8_t* base = (uint8_t*)plan_host;
  memset(base, 0, L.bytes);
  PlanHeader* hdr = (PlanHeader*)base;
  CtaHeader* ctas = (CtaHeader*)(base + L.off_cta);
  WorkItem* items = (WorkItem*)(base + L.off_items);
  SegInfo* segs = (SegInfo*)(base + L.off_seg);

  // rows per CTA: an equal share of all (charged) rows, rounded up to the split alignment
  int64_t quota = (charged + num_ctas - 1) / num_ctas;
  quota = (quota + kSplitAlign - 1) / kSplitAlign * kSplitAlign;
  if (quota < kSplitAlign) quota = kSplitAlign;

  int n_items = 0, n_slots = 0, max_pieces = 1;
  int seg = 0;
  int32_t pos = 0;  // next unassigned row of `seg`
  int seg_first_item = 0;
  for (int c = 0; c < num_ctas; ++c) {
    ctas[c].item_begin = n_items;
    int64_t room = quota;
    while (seg < n_segs) {
      const int32_t len = cache->seg_len[seg];
      if (len == 0) {
        // an empty segment still gets one (direct) item, so that the plan stays valid once it grows
        items[n_items++] = WorkItem{seg, 0, 0, -1, (int64_t)cache->seg_off[seg], 1, cache->seg_cap[seg]};
        segs[seg] = SegInfo{0, 1, 0, 0};
        ++seg;
        seg_first_item = n_items;
        continue;
      }
      if (room <= 0) break;
      const int32_t take = (int32_t)((int64_t)(len - pos) < room ? (len - pos) : room);
      items[n_items++] = WorkItem{seg, pos, pos + take, 0, (int64_t)cache->seg_off[seg] + pos, 0, cache->seg_cap[seg]};
      pos += take;
      room -= take;
      if (pos == len) {
        // segment finished: fix up its pieces
        const int pieces = n_items - seg_first_item;
        items[n_items - 1].last = 1;  // the last piece follows the segment's current length
        if (pieces == 1) {
          items[seg_first_item].slot = -1;
          segs[seg] = SegInfo{0, 1, len, 0};
        } else {
          for (int i = 0; i < pieces; ++i) items[seg_first_item + i].slot = n_slots + i;
          segs[seg] = SegInfo{n_slots, pieces, len, 0};
          n_slots += pieces;
          max_pieces = pieces > max_pieces ? pieces : max_pieces;
        }
        ++seg;
        pos = 0;
        seg_first_item = n_items;
        room -= kSegEndCharge;
      }
    }
    ctas[c].item_end = n_items;
  }
  if (seg != n_segs) return CATEKV_ERR_INVALID_ARG;  // cannot happen: quota * num_ctas >= the charged rows
  for (int c = 0; c < num_ctas; ++c)
    if (ctas[c].item_begin < ctas[c].item_end) ctas[c].first = items[ctas[c].item_begin];
  hdr->magic = kPlanMagic;
  hdr->num_ctas = num_ctas;
  hdr->n_segs = n_segs;
  hdr->n_items = n_items;
  hdr->n_slots = n_slots;
  hdr->tile = kTile;
  hdr->total_rows = total;
  hdr->off_cta = (int32_t)L.off_cta;
  hdr->off_items = (int32_t)L.off_items;
  hdr->off_seg = (int32_t)L.off_seg;
  hdr->max_pieces = max_pieces;
  if (plan_dev)
    CATEKV_CUDA_TRY(cudaMemcpyAsync(plan_dev, plan_host, L.bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream));
  return CATEKV_OK;
}
