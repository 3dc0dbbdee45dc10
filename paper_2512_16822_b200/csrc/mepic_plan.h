// Layout of the grouped-decode plan: one flat int32 buffer written by
// mepic_decode_plan_build on the host and read by the grouped decode kernels on
// the device (not part of the ABI: callers treat the buffer as opaque).
//
//   header   [kPlanHeaderInts]
//   items    [n_items][kItemFixed + R]   {n_req, rec_off, n_ent, tail_slot_start, tile_start, req[R]}
//   workers  [n_workers][3]              (item, kv head, tile) where each worker's piece of the line begins
//   req_off  [batch + 1]                 CSR over req_items
//   req_items[...]                       item * 16 + j for every (item, row-request j) a request takes part in
//   req_ent  [batch]                     table entries each request has in the plan
//   own_item [batch]                     the request's single-request item (-1: it has none)
//   rec_cap  [n_items]                   records the item's run has room for (>= n_ent; only own items have slack)
//   slot_base[n_items][n_kv_heads][R]    first partial slot of (item, kv head, row-request): the worker whose piece is
//                                        the k-th to overlap the unit writes slot_base + k
//   part_off [batch * n_kv_heads + 1]    the partial slots of (request, kv head) are part_off[u] .. part_off[u+1]-1
//   records  [n_records][1 + R]          {page_id, pos_base[R]}   one per page of an item; an item's run is rec_off ..
//                                        rec_off + rec_cap - 1, of which the first n_ent are in use
//
// Everything before the records is re-derived when a request gains pages (mepic_decode_plan_patch); of the records
// only the runs of the requests that grew get new entries.  The records come last so that a patch changes one
// prefix of the buffer plus a short stretch of records.
//
// R = requests per group.  The line is item-major, then kv head, then tile; an item's tile count
// per head is n_ent * (page_size / 16); tile_start is the sum of the tile counts of the items
// before it.
#ifndef MEPIC_PLAN_H_
#define MEPIC_PLAN_H_

#include <stdint.h>

constexpr int32_t kPlanMagic = 0x4d504c31;   // "MPL1"
constexpr int kPlanHeaderInts = 24;
constexpr int kItemFixed = 5;
enum PlanHeader {
  kPhMagic = 0, kPhItems, kPhWorkers, kPhPiece, kPhTotal, kPhR, kPhOffItems, kPhOffRecords, kPhOffWorkers,
  kPhOffReqOff, kPhOffReqItems, kPhBatch, kPhRecords, kPhInts, kPhOffReqEnt, kPhPageSize,
  kPhOffSlotBase, kPhOffPartOff, kPhSlots, kPhKvHeads, kPhOffOwnItem, kPhOffRecCap
};
enum PlanItem { kPiReq = 0, kPiRecOff, kPiEnt, kPiTail, kPiTileStart, kPiReqIds };

constexpr int kPlanTile = 16;        // tokens per tile
constexpr int kPlanMinPiece = 4;     // shortest piece of the line a worker gets
constexpr int kPlanWarps = 8;        // workers per SM
constexpr int kPlanReservePages = 16; // table entries a request can gain before its plan has to be rebuilt

// Requests whose heads share the 16 rows of one tensor-core tile.
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int plan_group_requests(int group_size) { return 16 / group_size < 8 ? 16 / group_size : 8; }

#endif
