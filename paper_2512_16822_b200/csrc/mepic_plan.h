// Layout of the grouped-decode plan: one flat int32 buffer written by
// mepic_decode_plan_build on the host and read by the grouped decode kernels on
// the device (not part of the ABI: callers treat the buffer as opaque).
//
//   header   [kPlanHeaderInts]
//   items    [n_items][kItemFixed + R]   {n_req, rec_off, n_ent, tail_slot_start, tile_start, req[R]}
//   records  [n_records][1 + R]          {page_id, pos_base[R]}   one per page of an item
//   workers  [n_workers][3]              (item, kv head, tile) where each worker's piece of the line begins
//   req_off  [batch + 1]                 CSR over req_items
//   req_items[...]                       item * 16 + j for every (item, row-request j) a request takes part in
//   req_ent  [batch]                     table entries each request had when the plan was built
//   slot_base[n_items][n_kv_heads][R]    first partial slot of (item, kv head, row-request): the worker whose piece is
//                                        the k-th to overlap the unit writes slot_base + k
//   part_off [batch * n_kv_heads + 1]    the partial slots of (request, kv head) are part_off[u] .. part_off[u+1]-1
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
  kPhOffSlotBase, kPhOffPartOff, kPhSlots, kPhKvHeads
};
enum PlanItem { kPiReq = 0, kPiRecOff, kPiEnt, kPiTail, kPiTileStart, kPiReqIds };

constexpr int kPlanTile = 16;        // tokens per tile
constexpr int kPlanMinPiece = 4;     // shortest piece of the line a worker gets
constexpr int kPlanWarps = 8;        // workers per SM

// Requests whose heads share the 16 rows of one tensor-core tile.
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int plan_group_requests(int group_size) { return 16 / group_size < 8 ? 16 / group_size : 8; }

#endif
