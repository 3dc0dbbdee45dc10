// Host planner of the grouped decode (shared-chunk batched decode).
//
// MEPIC makes requests alias the same physical pages for every block of a chunk but the first
// (Section 3.2.2).  A per-request decode reads such a page once per request; here the requests that
// alias a page are put in one group, so that a worker stages the page once and scores it against all
// of the group's query heads in one tensor-core tile (the shared-KV attention direction the paper's
// related-work section names as complementary to its cache layer).
//
// The planner only regroups block-table entries.  Every (request, entry) pair lands in exactly one
// item: pages with the same set of users are split into groups of at most R requests; what is left
// over (pages with one user, a set's remainder of one, a request's partly filled last page) goes to
// the request's own single-request item.  Items are laid on one line of (item, kv head, 16-token
// tile) triples which is cut into equal pieces, one per worker.
#include <algorithm>
#include <map>
#include <unordered_map>
#include <vector>

#include <cuda_runtime.h>

#include "mepic.h"
#include "mepic_internal.h"
#include "mepic_plan.h"

namespace {

struct Use { int32_t r, e; };

struct Item {
  std::vector<int32_t> req;                 // requests of the group (a request may appear twice)
  std::vector<std::vector<int32_t>> ent;    // per page of the item: entry index in each request's table
  int32_t tail_slot_start = -1;
};

int sm_count_or(int n_sms) {
  if (n_sms > 0) return n_sms;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

}  // namespace

extern "C" size_t mepic_decode_plan_max_ints(const mepic_config_t* cfg, int32_t batch, int32_t table_stride, int32_t n_sms) {
  if (!mepic_config_ok(cfg) || batch < 1 || table_stride < 1) return 0;
  const int sms = sm_count_or(n_sms);
  if (sms <= 0) { mepic_set_error("decode_plan: no CUDA device and no SM count given"); return 0; }
  const int R = plan_group_requests(cfg->n_q_heads / cfg->n_kv_heads);
  const size_t E = static_cast<size_t>(batch) * table_stride;     // every entry is one record of one item at most
  return kPlanHeaderInts + E * (kItemFixed + R) + E * (1 + R) + static_cast<size_t>(sms) * kPlanWarps * 3 +
         (batch + 1) + E + batch + E * cfg->n_kv_heads * R + static_cast<size_t>(batch) * cfg->n_kv_heads + 1;
}

extern "C" int32_t mepic_decode_plan_build(const mepic_config_t* cfg, const int32_t* page_ids, const int32_t* pos_base,
                                           const int32_t* kv_len, int32_t batch, int32_t table_stride, int32_t n_sms,
                                           int32_t* out_plan, size_t cap_ints, size_t* out_ints) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (!page_ids || !pos_base || !kv_len || !out_plan || !out_ints || batch < 1 || table_stride < 1) {
    mepic_set_error("decode_plan: bad argument"); return MEPIC_E_INVAL;
  }
  const int sms = sm_count_or(n_sms);
  if (sms <= 0) { mepic_set_error("decode_plan: no CUDA device and no SM count given"); return MEPIC_E_CUDA; }
  const int32_t P = cfg->page_size, Hkv = cfg->n_kv_heads;
  const int R = plan_group_requests(cfg->n_q_heads / Hkv);
  const int tpp = P / kPlanTile;

  // users of every page, in (request, entry) order; a request's partly filled last page stays private
  std::vector<int32_t> n_ent(batch);
  std::unordered_map<int32_t, std::vector<Use>> users;
  std::vector<int32_t> page_order;                       // pages in order of first appearance
  std::vector<std::vector<int32_t>> own(batch);          // entries of a request that no group takes
  for (int32_t r = 0; r < batch; ++r) {
    if (kv_len[r] < 1) { mepic_set_error("decode_plan: kv_len[%d] = %d < 1", r, kv_len[r]); return MEPIC_E_INVAL; }
    n_ent[r] = (kv_len[r] + P - 1) / P;
    if (n_ent[r] > table_stride) { mepic_set_error("decode_plan: request %d needs %d entries > stride", r, n_ent[r]); return MEPIC_E_INVAL; }
    for (int32_t e = 0; e < n_ent[r]; ++e) {
      const bool full = (e + 1) * P <= kv_len[r];
      if (!full) { own[r].push_back(e); continue; }
      const int32_t page = page_ids[static_cast<size_t>(r) * table_stride + e];
      auto it = users.find(page);
      if (it == users.end()) { page_order.push_back(page); it = users.emplace(page, std::vector<Use>()).first; }
      it->second.push_back(Use{r, e});
    }
  }

  // pages with the same user requests form a set; each set is cut into groups of R requests
  std::map<std::vector<int32_t>, size_t> item_of_group;
  std::vector<Item> shared_items;
  for (int32_t page : page_order) {
    const std::vector<Use>& u = users[page];
    if (u.size() == 1) { own[u[0].r].push_back(u[0].e); continue; }
    for (size_t at = 0; at < u.size(); at += R) {
      const size_t n = std::min<size_t>(R, u.size() - at);
      if (n == 1) { own[u[at].r].push_back(u[at].e); continue; }
      std::vector<int32_t> key(n), ent(n);
      for (size_t j = 0; j < n; ++j) { key[j] = u[at + j].r; ent[j] = u[at + j].e; }
      auto it = item_of_group.find(key);
      if (it == item_of_group.end()) {
        it = item_of_group.emplace(key, shared_items.size()).first;
        shared_items.emplace_back();
        shared_items.back().req = key;
      }
      shared_items[it->second].ent.push_back(ent);
    }
  }
  std::vector<Item> items;
  items.reserve(shared_items.size() + batch);
  for (Item& it : shared_items) items.push_back(std::move(it));
  for (int32_t r = 0; r < batch; ++r) {
    if (own[r].empty()) continue;
    std::sort(own[r].begin(), own[r].end());
    Item it;
    it.req = {r};
    for (int32_t e : own[r]) it.ent.push_back({e});
    if (own[r].back() == n_ent[r] - 1) it.tail_slot_start = (n_ent[r] - 1) * P;
    items.push_back(std::move(it));
  }

  // sizes and offsets
  size_t n_records = 0, n_req_items = 0;
  long long tiles_per_head = 0;
  for (const Item& it : items) { n_records += it.ent.size(); n_req_items += it.req.size(); tiles_per_head += static_cast<long long>(it.ent.size()) * tpp; }
  const long long total = tiles_per_head * Hkv;
  if (total >= (1ll << 31) || items.size() >= (1u << 27)) { mepic_set_error("decode_plan: batch too large for the plan's 32-bit fields"); return MEPIC_E_CAPACITY; }
  const int n_workers = sms * kPlanWarps;
  long long piece = (total + n_workers - 1) / n_workers;
  if (piece < kPlanMinPiece) piece = kPlanMinPiece;
  const size_t off_items = kPlanHeaderInts;
  const size_t off_records = off_items + items.size() * (kItemFixed + R);
  const size_t off_workers = off_records + n_records * (1 + R);
  const size_t off_req_off = off_workers + static_cast<size_t>(n_workers) * 3;
  const size_t off_req_items = off_req_off + batch + 1;
  const size_t off_req_ent = off_req_items + n_req_items;
  const size_t off_slot_base = off_req_ent + batch;
  const size_t off_part_off = off_slot_base + items.size() * Hkv * R;
  const size_t ints = off_part_off + static_cast<size_t>(batch) * Hkv + 1;
  *out_ints = ints;
  if (ints > cap_ints) { mepic_set_error("decode_plan: plan needs %zu ints, buffer holds %zu", ints, cap_ints); return MEPIC_E_CAPACITY; }

  int32_t* h = out_plan;
  h[kPhMagic] = kPlanMagic; h[kPhItems] = static_cast<int32_t>(items.size()); h[kPhWorkers] = n_workers;
  h[kPhPiece] = static_cast<int32_t>(piece); h[kPhTotal] = static_cast<int32_t>(total); h[kPhR] = R;
  h[kPhOffItems] = static_cast<int32_t>(off_items); h[kPhOffRecords] = static_cast<int32_t>(off_records);
  h[kPhOffWorkers] = static_cast<int32_t>(off_workers); h[kPhOffReqOff] = static_cast<int32_t>(off_req_off);
  h[kPhOffReqItems] = static_cast<int32_t>(off_req_items); h[kPhBatch] = batch; h[kPhRecords] = static_cast<int32_t>(n_records);
  h[kPhInts] = static_cast<int32_t>(ints); h[kPhOffReqEnt] = static_cast<int32_t>(off_req_ent); h[kPhPageSize] = P;
  h[kPhOffSlotBase] = static_cast<int32_t>(off_slot_base); h[kPhOffPartOff] = static_cast<int32_t>(off_part_off);
  h[kPhKvHeads] = Hkv;
  for (int k = kPhKvHeads + 1; k < kPlanHeaderInts; ++k) h[k] = 0;

  std::vector<std::vector<int32_t>> req_items(batch);
  int32_t rec = 0, tile_start = 0;
  for (size_t i = 0; i < items.size(); ++i) {
    const Item& it = items[i];
    int32_t* d = out_plan + off_items + i * (kItemFixed + R);
    d[kPiReq] = static_cast<int32_t>(it.req.size()); d[kPiRecOff] = rec; d[kPiEnt] = static_cast<int32_t>(it.ent.size());
    d[kPiTail] = it.tail_slot_start; d[kPiTileStart] = tile_start;
    for (int j = 0; j < R; ++j) d[kPiReqIds + j] = j < static_cast<int>(it.req.size()) ? it.req[j] : -1;
    for (size_t j = 0; j < it.req.size(); ++j) req_items[it.req[j]].push_back(static_cast<int32_t>(i) * 16 + static_cast<int32_t>(j));
    for (const std::vector<int32_t>& ent : it.ent) {
      int32_t* q = out_plan + off_records + static_cast<size_t>(rec) * (1 + R);
      q[0] = page_ids[static_cast<size_t>(it.req[0]) * table_stride + ent[0]];
      for (int j = 0; j < R; ++j)
        q[1 + j] = j < static_cast<int>(ent.size()) ? pos_base[static_cast<size_t>(it.req[j]) * table_stride + ent[j]] : 0;
      ++rec;
    }
    tile_start += static_cast<int32_t>(it.ent.size()) * tpp;
  }
  // where each worker's piece begins
  {
    size_t i = 0;
    for (int w = 0; w < n_workers; ++w) {
      int32_t* d = out_plan + off_workers + static_cast<size_t>(w) * 3;
      const long long x = static_cast<long long>(w) * piece;
      if (x >= total) { d[0] = static_cast<int32_t>(items.size()); d[1] = 0; d[2] = 0; continue; }
      while (true) {
        const long long nt = static_cast<long long>(items[i].ent.size()) * tpp;
        const long long start = static_cast<long long>(out_plan[off_items + i * (kItemFixed + R) + kPiTileStart]) * Hkv;
        if (x < start + nt * Hkv) {
          d[0] = static_cast<int32_t>(i); d[1] = static_cast<int32_t>((x - start) / nt); d[2] = static_cast<int32_t>((x - start) % nt);
          break;
        }
        ++i;
      }
    }
  }
  int32_t at = 0;
  for (int32_t r = 0; r < batch; ++r) {
    out_plan[off_req_off + r] = at;
    for (int32_t v : req_items[r]) out_plan[off_req_items + at++] = v;
    out_plan[off_req_ent + r] = n_ent[r];
  }
  out_plan[off_req_off + batch] = at;

  // partial slots: a unit (item, kv head) is overlapped by the pieces w_first..w_last of the line; each of its rows gets
  // one slot per piece, and the slots of a (request, kv head) pair are contiguous so that the merge reads one run
  std::vector<long long> count(static_cast<size_t>(batch) * Hkv + 1, 0);
  auto pieces_of = [&](size_t i, int hd) {
    const long long nt = static_cast<long long>(items[i].ent.size()) * tpp;
    const long long start = static_cast<long long>(out_plan[off_items + i * (kItemFixed + R) + kPiTileStart]) * Hkv + hd * nt;
    return (start + nt - 1) / piece - start / piece + 1;
  };
  for (size_t i = 0; i < items.size(); ++i)
    for (int hd = 0; hd < Hkv; ++hd)
      for (int32_t r : items[i].req) count[static_cast<size_t>(r) * Hkv + hd] += pieces_of(i, hd);
  long long run = 0;
  for (size_t u = 0; u < static_cast<size_t>(batch) * Hkv; ++u) {
    out_plan[off_part_off + u] = static_cast<int32_t>(run);
    const long long c = count[u]; count[u] = run; run += c;
  }
  if (run >= (1ll << 31)) { mepic_set_error("decode_plan: too many partials for the plan's 32-bit fields"); return MEPIC_E_CAPACITY; }
  out_plan[off_part_off + static_cast<size_t>(batch) * Hkv] = static_cast<int32_t>(run);
  h[kPhSlots] = static_cast<int32_t>(run);
  for (size_t i = 0; i < items.size(); ++i)
    for (int hd = 0; hd < Hkv; ++hd) {
      const long long c = pieces_of(i, hd);
      for (int j = 0; j < R; ++j) {
        int32_t v = 0;
        if (j < static_cast<int>(items[i].req.size())) {
          long long& cur = count[static_cast<size_t>(items[i].req[j]) * Hkv + hd];
          v = static_cast<int32_t>(cur); cur += c;
        }
        out_plan[off_slot_base + (i * Hkv + hd) * R + j] = v;
      }
    }
  return MEPIC_OK;
}
