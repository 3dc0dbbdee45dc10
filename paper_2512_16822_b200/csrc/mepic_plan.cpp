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
#include <cstdint>
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
  std::vector<int32_t> ent;                 // per page of the item, n_req entries: the entry index in each request's table
  size_t pages() const { return ent.size() / req.size(); }
  int32_t tail_slot_start = -1;
};

int sm_count_or(int n_sms) {
  if (n_sms > 0) return n_sms;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

// Everything in the plan that follows from the items and their page counts: each item's place on the line, the cut of
// the line into pieces, where each worker's piece begins, and the partial slots.  Written at build time and again after
// a patch (a request that gained pages moves every later item along the line).
int32_t derive_plan(int32_t* plan) {
  int32_t* h = plan;
  const int n_items = h[kPhItems], R = h[kPhR], Hkv = h[kPhKvHeads], batch = h[kPhBatch], n_workers = h[kPhWorkers];
  const int tpp = h[kPhPageSize] / kPlanTile;
  const size_t stride = kItemFixed + R;
  int32_t* items = plan + h[kPhOffItems];
  long long tiles_per_head = 0;
  for (int i = 0; i < n_items; ++i) {
    if (tiles_per_head >= (1ll << 31)) break;
    items[i * stride + kPiTileStart] = static_cast<int32_t>(tiles_per_head);
    tiles_per_head += static_cast<long long>(items[i * stride + kPiEnt]) * tpp;
  }
  const long long total = tiles_per_head * Hkv;
  if (total >= (1ll << 31)) { mepic_set_error("decode_plan: batch too large for the plan's 32-bit fields"); return MEPIC_E_CAPACITY; }
  long long piece = (total + n_workers - 1) / n_workers;
  if (piece < kPlanMinPiece) piece = kPlanMinPiece;
  h[kPhPiece] = static_cast<int32_t>(piece); h[kPhTotal] = static_cast<int32_t>(total);
  // where each worker's piece begins
  {
    int i = 0;
    for (int w = 0; w < n_workers; ++w) {
      int32_t* d = plan + h[kPhOffWorkers] + static_cast<size_t>(w) * 3;
      const long long x = static_cast<long long>(w) * piece;
      if (x >= total) { d[0] = n_items; d[1] = 0; d[2] = 0; continue; }
      while (true) {
        const long long nt = static_cast<long long>(items[i * stride + kPiEnt]) * tpp;
        const long long start = static_cast<long long>(items[i * stride + kPiTileStart]) * Hkv;
        if (x < start + nt * Hkv) {
          d[0] = i; d[1] = static_cast<int32_t>((x - start) / nt); d[2] = static_cast<int32_t>((x - start) % nt);
          break;
        }
        ++i;
      }
    }
  }
  // partial slots: a unit (item, kv head) is overlapped by the pieces w_first..w_last of the line; each of its rows gets
  // one slot per piece, and the slots of a (request, kv head) pair are contiguous so that the merge reads one run
  std::vector<long long> count(static_cast<size_t>(batch) * Hkv + 1, 0);
  auto pieces_of = [&](int i, int hd) {
    const long long nt = static_cast<long long>(items[i * stride + kPiEnt]) * tpp;
    const long long start = static_cast<long long>(items[i * stride + kPiTileStart]) * Hkv + hd * nt;
    return (start + nt - 1) / piece - start / piece + 1;
  };
  for (int i = 0; i < n_items; ++i)
    for (int hd = 0; hd < Hkv; ++hd)
      for (int j = 0; j < items[i * stride + kPiReq]; ++j)
        count[static_cast<size_t>(items[i * stride + kPiReqIds + j]) * Hkv + hd] += pieces_of(i, hd);
  int32_t* part_off = plan + h[kPhOffPartOff];
  long long run = 0;
  for (size_t u = 0; u < static_cast<size_t>(batch) * Hkv; ++u) {
    part_off[u] = static_cast<int32_t>(run);
    const long long c = count[u]; count[u] = run; run += c;
  }
  if (run >= (1ll << 31)) { mepic_set_error("decode_plan: too many partials for the plan's 32-bit fields"); return MEPIC_E_CAPACITY; }
  part_off[static_cast<size_t>(batch) * Hkv] = static_cast<int32_t>(run);
  h[kPhSlots] = static_cast<int32_t>(run);
  int32_t* slot_base = plan + h[kPhOffSlotBase];
  for (int i = 0; i < n_items; ++i)
    for (int hd = 0; hd < Hkv; ++hd) {
      const long long c = pieces_of(i, hd);
      for (int j = 0; j < R; ++j) {
        int32_t v = 0;
        if (j < items[i * stride + kPiReq]) {
          long long& cur = count[static_cast<size_t>(items[i * stride + kPiReqIds + j]) * Hkv + hd];
          v = static_cast<int32_t>(cur); cur += c;
        }
        slot_base[(static_cast<size_t>(i) * Hkv + hd) * R + j] = v;
      }
    }
  return MEPIC_OK;
}

}  // namespace

extern "C" size_t mepic_decode_plan_max_ints(const mepic_config_t* cfg, int32_t batch, int32_t table_stride, int32_t n_sms) {
  if (!mepic_config_ok(cfg) || batch < 1 || table_stride < 1) return 0;
  const int sms = sm_count_or(n_sms);
  if (sms <= 0) { mepic_set_error("decode_plan: no CUDA device and no SM count given"); return 0; }
  const int R = plan_group_requests(cfg->n_q_heads / cfg->n_kv_heads);
  const size_t E = static_cast<size_t>(batch) * table_stride;     // every entry is one record of one item at most
  return kPlanHeaderInts + E * (kItemFixed + R) + (E + static_cast<size_t>(batch) * kPlanReservePages) * (1 + R) +
         static_cast<size_t>(sms) * kPlanWarps * 3 + (batch + 1) + E + batch + batch + E + E * cfg->n_kv_heads * R +
         static_cast<size_t>(batch) * cfg->n_kv_heads + 1;
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

  // users of every page, in (request, entry) order (a counting sort over page ids); a request's partly filled last
  // page stays private, and so does an entry whose page id is outside the pool (the kernel reports it)
  std::vector<int32_t> n_ent(batch);
  std::vector<std::vector<int32_t>> own(batch);          // entries of a request that no group takes
  const int32_t NP = cfg->num_pages;
  std::vector<int32_t> first_use(static_cast<size_t>(NP) + 1, 0);   // becomes the offset of each page's users
  size_t n_full = 0;
  for (int32_t r = 0; r < batch; ++r) {
    if (kv_len[r] < 1) { mepic_set_error("decode_plan: kv_len[%d] = %d < 1", r, kv_len[r]); return MEPIC_E_INVAL; }
    n_ent[r] = (kv_len[r] + P - 1) / P;
    if (n_ent[r] > table_stride) { mepic_set_error("decode_plan: request %d needs %d entries > stride", r, n_ent[r]); return MEPIC_E_INVAL; }
    const int32_t n_whole = kv_len[r] / P;                // entries 0 .. n_whole-1 are full pages
    for (int32_t e = 0; e < n_whole; ++e) {
      const int32_t page = page_ids[static_cast<size_t>(r) * table_stride + e];
      if (static_cast<uint32_t>(page) >= static_cast<uint32_t>(NP)) { own[r].push_back(e); continue; }
      ++first_use[page + 1]; ++n_full;
    }
    if (n_whole < n_ent[r]) own[r].push_back(n_whole);
  }
  for (int32_t pg = 0; pg < NP; ++pg) first_use[pg + 1] += first_use[pg];
  std::vector<Use> uses(n_full);
  std::vector<int32_t> page_order;                       // pages in order of first appearance
  {
    std::vector<int32_t> fill(first_use.begin(), first_use.end() - 1);
    for (int32_t r = 0; r < batch; ++r) {
      const int32_t n_whole = kv_len[r] / P;
      for (int32_t e = 0; e < n_whole; ++e) {
        const int32_t page = page_ids[static_cast<size_t>(r) * table_stride + e];
        if (static_cast<uint32_t>(page) >= static_cast<uint32_t>(NP)) continue;
        if (fill[page] == first_use[page]) page_order.push_back(page);
        uses[fill[page]++] = Use{r, e};
      }
    }
  }

  // pages with the same user requests form a set; each set is cut into groups of R requests; a group's pages
  // accumulate in one item (found through a hash of its request list, confirmed by comparing the list)
  std::unordered_map<uint64_t, std::vector<size_t>> item_of_group;
  std::vector<Item> shared_items;
  for (int32_t page : page_order) {
    const Use* u = uses.data() + first_use[page];
    const size_t n_users = static_cast<size_t>(first_use[page + 1] - first_use[page]);
    if (n_users == 1) { own[u[0].r].push_back(u[0].e); continue; }
    for (size_t at = 0; at < n_users; at += R) {
      const size_t n = std::min<size_t>(R, n_users - at);
      if (n == 1) { own[u[at].r].push_back(u[at].e); continue; }
      uint64_t hsh = 0xcbf29ce484222325ULL;
      for (size_t j = 0; j < n; ++j) { hsh ^= static_cast<uint64_t>(static_cast<uint32_t>(u[at + j].r)) + 1; hsh *= 0x100000001b3ULL; }
      std::vector<size_t>& cands = item_of_group[hsh];
      size_t idx = SIZE_MAX;
      for (size_t c : cands) {
        const std::vector<int32_t>& rq = shared_items[c].req;
        bool same = rq.size() == n;
        for (size_t j = 0; same && j < n; ++j) same = rq[j] == u[at + j].r;
        if (same) { idx = c; break; }
      }
      if (idx == SIZE_MAX) {
        idx = shared_items.size();
        cands.push_back(idx);
        shared_items.emplace_back();
        for (size_t j = 0; j < n; ++j) shared_items.back().req.push_back(u[at + j].r);
      }
      for (size_t j = 0; j < n; ++j) shared_items[idx].ent.push_back(u[at + j].e);
    }
  }
  std::vector<Item> items;
  items.reserve(shared_items.size() + batch);
  const size_t n_shared_items = shared_items.size();          // the items after these are the requests' own ones
  for (Item& it : shared_items) items.push_back(std::move(it));
  for (int32_t r = 0; r < batch; ++r) {
    if (own[r].empty()) continue;
    std::sort(own[r].begin(), own[r].end());
    Item it;
    it.req = {r};
    it.ent = own[r];
    if (own[r].back() == n_ent[r] - 1) it.tail_slot_start = (n_ent[r] - 1) * P;
    items.push_back(std::move(it));
  }

  // sizes and offsets.  The run of records of a request's own item has room for kPlanReservePages more pages (as far as
  // the table's stride lets the request grow), so that a page gain can be patched in (mepic_decode_plan_patch).
  std::vector<int32_t> cap(items.size());
  size_t n_records = 0, n_req_items = 0;
  for (size_t i = 0; i < items.size(); ++i) {
    const Item& it = items[i];
    int32_t c = static_cast<int32_t>(it.pages());
    if (i >= n_shared_items) c += std::min<int32_t>(kPlanReservePages, table_stride - n_ent[it.req[0]]);
    cap[i] = c;
    n_records += static_cast<size_t>(c); n_req_items += it.req.size();
  }
  if (items.size() >= (1u << 27)) { mepic_set_error("decode_plan: batch too large for the plan's 32-bit fields"); return MEPIC_E_CAPACITY; }
  const int n_workers = sms * kPlanWarps;
  const size_t off_items = kPlanHeaderInts;
  const size_t off_workers = off_items + items.size() * (kItemFixed + R);
  const size_t off_req_off = off_workers + static_cast<size_t>(n_workers) * 3;
  const size_t off_req_items = off_req_off + batch + 1;
  const size_t off_req_ent = off_req_items + n_req_items;
  const size_t off_own_item = off_req_ent + batch;
  const size_t off_rec_cap = off_own_item + batch;
  const size_t off_slot_base = off_rec_cap + items.size();
  const size_t off_part_off = off_slot_base + items.size() * Hkv * R;
  const size_t off_records = off_part_off + static_cast<size_t>(batch) * Hkv + 1;
  const size_t ints = off_records + n_records * (1 + R);
  *out_ints = ints;
  if (ints >= (1ull << 31)) { mepic_set_error("decode_plan: batch too large for the plan's 32-bit fields"); return MEPIC_E_CAPACITY; }
  if (ints > cap_ints) { mepic_set_error("decode_plan: plan needs %zu ints, buffer holds %zu", ints, cap_ints); return MEPIC_E_CAPACITY; }

  int32_t* h = out_plan;
  for (int k = 0; k < kPlanHeaderInts; ++k) h[k] = 0;
  h[kPhMagic] = kPlanMagic; h[kPhItems] = static_cast<int32_t>(items.size()); h[kPhWorkers] = n_workers; h[kPhR] = R;
  h[kPhOffItems] = static_cast<int32_t>(off_items); h[kPhOffRecords] = static_cast<int32_t>(off_records);
  h[kPhOffWorkers] = static_cast<int32_t>(off_workers); h[kPhOffReqOff] = static_cast<int32_t>(off_req_off);
  h[kPhOffReqItems] = static_cast<int32_t>(off_req_items); h[kPhBatch] = batch; h[kPhRecords] = static_cast<int32_t>(n_records);
  h[kPhInts] = static_cast<int32_t>(ints); h[kPhOffReqEnt] = static_cast<int32_t>(off_req_ent); h[kPhPageSize] = P;
  h[kPhOffSlotBase] = static_cast<int32_t>(off_slot_base); h[kPhOffPartOff] = static_cast<int32_t>(off_part_off);
  h[kPhKvHeads] = Hkv; h[kPhOffOwnItem] = static_cast<int32_t>(off_own_item); h[kPhOffRecCap] = static_cast<int32_t>(off_rec_cap);

  std::vector<std::vector<int32_t>> req_items(batch);
  for (int32_t r = 0; r < batch; ++r) out_plan[off_own_item + r] = -1;
  int32_t rec = 0;
  for (size_t i = 0; i < items.size(); ++i) {
    const Item& it = items[i];
    int32_t* d = out_plan + off_items + i * (kItemFixed + R);
    d[kPiReq] = static_cast<int32_t>(it.req.size()); d[kPiRecOff] = rec; d[kPiEnt] = static_cast<int32_t>(it.pages());
    d[kPiTail] = it.tail_slot_start; d[kPiTileStart] = 0;
    for (int j = 0; j < R; ++j) d[kPiReqIds + j] = j < static_cast<int>(it.req.size()) ? it.req[j] : -1;
    for (size_t j = 0; j < it.req.size(); ++j) req_items[it.req[j]].push_back(static_cast<int32_t>(i) * 16 + static_cast<int32_t>(j));
    if (i >= n_shared_items) out_plan[off_own_item + it.req[0]] = static_cast<int32_t>(i);
    out_plan[off_rec_cap + i] = cap[i];
    const int nr = static_cast<int>(it.req.size());
    for (int32_t k = 0; k < cap[i]; ++k) {
      int32_t* q = out_plan + off_records + static_cast<size_t>(rec + k) * (1 + R);
      for (int j = 0; j <= R; ++j) q[j] = 0;                      // (the unused part of a run reads as page 0)
      if (static_cast<size_t>(k) >= it.pages()) continue;
      const int32_t* ent = it.ent.data() + static_cast<size_t>(k) * nr;
      q[0] = page_ids[static_cast<size_t>(it.req[0]) * table_stride + ent[0]];
      for (int j = 0; j < nr; ++j) q[1 + j] = pos_base[static_cast<size_t>(it.req[j]) * table_stride + ent[j]];
    }
    rec += cap[i];
  }
  int32_t at = 0;
  for (int32_t r = 0; r < batch; ++r) {
    out_plan[off_req_off + r] = at;
    for (int32_t v : req_items[r]) out_plan[off_req_items + at++] = v;
    out_plan[off_req_ent + r] = n_ent[r];
  }
  out_plan[off_req_off + batch] = at;
  return derive_plan(out_plan);
}

// A request gained table entries since the plan was built (its kv_len moved into new pages): its own item takes the new
// pages, everything derived from the items' sizes is written again, and the caller uploads the two stretches that
// changed.  Host work is O(items + workers), not the regrouping of every table entry.
extern "C" int32_t mepic_decode_plan_patch(const mepic_config_t* cfg, int32_t* plan, const int32_t* page_ids, const int32_t* pos_base,
                                           const int32_t* kv_len, int32_t batch, int32_t table_stride,
                                           int64_t* out_ranges, int32_t* out_n_ranges) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (!plan || !page_ids || !pos_base || !kv_len || !out_ranges || !out_n_ranges || batch < 1 || table_stride < 1) {
    mepic_set_error("decode_plan_patch: bad argument"); return MEPIC_E_INVAL;
  }
  int32_t* h = plan;
  const int R = plan_group_requests(cfg->n_q_heads / cfg->n_kv_heads);
  if (h[kPhMagic] != kPlanMagic || h[kPhBatch] != batch || h[kPhR] != R || h[kPhPageSize] != cfg->page_size ||
      h[kPhKvHeads] != cfg->n_kv_heads) { mepic_set_error("decode_plan_patch: the plan was built for another config or batch"); return MEPIC_E_INVAL; }
  const int32_t P = cfg->page_size;
  const size_t stride = kItemFixed + R;
  int32_t* items = plan + h[kPhOffItems];
  int32_t* req_ent = plan + h[kPhOffReqEnt];
  const int32_t* own_item = plan + h[kPhOffOwnItem];
  const int32_t* rec_cap = plan + h[kPhOffRecCap];
  // first pass: can every grown request be served?  (nothing is changed before that is known)
  bool any = false;
  for (int32_t r = 0; r < batch; ++r) {
    if (kv_len[r] < 1) { mepic_set_error("decode_plan_patch: kv_len[%d] = %d < 1", r, kv_len[r]); return MEPIC_E_INVAL; }
    const int32_t now = (kv_len[r] + P - 1) / P;
    if (now > table_stride) { mepic_set_error("decode_plan_patch: request %d needs %d entries > stride", r, now); return MEPIC_E_INVAL; }
    if (now < req_ent[r]) { mepic_set_error("decode_plan_patch: request %d lost pages: build a new plan", r); return MEPIC_E_INVAL; }
    if (now == req_ent[r]) continue;
    any = true;
    const int32_t i = own_item[r];
    if (i < 0 || items[i * stride + kPiEnt] + (now - req_ent[r]) > rec_cap[i]) {
      mepic_set_error("decode_plan_patch: no room left for request %d's new pages: build a new plan", r);
      return MEPIC_E_CAPACITY;
    }
  }
  *out_n_ranges = 0;
  if (!any) return MEPIC_OK;
  int64_t rec_lo = INT64_MAX, rec_hi = 0;      // the stretch of the buffer (in ints) that holds the new records
  for (int32_t r = 0; r < batch; ++r) {
    const int32_t now = (kv_len[r] + P - 1) / P;
    if (now == req_ent[r]) continue;
    int32_t* it = items + static_cast<size_t>(own_item[r]) * stride;
    for (int32_t e = req_ent[r]; e < now; ++e) {
      const int64_t at = h[kPhOffRecords] + static_cast<int64_t>(it[kPiRecOff] + it[kPiEnt]) * (1 + R);
      int32_t* q = plan + at;
      q[0] = page_ids[static_cast<size_t>(r) * table_stride + e];
      q[1] = pos_base[static_cast<size_t>(r) * table_stride + e];
      for (int j = 1; j < R; ++j) q[1 + j] = 0;
      it[kPiEnt] += 1;
      rec_lo = std::min(rec_lo, at); rec_hi = std::max<int64_t>(rec_hi, at + 1 + R);
    }
    it[kPiTail] = (now - 1) * P;               // the request's last page now lives in its own item
    req_ent[r] = now;
  }
  const int32_t rc = derive_plan(plan);
  if (rc != MEPIC_OK) return rc;
  out_ranges[0] = 0; out_ranges[1] = h[kPhOffRecords];
  out_ranges[2] = rec_lo; out_ranges[3] = rec_hi - rec_lo;
  *out_n_ranges = 2;
  return MEPIC_OK;
}
