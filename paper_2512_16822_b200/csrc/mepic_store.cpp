// Host side of the MEPIC hot path: the scheduling path of Section 3.2 / Algorithm 1.
//
// A store owns the metadata of one page pool: a FIFO free list, the index of
// resident chunks (identity = hash of the canonically padded token sequence,
// Section 3.2.3) and the private pages of every live request.  No device
// memory is touched here; the K/V bytes live in buffers the caller owns.
#include <cuda_runtime.h>

#include "mepic.h"
#include "mepic_internal.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <mutex>
#include <new>
#include <unordered_map>
#include <unordered_set>
#include <vector>

namespace {
thread_local char g_err[512] = "";
}

void mepic_set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

bool mepic_config_ok(const mepic_config_t* c) {
  if (!c) { mepic_set_error("config is NULL"); return false; }
  if (c->page_size < 16 || (c->page_size & (c->page_size - 1)) != 0) {
    mepic_set_error("page_size %d must be a power of two >= 16", c->page_size); return false;
  }
  if (c->head_dim != 64 && c->head_dim != 128) { mepic_set_error("head_dim %d must be 64 or 128", c->head_dim); return false; }
  if (c->n_kv_heads < 1 || c->n_q_heads < 1 || c->n_q_heads % c->n_kv_heads != 0) {
    mepic_set_error("n_q_heads %d must be a positive multiple of n_kv_heads %d", c->n_q_heads, c->n_kv_heads); return false;
  }
  const int g = c->n_q_heads / c->n_kv_heads;
  if (g < 1 || g > 8) { mepic_set_error("group size %d not in 1..8", g); return false; }
  if (c->num_pages < 1) { mepic_set_error("num_pages %d < 1", c->num_pages); return false; }
  if (c->max_position < c->page_size - 1) { mepic_set_error("max_position %d < page_size-1", c->max_position); return false; }
  if (!(c->rope_theta > 1.0f)) { mepic_set_error("rope_theta must exceed 1"); return false; }
  return true;
}

struct Chunk {
  std::vector<int32_t> padded;   // canonical form: leading pads + tokens
  std::vector<int32_t> shared;   // page ids of blocks 1..n-1
  int64_t refs = 0;
  uint64_t last_use = 0;         // store tick of the last register / table build / release that touched it
  bool uncomputed = false;       // the shared pages hold no K/V yet: the next request to alias the chunk computes them
};

struct LiveRequest {
  std::vector<int32_t> private_pages;
  std::vector<uint64_t> chunks;  // one entry per chunk segment
  int64_t entries = 0;
};

static uint64_t fnv1a64(const std::vector<int32_t>& v);

// The tier behind the HBM pool: evicted chunk KV kept in host memory, keyed by content.
struct RemoteChunk {
  std::vector<int32_t> padded;
  std::vector<int64_t> slots;    // one page slot of the tier per shareable block
  uint64_t last_use = 0;
};

struct RemoteTier {
  bool on = false, host_pools = false, failed = false;
  unsigned char* k_pool = nullptr;
  unsigned char* v_pool = nullptr;
  unsigned char* buf = nullptr;            // [capacity][K page | V page]
  int64_t capacity = 0;
  size_t page_bytes = 0;
  std::vector<int64_t> free_slots;
  std::unordered_map<uint64_t, RemoteChunk> chunks;   // key = hash of the padded tokens, bumped on collision
  cudaStream_t stream = nullptr;
  int64_t spilled = 0, fetched = 0;
  uint64_t tick = 0;
  int fail_next = 0;                       // test hook: this many of the next page copies report failure

  ~RemoteTier() {
    if (!buf) return;
    if (host_pools) std::free(buf); else cudaFreeHost(buf);
  }
  // key of `padded` in the tier, or of the free probe position when it is not there
  uint64_t find(const std::vector<int32_t>& padded, bool* found) const {
    uint64_t id = fnv1a64(padded);
    for (;; ++id) {
      auto it = chunks.find(id);
      if (it == chunks.end()) { *found = false; return id; }
      if (it->second.padded == padded) { *found = true; return id; }
    }
  }
  void copy(void* dst, const void* src, bool to_tier) {
    if (fail_next > 0) { --fail_next; failed = true; mepic_set_error("remote tier: page copy failed (injected)"); return; }
    if (host_pools) { std::memcpy(dst, src, page_bytes); return; }
    const cudaError_t e = cudaMemcpyAsync(dst, src, page_bytes, to_tier ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) { failed = true; mepic_set_error("remote tier: cudaMemcpyAsync: %s", cudaGetErrorString(e)); }
  }
  void drop(uint64_t key) {
    auto it = chunks.find(key);
    for (int64_t sl : it->second.slots) free_slots.push_back(sl);
    // keep probe chains intact: re-insert the entries that follow in the chain
    std::vector<RemoteChunk> chain;
    chunks.erase(it);
    for (uint64_t k = key + 1;; ++k) {
      auto nx = chunks.find(k);
      if (nx == chunks.end()) break;
      chain.push_back(std::move(nx->second));
      chunks.erase(nx);
    }
    for (RemoteChunk& c : chain) { bool f; const uint64_t k = find(c.padded, &f); chunks.emplace(k, std::move(c)); }
  }
  // Keep the K/V of an evicted chunk.  The tier gives up its own least recently used chunks for room.
  void spill(const std::vector<int32_t>& padded, const std::vector<int32_t>& pages) {
    bool found;
    uint64_t key = find(padded, &found);
    if (found) { chunks[key].last_use = ++tick; return; }        // shared pages never change once computed
    if (static_cast<int64_t>(pages.size()) > capacity) return;
    while (free_slots.size() < pages.size()) {
      uint64_t victim = 0, oldest = UINT64_MAX;
      for (const auto& kv : chunks) if (kv.second.last_use < oldest) { oldest = kv.second.last_use; victim = kv.first; }
      drop(victim);
    }
    key = find(padded, &found);
    RemoteChunk rc;
    rc.padded = padded;
    for (int32_t pg : pages) {
      const int64_t sl = free_slots.back(); free_slots.pop_back();
      rc.slots.push_back(sl);
      copy(buf + static_cast<size_t>(sl) * 2 * page_bytes, k_pool + static_cast<size_t>(pg) * page_bytes, true);
      copy(buf + static_cast<size_t>(sl) * 2 * page_bytes + page_bytes, v_pool + static_cast<size_t>(pg) * page_bytes, true);
    }
    if (failed) {
      // a copy could not be made: the tier must not claim K/V it does not hold.  Give the slots back (in the order
      // they were taken, so that the next spill sees the same slots) and keep no record of the chunk.
      for (auto it = rc.slots.rbegin(); it != rc.slots.rend(); ++it) free_slots.push_back(*it);
      return;
    }
    rc.last_use = ++tick;
    chunks.emplace(key, std::move(rc));
    spilled += 1;
  }
  // false (and nothing counted) when a copy failed: the caller's pages then hold no valid K/V
  bool fetch(uint64_t key, const std::vector<int32_t>& pages) {
    RemoteChunk& rc = chunks.at(key);
    for (size_t i = 0; i < pages.size(); ++i) {
      copy(k_pool + static_cast<size_t>(pages[i]) * page_bytes, buf + static_cast<size_t>(rc.slots[i]) * 2 * page_bytes, false);
      copy(v_pool + static_cast<size_t>(pages[i]) * page_bytes, buf + static_cast<size_t>(rc.slots[i]) * 2 * page_bytes + page_bytes, false);
    }
    if (failed) return false;
    rc.last_use = ++tick;
    fetched += 1;
    return true;
  }
};

struct mepic_store {
  mepic_config_t cfg;
  RemoteTier remote;
  std::deque<int32_t> free_pages;
  std::unordered_map<uint64_t, Chunk> chunks;          // id -> chunk; id = hash, bumped on collision
  std::unordered_set<uint64_t> erased;                 // ids of reclaimed chunks that other ids were probed past
  uint64_t hash_mask = ~0ull;                          // test hook: fewer hash bits, so that ids collide
  std::unordered_map<int64_t, LiveRequest> requests;
  int64_t dedup_hits = 0;
  int64_t shared_held = 0;
  int64_t private_held = 0;
  int64_t chunks_evicted = 0;
  int64_t pages_evicted = 0;
  uint64_t tick = 0;
  mutable std::mutex mu;

  void touch(Chunk& c) { c.last_use = ++tick; }

  // Section 3.2.3 "Eviction Policy" / Algorithm 1 admission check: if `need` pages are not free, reclaim whole
  // chunk objects with zero references, least recently used first, until they are; chunks named in `protect`
  // (those the call in progress is about to alias) are never taken.  Chunks are reclaimed lazily, only here.
  // Returns false, having evicted nothing, when free + evictable pages cannot cover the demand (Reject).
  bool make_room(size_t need, const std::vector<uint64_t>& protect) {
    if (need <= free_pages.size()) return true;
    std::vector<std::pair<uint64_t, uint64_t>> cand;     // (last_use, id) of evictable chunks that hold pages
    size_t evictable = 0;
    for (const auto& kv : chunks) {
      const Chunk& c = kv.second;
      if (c.refs != 0 || c.shared.empty()) continue;
      if (std::find(protect.begin(), protect.end(), kv.first) != protect.end()) continue;
      cand.emplace_back(c.last_use, kv.first);
      evictable += c.shared.size();
    }
    if (free_pages.size() + evictable < need) return false;
    std::sort(cand.begin(), cand.end());
    for (const auto& lu : cand) {
      if (need <= free_pages.size()) break;
      auto it = chunks.find(lu.second);
      if (remote.on && !it->second.uncomputed) remote.spill(it->second.padded, it->second.shared);
      std::vector<int32_t> pages = it->second.shared;
      std::sort(pages.begin(), pages.end());
      for (int32_t pg : pages) free_pages.push_back(pg);
      shared_held -= static_cast<int64_t>(pages.size());
      pages_evicted += static_cast<int64_t>(pages.size());
      chunks_evicted += 1;
      forget(it);
    }
    return true;
  }

  // Ids are handed out by linear probing from the hash (a chunk whose hash is taken by other content gets the next
  // free id), and callers hold ids, so an id can never move.  A lookup stops at the first id nobody holds; when a
  // chunk that others were probed past goes away its id is therefore remembered as erased and lookups walk on over it.
  // Only a chunk with a successor in its chain leaves such a mark, i.e. only after a 64-bit hash collision.
  void forget(std::unordered_map<uint64_t, Chunk>::iterator it) {
    const uint64_t id = it->first;
    chunks.erase(it);
    if (chunks.count(id + 1) || erased.count(id + 1)) erased.insert(id);
    else for (uint64_t k = id - 1; erased.count(k); --k) erased.erase(k);      // the chain now ends earlier: marks at its end go
  }
  // The id of `padded` if resident (*hit set), else the id a new chunk with this content gets: the first erased id
  // of its chain, else the chain's end.
  uint64_t locate(const std::vector<int32_t>& padded, const Chunk** hit) {
    *hit = nullptr;
    uint64_t id = fnv1a64(padded) & hash_mask;
    bool have_gap = false; uint64_t gap = 0;
    for (;; ++id) {
      auto it = chunks.find(id);
      if (it != chunks.end()) { if (it->second.padded == padded) { *hit = &it->second; return id; } continue; }
      if (erased.count(id)) { if (!have_gap) { have_gap = true; gap = id; } continue; }
      return have_gap ? gap : id;
    }
  }
};

static uint64_t fnv1a64(const std::vector<int32_t>& v) {
  uint64_t h = 0xcbf29ce484222325ULL;
  for (int32_t t : v) {
    uint32_t u = static_cast<uint32_t>(t);
    for (int b = 0; b < 4; ++b) {               // little-endian bytes of the int32
      h ^= static_cast<uint64_t>((u >> (8 * b)) & 0xffu);
      h *= 0x100000001b3ULL;
    }
  }
  return h;
}

extern "C" const char* mepic_last_error(void) { return g_err; }

extern "C" int32_t mepic_store_create(const mepic_config_t* cfg, mepic_store_t** out) {
  if (!out) { mepic_set_error("out is NULL"); return MEPIC_E_INVAL; }
  *out = nullptr;
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  mepic_store* s = new (std::nothrow) mepic_store();
  if (!s) { mepic_set_error("out of host memory"); return MEPIC_E_INVAL; }
  s->cfg = *cfg;
  for (int32_t p = 0; p < cfg->num_pages; ++p) s->free_pages.push_back(p);
  *out = s;
  return MEPIC_OK;
}

extern "C" void mepic_store_destroy(mepic_store_t* store) { delete store; }

extern "C" int32_t mepic_chunk_register(mepic_store_t* s, const int32_t* tokens, int32_t n_tokens,
                                        uint64_t* out_chunk_id, int32_t* out_was_resident, int32_t* out_lead_pad,
                                        int32_t* out_shared_pages, int32_t cap, int32_t* out_n_shared) {
  if (!s || !tokens || n_tokens <= 0 || cap < 0 || (cap > 0 && !out_shared_pages)) {
    mepic_set_error("chunk_register: bad argument"); return MEPIC_E_INVAL;
  }
  std::lock_guard<std::mutex> lock(s->mu);
  const int32_t P = s->cfg.page_size;
  const int32_t lead = (P - n_tokens % P) % P;                 // Section 3.2.1: chunks are padded at the FRONT
  std::vector<int32_t> padded(static_cast<size_t>(lead) + n_tokens, s->cfg.pad_token_id);
  std::copy(tokens, tokens + n_tokens, padded.begin() + lead);
  const Chunk* hit = nullptr;
  uint64_t id = s->locate(padded, &hit);                        // identity is by content: hash, confirm, else probe on
  int32_t resident = 0;
  const std::vector<int32_t>* shared = nullptr;
  if (hit) {
    resident = 1;
    s->dedup_hits += 1;
    s->touch(s->chunks.at(id));
    shared = &hit->shared;
  } else {
    const size_t n_shared = padded.size() / P - 1;              // first block is private to each request
    if (!s->make_room(n_shared, {})) {
      mepic_set_error("chunk_register: %zu shared pages needed, %zu free and not enough evictable", n_shared, s->free_pages.size());
      return MEPIC_E_NOSPACE;
    }
    // a spill made for room could not be copied out: the evicted chunks are gone from HBM and the tier kept no
    // record of the one that failed, so the state is consistent; report it before anything is allocated
    if (s->remote.failed) { s->remote.failed = false; return MEPIC_E_CUDA; }
    id = s->locate(padded, &hit);                               // the evictions may have freed an earlier id of the chain
    Chunk c;
    c.shared.reserve(n_shared);
    for (size_t i = 0; i < n_shared; ++i) { c.shared.push_back(s->free_pages.front()); s->free_pages.pop_front(); }
    if (s->remote.on && n_shared > 0) {
      // Algorithm 1, residency resolution: not in HBM, but is there a remote copy?  (Looked up after make_room: the
      // evictions it caused may have made the tier drop this very chunk.)
      bool found;
      const uint64_t key = s->remote.find(padded, &found);
      if (found) {
        if (!s->remote.fetch(key, c.shared)) {
          // the pages hold no valid K/V: hand them back where they came from and register nothing
          for (auto it = c.shared.rbegin(); it != c.shared.rend(); ++it) s->free_pages.push_front(*it);
          s->remote.failed = false;
          return MEPIC_E_CUDA;
        }
        resident = 2;
      }
    }
    s->touch(c);
    c.padded = std::move(padded);
    s->shared_held += static_cast<int64_t>(n_shared);
    s->erased.erase(id);
    shared = &s->chunks.emplace(id, std::move(c)).first->second.shared;
  }
  if (out_chunk_id) *out_chunk_id = id;
  if (out_was_resident) *out_was_resident = resident;
  if (out_lead_pad) *out_lead_pad = lead;
  if (out_n_shared) *out_n_shared = static_cast<int32_t>(shared->size());
  if (static_cast<size_t>(cap) < shared->size()) {
    if (out_shared_pages || cap > 0) { mepic_set_error("chunk_register: cap %d < %zu shared pages", cap, shared->size()); return MEPIC_E_CAPACITY; }
    return MEPIC_OK;   // caller did not ask for the page list
  }
  if (out_shared_pages) std::copy(shared->begin(), shared->end(), out_shared_pages);
  return MEPIC_OK;
}

extern "C" int32_t mepic_build_block_table(mepic_store_t* s, int64_t request_id,
                                           const mepic_segment_t* segs, int32_t n_segs,
                                           int32_t* out_page_ids, int32_t* out_pos_base, int32_t cap_entries,
                                           int32_t* out_n_entries, int32_t* out_kv_len,
                                           int32_t* out_recompute_slots, int32_t cap_slots, int32_t* out_n_slots) {
  if (!s || !segs || n_segs <= 0 || cap_entries < 0 || cap_slots < 0 ||
      (cap_entries > 0 && (!out_page_ids || !out_pos_base)) || (cap_slots > 0 && !out_recompute_slots)) {
    mepic_set_error("build_block_table: bad argument"); return MEPIC_E_INVAL;
  }
  std::lock_guard<std::mutex> lock(s->mu);
  if (s->requests.count(request_id)) { mepic_set_error("request %lld already live", (long long)request_id); return MEPIC_E_EXISTS; }
  const int64_t P = s->cfg.page_size;
  // Pass 1 (Algorithm 1, canonicalisation + admission check): sizes only, nothing allocated.
  int last = -1;
  for (int i = 0; i < n_segs; ++i) {
    if (segs[i].kind == MEPIC_SEG_CHUNK) {
      if (!s->chunks.count(segs[i].chunk_id)) { mepic_set_error("segment %d: unknown chunk id", i); return MEPIC_E_NOTFOUND; }
      last = i;
    } else if (segs[i].kind == MEPIC_SEG_PROMPT) {
      if (segs[i].n_tokens < 0) { mepic_set_error("segment %d: negative length", i); return MEPIC_E_INVAL; }
      if (segs[i].n_tokens > 0) last = i;                      // empty prompt segments are skipped
    } else { mepic_set_error("segment %d: bad kind %d", i, segs[i].kind); return MEPIC_E_INVAL; }
  }
  if (last < 0) { mepic_set_error("request has no tokens"); return MEPIC_E_INVAL; }
  int64_t entries = 0, need_private = 0, slots = 0, kv_len = 0;
  for (int i = 0; i <= last; ++i) {
    if (segs[i].kind == MEPIC_SEG_CHUNK) {
      const Chunk& c = s->chunks.at(segs[i].chunk_id);
      // Section 3.3.1: a cached chunk recomputes its first block only; a newly encountered one is recomputed whole
      // (once per request: a second occurrence of the same chunk in this request finds it computed)
      bool whole = c.uncomputed;
      for (int k = 0; k < i && whole; ++k)
        if (segs[k].kind == MEPIC_SEG_CHUNK && segs[k].chunk_id == segs[i].chunk_id) whole = false;
      entries += 1 + static_cast<int64_t>(c.shared.size());
      need_private += 1;
      slots += whole ? P * (1 + static_cast<int64_t>(c.shared.size())) : P;
      kv_len = entries * P;
    } else if (segs[i].n_tokens > 0) {
      const int64_t n = segs[i].n_tokens, pages = (n + P - 1) / P;
      const int64_t seg_len = (i == last) ? n : pages * P;     // trailing pad unless final segment
      kv_len = entries * P + seg_len;
      slots += seg_len;
      entries += pages;
      need_private += pages;
    }
  }
  if (kv_len > INT32_MAX || entries > INT32_MAX) { mepic_set_error("request too long"); return MEPIC_E_INVAL; }
  if (out_n_entries) *out_n_entries = static_cast<int32_t>(entries);
  if (out_n_slots) *out_n_slots = static_cast<int32_t>(slots);
  if (out_kv_len) *out_kv_len = static_cast<int32_t>(kv_len);
  if (entries > cap_entries || slots > cap_slots) {
    mepic_set_error("build_block_table: need %lld entries, %lld slots", (long long)entries, (long long)slots);
    return MEPIC_E_CAPACITY;
  }
  {
    std::vector<uint64_t> protect;                              // the chunks this request is about to alias
    for (int i = 0; i <= last; ++i)
      if (segs[i].kind == MEPIC_SEG_CHUNK) protect.push_back(segs[i].chunk_id);
    if (!s->make_room(static_cast<size_t>(need_private), protect)) {
      mepic_set_error("build_block_table: %lld private pages needed, %zu free and not enough evictable",
                      (long long)need_private, s->free_pages.size());
      return MEPIC_E_NOSPACE;                                   // Reject; nothing is held, nothing was evicted
    }
    if (s->remote.failed) { s->remote.failed = false; return MEPIC_E_CUDA; }
  }
  // Pass 2 (block assignment).
  LiveRequest live;
  int64_t e = 0, w = 0;
  auto take = [&]() { int32_t p = s->free_pages.front(); s->free_pages.pop_front(); live.private_pages.push_back(p); return p; };
  for (int i = 0; i <= last; ++i) {
    const int64_t start = e * P;
    if (segs[i].kind == MEPIC_SEG_CHUNK) {
      Chunk& c = s->chunks.at(segs[i].chunk_id);
      out_page_ids[e++] = take();                               // first block: private, recomputed
      for (int32_t p : c.shared) out_page_ids[e++] = p;         // remaining blocks: shared chunk KV
      const int64_t n_rec = c.uncomputed ? P * (1 + static_cast<int64_t>(c.shared.size())) : P;
      c.uncomputed = false;                                     // this request computes them; later ones reuse them
      for (int64_t t = 0; t < n_rec; ++t) out_recompute_slots[w++] = static_cast<int32_t>(start + t);
      c.refs += 1;
      s->touch(c);
      live.chunks.push_back(segs[i].chunk_id);
    } else if (segs[i].n_tokens > 0) {
      const int64_t n = segs[i].n_tokens, pages = (n + P - 1) / P;
      for (int64_t k = 0; k < pages; ++k) out_page_ids[e++] = take();
      const int64_t seg_len = (i == last) ? n : pages * P;
      for (int64_t t = 0; t < seg_len; ++t) out_recompute_slots[w++] = static_cast<int32_t>(start + t);
    }
  }
  for (int64_t k = 0; k < entries; ++k) out_pos_base[k] = static_cast<int32_t>(k * P);
  live.entries = entries;
  s->private_held += static_cast<int64_t>(live.private_pages.size());
  s->requests.emplace(request_id, std::move(live));
  return MEPIC_OK;
}

extern "C" int32_t mepic_chunk_mark_uncomputed(mepic_store_t* s, uint64_t chunk_id) {
  if (!s) { mepic_set_error("store is NULL"); return MEPIC_E_INVAL; }
  std::lock_guard<std::mutex> lock(s->mu);
  auto it = s->chunks.find(chunk_id);
  if (it == s->chunks.end()) { mepic_set_error("unknown chunk id"); return MEPIC_E_NOTFOUND; }
  if (it->second.refs != 0) { mepic_set_error("chunk is aliased by live requests"); return MEPIC_E_EXISTS; }
  it->second.uncomputed = true;
  return MEPIC_OK;
}

extern "C" int32_t mepic_request_release(mepic_store_t* s, int64_t request_id) {
  if (!s) { mepic_set_error("store is NULL"); return MEPIC_E_INVAL; }
  std::lock_guard<std::mutex> lock(s->mu);
  auto it = s->requests.find(request_id);
  if (it == s->requests.end()) { mepic_set_error("request %lld not live", (long long)request_id); return MEPIC_E_NOTFOUND; }
  LiveRequest& r = it->second;
  for (uint64_t id : r.chunks) { Chunk& c = s->chunks.at(id); c.refs -= 1; s->touch(c); }
  std::sort(r.private_pages.begin(), r.private_pages.end());
  for (int32_t p : r.private_pages) s->free_pages.push_back(p);
  s->private_held -= static_cast<int64_t>(r.private_pages.size());
  s->requests.erase(it);
  return MEPIC_OK;
}

extern "C" int32_t mepic_store_stats(const mepic_store_t* s, mepic_stats_t* out) {
  if (!s || !out) { mepic_set_error("stats: NULL argument"); return MEPIC_E_INVAL; }
  std::lock_guard<std::mutex> lock(s->mu);
  out->pages_total = s->cfg.num_pages;
  out->pages_free = static_cast<int64_t>(s->free_pages.size());
  out->pages_shared_held = s->shared_held;
  out->pages_private_held = s->private_held;
  out->chunks_resident = static_cast<int64_t>(s->chunks.size());
  int64_t refs = 0;
  for (const auto& kv : s->chunks) refs += kv.second.refs;
  out->chunk_refs = refs;
  out->dedup_hits = s->dedup_hits;
  int64_t ent = 0;
  for (const auto& kv : s->requests) ent += kv.second.entries;
  out->unshared_equivalent_pages = ent;
  out->live_requests = static_cast<int64_t>(s->requests.size());
  out->chunks_evicted = s->chunks_evicted;
  out->pages_evicted = s->pages_evicted;
  out->chunks_spilled = s->remote.spilled;
  out->chunks_fetched = s->remote.fetched;
  out->remote_chunks = static_cast<int64_t>(s->remote.chunks.size());
  out->remote_pages = s->remote.on ? s->remote.capacity - static_cast<int64_t>(s->remote.free_slots.size()) : 0;
  return MEPIC_OK;
}

extern "C" int32_t mepic_store_attach_remote(mepic_store_t* s, void* k_pool, void* v_pool, int32_t pools_on_host,
                                             int64_t capacity_pages, void* cuda_stream) {
  if (!s || !k_pool || !v_pool || capacity_pages < 1) { mepic_set_error("attach_remote: bad argument"); return MEPIC_E_INVAL; }
  std::lock_guard<std::mutex> lock(s->mu);
  RemoteTier& r = s->remote;
  if (r.on) { mepic_set_error("attach_remote: the store already has a remote tier"); return MEPIC_E_EXISTS; }
  r.page_bytes = static_cast<size_t>(s->cfg.n_kv_heads) * s->cfg.page_size * s->cfg.head_dim * 2;
  const size_t bytes = static_cast<size_t>(capacity_pages) * 2 * r.page_bytes;
  if (pools_on_host) {
    r.buf = static_cast<unsigned char*>(std::malloc(bytes));
    if (!r.buf) { mepic_set_error("attach_remote: out of host memory"); return MEPIC_E_INVAL; }
  } else {
    void* ptr = nullptr;
    const cudaError_t e = cudaHostAlloc(&ptr, bytes, cudaHostAllocDefault);
    if (e != cudaSuccess) { mepic_set_error("attach_remote: cudaHostAlloc(%zu): %s", bytes, cudaGetErrorString(e)); return MEPIC_E_CUDA; }
    r.buf = static_cast<unsigned char*>(ptr);
  }
  r.host_pools = pools_on_host != 0;
  r.k_pool = static_cast<unsigned char*>(k_pool);
  r.v_pool = static_cast<unsigned char*>(v_pool);
  r.capacity = capacity_pages;
  r.stream = static_cast<cudaStream_t>(cuda_stream);
  r.free_slots.reserve(static_cast<size_t>(capacity_pages));
  for (int64_t i = capacity_pages - 1; i >= 0; --i) r.free_slots.push_back(i);    // slot 0 is handed out first
  r.on = true;
  return MEPIC_OK;
}

extern "C" int32_t mepic_store_test_hooks(mepic_store_t* s, uint64_t hash_mask, int32_t fail_copies) {
  if (!s || fail_copies < 0) { mepic_set_error("test_hooks: bad argument"); return MEPIC_E_INVAL; }
  std::lock_guard<std::mutex> lock(s->mu);
  if (hash_mask != s->hash_mask && !s->chunks.empty()) { mepic_set_error("test_hooks: the hash mask can only change while no chunk is resident"); return MEPIC_E_EXISTS; }
  s->hash_mask = hash_mask;
  s->remote.fail_next = fail_copies;
  return MEPIC_OK;
}

// ---------------------------------------------------------------- rope table (set-up, host)
extern "C" size_t mepic_rope_table_floats(const mepic_config_t* cfg) {
  if (!mepic_config_ok(cfg)) return 0;
  return (static_cast<size_t>(cfg->max_position) + 1) * static_cast<size_t>(cfg->head_dim);
}

extern "C" int32_t mepic_rope_table_fill(const mepic_config_t* cfg, float* out) {
  if (!mepic_config_ok(cfg) || !out) { if (cfg && !out) mepic_set_error("rope_table_fill: out is NULL"); return MEPIC_E_INVAL; }
  const int half = cfg->head_dim / 2;
  std::vector<double> inv_freq(half);
  for (int i = 0; i < half; ++i) inv_freq[i] = std::pow(static_cast<double>(cfg->rope_theta), -2.0 * i / cfg->head_dim);
  for (int64_t p = 0; p <= cfg->max_position; ++p) {
    float* row = out + p * cfg->head_dim;
    for (int i = 0; i < half; ++i) {
      const double a = static_cast<double>(p) * inv_freq[i];
      row[2 * i] = static_cast<float>(std::cos(a));
      row[2 * i + 1] = static_cast<float>(std::sin(a));
    }
  }
  return MEPIC_OK;
}

// ---------------------------------------------------------------- kernel test hooks
static std::atomic<int> g_spin_limit{0}, g_skip_tile{-1};
int mepic_test_spin_limit(int built_in) { const int v = g_spin_limit.load(std::memory_order_relaxed); return v > 0 ? v : built_in; }
int mepic_test_skip_tile() { return g_skip_tile.load(std::memory_order_relaxed); }
extern "C" int32_t mepic_kernel_test_hooks(int32_t spin_limit, int32_t skip_tile) {
  if (spin_limit < 0 || skip_tile < -1) { mepic_set_error("kernel_test_hooks: bad argument"); return MEPIC_E_INVAL; }
  g_spin_limit.store(spin_limit, std::memory_order_relaxed);
  g_skip_tile.store(skip_tile, std::memory_order_relaxed);
  return MEPIC_OK;
}

static std::atomic<int> g_prefill_two_pass{0};
int mepic_test_prefill_two_pass() { return g_prefill_two_pass.load(std::memory_order_relaxed); }
extern "C" int32_t mepic_prefill_test_two_pass(int32_t on) {
  g_prefill_two_pass.store(on != 0, std::memory_order_relaxed);
  return MEPIC_OK;
}

// ---------------------------------------------------------------- launch counter
static std::atomic<int64_t> g_launches{0};
void mepic_count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
extern "C" int64_t mepic_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
