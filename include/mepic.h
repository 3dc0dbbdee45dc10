/*
 * mepic.h - C ABI of the B200 (sm_100a) hot path of MEPIC: attention over a
 * page-aligned, position-free chunk KV cache.
 *
 * Shared chunk pages hold UN-ROTATED keys (the paper's NoPE KV format,
 * Section 3.3.3); rotary position embedding is applied to K inside the
 * attention kernels, from the logical position base that every block-table
 * entry carries.  The host side implements the scheduling path of Section 3.2
 * / Algorithm 1 (canonical padding, chunk identity by hash of the padded
 * tokens, first KV block private per request, remaining blocks shared); the
 * device side implements the computation path of Section 3.3 (commit of
 * recomputed K/V into the assigned pages, fused-RoPE attention).
 *
 * Conventions
 *  - Every function returns an int32_t status: MEPIC_OK (0) or a negative
 *    MEPIC_E_* code.  Nothing throws or aborts across this boundary;
 *    mepic_last_error() returns thread-local text for the last failure.
 *  - "host" / "device" is stated for every pointer.  The CALLER owns every
 *    device buffer and the CUDA stream; the library owns only the host
 *    metadata inside mepic_store_t (and, when a remote tier is attached, that
 *    tier's page-locked HOST buffer).  The library never allocates or frees
 *    device memory and never synchronises the stream: kernels and copies are
 *    enqueued and the call returns.
 *  - Device-side problems (a page id outside the pool, a bounded wait that ran
 *    out) never fault or hang the GPU: the kernel records a code in the device
 *    status word the caller passes and carries on with safe values.  Read the
 *    word after synchronising; 0 means clean.
 *  - bf16 tensors are passed as plain pointers to 16-bit words.
 *  - Layouts (row-major, last index fastest):
 *        K pool, V pool : [num_pages][n_kv_heads][page_size][head_dim]  bf16
 *        q (decode)     : [batch][n_q_heads][head_dim]                   bf16
 *        block table    : page_ids[batch][table_stride], pos_base[batch][table_stride]  int32
 *        rope table     : [max_position + 1][head_dim / 2][2] fp32 = (cos, sin)
 *    q head h reads KV head h / (n_q_heads / n_kv_heads).
 *  - RoPE convention (the paper does not state one): split-half pairing
 *    (i, i + head_dim/2), angle = position * rope_theta^(-2 i / head_dim), no
 *    frequency scaling.  V is never rotated.
 *  - Logical slot t of a request lives in block-table entry e = t / page_size,
 *    at in-page slot t % page_size, and has position pos_base[e] + t % page_size.
 *    Causality is by logical slot; rotation is by position.
 */
#ifndef MEPIC_H_
#define MEPIC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MEPIC_OK                 0
#define MEPIC_E_INVAL           -1  /* bad argument, unsupported shape, misaligned pointer */
#define MEPIC_E_NOSPACE         -2  /* Algorithm 1's Reject: the page pool cannot supply the blocks */
#define MEPIC_E_NOTFOUND        -3  /* unknown chunk id or request id */
#define MEPIC_E_CAPACITY        -4  /* caller's output array too small; required count written back */
#define MEPIC_E_CUDA            -5  /* a CUDA runtime call failed; see mepic_last_error() */
#define MEPIC_E_EXISTS          -6  /* request id already has a live block table */

/* Codes a kernel may OR into the device status word. */
#define MEPIC_DEV_BAD_PAGE      0x1 /* a block-table entry named a page outside [0, num_pages) */
#define MEPIC_DEV_WAIT_EXPIRED  0x2 /* a bounded wait on an on-chip barrier ran out */
#define MEPIC_DEV_BAD_POSITION  0x4 /* a position fell outside the rope table */
#define MEPIC_DEV_BAD_SLOT      0x8 /* a new row's logical slot fell outside its request */
#define MEPIC_DEV_BAD_PLAN      0x10 /* a grouped-decode plan no longer matches kv_len (a request gained or lost a page) */

#define MEPIC_SEG_CHUNK  0
#define MEPIC_SEG_PROMPT 1

typedef struct mepic_store mepic_store_t;

typedef struct {
  int32_t page_size;     /* tokens per KV block ("page"); power of two, >= 16 */
  int32_t n_q_heads;
  int32_t n_kv_heads;    /* divides n_q_heads; group size n_q_heads/n_kv_heads in 1..8 */
  int32_t head_dim;      /* 64 or 128 */
  int32_t num_pages;     /* pages in the pool */
  int32_t pad_token_id;  /* token used for canonical padding; part of the hashed sequence */
  int32_t max_position;  /* largest position the rope table covers (inclusive) */
  float   rope_theta;
} mepic_config_t;

typedef struct {
  int64_t pages_total;
  int64_t pages_free;
  int64_t pages_shared_held;          /* pages owned by resident chunks (all but their first block) */
  int64_t pages_private_held;         /* pages owned by live requests */
  int64_t chunks_resident;
  int64_t chunk_refs;                 /* sum over chunks of live requests aliasing them */
  int64_t dedup_hits;                 /* mepic_chunk_register calls that found the chunk resident */
  int64_t unshared_equivalent_pages;  /* sum of block-table entries of live requests = pages a
                                         per-request copy of every chunk would hold */
  int64_t live_requests;
  int64_t chunks_evicted;             /* zero-reference chunk objects reclaimed under memory pressure */
  int64_t pages_evicted;              /* pages those evictions returned to the pool */
  int64_t chunks_spilled;             /* evicted chunks whose pages were copied to the remote tier */
  int64_t chunks_fetched;             /* registrations served from the remote tier */
  int64_t remote_chunks;              /* chunks the remote tier holds now */
  int64_t remote_pages;               /* page slots of the remote tier in use */
} mepic_stats_t;

typedef struct {
  int32_t  kind;       /* MEPIC_SEG_CHUNK or MEPIC_SEG_PROMPT */
  int32_t  n_tokens;   /* prompt segments: token count (0 = skipped); ignored for chunks */
  uint64_t chunk_id;   /* chunk segments: id returned by mepic_chunk_register */
} mepic_segment_t;

const char* mepic_last_error(void);

/* Number of kernels this library has launched in this process (all threads). */
int64_t mepic_launch_count(void);

/* ---------------------------------------------------------------- scheduling path (host only)
 *
 * mepic_store_create: make an empty store over a pool of cfg->num_pages pages.  Free pages are
 * handed out first-in-first-out starting from 0,1,2,...; released pages rejoin the queue in
 * ascending order (the paper leaves the order open; this one makes tables reproducible).
 *
 * Memory pressure (Section 3.2.3 "Eviction Policy"; Algorithm 1, admission check): when a call needs
 * more pages than are free, whole chunk objects with ZERO live references are reclaimed, least
 * recently used first (use = the last register, table build or release that touched the chunk),
 * until the demand is met; their pages rejoin the queue in ascending order per chunk.  Chunks the
 * call itself is about to alias, and every page private to a live request, are never reclaimed.
 * Reclaiming is lazy: it happens only inside such a call.  If free plus reclaimable pages cannot
 * cover the demand the call is rejected (MEPIC_E_NOSPACE) and nothing is reclaimed.  The id of a
 * reclaimed chunk becomes unknown; registering the same tokens again reports was_resident = 0.
 * References are taken by mepic_build_block_table, not by mepic_chunk_register: under pressure a
 * request's later registration may reclaim a chunk the same request registered just before; the
 * table build then returns MEPIC_E_NOTFOUND and the caller registers that chunk again.
 * cfg: host.  out: host, receives the handle.  Errors: E_INVAL.
 */
int32_t mepic_store_create(const mepic_config_t* cfg, mepic_store_t** out);
void    mepic_store_destroy(mepic_store_t* store);

/*
 * mepic_chunk_register - Section 3.2.1 (canonical leading pad), Section 3.2.2 (residency lookup),
 * Section 3.2.3 "KV Block Allocation" (identity = hash of the PADDED token sequence; the first
 * block is recomputed per request, the remaining blocks are the shareable chunk KV).
 *
 * tokens (host, n_tokens > 0 int32): the UNPADDED chunk.  The store pads it at the front with
 * pad_token_id to a multiple of page_size, hashes the padded sequence (64-bit FNV-1a, confirmed by
 * a full token compare, so identity is by content) and looks it up.  On a miss it takes
 * ceil(n/page_size) - 1 pages from the pool for the shareable blocks; on a hit it allocates
 * nothing (a miss may first reclaim idle chunks, see mepic_store_create).  out_chunk_id, out_was_resident
 * (0 = new, 1 = resident, 2 = brought back from the remote tier, see mepic_store_attach_remote), out_lead_pad (pad tokens added), out_n_shared:
 * host, each may be NULL.  out_shared_pages (host, cap entries, may be NULL when cap == 0)
 * receives the shared page ids in block order.
 * Errors: E_INVAL; E_NOSPACE (nothing allocated, chunk not registered); E_CAPACITY (cap too small:
 * *out_n_shared holds the count needed; the registration itself HAS taken place).
 */
int32_t mepic_chunk_register(mepic_store_t* store, const int32_t* tokens, int32_t n_tokens,
                             uint64_t* out_chunk_id, int32_t* out_was_resident, int32_t* out_lead_pad,
                             int32_t* out_shared_pages, int32_t cap, int32_t* out_n_shared);

/*
 * mepic_build_block_table - Algorithm 1 (segment -> pad -> admission check -> block assignment)
 * for one request whose chunks are already registered.
 *
 * segs (host, n_segs): the request's segments in order.  A chunk segment contributes one freshly
 * allocated PRIVATE first page followed by the chunk's shared pages; a prompt segment contributes
 * ceil(n_tokens/page_size) private pages and is padded at the back to a block boundary unless it
 * is the request's last segment.  Entry e gets pos_base[e] = e * page_size (a token's position is
 * its index in the padded sequence).  Outputs (host): out_page_ids / out_pos_base (cap_entries
 * each), *out_n_entries, *out_kv_len (padded length; pads are ordinary tokens), and
 * out_recompute_slots (cap_slots): the logical slots whose K/V the caller must compute and hand
 * to mepic_attn_prefill = every slot below kv_len that lives on a private page, plus every slot of a
 * chunk marked by mepic_chunk_mark_uncomputed (first occurrence in the request), ascending.
 * The admission check runs before any allocation: on E_NOSPACE nothing is held.
 * Errors: E_INVAL (no tokens, bad kind), E_NOTFOUND (chunk id), E_EXISTS (request id live),
 * E_NOSPACE, E_CAPACITY (required counts written to *out_n_entries / *out_n_slots; nothing held).
 */
int32_t mepic_build_block_table(mepic_store_t* store, int64_t request_id,
                                const mepic_segment_t* segs, int32_t n_segs,
                                int32_t* out_page_ids, int32_t* out_pos_base, int32_t cap_entries,
                                int32_t* out_n_entries, int32_t* out_kv_len,
                                int32_t* out_recompute_slots, int32_t cap_slots, int32_t* out_n_slots);

/*
 * mepic_chunk_mark_uncomputed - Section 3.3.1: a chunk seen for the first time is recomputed whole, a cached
 * one only in its first KV block.  A registered chunk is taken to have its shareable
 * pages filled by the caller (offline precompute, a load from a remote tier).  When that is not so - the chunk
 * is new (mepic_chunk_register reported was_resident = 0) and nobody has its K/V - mark it: the NEXT
 * mepic_build_block_table that aliases the chunk lists every slot of the chunk, shared pages included, among its
 * recompute slots, so that that request's mepic_attn_prefill call computes and commits the whole chunk; the mark
 * is cleared by that build, and later requests recompute the first block only.  The caller orders that prefill
 * before any other request's attention over the chunk (same stream, or an event).
 * Errors: E_NOTFOUND; E_EXISTS if live requests already alias the chunk.
 */
int32_t mepic_chunk_mark_uncomputed(mepic_store_t* store, uint64_t chunk_id);

/* Request end (Section 3.2.3 "Eviction Policy"): private pages go back to the pool in ascending
 * order, the reference count of every chunk the request aliased drops by one; chunks stay
 * resident.  Errors: E_NOTFOUND. */
int32_t mepic_request_release(mepic_store_t* store, int64_t request_id);

/* Snapshot of the pool ("HBM usage" of Section 4 in units of pages).  out: host. */
int32_t mepic_store_stats(const mepic_store_t* store, mepic_stats_t* out);

/*
 * mepic_store_attach_remote - a second tier behind the HBM pool for chunk KV, standing in for the
 * remote chunk store of the paper's serving stack (Section 3.1; Algorithm 1 "resolve HBM residency
 * and remote availability"; Section 3.2.3 eviction).  capacity_pages page slots of host memory are
 * allocated (page-locked when the pools are device memory).  From then on
 *   - a computed chunk reclaimed under memory pressure (Section 3.2.3) first has its shareable pages
 *     copied, K and V, into the tier; the tier drops its own least recently used chunks to make room,
 *     and a chunk larger than the whole tier is not kept;
 *   - mepic_chunk_register of a chunk that is not resident but is in the tier allocates its pages as
 *     for a miss and copies the K/V back into them: *out_was_resident = 2, the pages need no
 *     recomputation (only the first block does, per request, as for any cached chunk).  The tier keeps
 *     its copy.
 * k_pool / v_pool: the pools the kernels read, [num_pages][n_kv_heads][page_size][head_dim] bf16.
 * pools_on_host = 0: DEVICE pointers; copies are cudaMemcpyAsync on cuda_stream, so they are ordered
 * with the caller's kernels only if those run on the same stream (or the caller synchronises), and a
 * page handed out by a call may still be the source of a copy enqueued by that call.
 * pools_on_host = 1: HOST pointers and plain memcpy (no CUDA call at all; cuda_stream ignored) - for
 * host-only use and tests.  One tier per store; E_EXISTS if already attached, E_INVAL for bad
 * arguments, E_CUDA if page-locked memory cannot be had or (later, from the call that triggered it)
 * a copy cannot be enqueued.  The tier is freed by mepic_store_destroy.
 */
int32_t mepic_store_attach_remote(mepic_store_t* store, void* k_pool, void* v_pool, int32_t pools_on_host,
                                  int64_t capacity_pages, void* cuda_stream);

/*
 * mepic_store_test_hooks - host-side fault injection for the store's rare paths (the paper has no counterpart;
 * no GPU is involved).  hash_mask: chunk ids are taken from (hash & hash_mask), so a mask of a few bits makes
 * different chunks collide and exercises the probing that keeps identity by content (may only change while no
 * chunk is resident; ~0 = normal).  fail_copies: the next fail_copies page copies to or from the remote tier
 * report failure without copying, as a failed cudaMemcpyAsync would.  What a failed copy leaves behind: a spill
 * that failed keeps no record of the chunk in the tier (the eviction itself stands), a fetch that failed returns
 * the pages and registers nothing; the call that triggered it returns MEPIC_E_CUDA.  Errors: E_INVAL, E_EXISTS.
 */
int32_t mepic_store_test_hooks(mepic_store_t* store, uint64_t hash_mask, int32_t fail_copies);

/*
 * mepic_kernel_test_hooks - lets a test make a kernel's bounded wait run out, in the one form that harms nothing
 * (the paper has no counterpart).  Every wait of the kernels on an on-chip barrier polls a limited number of times
 * and then gives up: the kernel ORs MEPIC_DEV_WAIT_EXPIRED into the status word, lets whatever it still has in
 * flight land, releases what it holds and returns; the results of that call are undefined, the GPU and the
 * context stay usable.  spin_limit > 0 replaces the built-in poll limit (about a second) for calls made from now
 * on, 0 restores it.  skip_tile >= 0 makes the first worker of every such call (warp 0 of CTA 0 in the decode
 * kernels, the K loader of CTA 0 in the prefill kernel) leave out the staged copy of its tile with that index, so
 * that the barrier that copy would complete is a flag nothing sets and the wait on it expires; -1 restores normal
 * operation.  Process-wide; not for production use.  Errors: E_INVAL.
 */
int32_t mepic_kernel_test_hooks(int32_t spin_limit, int32_t skip_tile);

/*
 * mepic_prefill_test_two_pass - lets a test compare the two softmax schedules of mepic_attn_prefill (the paper has no
 * counterpart).  on != 0: calls made from now on enqueue the attention kernel once, with the reference found from each
 * tile's own scores (the repeat launch's schedule) for every item; the first word of the workspace stays clear;
 * 0 restores the fast launch followed by the conditional repeat launch.  Both schedules compute the same softmax;
 * their outputs differ by the rounding of P to bf16 under different references only.  Process-wide; not for
 * production use.  Always returns MEPIC_OK.
 */
int32_t mepic_prefill_test_two_pass(int32_t on);

/* ---------------------------------------------------------------- rope table (host, set-up)
 *
 * Section 3.3.3 has the kernel apply each block's rotary offset but gives no formula; the table
 * holds (cos, sin)(p * rope_theta^(-2i/head_dim)) for p in [0, max_position], i < head_dim/2,
 * computed in double precision and rounded to fp32.  The caller uploads it once and passes the
 * device copy to the attention calls.  mepic_rope_table_floats returns the float count
 * (max_position+1) * head_dim, or 0 for a bad config; mepic_rope_table_fill writes that many
 * floats to out (host).  Errors: E_INVAL.
 */
size_t  mepic_rope_table_floats(const mepic_config_t* cfg);
int32_t mepic_rope_table_fill(const mepic_config_t* cfg, float* out);

/* ---------------------------------------------------------------- decode (device)
 *
 * mepic_attn_decode - Section 3.3.3 for one new token per request: for every request b and query
 * head h,
 *     out[b,h,:] = sum_t softmax_t( sm_scale * < R(q_pos[b]) q[b,h,:] , R(pos_t) K_t > ) V_t ,
 * t over the kv_len[b] logical slots of the request, K_t / V_t read through the block table from
 * the un-rotated pools, R the rotary embedding.  The work is split over the KV axis across the
 * whole GPU; partial (max, sum, weighted V) triples go to the workspace and a second kernel
 * combines them (log-sum-exp merge) and writes bf16.
 *
 * All pointers in the struct are DEVICE pointers.  kv_len[b] >= 1; entries beyond
 * ceil(kv_len[b]/page_size) are not read; slots at or beyond kv_len[b] in the last page are
 * ignored whatever bits they hold.  workspace: at least mepic_attn_decode_workspace() bytes,
 * 16-byte aligned; contents need not be initialised and are overwritten.  status: one int32 the
 * caller zeroed; MEPIC_DEV_* bits are ORed in.  Two calls that overlap on the GPU must not share
 * a workspace.  Errors: E_INVAL (null/misaligned pointer, unsupported shape, workspace too small),
 * E_CUDA.
 */
typedef struct {
  const void*    q;            /* bf16 [batch][n_q_heads][head_dim], un-rotated */
  const void*    k_pool;       /* bf16 pool, K un-rotated; 16-byte aligned */
  const void*    v_pool;       /* bf16 pool; 16-byte aligned */
  const int32_t* page_ids;     /* [batch][table_stride] */
  const int32_t* pos_base;     /* [batch][table_stride] */
  const int32_t* kv_len;       /* [batch] */
  const int32_t* q_pos;        /* [batch] position of the query token */
  const float*   rope_table;   /* see above */
  void*          out;          /* bf16 [batch][n_q_heads][head_dim] */
  void*          workspace;
  size_t         workspace_bytes;
  int32_t*       status;
  int32_t        table_stride;
  int32_t        batch;
  float          sm_scale;
} mepic_decode_args_t;

/* Bytes of workspace mepic_attn_decode needs for this config and batch on the CURRENT device
 * (depends on its SM count); 0 on error. */
size_t  mepic_attn_decode_workspace(const mepic_config_t* cfg, int32_t batch);
int32_t mepic_attn_decode(const mepic_config_t* cfg, const mepic_decode_args_t* args, void* cuda_stream);

/*
 * mepic_attn_decode_static - the same decode, for callers that cannot allocate device memory.
 * (The paper has no counterpart; this entry point exists for deployment reasons only.)
 *
 * Who needs it: code that runs where asking the device allocator for memory is not allowed or
 * cannot succeed - inside an allocator or memory-pool callback, in a serving plug-in whose host
 * process forbids device allocation after start-up, or when the page pool has already been given
 * all the free device memory - and therefore cannot produce the workspace mepic_attn_decode asks
 * for.  Here the split-KV partials go to an array built into the library instead:
 * MEPIC_DECODE_STATIC_SCRATCH_BYTES bytes of device memory that every GPU which uses the library's
 * decode module holds until the process exits.  The CUDA runtime loads a module lazily by default,
 * so the array comes into existence on a device when the first decode call of any kind
 * (mepic_attn_decode, mepic_attn_decode_static) is made there, not when the library is loaded: a
 * caller that is about to hand all remaining device memory to its page pool makes one such call
 * first (a one-request warm-up will do), or that first call fails with MEPIC_E_CUDA later.
 *
 * Arguments are those of mepic_attn_decode; args->workspace and args->workspace_bytes are ignored.
 * The call allocates nothing and frees nothing, on the host's device allocator or through any
 * library.  The first call on each device looks up the array's device address (a cheap runtime
 * query, done once per device with that device current); make that first call outside any stream
 * capture.  Limit: the config and batch must need no more than the array holds, i.e.
 * mepic_attn_decode_workspace(cfg, batch) <= MEPIC_DECODE_STATIC_SCRATCH_BYTES; otherwise the call
 * fails with MEPIC_E_INVAL and a message that states both numbers, and nothing is launched.
 * All calls on a device share the one array, and it keeps whatever the last call left in it.  No
 * part of it has to start at zero (every partial that is read has been written by the same call),
 * so nothing is cleared.  Two calls whose kernels overlap on the GPU (different streams, or
 * different threads of the process) race on the array and corrupt each other's results: serialise
 * them, or give one of them mepic_attn_decode with its own workspace.
 * Errors: as mepic_attn_decode, plus MEPIC_E_CUDA if the address query fails.
 */
#define MEPIC_DECODE_STATIC_SCRATCH_BYTES (8u << 20)
int32_t mepic_attn_decode_static(const mepic_config_t* cfg, const mepic_decode_args_t* args, void* cuda_stream);

/* ---------------------------------------------------------------- grouped decode (host plan + device)
 *
 * The same decode, aware of chunk sharing.  MEPIC lets many requests alias the physical pages of a
 * chunk (Section 3.2.2); mepic_attn_decode still reads such a page once per request.  The paper's
 * related-work section (operator-level acceleration: shared-prefix / shared-KV attention kernels)
 * names kernels that serve all the requests sharing a piece of context from one pass over it as the
 * layer to put under MEPIC; this pair of calls is that layer.  The result is the one
 * mepic_attn_decode defines (same formula, same tolerance); only the order of the work differs.
 *
 * mepic_decode_plan_build (HOST pointers, host work only, no device call when n_sms > 0) regroups
 * the block tables: every (request, table entry) pair is put in exactly one item = a group of at
 * most R = min(16 / G, 8) requests plus the pages all of them alias; pages nobody else uses, a
 * set's remainder of one request and a request's partly filled last page go to the request's own
 * single-request item.  The (item, kv head, 16-token tile) triples are laid on one line and cut in
 * equal pieces for n_sms * 8 workers (n_sms = 0: the SM count of the current device).  The plan is a
 * flat int32 buffer the caller treats as opaque, copies to the device as is, and also keeps on the
 * host.  It bakes in page ids, position bases and the number of table entries of every request; it
 * stays valid while kv_len grows inside each request's last page; when a request gains a page it is
 * patched (mepic_decode_plan_patch) or rebuilt, when the batch changes it is rebuilt (the device sets
 * MEPIC_DEV_BAD_PLAN otherwise and the result is then undefined but the call does not fault).  mepic_decode_plan_max_ints bounds the buffer size
 * for any tables of that shape.  Errors: E_INVAL (bad argument, kv_len < 1, entries > stride),
 * E_CAPACITY (buffer too small: *out_ints holds the need; or a batch beyond the plan's 32-bit
 * fields), E_CUDA (n_sms = 0 without a device).
 *
 * mepic_attn_decode_grouped: all pointers DEVICE pointers except plan_host (the host copy of the
 * same plan; its header is read during the call).  q, kv_len, q_pos, out, status, rope_table and the
 * pools are as for mepic_attn_decode; the block tables are not passed: the plan replaces them.
 * The rope table must cover position 16 (max_position >= 16).  workspace: at least
 * mepic_attn_decode_grouped_workspace() bytes, 16-byte aligned, contents overwritten; plan: 16-byte
 * aligned.  Errors as for mepic_attn_decode, plus E_INVAL for a plan built for another config/batch.
 */
size_t  mepic_decode_plan_max_ints(const mepic_config_t* cfg, int32_t batch, int32_t table_stride, int32_t n_sms);
int32_t mepic_decode_plan_build(const mepic_config_t* cfg, const int32_t* page_ids_host, const int32_t* pos_base_host,
                                const int32_t* kv_len_host, int32_t batch, int32_t table_stride, int32_t n_sms,
                                int32_t* out_plan_host, size_t cap_ints, size_t* out_ints);

/*
 * mepic_decode_plan_patch - keeps a plan alive across a page gain (the paper has no counterpart; a plan is this
 * library's).  In a decode loop every request gains a table entry each page_size tokens; instead of regrouping every
 * entry again, the request's new pages are appended to its own single-request item (the plan reserves room for 16
 * more pages per request, as far as table_stride lets the request grow) and everything that follows from the items'
 * sizes (places on the line, the cut, the workers' starts, the partial slots) is written again: host work of
 * O(items + workers).  plan_host (HOST, in/out): the plan as built; page_ids_host / pos_base_host / kv_len_host (HOST):
 * the tables as they are NOW (entries that existed at build time must be unchanged).  On MEPIC_OK out_ranges (HOST,
 * 4 x int64) holds *out_n_ranges (0 or 2) pairs {first int, number of ints} of plan_host that changed: copy exactly
 * those to the device copy.  The workspace the plan needs may have grown (mepic_attn_decode_grouped_workspace).
 * Errors: E_INVAL (bad argument, another config or batch, a request that lost pages), E_CAPACITY (a request has no
 * own item or its reserve is used up: build a new plan; nothing was changed).
 */
int32_t mepic_decode_plan_patch(const mepic_config_t* cfg, int32_t* plan_host, const int32_t* page_ids_host,
                                const int32_t* pos_base_host, const int32_t* kv_len_host, int32_t batch, int32_t table_stride,
                                int64_t* out_ranges, int32_t* out_n_ranges);

typedef struct {
  const void*    q;            /* bf16 [batch][n_q_heads][head_dim], un-rotated */
  const void*    k_pool;
  const void*    v_pool;
  const int32_t* plan;         /* device copy of the plan */
  const int32_t* plan_host;    /* host copy of the same plan */
  const int32_t* kv_len;       /* [batch] */
  const int32_t* q_pos;        /* [batch] */
  const float*   rope_table;
  void*          out;          /* bf16 [batch][n_q_heads][head_dim] */
  void*          workspace;
  size_t         workspace_bytes;
  int32_t*       status;
  int32_t        batch;
  float          sm_scale;
} mepic_decode_grouped_args_t;

size_t  mepic_attn_decode_grouped_workspace(const mepic_config_t* cfg, const int32_t* plan_host);
int32_t mepic_attn_decode_grouped(const mepic_config_t* cfg, const mepic_decode_grouped_args_t* args, void* cuda_stream);

/* ---------------------------------------------------------------- fp8 (e4m3) pages (device)
 *
 * KV-cache quantisation is named by the paper's related-work section as complementary and no format
 * is given; this is this build's: a pool of 8-bit pages [num_pages][n_kv_heads][page_size][head_dim]
 * of OCP E4M3 codes (1-4-3, bias 7, no infinities, largest finite value 448) plus one fp32 scale per
 * (page, kv head) block [num_pages][n_kv_heads], for K and for V separately.  Keys stay un-rotated.
 *
 * mepic_pages_quantize: for every page listed in pages (DEVICE int32[n_pages]) and every kv head,
 *     scale = max|x| / 448 over the block's elements that are not NaN (1 if that maximum is zero: a block of
 *             zeros, of NaN, or of both),
 *     code  = E4M3(x / scale), rounded to nearest, ties to even, saturating; a NaN element -> the NaN code 0x7F
 *             whatever its sign, -0 -> 0x80; an infinite element makes the scale infinite, so the block's finite
 *             elements encode to zero and the infinite ones to the NaN code,
 * computed in fp32 from the bf16 pool src_pool (DEVICE) into dst_pool and scales (DEVICE).  Call it
 * once for the K pools and once for the V pools.  A page id outside the pool sets MEPIC_DEV_BAD_PAGE
 * in *status and that block is skipped.  Errors: E_INVAL, E_CUDA.
 *
 * mepic_attn_decode_fp8: mepic_attn_decode over such pools: args->k_pool / v_pool are the 8-bit pools,
 * k_scales / v_scales (DEVICE) their scales; every other field, the workspace size included, is as for
 * mepic_attn_decode.  What is computed is that call's formula with K_t, V_t replaced by
 * value(code) * scale; the tolerance against the fp64 oracle evaluated on the same codes and scales
 * is that call's.  head_dim must be 128.  The queries are carried in fp16 after rotation and scaling
 * (|q| * sm_scale * log2(e) must stay below 65504).
 */
int32_t mepic_pages_quantize(const mepic_config_t* cfg, const void* src_pool, void* dst_pool, float* scales,
                             const int32_t* pages, int32_t n_pages, int32_t* status, void* cuda_stream);
int32_t mepic_attn_decode_fp8(const mepic_config_t* cfg, const mepic_decode_args_t* args, const float* k_scales,
                              const float* v_scales, void* cuda_stream);

/* ---------------------------------------------------------------- prefill (device)
 *
 * mepic_attn_prefill - Sections 3.3.1-3.3.3 for the rows a request recomputes (the first block of
 * every chunk plus its prompt segments).  Step 1 (commit, Section 3.3.2): row i's k_new / v_new
 * bits are written, un-rotated, to page page_ids[b][q_slot[i]/P], slot q_slot[i]%P of the pools.
 * Step 2: every new row attends causally, by logical slot, over slots 0..q_slot[i] of its
 * request's paged context (which now contains the committed rows), K rotated at each slot's
 * position and the row's q at the position of its own slot:
 *     out[i,h,:] = sum_{t <= q_slot[i]} softmax_t( sm_scale * < R(pos_{q_slot[i]}) q_new[i,h,:], R(pos_t) K_t > ) V_t .
 * bf16 tensor-core products, fp32 accumulation.
 *
 * Rows are grouped by request: rows row_offsets[b] .. row_offsets[b+1]-1 belong to request b and
 * their q_slot values are strictly ascending.  The caller guarantees that the slots named lie on
 * the request's PRIVATE pages (shared pages are never written by a correct caller; the library
 * cannot tell).  All struct pointers are DEVICE pointers except row_offsets_host (host copy of
 * row_offsets, batch+1 entries, read during the call for launch sizing).
 * workspace: mepic_attn_prefill_workspace() bytes, 16-byte aligned.  Each CTA derives its share of the work on the
 * device from row_offsets; nothing is built or uploaded by the call, which only enqueues kernels.  When the work
 * items fill at least one wave of the GPU that amount is 16 bytes.  When they do not (one request, say), each item's
 * key range is cut into up to eight shares, one CTA each, whose per-row partials (reference, sum, unnormalised
 * output: 4 (head_dim + 2) bytes per row, q head and share) go to the workspace and are merged by a third kernel;
 * given a smaller workspace the call runs one CTA per item instead.  Errors as for decode.
 * The attention kernel is enqueued twice.  The first launch expresses a tile's softmax weights against the reference
 * its rows agreed on earlier (one pass over the scores); that is exact as long as no score lies more than 2^64 above
 * the running reference, which a CTA notices from its row sums and records in the first word of the workspace (also
 * its only use of the first 16 bytes; the commit kernel clears it).  The second launch returns at once unless that
 * word is set, and otherwise does every item again with the reference found from the tile's own scores first (two
 * passes), overwriting the first launch's results; either way `out` holds the exact-softmax result when the call's
 * kernels have run.
 * A request may have no rows (row_offsets[b] == row_offsets[b+1]).  A call with no rows at all returns MEPIC_OK
 * without launching anything or reading any pointer but row_offsets_host.
 */
typedef struct {
  const void*    q_new;        /* bf16 [rows][n_q_heads][head_dim], un-rotated */
  const void*    k_new;        /* bf16 [rows][n_kv_heads][head_dim], un-rotated */
  const void*    v_new;        /* bf16 [rows][n_kv_heads][head_dim] */
  const int32_t* row_offsets;  /* [batch+1] */
  const int32_t* q_slot;       /* [rows] logical slot of each new row */
  void*          k_pool;       /* read and written (commit) */
  void*          v_pool;
  const int32_t* page_ids;     /* [batch][table_stride] */
  const int32_t* pos_base;     /* [batch][table_stride] */
  const int32_t* kv_len;       /* [batch] */
  const float*   rope_table;
  void*          out;          /* bf16 [rows][n_q_heads][head_dim] */
  void*          workspace;
  size_t         workspace_bytes;
  int32_t*       status;
  const int32_t* row_offsets_host;
  int32_t        table_stride;
  int32_t        batch;
  float          sm_scale;
} mepic_prefill_args_t;

size_t  mepic_attn_prefill_workspace(const mepic_config_t* cfg, int32_t batch, const int32_t* row_offsets_host);
int32_t mepic_attn_prefill(const mepic_config_t* cfg, const mepic_prefill_args_t* args, void* cuda_stream);

/* mepic_attn_decode_grouped_fp8: mepic_attn_decode_grouped over 8-bit pools (args->k_pool / v_pool are the e4m3 pools,
 * k_scales / v_scales (DEVICE) their scales); plan, workspace and every other field as for mepic_attn_decode_grouped,
 * what is computed and the tolerance as for mepic_attn_decode_fp8.  head_dim must be 128. */
int32_t mepic_attn_decode_grouped_fp8(const mepic_config_t* cfg, const mepic_decode_grouped_args_t* args, const float* k_scales,
                                      const float* v_scales, void* cuda_stream);

/*
 * mepic_attn_prefill_fp8 - mepic_attn_prefill over 8-bit (e4m3) pools: Sections 3.3.1-3.3.3 with the KV-cache
 * quantisation the paper's related-work section calls combinable.  args->k_pool / v_pool are the 8-bit pools
 * (format above), k_scales / v_scales (DEVICE, [num_pages][n_kv_heads] fp32) their scales; both are read and
 * WRITTEN; q_new / k_new / v_new / out stay bf16.  No bf16 copy of the pool is needed anywhere.
 * Step 1 (commit): row i's k_new / v_new go to page page_ids[b][q_slot[i]/P], slot q_slot[i]%P as codes.  A block's
 * scale belongs to the whole (page, kv head) block and pages fill from slot 0 upwards, so: if the call's rows for a
 * block include the block's slot 0 the call STARTS the block and sets its scale to the largest non-NaN magnitude of
 * the rows it writes there / 448 (1 if that is zero); otherwise it APPENDS: the block keeps its scale and the codes
 * saturate at +-448 x scale.  code = E4M3(x / scale), to nearest even, in fp32.  (The paper commits rows as they
 * are, Section 3.3.2; this rule is this library's.)  Step 2: the attention of mepic_attn_prefill with K_t, V_t
 * replaced by value(code) x scale, committed rows included; same tolerance against the fp64 oracle evaluated on the
 * same codes and scales.  head_dim must be 128.  Everything else (row grouping, workspace, splitting of small
 * grids, errors) is as for mepic_attn_prefill.
 */
int32_t mepic_attn_prefill_fp8(const mepic_config_t* cfg, const mepic_prefill_args_t* args, float* k_scales, float* v_scales,
                               void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MEPIC_H_ */
