// Prefill (selective recompute, Sections 3.3.1-3.3.3): commit the recomputed K/V rows
// un-rotated into their private pages, then let every new row attend causally over its
// request's paged context with RoPE applied to K on the way from the page pool to the
// tensor cores.
//
// Attention kernel.  One CTA per (request, kv head, 2 x 128/G query positions).  An M-tile
// packs QT = 128 / G query positions x the G query heads of the kv head into the 128 rows
// of one tcgen05 MMA (M = 128); a CTA carries two M-tiles, so one staged and rotated K/V
// tile serves 2 x G x QT rows and the tensor core always has the other M-tile's MMAs to
// run while one M-tile is in its softmax.  The CTA is warp specialised and pipelines
// 128-key tiles through a three-stage K ring and a two-stage V ring:
//   loader warps  : TMA (cp.async.bulk.tensor, 128-byte swizzle) brings the un-rotated K
//                   rows (one warp) and the V rows (another) of the tile's pages straight
//                   into the layout the MMA reads; one 16-row box per 16-token group and
//                   64-dim half.  A K stage is reused as soon as its QK^T has completed, a
//                   V stage once its PV has.
//   rotator warps : rotate the K tile IN PLACE in shared memory (fp32 math, bf16 storage).
//                   A thread walks CH consecutive keys of one 8-pair chunk and advances
//                   (cos, sin) by one position per key with a complex multiply, starting
//                   from the table row of its first key: 8 KB of table per tile, not 64.
//   MMA warp      : one thread issues, per M-tile, S = Q' K'^T (8 x tcgen05.mma 128x128x16
//                   into tensor memory) and O += P V (8 x 128 x D x 16), alternating the
//                   two M-tiles: PV_a(j), QK_a(j+1), PV_b(j), QK_b(j+1).
//   softmax warps : two warpgroups per M-tile; row r is shared by two threads, one per half of
//                   the tile's 128 score columns: tcgen05.ld the scores, causal mask by logical
//                   slot, online softmax in the log2 domain against a reference that both threads
//                   of the row share.  The first tile finds it from its own scores (the two
//                   threads meet on a hardware barrier of their two warps, values through shared
//                   memory); later tiles of the fast launch keep the reference they have and raise
//                   it one tile late, from the sums of P, without a meeting; a row that outruns it
//                   asks for the repeat launch, which finds it from every tile's own scores,
//                   P -> bf16 -> tensor memory (over the first columns of each half of the S
//                   buffer, from where the PV MMA takes it as its A operand); each rescales its
//                   half of the O columns in tensor memory when the reference moved; the
//                   epilogue writes O / l.
// Q' carries the rotation at the row's own position and sm_scale * log2(e).
// Every mbarrier wait is bounded; a wait that runs out raises an abort flag every role checks, and a softmax warp
// that leaves early releases its partner from the hardware barrier.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <cmath>
#include <cstring>

#include "mepic.h"
#include "mepic_internal.h"
#include "mepic_ptx.cuh"

namespace {

using namespace mepic_dev;

constexpr int kTileN = 128;            // keys per staged tile
constexpr int kBlockBytes = 128 * 128; // one [128 rows x 64 bf16] swizzled block
constexpr int kTmemCols = 512;         // S of M-tile a: 0..127, of b: 128..255; O of a: 256.., of b: 384..
constexpr int kSoftmaxWarps = 16;       // 2 M-tiles x 2 column halves x 4 lane quadrants: two threads share a row
constexpr int kRotatorWarps = 4;
// 8-bit pages: chunks / keys a converter / rotator thread takes from the staging buffer at a time.  Small batches: the
// codes are a shared-memory load away, and the shorter the unrolled bodies the better the roles that share a scheduler
// fit its instruction cache (batches of 16 / 4 measured 2.54 ms on config 3, 8 / 4 2.00, 2 / 4 1.79).
constexpr int kFp8VBatch = 2, kFp8KBatch = 4;
constexpr int kKLoaderWarp = 20, kVLoaderWarp = 21, kMmaWarp = 22, kSpareWarp = 23;   // the spare warp idles unless the pages are 8-bit
constexpr int kThreads = 768;
constexpr float kRescaleThreshold = 8.f;   // move the reference maximum only when it lags by 2^8
constexpr float kSaturation = 64.f;        // fast launch: a score more than this above the reference it was scaled by means "repeat"

struct Item { int32_t b, h, row0, nq; };   // rows row0 .. row0+nq-1 (global row indices) of request b

struct PrefillParams {
  const uint16_t* q_new;
  const uint16_t* k_new;
  const uint16_t* v_new;
  const int32_t* row_offsets;
  const int32_t* q_slot;
  uint16_t* k_pool;
  uint16_t* v_pool;
  const int32_t* page_ids;
  const int32_t* pos_base;
  const int32_t* kv_len;
  const float* rope;
  uint16_t* out;
  int32_t* status;
  int table_stride, batch, n_kv_heads, page_size, num_pages, max_position, total_rows;
  int max_q_tiles;      // most CTA-sized tiles of query positions any request has (launch sizing, from the host copy)
  int n_splits;         // CTAs per work item: each takes a contiguous share of the item's key tiles (1 = no split)
  float* part_o;        // n_splits > 1: [split][row][q head][D] unnormalised O of the share
  float* part_ml;       // n_splits > 1: [split][row][q head][2] = (reference maximum in log2 units, sum)
  float scale_log2;
  float* k_scales;      // 8-bit pools only: [num_pages][n_kv_heads] scale of each (page, kv head) block of K (the commit writes them)
  float* v_scales;      // ... and of V
  int32_t* redo_flag;   // first word of the workspace: set by a CTA of the fast launch one of whose rows outran its reference
  int exact;            // 0: the fast launch; 1: the repeat launch (two passes on every tile; returns at once unless *redo_flag); 2: two passes, unconditionally (test hook)
  int spin_limit;       // polls before a bounded wait gives up
  int skip_tile;        // test hook: CTA 0's K loader leaves out the copies of its key tile with this index (-1: none)
};

// packed fp32 pairs (one instruction for two lanes of work)
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{ .reg .b64 ra, rb, rc, rd;\n mov.b64 ra, {%2,%3};\n mov.b64 rb, {%4,%5};\n mov.b64 rc, {%6,%7};\n"
      " fma.rn.f32x2 rd, ra, rb, rc;\n mov.b64 {%0,%1}, rd; }"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
  float2 d;
  asm("{ .reg .b64 ra, rb, rd;\n mov.b64 ra, {%2,%3};\n mov.b64 rb, {%4,%5};\n mul.rn.f32x2 rd, ra, rb;\n mov.b64 {%0,%1}, rd; }"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {
  float2 d;
  asm("{ .reg .b64 ra, rb, rd;\n mov.b64 ra, {%2,%3};\n mov.b64 rb, {%4,%5};\n sub.rn.f32x2 rd, ra, rb;\n mov.b64 {%0,%1}, rd; }"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  float2 d;
  asm("{ .reg .b64 ra, rb, rd;\n mov.b64 ra, {%2,%3};\n mov.b64 rb, {%4,%5};\n add.rn.f32x2 rd, ra, rb;\n mov.b64 {%0,%1}, rd; }"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
__device__ __forceinline__ uint32_t bf16x2_sub(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// byte offset of 16-byte chunk `chunk` of row `row` inside a [rows x 128 B] block with the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int row, int chunk) { return static_cast<uint32_t>(row * 128 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait that also gives up when another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int limit) {
  for (int i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023) == 1023 && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicOr(status, MEPIC_DEV_WAIT_EXPIRED);
  return false;
}
// Same, with one answer for the whole warp (the callers run warp-collective instructions afterwards).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int limit) {
  const bool w = mbar_wait(bar, parity, abort_flag, status, limit);
  return __all_sync(0xffffffffu, w) != 0;
}
// ---- tcgen05 wrappers
__device__ __forceinline__ void tmem_alloc(uint32_t smem_slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate; one thread issues
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{ .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// same with A taken from tensor memory (row i of A in lane i, 16-bit elements packed two per column)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{ .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }"
               ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((addr & 0x3ffffu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
         (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// instruction descriptor: fp32 accumulator, bf16 A and B, M x N, majors (0 = K-major, 1 = MN-major)
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn_major) << 15) |
         (static_cast<uint32_t>(b_mn_major) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

#define TMEM_LD32(taddr, r, o)                                                                                        \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                            \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26," \
               "%27,%28,%29,%30,%31}, [%32];"                                                                       \
               : "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]),     \
                 "=r"(r[o + 6]), "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]),   \
                 "=r"(r[o + 12]), "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15]), "=r"(r[o + 16]),                \
                 "=r"(r[o + 17]), "=r"(r[o + 18]), "=r"(r[o + 19]), "=r"(r[o + 20]), "=r"(r[o + 21]),                \
                 "=r"(r[o + 22]), "=r"(r[o + 23]), "=r"(r[o + 24]), "=r"(r[o + 25]), "=r"(r[o + 26]),                \
                 "=r"(r[o + 27]), "=r"(r[o + 28]), "=r"(r[o + 29]), "=r"(r[o + 30]), "=r"(r[o + 31])                 \
               : "r"(taddr) : "memory")

#define TMEM_ST32(taddr, r, o)                                                                                        \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                                      \
               "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27," \
               "%28,%29,%30,%31,%32};"                                                                              \
               ::"r"(taddr), "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), \
                 "r"(r[o + 6]), "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]),         \
                 "r"(r[o + 12]), "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15]), "r"(r[o + 16]), "r"(r[o + 17]),     \
                 "r"(r[o + 18]), "r"(r[o + 19]), "r"(r[o + 20]), "r"(r[o + 21]), "r"(r[o + 22]), "r"(r[o + 23]),     \
                 "r"(r[o + 24]), "r"(r[o + 25]), "r"(r[o + 26]), "r"(r[o + 27]), "r"(r[o + 28]), "r"(r[o + 29]),     \
                 "r"(r[o + 30]), "r"(r[o + 31]) : "memory")

#define TMEM_ST16(taddr, r)                                                                                          \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" \
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),  \
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- commit (Section 3.3.2)
// One warp per new row (eight rows to a CTA): its K and V bits go, un-rotated, to (page, slot) of the pools.
constexpr int kCommitRows = 8;          // rows per CTA of the commit kernel, one warp each
__global__ void __launch_bounds__(kCommitRows * 32) mepic_prefill_commit(const PrefillParams p, int chunks_per_row) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the attention kernel may stage its queries meanwhile
  if (blockIdx.x == 0 && threadIdx.x == 0) *p.redo_flag = 0;       // (an attention CTA that could set it waits for this grid first)
  // a warp per row: the row's look-ups (request, slot, page) are a chain of dependent loads, and a CTA's eight chains
  // run side by side
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * kCommitRows + (threadIdx.x >> 5);
  if (row >= p.total_rows) return;
  int b = 0;
  while (b + 1 < p.batch && row >= p.row_offsets[b + 1]) ++b;
  const int slot = p.q_slot[row];
  if (slot < 0 || slot >= p.kv_len[b]) { if (lane == 0) atomicOr(p.status, MEPIC_DEV_BAD_SLOT); return; }
  const int page = p.page_ids[static_cast<size_t>(b) * p.table_stride + slot / p.page_size];
  if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { if (lane == 0) atomicOr(p.status, MEPIC_DEV_BAD_PAGE); return; }
  const int D8 = chunks_per_row / p.n_kv_heads;        // 16-byte chunks per head row
  for (int c = lane; c < chunks_per_row; c += 32) {
    const int h = c / D8, cc = c % D8;
    const size_t dst = (((static_cast<size_t>(page) * p.n_kv_heads + h) * p.page_size + slot % p.page_size) * D8 + cc);
    const size_t src = static_cast<size_t>(row) * chunks_per_row + c;
    reinterpret_cast<uint4*>(p.k_pool)[dst] = reinterpret_cast<const uint4*>(p.k_new)[src];
    reinterpret_cast<uint4*>(p.v_pool)[dst] = reinterpret_cast<const uint4*>(p.v_new)[src];
  }
}

// The same commit into 8-bit (e4m3) pages.  A block's scale belongs to the whole (page, kv head) block and pages fill
// from slot 0 upwards: a call whose rows for a block include its slot 0 starts the block and sets the scale from the rows
// it writes there (largest non-NaN magnitude / 448, 1 if zero); otherwise the call appends, the block keeps its scale
// and the codes saturate.  One CTA per new row; the first row of each run of rows that share a page does the run's work
// (a request's slots ascend, so a page's rows are neighbours), the others leave at once.
__device__ __forceinline__ uint32_t e4m3x4_of(float a, float b, float c, float d) {     // byte i = element i
  uint16_t lo, hi;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(b), "f"(a));
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(d), "f"(c));
  return static_cast<uint32_t>(lo) | (static_cast<uint32_t>(hi) << 16);
}
__global__ void __launch_bounds__(256) mepic_prefill_commit_fp8(const PrefillParams p, int head_dim) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int row = blockIdx.x;
  if (row == 0 && threadIdx.x == 0) *p.redo_flag = 0;
  __shared__ int sh_b;
  __shared__ unsigned sh_amax[2][8];         // [K | V][kv head], bit patterns of non-negative floats order like integers
  __shared__ float sh_scale[2][8];
  if (threadIdx.x == 0) {
    int b = 0;
    while (b + 1 < p.batch && row >= p.row_offsets[b + 1]) ++b;
    sh_b = b;
  }
  if (threadIdx.x < 16) sh_amax[threadIdx.x >> 3][threadIdx.x & 7] = 0u;
  __syncthreads();
  const int b = sh_b, P = p.page_size, kvl = p.kv_len[b];
  const int slot = p.q_slot[row];
  if (slot < 0 || slot >= kvl) { if (threadIdx.x == 0) atomicOr(p.status, MEPIC_DEV_BAD_SLOT); return; }
  const int e = slot / P;
  if (row > p.row_offsets[b]) {
    const int prev = p.q_slot[row - 1];
    if (prev >= 0 && prev < kvl && prev / P == e) return;         // not the first row of its page's run
  }
  const int page = p.page_ids[static_cast<size_t>(b) * p.table_stride + e];
  if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { if (threadIdx.x == 0) atomicOr(p.status, MEPIC_DEV_BAD_PAGE); return; }
  int n = 1;                                                      // rows of the run (at most one page's worth)
  const int row_end = p.row_offsets[b + 1];
  while (row + n < row_end && n < P) {
    const int s2 = p.q_slot[row + n];
    if (s2 < 0 || s2 >= kvl || s2 / P != e) break;
    ++n;
  }
  const bool fresh = slot % P == 0;
  const int H = p.n_kv_heads, D8 = head_dim / 8;                  // 16-byte chunks (8 bf16) per head row
  const int chunks = n * H * D8;
  const uint16_t* srcs[2] = {p.k_new, p.v_new};
  unsigned char* dsts[2] = {reinterpret_cast<unsigned char*>(p.k_pool), reinterpret_cast<unsigned char*>(p.v_pool)};
  float* scl[2] = {p.k_scales, p.v_scales};
  if (fresh) {
    for (int w = 0; w < 2; ++w)
      for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        const int r = c / (H * D8), h = (c / D8) % H;
        const uint4 v = *reinterpret_cast<const uint4*>(srcs[w] + (static_cast<size_t>(row + r) * H + h) * head_dim + 8 * (c % D8));
        const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
        float amax = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 f = bf16x2_to_float2(ww[k]);
          amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));       // fmaxf drops NaN operands: a NaN element does not set the scale
        }
        atomicMax(&sh_amax[w][h], __float_as_uint(amax));
      }
  }
  __syncthreads();
  if (threadIdx.x < 2 * H) {
    const int w = threadIdx.x / H, h = threadIdx.x % H;
    float sc;
    if (fresh) {
      const float amax = __uint_as_float(sh_amax[w][h]);
      sc = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
      scl[w][static_cast<size_t>(page) * H + h] = sc;
    } else {
      sc = scl[w][static_cast<size_t>(page) * H + h];
    }
    sh_scale[w][h] = sc;
  }
  __syncthreads();
  for (int w = 0; w < 2; ++w)
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
      const int r = c / (H * D8), h = (c / D8) % H, cc = c % D8;
      const uint4 v = *reinterpret_cast<const uint4*>(srcs[w] + (static_cast<size_t>(row + r) * H + h) * head_dim + 8 * cc);
      const float sc = sh_scale[w][h];
      const float2 f0 = bf16x2_to_float2(v.x), f1 = bf16x2_to_float2(v.y), f2 = bf16x2_to_float2(v.z), f3 = bf16x2_to_float2(v.w);
      uint2 out;
      out.x = e4m3x4_of(__fdiv_rn(f0.x, sc), __fdiv_rn(f0.y, sc), __fdiv_rn(f1.x, sc), __fdiv_rn(f1.y, sc));
      out.y = e4m3x4_of(__fdiv_rn(f2.x, sc), __fdiv_rn(f2.y, sc), __fdiv_rn(f3.x, sc), __fdiv_rn(f3.y, sc));
      const int in_page = p.q_slot[row + r] % P;
      *reinterpret_cast<uint2*>(dsts[w] + ((static_cast<size_t>(page) * H + h) * P + in_page) * head_dim + 8 * cc) = out;
    }
}

// The work item of CTA `i`, derived on the device from row_offsets alone (no list to build or upload).  Items are
// ordered heaviest first: level t = index of the tile of query positions inside its request, highest level first
// (later tiles see more keys); inside a level by request, then kv head.  Executed by one full warp.
__device__ __forceinline__ Item item_of_cta(const int32_t* row_offsets, int batch, int n_kv_heads, int qt, int max_q_tiles, int i, int lane) {
  Item it{0, 0, 0, 0};
  int before = 0;                                   // items of the levels above
  // row counts of the first 32 requests stay in registers: the level loop below would otherwise reload them
  const int r_first = lane < batch ? __ldg(row_offsets + lane) : 0;
  const int n_first = lane < batch ? __ldg(row_offsets + lane + 1) - r_first : 0;
  for (int t = max_q_tiles - 1; t >= 0; --t) {
    int cnt = 0;                                    // requests that have a tile at this level
    for (int b0 = 0; b0 < batch; b0 += 32) {
      const int b = b0 + lane;
      const int n = b0 == 0 ? n_first : (b < batch ? row_offsets[b + 1] - row_offsets[b] : 0);
      cnt += __popc(__ballot_sync(0xffffffffu, n > t * qt));
    }
    if (i < before + cnt * n_kv_heads) {
      const int j = i - before, want = j / n_kv_heads;      // the want-th such request, kv head j % n_kv_heads
      int seen = 0;
      for (int b0 = 0; b0 < batch; b0 += 32) {
        const int b = b0 + lane;
        const int n = b0 == 0 ? n_first : (b < batch ? row_offsets[b + 1] - row_offsets[b] : 0);
        const unsigned m = __ballot_sync(0xffffffffu, n > t * qt);
        const int here = __popc(m);
        if (want < seen + here) {
          unsigned mm = m;
          for (int k = 0; k < want - seen; ++k) mm &= mm - 1;     // drop the lower set bits
          const int src = __ffs(mm) - 1;
          const int bb = b0 + src;
          const int nn = __shfl_sync(0xffffffffu, n, src);
          it.b = bb; it.h = j % n_kv_heads;
          it.row0 = __shfl_sync(0xffffffffu, b0 == 0 ? r_first : (b < batch ? row_offsets[b] : 0), src) + t * qt;
          it.nq = min(qt, nn - t * qt);
          return it;
        }
        seen += here;
      }
    }
    before += cnt * n_kv_heads;
  }
  return it;       // not reached for i < number of items; nq = 0 makes the CTA do nothing
}

// ---------------------------------------------------------------- attention
constexpr int kKStages = 3;            // K ring depth (rotation runs ahead of the MMA)
constexpr int kVStages = 2;            // V ring depth

template <int D>
struct PrefillSmem {
  static constexpr int NB = D / 64;
  static constexpr int kQ = 0;                                     // two M-tiles of Q'
  static constexpr int kK = kQ + 2 * NB * kBlockBytes;
  static constexpr int kV = kK + kKStages * NB * kBlockBytes;
  static constexpr int kXchg = kV + kVStages * NB * kBlockBytes;   // float [2 M-tiles][2 halves][128 rows], then a byte each: the exchange of a row's two threads
  static constexpr int kBars = kXchg + 2 * 2 * 128 * 4 + 2 * 2 * 128;   // mbarriers and small state
  static constexpr int kBytes = kBars + 512;
};

// barrier indices inside the barrier block
constexpr int kBarKLanded = 0;                          // [kKStages] TMA bytes of a K stage
constexpr int kBarKReady = kBarKLanded + kKStages;      // [kKStages] K stage rotated
constexpr int kBarKFree = kBarKReady + kKStages;        // [kKStages] every QK^T that reads the stage is complete
constexpr int kBarVLanded = kBarKFree + kKStages;       // [kVStages] TMA bytes of a V stage
constexpr int kBarVFree = kBarVLanded + kVStages;       // [kVStages] every PV that reads the stage is complete
constexpr int kBarSFull = kBarVFree + kVStages;         // [2 M-tiles] S of the current tile is in tensor memory
constexpr int kBarPFull = kBarSFull + 2;                // [2] P of the current tile is in tensor memory
constexpr int kBarPvDone = kBarPFull + 2;               // [2] PV of the current tile complete
constexpr int kBarVPatched = kBarPvDone + 2;            // [1] rows past kv_len of the last V tile zeroed
constexpr int kBarQReady = kBarVPatched + 1;                // [1] Q' of both M-tiles is staged
constexpr int kBarDrain = kBarQReady + 1;                   // [1] after a lost wait: every MMA issued so far has completed
constexpr int kBarVReady = kBarDrain + 1;                   // [kVStages] 8-bit pages only: the V stage has been widened to bf16
constexpr int kNumBars = kBarVReady + kVStages;

// FP8 = the pools hold e4m3 codes with one scale per (page, kv head) block.  The tensor cores need bf16 operands in the
// swizzled layout, so the codes are widened on the way: the K ring has two stages, the third stage's room stages the raw
// codes of one K and one V tile, which the K loader warp brings with untiled bulk copies; the rotator warps read the K
// codes there, fold the block's scale into the rotation constants and write the bf16 stage the MMA reads, and two
// converter warps (the V loader, which has nothing to copy, and the spare warp) do the same for V.  Everything
// downstream of the stages is unchanged.
// HOOKS = the test build of the kernel: the poll limit of the bounded waits and the one left-out K tile come from the
// launch parameters (mepic_kernel_test_hooks).  The production instantiation has the limit as a compile-time constant
// and no such check: the issuing thread's wait loops are on the critical path of every tile (measured: 2 % of the call).
template <int D, int G, bool FP8, bool HOOKS>
__global__ void __launch_bounds__(kThreads, 1)
mepic_prefill_attn(const PrefillParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  using L = PrefillSmem<D>;
  constexpr int NB = D / 64;              // 64-dim blocks per row
  constexpr int QT = 128 / G;             // query positions per M-tile
  constexpr int CH = D / 16;              // (lo, hi) chunk pairs per row: chunk c pairs dims [8c,8c+8) with [D/2+8c, ...)
  constexpr uint32_t kIdescQK = instr_desc(128, kTileN, 0, 0);
  constexpr uint32_t kIdescPV = instr_desc(128, D, 0, 1);
  constexpr uint32_t kGroupBytes = 16u * D * 2u;        // the rows of one 16-token group in one pool
  // 8-bit pages: the K ring has two stages and the third stage's 32 KB stage the raw codes of one K tile and one V tile
  // (16 KB each, [key][128 bytes]), brought by bulk copies; the barriers of the unused K / V "landed" slots serve them
  constexpr int KD = FP8 ? 2 : kKStages;                // depth of the bf16 K ring
  constexpr uint32_t kCodeGroupBytes = 16u * 128u;      // the codes of one 16-token group

  // 1024-byte alignment: the swizzle pattern is a function of the address bits (checked below; there is no slack left)
  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn;
  unsigned char* Qs = smem + L::kQ;
  unsigned char* Ks = smem + L::kK;
  unsigned char* Vs = smem + L::kV;
  float* xchg = reinterpret_cast<float*>(smem + L::kXchg);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBars);
  const uint32_t bar0 = smem_u32(bars);
  auto BAR = [&](int which, int slot) { return bar0 + static_cast<uint32_t>((which + slot) * 8); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + kNumBars + 1);
  volatile int* gbase = reinterpret_cast<volatile int*>(bars + kNumBars + 2);   // [kKStages][8] position of each 16-key group's first key
  volatile float* kscl = reinterpret_cast<volatile float*>(bars + kNumBars + 18);   // 8-bit pages: [2][8] scale of each group's K block, by tile parity
  volatile float* vscl = reinterpret_cast<volatile float*>(bars + kNumBars + 30);   // ... and of its V block
  unsigned char* Kc = Ks + 2 * NB * kBlockBytes;            // 8-bit pages: staged K codes of one tile (the third K stage's room)
  unsigned char* Vc = Kc + 128 * 128;                       // ... and V codes
  const uint32_t bar_kc_landed = BAR(kBarKLanded, 0), bar_kc_free = BAR(kBarKLanded, 1);   // 8-bit pages: staging full / read out
  const uint32_t bar_vc_landed = BAR(kBarVLanded, 0), bar_vc_free = BAR(kBarVLanded, 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int spin = HOOKS ? p.spin_limit : kSpinLimit;
  if (p.exact == 1) {
    // the repeat launch: nothing to do unless a CTA of the fast launch asked for it (then every item is done again)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (*reinterpret_cast<volatile int32_t*>(p.redo_flag) == 0) return;
  }
  volatile int* sat_flag = reinterpret_cast<volatile int*>(bars + kNumBars + 14);   // fast launch: a row outran its reference
  Item* item_slot = reinterpret_cast<Item*>(bars + kNumBars + 16);
  if (warp == 1) {
    const Item it = item_of_cta(p.row_offsets, p.batch, p.n_kv_heads, 2 * QT, p.max_q_tiles, blockIdx.x / p.n_splits, lane);
    if (lane == 0) *item_slot = it;
  }
  __syncthreads();
  const Item item = *item_slot;
  if (item.nq <= 0) return;
  const int b = item.b, h = item.h;
  const int kvl = p.kv_len[b];
  const int32_t* ids = p.page_ids + static_cast<size_t>(b) * p.table_stride;
  const int32_t* bases = p.pos_base + static_cast<size_t>(b) * p.table_stride;
  const int n_q_heads = p.n_kv_heads * G;

  if ((smem_u32(smem) & 1023u) != 0) {       // cannot happen with the alignment requested above; never run misaligned
    if (tid == 0) atomicOr(p.status, MEPIC_DEV_WAIT_EXPIRED);
    return;
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  if (tid == 32) {
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(BAR(kBarKLanded, s), (FP8 && s == 1) ? kRotatorWarps * 32 : 1);   // loader's expect_tx + TMA bytes (8-bit pages: slot 1 = K codes read out)
      mbar_init(BAR(kBarKReady, s), kRotatorWarps * 32);
      mbar_init(BAR(kBarKFree, s), 1);                       // tcgen05.commit
    }
    for (int s = 0; s < kVStages; ++s) {
      mbar_init(BAR(kBarVLanded, s), (FP8 && s == 1) ? 2 * 32 : 1);                   // (8-bit pages: slot 1 = V codes read out by the two converter warps)
      mbar_init(BAR(kBarVFree, s), 1);                       // tcgen05.commit
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(BAR(kBarSFull, s), 1);                       // tcgen05.commit
      mbar_init(BAR(kBarPFull, s), 256);                     // the M-tile's two softmax warpgroups
      mbar_init(BAR(kBarPvDone, s), 1);                      // tcgen05.commit
    }
    mbar_init(BAR(kBarVPatched, 0), 1);
    mbar_init(BAR(kBarQReady, 0), kSoftmaxWarps * 32);      // the softmax warps stage Q'
    mbar_init(BAR(kBarDrain, 0), 1);                         // tcgen05.commit
    for (int s = 0; s < kVStages; ++s) mbar_init(BAR(kBarVReady, s), 2 * 32);            // the two V converter warps
    *abort_flag = 0;
    *sat_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }

  // key tiles each M-tile needs: up to the causal limit of its last live row (rows ascend by slot)
  int lim[2], nt[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    const int last_q = min((x + 1) * QT, item.nq) - 1;            // last live position of M-tile x, or < x*QT when it has none
    if (last_q < x * QT) { lim[x] = -1; nt[x] = 0; continue; }
    int l = p.q_slot[item.row0 + last_q];
    l = l < 0 ? 0 : (l >= kvl ? kvl - 1 : l);
    lim[x] = l;
    nt[x] = l / kTileN + 1;
  }
  // With few work items (a single request, say) each item is cut into n_splits CTAs so that the grid still fills
  // the GPU: this CTA takes key tiles [tile_base, tile_base + n_tiles) of the item's n_all and leaves a partial
  // (reference, sum, unnormalised O) per row that a second kernel merges.  From here on nt[] and n_tiles count
  // this CTA's tiles.
  const int n_all = nt[1] > nt[0] ? nt[1] : nt[0];
  const int split = blockIdx.x % p.n_splits;
  const int tile_base = static_cast<int>(static_cast<long long>(n_all) * split / p.n_splits);
  const int tile_end = static_cast<int>(static_cast<long long>(n_all) * (split + 1) / p.n_splits);
#pragma unroll
  for (int x = 0; x < 2; ++x) nt[x] = min(max(nt[x], tile_base), tile_end) - tile_base;
  const int n_tiles = tile_end - tile_base;
  const bool last_has_tail = n_tiles > 0 && tile_end == n_all && n_all * kTileN > kvl;

  tc_fence_before();
  __syncthreads();             // barriers initialised, tensor memory allocated
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // ---- stage Q (the softmax warps; meanwhile the loaders and rotators already work on the first key tiles):
  // rotate each row at its own position, fold in sm_scale*log2e, round to bf16
  if (warp < kSoftmaxWarps) {
  for (int task = tid; task < 256 * CH; task += kSoftmaxWarps * 32) {
    const int rr2 = task / CH, c = task % CH;
    const int x = rr2 >> 7, rr = rr2 & 127;
    const int qq = x * QT + rr / G, gg = rr % G;
    uint32_t lo_w[4] = {0, 0, 0, 0}, hi_w[4] = {0, 0, 0, 0};
    if (rr < QT * G && qq < item.nq) {
      const int row = item.row0 + qq;
      int slot = p.q_slot[row];
      slot = slot < 0 ? 0 : (slot >= kvl ? kvl - 1 : slot);
      int pos = bases[slot / p.page_size] + slot % p.page_size;
      if (pos < 0 || pos > p.max_position) { atomicOr(p.status, MEPIC_DEV_BAD_POSITION); pos = pos < 0 ? 0 : p.max_position; }
      const uint16_t* src = p.q_new + (static_cast<size_t>(row) * n_q_heads + static_cast<size_t>(h) * G + gg) * D;
      const uint4 lo = *reinterpret_cast<const uint4*>(src + 8 * c);
      const uint4 hi = *reinterpret_cast<const uint4*>(src + D / 2 + 8 * c);
      const float4* cs = reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(pos) * D + 16 * c);
      const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w}, hw[4] = {hi.x, hi.y, hi.z, hi.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 t = __ldg(cs + j);       // (cos, sin) of pairs 8c+2j and 8c+2j+1
        const float2 a = bf16x2_to_float2(lw[j]), bq = bf16x2_to_float2(hw[j]);
        const float l0 = (a.x * t.x - bq.x * t.y) * p.scale_log2, h0 = (a.x * t.y + bq.x * t.x) * p.scale_log2;
        const float l1 = (a.y * t.z - bq.y * t.w) * p.scale_log2, h1 = (a.y * t.w + bq.y * t.z) * p.scale_log2;
        lo_w[j] = pack_bf16x2(l0, l1);
        hi_w[j] = pack_bf16x2(h0, h1);
      }
    }
    // chunk index within the row: lo chunk = c, hi chunk = CH + c ; 8 chunks per 64-dim block
    const int lc = c, hc = CH + c;
    unsigned char* Qx = Qs + x * NB * kBlockBytes;
    *reinterpret_cast<uint4*>(Qx + (lc / 8) * kBlockBytes + sw128(rr, lc % 8)) = make_uint4(lo_w[0], lo_w[1], lo_w[2], lo_w[3]);
    *reinterpret_cast<uint4*>(Qx + (hc / 8) * kBlockBytes + sw128(rr, hc % 8)) = make_uint4(hi_w[0], hi_w[1], hi_w[2], hi_w[3]);
  }
  fence_async_smem();          // Q is read by the tensor core (async proxy)
  mbar_arrive(BAR(kBarQReady, 0));
  }

  if (warp < kSoftmaxWarps) {
    // =============================================================== softmax warps
    // Row r of M-tile x is shared by two threads (same tensor-memory lane, warps w and w + 4 of the M-tile's
    // eight): one takes the scores of keys 0..63 of the tile, the other keys 64..127.  They agree on the row's
    // reference maximum through shared memory once per tile; everything else is private.
    const int x = warp >> 3;                      // M-tile
    const int ch = (warp >> 2) & 1;               // column half
    const int q4 = warp & 3;                      // lane quadrant of tensor memory
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q4 * 32) << 16);
    const uint32_t t_H = t_row + static_cast<uint32_t>(x * 128 + ch * 64);     // my 64 score columns; P goes over the first 32
    const uint32_t t_O = t_row + 256u + static_cast<uint32_t>(x * 128 + ch * (D / 2));   // my half of the row's O columns
    const int r = q4 * 32 + lane;
    const int qi = x * QT + r / G, g = r % G;
    const bool row_live = (r < QT * G) && (qi < item.nq);
    int limit = lim[x];
    if (row_live) {
      limit = p.q_slot[item.row0 + qi];
      if (limit < 0 || limit >= kvl) { atomicOr(p.status, MEPIC_DEV_BAD_SLOT); limit = limit < 0 ? 0 : kvl - 1; }
    }
    // exchange slots of the row's two threads.  2 KB: the fp32 maximum of a two-pass tile, one word per thread.  512
    // bytes after them: one byte per thread that tells the partner, one tile later and without a meeting, how far the
    // thread's sum of P over a tile ran ahead of the reference: two 4-bit codes, low nibble for even tiles, high nibble
    // for odd ones (the owner keeps the byte in a register and stores all of it, so a tile's code stays readable until
    // the tile after next overwrites it).
    volatile float* mine = xchg + (x * 2 + ch) * 128 + r;
    const volatile float* theirs = xchg + (x * 2 + (ch ^ 1)) * 128 + r;
    volatile unsigned char* lz_mine = reinterpret_cast<volatile unsigned char*>(xchg + 512) + (x * 2 + ch) * 128 + r;
    const volatile unsigned char* lz_theirs = reinterpret_cast<const volatile unsigned char*>(xchg + 512) + (x * 2 + (ch ^ 1)) * 128 + r;
    const int pair_id = 1 + x * 4 + q4;         // hardware barrier of the two warps that share these 32 rows (0 is the CTA's)
    // publish `v`, meet the partner warp, return the partner's value of the same row.  The meeting point is a
    // hardware barrier (a waiting warp takes no issue slots and wakes at once); it has no time limit of its own, so
    // a warp that leaves this role early after a lost wait arrives on it once (below) and every warp looks at the
    // abort flag, which is raised before that arrival, as soon as it is through.
    auto swap_with_partner = [&](float v, bool& ok_io, float* dst, const float* src) {
      *dst = v;
      asm volatile("bar.sync %0, 64;" ::"r"(pair_id) : "memory");
      if (*abort_flag) ok_io = false;
      return *src;
    };
    // the row's maximum over both halves.  (The partner reads this thread's word right after the meeting; the word
    // is next written in a later two-pass tile, after an S that was issued once both threads had handed P over.)
    auto row_max_of = [&](float v, bool& ok_io) {
      *mine = v;
      asm volatile("bar.sync %0, 64;" ::"r"(pair_id) : "memory");
      if (*abort_flag) ok_io = false;
      return fmaxf(v, *theirs);
    };
    // The reference 2^m_ref that P is expressed in only has to be the same for both threads of the row, not far above
    // the row's maximum so far (else every P of a row could vanish) and close enough below the scores for P to stay in
    // range.  The first tile finds it in a pass of its own over the scores and a meeting of the two threads (two
    // passes).  In the fast launch later tiles make one pass with the reference they have; what tells them to raise it
    // is the sum of P of the tile before: a thread whose sum exceeds 2^8 leaves the code c = ceil((floor(log2(sum)) + 1)
    // / 8) in shared memory before it hands P over, and reads its partner's at the next tile (the hand-over, the MMA
    // and the next S order the two); 8 max(c, c') added to the reference puts it above every score of that tile by
    // less than 16.  A thread whose sum reaches 2^kSaturation (or overflows) raises sat_flag: the call then repeats
    // every item with two passes on every tile (the repeat launch).
    float m_ref = -INFINITY, m_next = -INFINITY, l_run = 0.f;
    int c_prev = 0;                               // my code for the tile before
    uint32_t lz_byte = 0;                         // my byte of codes as it stands in shared memory
    bool ok = true;
    const int my_tiles = nt[x];
    for (int tile = 0; tile < my_tiles; ++tile) {
      if (!mbar_wait_warp(BAR(kBarSFull, x), static_cast<uint32_t>(tile) & 1u, abort_flag, p.status, spin)) { ok = false; break; }
      tc_fence_after();
      const int n_vis = limit - (tile_base + tile) * kTileN + 1 - 64 * ch;     // my columns [0, n_vis) are visible to this row
      const bool boundary = n_vis < 64;                          // only the tile(s) on the causal boundary need the mask
      // two passes: the repeat launch, the first tile, and any tile at which a row of this warp has no reference yet
      // (both warps of the pair hold the same rows and the same references: they decide alike)
      if (!p.exact && tile > 0) {
        const int c = max(c_prev, (static_cast<int>(*lz_theirs) >> (4 * ((tile - 1) & 1))) & 15);
        if (c > 0 && m_ref != -INFINITY) m_next = m_ref + static_cast<float>(8 * c);
      }
      const bool two_pass = p.exact || tile == 0 || __any_sync(0xffffffffu, m_next == -INFINITY);
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      float alpha = 1.f;
      if (two_pass) {
        // ---- pass 1: maximum of my 64 scores
        uint32_t sv[64];                  // both loads in flight at once: one wait
        TMEM_LD32(t_H, sv, 0);
        TMEM_LD32(t_H + 32, sv, 32);
        tmem_wait_ld();
        if (boundary) {
#pragma unroll
          for (int c = 0; c < 64; ++c) sv[c] = c < n_vis ? sv[c] : 0xff800000u;   // -inf
        }
#pragma unroll
        for (int c = 0; c < 64; c += 4) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mx4[k] = fmaxf(mx4[k], __uint_as_float(sv[c + k]));
        }
        const float mx = row_max_of(fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])), ok);
        if (!ok) break;
        // move the reference only when it lags by more than the threshold (both threads of the row decide alike);
        // always true on the first tile that shows the row a key
        const float m_new = mx > m_next + kRescaleThreshold ? mx : m_next;      // m_next >= m_ref: a raise still pending
        if (m_new != m_ref) {
          alpha = ex2(m_ref - m_new);
          m_ref = m_new;
        }
        m_next = m_ref;
      } else if (m_next != m_ref) {
        alpha = ex2(m_ref - m_next);
        m_ref = m_next;
      }
      // O holds every earlier tile's PV, all complete: this tile's S was issued after them.  Each thread of the
      // row rescales its own half of the O columns.
      if (tile > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
        for (int cb = 0; cb < D / 2; cb += 32) {
          uint32_t o[32];
          TMEM_LD32(t_O + cb, o, 0);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          TMEM_ST32(t_O + cb, o, 0);
        }
      }
      // ---- pass 2: P = 2^(S - reference) as bf16 pairs over the first 32 of my 64 columns
      float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      // a row none of whose keys lies in this CTA's share so far still has m_ref = -inf: every score is masked
      // (-inf) and must give P = 0, not 2^(-inf + inf)
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      const float2 ref2 = make_float2(m_use, m_use);
#pragma unroll 1
      for (int q = 0; q < 2; ++q) {
        uint32_t sv[32], pw[16];
        TMEM_LD32(t_H + 32 * q, sv, 0);
        tmem_wait_ld();
        if (boundary) {
#pragma unroll
          for (int c = 0; c < 32; ++c) sv[c] = (32 * q + c) < n_vis ? sv[c] : 0xff800000u;   // -inf -> P = 0
        }
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          const float2 d0 = sub2(make_float2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), ref2);
          const float2 d1 = sub2(make_float2(__uint_as_float(sv[c + 2]), __uint_as_float(sv[c + 3])), ref2);
          const float2 p0 = make_float2(ex2(d0.x), ex2(d0.y)), p1 = make_float2(ex2(d1.x), ex2(d1.y));
          sum2[0] = add2(sum2[0], p0);
          sum2[1] = add2(sum2[1], p1);
          pw[c / 2] = pack_bf16x2(p0.x, p0.y);
          pw[c / 2 + 1] = pack_bf16x2(p1.x, p1.y);
        }
        TMEM_ST16(t_H + 16 * q, pw);      // chunk q's P over columns that hold only consumed scores
      }
      const float l_tile = (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
      l_run = l_run * alpha + l_tile;
      {
        const int e = static_cast<int>((__float_as_uint(l_tile) >> 23) & 0xffu);       // floor(log2(sum)) + 127
        c_prev = e > 127 + static_cast<int>(kRescaleThreshold) ? min(15, (e - 126 + 7) >> 3) : 0;
        lz_byte = (tile & 1) ? (lz_byte & 0x0fu) | (static_cast<uint32_t>(c_prev) << 4) : (lz_byte & 0xf0u) | static_cast<uint32_t>(c_prev);
        *lz_mine = static_cast<unsigned char>(lz_byte);
      }
      if (!(l_tile < 1.8446744e19f)) *sat_flag = 1;             // 2^64 and beyond, inf or NaN: repeat (the repeat launch never gets here with such a sum)
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(BAR(kBarPFull, x));
    }
    // ---- epilogue once the last PV has completed; each thread of the row writes its half of the head dims:
    // out = O / l, or (when the item is split) this share's unnormalised O with its reference and sum
    if (p.n_splits > 1 && my_tiles == 0 && row_live && ch == 0) {
      const size_t at = (static_cast<size_t>(split) * p.total_rows + item.row0 + qi) * n_q_heads + static_cast<size_t>(h) * G + g;
      *reinterpret_cast<float2*>(p.part_ml + at * 2) = make_float2(-INFINITY, 0.f);      // nothing of this row in the share
    }
    if (ok && my_tiles > 0) {
      // The row sums go through a second pair of slots: the partner may not have read this thread's last maximum yet
      // (nothing orders that read before this write, unlike inside the loop, where the next write follows a QK^T that
      // was issued after both threads handed P over).  The M-tile's Q' block is free by now: its last QK^T has completed.
      float* ep = reinterpret_cast<float*>(Qs + x * NB * kBlockBytes);
      const float l_tot = l_run + swap_with_partner(l_run, ok, ep + ch * 128 + r, ep + (ch ^ 1) * 128 + r);
      if (ok) ok = mbar_wait_warp(BAR(kBarPvDone, x), static_cast<uint32_t>(my_tiles - 1) & 1u, abort_flag, p.status, spin);
      if (ok) {
        tc_fence_after();
        const size_t rh = static_cast<size_t>(item.row0 + qi) * n_q_heads + static_cast<size_t>(h) * G + g;
        if (p.n_splits == 1) {
          const float inv = 1.f / l_tot;
          uint16_t* dst = p.out + rh * D + ch * (D / 2);
#pragma unroll 1
          for (int cb = 0; cb < D / 2; cb += 32) {
            uint32_t o[32];
            TMEM_LD32(t_O + cb, o, 0);
            tmem_wait_ld();
            if (row_live) {
#pragma unroll
              for (int c = 0; c < 32; c += 8) {
                uint4 w;
                w.x = pack_bf16x2(__uint_as_float(o[c + 0]) * inv, __uint_as_float(o[c + 1]) * inv);
                w.y = pack_bf16x2(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
                w.z = pack_bf16x2(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
                w.w = pack_bf16x2(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
                *reinterpret_cast<uint4*>(dst + cb + c) = w;
              }
            }
          }
        } else {
          const size_t at = static_cast<size_t>(split) * p.total_rows * n_q_heads + rh;
          float* dst = p.part_o + at * D + ch * (D / 2);
          if (row_live && ch == 0) *reinterpret_cast<float2*>(p.part_ml + at * 2) = make_float2(m_ref, l_tot);
#pragma unroll 1
          for (int cb = 0; cb < D / 2; cb += 32) {
            uint32_t o[32];
            TMEM_LD32(t_O + cb, o, 0);
            tmem_wait_ld();
            if (row_live) {
#pragma unroll
              for (int c = 0; c < 32; c += 4) *reinterpret_cast<uint4*>(dst + cb + c) = make_uint4(o[c], o[c + 1], o[c + 2], o[c + 3]);
            }
          }
        }
      }
    }
    if (!ok) asm volatile("bar.arrive %0, 64;" ::"r"(pair_id) : "memory");   // never leave the partner at the barrier
  } else if (warp < kSoftmaxWarps + kRotatorWarps) {
    // =============================================================== rotator warps: K tile, in place
    const int rt = tid - kSoftmaxWarps * 32;     // 0..127
    const int c = rt % CH;                       // chunk pair: dims [8c, 8c+8) and [D/2+8c, ...)
    const int k0 = (rt / CH) * CH;               // first of this thread's CH consecutive keys
    // one-position step of this chunk's 8 pairs: table row 1, as packed pairs (cos, sin, -sin)
    float2 c1[4], s1[4], ns1[4];
    {
      const float4* row1 = reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(1) * D + 16 * c);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 t = __ldg(row1 + j);
        c1[j] = make_float2(t.x, t.z); s1[j] = make_float2(t.y, t.w); ns1[j] = make_float2(-t.y, -t.w);
      }
    }
    const int lc = c, hc = CH + c;
    for (int tile = 0; tile < n_tiles; ++tile) {
      const int st = tile % KD;
      const uint32_t ph = static_cast<uint32_t>(tile / KD) & 1u;
      if constexpr (FP8) {
        // the tile's codes are staged, and (this role writes the bf16 stage itself) every QK^T that read the stage's
        // previous tenant has completed
        if (!mbar_wait(bar_kc_landed, static_cast<uint32_t>(tile) & 1u, abort_flag, p.status, spin)) break;
        if (tile >= KD && !mbar_wait(BAR(kBarKFree, st), static_cast<uint32_t>(tile / KD - 1) & 1u, abort_flag, p.status, spin)) break;
      } else {
        if (!mbar_wait(BAR(kBarKLanded, st), ph, abort_flag, p.status, spin)) break;
      }
      unsigned char* Kb = Ks + st * NB * kBlockBytes;
      const int key0 = (tile_base + tile) * kTileN;
      int pos = gbase[(FP8 ? (tile & 1) : st) * 8 + k0 / 16] + (k0 & 15);
      if (pos < 0 || pos > p.max_position) {
        if (key0 + k0 < kvl) atomicOr(p.status, MEPIC_DEV_BAD_POSITION);
        pos = 0;
      }
      float2 cc[4], ss[4];
      {
        const float4* row = reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(pos) * D + 16 * c);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 t = __ldg(row + j);
          cc[j] = make_float2(t.x, t.z); ss[j] = make_float2(t.y, t.w);
        }
      }
      if constexpr (FP8) {
        // ---- 8-bit pages: codes from the staging buffer, widened exactly, rotated in fp32 with the block's scale
        // folded into (cos, sin) (the one-position step is a pure rotation, so the factor rides along), rounded to
        // bf16 once.  A group with no key below kv_len was not copied: its rows become zero.
        const bool have = key0 + (k0 & ~15) < kvl;
        const unsigned char* src0 = Kc + k0 * 128;
        if (have) {
          const float sc = kscl[(tile & 1) * 8 + k0 / 16];
#pragma unroll
          for (int j = 0; j < 4; ++j) { cc[j].x *= sc; cc[j].y *= sc; ss[j].x *= sc; ss[j].y *= sc; }
        }
#pragma unroll 1
        for (int i0 = 0; i0 < CH; i0 += kFp8KBatch) {
          uint2 lo8[kFp8KBatch], hi8[kFp8KBatch];
#pragma unroll
          for (int u = 0; u < kFp8KBatch; ++u) {
            lo8[u] = have ? *reinterpret_cast<const uint2*>(src0 + (i0 + u) * 128 + 8 * c) : make_uint2(0, 0);
            hi8[u] = have ? *reinterpret_cast<const uint2*>(src0 + (i0 + u) * 128 + 64 + 8 * c) : make_uint2(0, 0);
          }
#pragma unroll
          for (int u = 0; u < kFp8KBatch; ++u) {
            const int kk = k0 + i0 + u;
            const uint32_t lw[2] = {lo8[u].x, lo8[u].y}, hw[2] = {hi8[u].x, hi8[u].y};
            uint32_t lo_w[4], hi_w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {          // pairs 8c + 2j, 8c + 2j + 1 = bytes 2j, 2j + 1 of the 8
              const uint16_t lb = static_cast<uint16_t>(lw[j >> 1] >> (16 * (j & 1))), hb = static_cast<uint16_t>(hw[j >> 1] >> (16 * (j & 1)));
              uint32_t lh, hh;
              asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(lh) : "h"(lb));
              asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(hh) : "h"(hb));
              const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&lh)), bq = __half22float2(*reinterpret_cast<const __half2*>(&hh));
              const float2 l = fma2(a, cc[j], mul2(bq, make_float2(-ss[j].x, -ss[j].y)));      // lo cos - hi sin
              const float2 hgh = fma2(a, ss[j], mul2(bq, cc[j]));                                // lo sin + hi cos
              lo_w[j] = pack_bf16x2(l.x, l.y);
              hi_w[j] = pack_bf16x2(hgh.x, hgh.y);
            }
            *reinterpret_cast<uint4*>(Kb + (lc / 8) * kBlockBytes + sw128(kk, lc % 8)) = make_uint4(lo_w[0], lo_w[1], lo_w[2], lo_w[3]);
            *reinterpret_cast<uint4*>(Kb + (hc / 8) * kBlockBytes + sw128(kk, hc % 8)) = make_uint4(hi_w[0], hi_w[1], hi_w[2], hi_w[3]);
            if (i0 + u + 1 < CH) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float2 cn = fma2(ss[j], ns1[j], mul2(cc[j], c1[j]));
                ss[j] = fma2(ss[j], c1[j], mul2(cc[j], s1[j]));
                cc[j] = cn;
              }
            }
          }
        }
        fence_async_smem();
        mbar_arrive(BAR(kBarKReady, st));
        mbar_arrive(bar_kc_free);    // the staged codes have been read: the next tile's may come
        continue;                    // (the V tile is the V converters' work)
      }
#pragma unroll 2
      for (int i = 0; i < CH; ++i) {
        const int kk = k0 + i;
        uint4* plo = reinterpret_cast<uint4*>(Kb + (lc / 8) * kBlockBytes + sw128(kk, lc % 8));
        uint4* phi = reinterpret_cast<uint4*>(Kb + (hc / 8) * kBlockBytes + sw128(kk, hc % 8));
        const uint4 lo = *plo, hi = *phi;
        const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w}, hw[4] = {hi.x, hi.y, hi.z, hi.w};
        uint32_t lo_w[4], hi_w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          // packed bf16 arithmetic: the result is rounded to bf16 for the MMA anyway, and two elements rotate per
          // instruction without being widened first; cos/sin are carried in fp32 and rounded once per key
          const uint32_t cb = pack_bf16x2(cc[j].x, cc[j].y), sb = pack_bf16x2(ss[j].x, ss[j].y);
          lo_w[j] = bf16x2_sub(bf16x2_mul(lw[j], cb), bf16x2_mul(hw[j], sb));      // lo cos - hi sin
          hi_w[j] = bf16x2_fma(lw[j], sb, bf16x2_mul(hw[j], cb));                  // lo sin + hi cos
        }
        *plo = make_uint4(lo_w[0], lo_w[1], lo_w[2], lo_w[3]);
        *phi = make_uint4(hi_w[0], hi_w[1], hi_w[2], hi_w[3]);
        if (i + 1 < CH) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {          // (cos, sin)(pos+1) = (cos, sin)(pos) x (cos, sin)(1)
            const float2 cn = fma2(ss[j], ns1[j], mul2(cc[j], c1[j]));
            ss[j] = fma2(ss[j], c1[j], mul2(cc[j], s1[j]));
            cc[j] = cn;
          }
        }
      }
      fence_async_smem();
      mbar_arrive(BAR(kBarKReady, st));
    }
  } else if (FP8 && (warp == kVLoaderWarp || warp == kSpareWarp)) {
    // =============================================================== 8-bit pages: the V converters
    // The V loader (which has nothing to copy: the K loader stages the codes of both pools) and the spare warp widen
    // the V tile, 64 keys each: codes from the staging buffer, times the block's scale, rounded to bf16 into the stage
    // the PV MMA reads; rows at or past kv_len become zero (P is 0 there, but 0 x NaN is NaN).
    const int half = warp == kVLoaderWarp ? 0 : 1;
    for (int tile = 0; tile < n_tiles; ++tile) {
      const int vst = tile % kVStages;
      if (!mbar_wait_warp(bar_vc_landed, static_cast<uint32_t>(tile) & 1u, abort_flag, p.status, spin)) break;
      if (tile >= kVStages &&
          !mbar_wait_warp(BAR(kBarVFree, vst), static_cast<uint32_t>(tile / kVStages - 1) & 1u, abort_flag, p.status, spin)) break;
      const int key0 = (tile_base + tile) * kTileN;
      unsigned char* Vb = Vs + vst * NB * kBlockBytes;
#pragma unroll 1
      for (int i0 = 0; i0 < 16; i0 += kFp8VBatch) {
        // a lane's 16 chunks of 16 codes in small batches (the codes are a shared-memory load away, and short loop bodies
        // keep the kernel's code small): chunk idx = lane + 32 i of the warp's 64 keys is key idx / 8, dims [16 (idx % 8), +16)
        uint4 cd[kFp8VBatch];
        float sc[kFp8VBatch];
#pragma unroll
        for (int u = 0; u < kFp8VBatch; ++u) {
          const int idx = lane + 32 * (i0 + u), kk = half * 64 + (idx >> 3), c16 = idx & 7;
          cd[u] = make_uint4(0, 0, 0, 0); sc[u] = 0.f;
          if (key0 + kk < kvl) {
            cd[u] = *reinterpret_cast<const uint4*>(Vc + kk * 128 + 16 * c16);
            sc[u] = vscl[(tile & 1) * 8 + (kk >> 4)];
          }
        }
#pragma unroll
        for (int u = 0; u < kFp8VBatch; ++u) {
          const int idx = lane + 32 * (i0 + u), kk = half * 64 + (idx >> 3), c16 = idx & 7;
          const uint32_t cw[4] = {cd[u].x, cd[u].y, cd[u].z, cd[u].w};
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t hh;
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(hh) : "h"(static_cast<uint16_t>(cw[j >> 1] >> (16 * (j & 1)))));
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hh));
            w[j] = pack_bf16x2(f.x * sc[u], f.y * sc[u]);       // a dead row: codes 0 and scale 0 give zeros
          }
          const int ch0 = 2 * c16;                   // bf16 chunk (8 dims) index within the row
          *reinterpret_cast<uint4*>(Vb + (ch0 / 8) * kBlockBytes + sw128(kk, ch0 % 8)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(Vb + (ch0 / 8) * kBlockBytes + sw128(kk, ch0 % 8 + 1)) = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      fence_async_smem();
      mbar_arrive(BAR(kBarVReady, vst));
      mbar_arrive(bar_vc_free);      // the staged codes have been read: the next tile's may come
    }
  } else if (FP8 && warp == kKLoaderWarp) {
    // =============================================================== 8-bit pages: the code loader
    // Lane g < 8 brings the codes of 16-key group g of the tile into the staging buffers, K then V, one bulk copy of
    // 2 KB each (a group's rows are contiguous in a pool), and publishes the group's position and the two scales.  The
    // staging buffers hold one tile: the copies of tile j + 1 wait until the rotators (K) and the converters (V) have
    // read tile j out.
    asm volatile("griddepcontrol.wait;" ::: "memory");   // after the commit kernel: the pools may be read
    int issued = 0;                                      // tiles whose copies have been started
    for (int tile = 0; tile < n_tiles; ++tile) {
      const int key0 = (tile_base + tile) * kTileN;
      const int gkey = key0 + lane * 16;
      const bool live = lane < 8 && gkey < kvl;
      int page = 0, pos = 0, slot0 = 0;
      float ks = 0.f, vs = 0.f;
      if (live) {
        const int e = gkey / p.page_size;
        slot0 = gkey % p.page_size;
        page = __ldg(ids + e);
        pos = __ldg(bases + e) + slot0;
        if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { atomicOr(p.status, MEPIC_DEV_BAD_PAGE); page = 0; }
        ks = __ldg(p.k_scales + page * p.n_kv_heads + h);
        vs = __ldg(p.v_scales + page * p.n_kv_heads + h);
      }
      const size_t row = static_cast<size_t>(page * p.n_kv_heads + h) * p.page_size + slot0;      // of the pool viewed as [rows][128 bytes]
      const uint32_t bytes = static_cast<uint32_t>(__popc(__ballot_sync(0xffffffffu, live))) * kCodeGroupBytes;
      // ---- K codes
      if (tile >= 1 && !mbar_wait_warp(bar_kc_free, static_cast<uint32_t>(tile - 1) & 1u, abort_flag, p.status, spin)) break;
      if (lane < 8) { gbase[(tile & 1) * 8 + lane] = pos; kscl[(tile & 1) * 8 + lane] = ks; }
      __syncwarp();
      if (!(HOOKS && blockIdx.x == 0 && tile == p.skip_tile)) {      // (test hook: a K tile that never comes)
        if (lane == 0) mbar_expect_tx(bar_kc_landed, bytes);
        __syncwarp();
        if (live) bulk_g2s(smem_u32(Kc) + static_cast<uint32_t>(lane) * kCodeGroupBytes,
                           reinterpret_cast<const unsigned char*>(p.k_pool) + row * 128, kCodeGroupBytes, bar_kc_landed);
      }
      // ---- V codes
      if (tile >= 1 && !mbar_wait_warp(bar_vc_free, static_cast<uint32_t>(tile - 1) & 1u, abort_flag, p.status, spin)) break;
      if (lane < 8) vscl[(tile & 1) * 8 + lane] = vs;
      __syncwarp();
      if (lane == 0) mbar_expect_tx(bar_vc_landed, bytes);
      __syncwarp();
      if (live) bulk_g2s(smem_u32(Vc) + static_cast<uint32_t>(lane) * kCodeGroupBytes,
                         reinterpret_cast<const unsigned char*>(p.v_pool) + row * 128, kCodeGroupBytes, bar_vc_landed);
      issued = tile + 1;
    }
    // after a lost wait: the copies started last may still be in flight; give them a bounded chance to land before the
    // CTA's shared memory is given up (the tile that the test hook left out never lands: the bound ends that wait)
    if (*abort_flag && issued > 0) {
      for (int i = 0; i < spin && !mbar_try_wait(bar_kc_landed, static_cast<uint32_t>(issued - 1) & 1u); ++i) {}
      for (int i = 0; i < spin && !mbar_try_wait(bar_vc_landed, static_cast<uint32_t>(issued - 1) & 1u); ++i) {}
    }
  } else if (!FP8 && (warp == kKLoaderWarp || warp == kVLoaderWarp)) {
    // =============================================================== loader warps: lane g loads 16-key group g
    const bool is_k = warp == kKLoaderWarp;
    const CUtensorMap* map = is_k ? &map_k : &map_v;
    unsigned char* ring = is_k ? Ks : Vs;
    const int depth = is_k ? kKStages : kVStages;
    bool ok = true;
    // This kernel is launched as a programmatic dependent of the commit kernel: everything up to here read only
    // the call's inputs; the pools may be read once that kernel has completed and its writes are visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int tile = 0; tile < n_tiles; ++tile) {
      const int st = tile % depth;
      if (tile >= depth) {
        // the stage is free once every MMA that reads its previous tenant has completed
        const uint32_t bar = BAR(is_k ? kBarKFree : kBarVFree, st);
        if (!mbar_wait_warp(bar, static_cast<uint32_t>(tile / depth - 1) & 1u, abort_flag, p.status, spin)) { ok = false; break; }
      }
      const int key0 = (tile_base + tile) * kTileN;
      const int gkey = key0 + lane * 16;
      const bool live = lane < 8 && gkey < kvl;
      int page = 0, pos = 0, slot0 = 0;
      if (live) {
        const int e = gkey / p.page_size;
        slot0 = gkey % p.page_size;
        page = __ldg(ids + e);
        pos = __ldg(bases + e) + slot0;
        if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { atomicOr(p.status, MEPIC_DEV_BAD_PAGE); page = 0; }
      }
      if (is_k && lane < 8) gbase[st * 8 + lane] = pos;
      const unsigned live_mask = __ballot_sync(0xffffffffu, live);
      __syncwarp();
      const uint32_t landed = BAR(is_k ? kBarKLanded : kBarVLanded, st);
      if (HOOKS && is_k && blockIdx.x == 0 && tile == p.skip_tile) continue;      // (test hook: a K tile that never comes)
      if (lane == 0) mbar_expect_tx(landed, static_cast<uint32_t>(__popc(live_mask)) * kGroupBytes);
      __syncwarp();
      if (live) {
        const int y = (page * p.n_kv_heads + h) * p.page_size + slot0;     // row of the pool viewed as [rows][D]
        const uint32_t dst = smem_u32(ring + st * NB * kBlockBytes) + static_cast<uint32_t>(lane * 16 * 128);
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) tma_load_2d(dst + nb * kBlockBytes, map, nb * 64, y, landed);
      }
    }
    // Rows at or past kv_len of the last V tile may hold anything (NaN bit patterns included): P is 0 there,
    // but 0 x NaN is NaN, so V must be finite.  Zero them once the tile has landed.
    if (!is_k && ok && last_has_tail) {
      const int lt = n_tiles - 1, st = lt % kVStages;
      if (mbar_wait_warp(BAR(kBarVLanded, st), static_cast<uint32_t>(lt / kVStages) & 1u, abort_flag, p.status, spin)) {
        unsigned char* Vb = Vs + st * NB * kBlockBytes;
        const int first = kvl - (tile_base + lt) * kTileN;       // first row to clear (0 < first < 128)
        for (int idx = first * 2 * CH + lane; idx < kTileN * 2 * CH; idx += 32) {
          const int kk = idx / (2 * CH), ch = idx % (2 * CH);
          *reinterpret_cast<uint4*>(Vb + (ch / 8) * kBlockBytes + sw128(kk, ch % 8)) = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(kBarVPatched, 0));
      }
    }
    // (After a lost wait somewhere this warp leaves its loop from a wait that has polled at least 1024 times since its
    // last copy was started - the flag is looked at every 1024 polls - which is tens of microseconds against the one or
    // two a copy takes: nothing of it is still in flight at the CTA's exit.  An explicit wait for the landed barriers
    // here, even out of line and never executed, cost the kernel 1.3 % in the way the compiler lays the roles out.)
  } else if (warp == kMmaWarp && lane == 0) {
    // =============================================================== MMA issuer (one thread)
    // Order per key tile j:  PV_a(j), QK_a(j+1), PV_b(j), QK_b(j+1): while one M-tile's softmax runs, the
    // tensor core works on the other M-tile.  S of an M-tile is reused by its P, so QK_x(j+1) follows PV_x(j).
    // The issuing thread shares its scheduler with softmax and rotator warps and the tensor pipe waits on it between
    // an M-tile's P and its next S, so the issue loops carry as few instructions as possible: every descriptor is a
    // base computed once plus a compile-time constant in its 16-byte-unit address field.
    const uint64_t q_desc[2] = {smem_desc(smem_u32(Qs), 16, 1024), smem_desc(smem_u32(Qs + NB * kBlockBytes), 16, 1024)};
    const uint64_t k_desc0 = smem_desc(smem_u32(Ks), 16, 1024);
    const uint64_t v_desc0 = smem_desc(smem_u32(Vs), kBlockBytes, 1024);
    constexpr uint64_t kStageUnits = (NB * kBlockBytes) >> 4;
    bool ok = true;
    auto issue_qk = [&](int x, int j) {
      const uint64_t kd = k_desc0 + static_cast<uint64_t>(j % KD) * kStageUnits;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint64_t off = static_cast<uint64_t>(((ks / 4) * kBlockBytes + (ks % 4) * 32) >> 4);
        tc_mma(tmem_base + static_cast<uint32_t>(x * 128), q_desc[x] + off, kd + off, kIdescQK, ks > 0);
      }
      tc_commit(BAR(kBarSFull, x));
    };
    auto issue_pv = [&](int x, int j) {
      const uint64_t vd = v_desc0 + static_cast<uint64_t>(j % kVStages) * kStageUnits;
#pragma unroll
      for (int ks = 0; ks < kTileN / 16; ++ks) {
        // A = P from tensor memory: 16 bf16 per k-step = 8 columns, keys 0..63 at columns 0.., keys 64..127 at 64..; B = V, MN-major
        tc_mma_ts(tmem_base + 256u + static_cast<uint32_t>(x * 128), tmem_base + static_cast<uint32_t>(x * 128 + (ks / 4) * 64 + (ks % 4) * 8),
                  vd + static_cast<uint64_t>((ks * 2048) >> 4), kIdescPV, (j > 0 || ks > 0) ? 1u : 0u);
      }
      tc_commit(BAR(kBarPvDone, x));
    };
    auto wait_k = [&](int j) {
      const bool w = mbar_wait(BAR(kBarKReady, j % KD), static_cast<uint32_t>(j / KD) & 1u, abort_flag, p.status, spin);
      tc_fence_after();
      return w;
    };
    // prologue: S of key tile 0 for both M-tiles
    ok = n_tiles > 0 && mbar_wait(BAR(kBarQReady, 0), 0, abort_flag, p.status, spin) && wait_k(0);
    if (ok) {
      if (nt[0] > 0) issue_qk(0, 0);
      if (nt[1] > 0) issue_qk(1, 0);
      tc_commit(BAR(kBarKFree, 0));
    }
    for (int j = 0; j < n_tiles && ok; ++j) {
      bool v_here = false;
      auto wait_v = [&]() {
        if (v_here) return true;
        bool w = mbar_wait(BAR(FP8 ? kBarVReady : kBarVLanded, j % kVStages), static_cast<uint32_t>(j / kVStages) & 1u, abort_flag, p.status, spin);
        if (!FP8 && w && j == n_tiles - 1 && last_has_tail) w = mbar_wait(BAR(kBarVPatched, 0), 0, abort_flag, p.status, spin);
        v_here = w;
        return w;
      };
      const bool more = j + 1 < n_tiles;
      // ---- M-tile a.  The next K tile was rotated long ago (the rotators run ahead): its wait comes first so that
      // nothing stands between the issue of PV_a and of QK_a(next) and the pipe's queue does not run dry.
      if (more && !wait_k(j + 1)) { ok = false; break; }
      if (j < nt[0]) {
        if (!mbar_wait(BAR(kBarPFull, 0), static_cast<uint32_t>(j) & 1u, abort_flag, p.status, spin) || !wait_v()) { ok = false; break; }
        tc_fence_after();
        issue_pv(0, j);
      }
      if (more && j + 1 < nt[0]) issue_qk(0, j + 1);
      // ---- M-tile b
      if (j < nt[1]) {
        if (!mbar_wait(BAR(kBarPFull, 1), static_cast<uint32_t>(j) & 1u, abort_flag, p.status, spin) || !wait_v()) { ok = false; break; }
        tc_fence_after();
        issue_pv(1, j);
      }
      tc_commit(BAR(kBarVFree, j % kVStages));
      if (more) {
        if (j + 1 < nt[1]) issue_qk(1, j + 1);
        tc_commit(BAR(kBarKFree, (j + 1) % KD));
      }
    }
    if (!ok) {
      // a wait was lost: the MMAs issued so far still run; tensor memory may only be released once they are done
      tc_commit(BAR(kBarDrain, 0));
      for (int i = 0; i < spin && !mbar_try_wait(BAR(kBarDrain, 0), 0); ++i) {}
    }
  }

  // ---- common exit: nothing of this CTA may still be in flight when tensor memory is released
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
  if (tid == 0 && *sat_flag) *p.redo_flag = 1;
}

constexpr int kMaxSplits = 8;           // most shares a work item's key range is cut into

// Merge of the shares of a split item: one warp per (row, q head), a lane per four head dims.
template <int D>
__global__ void __launch_bounds__(128) mepic_prefill_merge(const PrefillParams p, int n_q_heads) {
  const long long pair = static_cast<long long>(blockIdx.x) * 4 + (threadIdx.x >> 5);
  const long long n_pairs = static_cast<long long>(p.total_rows) * n_q_heads;
  const int lane = threadIdx.x & 31;
  if (pair >= n_pairs) return;
  asm volatile("griddepcontrol.wait;" ::: "memory");              // launched as a programmatic dependent of the attention kernel
  // every load of the pair is issued before the first use (the share count is at most kMaxSplits)
  float2 ml[kMaxSplits];
  float4 x[kMaxSplits];
#pragma unroll
  for (int s = 0; s < kMaxSplits; ++s) {
    ml[s] = make_float2(-INFINITY, 0.f);
    x[s] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (s < p.n_splits) {
      const size_t at = static_cast<size_t>(s) * n_pairs + pair;
      ml[s] = *reinterpret_cast<const float2*>(p.part_ml + at * 2);
      if (lane < D / 4) x[s] = *reinterpret_cast<const float4*>(p.part_o + at * D + 4 * lane);
    }
  }
  float m_star = -INFINITY;
#pragma unroll
  for (int s = 0; s < kMaxSplits; ++s)
    if (ml[s].y > 0.f) m_star = fmaxf(m_star, ml[s].x);
  float l_star = 0.f;
  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int s = 0; s < kMaxSplits; ++s) {
    if (!(ml[s].y > 0.f)) continue;                  // the share held none of this row's keys (or does not exist)
    const float wgt = ex2(ml[s].x - m_star);
    l_star += ml[s].y * wgt;
    o.x += x[s].x * wgt; o.y += x[s].y * wgt; o.z += x[s].z * wgt; o.w += x[s].w * wgt;
  }
  if (lane < D / 4) {
    const float inv = l_star > 0.f ? 1.f / l_star : 0.f;
    *reinterpret_cast<uint2*>(p.out + pair * D + 4 * lane) = make_uint2(pack_bf16x2(o.x * inv, o.y * inv), pack_bf16x2(o.z * inv, o.w * inv));
  }
}

template <int D, int G, bool FP8, bool HOOKS = false>
int32_t launch_prefill(const PrefillParams& p, int n_items, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
  constexpr size_t smem = PrefillSmem<D>::kBytes;
  cudaError_t e = cudaFuncSetAttribute(mepic_prefill_attn<D, G, FP8, HOOKS>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) { mepic_set_error("prefill: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  const int chunks_per_row = p.n_kv_heads * D / 8;
  if (FP8) mepic_prefill_commit_fp8<<<p.total_rows, 256, 0, stream>>>(p, D);
  else mepic_prefill_commit<<<(p.total_rows + kCommitRows - 1) / kCommitRows, kCommitRows * 32, 0, stream>>>(p, chunks_per_row);
  // each kernel may become resident while its predecessor drains (programmatic dependent launch); it waits with
  // griddepcontrol.wait before it touches what the predecessor writes
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(static_cast<unsigned>(n_items * p.n_splits)); lc.blockDim = dim3(kThreads); lc.dynamicSmemBytes = smem; lc.stream = stream;
  lc.attrs = pdl; lc.numAttrs = 1;
  // the fast launch, then the repeat launch, which does nothing unless a row outran its reference in the first
  PrefillParams pf = p;
  const bool two_pass_only = mepic_test_prefill_two_pass() != 0;       // (test hook: the repeat launch's schedule, unconditionally)
  pf.exact = two_pass_only ? 2 : 0;
  e = cudaLaunchKernelEx(&lc, mepic_prefill_attn<D, G, FP8, HOOKS>, pf, map_k, map_v);
  if (e == cudaSuccess && !two_pass_only) {
    pf.exact = 1;
    e = cudaLaunchKernelEx(&lc, mepic_prefill_attn<D, G, FP8, HOOKS>, pf, map_k, map_v);
  }
  if (e == cudaSuccess && p.n_splits > 1) {
    const long long n_pairs = static_cast<long long>(p.total_rows) * p.n_kv_heads * G;
    lc.gridDim = dim3(static_cast<unsigned>((n_pairs + 3) / 4)); lc.blockDim = dim3(128); lc.dynamicSmemBytes = 0;
    e = cudaLaunchKernelEx(&lc, mepic_prefill_merge<D>, p, p.n_kv_heads * G);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { mepic_set_error("prefill: launch: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_count_launches((p.n_splits > 1 ? 4 : 3) - (two_pass_only ? 1 : 0));
  return MEPIC_OK;
}

// Launch sizing from the host copy of row_offsets: number of CTAs and the deepest level (see item_of_cta).
bool count_items(const mepic_config_t* cfg, int batch, const int32_t* row_offsets_host, int* n_items, int* max_q_tiles) {
  const int G = cfg->n_q_heads / cfg->n_kv_heads, QT = 2 * (128 / G);   // two M-tiles of query positions per CTA
  long long items = 0;
  int deepest = 0;
  for (int b = 0; b < batch; ++b) {
    const int n = row_offsets_host[b + 1] - row_offsets_host[b];
    if (n < 0) return false;
    const int tiles = (n + QT - 1) / QT;
    items += static_cast<long long>(tiles) * cfg->n_kv_heads;
    deepest = std::max(deepest, tiles);
  }
  if (items > 0x7fffffffLL) return false;
  *n_items = static_cast<int>(items);
  *max_q_tiles = deepest;
  return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// How many CTAs share a work item: 1 when the items fill at least one wave of the GPU; below that
// round((1.2 SMs / items)^0.8), at most kMaxSplits.  The host knows the number of items but not their sizes (slots and
// lengths are device data), so this is a fit: CTAs are handed to SMs in index order and a share costs about eight key
// tiles of fixed work (Q staging, pipeline fill, partials); a model of exactly that reproduces the measured times of
// seven small batches to within ten tiles, and over those and a dozen more shapes this rule is at or next to the model's
// best uniform share count.  Depends on the SM count of the current device; 1 without a device.
int splits_for(int n_items) {
  int dev = 0, sms = 0;
  if (n_items <= 0 || cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return 1;
  if (n_items >= sms) return 1;                  // a full wave or more: a share's fixed cost (Q staging, pipeline fill, partials) outweighs the balance
  const int s = static_cast<int>(std::lround(std::pow(1.2 * sms / n_items, 0.8)));
  return std::max(1, std::min(kMaxSplits, s));
}
size_t split_workspace_bytes(const mepic_config_t* cfg, long long total_rows, int splits) {
  if (splits <= 1) return 16;
  return 16 + static_cast<size_t>(splits) * static_cast<size_t>(total_rows) * cfg->n_q_heads * (cfg->head_dim + 2) * sizeof(float);
}

}  // namespace

extern "C" size_t mepic_attn_prefill_workspace(const mepic_config_t* cfg, int32_t batch, const int32_t* row_offsets_host) {
  if (!mepic_config_ok(cfg) || batch < 1 || !row_offsets_host) { if (cfg) mepic_set_error("prefill_workspace: bad argument"); return 0; }
  int n_items = 0, deepest = 0;
  if (!count_items(cfg, batch, row_offsets_host, &n_items, &deepest)) { mepic_set_error("prefill_workspace: row_offsets must be non-decreasing"); return 0; }
  // 16 bytes when the items fill the GPU by themselves (the kernels derive their work on the device; nothing is
  // staged); else room for the partials of the items' key-range shares
  return split_workspace_bytes(cfg, row_offsets_host[batch], splits_for(n_items));
}

static int32_t prefill_call(const mepic_config_t* cfg, const mepic_prefill_args_t* a, float* k_scales, float* v_scales, bool fp8, void* cuda_stream) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (fp8 && cfg->head_dim != 128) { mepic_set_error("prefill_fp8: head_dim %d: 8-bit pages are built for head_dim 128", cfg->head_dim); return MEPIC_E_INVAL; }
  if (!a || !a->row_offsets_host) { mepic_set_error("prefill: NULL pointer argument"); return MEPIC_E_INVAL; }
  if (a->batch < 1 || a->table_stride < 1) { mepic_set_error("prefill: batch and table_stride must be positive"); return MEPIC_E_INVAL; }
  if (a->row_offsets_host[0] == 0 && a->row_offsets_host[a->batch] == 0) return MEPIC_OK;   // no rows at all: the row buffers may be absent
  if (!a->q_new || !a->k_new || !a->v_new || !a->row_offsets || !a->q_slot || !a->k_pool || !a->v_pool ||
      !a->page_ids || !a->pos_base || !a->kv_len || !a->rope_table || !a->out || !a->workspace || !a->status) {
    mepic_set_error("prefill: NULL pointer argument"); return MEPIC_E_INVAL;
  }
  if (!aligned16(a->q_new) || !aligned16(a->k_new) || !aligned16(a->v_new) || !aligned16(a->k_pool) || !aligned16(a->v_pool) ||
      !aligned16(a->rope_table) || !aligned16(a->out) || !aligned16(a->workspace)) {
    mepic_set_error("prefill: pointers must be 16-byte aligned"); return MEPIC_E_INVAL;
  }
  if (cfg->max_position < 16) { mepic_set_error("prefill: rope table must cover positions 0..16"); return MEPIC_E_INVAL; }
  if (a->row_offsets_host[0] != 0) { mepic_set_error("prefill: row_offsets[0] must be 0"); return MEPIC_E_INVAL; }
  int n_items = 0, max_q_tiles = 0;
  if (!count_items(cfg, a->batch, a->row_offsets_host, &n_items, &max_q_tiles)) { mepic_set_error("prefill: row_offsets must be non-decreasing"); return MEPIC_E_INVAL; }
  const int total_rows = a->row_offsets_host[a->batch];
  if (n_items == 0 || total_rows == 0) return MEPIC_OK;      // nothing to recompute
  if (fp8 && (!k_scales || !v_scales)) { mepic_set_error("prefill_fp8: NULL scale pointer"); return MEPIC_E_INVAL; }
  alignas(64) CUtensorMap map_k, map_v;
  if (fp8) {
    memset(&map_k, 0, sizeof(map_k)); memset(&map_v, 0, sizeof(map_v));        // the 8-bit kernel does not use TMA
  } else {
    int32_t rc = mepic_make_pool_map(cfg, a->k_pool, &map_k);
    if (rc != MEPIC_OK) return rc;
    rc = mepic_make_pool_map(cfg, a->v_pool, &map_v);
    if (rc != MEPIC_OK) return rc;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  PrefillParams p;
  p.k_scales = k_scales; p.v_scales = v_scales;
  p.q_new = static_cast<const uint16_t*>(a->q_new);
  p.k_new = static_cast<const uint16_t*>(a->k_new);
  p.v_new = static_cast<const uint16_t*>(a->v_new);
  p.row_offsets = a->row_offsets; p.q_slot = a->q_slot;
  p.k_pool = static_cast<uint16_t*>(a->k_pool); p.v_pool = static_cast<uint16_t*>(a->v_pool);
  p.page_ids = a->page_ids; p.pos_base = a->pos_base; p.kv_len = a->kv_len;
  p.rope = a->rope_table;
  p.out = static_cast<uint16_t*>(a->out);
  p.status = a->status;
  p.table_stride = a->table_stride; p.batch = a->batch; p.n_kv_heads = cfg->n_kv_heads; p.page_size = cfg->page_size;
  p.num_pages = cfg->num_pages; p.max_position = cfg->max_position; p.total_rows = total_rows;
  p.max_q_tiles = max_q_tiles;
  p.n_splits = splits_for(n_items);
  if (a->workspace_bytes < split_workspace_bytes(cfg, total_rows, p.n_splits)) p.n_splits = 1;     // no room for partials: one CTA per item
  p.redo_flag = static_cast<int32_t*>(a->workspace);
  p.exact = 0;
  p.part_o = reinterpret_cast<float*>(static_cast<unsigned char*>(a->workspace) + 16);
  p.part_ml = p.part_o + static_cast<size_t>(p.n_splits) * total_rows * cfg->n_q_heads * cfg->head_dim;
  p.scale_log2 = a->sm_scale * 1.4426950408889634f;
  p.spin_limit = mepic_test_spin_limit(kSpinLimit); p.skip_tile = mepic_test_skip_tile();
  const int D = cfg->head_dim, G = cfg->n_q_heads / cfg->n_kv_heads;
  if (p.spin_limit != kSpinLimit || p.skip_tile >= 0) {
    // test hooks are set: the instrumented instantiation, built for the shape the give-up test uses
    if (D == 128 && G == 4) return fp8 ? launch_prefill<128, 4, true, true>(p, n_items, map_k, map_v, st) : launch_prefill<128, 4, false, true>(p, n_items, map_k, map_v, st);
    mepic_set_error("prefill: the kernel test hooks are built for head_dim 128 and group size 4 only");
    return MEPIC_E_INVAL;
  }
  if (fp8) {
#define MEPIC_PREFILL_FP8_CASE(GG) if (G == GG) return launch_prefill<128, GG, true>(p, n_items, map_k, map_v, st);
    MEPIC_PREFILL_FP8_CASE(1) MEPIC_PREFILL_FP8_CASE(2) MEPIC_PREFILL_FP8_CASE(3) MEPIC_PREFILL_FP8_CASE(4) MEPIC_PREFILL_FP8_CASE(5) MEPIC_PREFILL_FP8_CASE(6) MEPIC_PREFILL_FP8_CASE(7) MEPIC_PREFILL_FP8_CASE(8)
#undef MEPIC_PREFILL_FP8_CASE
  }
#define MEPIC_PREFILL_CASE(DD, GG) if (D == DD && G == GG) return launch_prefill<DD, GG, false>(p, n_items, map_k, map_v, st);
  MEPIC_PREFILL_CASE(128, 1) MEPIC_PREFILL_CASE(128, 2) MEPIC_PREFILL_CASE(128, 3) MEPIC_PREFILL_CASE(128, 4) MEPIC_PREFILL_CASE(128, 5) MEPIC_PREFILL_CASE(128, 6) MEPIC_PREFILL_CASE(128, 7) MEPIC_PREFILL_CASE(128, 8)
  MEPIC_PREFILL_CASE(64, 1) MEPIC_PREFILL_CASE(64, 2) MEPIC_PREFILL_CASE(64, 3) MEPIC_PREFILL_CASE(64, 4) MEPIC_PREFILL_CASE(64, 5) MEPIC_PREFILL_CASE(64, 6) MEPIC_PREFILL_CASE(64, 7) MEPIC_PREFILL_CASE(64, 8)
#undef MEPIC_PREFILL_CASE
  mepic_set_error("prefill: unsupported head_dim %d / group size %d", D, G);
  return MEPIC_E_INVAL;
}

extern "C" int32_t mepic_attn_prefill(const mepic_config_t* cfg, const mepic_prefill_args_t* a, void* cuda_stream) {
  return prefill_call(cfg, a, nullptr, nullptr, false, cuda_stream);
}

extern "C" int32_t mepic_attn_prefill_fp8(const mepic_config_t* cfg, const mepic_prefill_args_t* a, float* k_scales, float* v_scales,
                                          void* cuda_stream) {
  return prefill_call(cfg, a, k_scales, v_scales, true, cuda_stream);
}
