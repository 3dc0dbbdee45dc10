// The tile line of the per-request decode kernels and what they share: launch parameters, the cut of the line
// into equal pieces, the cursor that walks it, and the kernel that merges the partials of each unit.
#ifndef MEPIC_DECODE_LINE_CUH_
#define MEPIC_DECODE_LINE_CUH_

#include "mepic.h"
#include "mepic_ptx.cuh"

namespace mepic_dev {

constexpr int kTile = 16;      // tokens per staged tile
#ifndef MEPIC_DECODE_WARPS
#define MEPIC_DECODE_WARPS 8
#endif
constexpr int kWarps = MEPIC_DECODE_WARPS;      // warps per CTA of the bf16 kernel that take part when every byte may come from DRAM
constexpr int kWarpsShared = 12;                // ... and when the requests are known to alias pages (see cut_of_line)
#ifndef MEPIC_FP8_WARPS
#define MEPIC_FP8_WARPS 12
#endif
constexpr int kWarpsFp8 = MEPIC_FP8_WARPS;      // ... of the 8-bit kernel (half the bytes per stage, fewer registers: room for more)
constexpr int kMaxWarps = kWarpsFp8 > kWarpsShared ? kWarpsFp8 : kWarpsShared;   // the workspace holds a partial per worker of either kernel
constexpr int kMinPiece = 4;   // never cut the line into pieces shorter than this many tiles

struct DecodeParams {
  const uint16_t* q;
  const uint16_t* k_pool;
  const uint16_t* v_pool;
  const int32_t* page_ids;
  const int32_t* pos_base;
  const int32_t* kv_len;
  const int32_t* q_pos;
  const float* rope;
  const float* k_scales;   // fp8 pools only: [num_pages][n_kv_heads] scale of each (page, kv head) block of K
  const float* v_scales;   // ... and of V
  float* part_o;    // [slots][G][D]
  float* part_ml;   // [slots][G][2] = (max in log2 units, sum)
  uint16_t* out;
  int32_t* status;
  int table_stride, batch, n_kv_heads, page_size, log2_tpp, num_pages, max_position, n_workers;
  int n_workers_dram;   // workers used when the batch cannot be known to alias pages (see cut_of_line); <= n_workers
  int spin_limit;   // polls before a bounded wait gives up
  int skip_tile;    // test hook: worker 0 leaves out the staged copy of its tile with this index (-1: none)
  float scale_log2;   // sm_scale * log2(e)
};

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}
__device__ __forceinline__ int tiles_of(int kv_len) { return kv_len > 0 ? (kv_len + kTile - 1) / kTile : 0; }

// The cut of the tile line, recomputed by every warp from kv_len (no host mirror, no plan upload).
//
// How many workers take part is decided here as well, the same way by every warp of both kernels.  The decode has two
// regimes: when every byte comes from DRAM it is bound by DRAM, and more tiles in flight than n_workers_dram workers
// keep there only lower the DRAM rate; when requests alias pages most tile loads are L2 hits, the kernel is bound by
// the latency of its own dependent instructions and all n_workers help.  If the batch has at least 1.5 table entries
// per page of the pool its requests must alias pages, and all workers run; otherwise only the first n_workers_dram
// (the warps beyond them in each CTA leave at once).
struct Cut { long long total; long long piece; int workers; };
__device__ __forceinline__ Cut cut_of_line(const DecodeParams& p, int lane) {
  long long tiles = 0;
  for (int b0 = 0; b0 < p.batch; b0 += 32) {
    const int n = (b0 + lane < p.batch) ? tiles_of(p.kv_len[b0 + lane]) : 0;
    tiles += warp_sum(n);
  }
  Cut c;
  c.total = tiles * p.n_kv_heads;
  c.workers = 2 * (tiles >> p.log2_tpp) >= 3ll * p.num_pages ? p.n_workers : p.n_workers_dram;
  long long piece = (c.total + c.workers - 1) / c.workers;
  c.piece = piece < kMinPiece ? kMinPiece : piece;
  return c;
}

// Position on the line: request b, kv head h, tile t of the request's nt tiles.
struct Cursor { int b, h, t, nt, kvl; };

__device__ __forceinline__ Cursor locate(const int32_t* kv_len, int batch, int n_kv_heads, long long x, int lane) {
  Cursor c{batch, 0, 0, 0, 0};
  long long before = 0;   // tiles of the requests before the 32 under inspection
  for (int b0 = 0; b0 < batch; b0 += 32) {
    const int kvl = (b0 + lane < batch) ? kv_len[b0 + lane] : 0;
    const int n = tiles_of(kvl);
    int incl = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(kFull, incl, o); if (lane >= o) incl += y; }
    const bool past = (before + incl) * n_kv_heads > x;
    const unsigned m = __ballot_sync(kFull, past);
    if (m) {
      const int l = __ffs(m) - 1;
      const long long pre = before + __shfl_sync(kFull, incl - n, l);
      c.b = b0 + l;
      c.nt = __shfl_sync(kFull, n, l);
      c.kvl = __shfl_sync(kFull, kvl, l);
      const long long r = x - pre * n_kv_heads;
      c.h = static_cast<int>(r / c.nt);
      c.t = static_cast<int>(r % c.nt);
      return c;
    }
    before += __shfl_sync(kFull, incl, 31);
  }
  return c;
}

__device__ __forceinline__ void advance(Cursor& c, const int32_t* kv_len, int batch, int n_kv_heads) {
  if (++c.t < c.nt) return;
  c.t = 0;
  if (++c.h < n_kv_heads) return;
  c.h = 0;
  do {
    ++c.b;
    c.kvl = (c.b < batch) ? kv_len[c.b] : 0;
    c.nt = tiles_of(c.kvl);
  } while (c.b < batch && c.nt == 0);
}

// ---------------------------------------------------------------- merge of the partials of each unit
// One CTA per (request, kv head); thread (g, d) combines the unit's partials:
// m* = max m, l* = sum l 2^(m - m*), out = sum o 2^(m - m*) / l*  -> bf16.
template <int D, int G>
__global__ void mepic_decode_merge(const DecodeParams p) {
  const int b = blockIdx.x / p.n_kv_heads, h = blockIdx.x % p.n_kv_heads;
  const int lane = threadIdx.x & 31;
  __shared__ long long sh[3];
  if (threadIdx.x < 32) {
    const Cut cut = cut_of_line(p, lane);
    long long before = 0;
    for (int b0 = 0; b0 < b; b0 += 32) {
      const int n = (b0 + lane < b) ? tiles_of(p.kv_len[b0 + lane]) : 0;
      before += warp_sum(n);
    }
    if (lane == 0) { sh[0] = cut.piece; sh[1] = before; sh[2] = tiles_of(p.kv_len[b]); }
  }
  __syncthreads();
  // Everything above read only the call's inputs.  The partials come from the split-KV kernel launched just before
  // on the same stream: with programmatic dependent launch this kernel may already be resident, so wait for that
  // kernel's completion (and the visibility of its writes) here rather than at launch.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const long long piece = sh[0], nt = sh[2];
  const int g = threadIdx.x / D, d = threadIdx.x % D;
  const size_t o_at = (static_cast<size_t>(b) * p.n_kv_heads * G + static_cast<size_t>(h) * G + g) * D + d;
  if (nt == 0) { p.out[o_at] = 0; return; }
  const long long u0 = sh[1] * p.n_kv_heads + static_cast<long long>(h) * nt;
  const long long w_first = u0 / piece, w_last = (u0 + nt - 1) / piece;
  const long long unit = static_cast<long long>(b) * p.n_kv_heads + h;
  // the partials of a line are read four pieces at a time (the loads of a batch are independent: one round trip to L2
  // instead of four) and combined in piece order
  float m_star = -INFINITY;
  for (long long wk = w_first; wk <= w_last; wk += 4) {
    float m4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) m4[k] = wk + k <= w_last ? p.part_ml[((unit + wk + k) * G + g) * 2] : -INFINITY;
#pragma unroll
    for (int k = 0; k < 4; ++k) m_star = fmaxf(m_star, m4[k]);
  }
  float l_star = 0.f, o_star = 0.f;
  for (long long wk = w_first; wk <= w_last; wk += 4) {
    float2 ml4[4];
    float o4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const bool in = wk + k <= w_last;
      ml4[k] = in ? *reinterpret_cast<const float2*>(p.part_ml + ((unit + wk + k) * G + g) * 2) : make_float2(-INFINITY, 0.f);
      o4[k] = in ? p.part_o[((unit + wk + k) * G + g) * D + d] : 0.f;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (wk + k <= w_last) {
        const float wgt = ex2(ml4[k].x - m_star);
        l_star += ml4[k].y * wgt;
        o_star += o4[k] * wgt;
      }
    }
  }
  const float r = o_star / l_star;
  // fp32 -> bf16, round to nearest even
  uint32_t u = __float_as_uint(r);
  u += 0x7fffu + ((u >> 16) & 1u);
  p.out[o_at] = (r != r) ? 0x7fc0 : static_cast<uint16_t>(u >> 16);
}

}  // namespace mepic_dev

#endif
