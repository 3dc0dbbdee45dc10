// Decode: RoPE-fused, split-KV, GQA, online-softmax attention over paged,
// un-rotated K (Section 3.3.3 of the paper: the rotation is applied when the
// kernel brings NoPE KV blocks on chip, right before the scores).
//
// Work decomposition.  The context of request b is cut into tiles of 16 tokens;
// the (request, kv head, tile) triples of the whole batch are laid on one line
// in that order and cut into equal contiguous pieces, one per WARP of a
// persistent grid (one CTA per SM, 8 warps).  A warp is a self-contained
// worker: it owns a ring of shared-memory stages that bulk-async copies
// (cp.async.bulk + mbarrier complete_tx) fill with the 16 x D K tile and V tile
// of its next tiles, and it keeps one online-softmax state per query head of
// the kv head it is on.  When its piece crosses into another (request, head)
// unit, or ends, it writes a partial (max, sum, weighted V) for the unit; a
// second kernel merges the partials of each unit.  Equal pieces balance the
// ragged batches; no warp ever waits on another warp.
//
// Rotation.  <R(qpos) q, R(base+tau) k> = <R(qpos-base) q, R(tau) k>: per tile
// the warp rotates the G query vectors by (qpos - tile base) from one row of
// the cos/sin table, and rotates every key only by its offset tau < 16 inside
// the tile, with cos/sin of those 16 offsets held in registers for the whole
// kernel.  Keys are rotated in registers in fp32 and never written back.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "mepic.h"
#include "mepic_internal.h"

namespace {

constexpr int kTile = 16;      // tokens per staged tile
constexpr int kWarps = 8;      // workers per CTA
// ring depth per worker: 3 stages, 2 where the per-warp buffers of a large group would not fit
__host__ __device__ constexpr int stages_for(int D, int G) { return G * D > 640 ? 2 : 3; }
constexpr int kMinPiece = 4;   // never cut the line into pieces shorter than this many tiles
constexpr unsigned kFull = 0xffffffffu;
constexpr int kSpinLimit = 1 << 22;

struct DecodeParams {
  const uint16_t* q;
  const uint16_t* k_pool;
  const uint16_t* v_pool;
  const int32_t* page_ids;
  const int32_t* pos_base;
  const int32_t* kv_len;
  const int32_t* q_pos;
  const float* rope;
  float* part_o;    // [slots][G][D]
  float* part_ml;   // [slots][G][2] = (max in log2 units, sum)
  uint16_t* out;
  int32_t* status;
  int table_stride, batch, n_kv_heads, page_size, log2_tpp, num_pages, max_position, n_workers;
  float scale_log2;   // sm_scale * log2(e)
};

// ---------------------------------------------------------------- small PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

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
// two bf16 packed in a 32-bit word (low half = even element) -> two floats, exactly
__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{ .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p; }"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls instead of hanging the SM.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (int i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}
__device__ __forceinline__ int tiles_of(int kv_len) { return kv_len > 0 ? (kv_len + kTile - 1) / kTile : 0; }

// The cut of the tile line, recomputed by every warp from kv_len (no host mirror, no plan upload).
struct Cut { long long total; long long piece; };
__device__ __forceinline__ Cut cut_of_line(const int32_t* kv_len, int batch, int n_kv_heads, int n_workers, int lane) {
  long long tiles = 0;
  for (int b0 = 0; b0 < batch; b0 += 32) {
    const int n = (b0 + lane < batch) ? tiles_of(kv_len[b0 + lane]) : 0;
    tiles += warp_sum(n);
  }
  Cut c;
  c.total = tiles * n_kv_heads;
  long long piece = (c.total + n_workers - 1) / n_workers;
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

// ---------------------------------------------------------------- the split-KV kernel
template <int D, int G>
__global__ void __launch_bounds__(kWarps * 32, 1) mepic_decode_splitkv(const DecodeParams p) {
  constexpr int kStages = stages_for(D, G);
  constexpr int DL = D / 16;                 // K phase: bf16 per lane per half row (8 lanes span a half row)
  constexpr int NP = DL / 2;                 // ... as packed pairs (32-bit words / float2)
  constexpr int DV = D / 16;                 // V phase: dims per lane (16 lanes span a row)
  constexpr int GP = G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8;   // heads padded to a power of two
  constexpr int LPH = 8 / GP;                // dim-lanes that end up holding the same head's score
  constexpr int HPL = (G + 3) / 4;           // heads each key-group rotates per tile
  constexpr int PSTR = GP < 4 ? 4 : GP;      // floats per key in the probability buffer
  constexpr int kTileElems = kTile * D;
  constexpr int kStageBytes = 2 * kTileElems * 2;
  constexpr int kQrotFloats = G * D;
  constexpr int kWarpBytes = kStages * kStageBytes + kQrotFloats * 4 + kTile * PSTR * 4 + 64;

  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  unsigned char* wbase = smem_raw + static_cast<size_t>(wic) * kWarpBytes;
  uint16_t* stage0 = reinterpret_cast<uint16_t*>(wbase);
  float4* qrot = reinterpret_cast<float4*>(wbase + kStages * kStageBytes);
  float* pbuf = reinterpret_cast<float*>(wbase + kStages * kStageBytes + kQrotFloats * 4);
  unsigned char* tail = wbase + kStages * kStageBytes + kQrotFloats * 4 + kTile * PSTR * 4;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail);          // kStages x 8 bytes
  volatile int* meta = reinterpret_cast<volatile int*>(tail + 32);   // tile position base per stage

  const int kg = lane >> 3;      // key group (K phase): keys kg, kg+4, kg+8, kg+12 of the tile
  const int l8 = lane & 7;       // dim lane (K phase)
  const int hw = lane >> 4;      // half warp (V phase): keys of parity hw
  const int l16 = lane & 15;     // dim lane (V phase)
  const int my_head = l8 / LPH;  // head whose score this lane holds after the reduction

  const long long w = static_cast<long long>(blockIdx.x) * kWarps + wic;
  const Cut cut = cut_of_line(p.kv_len, p.batch, p.n_kv_heads, p.n_workers, lane);
  const long long x0 = w * cut.piece;
  if (x0 >= cut.total) return;
  const long long x1 = (x0 + cut.piece < cut.total) ? x0 + cut.piece : cut.total;
  const int n_tiles = static_cast<int>(x1 - x0);

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // cos/sin of the 16 in-tile offsets, this lane's dims: rows 0..15 of the table.
  float2 c2[4][NP], s2[4][NP];
#pragma unroll
  for (int ps = 0; ps < 4; ++ps) {
    const float4* row = reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(kg + 4 * ps) * D + l8 * DL * 2);
#pragma unroll
    for (int j = 0; j < NP; ++j) {
      const float4 cs = __ldg(row + j);      // (cos, sin) of dims 2j and 2j+1 of this lane's slice
      c2[ps][j] = make_float2(cs.x, cs.z);
      s2[ps][j] = make_float2(cs.y, cs.w);
    }
  }

  Cursor pc = locate(p.kv_len, p.batch, p.n_kv_heads, x0, lane);   // producer cursor
  Cursor cc = pc;                                                  // consumer cursor
  int win_b = -1, win_e0 = 0, win_page = 0, win_pos = 0;           // 32 block-table entries, one per lane

  auto issue = [&](int stage) {
    const int e = pc.t >> p.log2_tpp;
    const int sub = pc.t & ((1 << p.log2_tpp) - 1);
    if (pc.b != win_b || e < win_e0 || e >= win_e0 + 32) {
      win_b = pc.b; win_e0 = e;
      const int n_ent = (pc.kvl + p.page_size - 1) / p.page_size;
      const bool ok = e + lane < n_ent;
      const size_t at = static_cast<size_t>(pc.b) * p.table_stride + e + lane;
      win_page = ok ? __ldg(p.page_ids + at) : 0;
      win_pos = ok ? __ldg(p.pos_base + at) : 0;
    }
    int page = __shfl_sync(kFull, win_page, e - win_e0);
    const int pos = __shfl_sync(kFull, win_pos, e - win_e0);
    if (lane == 0) {
      if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { atomicOr(p.status, MEPIC_DEV_BAD_PAGE); page = 0; }
      const size_t off = ((static_cast<size_t>(page) * p.n_kv_heads + pc.h) * p.page_size + static_cast<size_t>(sub) * kTile) * D;
      const uint32_t bar = smem_u32(&bars[stage]);
      const uint32_t dst = smem_u32(stage0 + static_cast<size_t>(stage) * 2 * kTileElems);
      meta[stage] = pos + sub * kTile;
      mbar_expect_tx(bar, kStageBytes);
      bulk_g2s(dst, p.k_pool + off, kTileElems * 2, bar);
      bulk_g2s(dst + kTileElems * 2, p.v_pool + off, kTileElems * 2, bar);
    }
    advance(pc, p.kv_len, p.batch, p.n_kv_heads);
  };

  int issued = 0;
  for (; issued < kStages && issued < n_tiles; ++issued) issue(issued);

  // per-unit state
  int ub = -1, uh = -1, qpos = 0;
  float qraw_lo[HPL][DL], qraw_hi[HPL][DL];   // this key group's heads, un-rotated, pre-scaled
  float m_mine = -INFINITY, l_mine = 0.f;
  float2 acc[G][DV / 2];

  auto flush = [&]() {
    if (ub < 0) return;
    float l_tot = l_mine;
    l_tot += __shfl_xor_sync(kFull, l_tot, 8);
    l_tot += __shfl_xor_sync(kFull, l_tot, 16);
    const long long slot = static_cast<long long>(ub) * p.n_kv_heads + uh + w;
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
      for (int j = 0; j < DV / 2; ++j) {
        acc[g][j].x += __shfl_xor_sync(kFull, acc[g][j].x, 16);
        acc[g][j].y += __shfl_xor_sync(kFull, acc[g][j].y, 16);
      }
      if (hw == 0) {
        float2* dst = reinterpret_cast<float2*>(p.part_o + (slot * G + g) * D + l16 * DV);
#pragma unroll
        for (int j = 0; j < DV / 2; ++j) dst[j] = acc[g][j];
      }
    }
    if (kg == 0 && (l8 % LPH) == 0 && my_head < G)
      *reinterpret_cast<float2*>(p.part_ml + (slot * G + my_head) * 2) = make_float2(m_mine, l_tot);
  };

  int stage = 0;
  uint32_t parity = 0;
  for (int it = 0; it < n_tiles; ++it) {
    if (cc.b != ub || cc.h != uh) {
      flush();
      ub = cc.b; uh = cc.h;
      qpos = __ldg(p.q_pos + ub);
      const int n_q_heads = p.n_kv_heads * G;
#pragma unroll
      for (int hh = 0; hh < HPL; ++hh) {
        const int head = kg + 4 * hh;
        if (head < G) {
          const uint32_t* src = reinterpret_cast<const uint32_t*>(
              p.q + (static_cast<size_t>(ub) * n_q_heads + static_cast<size_t>(uh) * G + head) * D);
#pragma unroll
          for (int j = 0; j < NP; ++j) {
            const float2 lo = bf16x2_to_float2(__ldg(src + l8 * NP + j));
            const float2 hi = bf16x2_to_float2(__ldg(src + D / 4 + l8 * NP + j));
            qraw_lo[hh][2 * j] = lo.x * p.scale_log2; qraw_lo[hh][2 * j + 1] = lo.y * p.scale_log2;
            qraw_hi[hh][2 * j] = hi.x * p.scale_log2; qraw_hi[hh][2 * j + 1] = hi.y * p.scale_log2;
          }
        } else {
#pragma unroll
          for (int j = 0; j < DL; ++j) { qraw_lo[hh][j] = 0.f; qraw_hi[hh][j] = 0.f; }
        }
      }
      m_mine = -INFINITY; l_mine = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int j = 0; j < DV / 2; ++j) acc[g][j] = make_float2(0.f, 0.f);
    }

    if (!mbar_wait_bounded(smem_u32(&bars[stage]), parity)) {
      // Give the copies still in flight a last bounded chance to land, then leave cleanly.
      if (lane == 0) atomicOr(p.status, MEPIC_DEV_WAIT_EXPIRED);
      for (int s = 0; s < kStages; ++s) mbar_wait_bounded(smem_u32(&bars[s]), s == stage ? parity : (s < stage ? parity ^ 1u : parity));
      return;
    }
    const uint16_t* ks = stage0 + static_cast<size_t>(stage) * 2 * kTileElems;
    const uint16_t* vs = ks + kTileElems;
    const int base = meta[stage];
    const int n_valid = min(kTile, cc.kvl - cc.t * kTile);

    // ---- rotate the G query vectors by (qpos - base): one table row, each key group does its heads
    {
      const int rel = qpos - base;
      int arel = rel < 0 ? -rel : rel;
      const float sgn = rel < 0 ? -1.f : 1.f;
      if (arel > p.max_position) { if (lane == 0) atomicOr(p.status, MEPIC_DEV_BAD_POSITION); arel = p.max_position; }
      const float4* row = reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(arel) * D + l8 * DL * 2);
      float4 cs[NP];
#pragma unroll
      for (int j = 0; j < NP; ++j) cs[j] = __ldg(row + j);
#pragma unroll
      for (int hh = 0; hh < HPL; ++hh) {
        const int head = kg + 4 * hh;
        if (head < G) {
          float lo[DL], hi[DL];
#pragma unroll
          for (int j = 0; j < NP; ++j) {
            const float c0 = cs[j].x, s0 = cs[j].y * sgn, c1 = cs[j].z, s1 = cs[j].w * sgn;
            lo[2 * j] = qraw_lo[hh][2 * j] * c0 - qraw_hi[hh][2 * j] * s0;
            hi[2 * j] = qraw_lo[hh][2 * j] * s0 + qraw_hi[hh][2 * j] * c0;
            lo[2 * j + 1] = qraw_lo[hh][2 * j + 1] * c1 - qraw_hi[hh][2 * j + 1] * s1;
            hi[2 * j + 1] = qraw_lo[hh][2 * j + 1] * s1 + qraw_hi[hh][2 * j + 1] * c1;
          }
          // layout: float4 index (head * 2*DL/4 + part) * 8 + l8 ; parts = lo quads then hi quads
#pragma unroll
          for (int part = 0; part < DL / 4; ++part) {
            qrot[(head * (DL / 2) + part) * 8 + l8] = make_float4(lo[4 * part], lo[4 * part + 1], lo[4 * part + 2], lo[4 * part + 3]);
            qrot[(head * (DL / 2) + DL / 4 + part) * 8 + l8] = make_float4(hi[4 * part], hi[4 * part + 1], hi[4 * part + 2], hi[4 * part + 3]);
          }
        }
      }
    }
    __syncwarp();
    float2 qlo[G][NP], qhi[G][NP];
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
      for (int part = 0; part < DL / 4; ++part) {
        const float4 a = qrot[(g * (DL / 2) + part) * 8 + l8];
        const float4 b = qrot[(g * (DL / 2) + DL / 4 + part) * 8 + l8];
        qlo[g][2 * part] = make_float2(a.x, a.y); qlo[g][2 * part + 1] = make_float2(a.z, a.w);
        qhi[g][2 * part] = make_float2(b.x, b.y); qhi[g][2 * part + 1] = make_float2(b.z, b.w);
      }
    }

    // ---- K phase: rotate each key by its in-tile offset, dot with the G queries, reduce over 8 lanes
    float sc[4];
#pragma unroll
    for (int ps = 0; ps < 4; ++ps) {
      const int r = kg + 4 * ps;
      const uint32_t* krow = reinterpret_cast<const uint32_t*>(ks + r * D);
      uint32_t wlo[NP], whi[NP];
      if constexpr (NP == 4) {
        const uint4 a = *reinterpret_cast<const uint4*>(krow + l8 * 4);
        const uint4 b = *reinterpret_cast<const uint4*>(krow + D / 4 + l8 * 4);
        wlo[0] = a.x; wlo[1] = a.y; wlo[2] = a.z; wlo[3] = a.w;
        whi[0] = b.x; whi[1] = b.y; whi[2] = b.z; whi[3] = b.w;
      } else {
        const uint2 a = *reinterpret_cast<const uint2*>(krow + l8 * 2);
        const uint2 b = *reinterpret_cast<const uint2*>(krow + D / 4 + l8 * 2);
        wlo[0] = a.x; wlo[1] = a.y; whi[0] = b.x; whi[1] = b.y;
      }
      float2 dot[GP];
#pragma unroll
      for (int g = 0; g < GP; ++g) dot[g] = make_float2(0.f, 0.f);
#pragma unroll
      for (int j = 0; j < NP; ++j) {
        const float2 lo = bf16x2_to_float2(wlo[j]);
        const float2 hi = bf16x2_to_float2(whi[j]);
        const float2 klo = sub2(mul2(lo, c2[ps][j]), mul2(hi, s2[ps][j]));
        const float2 khi = fma2(lo, s2[ps][j], mul2(hi, c2[ps][j]));
#pragma unroll
        for (int g = 0; g < G; ++g) {
          dot[g] = fma2(qlo[g][j], klo, dot[g]);
          dot[g] = fma2(qhi[g][j], khi, dot[g]);
        }
      }
      float v[GP];
#pragma unroll
      for (int g = 0; g < GP; ++g) v[g] = dot[g].x + dot[g].y;
      // reduce-scatter over the 8 dim lanes: halve the number of live heads per step while any remain
      int cnt = GP;
#pragma unroll
      for (int msk = 4; msk >= 1; msk >>= 1) {
        if (cnt > 1) {
          const bool upper = (l8 & msk) != 0;
#pragma unroll
          for (int i = 0; i < GP / 2; ++i) {
            if (i < cnt / 2) {
              const float keep = upper ? v[i + cnt / 2] : v[i];
              const float send = upper ? v[i] : v[i + cnt / 2];
              v[i] = keep + __shfl_xor_sync(kFull, send, msk);
            }
          }
          cnt >>= 1;
        } else {
          v[0] += __shfl_xor_sync(kFull, v[0], msk);
        }
      }
      sc[ps] = (r < n_valid) ? v[0] : -INFINITY;
    }

    // ---- online softmax for this lane's head (log2 domain)
    float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 8));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 16));
    if (__any_sync(kFull, mx > m_mine)) {
      const float m_new = fmaxf(m_mine, mx);
      const float alpha = ex2(m_mine - m_new);     // 0 on the first tile (m_mine = -inf)
      m_mine = m_new;
      l_mine *= alpha;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float a = __shfl_sync(kFull, alpha, g * LPH);
#pragma unroll
        for (int j = 0; j < DV / 2; ++j) { acc[g][j].x *= a; acc[g][j].y *= a; }
      }
    }
#pragma unroll
    for (int ps = 0; ps < 4; ++ps) {
      const float pr = ex2(sc[ps] - m_mine);
      l_mine += pr;
      if ((l8 % LPH) == 0) pbuf[(kg + 4 * ps) * PSTR + my_head] = pr;
    }
    __syncwarp();

    // ---- V phase: half warps take alternate keys, 16 lanes span the row
#pragma unroll
    for (int i = 0; i < kTile / 2; ++i) {
      const int key = 2 * i + hw;
      if (key < n_valid) {
        float pg[8];
        const float4 p0 = *reinterpret_cast<const float4*>(pbuf + key * PSTR);
        pg[0] = p0.x; pg[1] = p0.y; pg[2] = p0.z; pg[3] = p0.w;
        if constexpr (GP == 8) {
          const float4 p1 = *reinterpret_cast<const float4*>(pbuf + key * PSTR + 4);
          pg[4] = p1.x; pg[5] = p1.y; pg[6] = p1.z; pg[7] = p1.w;
        }
        const uint32_t* vrow = reinterpret_cast<const uint32_t*>(vs + key * D + l16 * DV);
        uint32_t wv[DV / 2];
        if constexpr (DV == 8) {
          const uint4 a = *reinterpret_cast<const uint4*>(vrow);
          wv[0] = a.x; wv[1] = a.y; wv[2] = a.z; wv[3] = a.w;
        } else {
          const uint2 a = *reinterpret_cast<const uint2*>(vrow);
          wv[0] = a.x; wv[1] = a.y;
        }
#pragma unroll
        for (int j = 0; j < DV / 2; ++j) {
          const float2 vv = bf16x2_to_float2(wv[j]);
#pragma unroll
          for (int g = 0; g < G; ++g) acc[g][j] = fma2(make_float2(pg[g], pg[g]), vv, acc[g][j]);
        }
      }
    }
    __syncwarp();   // every lane is done with this stage, qrot and pbuf

    if (issued < n_tiles) { issue(stage); ++issued; }
    advance(cc, p.kv_len, p.batch, p.n_kv_heads);
    if (++stage == kStages) { stage = 0; parity ^= 1u; }
  }
  flush();
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
    const Cut cut = cut_of_line(p.kv_len, p.batch, p.n_kv_heads, p.n_workers, lane);
    long long before = 0;
    for (int b0 = 0; b0 < b; b0 += 32) {
      const int n = (b0 + lane < b) ? tiles_of(p.kv_len[b0 + lane]) : 0;
      before += warp_sum(n);
    }
    if (lane == 0) { sh[0] = cut.piece; sh[1] = before; sh[2] = tiles_of(p.kv_len[b]); }
  }
  __syncthreads();
  const long long piece = sh[0], nt = sh[2];
  const int g = threadIdx.x / D, d = threadIdx.x % D;
  const size_t o_at = (static_cast<size_t>(b) * p.n_kv_heads * G + static_cast<size_t>(h) * G + g) * D + d;
  if (nt == 0) { p.out[o_at] = 0; return; }
  const long long u0 = sh[1] * p.n_kv_heads + static_cast<long long>(h) * nt;
  const long long w_first = u0 / piece, w_last = (u0 + nt - 1) / piece;
  const long long unit = static_cast<long long>(b) * p.n_kv_heads + h;
  float m_star = -INFINITY;
  for (long long wk = w_first; wk <= w_last; ++wk) m_star = fmaxf(m_star, p.part_ml[((unit + wk) * G + g) * 2]);
  float l_star = 0.f, o_star = 0.f;
  for (long long wk = w_first; wk <= w_last; ++wk) {
    const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + ((unit + wk) * G + g) * 2);
    const float wgt = ex2(ml.x - m_star);
    l_star += ml.y * wgt;
    o_star += p.part_o[((unit + wk) * G + g) * D + d] * wgt;
  }
  const float r = o_star / l_star;
  // fp32 -> bf16, round to nearest even
  uint32_t u = __float_as_uint(r);
  u += 0x7fffu + ((u >> 16) & 1u);
  p.out[o_at] = (r != r) ? 0x7fc0 : static_cast<uint16_t>(u >> 16);
}

template <int D, int G>
constexpr size_t decode_smem_bytes() {
  constexpr int GP = G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8;
  constexpr int PSTR = GP < 4 ? 4 : GP;
  return static_cast<size_t>(kWarps) * (stages_for(D, G) * (2 * kTile * D * 2) + G * D * 4 + kTile * PSTR * 4 + 64);
}

template <int D, int G>
int32_t launch_decode(const DecodeParams& p, int n_ctas, cudaStream_t stream) {
  constexpr size_t smem = decode_smem_bytes<D, G>();
  cudaError_t e = cudaFuncSetAttribute(mepic_decode_splitkv<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) { mepic_set_error("decode: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_decode_splitkv<D, G><<<n_ctas, kWarps * 32, smem, stream>>>(p);
  mepic_decode_merge<D, G><<<p.batch * p.n_kv_heads, G * D, 0, stream>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) { mepic_set_error("decode: launch: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_count_launches(2);
  return MEPIC_OK;
}

int sm_count_of_current_device() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

size_t decode_slots(const mepic_config_t* cfg, int batch, int sms) {
  return static_cast<size_t>(batch) * cfg->n_kv_heads + static_cast<size_t>(sms) * kWarps;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" size_t mepic_attn_decode_workspace(const mepic_config_t* cfg, int32_t batch) {
  if (!mepic_config_ok(cfg) || batch < 1) return 0;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) { mepic_set_error("decode_workspace: no CUDA device"); return 0; }
  const int G = cfg->n_q_heads / cfg->n_kv_heads;
  return decode_slots(cfg, batch, sms) * G * (cfg->head_dim + 2) * sizeof(float);
}

extern "C" int32_t mepic_attn_decode(const mepic_config_t* cfg, const mepic_decode_args_t* a, void* cuda_stream) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (!a || !a->q || !a->k_pool || !a->v_pool || !a->page_ids || !a->pos_base || !a->kv_len || !a->q_pos ||
      !a->rope_table || !a->out || !a->workspace || !a->status) { mepic_set_error("decode: NULL pointer argument"); return MEPIC_E_INVAL; }
  if (a->batch < 1 || a->table_stride < 1) { mepic_set_error("decode: batch and table_stride must be positive"); return MEPIC_E_INVAL; }
  if (!aligned16(a->q) || !aligned16(a->k_pool) || !aligned16(a->v_pool) || !aligned16(a->workspace) ||
      !aligned16(a->rope_table) || !aligned16(a->out)) { mepic_set_error("decode: pointers must be 16-byte aligned"); return MEPIC_E_INVAL; }
  if (cfg->max_position < kTile - 1) { mepic_set_error("decode: rope table must cover positions 0..15"); return MEPIC_E_INVAL; }
  const int sms = sm_count_of_current_device();
  if (sms <= 0) { mepic_set_error("decode: no CUDA device"); return MEPIC_E_CUDA; }
  const int G = cfg->n_q_heads / cfg->n_kv_heads, D = cfg->head_dim;
  const size_t slots = decode_slots(cfg, a->batch, sms);
  const size_t need = slots * G * (D + 2) * sizeof(float);
  if (a->workspace_bytes < need) { mepic_set_error("decode: workspace %zu < %zu bytes", a->workspace_bytes, need); return MEPIC_E_INVAL; }

  DecodeParams p;
  p.q = static_cast<const uint16_t*>(a->q);
  p.k_pool = static_cast<const uint16_t*>(a->k_pool);
  p.v_pool = static_cast<const uint16_t*>(a->v_pool);
  p.page_ids = a->page_ids; p.pos_base = a->pos_base; p.kv_len = a->kv_len; p.q_pos = a->q_pos;
  p.rope = a->rope_table;
  p.part_o = static_cast<float*>(a->workspace);
  p.part_ml = p.part_o + slots * G * D;
  p.out = static_cast<uint16_t*>(a->out);
  p.status = a->status;
  p.table_stride = a->table_stride; p.batch = a->batch; p.n_kv_heads = cfg->n_kv_heads;
  p.page_size = cfg->page_size;
  int l2 = 0; while ((kTile << l2) < cfg->page_size) ++l2;
  p.log2_tpp = l2;
  p.num_pages = cfg->num_pages; p.max_position = cfg->max_position;
  p.n_workers = sms * kWarps;
  p.scale_log2 = a->sm_scale * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

#define MEPIC_DECODE_CASE(DD, GG) if (D == DD && G == GG) return launch_decode<DD, GG>(p, sms, st);
  MEPIC_DECODE_CASE(128, 1) MEPIC_DECODE_CASE(128, 2) MEPIC_DECODE_CASE(128, 4) MEPIC_DECODE_CASE(128, 5) MEPIC_DECODE_CASE(128, 8)
  MEPIC_DECODE_CASE(64, 1) MEPIC_DECODE_CASE(64, 2) MEPIC_DECODE_CASE(64, 4) MEPIC_DECODE_CASE(64, 5) MEPIC_DECODE_CASE(64, 8)
#undef MEPIC_DECODE_CASE
  mepic_set_error("decode: unsupported head_dim %d / group size %d", D, G);
  return MEPIC_E_INVAL;
}

// ---------------------------------------------------------------- decode without any allocation by anyone
//
// Some callers cannot obtain device memory at the moment they need to decode: code running
// inside a memory-pool or allocator callback, an inference plug-in whose host forbids calls
// into the device allocator after start-up, a process whose device memory is fully handed to
// the page pool.  For them the split-KV partials live in the fixed array below instead of a
// caller-provided workspace.  Every GPU that loads this library holds the array until the
// process exits.
namespace {

__device__ __align__(256) unsigned char g_decode_static_scratch[MEPIC_DECODE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal; filled on first use

// In host code the array's name is only a host-side handle, not a device address: the address a
// kernel can use has to be asked from the runtime, once per device, with that device current.
int32_t static_scratch_of_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { mepic_set_error("decode_static: cudaGetDevice: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) { mepic_set_error("decode_static: device ordinal %d not supported", dev); return MEPIC_E_INVAL; }
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_decode_static_scratch);
    if (e != cudaSuccess || !ptr) {
      mepic_set_error("decode_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
      return MEPIC_E_CUDA;
    }
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return MEPIC_OK;
}

}  // namespace

extern "C" int32_t mepic_attn_decode_static(const mepic_config_t* cfg, const mepic_decode_args_t* a, void* cuda_stream) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (!a) { mepic_set_error("decode_static: args is NULL"); return MEPIC_E_INVAL; }
  if (a->batch < 1) { mepic_set_error("decode_static: batch must be positive"); return MEPIC_E_INVAL; }
  const size_t need = mepic_attn_decode_workspace(cfg, a->batch);
  if (need == 0) return MEPIC_E_CUDA;
  if (need > static_cast<size_t>(MEPIC_DECODE_STATIC_SCRATCH_BYTES)) {
    mepic_set_error("decode_static: this batch and config need %zu bytes of scratch; the built-in array holds %zu "
                    "(use mepic_attn_decode with a caller workspace)", need, static_cast<size_t>(MEPIC_DECODE_STATIC_SCRATCH_BYTES));
    return MEPIC_E_INVAL;
  }
  void* scratch = nullptr;
  const int32_t rc = static_scratch_of_current_device(&scratch);
  if (rc != MEPIC_OK) return rc;
  mepic_decode_args_t with_scratch = *a;
  with_scratch.workspace = scratch;
  with_scratch.workspace_bytes = MEPIC_DECODE_STATIC_SCRATCH_BYTES;
  return mepic_attn_decode(cfg, &with_scratch, cuda_stream);
}
