// fp8 (e4m3) chunk pages: the quantiser that turns bf16 pages into 8-bit pages with one scale per
// (page, kv head) block, and the RoPE-fused split-KV decode that reads them.
//
// The paper leaves KV compression to related work; the format here is this build's: OCP E4M3 codes,
// scale = max|x| / 448 of the block (1 for an all-zero block), code = E4M3(x / scale) rounded to
// nearest-even and saturating, all in fp32.  Keys stay un-rotated in the pages, exactly as in bf16.
//
// Decode kernel.  Same work decomposition, ring, cursor, partials and merge as the bf16 per-request
// kernel (mepic_decode.cu); what differs is the way a tile reaches the tensor cores:
//   * a 16-token tile of one head is 16 rows x 128 bytes, one TMA box per pool (2 KB instead of 4);
//   * E4M3 values are exact in fp16, so codes are widened with cvt.f16x2.e4m3x2 and both
//     contractions run as fp16 MMAs (fp32 accumulate); the scales are applied to the fp32 scores
//     (K) and to P before it is packed (V), never to the 8-bit data;
//   * the keys are the M rows of both MMAs (S^T = K' Q^T, O^T = V^T P^T), the query heads the N columns, as in the
//     bf16 kernel.  ldmatrix (16-bit elements) on 8-bit rows hands a lane FOUR consecutive dims of a key where the
//     bf16 layout hands it two, and the transposing 8-bit ldmatrix (m16n16) hands it four consecutive KEYS of a dim.
//     The MMA does not care which physical index sits at which k position as long as A and B agree, so the query
//     fragments use the same dim order (pairs 16j + 4t + 2r), and the M rows of the score MMA are the keys in the
//     order {0,1,4,5,8,9,12,13} / {2,3,6,7,10,11,14,15}: after the movmatrix transposition of the probabilities a
//     lane's P^T fragments are keys 4t..4t+3 - the four keys its V^T fragments carry;
//   * the query rotation runs in packed fp16 (the rotated query is rounded to fp16 for the MMA anyway), which with
//     the halved accumulators leaves a thread at 168 registers: 12 warps per SM with a 3-stage ring each.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mepic.h"
#include "mepic_internal.h"
#include "mepic_decode_line.cuh"

namespace {

using namespace mepic_dev;

// ---------------------------------------------------------------- quantiser
// One CTA per (listed page, kv head): block maximum, scale, codes.
__global__ void __launch_bounds__(256) mepic_quantize_pages(const uint16_t* src, unsigned char* dst, float* scales, const int32_t* pages,
                                                            int n_kv_heads, int elems, int num_pages, int32_t* status) {
  const int page = pages[blockIdx.x / n_kv_heads], h = blockIdx.x % n_kv_heads;
  if (static_cast<unsigned>(page) >= static_cast<unsigned>(num_pages)) { if (threadIdx.x == 0) atomicOr(status, MEPIC_DEV_BAD_PAGE); return; }
  const size_t base = (static_cast<size_t>(page) * n_kv_heads + h) * elems;
  const uint4* in = reinterpret_cast<const uint4*>(src + base);
  float amax = 0.f;
  for (int c = threadIdx.x; c < elems / 8; c += blockDim.x) {
    const uint4 w = in[c];
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 f = bf16x2_to_float2(ww[k]);
      amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));       // fmaxf drops NaN operands: a NaN element does not set the scale
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, o));
  __shared__ float part[8];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = part[0];
#pragma unroll
  for (int k = 1; k < 8; ++k) amax = fmaxf(amax, part[k]);
  const float scale = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
  if (threadIdx.x == 0) scales[static_cast<size_t>(page) * n_kv_heads + h] = scale;
  uint2* out = reinterpret_cast<uint2*>(dst + base);
  for (int c = threadIdx.x; c < elems / 8; c += blockDim.x) {
    const uint4 w = in[c];
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    uint32_t codes[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 f = bf16x2_to_float2(ww[k]);
      uint16_t pair;      // low byte = the lower element
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(__fdiv_rn(f.y, scale)), "f"(__fdiv_rn(f.x, scale)));
      codes[k] = pair;
    }
    out[c] = make_uint2(codes[0] | (codes[1] << 16), codes[2] | (codes[3] << 16));
  }
}

#ifndef MEPIC_FP8_STAGES
#define MEPIC_FP8_STAGES 3
#endif
constexpr int kFp8Stages = MEPIC_FP8_STAGES;               // depth of each warp's ring of staged tiles

template <int G>
__global__ void __launch_bounds__(kWarpsFp8 * 32, 1)
mepic_decode_splitkv_fp8(const DecodeParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  constexpr int D = 128;
  constexpr int kStages = kFp8Stages;
  constexpr int KH = D / 32;                 // k-steps per half: 16-dim block j pairs with block j + KH
  constexpr int NV = D / 16;                 // 16-dim blocks of the output (M tiles of the PV product)
  constexpr int kBlockBytes = kTile * 128;   // one tile of one pool: 16 rows x 128 bytes
  constexpr int kStageBytes = 2 * kBlockBytes;
  constexpr int kWarpBytes = kStages * kStageBytes;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  unsigned char* stage0 = smem + static_cast<size_t>(wic) * kWarpBytes;
  float* rope_rows = reinterpret_cast<float*>(smem + static_cast<size_t>(kWarpsFp8) * kWarpBytes) + static_cast<size_t>(wic) * kStages * D;
  unsigned char* misc = smem + static_cast<size_t>(kWarpsFp8) * (kWarpBytes + kStages * D * 4) + wic * 128;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);                   // kStages x 8 bytes
  volatile float* meta = reinterpret_cast<volatile float*>(misc + 32);  // per stage: sign of (q position - tile base), K scale, V scale

  const int g = lane >> 2;       // fragment row group: head g (A, C) / row g of a key n-tile (B)
  const int t = lane & 3;        // fragment column group
  // keys behind row g of the two key n-tiles
  const int key0 = 4 * (g >> 1) + (g & 1), key1 = key0 + 2;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const long long w = static_cast<long long>(blockIdx.x) * kWarpsFp8 + wic;
  const Cut cut = cut_of_line(p, lane);
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

  // cos/sin of the in-tile offsets of this lane's two keys, pairs 16j + 4t + 2r + {0,1}, as packed fp16 (cos, sin)
  uint32_t kc[2][KH][2], ksn[2][KH][2];      // [key set][k-step][column pair]
#pragma unroll
  for (int kq = 0; kq < 2; ++kq)
#pragma unroll
    for (int j = 0; j < KH; ++j)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float4 cs = __ldg(reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(kq ? key1 : key0) * D + 2 * (16 * j + 4 * t + 2 * r)));
        kc[kq][j][r] = pack_f16x2(cs.x, cs.z);
        ksn[kq][j][r] = pack_f16x2(cs.y, cs.w);
      }

  Cursor pc = locate(p.kv_len, p.batch, p.n_kv_heads, x0, lane);   // producer cursor
  Cursor cc = pc;                                                  // consumer cursor
  int win_b = -1, win_h = -1, win_e0 = 0, win_page = 0, win_pos = 0;   // 32 block-table entries, one per lane
  float win_ks = 1.f, win_vs = 1.f;                                // and the scales of their (page, head) blocks
  int win_qpos = 0;

  int issued = 0;     // tiles handed to the ring so far = index of the tile issue() is called for
  auto issue = [&](int stage) {
    const int e = pc.t >> p.log2_tpp;
    const int sub = pc.t & ((1 << p.log2_tpp) - 1);
    if (pc.b != win_b || pc.h != win_h || e < win_e0 || e >= win_e0 + 32) {
      if (pc.b != win_b) win_qpos = __ldg(p.q_pos + pc.b);
      win_b = pc.b; win_h = pc.h; win_e0 = e;
      const int n_ent = (pc.kvl + p.page_size - 1) / p.page_size;
      const bool ok = e + lane < n_ent;
      const size_t at = static_cast<size_t>(pc.b) * p.table_stride + e + lane;
      win_page = ok ? __ldg(p.page_ids + at) : 0;
      win_pos = ok ? __ldg(p.pos_base + at) : 0;
      const bool page_ok = ok && static_cast<unsigned>(win_page) < static_cast<unsigned>(p.num_pages);
      win_ks = page_ok ? __ldg(p.k_scales + static_cast<size_t>(win_page) * p.n_kv_heads + pc.h) : 1.f;
      win_vs = page_ok ? __ldg(p.v_scales + static_cast<size_t>(win_page) * p.n_kv_heads + pc.h) : 1.f;
    }
    int page = __shfl_sync(kFull, win_page, e - win_e0);
    const int pos = __shfl_sync(kFull, win_pos, e - win_e0);
    const float ks = __shfl_sync(kFull, win_ks, e - win_e0), vs = __shfl_sync(kFull, win_vs, e - win_e0);
    if (lane == 0 && !(w == 0 && issued == p.skip_tile)) {     // (test hook: one copy that never comes)
      if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { atomicOr(p.status, MEPIC_DEV_BAD_PAGE); page = 0; }
      const int y = (page * p.n_kv_heads + pc.h) * p.page_size + sub * kTile;     // row of the pool viewed as [rows][128 bytes]
      const uint32_t bar = smem_u32(&bars[stage]);
      const uint32_t dst = smem_u32(stage0 + static_cast<size_t>(stage) * kStageBytes);
      const int rel = win_qpos - (pos + sub * kTile);
      int arel = rel < 0 ? -rel : rel;
      if (arel > p.max_position) { atomicOr(p.status, MEPIC_DEV_BAD_POSITION); arel = p.max_position; }
      meta[stage * 4] = rel < 0 ? -1.f : 1.f;
      meta[stage * 4 + 1] = ks;
      meta[stage * 4 + 2] = vs;
      mbar_expect_tx(bar, kStageBytes + D * 4);
      tma_load_2d(dst, &map_k, 0, y, bar);
      tma_load_2d(dst + kBlockBytes, &map_v, 0, y, bar);
      bulk_g2s(smem_u32(rope_rows + stage * D), p.rope + static_cast<size_t>(arel) * D, D * 4, bar);
    }
    advance(pc, p.kv_len, p.batch, p.n_kv_heads);
  };

  for (; issued < kStages && issued < n_tiles; ++issued) issue(issued);
  __syncwarp();

  // The keys are the M rows of both MMAs (S^T = K' Q^T, O^T = V^T P^T) and the query heads the N columns: this lane's B
  // fragments of Q^T hold head g; its accumulators hold heads 2t, 2t+1 for the keys key0 / key1 (scores) and for dims g,
  // g+8 of every 16-dim block (output).
  int ub = -1, uh = -1;
  uint32_t q_lo[KH][2], q_hi[KH][2];        // un-rotated q of head g as packed fp16 pairs, pre-scaled by sm_scale*log2e: pairs as for kc/ksn
  float m_run[2] = {-INFINITY, -INFINITY};  // running maximum of heads 2t, 2t+1 (the same in the 8 lanes that share t)
  float l_run[2] = {0.f, 0.f};              // this lane's share (its two keys of every tile) of the two heads' sums
  float acc[NV][4];                         // O^T fragments: [16-dim block][dim g: head 2t, 2t+1 | dim g+8: head 2t, 2t+1]

  auto flush = [&]() {
    if (ub < 0) return;
    float l0 = l_run[0], l1 = l_run[1];
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) { l0 += __shfl_xor_sync(kFull, l0, o); l1 += __shfl_xor_sync(kFull, l1, o); }
    const long long slot = static_cast<long long>(ub) * p.n_kv_heads + uh + w;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int hh = 2 * t + c;
      if (hh < G) {
        float* dst = p.part_o + (slot * G + hh) * D;
#pragma unroll
        for (int db = 0; db < NV; ++db) { dst[16 * db + g] = acc[db][c]; dst[16 * db + 8 + g] = acc[db][2 + c]; }
        if (g == 0) *reinterpret_cast<float2*>(p.part_ml + (slot * G + hh) * 2) = make_float2(m_run[c], c ? l1 : l0);
      }
    }
  };

  // ---- the pieces of one tile's work, as functions of the ring stage
  // bounded wait for a stage; on expiry the status bit is set and the other stages get one more bounded wait each
  int stage = 0;
  uint32_t parity = 0;
  auto landed = [&](int st, uint32_t par) {
    if (mbar_wait_bounded(smem_u32(&bars[st]), par, p.spin_limit)) return true;
    if (lane == 0) atomicOr(p.status, MEPIC_DEV_WAIT_EXPIRED);
    for (int s = 0; s < kStages; ++s) mbar_wait_bounded(smem_u32(&bars[s]), s == stage ? parity : (s < stage ? parity ^ 1u : parity), p.spin_limit);
    return false;
  };
  // S^T of the tile in stage st (log2 domain, K scale applied): sc = {key0: head 2t, 2t+1 | key1: head 2t, 2t+1}
  auto scores = [&](int st, float (&sc)[4]) {
    const uint32_t ks_addr = smem_u32(stage0 + static_cast<size_t>(st) * kStageBytes);
    const uint32_t sgn_bits = meta[st * 4] < 0.f ? 0x80008000u : 0u;     // a negative angle flips the sines
    const float k_scale = meta[st * 4 + 1];
    // B fragments of Q^T: head g rotated by (qpos - tile base), fp16, from the table row that came with the tile
    uint32_t qa[2 * KH][2];                     // [k-step][b0 (dims 16j+4t,+1) | b1 (dims 16j+4t+2,+3)], column = head g
    const float* row = rope_rows + st * D;
#pragma unroll
    for (int j = 0; j < KH; ++j)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        // packed fp16 arithmetic: the rotated query is rounded to fp16 for the MMA anyway
        const float4 cs = *reinterpret_cast<const float4*>(row + 2 * (16 * j + 4 * t + 2 * r));
        const uint32_t c2 = pack_f16x2(cs.x, cs.z), s2 = pack_f16x2(cs.y, cs.w) ^ sgn_bits;
        qa[j][r] = f16x2_fma(q_lo[j][r], c2, f16x2_neg(f16x2_mul(q_hi[j][r], s2)));       // lo cos - hi sin
        qa[j + KH][r] = f16x2_fma(q_lo[j][r], s2, f16x2_mul(q_hi[j][r], c2));             // lo sin + hi cos
      }
    // one ldmatrix per k-step pair brings, for both key sets (M rows 0-7 and 8-15), 16 dims of the lower half and their
    // partners of the upper half; widened to fp16 and rotated in registers.  Two accumulators so that the MMAs of the
    // two halves do not wait on each other.
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < KH; ++j) {
      uint32_t raw[4];            // [key set 0 lower, key set 1 lower, key set 0 upper, key set 1 upper], 4 dims each
      {
        // lane -> (matrix mi = lane / 8, row = lane % 8): key of that row in key set (mi & 1), 16-byte chunk j (+ KH)
        const int mi = lane >> 3, rr = lane & 7;
        const int key = 4 * (rr >> 1) + (rr & 1) + 2 * (mi & 1);
        const int ch = j + KH * (mi >> 1);
        ldmatrix_x4(raw, ks_addr + key * 128 + ((ch ^ (key & 7)) << 4));
      }
      uint32_t lo[4], hi[4];      // [key0: dims 4t,+1 | key0: dims 4t+2,+3 | key1: ... | key1: ...] of k-step j / j + KH
      e4m3x4_to_f16x2x2(raw[0], lo[0], lo[1]);
      e4m3x4_to_f16x2x2(raw[1], lo[2], lo[3]);
      e4m3x4_to_f16x2x2(raw[2], hi[0], hi[1]);
      e4m3x4_to_f16x2x2(raw[3], hi[2], hi[3]);
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const int kq = f >> 1, r = f & 1;       // key of set kq, column pair r
        const uint32_t a = lo[f], b = hi[f];
        lo[f] = f16x2_fma(a, kc[kq][j][r], f16x2_neg(f16x2_mul(b, ksn[kq][j][r])));     // lo cos - hi sin
        hi[f] = f16x2_fma(a, ksn[kq][j][r], f16x2_mul(b, kc[kq][j][r]));                // lo sin + hi cos
      }
      // A = (row g: key0, row g+8: key1) x (k columns 2t,+1 <-> dims 4t,+1 ; k columns 2t+8,+9 <-> dims 4t+2,+3)
      mma_f16(sa, lo[0], lo[2], lo[1], lo[3], qa[j][0], qa[j][1]);
      mma_f16(sb, hi[0], hi[2], hi[1], hi[3], qa[j + KH][0], qa[j + KH][1]);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) sc[k] = (sa[k] + sb[k]) * k_scale;
  };
  // slots at or past kv_len may hold any code (NaN included): P is 0 there, but 0 x NaN is NaN, so V must be finite;
  // their scores are masked
  auto tail = [&](int st, int n_valid, float (&sc)[4]) {
    const uint32_t vs_addr = smem_u32(stage0 + static_cast<size_t>(st) * kStageBytes) + kBlockBytes;
    for (int idx = n_valid * 8 + lane; idx < kTile * 8; idx += 32) {
      const int key = idx / 8, ch = idx % 8;
      const uint32_t a = vs_addr + key * 128 + ((ch ^ (key & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
    }
    // these generic-proxy stores must be ordered before the TMA (async proxy) write that refills this stage
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (key0 >= n_valid) { sc[0] = -INFINITY; sc[1] = -INFINITY; }
    if (key1 >= n_valid) { sc[2] = -INFINITY; sc[3] = -INFINITY; }
  };
  // O^T += V^T P^T for the tile in stage st; p = the tile's four probabilities of this lane (V scale not yet applied)
  auto pv = [&](int st, float p0, float p1, float p2, float p3) {
    const uint32_t vs_addr = smem_u32(stage0 + static_cast<size_t>(st) * kStageBytes) + kBlockBytes;
    const float v_scale = meta[st * 4 + 2];
    // B fragments of P^T carrying the V scale of the tile: the transposes of the two 8 x 8 blocks (key row, head columns);
    // row r of block 0 is key 4 (r / 2) + r % 2 and of block 1 that key + 2, so b0 = keys 4t, 4t+1 and b1 = keys 4t+2, 4t+3
    const uint32_t pb0 = movmatrix_trans(pack_f16x2(p0 * v_scale, p1 * v_scale)), pb1 = movmatrix_trans(pack_f16x2(p2 * v_scale, p3 * v_scale));
    // the transposing 8-bit ldmatrix hands this lane keys 4t..4t+3 of dims g and g + 8 of a 16-dim block
#pragma unroll
    for (int c = 0; c < NV; c += 2) {
      uint32_t raw[4];            // [block c: dim g, dim g + 8 | block c + 1: dim g, dim g + 8]
      {
        const int key = lane & 15, ch = c + (lane >> 4);
        ldmatrix_b8_trans_x2(raw, vs_addr + key * 128 + ((ch ^ (key & 7)) << 4));
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        uint32_t a0, a2, a1, a3;  // dim g: keys 4t,+1 | keys 4t+2,+3 ; dim g + 8: the same
        e4m3x4_to_f16x2x2(raw[2 * k], a0, a2);
        e4m3x4_to_f16x2x2(raw[2 * k + 1], a1, a3);
        mma_f16(acc[c + k], a0, a1, a2, a3, pb0, pb1);
      }
    }
  };
  // the running maxima move only if some lane saw a larger score: only then is the maximum over the lanes worked out
  auto raise = [&](float mx0, float mx1) {
    if (!__any_sync(kFull, mx0 > m_run[0] || mx1 > m_run[1])) return;
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) { mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, o)); mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, o)); }
    const float n0 = fmaxf(m_run[0], mx0), n1 = fmaxf(m_run[1], mx1);
    const float a0 = ex2(m_run[0] - n0), a1 = ex2(m_run[1] - n1);     // 0 on the first tile (m_run = -inf)
    m_run[0] = n0; m_run[1] = n1;
    l_run[0] *= a0; l_run[1] *= a1;
#pragma unroll
    for (int db = 0; db < NV; ++db) { acc[db][0] *= a0; acc[db][1] *= a1; acc[db][2] *= a0; acc[db][3] *= a1; }
  };

  int it = 0;
  while (it < n_tiles) {
    if (cc.b != ub || cc.h != uh) {
      flush();
      ub = cc.b; uh = cc.h;
      const int n_q_heads = p.n_kv_heads * G;
      const uint32_t* src = reinterpret_cast<const uint32_t*>(
          p.q + (static_cast<size_t>(ub) * n_q_heads + static_cast<size_t>(uh) * G + (g < G ? g : 0)) * D);
#pragma unroll
      for (int j = 0; j < KH; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int pair = 16 * j + 4 * t + 2 * r;              // dims pair, pair+1 and their partners + D/2
          const float2 lo = bf16x2_to_float2(__ldg(src + pair / 2));
          const float2 hi = bf16x2_to_float2(__ldg(src + (pair + D / 2) / 2));
          const float sc = g < G ? p.scale_log2 : 0.f;
          q_lo[j][r] = pack_f16x2(lo.x * sc, lo.y * sc);
          q_hi[j][r] = pack_f16x2(hi.x * sc, hi.y * sc);
        }
      m_run[0] = m_run[1] = -INFINITY; l_run[0] = l_run[1] = 0.f;
#pragma unroll
      for (int db = 0; db < NV; ++db) { acc[db][0] = 0.f; acc[db][1] = 0.f; acc[db][2] = 0.f; acc[db][3] = 0.f; }
    }
    if (!landed(stage, parity)) return;
    {
      float sA[4];
      scores(stage, sA);
      const int n_valid = min(kTile, cc.kvl - cc.t * kTile);
      if (n_valid < kTile) tail(stage, n_valid, sA);
      raise(fmaxf(sA[0], sA[2]), fmaxf(sA[1], sA[3]));
      const float a0 = ex2(sA[0] - m_run[0]), a1 = ex2(sA[1] - m_run[1]), a2 = ex2(sA[2] - m_run[0]), a3 = ex2(sA[3] - m_run[1]);
      l_run[0] += a0 + a2; l_run[1] += a1 + a3;
      pv(stage, a0, a1, a2, a3);
      __syncwarp();   // every lane is done with this stage
      if (issued < n_tiles) { issue(stage); ++issued; }
      advance(cc, p.kv_len, p.batch, p.n_kv_heads);
      it += 1;
      if (++stage == kStages) { stage = 0; parity ^= 1u; }
    }
  }
  flush();
}

constexpr size_t fp8_smem_bytes() {
  // per warp: 4 stages of (K tile + V tile), 4 table rows, 128 bytes of barriers and per-stage scalars; 1 KB alignment slack
  return static_cast<size_t>(kWarpsFp8) * (kFp8Stages * 2 * kTile * 128 + kFp8Stages * 128 * 4) + kWarpsFp8 * 128 + 1024;
}

template <int G>
int32_t launch_fp8(const DecodeParams& p, int n_ctas, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
  constexpr size_t smem = fp8_smem_bytes();
  cudaError_t e = cudaFuncSetAttribute(mepic_decode_splitkv_fp8<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) { mepic_set_error("decode_fp8: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_decode_splitkv_fp8<G><<<n_ctas, kWarpsFp8 * 32, smem, stream>>>(p, map_k, map_v);
  e = launch_dependent(mepic_decode_merge<128, G>, dim3(p.batch * p.n_kv_heads), dim3(G * 128), stream, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { mepic_set_error("decode_fp8: launch: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_count_launches(2);
  return MEPIC_OK;
}

int sm_count_of_current_device() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int32_t mepic_pages_quantize(const mepic_config_t* cfg, const void* src_pool, void* dst_pool, float* scales,
                                        const int32_t* pages, int32_t n_pages, int32_t* status, void* cuda_stream) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (!src_pool || !dst_pool || !scales || !pages || !status || n_pages < 0) { mepic_set_error("pages_quantize: bad argument"); return MEPIC_E_INVAL; }
  if (!aligned16(src_pool) || !aligned16(dst_pool)) { mepic_set_error("pages_quantize: pools must be 16-byte aligned"); return MEPIC_E_INVAL; }
  if (n_pages == 0) return MEPIC_OK;
  const int elems = cfg->page_size * cfg->head_dim;
  mepic_quantize_pages<<<n_pages * cfg->n_kv_heads, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint16_t*>(src_pool), static_cast<unsigned char*>(dst_pool), scales, pages, cfg->n_kv_heads, elems,
      cfg->num_pages, status);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { mepic_set_error("pages_quantize: launch: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_count_launches(1);
  return MEPIC_OK;
}

extern "C" int32_t mepic_attn_decode_fp8(const mepic_config_t* cfg, const mepic_decode_args_t* a, const float* k_scales,
                                         const float* v_scales, void* cuda_stream) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (!a || !a->q || !a->k_pool || !a->v_pool || !a->page_ids || !a->pos_base || !a->kv_len || !a->q_pos ||
      !a->rope_table || !a->out || !a->workspace || !a->status || !k_scales || !v_scales) {
    mepic_set_error("decode_fp8: NULL pointer argument"); return MEPIC_E_INVAL;
  }
  if (cfg->head_dim != 128) { mepic_set_error("decode_fp8: head_dim %d: 8-bit pages are built for head_dim 128", cfg->head_dim); return MEPIC_E_INVAL; }
  if (a->batch < 1 || a->table_stride < 1) { mepic_set_error("decode_fp8: batch and table_stride must be positive"); return MEPIC_E_INVAL; }
  if (!aligned16(a->q) || !aligned16(a->k_pool) || !aligned16(a->v_pool) || !aligned16(a->workspace) ||
      !aligned16(a->rope_table) || !aligned16(a->out)) { mepic_set_error("decode_fp8: pointers must be 16-byte aligned"); return MEPIC_E_INVAL; }
  if (cfg->max_position < kTile - 1) { mepic_set_error("decode_fp8: rope table must cover positions 0..15"); return MEPIC_E_INVAL; }
  const int sms = sm_count_of_current_device();
  if (sms <= 0) { mepic_set_error("decode_fp8: no CUDA device"); return MEPIC_E_CUDA; }
  const int G = cfg->n_q_heads / cfg->n_kv_heads, D = cfg->head_dim;
  const size_t slots = static_cast<size_t>(a->batch) * cfg->n_kv_heads + static_cast<size_t>(sms) * kMaxWarps;
  const size_t need = slots * G * (D + 2) * sizeof(float);      // the same as mepic_attn_decode_workspace
  if (a->workspace_bytes < need) { mepic_set_error("decode_fp8: workspace %zu < %zu bytes", a->workspace_bytes, need); return MEPIC_E_INVAL; }

  DecodeParams p;
  p.q = static_cast<const uint16_t*>(a->q);
  p.k_pool = static_cast<const uint16_t*>(a->k_pool);
  p.v_pool = static_cast<const uint16_t*>(a->v_pool);
  p.page_ids = a->page_ids; p.pos_base = a->pos_base; p.kv_len = a->kv_len; p.q_pos = a->q_pos;
  p.rope = a->rope_table;
  p.k_scales = k_scales; p.v_scales = v_scales;
  p.part_o = static_cast<float*>(a->workspace);
  p.part_ml = p.part_o + slots * G * D;
  p.out = static_cast<uint16_t*>(a->out);
  p.status = a->status;
  p.table_stride = a->table_stride; p.batch = a->batch; p.n_kv_heads = cfg->n_kv_heads;
  p.page_size = cfg->page_size;
  int l2 = 0; while ((kTile << l2) < cfg->page_size) ++l2;
  p.log2_tpp = l2;
  p.num_pages = cfg->num_pages; p.max_position = cfg->max_position;
  p.n_workers = sms * kWarpsFp8; p.n_workers_dram = p.n_workers;       // half the bytes per tile: never DRAM-bound
  p.scale_log2 = a->sm_scale * 1.4426950408889634f;
  p.spin_limit = mepic_test_spin_limit(kSpinLimit); p.skip_tile = mepic_test_skip_tile();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  alignas(64) CUtensorMap map_k, map_v;
  int32_t rc = mepic_make_pool_map_u8(cfg, a->k_pool, &map_k);
  if (rc != MEPIC_OK) return rc;
  rc = mepic_make_pool_map_u8(cfg, a->v_pool, &map_v);
  if (rc != MEPIC_OK) return rc;
  switch (G) {
    case 1: return launch_fp8<1>(p, sms, map_k, map_v, st);
    case 2: return launch_fp8<2>(p, sms, map_k, map_v, st);
    case 3: return launch_fp8<3>(p, sms, map_k, map_v, st);
    case 4: return launch_fp8<4>(p, sms, map_k, map_v, st);
    case 5: return launch_fp8<5>(p, sms, map_k, map_v, st);
    case 6: return launch_fp8<6>(p, sms, map_k, map_v, st);
    case 7: return launch_fp8<7>(p, sms, map_k, map_v, st);
    case 8: return launch_fp8<8>(p, sms, map_k, map_v, st);
  }
  mepic_set_error("decode_fp8: unsupported group size %d", G);
  return MEPIC_E_INVAL;
}
