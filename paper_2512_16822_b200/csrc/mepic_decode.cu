// Decode: RoPE-fused, split-KV, GQA, online-softmax attention over paged,
// un-rotated K (Section 3.3.3 of the paper: the rotation is applied when the
// kernel brings NoPE KV blocks on chip, right before the scores).
//
// Work decomposition.  The context of request b is cut into tiles of 16 tokens;
// the (request, kv head, tile) triples of the whole batch are laid on one line
// in that order and cut into equal contiguous pieces, one per WARP of a
// persistent grid (one CTA per SM, 8 or 12 warps).  A warp is a self-contained
// worker: it owns a ring of shared-memory stages that TMA tensor copies
// (cp.async.bulk.tensor + mbarrier complete_tx, 128-byte swizzle) fill with the
// K tile and V tile of its next tiles, together with the one row of the cos/sin
// table the tile's query rotation needs, and it keeps one online-softmax state
// per query head of the kv head it is on.  When its piece crosses into another
// (request, head) unit, or ends, it writes a partial (max, sum, weighted V) for
// the unit; a second kernel merges the partials of each unit.  Equal pieces
// balance ragged batches; no warp ever waits on another warp.
//
// Arithmetic.  <R(qpos) q, R(base+tau) k> = <R(qpos-base) q, R(tau) k>: per tile
// the G query vectors are rotated by (qpos - tile base) in fp32 and rounded to
// bf16, and every key only by its offset tau < 16 inside the tile, with cos/sin
// of those 16 offsets held in registers for the whole kernel.  Both contractions
// of a tile run on the tensor cores (mma.sync m16n8k16, fp32 accumulate) with the
// keys as the M rows; the K rotation is applied to the MMA's A fragments in
// registers (packed bf16), so rotated keys never touch shared or global memory.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "mepic.h"
#include "mepic_internal.h"

#include "mepic_decode_line.cuh"

namespace {

using namespace mepic_dev;

// ---------------------------------------------------------------- the split-KV kernel
// Warp-level tensor-core MMA (mma.sync m16n8k16, bf16 in, fp32 accumulate) for the two contractions of a tile:
//   S^T[key][head]  = K'[key][dim] . Q^T[dim][head]           A = rotated K (16 keys = the M rows), B = rotated q (heads = N <= 8)
//   O^T[dim][head] += V^T[dim][key] . P^T[key][head]          A = V^T by transposing ldmatrix, B = P^T (movmatrix of the S fragments)
// The keys and the head dims fill the 16 M rows completely and the G <= 8 query heads sit in the 8 N columns, so a tile
// costs 8 + 8 MMAs and 32 output accumulators per lane at D = 128 (with the heads as M rows, padded to 16, it was 16 + 16
// and 64).  Only the rotation of K (thread-local on the A fragments: the partner dim i + D/2 sits in the fragment of
// k-step j + D/32, same lane, same position) and the softmax stay on the CUDA cores.
#ifndef MEPIC_DECODE_STAGES
#define MEPIC_DECODE_STAGES 2
#endif
constexpr int kDecodeStages = MEPIC_DECODE_STAGES;     // depth of each warp's ring of staged tiles

// W = warps per CTA (12); how many of them take part (8 or 12) is decided on the device, see cut_of_line.
template <int D, int G, int W>
__global__ void __launch_bounds__(W * 32, 1)
mepic_decode_splitkv(const DecodeParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  constexpr int kStages = kDecodeStages;
  constexpr int NB = D / 64;                 // 64-dim blocks (128-byte swizzled rows) per K or V row
  constexpr int KS = D / 16;                 // k-steps of the QK^T contraction
  constexpr int KH = KS / 2;                 // k-steps per half: step j pairs with step j + KH
  constexpr int NV = D / 16;                 // 16-dim blocks of the output (M tiles of the PV product)
  constexpr int kBlockBytes = kTile * 128;   // one [16 rows x 64 dims] block
  constexpr int kStageBytes = 2 * NB * kBlockBytes;   // K blocks then V blocks
  constexpr int kWarpBytes = kStages * kStageBytes;

  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment: the swizzle pattern is a function of the address bits
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  unsigned char* stage0 = smem + static_cast<size_t>(wic) * kWarpBytes;
  // after the K/V rings: per warp, per stage, the cos/sin table row the tile's query rotation needs (D floats)
  float* rope_rows = reinterpret_cast<float*>(smem + static_cast<size_t>(W) * kWarpBytes) + static_cast<size_t>(wic) * kStages * D;
  unsigned char* misc = smem + static_cast<size_t>(W) * (kWarpBytes + kStages * D * 4) + wic * 64;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);                 // kStages x 8 bytes
  volatile float* meta = reinterpret_cast<volatile float*>(misc + 32);  // per stage: sign of (query position - tile base)

  const int g = lane >> 2;       // fragment row group: head g (A, C) / key g (B)
  const int t = lane & 3;        // fragment column group

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the merge kernel may move in as CTAs of this one retire
  const Cut cut = cut_of_line(p, lane);
  const int w_active = cut.workers / static_cast<int>(gridDim.x);     // warps of this CTA that take part (8 or all 12)
  if (wic >= w_active) return;
  const long long w = static_cast<long long>(blockIdx.x) * w_active + wic;
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

  // cos/sin of the in-tile offsets this lane's B fragments cover: keys g and g+8, pairs 16j + 2t + 8r + {0,1},
  // kept as packed bf16 pairs (cos, sin, -sin): the rotated K is rounded to bf16 for the MMA anyway, and packed
  // bf16 arithmetic rotates two elements per instruction without widening them first.
  uint32_t kc[2][KH][2], ksn[2][KH][2];      // [key g / g+8][k-step][fragment register]
#pragma unroll
  for (int kq = 0; kq < 2; ++kq)
#pragma unroll
    for (int j = 0; j < KH; ++j)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float4 cs = __ldg(reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(g + 8 * kq) * D + 2 * (16 * j + 2 * t + 8 * r)));
        kc[kq][j][r] = pack_bf16x2(cs.x, cs.z);
        ksn[kq][j][r] = pack_bf16x2(cs.y, cs.w);
      }

  Cursor pc = locate(p.kv_len, p.batch, p.n_kv_heads, x0, lane);   // producer cursor
  Cursor cc = pc;                                                  // consumer cursor
  int win_b = -1, win_e0 = 0, win_page = 0, win_pos = 0;           // 32 block-table entries, one per lane
  int win_qpos = 0;                                                // query position of the window's request

  int issued = 0;     // tiles handed to the ring so far = index of the tile issue() is called for
  auto issue = [&](int stage) {
    const int e = pc.t >> p.log2_tpp;
    const int sub = pc.t & ((1 << p.log2_tpp) - 1);
    if (pc.b != win_b || e < win_e0 || e >= win_e0 + 32) {
      if (pc.b != win_b) win_qpos = __ldg(p.q_pos + pc.b);
      win_b = pc.b; win_e0 = e;
      const int n_ent = (pc.kvl + p.page_size - 1) / p.page_size;
      const bool ok = e + lane < n_ent;
      const size_t at = static_cast<size_t>(pc.b) * p.table_stride + e + lane;
      win_page = ok ? __ldg(p.page_ids + at) : 0;
      win_pos = ok ? __ldg(p.pos_base + at) : 0;
    }
    int page = __shfl_sync(kFull, win_page, e - win_e0);
    const int pos = __shfl_sync(kFull, win_pos, e - win_e0);
    if (lane == 0 && !(w == 0 && issued == p.skip_tile)) {     // (test hook: one copy that never comes)
      if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { atomicOr(p.status, MEPIC_DEV_BAD_PAGE); page = 0; }
      const int y = (page * p.n_kv_heads + pc.h) * p.page_size + sub * kTile;     // row of the pool viewed as [rows][D]
      const uint32_t bar = smem_u32(&bars[stage]);
      const uint32_t dst = smem_u32(stage0 + static_cast<size_t>(stage) * kStageBytes);
      // the query is rotated by (its position - tile base): that table row travels with the tile
      const int rel = win_qpos - (pos + sub * kTile);
      int arel = rel < 0 ? -rel : rel;
      if (arel > p.max_position) { atomicOr(p.status, MEPIC_DEV_BAD_POSITION); arel = p.max_position; }
      meta[stage] = rel < 0 ? -1.f : 1.f;
      mbar_expect_tx(bar, kStageBytes + D * 4);
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        tma_load_2d(dst + nb * kBlockBytes, &map_k, nb * 64, y, bar);
        tma_load_2d(dst + (NB + nb) * kBlockBytes, &map_v, nb * 64, y, bar);
      }
      bulk_g2s(smem_u32(rope_rows + stage * D), p.rope + static_cast<size_t>(arel) * D, D * 4, bar);
    }
    advance(pc, p.kv_len, p.batch, p.n_kv_heads);
  };

  for (; issued < kStages && issued < n_tiles; ++issued) issue(issued);

  // per-unit state.  The keys are the M rows of both MMAs (S^T = K' Q^T and O^T = V^T P^T), the query heads the N
  // columns: this lane's B fragments of Q^T hold head g (lanes with g >= G carry zeros); its accumulators hold heads
  // 2t and 2t+1 (columns) for keys g, g+8 (scores) and for dims g, g+8 of every 16-dim block (output).
  int ub = -1, uh = -1;
  uint32_t q_lo[KH][2], q_hi[KH][2];        // un-rotated q of head g as packed bf16 pairs, pre-scaled by sm_scale*log2e: pairs as for kc/ksn
  float m_run[2] = {-INFINITY, -INFINITY};  // running maximum of heads 2t, 2t+1 (the same in the 8 lanes that share t)
  float l_run[2] = {0.f, 0.f};              // this lane's share (keys g, g+8 of every tile) of the two heads' sums
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

  int stage = 0;
  uint32_t parity = 0;
  for (int it = 0; it < n_tiles; ++it) {
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
          const int pair = 16 * j + 2 * t + 8 * r;              // dims pair, pair+1 and their partners + D/2
          const float2 lo = bf16x2_to_float2(__ldg(src + pair / 2));
          const float2 hi = bf16x2_to_float2(__ldg(src + (pair + D / 2) / 2));
          const float sc = g < G ? p.scale_log2 : 0.f;
          q_lo[j][r] = pack_bf16x2(lo.x * sc, lo.y * sc);
          q_hi[j][r] = pack_bf16x2(hi.x * sc, hi.y * sc);
        }
      m_run[0] = m_run[1] = -INFINITY; l_run[0] = l_run[1] = 0.f;
#pragma unroll
      for (int db = 0; db < NV; ++db) { acc[db][0] = 0.f; acc[db][1] = 0.f; acc[db][2] = 0.f; acc[db][3] = 0.f; }
    }

    if (!mbar_wait_bounded(smem_u32(&bars[stage]), parity, p.spin_limit)) {
      // Give the copies still in flight a last bounded chance to land, then leave cleanly.
      if (lane == 0) atomicOr(p.status, MEPIC_DEV_WAIT_EXPIRED);
      for (int s = 0; s < kStages; ++s) mbar_wait_bounded(smem_u32(&bars[s]), s == stage ? parity : (s < stage ? parity ^ 1u : parity), p.spin_limit);
      return;
    }
    const uint32_t ks_addr = smem_u32(stage0 + static_cast<size_t>(stage) * kStageBytes);
    const uint32_t vs_addr = ks_addr + NB * kBlockBytes;
    const uint32_t sgn_bits = meta[stage] < 0.f ? 0x80008000u : 0u;      // a negative angle flips the sines
    const int n_valid = min(kTile, cc.kvl - cc.t * kTile);
    // ---- B fragments of Q^T: head g rotated by (qpos - tile base), from the table row that came with the tile
    uint32_t qa[KS][2];                         // [k-step][b0 (dims 16j+2t,+1) | b1 (dims 16j+8+2t,+1)], column = head g
    {
      const float* row = rope_rows + stage * D;
#pragma unroll
      for (int j = 0; j < KH; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          // packed bf16 arithmetic, as for the keys: the rotated query is rounded to bf16 for the MMA anyway
          const float4 cs = *reinterpret_cast<const float4*>(row + 2 * (16 * j + 2 * t + 8 * r));
          const uint32_t c2 = pack_bf16x2(cs.x, cs.z), s2 = pack_bf16x2(cs.y, cs.w) ^ sgn_bits;
          qa[j][r] = bf16x2_fma(q_lo[j][r], c2, bf16x2_neg(bf16x2_mul(q_hi[j][r], s2)));      // lo cos - hi sin
          qa[j + KH][r] = bf16x2_fma(q_lo[j][r], s2, bf16x2_mul(q_hi[j][r], c2));            // lo sin + hi cos
        }
    }
    // rows at or past kv_len may hold anything (NaN bit patterns included): their P is 0, but 0 x NaN is NaN,
    // so V must be finite there.  Only a request's last tile has such rows.
    if (n_valid < kTile) {
      for (int idx = n_valid * 8 * NB + lane; idx < kTile * 8 * NB; idx += 32) {
        const int key = idx / (8 * NB), ch = idx % (8 * NB);
        const uint32_t a = vs_addr + (ch / 8) * kBlockBytes + key * 128 + (((ch % 8) ^ (key & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
      }
      // these generic-proxy stores must be ordered before the TMA (async proxy) write that refills this stage
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
    }

    // ---- S^T = K' Q^T : A fragments of K by ldmatrix (keys g, g+8 x 16 dims), rotated in registers; two
    // accumulators so that the MMAs of the lower and the upper half of the head dimension do not wait on each other
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < KH; ++j) {
      uint32_t lo[4], hi[4];      // lo: k-step j, hi: k-step j + KH; [a0 key g, a1 key g+8 | a2 key g, a3 key g+8 (dims + 8)]
      {
        // lane -> (matrix mi = lane / 8, row = lane % 8): key = 8 (mi & 1) + row, 16-byte chunk 2 j + (mi >> 1)
        const int mi = lane >> 3, key = ((mi & 1) << 3) + (lane & 7);
        const int cl = 2 * j + (mi >> 1), chh = 2 * (j + KH) + (mi >> 1);
        ldmatrix_x4(lo, ks_addr + (cl / 8) * kBlockBytes + key * 128 + (((cl % 8) ^ (key & 7)) << 4));
        ldmatrix_x4(hi, ks_addr + (chh / 8) * kBlockBytes + key * 128 + (((chh % 8) ^ (key & 7)) << 4));
      }
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const int kq = f & 1, r = f >> 1;       // key g + 8 kq, column half r
        const uint32_t a = lo[f], b = hi[f];
        lo[f] = bf16x2_fma(a, kc[kq][j][r], bf16x2_neg(bf16x2_mul(b, ksn[kq][j][r])));     // lo cos - hi sin
        hi[f] = bf16x2_fma(a, ksn[kq][j][r], bf16x2_mul(b, kc[kq][j][r]));     // lo sin + hi cos
      }
      mma_bf16(sa, lo[0], lo[1], lo[2], lo[3], qa[j][0], qa[j][1]);
      mma_bf16(sb, hi[0], hi[1], hi[2], hi[3], qa[j + KH][0], qa[j + KH][1]);
    }

    // ---- online softmax (log2 domain): this lane holds keys g (c0, c1) and g+8 (c2, c3) of heads 2t (c0, c2), 2t+1 (c1, c3)
    float sc[4] = {sa[0] + sb[0], sa[1] + sb[1], sa[2] + sb[2], sa[3] + sb[3]};
    if (n_valid < kTile) {
      if (g >= n_valid) { sc[0] = -INFINITY; sc[1] = -INFINITY; }
      if (g + 8 >= n_valid) { sc[2] = -INFINITY; sc[3] = -INFINITY; }
    }
    float mx0 = fmaxf(sc[0], sc[2]), mx1 = fmaxf(sc[1], sc[3]);
    // the running maximum moves only if some lane saw a larger score: only then is the tile's maximum worked out
    if (__any_sync(kFull, mx0 > m_run[0] || mx1 > m_run[1])) {
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) { mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, o)); mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, o)); }
      const float n0 = fmaxf(m_run[0], mx0), n1 = fmaxf(m_run[1], mx1);
      const float a0 = ex2(m_run[0] - n0), a1 = ex2(m_run[1] - n1);     // 0 on the first tile (m_run = -inf)
      m_run[0] = n0; m_run[1] = n1;
      l_run[0] *= a0; l_run[1] *= a1;
#pragma unroll
      for (int db = 0; db < NV; ++db) { acc[db][0] *= a0; acc[db][1] *= a1; acc[db][2] *= a0; acc[db][3] *= a1; }
    }
    const float p0 = ex2(sc[0] - m_run[0]), p1 = ex2(sc[1] - m_run[1]), p2 = ex2(sc[2] - m_run[0]), p3 = ex2(sc[3] - m_run[1]);
    l_run[0] += p0 + p2; l_run[1] += p1 + p3;
    // B fragments of P^T (keys x heads) = the transposes of the two 8 x 8 blocks this warp holds as (key row, head columns)
    const uint32_t pb0 = movmatrix_trans(pack_bf16x2(p0, p1)), pb1 = movmatrix_trans(pack_bf16x2(p2, p3));

    // ---- O^T += V^T P^T : A fragments of V^T by transposing ldmatrix, one 16-dim block per MMA
#pragma unroll
    for (int db = 0; db < NV; ++db) {
      uint32_t va[4];             // a0 dims g x keys 0-7, a1 dims g+8 x keys 0-7, a2 dims g x keys 8-15, a3 dims g+8 x keys 8-15
      {
        // lane -> (matrix mi, row): key = 8 (mi >> 1) + row, 16-byte chunk 2 db + (mi & 1)
        const int mi = lane >> 3, key = ((mi >> 1) << 3) + (lane & 7);
        const int ch = 2 * db + (mi & 1);
        ldmatrix_x4_trans(va, vs_addr + (ch / 8) * kBlockBytes + key * 128 + (((ch % 8) ^ (key & 7)) << 4));
      }
      mma_bf16(acc[db], va[0], va[1], va[2], va[3], pb0, pb1);
    }
    __syncwarp();   // every lane is done with this stage

    if (issued < n_tiles) { issue(stage); ++issued; }
    advance(cc, p.kv_len, p.batch, p.n_kv_heads);
    if (++stage == kStages) { stage = 0; parity ^= 1u; }
  }
  flush();
}

template <int D, int G, int W>
constexpr size_t decode_smem_bytes() {
  // per warp: the stages of (K blocks + V blocks) and their table rows, 64 bytes of barriers and flags; 1 KB alignment slack
  return static_cast<size_t>(W) * (kDecodeStages * 2 * (D / 64) * kTile * 128 + kDecodeStages * D * 4) + W * 64 + 1024;
}

template <int D, int G, int W>
int32_t launch_decode_w(const DecodeParams& p, int n_ctas, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
  constexpr size_t smem = decode_smem_bytes<D, G, W>();
  cudaError_t e = cudaFuncSetAttribute(mepic_decode_splitkv<D, G, W>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) { mepic_set_error("decode: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_decode_splitkv<D, G, W><<<n_ctas, W * 32, smem, stream>>>(p, map_k, map_v);
  e = launch_dependent(mepic_decode_merge<D, G>, dim3(p.batch * p.n_kv_heads), dim3(G * D), stream, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { mepic_set_error("decode: launch: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_count_launches(2);
  return MEPIC_OK;
}

template <int D, int G>
int32_t launch_decode(const DecodeParams& p, int n_ctas, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
  return launch_decode_w<D, G, kWarpsShared>(p, n_ctas, map_k, map_v, stream);
}

int sm_count_of_current_device() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

size_t decode_slots(const mepic_config_t* cfg, int batch, int sms) {
  return static_cast<size_t>(batch) * cfg->n_kv_heads + static_cast<size_t>(sms) * kMaxWarps;
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
  p.k_scales = nullptr; p.v_scales = nullptr;
  p.part_o = static_cast<float*>(a->workspace);
  p.part_ml = p.part_o + slots * G * D;
  p.out = static_cast<uint16_t*>(a->out);
  p.status = a->status;
  p.table_stride = a->table_stride; p.batch = a->batch; p.n_kv_heads = cfg->n_kv_heads;
  p.page_size = cfg->page_size;
  int l2 = 0; while ((kTile << l2) < cfg->page_size) ++l2;
  p.log2_tpp = l2;
  p.num_pages = cfg->num_pages; p.max_position = cfg->max_position;
  p.n_workers = sms * kWarpsShared; p.n_workers_dram = sms * kWarps;
  p.scale_log2 = a->sm_scale * 1.4426950408889634f;
  p.spin_limit = mepic_test_spin_limit(kSpinLimit); p.skip_tile = mepic_test_skip_tile();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  alignas(64) CUtensorMap map_k, map_v;
  int32_t rc = mepic_make_pool_map(cfg, a->k_pool, &map_k);
  if (rc != MEPIC_OK) return rc;
  rc = mepic_make_pool_map(cfg, a->v_pool, &map_v);
  if (rc != MEPIC_OK) return rc;

#define MEPIC_DECODE_CASE(DD, GG) if (D == DD && G == GG) return launch_decode<DD, GG>(p, sms, map_k, map_v, st);
  MEPIC_DECODE_CASE(128, 1) MEPIC_DECODE_CASE(128, 2) MEPIC_DECODE_CASE(128, 3) MEPIC_DECODE_CASE(128, 4) MEPIC_DECODE_CASE(128, 5) MEPIC_DECODE_CASE(128, 6) MEPIC_DECODE_CASE(128, 7) MEPIC_DECODE_CASE(128, 8)
  MEPIC_DECODE_CASE(64, 1) MEPIC_DECODE_CASE(64, 2) MEPIC_DECODE_CASE(64, 3) MEPIC_DECODE_CASE(64, 4) MEPIC_DECODE_CASE(64, 5) MEPIC_DECODE_CASE(64, 6) MEPIC_DECODE_CASE(64, 7) MEPIC_DECODE_CASE(64, 8)
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
