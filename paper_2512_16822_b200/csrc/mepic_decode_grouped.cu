// Grouped decode: the RoPE-fused split-KV decode in which the requests that alias the same
// shared chunk pages (Section 3.2.2) are scored against a staged page together.
//
// The host plan (mepic_plan.cpp) regroups the block tables into items: a group of up to R
// requests and the pages all of them alias.  The 16 rows of a tensor-core tile hold the G query
// heads of up to R = 16 / G requests, so a K/V tile is brought on chip once and its keys rotated
// once per GROUP instead of once per request; with per-request decode the same rows carry one
// request's G heads and padding.  The line of (item, kv head, tile) triples is cut into equal
// pieces, one per warp of a persistent grid, exactly as in the per-request kernel.
//
// Rotation.  <R(qpos) q, R(base + tau) k> = <R(qpos - base) q, R(tau) k>, and base differs between
// the requests of a group, so the per-request part of the angle goes to the query: row (j, h)
// carries q rotated by (qpos_j - tile base_j) in fp32 registers.  From one tile to the next of a
// chunk that angle drops by exactly 16 positions, so the row is advanced by one fixed rotation
// (cos/sin of 16 positions, one table row kept in shared memory); only where the angle jumps
// (first tile of a unit, chunk boundary, non-contiguous private pages) is the row rebuilt from
// the un-rotated q and the cos/sin table.  Keys are rotated by their in-tile offset on the MMA's
// B fragments with packed bf16 constants held in registers, as in the per-request kernel.
#include <cuda.h>
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "mepic.h"
#include "mepic_internal.h"
#include "mepic_plan.h"
#include "mepic_ptx.cuh"

namespace {

using namespace mepic_dev;

constexpr int kTile = kPlanTile;
constexpr int kWarps = kPlanWarps;

struct GroupedParams {
  const uint16_t* q;
  const int32_t* kv_len;
  const int32_t* q_pos;
  const float* rope;
  const int32_t* plan;
  const float* k_scales;   // 8-bit pools only: [num_pages][n_kv_heads] scale of each (page, kv head) block of K
  const float* v_scales;   // ... and of V
  float* part_o;    // [slots][G][D]
  float* part_ml;   // [slots][G][2] = (max in log2 units, sum)
  uint16_t* out;
  int32_t* status;
  int n_kv_heads, page_size, log2_tpp, num_pages, max_position, batch;
  int n_items, piece, total;
  int off_items, off_records, off_workers, off_req_ent, off_slot_base, off_part_off;
  int spin_limit;   // polls before a bounded wait gives up
  int skip_tile;    // test hook: worker 0 leaves out the staged copy of its tile with this index (-1: none)
  float scale_log2;   // sm_scale * log2(e)
};

// FP8: the pools hold e4m3 codes with one scale per (page, kv head) block (head_dim 128 only).  A staged tile is then
// 16 rows x 128 bytes per pool; codes are widened exactly to fp16, both contractions run as fp16 MMAs, the K scale
// goes on the fp32 scores and the V scale on P.  16-bit ldmatrix on 8-bit rows hands a lane four consecutive dims of a
// key and the transposing 8-bit ldmatrix four consecutive keys of a dim, so the dim pairs of a lane are 16j + 4t + 2r
// (bf16: 16j + 2t + 8r) and the key columns of the two score n-tiles are {0,1,4,5,..} / {2,3,6,7,..}: a lane's four
// scores are keys 4t..4t+3, the keys its V fragments carry.
template <int D, int G, bool FP8>
__global__ void __launch_bounds__(kWarps * 32, 1)
mepic_decode_grouped(const GroupedParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  constexpr int R = plan_group_requests(G);
  constexpr int kItemInts = kItemFixed + R;
  constexpr int kStages = 3;
  constexpr int NB = D / 64;                 // 64-dim blocks (128-byte swizzled rows) per K or V row
  constexpr int KS = D / 16;                 // k-steps of the QK^T contraction
  constexpr int KH = KS / 2;                 // k-steps per half: step j pairs with step j + KH
  constexpr int ND = D / 8;                  // n-tiles of the PV product
  constexpr int kBlockBytes = kTile * 128;   // one [16 rows x 128 bytes] block: 64 bf16 dims, or all 128 dims of 8-bit pages
  constexpr int KB = FP8 ? 1 : NB;           // such blocks per K or V tile
  constexpr int kStageBytes = 2 * KB * kBlockBytes;   // K blocks then V blocks
  constexpr int kWarpBytes = kStages * kStageBytes;

  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment: the swizzle pattern is a function of the address bits
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;
  unsigned char* stage0 = smem + static_cast<size_t>(wic) * kWarpBytes;
  // after the rings: the table row of 16 positions (cos, sin interleaved, D floats), then per warp its barriers
  // and, per stage, the tile base position of each request of the group
  float* step16 = reinterpret_cast<float*>(smem + static_cast<size_t>(kWarps) * kWarpBytes);
  unsigned char* misc = smem + static_cast<size_t>(kWarps) * kWarpBytes + D * 4 + wic * 128;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);                       // kStages x 8 bytes
  volatile int32_t* meta = reinterpret_cast<volatile int32_t*>(misc + 32);  // [kStages][8] (64-byte misc + 32 .. + 128)
  volatile float* scl = reinterpret_cast<volatile float*>(smem + static_cast<size_t>(kWarps) * (kWarpBytes + 128) + D * 4 + wic * 32);   // 8-bit pools: [kStages][2] K / V scale of the staged tile

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the merge kernel may move in as CTAs of this one retire
  for (int i = threadIdx.x; i < D; i += kWarps * 32) step16[i] = __ldg(p.rope + static_cast<size_t>(kTile) * D + i);
  __syncthreads();

  const int g = lane >> 2;       // fragment row group: rows g and g + 8 (A, C) / key column g of a score n-tile (B)
  const int t = lane & 3;        // fragment column group
  // first dim of the pair this lane's fragment register r of k-step j covers; the keys behind column g of the two n-tiles
  auto pair_of = [&](int j, int r) { return FP8 ? 16 * j + 4 * t + 2 * r : 16 * j + 2 * t + 8 * r; };
  const int keyA = FP8 ? 4 * (g >> 1) + (g & 1) : g, keyB = FP8 ? keyA + 2 : g + 8;
  // the two rows this lane owns: row = j * G + h = (request of the group, query head of the kv head)
  const int jA = g / G, hA = g % G, jB = (g + 8) / G, hB = (g + 8) % G;

  const long long w = static_cast<long long>(blockIdx.x) * kWarps + wic;
  const long long x0 = w * p.piece;
  if (x0 >= p.total) return;
  const long long x1 = (x0 + p.piece < p.total) ? x0 + p.piece : p.total;
  const int n_tiles = static_cast<int>(x1 - x0);

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // cos/sin of the in-tile offsets this lane's B fragments cover: keys g and g+8, pairs 16j + 2t + 8r + {0,1},
  // as packed bf16 pairs (cos, sin, -sin)
  uint32_t kc[2][KH][2], ksn[2][KH][2], kns[2][KH][2];      // [key g / g+8][k-step][fragment register]
#pragma unroll
  for (int kq = 0; kq < 2; ++kq)
#pragma unroll
    for (int j = 0; j < KH; ++j)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float4 cs = __ldg(reinterpret_cast<const float4*>(p.rope + static_cast<size_t>(kq ? keyB : keyA) * D + 2 * pair_of(j, r)));
        kc[kq][j][r] = FP8 ? pack_f16x2(cs.x, cs.z) : pack_bf16x2(cs.x, cs.z);
        ksn[kq][j][r] = FP8 ? pack_f16x2(cs.y, cs.w) : pack_bf16x2(cs.y, cs.w);
        kns[kq][j][r] = FP8 ? pack_f16x2(-cs.y, -cs.w) : pack_bf16x2(-cs.y, -cs.w);
      }

  const int32_t* items = p.plan + p.off_items;
  const int32_t* ws = p.plan + p.off_workers + w * 3;
  // producer cursor: item, kv head, tile; the item's tile count per head and first record
  int pi = __ldg(ws), ph = __ldg(ws + 1), pt = __ldg(ws + 2);
  int p_nt = 0, p_rec = 0;
  auto producer_item = [&]() {
    if (pi < p.n_items) {
      p_nt = __ldg(items + static_cast<size_t>(pi) * kItemInts + kPiEnt) << p.log2_tpp;
      p_rec = __ldg(items + static_cast<size_t>(pi) * kItemInts + kPiRecOff);
    }
  };
  producer_item();
  // consumer cursor
  int ci = pi, ch = ph, ct = pt, c_nt = p_nt;

  int win_item = -1, win_e0 = 0, win_page = 0, win_pos[R];   // 32 records of the producer's item, one per lane

  int issued = 0;     // tiles handed to the ring so far = index of the tile issue() is called for
  auto issue = [&](int stage) {
    const int e = pt >> p.log2_tpp;
    const int sub = pt & ((1 << p.log2_tpp) - 1);
    if (pi != win_item || e < win_e0 || e >= win_e0 + 32) {
      win_item = pi; win_e0 = e;
      const bool ok = e + lane < (p_nt >> p.log2_tpp);
      const int32_t* rec = p.plan + p.off_records + static_cast<size_t>(p_rec + e + lane) * (1 + R);
      win_page = ok ? __ldg(rec) : 0;
#pragma unroll
      for (int j = 0; j < R; ++j) win_pos[j] = ok ? __ldg(rec + 1 + j) : 0;
    }
    int page = __shfl_sync(kFull, win_page, e - win_e0);
    int pos[R];
#pragma unroll
    for (int j = 0; j < R; ++j) pos[j] = __shfl_sync(kFull, win_pos[j], e - win_e0);
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < R; ++j) meta[stage * 8 + j] = pos[j] + sub * kTile;
    }
    if (lane == 0 && !(w == 0 && issued == p.skip_tile)) {     // (test hook: one copy that never comes)
      if (static_cast<unsigned>(page) >= static_cast<unsigned>(p.num_pages)) { atomicOr(p.status, MEPIC_DEV_BAD_PAGE); page = 0; }
      const int y = (page * p.n_kv_heads + ph) * p.page_size + sub * kTile;     // row of the pool viewed as [rows][D]
      const uint32_t bar = smem_u32(&bars[stage]);
      const uint32_t dst = smem_u32(stage0 + static_cast<size_t>(stage) * kStageBytes);
      mbar_expect_tx(bar, kStageBytes);
      if constexpr (FP8) {
        scl[stage * 2] = __ldg(p.k_scales + static_cast<size_t>(page) * p.n_kv_heads + ph);      // (an out-of-range page was replaced by 0 above)
        scl[stage * 2 + 1] = __ldg(p.v_scales + static_cast<size_t>(page) * p.n_kv_heads + ph);
        tma_load_2d(dst, &map_k, 0, y, bar);
        tma_load_2d(dst + kBlockBytes, &map_v, 0, y, bar);
      } else {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          tma_load_2d(dst + nb * kBlockBytes, &map_k, nb * 64, y, bar);
          tma_load_2d(dst + (NB + nb) * kBlockBytes, &map_v, nb * 64, y, bar);
        }
      }
    }
    if (++pt == p_nt) {
      pt = 0;
      if (++ph == p.n_kv_heads) { ph = 0; ++pi; producer_item(); }
    }
  };

  for (; issued < kStages && issued < n_tiles; ++issued) issue(issued);
  __syncwarp();

  // per-unit state of the lane's two rows
  int ui = -1, uh = -1, u_tail = -1, u_kvl = 0, u_ts = 0;
  int reqA = -1, reqB = -1, qposA = 0, qposB = 0, angA = INT_MIN, angB = INT_MIN;
  float qlA[KH][2][2], qhA[KH][2][2], qlB[KH][2][2], qhB[KH][2][2];   // rotated, pre-scaled q: halves lo / hi
  float mA = -INFINITY, lA = 0.f, mB = -INFINITY, lB = 0.f;
  float acc[ND][4];                         // O fragments: [n-tile][c0,c1 = row g | c2,c3 = row g + 8]

  auto flush = [&]() {
    if (ui < 0) return;
    float la = lA, lb = lB;
    la += __shfl_xor_sync(kFull, la, 1); la += __shfl_xor_sync(kFull, la, 2);
    lb += __shfl_xor_sync(kFull, lb, 1); lb += __shfl_xor_sync(kFull, lb, 2);
    // this worker is the k-th whose piece overlaps the unit
    const long long k = w - (static_cast<long long>(u_ts) * p.n_kv_heads + static_cast<long long>(uh) * c_nt) / p.piece;
    const int32_t* sb = p.plan + p.off_slot_base + (static_cast<size_t>(ui) * p.n_kv_heads + uh) * R;
    if (reqA >= 0) {
      const long long slot = __ldg(sb + jA) + k;
      float* dst = p.part_o + (slot * G + hA) * D;
#pragma unroll
      for (int nd = 0; nd < ND; ++nd) *reinterpret_cast<float2*>(dst + 8 * nd + 2 * t) = make_float2(acc[nd][0], acc[nd][1]);
      if (t == 0) *reinterpret_cast<float2*>(p.part_ml + (slot * G + hA) * 2) = make_float2(mA, la);
    }
    if (reqB >= 0) {
      const long long slot = __ldg(sb + jB) + k;
      float* dst = p.part_o + (slot * G + hB) * D;
#pragma unroll
      for (int nd = 0; nd < ND; ++nd) *reinterpret_cast<float2*>(dst + 8 * nd + 2 * t) = make_float2(acc[nd][2], acc[nd][3]);
      if (t == 0) *reinterpret_cast<float2*>(p.part_ml + (slot * G + hB) * 2) = make_float2(mB, lb);
    }
  };

  // Row (request req, query head h of kv head uh) rotated by `need` positions: rebuilt from the un-rotated q and the
  // table where the angle jumped, advanced by the fixed 16-position rotation otherwise.
  auto rotate_row = [&](float (&ql)[KH][2][2], float (&qh)[KH][2][2], int& ang, int need, int req, int h) {
    if (need == ang - kTile) {
#pragma unroll
      for (int j = 0; j < KH; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const float4 cs = *reinterpret_cast<const float4*>(step16 + 2 * pair_of(j, r));
          const float l0 = ql[j][r][0], h0 = qh[j][r][0], l1 = ql[j][r][1], h1 = qh[j][r][1];
          ql[j][r][0] = l0 * cs.x + h0 * cs.y; qh[j][r][0] = h0 * cs.x - l0 * cs.y;      // rotation by -16 positions
          ql[j][r][1] = l1 * cs.z + h1 * cs.w; qh[j][r][1] = h1 * cs.z - l1 * cs.w;
        }
    } else {
      int arel = need < 0 ? -need : need;
      if (arel > p.max_position) { atomicOr(p.status, MEPIC_DEV_BAD_POSITION); arel = p.max_position; }
      const float sgn = need < 0 ? -1.f : 1.f;
      const float* row = p.rope + static_cast<size_t>(arel) * D;
      const uint32_t* src = reinterpret_cast<const uint32_t*>(
          p.q + (static_cast<size_t>(req) * (p.n_kv_heads * G) + static_cast<size_t>(uh) * G + h) * D);
#pragma unroll
      for (int j = 0; j < KH; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int pair = pair_of(j, r);                        // dims pair, pair+1 and their partners + D/2
          const float2 lo = bf16x2_to_float2(__ldg(src + pair / 2));
          const float2 hi = bf16x2_to_float2(__ldg(src + (pair + D / 2) / 2));
          const float4 cs = __ldg(reinterpret_cast<const float4*>(row + 2 * pair));
          const float c0 = cs.x * p.scale_log2, s0 = cs.y * sgn * p.scale_log2, c1 = cs.z * p.scale_log2, s1 = cs.w * sgn * p.scale_log2;
          ql[j][r][0] = lo.x * c0 - hi.x * s0; qh[j][r][0] = lo.x * s0 + hi.x * c0;
          ql[j][r][1] = lo.y * c1 - hi.y * s1; qh[j][r][1] = lo.y * s1 + hi.y * c1;
        }
    }
    ang = need;
  };

  int stage = 0;
  uint32_t parity = 0;
  for (int it = 0; it < n_tiles; ++it) {
    if (ci != ui || ch != uh) {
      flush();
      if (ci != ui) {
        const int32_t* hd = items + static_cast<size_t>(ci) * kItemInts;
        const int n_req = __ldg(hd + kPiReq);
        c_nt = __ldg(hd + kPiEnt) << p.log2_tpp;
        u_tail = __ldg(hd + kPiTail);
        u_ts = __ldg(hd + kPiTileStart);
        reqA = jA < n_req ? __ldg(hd + kPiReqIds + jA) : -1;
        reqB = (jB < R && jB < n_req) ? __ldg(hd + kPiReqIds + jB) : -1;
        if (static_cast<unsigned>(reqA) >= static_cast<unsigned>(p.batch)) reqA = -1;
        if (static_cast<unsigned>(reqB) >= static_cast<unsigned>(p.batch)) reqB = -1;
        qposA = reqA >= 0 ? __ldg(p.q_pos + reqA) : 0;
        qposB = reqB >= 0 ? __ldg(p.q_pos + reqB) : 0;
        const int r0 = __ldg(hd + kPiReqIds);
        u_kvl = (u_tail >= 0 && static_cast<unsigned>(r0) < static_cast<unsigned>(p.batch)) ? __ldg(p.kv_len + r0) : 0;
      }
      ui = ci; uh = ch;
      angA = INT_MIN; angB = INT_MIN;
#pragma unroll
      for (int j = 0; j < KH; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          qlA[j][r][0] = 0.f; qlA[j][r][1] = 0.f; qhA[j][r][0] = 0.f; qhA[j][r][1] = 0.f;
          qlB[j][r][0] = 0.f; qlB[j][r][1] = 0.f; qhB[j][r][0] = 0.f; qhB[j][r][1] = 0.f;
        }
      mA = -INFINITY; lA = 0.f; mB = -INFINITY; lB = 0.f;
#pragma unroll
      for (int nd = 0; nd < ND; ++nd) { acc[nd][0] = 0.f; acc[nd][1] = 0.f; acc[nd][2] = 0.f; acc[nd][3] = 0.f; }
    }

    const uint32_t ks_addr = smem_u32(stage0 + static_cast<size_t>(stage) * kStageBytes);
    const uint32_t vs_addr = ks_addr + KB * kBlockBytes;
    // only the partly filled last page of a request (always in its single-request item) has invalid slots
    int n_valid = kTile;
    if (u_tail >= 0 && (ct >> p.log2_tpp) == (c_nt >> p.log2_tpp) - 1)
      n_valid = min(kTile, u_kvl - u_tail - (ct & ((1 << p.log2_tpp) - 1)) * kTile);

    // the query rows need only the tile's base positions (written when the stage was issued), not its data
    if (n_valid > 0) {
      if (reqA >= 0) rotate_row(qlA, qhA, angA, qposA - meta[stage * 8 + jA], reqA, hA);
      if (reqB >= 0) rotate_row(qlB, qhB, angB, qposB - meta[stage * 8 + (jB < R ? jB : 0)], reqB, hB);
    }
    if (!mbar_wait_bounded(smem_u32(&bars[stage]), parity, p.spin_limit)) {
      // Give the copies still in flight a last bounded chance to land, then leave cleanly.
      if (lane == 0) atomicOr(p.status, MEPIC_DEV_WAIT_EXPIRED);
      for (int s = 0; s < kStages; ++s) mbar_wait_bounded(smem_u32(&bars[s]), s == stage ? parity : (s < stage ? parity ^ 1u : parity), p.spin_limit);
      return;
    }
    if (n_valid > 0) {

      // slots at or past kv_len may hold anything (NaN bit patterns included): their P is 0, but 0 x NaN is NaN,
      // so V must be finite there.
      if (n_valid < kTile) {
        for (int idx = n_valid * 8 * KB + lane; idx < kTile * 8 * KB; idx += 32) {
          const int key = idx / (8 * KB), chk = idx % (8 * KB);
          const uint32_t a = vs_addr + (chk / 8) * kBlockBytes + key * 128 + (((chk % 8) ^ (key & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
        }
        // these generic-proxy stores must be ordered before the TMA (async proxy) write that refills this stage
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
      }

      // ---- S^T = Q K'^T : B fragments by ldmatrix, rotated in registers, two key n-tiles
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < KH; ++j) {
        uint32_t lo[4], hi[4];      // lo: k-step j, hi: k-step j + KH; [b0 nt0, b1 nt0, b0 nt1, b1 nt1]
        if constexpr (FP8) {
          uint32_t raw[4];          // [n-tile 0 lower, n-tile 1 lower, n-tile 0 upper, n-tile 1 upper], 4 dims each
          {
            // lane -> (matrix mi = lane / 8, row = lane % 8): key of that row in n-tile (mi & 1), 16-byte chunk j (+ KH)
            const int mi = lane >> 3, rr = lane & 7;
            const int key = 4 * (rr >> 1) + (rr & 1) + 2 * (mi & 1);
            const int chk = j + KH * (mi >> 1);
            ldmatrix_x4(raw, ks_addr + key * 128 + ((chk ^ (key & 7)) << 4));
          }
          e4m3x4_to_f16x2x2(raw[0], lo[0], lo[1]);
          e4m3x4_to_f16x2x2(raw[1], lo[2], lo[3]);
          e4m3x4_to_f16x2x2(raw[2], hi[0], hi[1]);
          e4m3x4_to_f16x2x2(raw[3], hi[2], hi[3]);
        } else {
          // lane -> (matrix mi = lane / 8, row = lane % 8): key = 8 (mi / 2) + row, 16-byte chunk 2 j + (mi & 1)
          const int mi = lane >> 3, key = ((mi >> 1) << 3) + (lane & 7);
          const int cl = 2 * j + (mi & 1), chh = 2 * (j + KH) + (mi & 1);
          ldmatrix_x4(lo, ks_addr + (cl / 8) * kBlockBytes + key * 128 + (((cl % 8) ^ (key & 7)) << 4));
          ldmatrix_x4(hi, ks_addr + (chh / 8) * kBlockBytes + key * 128 + (((chh % 8) ^ (key & 7)) << 4));
        }
#pragma unroll
        for (int f = 0; f < 4; ++f) {
          const int kq = f >> 1, r = f & 1;       // key column of n-tile kq, fragment register r
          const uint32_t a = lo[f], b = hi[f];
          if constexpr (FP8) {
            lo[f] = f16x2_fma(a, kc[kq][j][r], f16x2_mul(b, kns[kq][j][r]));     // lo cos - hi sin
            hi[f] = f16x2_fma(a, ksn[kq][j][r], f16x2_mul(b, kc[kq][j][r]));     // lo sin + hi cos
          } else {
            lo[f] = bf16x2_fma(a, kc[kq][j][r], bf16x2_mul(b, kns[kq][j][r]));
            hi[f] = bf16x2_fma(a, ksn[kq][j][r], bf16x2_mul(b, kc[kq][j][r]));
          }
        }
        // A fragments: a0 / a2 = row g, the pairs of fragment registers 0 / 1 of this k-step; a1 / a3 = row g + 8
        auto pk = [](float x, float y) { return FP8 ? pack_f16x2(x, y) : pack_bf16x2(x, y); };
        const uint32_t a0 = pk(qlA[j][0][0], qlA[j][0][1]), a2 = pk(qlA[j][1][0], qlA[j][1][1]);
        const uint32_t a1 = pk(qlB[j][0][0], qlB[j][0][1]), a3 = pk(qlB[j][1][0], qlB[j][1][1]);
        const uint32_t b0 = pk(qhA[j][0][0], qhA[j][0][1]), b2 = pk(qhA[j][1][0], qhA[j][1][1]);
        const uint32_t b1 = pk(qhB[j][0][0], qhB[j][0][1]), b3 = pk(qhB[j][1][0], qhB[j][1][1]);
        if constexpr (FP8) {
          mma_f16(s0, a0, a1, a2, a3, lo[0], lo[1]);
          mma_f16(s1, a0, a1, a2, a3, lo[2], lo[3]);
          mma_f16(s0, b0, b1, b2, b3, hi[0], hi[1]);
          mma_f16(s1, b0, b1, b2, b3, hi[2], hi[3]);
        } else {
          mma_bf16(s0, a0, a1, a2, a3, lo[0], lo[1]);
          mma_bf16(s1, a0, a1, a2, a3, lo[2], lo[3]);
          mma_bf16(s0, b0, b1, b2, b3, hi[0], hi[1]);
          mma_bf16(s1, b0, b1, b2, b3, hi[2], hi[3]);
        }
      }

      // ---- online softmax of the two rows (log2 domain); this lane holds, of each row, the keys kk[0..3]:
      // 2t, 2t+1, 8+2t, 9+2t (bf16 pages) or 4t .. 4t+3 (8-bit pages)
      const float k_scale = FP8 ? scl[stage * 2] : 1.f, v_scale = FP8 ? scl[stage * 2 + 1] : 1.f;
      float sa[4] = {s0[0] * k_scale, s0[1] * k_scale, s1[0] * k_scale, s1[1] * k_scale};
      float sb[4] = {s0[2] * k_scale, s0[3] * k_scale, s1[2] * k_scale, s1[3] * k_scale};
      if (n_valid < kTile) {
        const int kk[4] = {FP8 ? 4 * t : 2 * t, FP8 ? 4 * t + 1 : 2 * t + 1, FP8 ? 4 * t + 2 : 2 * t + 8, FP8 ? 4 * t + 3 : 2 * t + 9};
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (kk[i] >= n_valid) { sa[i] = -INFINITY; sb[i] = -INFINITY; }
      }
      float mxa = fmaxf(fmaxf(sa[0], sa[1]), fmaxf(sa[2], sa[3])), mxb = fmaxf(fmaxf(sb[0], sb[1]), fmaxf(sb[2], sb[3]));
      mxa = fmaxf(mxa, __shfl_xor_sync(kFull, mxa, 1)); mxb = fmaxf(mxb, __shfl_xor_sync(kFull, mxb, 1));
      mxa = fmaxf(mxa, __shfl_xor_sync(kFull, mxa, 2)); mxb = fmaxf(mxb, __shfl_xor_sync(kFull, mxb, 2));
      if (__any_sync(kFull, mxa > mA || mxb > mB)) {
        const float na = fmaxf(mA, mxa), nb = fmaxf(mB, mxb);
        const float fa = ex2(mA - na), fb = ex2(mB - nb);     // 0 on the first tile (running max = -inf)
        mA = na; mB = nb; lA *= fa; lB *= fb;
#pragma unroll
        for (int nd = 0; nd < ND; ++nd) { acc[nd][0] *= fa; acc[nd][1] *= fa; acc[nd][2] *= fb; acc[nd][3] *= fb; }
      }
      const float pa0 = ex2(sa[0] - mA), pa1 = ex2(sa[1] - mA), pa2 = ex2(sa[2] - mA), pa3 = ex2(sa[3] - mA);
      const float pb0 = ex2(sb[0] - mB), pb1 = ex2(sb[1] - mB), pb2 = ex2(sb[2] - mB), pb3 = ex2(sb[3] - mB);
      lA += (pa0 + pa1) + (pa2 + pa3);
      lB += (pb0 + pb1) + (pb2 + pb3);
      // A fragment of P (carrying the V scale of the tile on 8-bit pages): a0 row g keys kk[0], kk[1]; a1 row g+8 the
      // same keys; a2 row g keys kk[2], kk[3]; a3 row g+8 the same
      uint32_t f0, f1, f2, f3;
      if constexpr (FP8) {
        f0 = pack_f16x2(pa0 * v_scale, pa1 * v_scale); f1 = pack_f16x2(pb0 * v_scale, pb1 * v_scale);
        f2 = pack_f16x2(pa2 * v_scale, pa3 * v_scale); f3 = pack_f16x2(pb2 * v_scale, pb3 * v_scale);
      } else {
        f0 = pack_bf16x2(pa0, pa1); f1 = pack_bf16x2(pb0, pb1); f2 = pack_bf16x2(pa2, pa3); f3 = pack_bf16x2(pb2, pb3);
      }

      // ---- O += P V : B fragments of V by transposing ldmatrix
      if constexpr (FP8) {
        // the transposing 8-bit ldmatrix hands this lane keys 4t..4t+3 of dims g and g + 8 of a 16-dim block
#pragma unroll
        for (int c = 0; c < D / 16; c += 2) {
          uint32_t raw[4];          // [block c: dim g, dim g + 8 | block c + 1: dim g, dim g + 8]
          {
            const int key = lane & 15, chk = c + (lane >> 4);
            ldmatrix_b8_trans_x2(raw, vs_addr + key * 128 + ((chk ^ (key & 7)) << 4));
          }
#pragma unroll
          for (int m = 0; m < 4; ++m) {
            uint32_t v0, v1;
            e4m3x4_to_f16x2x2(raw[m], v0, v1);
            mma_f16(acc[2 * c + m], f0, f1, f2, f3, v0, v1);
          }
        }
      } else {
#pragma unroll
        for (int nd = 0; nd < ND; nd += 2) {
          uint32_t vb[4];             // [b0, b1] of n-tile nd, [b0, b1] of n-tile nd+1
          {
            // lane -> (matrix mi, row): key = 8 (mi & 1) + row, 16-byte chunk nd + (mi >> 1)
            const int mi = lane >> 3, key = ((mi & 1) << 3) + (lane & 7);
            const int chk = nd + (mi >> 1);
            ldmatrix_x4_trans(vb, vs_addr + (chk / 8) * kBlockBytes + key * 128 + (((chk % 8) ^ (key & 7)) << 4));
          }
          mma_bf16(acc[nd], f0, f1, f2, f3, vb[0], vb[1]);
          mma_bf16(acc[nd + 1], f0, f1, f2, f3, vb[2], vb[3]);
        }
      }
    }
    __syncwarp();   // every lane is done with this stage

    if (issued < n_tiles) { issue(stage); ++issued; }
    if (++ct == c_nt) {
      ct = 0;
      if (++ch == p.n_kv_heads) { ch = 0; ++ci; }
    }
    if (++stage == kStages) { stage = 0; parity ^= 1u; }
  }
  flush();
}

// ---------------------------------------------------------------- merge
// One CTA of four warps per (request, kv head, query head): the row's partials, which the plan laid out as one
// contiguous run of slots, are dealt round-robin to the warps; a lane owns four output dims.  Two passes
// (m* = max m; l* = sum l 2^(m - m*), o* = sum o 2^(m - m*)), the warps' results combined through shared memory,
// out = o* / l* -> bf16.  Many small CTAs with short load chains: the kernel is pure latency.
template <int D, int G>
__global__ void __launch_bounds__(128) mepic_decode_grouped_merge(const GroupedParams p) {
  const int unit = blockIdx.x / G, g = blockIdx.x % G;          // unit = request * n_kv_heads + kv head
  const int b = unit / p.n_kv_heads, h = unit % p.n_kv_heads;
  const int wv = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float sh_m[4], sh_l[4];
  __shared__ float4 sh_o[4][D / 4];
  if (h == 0 && g == 0 && threadIdx.x == 0) {
    const int kvl = p.kv_len[b];
    if ((kvl + p.page_size - 1) / p.page_size != p.plan[p.off_req_ent + b]) atomicOr(p.status, MEPIC_DEV_BAD_PLAN);
  }
  const int k0 = __ldg(p.plan + p.off_part_off + unit), k1 = __ldg(p.plan + p.off_part_off + unit + 1);
  // launched as a programmatic dependent of the grouped kernel: its partials are complete and visible after this
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // a piece that saw no valid slot of the row left (max, sum) = (-inf, 0): it drops out of both passes
  float m_mine = -INFINITY;
  for (int k = k0 + wv; k < k1; k += 4) m_mine = fmaxf(m_mine, p.part_ml[(static_cast<size_t>(k) * G + g) * 2]);
  if (lane == 0) sh_m[wv] = m_mine;
  __syncthreads();
  const float m_star = fmaxf(fmaxf(sh_m[0], sh_m[1]), fmaxf(sh_m[2], sh_m[3]));
  float l_mine = 0.f;
  float4 o_mine = make_float4(0.f, 0.f, 0.f, 0.f);
  const bool has_dims = lane < D / 4;
#pragma unroll 2
  for (int k = k0 + wv; k < k1; k += 4) {
    const size_t row = static_cast<size_t>(k) * G + g;
    const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + row * 2);
    const float wgt = ml.y > 0.f ? ex2(ml.x - m_star) : 0.f;
    l_mine += ml.y * wgt;
    if (has_dims) {
      const float4 o = *reinterpret_cast<const float4*>(p.part_o + row * D + 4 * lane);
      o_mine.x += o.x * wgt; o_mine.y += o.y * wgt; o_mine.z += o.z * wgt; o_mine.w += o.w * wgt;
    }
  }
  if (lane == 0) sh_l[wv] = l_mine;
  if (has_dims) sh_o[wv][lane] = o_mine;
  __syncthreads();
  if (wv == 0 && has_dims) {
    const float l_star = (sh_l[0] + sh_l[1]) + (sh_l[2] + sh_l[3]);
    float4 o = sh_o[0][lane];
#pragma unroll
    for (int k = 1; k < 4; ++k) { const float4 x = sh_o[k][lane]; o.x += x.x; o.y += x.y; o.z += x.z; o.w += x.w; }
    const float inv = l_star > 0.f ? 1.f / l_star : 0.f;
    const size_t o_at = (static_cast<size_t>(b) * p.n_kv_heads * G + static_cast<size_t>(h) * G + g) * D + 4 * lane;
    const uint32_t lo = static_cast<uint32_t>(f32_to_bf16_bits(o.x * inv)) | (static_cast<uint32_t>(f32_to_bf16_bits(o.y * inv)) << 16);
    const uint32_t hi = static_cast<uint32_t>(f32_to_bf16_bits(o.z * inv)) | (static_cast<uint32_t>(f32_to_bf16_bits(o.w * inv)) << 16);
    *reinterpret_cast<uint2*>(p.out + o_at) = make_uint2(lo, hi);
  }
}

template <int D, int G, bool FP8>
constexpr size_t grouped_smem_bytes() {
  // per warp: 3 stages of (K blocks + V blocks), 128 bytes of barriers and tile bases, 32 bytes of tile scales; one table
  // row; 1 KB alignment slack
  return static_cast<size_t>(kWarps) * (3 * 2 * (FP8 ? 1 : D / 64) * kTile * 128 + 128 + 32) + D * 4 + 1024;
}

template <int D, int G, bool FP8>
int32_t launch_grouped(const GroupedParams& p, int n_ctas, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream) {
  constexpr size_t smem = grouped_smem_bytes<D, G, FP8>();
  cudaError_t e = cudaFuncSetAttribute(mepic_decode_grouped<D, G, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) { mepic_set_error("decode_grouped: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_decode_grouped<D, G, FP8><<<n_ctas, kWarps * 32, smem, stream>>>(p, map_k, map_v);
  e = launch_dependent(mepic_decode_grouped_merge<D, G>, dim3(p.batch * p.n_kv_heads * G), dim3(128), stream, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { mepic_set_error("decode_grouped: launch: %s", cudaGetErrorString(e)); return MEPIC_E_CUDA; }
  mepic_count_launches(2);
  return MEPIC_OK;
}

bool plan_header_ok(const mepic_config_t* cfg, const int32_t* h, int32_t batch) {
  if (!h || h[kPhMagic] != kPlanMagic) { mepic_set_error("decode_grouped: plan_host is not a plan"); return false; }
  const int G = cfg->n_q_heads / cfg->n_kv_heads;
  if (h[kPhR] != plan_group_requests(G) || h[kPhPageSize] != cfg->page_size || (batch >= 0 && h[kPhBatch] != batch) ||
      h[kPhKvHeads] != cfg->n_kv_heads || h[kPhWorkers] < kWarps || h[kPhWorkers] % kWarps != 0 || h[kPhPiece] < 1 || h[kPhItems] < 1) {
    mepic_set_error("decode_grouped: the plan was built for another config or batch"); return false;
  }
  return true;
}

size_t grouped_slots(const mepic_config_t*, const int32_t* h) { return static_cast<size_t>(h[kPhSlots]) + 1; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" size_t mepic_attn_decode_grouped_workspace(const mepic_config_t* cfg, const int32_t* plan_host) {
  if (!mepic_config_ok(cfg) || !plan_header_ok(cfg, plan_host, -1)) return 0;
  const int G = cfg->n_q_heads / cfg->n_kv_heads;
  return grouped_slots(cfg, plan_host) * G * (cfg->head_dim + 2) * sizeof(float);
}

static int32_t grouped_call(const mepic_config_t* cfg, const mepic_decode_grouped_args_t* a, const float* k_scales, const float* v_scales,
                            bool fp8, void* cuda_stream) {
  if (!mepic_config_ok(cfg)) return MEPIC_E_INVAL;
  if (fp8 && cfg->head_dim != 128) { mepic_set_error("decode_grouped_fp8: head_dim %d: 8-bit pages are built for head_dim 128", cfg->head_dim); return MEPIC_E_INVAL; }
  if (fp8 && (!k_scales || !v_scales)) { mepic_set_error("decode_grouped_fp8: NULL scale pointer"); return MEPIC_E_INVAL; }
  if (!a || !a->q || !a->k_pool || !a->v_pool || !a->plan || !a->plan_host || !a->kv_len || !a->q_pos ||
      !a->rope_table || !a->out || !a->workspace || !a->status) { mepic_set_error("decode_grouped: NULL pointer argument"); return MEPIC_E_INVAL; }
  if (a->batch < 1) { mepic_set_error("decode_grouped: batch must be positive"); return MEPIC_E_INVAL; }
  if (!aligned16(a->q) || !aligned16(a->k_pool) || !aligned16(a->v_pool) || !aligned16(a->workspace) ||
      !aligned16(a->rope_table) || !aligned16(a->out) || !aligned16(a->plan)) { mepic_set_error("decode_grouped: pointers must be 16-byte aligned"); return MEPIC_E_INVAL; }
  if (cfg->max_position < kTile) { mepic_set_error("decode_grouped: rope table must cover positions 0..16"); return MEPIC_E_INVAL; }
  const int32_t* h = a->plan_host;
  if (!plan_header_ok(cfg, h, a->batch)) return MEPIC_E_INVAL;
  const int G = cfg->n_q_heads / cfg->n_kv_heads, D = cfg->head_dim;
  const size_t slots = grouped_slots(cfg, h);
  const size_t need = slots * G * (D + 2) * sizeof(float);
  if (a->workspace_bytes < need) { mepic_set_error("decode_grouped: workspace %zu < %zu bytes", a->workspace_bytes, need); return MEPIC_E_INVAL; }

  GroupedParams p;
  p.q = static_cast<const uint16_t*>(a->q);
  p.kv_len = a->kv_len; p.q_pos = a->q_pos; p.rope = a->rope_table; p.plan = a->plan;
  p.k_scales = k_scales; p.v_scales = v_scales;
  p.part_o = static_cast<float*>(a->workspace);
  p.part_ml = p.part_o + slots * G * D;
  p.out = static_cast<uint16_t*>(a->out);
  p.status = a->status;
  p.n_kv_heads = cfg->n_kv_heads; p.page_size = cfg->page_size;
  int l2 = 0; while ((kTile << l2) < cfg->page_size) ++l2;
  p.log2_tpp = l2;
  p.num_pages = cfg->num_pages; p.max_position = cfg->max_position; p.batch = a->batch;
  p.n_items = h[kPhItems]; p.piece = h[kPhPiece]; p.total = h[kPhTotal];
  p.off_items = h[kPhOffItems]; p.off_records = h[kPhOffRecords]; p.off_workers = h[kPhOffWorkers];
  p.off_req_ent = h[kPhOffReqEnt]; p.off_slot_base = h[kPhOffSlotBase]; p.off_part_off = h[kPhOffPartOff];
  p.scale_log2 = a->sm_scale * 1.4426950408889634f;
  p.spin_limit = mepic_test_spin_limit(kSpinLimit); p.skip_tile = mepic_test_skip_tile();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  alignas(64) CUtensorMap map_k, map_v;
  int32_t rc = fp8 ? mepic_make_pool_map_u8(cfg, a->k_pool, &map_k) : mepic_make_pool_map(cfg, a->k_pool, &map_k);
  if (rc != MEPIC_OK) return rc;
  rc = fp8 ? mepic_make_pool_map_u8(cfg, a->v_pool, &map_v) : mepic_make_pool_map(cfg, a->v_pool, &map_v);
  if (rc != MEPIC_OK) return rc;
  const int n_ctas = h[kPhWorkers] / kWarps;
  if (fp8) {
    switch (G) {
#define MEPIC_GROUPED_FP8_CASE(GG) case GG: return launch_grouped<128, GG, true>(p, n_ctas, map_k, map_v, st);
      MEPIC_GROUPED_FP8_CASE(1) MEPIC_GROUPED_FP8_CASE(2) MEPIC_GROUPED_FP8_CASE(3) MEPIC_GROUPED_FP8_CASE(4)
      MEPIC_GROUPED_FP8_CASE(5) MEPIC_GROUPED_FP8_CASE(6) MEPIC_GROUPED_FP8_CASE(7) MEPIC_GROUPED_FP8_CASE(8)
#undef MEPIC_GROUPED_FP8_CASE
    }
  }

#define MEPIC_GROUPED_CASE(DD, GG) if (D == DD && G == GG) return launch_grouped<DD, GG, false>(p, n_ctas, map_k, map_v, st);
  MEPIC_GROUPED_CASE(128, 1) MEPIC_GROUPED_CASE(128, 2) MEPIC_GROUPED_CASE(128, 3) MEPIC_GROUPED_CASE(128, 4) MEPIC_GROUPED_CASE(128, 5) MEPIC_GROUPED_CASE(128, 6) MEPIC_GROUPED_CASE(128, 7) MEPIC_GROUPED_CASE(128, 8)
  MEPIC_GROUPED_CASE(64, 1) MEPIC_GROUPED_CASE(64, 2) MEPIC_GROUPED_CASE(64, 3) MEPIC_GROUPED_CASE(64, 4) MEPIC_GROUPED_CASE(64, 5) MEPIC_GROUPED_CASE(64, 6) MEPIC_GROUPED_CASE(64, 7) MEPIC_GROUPED_CASE(64, 8)
#undef MEPIC_GROUPED_CASE
  mepic_set_error("decode_grouped: unsupported head_dim %d / group size %d", D, G);
  return MEPIC_E_INVAL;
}

extern "C" int32_t mepic_attn_decode_grouped(const mepic_config_t* cfg, const mepic_decode_grouped_args_t* a, void* cuda_stream) {
  return grouped_call(cfg, a, nullptr, nullptr, false, cuda_stream);
}

extern "C" int32_t mepic_attn_decode_grouped_fp8(const mepic_config_t* cfg, const mepic_decode_grouped_args_t* a, const float* k_scales,
                                                 const float* v_scales, void* cuda_stream) {
  return grouped_call(cfg, a, k_scales, v_scales, true, cuda_stream);
}
