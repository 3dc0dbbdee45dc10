"""8-bit (e4m3) pages end to end, on a pool that has NO bf16 copy: store -> block tables -> prefill that commits codes
and attends over them -> decode over the same pools, against the oracle.

Every chunk starts uncomputed (Section 3.3.1: a newly encountered chunk is recomputed whole), so the first request that
uses a chunk commits ALL of its pages through mepic_attn_prefill_fp8; later requests alias those 8-bit pages and
commit only their own first blocks and prompt pages.  Checked: the code pools and the scales bit for bit against the
oracle's commit rule (whole pages, a NaN element, and rows appended later to a partly filled page under the kept
scale), the prefill outputs and the decode outputs against the fp64 oracle evaluated on the same codes and scales at
the bf16 path's tolerance (max-abs 2e-2, mean-abs 2e-3; relative L2 2e-2 / 1e-2)."""
import numpy as np
import pytest
import torch

import paper_2512_16822_b200 as M
from paper_2512_16822_b200 import runtime as RT
from paper_2512_16822_b200.build import build_library
from mepic_inputs import f32_to_bf16_bits, bf16_bits_to_f64
from oracle import mepic_oracle as O

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"


def _check(got_bits, want, rel_bar, what=""):
    got = bf16_bits_to_f64(got_bits)
    d = np.abs(got - want)
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert np.isfinite(got).all(), what
    assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (what, d.max(), d.mean())
    assert rel <= rel_bar, (what, rel)


class _Side:
    """The library's pools on the GPU and the oracle's on the host, driven with the same calls."""

    def __init__(self, cfg, theta):
        self.cfg, self.theta = cfg, theta
        self.dev = RT.Device(cfg, bf16_pools=False)
        self.pools = RT.Fp8Pools(self.dev)
        shape = (cfg.num_pages, cfg.n_kv_heads, cfg.page_size, cfg.head_dim)
        self.okc, self.ovc = np.zeros(shape, dtype=np.uint8), np.zeros(shape, dtype=np.uint8)
        self.oks = np.ones((cfg.num_pages, cfg.n_kv_heads), dtype=np.float32); self.ovs = self.oks.copy()

    def prefill(self, tables, rows, sm, rel_bar=2e-2, what=""):
        """tables: list of (page_ids, pos_base, kv_len, slots); rows: list of (q, k, v) bit arrays per request."""
        B = len(tables)
        stride = max(len(t[0]) for t in tables)
        ids = np.zeros((B, stride), dtype=np.int32); base = np.zeros((B, stride), dtype=np.int32)
        for b, t in enumerate(tables):
            ids[b, :len(t[0])] = t[0]; base[b, :len(t[1])] = t[1]
        kvl = np.array([t[2] for t in tables], dtype=np.int32)
        ro = np.concatenate([[0], np.cumsum([len(t[3]) for t in tables])]).astype(np.int32)
        pb = RT.Fp8PrefillBatch(self.pools, ids, base, kvl, ro, np.concatenate([t[3] for t in tables]).astype(np.int32),
                                np.concatenate([r[0] for r in rows]), np.concatenate([r[1] for r in rows]),
                                np.concatenate([r[2] for r in rows]))
        out = pb.run(sm); torch.cuda.synchronize()
        assert self.dev.read_status() == 0, what
        got = RT.bf16_bits(out)
        # the oracle: commit every request's rows first (the library's commit kernel precedes its attention kernel),
        # then attention over the de-quantised pools
        for t, r in zip(tables, rows):
            O.commit_rows_fp8(self.okc, self.oks, self.ovc, self.ovs, list(t[0]), list(t[3]), r[1], r[2])
        self.compare_pools(what)
        kf, vf = O.dequantize_pages(self.okc, self.oks), O.dequantize_pages(self.ovc, self.ovs)
        for b, (t, r) in enumerate(zip(tables, rows)):
            want = O.prefill_attention_one(r[0], r[1], r[2], list(t[3]), kf, vf, list(t[0]), list(t[1]), int(t[2]), sm, self.theta)
            _check(got[ro[b]:ro[b + 1]], want, rel_bar, f"{what} prefill request {b}")

    def compare_pools(self, what=""):
        assert np.array_equal(self.pools.k_codes.cpu().numpy(), self.okc), what
        assert np.array_equal(self.pools.v_codes.cpu().numpy(), self.ovc), what
        assert np.array_equal(self.pools.k_scales.cpu().numpy(), self.oks) and np.array_equal(self.pools.v_scales.cpu().numpy(), self.ovs), what

    def decode(self, tables, q, sm, what=""):
        B = len(tables)
        stride = max(len(t[0]) for t in tables)
        ids = np.zeros((B, stride), dtype=np.int32); base = np.zeros((B, stride), dtype=np.int32)
        for b, t in enumerate(tables):
            ids[b, :len(t[0])] = t[0]; base[b, :len(t[1])] = t[1]
        kvl = np.array([t[2] for t in tables], dtype=np.int32)
        P = self.cfg.page_size
        q_pos = np.array([t[1][(t[2] - 1) // P] + (t[2] - 1) % P for t in tables], dtype=np.int32)
        out = RT.Fp8DecodeBatch(self.pools, ids, base, kvl, q_pos, q).run(sm); torch.cuda.synchronize()
        assert self.dev.read_status() == 0, what
        got = RT.bf16_bits(out).copy()
        kf, vf = O.dequantize_pages(self.okc, self.oks), O.dequantize_pages(self.ovc, self.ovs)
        gout = RT.Fp8GroupedDecodeBatch(self.pools, ids, base, kvl, q_pos, q).run(sm); torch.cuda.synchronize()
        assert self.dev.read_status() == 0, what
        ggot = RT.bf16_bits(gout)
        for b, t in enumerate(tables):
            want = O.decode_attention_one(q[b], kf, vf, list(t[0]), list(t[1]), int(t[2]), int(q_pos[b]), sm, self.theta)
            _check(got[b], want, 1e-2, f"{what} decode request {b}")
            _check(ggot[b], want, 1e-2, f"{what} grouped decode request {b}")


@pytest.mark.parametrize("Hq,Hkv,P,n_chunks,chunk_pages,question", [(8, 2, 16, 3, 9, 40), (10, 2, 16, 2, 5, 21), (4, 4, 64, 2, 3, 70),
                                                                    (32, 8, 16, 4, 32, 64)])
def test_store_prefill_decode_on_8bit_pools_only(Hq, Hkv, P, n_chunks, chunk_pages, question):
    D, theta = 128, 5e5
    sm = 1.0 / np.sqrt(D)
    rng = np.random.default_rng(1000 * Hq + P + n_chunks)
    bits = lambda shape, std=1.0: f32_to_bf16_bits((rng.standard_normal(shape) * std).astype(np.float32))
    chunks = [rng.integers(1, 32000, size=chunk_pages * P, dtype=np.int32) for _ in range(n_chunks)]
    num_pages = n_chunks * chunk_pages + 3 * (n_chunks + 8) + 8 + 2 * (P + 3)     # the top 2 (P + 3) pages stay outside the store's reach
    cfg = M.Config(P, Hq, Hkv, D, num_pages, (n_chunks * chunk_pages + 8) * P, theta)
    side = _Side(cfg, theta)
    ost = O.OracleStore(P, num_pages)
    with M.Store(cfg) as st:
        assert n_chunks * (chunk_pages - 1) + 2 * (n_chunks + -(-question // P)) <= num_pages - 2 * (P + 3)
        cids, keys = [], []
        for toks in chunks:
            cid, res, _, _ = st.chunk_register(toks); key, _, _ = ost.register_chunk(toks)
            st.chunk_mark_uncomputed(cid); ost.mark_uncomputed(key)           # nobody has any K/V yet
            cids.append(cid); keys.append(key)
        orders = [list(range(n_chunks)), list(reversed(range(n_chunks)))]
        tabs = []
        for rid, order in enumerate(orders):
            segs = [M.Segment(M.MEPIC_SEG_CHUNK, cids[c]) for c in order] + [M.Segment(M.MEPIC_SEG_PROMPT, question)]
            osegs = [(O.KIND_CHUNK, keys[c]) for c in order] + [(O.KIND_PROMPT, question)]
            pages, base, kv_len, slots = st.build_block_table(rid, segs)
            ot = ost.build_block_table(rid, osegs)
            assert list(pages) == ot.page_ids and list(slots) == ot.recompute_slots and kv_len == ot.kv_len
            tabs.append((pages, base, kv_len, np.asarray(slots, dtype=np.int32)))
        # request 0 computes every chunk whole (all slots are recompute slots), request 1 only first blocks + question
        assert len(tabs[0][3]) == tabs[0][2] and len(tabs[1][3]) == n_chunks * P + question
        rows = [(bits((len(t[3]), Hq, D), 1.0), bits((len(t[3]), Hkv, D)), bits((len(t[3]), Hkv, D))) for t in tabs]
        rows[0][1][3, 0, 5] = 0x7FC0                                           # one NaN element in a committed K row ...
        # ... which, by the commit rule, must not set its block's scale.  (It does poison request 0's scores of that
        # key, so the NaN is put back to a number before the attention is compared: the commit is checked first.)
        # commit-only check of the NaN rule on a throw-away pair of pools
        probe = _Side(cfg, theta)
        nan_rows = (rows[0][0][:P], rows[0][1][:P].copy(), rows[0][2][:P])
        t0 = (tabs[0][0], tabs[0][1], P, tabs[0][3][:P])
        B = RT.Fp8PrefillBatch(probe.pools, np.asarray([t0[0]], dtype=np.int32), np.asarray([t0[1]], dtype=np.int32), np.array([P], dtype=np.int32),
                               np.array([0, P], dtype=np.int32), t0[3], *nan_rows)
        B.run(sm); torch.cuda.synchronize()
        O.commit_rows_fp8(probe.okc, probe.oks, probe.ovc, probe.ovs, list(t0[0]), list(t0[3]), nan_rows[1], nan_rows[2])
        probe.compare_pools("NaN element in a committed row")
        assert probe.okc[t0[0][0], 0, 3, 5] == 0x7F and np.isfinite(probe.oks).all()
        rows[0][1][3, 0, 5] = 0x3F80
        # one call per request, in order (request 1 attends over pages request 0 committed)
        side.prefill([tabs[0]], [rows[0]], sm, what="whole-chunk materialisation")
        side.prefill([tabs[1]], [rows[1]], sm, what="aliasing request")
        q = bits((2, Hq, D))
        side.decode(tabs, q, sm, what="after prefill")
        # decode steps append one token each into the question's last page: rows that do not include the page's slot 0
        # keep the page's scale (and saturate); a row that opens a new page sets that page's scale
        for step in range(P + 2):
            new_tabs, new_rows = [], []
            for rid, t in enumerate(tabs):
                pages, base, kv_len, _ = t
                if kv_len % P == 0:                                            # the last page is full: a fresh private page
                    spare = num_pages - 1 - 2 * step - rid                     # pages nobody uses (the pool has slack at the top)
                    pages = np.append(pages, spare).astype(np.int32); base = np.append(base, base[-1] + P).astype(np.int32)
                new_tabs.append((pages, base, kv_len + 1, np.array([kv_len], dtype=np.int32)))
                big = 6.0 if step == 2 else 1.0                                # one appended row larger than its block's range
                new_rows.append((bits((1, Hq, D)), bits((1, Hkv, D), big), bits((1, Hkv, D), big)))
            side.prefill(new_tabs, new_rows, sm, what=f"append step {step}")
            tabs = new_tabs
        side.decode(tabs, bits((2, Hq, D)), sm, what="after the appends")


def test_config3_full_size_prefill_on_8bit_pools_sampled_rows():
    # The launch bench.py times (8 requests x 768 rows over 16 640 cached tokens, 8-bit pools, no bf16 copy while the
    # call runs).  The oracle quantises the pages request 0 reads (the library's codes and scales for them must agree
    # bit for bit), commits request 0's rows by its own rule and evaluates sampled rows on those codes and scales.
    from mepic_inputs import make_workload
    wl = make_workload(3)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.prefill_requests)
    page_ids, pos_base, kv_len, _ = RT.pack_tables(tables, wl.page_size)
    q_slots = [np.asarray(t.recompute_slots, dtype=np.int32) for t in tables]
    rows = [wl.prefill_rows(i, len(s)) for i, s in enumerate(q_slots)]
    ro = np.concatenate([[0], np.cumsum([len(s) for s in q_slots])]).astype(np.int32)
    dev = RT.Device(cfg, kp, vp)
    pools = RT.Fp8Pools(dev)                              # the library's quantiser over the whole pool
    torch.cuda.synchronize()
    dev.k_pool = dev.v_pool = None                        # from here on the 8-bit pools are the only pools
    torch.cuda.empty_cache()
    n0 = -(-int(kv_len[0]) // wl.page_size)
    mine = np.unique(page_ids[0, :n0])
    okc, oks = O.quantize_pages(kp[mine]); ovc, ovs = O.quantize_pages(vp[mine])
    sel = torch.from_numpy(mine.astype(np.int64)).to(dev.device)
    assert np.array_equal(pools.k_codes[sel].cpu().numpy(), okc) and np.array_equal(pools.k_scales[sel].cpu().numpy(), oks)
    assert np.array_equal(pools.v_codes[sel].cpu().numpy(), ovc) and np.array_equal(pools.v_scales[sel].cpu().numpy(), ovs)
    pb = RT.Fp8PrefillBatch(pools, page_ids, pos_base, kv_len, ro, np.concatenate(q_slots),
                            np.concatenate([r.q_new for r in rows]), np.concatenate([r.k_new for r in rows]),
                            np.concatenate([r.v_new for r in rows]))
    out = pb.run(wl.sm_scale); torch.cuda.synchronize()
    assert dev.read_status() == 0 and not pb.repeated()
    # the oracle's copy of request 0's pages, renumbered 0 .. len(mine) - 1
    local = {int(pg): i for i, pg in enumerate(mine)}
    ids0 = [local[int(pg)] for pg in page_ids[0, :n0]]
    O.commit_rows_fp8(okc, oks, ovc, ovs, ids0, list(q_slots[0]), rows[0].k_new, rows[0].v_new)
    assert np.array_equal(pools.k_codes[sel].cpu().numpy(), okc) and np.array_equal(pools.k_scales[sel].cpu().numpy(), oks)
    assert np.array_equal(pools.v_codes[sel].cpu().numpy(), ovc) and np.array_equal(pools.v_scales[sel].cpu().numpy(), ovs)
    R = len(q_slots[0])
    pick = sorted(set([0, 1, 15, 16, 255, 256, R // 2, R - 257, R - 256, R - 2, R - 1] + list(range(5, R, 61))))
    want = O.prefill_attention_one(rows[0].q_new, rows[0].k_new, rows[0].v_new, list(q_slots[0]),
                                   O.dequantize_pages(okc, oks), O.dequantize_pages(ovc, ovs), ids0, list(pos_base[0, :n0]),
                                   int(kv_len[0]), wl.sm_scale, wl.rope_theta, rows=pick)
    _check(RT.bf16_bits(out)[:R][pick], want, 2e-2, "config 3, request 0, 8-bit pools")
