"""The whole path on ragged inputs: store -> block tables -> prefill (commit + attention) -> decode, vs the oracle.

Chunk lengths are not page multiples (leading pads), prompts in the middle get trailing pads (Section 3.2.1), pads
are ordinary attended tokens; one chunk is new and is therefore recomputed whole by the first request that uses
it (Section 3.3.1), after which a second request aliases the pages that first request committed.
"""
import numpy as np
import pytest
import torch

import paper_2512_16822_b200 as M
from paper_2512_16822_b200 import runtime as RT
from paper_2512_16822_b200.build import build_library
from mepic_inputs import f32_to_bf16_bits, bf16_bits_to_f64
from oracle import mepic_oracle as O

pytestmark = pytest.mark.gpu


class _Rows:
    def __init__(self, q, k, v): self.q_new, self.k_new, self.v_new = q, k, v


@pytest.mark.parametrize("Hq,Hkv,D,P", [(8, 2, 128, 16), (10, 2, 64, 32)])
def test_ragged_chunks_full_materialisation_then_sharing(Hq, Hkv, D, P):
    build_library()
    rng = np.random.default_rng(77 + D + P)
    theta, sm = 1e4, 1.0 / np.sqrt(D)
    A = rng.integers(1, 999, size=5 * P + 9, dtype=np.int32)        # leading pads: P - 9
    B = rng.integers(1, 999, size=3 * P + 1, dtype=np.int32)
    Cc = rng.integers(1, 999, size=P - 3, dtype=np.int32)           # a one-page chunk: nothing shareable
    num_pages = 80
    cfg = M.Config(P, Hq, Hkv, D, num_pages, 2048, theta)
    bits = lambda shape, std=1.0: f32_to_bf16_bits((rng.standard_normal(shape) * std).astype(np.float32))
    kp, vp = bits((num_pages, Hkv, P, D)), bits((num_pages, Hkv, P, D))
    ost = O.OracleStore(P, num_pages)
    ok_pool, ov_pool = kp.copy(), vp.copy()
    dev = RT.Device(cfg, kp, vp)
    with M.Store(cfg) as st:
        ids = {}
        for name, toks in (("A", A), ("B", B), ("C", Cc)):
            key, _, _ = ost.register_chunk(toks)
            cid, res, lead, _ = st.chunk_register(toks)
            assert not res and lead == (-len(toks)) % P
            ids[name] = (key, cid)
        ost.mark_uncomputed(ids["A"][0]); st.chunk_mark_uncomputed(ids["A"][1])     # nobody has A's K/V yet
        plans = {1: [("P", 5), ("A",), ("B",), ("C",), ("P", 7)], 2: [("P", P + 4), ("B",), ("A",), ("A",), ("P", 3)]}
        tables = {}
        for rid, plan in plans.items():
            osegs = [(O.KIND_PROMPT, s[1]) if s[0] == "P" else (O.KIND_CHUNK, ids[s[0]][0]) for s in plan]
            lsegs = [M.Segment(1, s[1]) if s[0] == "P" else M.Segment(0, ids[s[0]][1]) for s in plan]
            ot = ost.build_block_table(rid, osegs)
            pages, base, kv_len, slots = st.build_block_table(rid, lsegs)
            assert list(pages) == ot.page_ids and list(base) == ot.pos_base and kv_len == ot.kv_len
            assert list(slots) == ot.recompute_slots
            tables[rid] = RT.Table(rid, pages, base, kv_len, slots)
        assert st.stats() == ost.stats()
    # request 1 recomputes A whole, request 2 only first blocks (and aliases what request 1 committed)
    n_a = -(-len(A) // P) * P
    assert len(tables[1].recompute_slots) == P + n_a + P + P + 7
    assert len(tables[2].recompute_slots) == 2 * P + P + P + P + 3
    for rid in (1, 2):                                   # one prefill call per request, in stream order
        t = tables[rid]
        R = len(t.recompute_slots)
        rows = _Rows(bits((R, Hq, D)), bits((R, Hkv, D)), bits((R, Hkv, D)))
        page_ids, pos_base, kv_len, _ = RT.pack_tables([t], P)
        pb = RT.PrefillBatch(dev, page_ids, pos_base, kv_len, np.array([0, R], dtype=np.int32), t.recompute_slots,
                             rows.q_new, rows.k_new, rows.v_new)
        out = pb.run(sm)
        torch.cuda.synchronize()
        assert dev.read_status() == 0
        want = O.prefill_attention_one(rows.q_new, rows.k_new, rows.v_new, list(t.recompute_slots), ok_pool, ov_pool,
                                       list(t.page_ids), list(t.pos_base), t.kv_len, sm, theta)
        d = np.abs(bf16_bits_to_f64(RT.bf16_bits(out)) - want)
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, (rid, d.max(), d.mean())
        assert np.array_equal(RT.bf16_bits(dev.k_pool), ok_pool) and np.array_equal(RT.bf16_bits(dev.v_pool), ov_pool)
    # decode both requests over the pool the prefills left behind
    both = [tables[1], tables[2]]
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(both, P)
    q = bits((2, Hq, D))
    out = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q).run(sm)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    got = bf16_bits_to_f64(RT.bf16_bits(out))
    for b, t in enumerate(both):
        want = O.decode_attention_one(q[b], ok_pool, ov_pool, list(t.page_ids), list(t.pos_base), t.kv_len, int(q_pos[b]), sm, theta)
        d = np.abs(got[b] - want)
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, ("decode", b, d.max(), d.mean())
    # the two requests alias the same physical pages for B's and A's shareable blocks, at different positions
    sh_a = set(tables[1].page_ids) & set(tables[2].page_ids)
    assert len(sh_a) == (n_a // P - 1) + (-(-len(B) // P) - 1)
