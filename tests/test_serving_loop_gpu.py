"""A serving loop on the GPU, every piece together, checked against the oracle after every step.

Requests arrive (chunks registered, block table built under memory pressure, new chunks computed whole and
cached ones by their first block only through the prefill call), every live request decodes a token (per-request
and sharing-aware kernels alternate), requests leave.  The pool is too small for every chunk, so chunks are
evicted to the remote tier and brought back (Algorithm 1: residency resolution, admission check, block assignment;
Sections 3.2.3 and 3.3.1-3.3.3).  Compared at every step: tables, residency answers, counters, prefill and decode
outputs (tolerance of the bf16 kernels) and the K/V pools bit for bit.
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


def _close(got_bits, want, what):
    d = np.abs(bf16_bits_to_f64(got_bits) - want)
    assert d.max() <= 2e-2 and d.mean() <= 2e-3, (what, d.max(), d.mean())


@pytest.mark.parametrize("seed,num_pages,remote_pages", [(0, 44, 80), (1, 38, 14)])
def test_serving_loop_under_memory_pressure(seed, num_pages, remote_pages):
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    P, Hq, Hkv, D, theta = 16, 8, 2, 128, 1e4
    sm = 1.0 / np.sqrt(D)
    rng = np.random.default_rng(seed)
    bits = lambda shape: f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    chunks = [rng.integers(1, 30000, size=int(n)).astype(np.int32) for n in rng.integers(3 * P - 5, 8 * P, size=14)]
    cfg = M.Config(P, Hq, Hkv, D, num_pages, 1024, theta)
    kp, vp = bits((num_pages, Hkv, P, D)), bits((num_pages, Hkv, P, D))
    okp, ovp = kp.copy(), vp.copy()
    dev = RT.Device(cfg, kp, vp)
    ost = O.OracleStore(P, num_pages)
    ost.attach_remote(okp, ovp, remote_pages)
    live = {}                                              # request id -> RT.Table
    seen = {0: 0, 1: 0, 2: 0}
    rejected = 0
    with M.Store(cfg) as st:
        st.attach_remote(dev.k_pool, dev.v_pool, remote_pages, torch.cuda.current_stream())
        for step in range(48):
            # ---- departures
            for rid in [r for r in list(live) if rng.random() < 0.3]:
                st.request_release(rid); ost.release(rid)
                del live[rid]
            # ---- one arrival
            picks = [int(c) for c in rng.choice(len(chunks), size=int(rng.integers(1, 4)), replace=False)]
            lsegs, osegs, ok = [], [], True
            for c in picks:
                try:
                    cid, res, _, pages = st.chunk_register(chunks[c])
                except M.MepicError as e:
                    assert e.code == M.MEPIC_E_NOSPACE
                    with pytest.raises(O.Reject):
                        ost.register_chunk(chunks[c])
                    ok = False
                    break
                okey, ores, opages = ost.register_chunk(chunks[c])
                assert res == ores and list(pages) == opages, (step, c)
                seen[res] += 1
                if res == 0 and len(pages):                # nobody has this chunk's K/V: the first user computes it whole
                    st.chunk_mark_uncomputed(cid); ost.mark_uncomputed(okey)
                lsegs.append(M.Segment(M.MEPIC_SEG_CHUNK, cid)); osegs.append((O.KIND_CHUNK, okey))
            if ok:
                qlen = int(rng.integers(1, 30))
                lsegs.append(M.Segment(M.MEPIC_SEG_PROMPT, qlen)); osegs.append((O.KIND_PROMPT, qlen))
                try:
                    pages, base, kvl, slots = st.build_block_table(step, lsegs)
                except M.MepicError as e:
                    assert e.code in (M.MEPIC_E_NOSPACE, M.MEPIC_E_NOTFOUND)
                    with pytest.raises((O.Reject, KeyError)):
                        ost.build_block_table(step, osegs)
                    rejected += 1
                else:
                    ot = ost.build_block_table(step, osegs)
                    assert list(pages) == ot.page_ids and list(base) == ot.pos_base and kvl == ot.kv_len
                    assert list(slots) == ot.recompute_slots
                    t = RT.Table(step, pages, base, kvl, slots)
                    live[step] = t
                    # ---- materialise: commit the recomputed rows and attend (one prefill call for the new request)
                    R = len(slots)
                    qn, kn, vn = bits((R, Hq, D)), bits((R, Hkv, D)), bits((R, Hkv, D))
                    page_ids, pos_base, kv_len, _ = RT.pack_tables([t], P)
                    pb = RT.PrefillBatch(dev, page_ids, pos_base, kv_len, np.array([0, R], dtype=np.int32), slots, qn, kn, vn)
                    out = pb.run(sm)
                    torch.cuda.synchronize()
                    assert dev.read_status() == 0
                    want = O.prefill_attention_one(qn, kn, vn, list(slots), okp, ovp, list(pages), list(base), kvl, sm, theta)
                    _close(RT.bf16_bits(out), want, ("prefill", step))
            assert st.stats() == ost.stats(), step
            torch.cuda.synchronize()
            assert np.array_equal(RT.bf16_bits(dev.k_pool), okp) and np.array_equal(RT.bf16_bits(dev.v_pool), ovp), step
            # ---- every live request decodes one token
            if live:
                order = sorted(live)
                page_ids, pos_base, kv_len, q_pos = RT.pack_tables([live[r] for r in order], P)
                q = bits((len(order), Hq, D))
                kind = RT.GroupedDecodeBatch if step % 2 else RT.DecodeBatch
                out = kind(dev, page_ids, pos_base, kv_len, q_pos, q).run(sm)
                torch.cuda.synchronize()
                assert dev.read_status() == 0
                got = RT.bf16_bits(out)
                for b, r in enumerate(order):
                    t = live[r]
                    want = O.decode_attention_one(q[b], okp, ovp, list(t.page_ids), list(t.pos_base), t.kv_len, int(q_pos[b]), sm, theta)
                    _close(got[b], want, ("decode", step, r))
        s = st.stats()
    assert s["chunks_evicted"] > 3 and s["chunks_spilled"] > 0 and seen[1] > 0, (s, seen)
    assert seen[2] > 0 or remote_pages < 20, (s, seen)
