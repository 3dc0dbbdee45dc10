"""Host side of the library (C ABI) against the oracle: tables and counters bit-exact.

No GPU is needed: the scheduling path is host code, and the library must load
and export every declared symbol on a machine without a driver.
"""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2512_16822_b200 as M
from paper_2512_16822_b200.build import LIB_PATH, build_library
from mepic_inputs import make_workload
from oracle import mepic_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def _cfg(P=16, num_pages=64, **kw):
    base = dict(page_size=P, n_q_heads=8, n_kv_heads=2, head_dim=64, num_pages=num_pages,
                max_position=max(4095, P - 1), rope_theta=1e4)
    base.update(kw)
    return M.Config(**base)


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "mepic.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(mepic_[a-z_]+)\s*\(", text))
    assert {"mepic_chunk_register", "mepic_build_block_table", "mepic_attn_decode", "mepic_attn_prefill"} <= declared
    handle = ctypes.CDLL(LIB_PATH)
    missing = [n for n in sorted(declared) if not hasattr(handle, n)]
    assert not missing, missing


def _run_both(wl, requests):
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    ost = O.OracleStore(wl.page_size, wl.num_pages, wl.pad_token_id)
    out = []
    with M.Store(cfg) as st:
        for r in requests:
            osegs, lsegs = [], []
            for kind, val in r.segments:
                if kind == O.KIND_CHUNK:
                    key, ores, oshared = ost.register_chunk(wl.chunks[val])
                    cid, lres, lead, lshared = st.chunk_register(wl.chunks[val])
                    assert lres == ores and list(lshared) == oshared
                    assert lead == (-len(wl.chunks[val])) % wl.page_size
                    osegs.append((kind, key)); lsegs.append(M.Segment(kind, cid))
                else:
                    osegs.append((kind, val)); lsegs.append(M.Segment(kind, val))
            ot = ost.build_block_table(r.request_id, osegs)
            pages, base, kv_len, slots = st.build_block_table(r.request_id, lsegs)
            assert list(pages) == ot.page_ids and list(base) == ot.pos_base
            assert kv_len == ot.kv_len and list(slots) == ot.recompute_slots
            out.append(ot)
        assert st.stats() == ost.stats()
        # release half of the requests on both sides, then compare the free-list order through new allocations
        for r in requests[::2]:
            ost.release(r.request_id); st.request_release(r.request_id)
        assert st.stats() == ost.stats()
        probe_o = ost.build_block_table(10 ** 9, [(O.KIND_PROMPT, 3 * wl.page_size + 1)])
        probe_l = st.build_block_table(10 ** 9, [M.Segment(M.MEPIC_SEG_PROMPT, 3 * wl.page_size + 1)])
        assert list(probe_l[0]) == probe_o.page_ids
    return out


@pytest.mark.parametrize("cfg_index,scale", [(1, 1.0), (2, 1.0), (3, 1.0), (4, 1.0), (5, 1.0), (5, 0.2)])
def test_tables_and_counters_bit_exact_on_configs(cfg_index, scale):
    wl = make_workload(cfg_index, scale=scale)
    # four spare pages so that the post-release probe request always fits
    wl.num_pages += 4
    _run_both(wl, wl.decode_requests + wl.prefill_requests)


def test_ragged_chunk_lengths_and_mid_prompts_bit_exact():
    rng = np.random.default_rng(5)
    P = 16
    chunks = [rng.integers(1, 1000, size=int(n), dtype=np.int32) for n in (1, 15, 16, 17, 40, 64, 100)]

    class R:
        def __init__(self, rid, segs): self.request_id, self.segments = rid, segs

    class W:
        pass
    wl = W()
    wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim = P, 8, 2, 64
    wl.num_pages, wl.max_position, wl.rope_theta, wl.pad_token_id, wl.chunks = 400, 4095, 1e4, 0, chunks
    reqs = []
    for rid in range(12):
        segs = []
        for _ in range(int(rng.integers(1, 6))):
            if rng.random() < 0.6:
                segs.append((O.KIND_CHUNK, int(rng.integers(0, len(chunks)))))
            else:
                segs.append((O.KIND_PROMPT, int(rng.integers(0, 50))))
        if all(k == O.KIND_PROMPT and v == 0 for k, v in segs):
            segs.append((O.KIND_PROMPT, 3))
        reqs.append(R(rid, segs))
    _run_both(wl, reqs)


def test_hand_worked_example_through_the_abi():
    with M.Store(_cfg(num_pages=32)) as st:
        a = st.chunk_register(np.arange(100, 140, dtype=np.int32))
        b = st.chunk_register(np.arange(900, 916, dtype=np.int32))
        assert list(a[3]) == [0, 1] and list(b[3]) == [] and a[2] == 8 and b[2] == 0
        S = M.Segment
        pages, base, kv_len, slots = st.build_block_table(
            7, [S(1, 5), S(0, a[0]), S(1, 20), S(0, b[0]), S(1, 7)])
        assert list(pages) == [2, 3, 0, 1, 4, 5, 6, 7]
        assert list(base) == [0, 16, 32, 48, 64, 80, 96, 112] and kv_len == 119
        assert list(slots) == list(range(0, 32)) + list(range(64, 119))


def test_error_codes_and_reject_is_transactional():
    cfg = _cfg(P=16, num_pages=6)
    with M.Store(cfg) as st:
        cid, _, _, shared = st.chunk_register(np.arange(1, 41, dtype=np.int32))     # 3 pages, 2 shared
        assert list(shared) == [0, 1]
        before = st.stats()
        with pytest.raises(M.MepicError) as e:
            st.build_block_table(1, [M.Segment(0, cid), M.Segment(1, 16 * 4)])       # 1 + 4 > 4 free, own chunk protected
        assert e.value.code == M.MEPIC_E_NOSPACE and st.stats() == before
        with pytest.raises(M.MepicError) as e:
            st.build_block_table(1, [M.Segment(0, cid + 12345)])
        assert e.value.code == M.MEPIC_E_NOTFOUND
        with pytest.raises(M.MepicError) as e:
            st.build_block_table(1, [M.Segment(1, 0)])
        assert e.value.code == M.MEPIC_E_INVAL
        st.build_block_table(1, [M.Segment(0, cid), M.Segment(1, 5)])
        held = st.stats()
        with pytest.raises(M.MepicError) as e:
            st.chunk_register(np.arange(1, 16 * 6 + 1, dtype=np.int32))              # 5 shared > 3 free, chunk in use stays
        assert e.value.code == M.MEPIC_E_NOSPACE and st.stats() == held
        with pytest.raises(M.MepicError) as e:
            st.build_block_table(1, [M.Segment(1, 5)])
        assert e.value.code == M.MEPIC_E_EXISTS
        with pytest.raises(M.MepicError) as e:
            st.request_release(2)
        assert e.value.code == M.MEPIC_E_NOTFOUND
        st.request_release(1)
        assert st.stats()["pages_free"] == 4 and st.stats()["chunk_refs"] == 0
        # now the chunk is idle: a registration that needs its pages reclaims it instead of failing
        big, res, _, pages = st.chunk_register(np.arange(1, 16 * 6 + 1, dtype=np.int32))
        assert not res and len(pages) == 5 and st.stats()["chunks_evicted"] == 1 and st.stats()["pages_evicted"] == 2
        with pytest.raises(M.MepicError) as e:
            st.build_block_table(9, [M.Segment(0, cid)])                              # its id is gone
        assert e.value.code == M.MEPIC_E_NOTFOUND
    for bad in (dict(page_size=24), dict(page_size=8), dict(head_dim=96), dict(n_q_heads=7), dict(num_pages=0),
                dict(n_q_heads=18, n_kv_heads=2)):
        with pytest.raises(M.MepicError) as e:
            M.Store(_cfg(**bad))
        assert e.value.code == M.MEPIC_E_INVAL


def test_serving_trace_under_memory_pressure_matches_oracle_step_by_step():
    """A long random trace of arrivals and departures over a pool far too small to keep every chunk: tables,
    rejections, evictions and counters must agree with the oracle after every single call."""
    rng = np.random.default_rng(21)
    P = 16
    chunks = [rng.integers(1, 5000, size=int(n), dtype=np.int32) for n in rng.integers(10, 200, size=24)]
    cfg = _cfg(P=P, num_pages=90)
    ost = O.OracleStore(P, 90)
    live, rid, rejected = [], 0, 0
    with M.Store(cfg) as st:
        for step in range(600):
            if live and (rng.random() < 0.45 or len(live) > 6):
                r = live.pop(int(rng.integers(0, len(live))))
                ost.release(r); st.request_release(r)
            else:
                rid += 1
                picks = rng.choice(len(chunks), size=int(rng.integers(1, 4)), replace=False)
                osegs, lsegs, ok = [], [], True
                for c in picks:
                    try:
                        key, ores, oshared = ost.register_chunk(chunks[c])
                    except O.Reject:
                        with pytest.raises(M.MepicError) as e:
                            st.chunk_register(chunks[c])
                        assert e.value.code == M.MEPIC_E_NOSPACE
                        ok = False
                        break
                    cid, lres, _, lshared = st.chunk_register(chunks[c])
                    assert lres == ores and list(lshared) == oshared
                    osegs.append((O.KIND_CHUNK, key)); lsegs.append(M.Segment(0, cid))
                if ok:
                    q = int(rng.integers(0, 40))
                    osegs.append((O.KIND_PROMPT, q)); lsegs.append(M.Segment(1, q))
                    try:
                        ot = ost.build_block_table(rid, osegs)
                    except KeyError:
                        # a chunk registered earlier in this very request was reclaimed by a later registration
                        with pytest.raises(M.MepicError) as e:
                            st.build_block_table(rid, lsegs)
                        assert e.value.code == M.MEPIC_E_NOTFOUND
                        ot = None
                    except O.Reject:
                        with pytest.raises(M.MepicError) as e:
                            st.build_block_table(rid, lsegs)
                        assert e.value.code == M.MEPIC_E_NOSPACE
                        rejected += 1
                        ot = None
                    if ot is not None:
                        pages, base, kv_len, slots = st.build_block_table(rid, lsegs)
                        assert list(pages) == ot.page_ids and list(base) == ot.pos_base and kv_len == ot.kv_len
                        assert list(slots) == ot.recompute_slots
                        live.append(rid)
            assert st.stats() == ost.stats(), step
        s = st.stats()
        assert s["chunks_evicted"] > 10 and rejected >= 0 and s["pages_free"] + s["pages_shared_held"] + s["pages_private_held"] == 90


def test_identity_is_the_padded_sequence():
    with M.Store(_cfg(P=16, num_pages=40)) as st:
        a = st.chunk_register(np.arange(5, 25, dtype=np.int32))                        # 20 tokens -> 12 pads
        padded = np.concatenate([np.zeros(12, np.int32), np.arange(5, 25, dtype=np.int32)])
        b = st.chunk_register(padded)                                                  # already canonical
        assert b[0] == a[0] and b[1] and list(b[3]) == list(a[3]) and b[2] == 0
        c = st.chunk_register(np.arange(5, 26, dtype=np.int32))                        # different content
        assert c[0] != a[0] and not c[1]
        assert st.stats()["dedup_hits"] == 1 and st.stats()["chunks_resident"] == 2


def test_rope_table_matches_oracle_angles():
    cfg = _cfg(P=16, num_pages=4, head_dim=128, n_q_heads=8, n_kv_heads=2, max_position=70000, rope_theta=5e5)
    tab = M.mepic_rope_table_fill(cfg)
    assert tab.shape == (70001, 64, 2) and tab.dtype == np.float32
    for p in (0, 1, 15, 16, 4097, 65535, 70000):
        phi = O.rope_angles(np.int64(p), 128, 5e5)
        assert np.abs(tab[p, :, 0] - np.cos(phi)).max() <= 2.0 ** -24
        assert np.abs(tab[p, :, 1] - np.sin(phi)).max() <= 2.0 ** -24


def test_new_chunk_is_recomputed_whole_once_then_first_block_only():
    # Section 3.3.1 through the ABI and the oracle: tables identical; the marked chunk lists all its slots for the
    # first request that uses it (first occurrence only), and only its first block afterwards.
    P = 16
    rng = np.random.default_rng(31)
    A = rng.integers(1, 999, size=40, dtype=np.int32)      # 3 pages (8 leading pads)
    B = rng.integers(1, 999, size=64, dtype=np.int32)      # 4 pages
    ost = O.OracleStore(P, 64)
    with M.Store(_cfg(P=P, num_pages=64)) as st:
        ka, _, _ = ost.register_chunk(A); kb, _, _ = ost.register_chunk(B)
        ca, ra, _, _ = st.chunk_register(A); cb, rb, _, _ = st.chunk_register(B)
        assert not ra and not rb
        ost.mark_uncomputed(ka); st.chunk_mark_uncomputed(ca)
        o1 = ost.build_block_table(1, [(O.KIND_PROMPT, 5), (O.KIND_CHUNK, ka), (O.KIND_CHUNK, kb), (O.KIND_CHUNK, ka), (O.KIND_PROMPT, 3)])
        l1 = st.build_block_table(1, [M.Segment(1, 5), M.Segment(0, ca), M.Segment(0, cb), M.Segment(0, ca), M.Segment(1, 3)])
        assert list(l1[0]) == o1.page_ids and l1[2] == o1.kv_len and list(l1[3]) == o1.recompute_slots
        # prompt(5) -> slots 0..15; A whole -> 16..63; B first block -> 64..79; A again, first block -> 128..143; prompt(3)
        assert o1.recompute_slots == list(range(0, 16)) + list(range(16, 64)) + list(range(64, 80)) + list(range(128, 144)) + list(range(176, 179))
        o2 = ost.build_block_table(2, [(O.KIND_CHUNK, ka)])
        l2 = st.build_block_table(2, [M.Segment(0, ca)])
        assert list(l2[3]) == o2.recompute_slots == list(range(0, 16))
        with pytest.raises(M.MepicError) as e:
            st.chunk_mark_uncomputed(ca)                      # aliased by live requests
        assert e.value.code == M.MEPIC_E_EXISTS
        with pytest.raises(M.MepicError) as e:
            st.chunk_mark_uncomputed(ca + 77)
        assert e.value.code == M.MEPIC_E_NOTFOUND
        assert st.stats() == ost.stats()
