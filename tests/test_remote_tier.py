"""Remote tier behind the HBM pool (Algorithm 1 "resolve HBM residency and remote availability",
Section 3.2.3 eviction): evicted chunk KV is kept in host memory and copied back on the next use.

Checked three ways on serving traces over a pool too small for every chunk:
  * against the oracle store, which mirrors the tier with copies of page arrays: tables, residency
    answers (0 new / 1 resident / 2 brought back), every counter, and the pools bit for bit;
  * against a pin that does not involve the oracle: a new chunk's pages are filled with a pattern
    that is a function of the chunk and the block only, and after every call each resident chunk's
    pages must still hold exactly that pattern - whichever pages it was given and however often it
    went out to the tier and came back;
  * brought-back chunks are not recomputed (only their first block is, per request).
The host-pool mode (plain memcpy) runs without a GPU; the device mode runs the same trace on
device pools with the copies enqueued on a stream.
"""
import numpy as np
import pytest

import paper_2512_16822_b200 as M
from oracle import mepic_oracle as O

P, HKV, D = 16, 2, 64


def _pattern(chunk_index: int, block: int, which: int) -> np.ndarray:
    """bf16 bit patterns of one page [HKV, P, D] of chunk `chunk_index`, shareable block `block`; which: 0 K, 1 V."""
    rng = np.random.default_rng([7, chunk_index, block, which])
    return rng.integers(0, 0x7F00, size=(HKV, P, D), dtype=np.uint16)


def _trace(st, ost, kp, vp, okp, ovp, after_call, steps=400, n_chunks=14, seed=0):
    """Drive the library store `st` and the oracle store `ost` with the same calls; `kp/vp` are the library's pools
    as numpy views the test may write (new chunks) and read, `okp/ovp` the oracle's."""
    rng = np.random.default_rng(seed)
    lens = rng.integers(2 * P, 6 * P + 1, size=n_chunks)
    chunks = [rng.integers(1, 32000, size=int(n)).astype(np.int32) for n in lens]
    live, resident = {}, {}                 # request id -> chunk indices ; chunk index -> shared pages
    next_id = 0
    seen = {0: 0, 1: 0, 2: 0}
    for step in range(steps):
        if live and (rng.random() < 0.45 or len(live) >= 3):
            rid = int(rng.choice(list(live)))
            st.request_release(rid); ost.release(rid)
            del live[rid]
        else:
            picks = [int(c) for c in rng.choice(n_chunks, size=int(rng.integers(1, 4)), replace=False)]
            segs, osegs, ok = [], [], True
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
                if res == 0:                 # a new chunk: "compute" its shareable pages (both sides hold the same bits)
                    for blk, pg in enumerate(pages):
                        kp[pg] = _pattern(c, blk, 0); vp[pg] = _pattern(c, blk, 1)
                        okp[pg] = _pattern(c, blk, 0); ovp[pg] = _pattern(c, blk, 1)
                after_call()
                resident[c] = list(pages)
                segs.append(M.Segment(M.MEPIC_SEG_CHUNK, cid)); osegs.append((O.KIND_CHUNK, okey))
            if ok:
                q = int(rng.integers(1, 40))
                segs.append(M.Segment(M.MEPIC_SEG_PROMPT, q)); osegs.append((O.KIND_PROMPT, q))
                try:
                    pages, base, kvl, slots = st.build_block_table(next_id, segs)
                    ot = ost.build_block_table(next_id, osegs)
                    assert list(pages) == ot.page_ids and list(base) == ot.pos_base and kvl == ot.kv_len
                    # a chunk that came back from the tier is a cached chunk: first block only
                    assert list(slots) == ot.recompute_slots
                    live[next_id] = picks
                except M.MepicError as e:
                    assert e.code in (M.MEPIC_E_NOSPACE, M.MEPIC_E_NOTFOUND)
                    with pytest.raises((O.Reject, KeyError)):
                        ost.build_block_table(next_id, osegs)
                next_id += 1
        after_call()
        assert st.stats() == ost.stats(), step
        # which chunks are resident now, and do their pages still hold their own K/V?
        for c in list(resident):
            try:
                key = ost.canonical_chunk(chunks[c])
            except Exception:
                key = None
            if key not in ost.chunks:
                del resident[c]
                continue
            assert ost.chunks[key]["shared"] == resident[c]
            for blk, pg in enumerate(resident[c]):
                assert np.array_equal(kp[pg], _pattern(c, blk, 0)) and np.array_equal(vp[pg], _pattern(c, blk, 1)), (step, c, blk)
    return seen


def _stores(num_pages, remote_pages, kp, vp, okp, ovp, stream=None):
    cfg = M.Config(P, 4, HKV, D, num_pages, 1024, 1e4)
    st = M.Store(cfg)
    st.attach_remote(kp, vp, remote_pages, stream)
    ost = O.OracleStore(P, num_pages)
    ost.attach_remote(okp, ovp, remote_pages)
    return st, ost


@pytest.mark.parametrize("num_pages,remote_pages,seed", [(26, 40, 0), (26, 9, 1), (34, 200, 2)])
def test_trace_with_host_pools(num_pages, remote_pages, seed):
    shape = (num_pages, HKV, P, D)
    kp, vp, okp, ovp = (np.zeros(shape, dtype=np.uint16) for _ in range(4))
    st, ost = _stores(num_pages, remote_pages, kp, vp, okp, ovp)
    with st:
        def same_pools():
            assert np.array_equal(kp, okp) and np.array_equal(vp, ovp)
        seen = _trace(st, ost, kp, vp, okp, ovp, same_pools, seed=seed)
        s = st.stats()
    assert seen[2] > 5 and seen[1] > 5 and seen[0] > 5, seen          # all three residency answers occur
    assert s["chunks_spilled"] > 5 and s["chunks_fetched"] == seen[2]
    if remote_pages == 9:
        assert s["remote_pages"] <= 9                                   # the small tier had to drop chunks of its own


def test_attach_errors_and_no_tier_means_old_behaviour():
    cfg = M.Config(P, 4, HKV, D, 8, 1024, 1e4)
    pool = np.zeros((8, HKV, P, D), dtype=np.uint16)
    with M.Store(cfg) as st:
        with pytest.raises(M.MepicError) as e:
            st.attach_remote(pool, pool.copy(), 0)
        assert e.value.code == M.MEPIC_E_INVAL
        st.attach_remote(pool, pool.copy(), 4)
        with pytest.raises(M.MepicError) as e:
            st.attach_remote(pool, pool.copy(), 4)
        assert e.value.code == M.MEPIC_E_EXISTS
    with M.Store(cfg) as st:                                            # no tier: an evicted chunk comes back as new
        a = np.arange(1, 5 * P + 1, dtype=np.int32); b = a + 1000
        assert st.chunk_register(a)[1] == 0
        assert st.chunk_register(b)[1] == 0                              # 4 + 4 shared pages: the pool is full
        c = a + 2000
        assert st.chunk_register(c)[1] == 0 and st.stats()["chunks_evicted"] == 1
        assert st.chunk_register(a)[1] == 0 and st.stats()["chunks_spilled"] == 0


def test_uncomputed_chunks_are_not_kept():
    cfg = M.Config(P, 4, HKV, D, 8, 1024, 1e4)
    kp = np.zeros((8, HKV, P, D), dtype=np.uint16); vp = kp.copy()
    with M.Store(cfg) as st:
        st.attach_remote(kp, vp, 16)
        a = np.arange(1, 5 * P + 1, dtype=np.int32); b = a + 1000; c = a + 2000
        ida = st.chunk_register(a)[0]
        st.chunk_mark_uncomputed(ida)                                   # nobody has computed a's K/V
        st.chunk_register(b)
        st.chunk_register(c)                                            # evicts a (least recently used)
        s = st.stats()
        assert s["chunks_evicted"] == 1 and s["chunks_spilled"] == 0
        assert st.chunk_register(a)[1] == 0                             # a is new again, not "brought back"
        assert st.stats()["chunks_spilled"] == 1                        # ... and that eviction (of b, computed) was kept


@pytest.mark.gpu
def test_trace_with_device_pools():
    import torch
    from paper_2512_16822_b200.build import build_library
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    num_pages, remote_pages = 26, 40
    shape = (num_pages, HKV, P, D)
    dk = torch.zeros(shape, dtype=torch.int16, device="cuda"); dv = torch.zeros_like(dk)
    okp, ovp = np.zeros(shape, dtype=np.uint16), np.zeros(shape, dtype=np.uint16)
    stream = torch.cuda.Stream()
    st, ost = _stores(num_pages, remote_pages, dk, dv, okp, ovp, stream)

    class DevicePool:                      # numpy-like access for the trace: writes and reads go through the tier's stream
        def __init__(self, t): self.t = t
        def __setitem__(self, pg, bits):
            with torch.cuda.stream(stream):
                self.t[pg].copy_(torch.from_numpy(bits.view(np.int16)), non_blocking=False)
        def __getitem__(self, pg):
            stream.synchronize()
            return self.t[pg].cpu().numpy().view(np.uint16)

    kp, vp = DevicePool(dk), DevicePool(dv)
    with st:
        def same_pools():
            stream.synchronize()
            assert np.array_equal(dk.cpu().numpy().view(np.uint16), okp) and np.array_equal(dv.cpu().numpy().view(np.uint16), ovp)
        seen = _trace(st, ost, kp, vp, okp, ovp, same_pools, steps=150, seed=3)
        stream.synchronize()
    assert seen[2] > 2
