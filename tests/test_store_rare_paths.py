"""Rare paths of the host store, reached through its fault-injection hook (no GPU involved).

  * Hash collisions.  Chunk identity is the padded token sequence (Section 3.2.3); the hash only finds it.  With
    the hash cut to two bits every chunk collides with others, ids are handed out by probing, and reclaiming a
    chunk that others were probed past must not hide them: a resident chunk is always found again (one resident
    copy per content), whatever was evicted before it in its chain.  Tables, residency answers and counters are
    compared with the oracle store, which keys on the token tuple itself and has no hash at all.
  * A copy to or from the remote tier that cannot be made.  The call reports MEPIC_E_CUDA and leaves a state in
    which nothing claims K/V it does not hold: a failed spill leaves no record in the tier, a failed fetch
    registers nothing and returns its pages to the head of the free list.
"""
import numpy as np
import pytest

import paper_2512_16822_b200 as M
from oracle import mepic_oracle as O

P = 16


def _cfg(num_pages):
    return M.Config(P, 4, 2, 64, num_pages, 4096, 1e4)


def test_colliding_chunks_stay_one_copy_per_content_across_evictions():
    rng = np.random.default_rng(3)
    chunks = [rng.integers(1, 32000, size=3 * P).astype(np.int32) for _ in range(12)]     # 2 shared pages each
    with M.Store(_cfg(12)) as st:
        M.mepic_store_test_hooks(st.handle, hash_mask=0x3)
        ost = O.OracleStore(P, 12)
        ids = {}
        for step in range(600):
            c = int(rng.integers(0, len(chunks)))
            try:
                cid, res, _, pages = st.chunk_register(chunks[c])
            except M.MepicError as e:
                assert e.code == M.MEPIC_E_NOSPACE
                with pytest.raises(O.Reject):
                    ost.register_chunk(chunks[c])
                continue
            _, ores, opages = ost.register_chunk(chunks[c])
            assert res == ores and list(pages) == opages, (step, c)
            # an id names one content for as long as the chunk is resident, and two resident contents never share one
            if res == 1:
                assert ids[c] == cid, (step, c)
            ids[c] = cid
            live = {k: v for k, v in ids.items() if ost.canonical_chunk(chunks[k]) in ost.chunks}
            assert len(set(live.values())) == len(live)
            assert st.stats() == ost.stats(), step
        assert st.stats()["chunks_evicted"] > 50 and st.stats()["dedup_hits"] > 50


def test_evicting_the_head_of_a_probe_chain_keeps_its_successor_findable():
    """The smallest case, by hand: A and B collide (mask 0: every id starts at 0), A is registered first (id 0), B is
    probed past it (id 1).  A is reclaimed for room; B must still be found as resident, not registered a second time."""
    rng = np.random.default_rng(4)
    A, B, Cc = (rng.integers(1, 32000, size=3 * P).astype(np.int32) for _ in range(3))
    with M.Store(_cfg(5)) as st:
        M.mepic_store_test_hooks(st.handle, hash_mask=0x0)
        ida, ra, _, pa = st.chunk_register(A)
        idb, rb, _, pb = st.chunk_register(B)
        assert (ida, idb, ra, rb) == (0, 1, 0, 0) and list(pa) == [0, 1] and list(pb) == [2, 3]
        # B in use, A idle: a third chunk needs 2 pages, 1 is free -> A (the only idle chunk) is reclaimed
        st.build_block_table(7, [M.Segment(M.MEPIC_SEG_CHUNK, idb)])
        idc, rc, _, pc = st.chunk_register(Cc)
        assert rc == 0 and st.stats()["chunks_evicted"] == 1
        idb2, rb2, _, pb2 = st.chunk_register(B)
        assert (idb2, rb2, list(pb2)) == (idb, 1, [2, 3])
        assert st.stats()["chunks_resident"] == 2
        assert idc == 0                      # the freed head of the chain is the new chunk's id; B keeps id 1


def _pools(n):
    return np.zeros((n, 2, P, 64), dtype=np.uint16), np.zeros((n, 2, P, 64), dtype=np.uint16)


def test_failed_spill_leaves_no_record_in_the_tier():
    rng = np.random.default_rng(5)
    A, B = (rng.integers(1, 32000, size=3 * P).astype(np.int32) for _ in range(2))
    kp, vp = _pools(3)
    with M.Store(_cfg(3)) as st:
        st.attach_remote(kp, vp, 8)
        st.chunk_register(A)
        M.mepic_store_test_hooks(st.handle, fail_copies=1)
        with pytest.raises(M.MepicError) as e:
            st.chunk_register(B)             # needs A's pages: A is spilled first, and that copy fails
        assert e.value.code == M.MEPIC_E_CUDA
        s = st.stats()
        assert s["remote_chunks"] == 0 and s["remote_pages"] == 0 and s["chunks_spilled"] == 0
        assert s["chunks_resident"] == 0 and s["pages_free"] == 3 and s["pages_shared_held"] == 0
        # the store works on: B registers as new, A comes back as new (the tier never held it)
        _, rb, _, _ = st.chunk_register(B)
        assert rb == 0
        st2 = st.stats()
        assert st2["chunks_resident"] == 1 and st2["pages_free"] == 1


def test_failed_fetch_registers_nothing_and_returns_the_pages_in_order():
    rng = np.random.default_rng(6)
    A, B = (rng.integers(1, 32000, size=3 * P).astype(np.int32) for _ in range(2))
    kp, vp = _pools(3)
    with M.Store(_cfg(3)) as st:
        st.attach_remote(kp, vp, 8)
        _, _, _, pa = st.chunk_register(A)
        kp[pa[0]] = 0x1234; vp[pa[1]] = 0x4321
        st.chunk_register(B)                 # A goes to the tier
        assert st.stats()["remote_chunks"] == 1
        kp[:] = 0; vp[:] = 0
        M.mepic_store_test_hooks(st.handle, fail_copies=1)
        with pytest.raises(M.MepicError) as e:
            st.chunk_register(A)             # B is spilled for room (that copy is the one that fails)
        assert e.value.code == M.MEPIC_E_CUDA
        M.mepic_store_test_hooks(st.handle, fail_copies=3)       # now the fetch itself fails part of the way
        before = st.stats()
        with pytest.raises(M.MepicError) as e:
            st.chunk_register(A)
        assert e.value.code == M.MEPIC_E_CUDA
        after = st.stats()
        assert after["chunks_resident"] == 0 and after["pages_free"] == before["pages_free"] == 3
        assert after["chunks_fetched"] == 0 and after["remote_chunks"] == 1
        M.mepic_store_test_hooks(st.handle, fail_copies=0)
        _, ra, _, pa2 = st.chunk_register(A)                       # and with copies working it comes back whole
        assert ra == 2 and (kp[pa2[0]] == 0x1234).all() and (vp[pa2[1]] == 0x4321).all()
        # the queue was [1, 0, 2] before the failed try (page 1 left over, then B's pages 0 and 2 in ascending order);
        # the failed try put its two pages back at the head in their order, so the retry gets what a first try would
        assert list(pa2) == [1, 0]
