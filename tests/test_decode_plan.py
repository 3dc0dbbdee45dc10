"""Host planner of the grouped decode: invariants every plan must satisfy (no GPU).

The plan has no counterpart in the paper; what is fixed is that it only REGROUPS the block
tables.  So the tests read the plan back and check, against the tables themselves: every
(request, entry) is covered exactly once with its own page id and position base; the requests of
a group really alias each page they are grouped on; partly filled last pages stay with their
request; the line, its cut and the per-request index are consistent.
"""
from collections import Counter

import numpy as np
import pytest

import paper_2512_16822_b200 as M
from paper_2512_16822_b200 import runtime as RT
from mepic_inputs import make_workload

HEADER, ITEM_FIXED = 24, 5
MAGIC = 0x4d504c31


def _parse(plan, Hkv, P):
    h = plan[:HEADER]
    assert h[0] == MAGIC and h[13] == len(plan) and h[15] == P
    n_items, n_workers, piece, total, R = (int(x) for x in h[1:6])
    off_items, off_rec, off_work, off_req_off, off_req_items = (int(x) for x in h[6:11])
    batch, n_rec, off_req_ent = int(h[11]), int(h[12]), int(h[14])
    items = plan[off_items:off_items + n_items * (ITEM_FIXED + R)].reshape(n_items, ITEM_FIXED + R)
    recs = plan[off_rec:off_rec + n_rec * (1 + R)].reshape(n_rec, 1 + R)
    workers = plan[off_work:off_work + n_workers * 3].reshape(n_workers, 3)
    req_off = plan[off_req_off:off_req_off + batch + 1]
    req_items = plan[off_req_items:off_req_items + req_off[-1]]
    req_ent = plan[off_req_ent:off_req_ent + batch]
    off_slot_base, off_part_off, n_slots = int(h[16]), int(h[17]), int(h[18])
    assert int(h[19]) == Hkv
    slot_base = plan[off_slot_base:off_slot_base + n_items * Hkv * R].reshape(n_items, Hkv, R)
    part_off = plan[off_part_off:off_part_off + batch * Hkv + 1]
    assert part_off[0] == 0 and part_off[-1] == n_slots and (np.diff(part_off) >= 1).all()
    return dict(slot_base=slot_base, part_off=part_off, n_items=n_items, n_workers=n_workers, piece=piece, total=total, R=R, items=items, recs=recs,
                workers=workers, req_off=req_off, req_items=req_items, req_ent=req_ent, batch=batch)


def _check_plan(cfg, page_ids, pos_base, kv_len, n_sms=148, plan=None):
    P, Hkv = cfg.page_size, cfg.n_kv_heads
    G = cfg.n_q_heads // Hkv
    if plan is None:
        plan = M.mepic_decode_plan_build(cfg, page_ids, pos_base, kv_len, n_sms)
    pl = _parse(plan, Hkv, P)
    R, tpp = pl["R"], P // 16
    assert R == min(16 // G, 8) and pl["n_workers"] == n_sms * 8 and pl["batch"] == len(kv_len)
    n_ent = [-(-int(k) // P) for k in kv_len]
    assert list(pl["req_ent"]) == n_ent
    want = Counter((r, int(page_ids[r, e]), int(pos_base[r, e])) for r in range(len(kv_len)) for e in range(n_ent[r]))
    got = Counter()
    listed = Counter()
    tile_start = 0
    for i, it in enumerate(pl["items"]):
        n_req, rec_off, n_e, tail, ts = (int(x) for x in it[:ITEM_FIXED])
        reqs = [int(x) for x in it[ITEM_FIXED:ITEM_FIXED + n_req]]
        assert 1 <= n_req <= R and n_e >= 1 and ts == tile_start
        assert all(x == -1 for x in it[ITEM_FIXED + n_req:])
        tile_start += n_e * tpp
        for j, r in enumerate(reqs):
            listed[(r, i * 16 + j)] += 1
        for k in range(n_e):
            rec = pl["recs"][rec_off + k]
            for j, r in enumerate(reqs):
                got[(r, int(rec[0]), int(rec[1 + j]))] += 1
        if n_req > 1:
            assert tail == -1
        else:
            r = reqs[0]
            last_page_partial = kv_len[r] % P != 0
            if tail >= 0:
                assert tail == (n_ent[r] - 1) * P
                last = pl["recs"][rec_off + n_e - 1]
                assert int(last[0]) == page_ids[r, n_ent[r] - 1] and int(last[1]) == pos_base[r, n_ent[r] - 1]
            else:
                assert not last_page_partial or all(
                    (int(pl["recs"][rec_off + k][0]), int(pl["recs"][rec_off + k][1])) !=
                    (int(page_ids[r, n_ent[r] - 1]), int(pos_base[r, n_ent[r] - 1])) for k in range(n_e))
    assert got == want, "the plan does not cover the block tables exactly once"
    # a partly filled last page is never grouped: it must be the tail of some single-request item
    for r, k in enumerate(kv_len):
        if k % P:
            assert any(int(it[0]) == 1 and int(it[ITEM_FIXED]) == r and int(it[3]) == (n_ent[r] - 1) * P for it in pl["items"])
    # the line and its cut
    assert pl["total"] == tile_start * Hkv
    assert pl["piece"] == max(4, -(-pl["total"] // pl["n_workers"]))
    for w, (item, head, tile) in enumerate(pl["workers"]):
        x = w * pl["piece"]
        if x >= pl["total"]:
            assert item == pl["n_items"]
            continue
        it = pl["items"][item]
        nt = int(it[2]) * tpp
        assert 0 <= head < Hkv and 0 <= tile < nt and int(it[4]) * Hkv + head * nt + tile == x
    # partial slots: unit (item, head) overlaps pieces w_first..w_last; its rows' slots tile each (request, head) run exactly
    taken = np.zeros(int(pl["part_off"][-1]), dtype=np.int32)
    for i, it in enumerate(pl["items"]):
        nt = int(it[2]) * tpp
        for hd in range(Hkv):
            start = int(it[4]) * Hkv + hd * nt
            cnt = (start + nt - 1) // pl["piece"] - start // pl["piece"] + 1
            for j in range(int(it[0])):
                r = int(it[ITEM_FIXED + j]); s0 = int(pl["slot_base"][i, hd, j])
                assert pl["part_off"][r * Hkv + hd] <= s0 and s0 + cnt <= pl["part_off"][r * Hkv + hd + 1]
                taken[s0:s0 + cnt] += 1
    assert (taken == 1).all()
    # per-request index of (item, row)
    for r in range(len(kv_len)):
        mine = [int(v) for v in pl["req_items"][pl["req_off"][r]:pl["req_off"][r + 1]]]
        assert Counter(mine) == Counter(v for (rr, v), c in listed.items() if rr == r for _ in range(c))
    return pl


def _tables_of(idx, scale=1.0):
    wl = make_workload(idx, scale=scale)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    ids, base, kvl, _ = RT.pack_tables(tables, wl.page_size)
    return cfg, ids, base, kvl


@pytest.mark.parametrize("idx", [1, 2, 4, 5])
def test_plan_covers_the_tables_of_every_config(idx):
    cfg, ids, base, kvl = _tables_of(idx)
    pl = _check_plan(cfg, ids, base, kvl)
    # sharing must show: far fewer staged pages than table entries on the Zipf-shared configurations
    entries = sum(-(-int(k) // cfg.page_size) for k in kvl)
    if idx in (2, 4):
        assert len(pl["recs"]) * 2.5 < entries
    # pages read once per group: the records of an item never repeat a page
    for it in pl["items"]:
        pages = pl["recs"][int(it[1]):int(it[1]) + int(it[2]), 0]
        assert len(set(pages.tolist())) == len(pages)


def test_groups_really_alias_their_pages_and_sizes_follow_the_users():
    # 9 requests use page 100..103 (a "chunk"), 2 of them also share 200..201, everyone has private pages
    P, Hq, Hkv, D = 16, 8, 2, 64            # G = 4 -> R = 4
    B, stride = 9, 12
    ids = np.full((B, stride), -1, dtype=np.int32); base = np.zeros((B, stride), dtype=np.int32)
    kvl = np.zeros(B, dtype=np.int32)
    nxt = 0
    for r in range(B):
        row = [nxt, 100, 101, 102, 103]; nxt += 1
        if r in (2, 5):
            row += [nxt, 200, 201]; nxt += 1
        row += [nxt]; nxt += 1
        ids[r, :len(row)] = row
        base[r, :len(row)] = np.arange(len(row)) * P + 3 * r
        kvl[r] = len(row) * P - (5 if r % 2 else 0)          # odd requests end inside their last page
    cfg = M.Config(P, Hq, Hkv, D, 300, 4096, 1e4)
    pl = _check_plan(cfg, ids, base, kvl, n_sms=4)
    shared = [it for it in pl["items"] if it[0] > 1]
    sizes = sorted(int(it[0]) for it in shared)
    # 9 users of pages 100..103 -> groups of 4 + 4 (+ 1 left to its own item); 2 users of 200..201 -> one group of 2
    assert sizes == [2, 4, 4]
    for it in shared:
        pages = pl["recs"][int(it[1]):int(it[1]) + int(it[2]), 0].tolist()
        for r in it[ITEM_FIXED:ITEM_FIXED + int(it[0])]:
            assert set(pages) <= set(ids[int(r)].tolist())


def test_same_page_twice_in_one_request_and_unshared_layout():
    P = 16
    cfg = M.Config(P, 4, 1, 128, 64, 2048, 1e4)              # G = 4
    ids = np.array([[5, 6, 7, 5, 6, 9], [5, 6, 8, 10, 0, 0]], dtype=np.int32)
    base = np.array([[0, 16, 32, 48, 64, 80], [0, 16, 32, 48, 0, 0]], dtype=np.int32)
    kvl = np.array([96, 60], dtype=np.int32)
    pl = _check_plan(cfg, ids, base, kvl, n_sms=2)
    # pages 5 and 6 have three users (request 0 twice, request 1 once): one group of three rows
    assert sorted(int(it[0]) for it in pl["items"]) == [1, 1, 3]
    # nothing shared: one record per table entry, one item per request
    ids2 = np.arange(12, dtype=np.int32).reshape(2, 6); kvl2 = np.array([96, 81], dtype=np.int32)
    pl2 = _check_plan(cfg, ids2, np.tile(np.arange(6, dtype=np.int32) * P, (2, 1)), kvl2, n_sms=2)
    assert len(pl2["recs"]) == 12 and pl2["n_items"] == 2


@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (2, 1), (3, 1), (5, 1), (6, 1), (7, 1), (8, 1), (40, 8)])
def test_group_capacity_for_every_group_size(Hq, Hkv):
    P, B = 32, 11
    ids = np.tile(np.array([[50, 51, 52]], dtype=np.int32), (B, 1)); ids = np.concatenate([np.arange(B, dtype=np.int32)[:, None], ids], axis=1)
    base = np.tile(np.arange(4, dtype=np.int32) * P, (B, 1))
    kvl = np.full(B, 4 * P, dtype=np.int32)
    cfg = M.Config(P, Hq, Hkv, 64, 64, 1024, 1e4)
    pl = _check_plan(cfg, ids, base, kvl, n_sms=3)
    R = min(16 // (Hq // Hkv), 8)
    assert max(int(it[0]) for it in pl["items"]) == min(R, B)


def test_errors():
    cfg = M.Config(16, 8, 2, 64, 32, 1024, 1e4)
    ids = np.zeros((2, 4), dtype=np.int32); base = np.zeros((2, 4), dtype=np.int32)
    with pytest.raises(M.MepicError) as e:
        M.mepic_decode_plan_build(cfg, ids, base, np.array([16, 0], dtype=np.int32), 4)
    assert e.value.code == M.MEPIC_E_INVAL
    with pytest.raises(M.MepicError) as e:
        M.mepic_decode_plan_build(cfg, ids, base, np.array([16, 5 * 16], dtype=np.int32), 4)     # 5 entries > stride 4
    assert e.value.code == M.MEPIC_E_INVAL
    # a buffer that is too small: E_CAPACITY and the needed size
    import ctypes as C
    c = cfg.c(); out = np.empty(8, dtype=np.int32); used = C.c_size_t(0)
    kvl = np.array([64, 64], dtype=np.int32)
    rc = M.lib().mepic_decode_plan_build(C.byref(c), ids.ctypes.data, base.ctypes.data, kvl.ctypes.data, 2, 4, 4,
                                         out.ctypes.data, 8, C.byref(used))
    assert rc == M.MEPIC_E_CAPACITY and used.value == len(M.mepic_decode_plan_build(cfg, ids, base, kvl, 4))


def test_patched_plan_satisfies_every_invariant_of_a_fresh_one_step_after_step():
    """A decode loop: every request grows by one token per step, gaining a page now and then (some requests start on a
    full page, some in the middle of one).  After every step the plan is patched, not rebuilt, and must still cover
    the tables as they are now exactly once, keep the tail rule, the cut and the partial slots consistent; the ranges
    the patch reports are exactly where the buffer changed."""
    cfg, ids, base, kvl = _tables_of(2, scale=0.25)
    P = cfg.page_size
    B, stride0 = ids.shape
    grow = 40                                                           # tokens per request: 2-3 page gains each
    stride = stride0 + 4
    ids2 = np.zeros((B, stride), dtype=np.int32); base2 = np.zeros((B, stride), dtype=np.int32)
    ids2[:, :stride0] = ids; base2[:, :stride0] = base
    kvl = kvl.copy(); kvl[1] -= 5; kvl[2] -= P - 1                      # ragged starts
    cfg = M.Config(P, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.num_pages + 4 * B, cfg.max_position + 4 * P, cfg.rope_theta)
    plan = M.mepic_decode_plan_build(cfg, ids2, base2, kvl, 148)
    _check_plan(cfg, ids2, base2, kvl, plan=plan)
    next_page = cfg.num_pages - 4 * B
    gains = 0
    for step in range(grow):
        before = plan.copy()
        for r in range(B):
            if kvl[r] % P == 0:                                         # the last page is full: the new token opens a page
                e = kvl[r] // P
                ids2[r, e] = next_page; next_page += 1
                base2[r, e] = base2[r, e - 1] + P
                gains += 1
            kvl[r] += 1
        ranges = M.mepic_decode_plan_patch(cfg, plan, ids2, base2, kvl)
        changed = np.flatnonzero(plan != before)
        if len(changed):
            assert len(ranges) == 2
            covered = np.zeros(len(plan), dtype=bool)
            for lo, n in ranges:
                covered[lo:lo + n] = True
            assert covered[changed].all()
            assert ranges[0] == (0, int(plan[7])) and ranges[1][0] >= int(plan[7])     # the derived prefix, then records
        else:
            assert ranges == []
        _check_plan(cfg, ids2, base2, kvl, plan=plan)
    assert gains >= 2 * B
    # the patched plan stages the same pages as a plan built from scratch on the final tables
    fresh = _parse(M.mepic_decode_plan_build(cfg, ids2, base2, kvl, 148), cfg.n_kv_heads, P)
    mine = _parse(plan, cfg.n_kv_heads, P)
    assert mine["total"] == fresh["total"] and mine["piece"] == fresh["piece"]


def test_patch_refuses_what_it_cannot_do_and_changes_nothing_then():
    cfg, ids, base, kvl = _tables_of(1)
    P = cfg.page_size
    B, stride0 = ids.shape
    stride = stride0 + 40
    ids2 = np.zeros((B, stride), dtype=np.int32); base2 = np.zeros((B, stride), dtype=np.int32)
    ids2[:, :stride0] = ids; base2[:, :stride0] = base
    base2[:, stride0:] = (np.arange(stride0, stride) * P)[None, :]
    plan = M.mepic_decode_plan_build(cfg, ids2, base2, kvl, 148)
    keep = plan.copy()
    shrunk = kvl.copy(); shrunk[0] -= 2 * P
    with pytest.raises(M.MepicError) as e:
        M.mepic_decode_plan_patch(cfg, plan, ids2, base2, shrunk)
    assert e.value.code == M.MEPIC_E_INVAL and np.array_equal(plan, keep)
    far = kvl.copy(); far[1] += 17 * P                                  # more pages than the reserve of 16
    with pytest.raises(M.MepicError) as e:
        M.mepic_decode_plan_patch(cfg, plan, ids2, base2, far)
    assert e.value.code == M.MEPIC_E_CAPACITY and np.array_equal(plan, keep)
    ok = kvl.copy(); ok[1] += 16 * P                                    # exactly the reserve
    assert len(M.mepic_decode_plan_patch(cfg, plan, ids2, base2, ok)) == 2
    _check_plan(cfg, ids2, base2, ok, plan=plan)
