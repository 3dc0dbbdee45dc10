"""Grouped (sharing-aware) decode through the C ABI against the fp64 oracle, element by element.

The call must produce what mepic_attn_decode defines, so the oracle and the tolerance are the same:
max-abs <= 2e-2, mean-abs <= 2e-3, and the tighter internal bar relative L2 <= 1e-2.  Cases cover
groups of every size, requests that hold a page twice, position bases that differ per request and
jump between pages (the rotation is rebuilt there instead of advanced), partly filled last pages with
NaN bit patterns behind kv_len, page sizes above the tile, and every group size G.
"""
import numpy as np
import pytest
import torch

import paper_2512_16822_b200 as M
from paper_2512_16822_b200 import runtime as RT
from paper_2512_16822_b200.build import build_library
from mepic_inputs import make_workload, f32_to_bf16_bits, bf16_bits_to_f64
from oracle import mepic_oracle as O

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_L2 = 2e-2, 2e-3, 1e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"


def _check(got_bits, want, what=""):
    got = bf16_bits_to_f64(got_bits)
    d = np.abs(got - want)
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert np.isfinite(got).all(), what
    assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (what, d.max(), d.mean())
    assert rel <= REL_L2, (what, rel)


def _run(cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm_scale, theta, sample=None, also_plain=True):
    dev = RT.Device(cfg, kp, vp)
    gb = RT.GroupedDecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q)
    out = gb.run(sm_scale)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    got = RT.bf16_bits(out)
    P = cfg.page_size
    for b in (range(len(kv_len)) if sample is None else sample):
        n = -(-int(kv_len[b]) // P)
        want = O.decode_attention_one(q[b], kp, vp, list(page_ids[b, :n]), list(pos_base[b, :n]), int(kv_len[b]),
                                      int(q_pos[b]), sm_scale, theta)
        _check(got[b], want, f"request {b}")
    if also_plain:
        # the per-request kernel on the same inputs: same definition, so the two bf16 results sit within rounding
        pb = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q)
        ref = bf16_bits_to_f64(RT.bf16_bits(pb.run(sm_scale)))
        torch.cuda.synchronize()
        assert np.abs(bf16_bits_to_f64(got) - ref).max() <= max(6e-3, 2.0 ** -7 * np.abs(ref).max())     # two bf16 ulps
    return dev, gb


def _workload(idx, scale=1.0, sample=None):
    wl = make_workload(idx, scale=scale)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    _run(cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, wl.decode_q(), wl.sm_scale, wl.rope_theta, sample)


def test_config1_all_elements():
    _workload(1)


@pytest.mark.parametrize("idx,scale", [(2, 0.25), (4, 0.25), (5, 0.1)])
def test_scaled_configs_all_elements(idx, scale):
    _workload(idx, scale)


@pytest.mark.parametrize("idx,sample", [(2, [0, 13, 31]), (4, [0, 7]), (5, [0, 1, 64, 127])])
def test_full_size_configs_sampled_requests(idx, sample):
    _workload(idx, 1.0, sample)


def _shared_case(seed, *, Hq, Hkv, D, P, n_req, chunk_pages, uses, tail_tokens, jitter, theta=1e4, q_std=1.0):
    """Hand-built tables: every request = [private page, the shared pages of a chunk] per used chunk, then private
    tail pages holding ``tail_tokens[r]`` tokens.  ``uses[r]`` lists the chunks (repeats allowed) of request r."""
    rng = np.random.default_rng(seed)
    n_chunks = len(chunk_pages)
    total_shared = sum(chunk_pages)
    ents = [sum(1 + chunk_pages[c] for c in uses[r]) + -(-tail_tokens[r] // P) for r in range(n_req)]
    num_pages = total_shared + sum(ents) + 3
    perm = rng.permutation(num_pages).astype(np.int32)
    at = 0
    shared = []
    for c in range(n_chunks):
        shared.append(perm[at:at + chunk_pages[c]]); at += chunk_pages[c]
    stride = max(ents) + 1
    page_ids = np.full((n_req, stride), -7, dtype=np.int32); pos_base = np.zeros((n_req, stride), dtype=np.int32)
    kv_len = np.zeros(n_req, dtype=np.int32)
    for r in range(n_req):
        row = []
        for c in uses[r]:
            row.append(perm[at]); at += 1
            row.extend(shared[c].tolist())
        n_tail = -(-tail_tokens[r] // P)
        row.extend(perm[at:at + n_tail].tolist()); at += n_tail
        page_ids[r, :len(row)] = row
        b = np.arange(len(row)) * P + int(rng.integers(0, 200))
        if jitter:
            b = b + np.cumsum(rng.integers(0, 3, size=len(row)) * int(rng.integers(1, 50)))   # jumps at some pages
        pos_base[r, :len(row)] = b
        kv_len[r] = (len(row) - n_tail) * P + tail_tokens[r]
    last = kv_len - 1
    q_pos = (pos_base[np.arange(n_req), last // P] + last % P).astype(np.int32)
    cfg = M.Config(P, Hq, Hkv, D, num_pages, int(max(q_pos.max(), pos_base.max() + P)) + 1, theta)
    kp = f32_to_bf16_bits(rng.standard_normal((num_pages, Hkv, P, D)).astype(np.float32))
    vp = f32_to_bf16_bits(rng.standard_normal((num_pages, Hkv, P, D)).astype(np.float32))
    for r in range(n_req):                     # slots past kv_len hold NaN bit patterns: they must be ignored
        t = int(kv_len[r]) % P
        if t:
            pg = page_ids[r, -(-int(kv_len[r]) // P) - 1]
            kp[pg, :, t:, :] = 0x7FC0; vp[pg, :, t:, :] = 0x7FC0
    q = f32_to_bf16_bits((rng.standard_normal((n_req, Hq, D)) * q_std).astype(np.float32))
    return cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q


@pytest.mark.parametrize("Hq,Hkv,D,P", [(8, 2, 128, 16), (8, 2, 64, 16), (4, 4, 128, 16), (2, 1, 64, 32), (3, 1, 128, 16),
                                        (10, 2, 128, 16), (6, 1, 64, 16), (7, 1, 128, 64), (8, 1, 128, 16), (4, 1, 64, 64)])
def test_groups_of_every_size_and_shape(Hq, Hkv, D, P):
    n_req = 11
    uses = [[0, 1], [0], [1, 0], [0, 2], [2], [0, 1, 2], [1], [0], [0, 0], [2, 1], [0]]      # request 8 holds chunk 0 twice
    tails = [5, 16, 1, P + 3, 17, 2 * P, 9, 33, 7, 16, P]
    args = _shared_case(100 + Hq + D + P, Hq=Hq, Hkv=Hkv, D=D, P=P, n_req=n_req, chunk_pages=[9, 5, 3], uses=uses,
                        tail_tokens=tails, jitter=False)
    _run(*args, 1.0 / np.sqrt(D), 1e4)


def test_position_bases_that_jump_and_differ_per_request():
    uses = [[0, 1, 2, 3], [3, 2, 1, 0], [0, 2], [1, 3], [0, 1, 2, 3], [2], [3, 0]]
    args = _shared_case(7, Hq=8, Hkv=2, D=128, P=16, n_req=7, chunk_pages=[31, 31, 12, 7], uses=uses,
                        tail_tokens=[64, 3, 20, 16, 40, 1, 15], jitter=True, theta=5e5)
    _run(*args, 0.11, 5e5)


def test_long_runs_keep_the_advanced_rotation_accurate():
    # one chunk of 400 pages shared by 5 requests: 400 consecutive 16-position steps of the query rotation
    uses = [[0]] * 5
    args = _shared_case(9, Hq=8, Hkv=2, D=128, P=16, n_req=5, chunk_pages=[400], uses=uses,
                        tail_tokens=[30, 2, 16, 7, 40], jitter=False, theta=5e5, q_std=3.0)
    _run(*args, 1.0 / np.sqrt(128), 5e5)


def test_query_position_before_the_context():
    # q_pos is an input: the rotation angle may be negative for every page
    cfg, kp, vp, ids, base, kvl, q_pos, q = _shared_case(11, Hq=8, Hkv=2, D=64, P=16, n_req=4, chunk_pages=[6, 4],
                                                         uses=[[0, 1], [1, 0], [0], [1]], tail_tokens=[9, 16, 3, 20], jitter=False)
    _run(cfg, kp, vp, ids, base, kvl, (q_pos // 3).astype(np.int32), q, 0.125, 1e4)


def test_stale_plan_sets_the_status_bit_without_faulting():
    cfg, kp, vp, ids, base, kvl, q_pos, q = _shared_case(13, Hq=8, Hkv=2, D=64, P=16, n_req=3, chunk_pages=[4],
                                                         uses=[[0], [0], [0]], tail_tokens=[16, 5, 9], jitter=False)
    dev = RT.Device(cfg, kp, vp)
    gb = RT.GroupedDecodeBatch(dev, ids, base, kvl, q_pos, q)
    # growing inside the last page keeps the plan valid ...
    gb.kv_len[1] += 3
    gb.run(0.125); torch.cuda.synchronize()
    assert dev.read_status() == 0
    # ... gaining a page does not: request 0 filled its last page and now needs another entry
    gb.kv_len[0] += 1
    gb.run(0.125); torch.cuda.synchronize()
    assert dev.read_status() & M.MEPIC_DEV_BAD_PLAN
    dev.status.zero_()


def test_argument_errors():
    cfg, kp, vp, ids, base, kvl, q_pos, q = _shared_case(15, Hq=8, Hkv=2, D=64, P=16, n_req=2, chunk_pages=[2],
                                                         uses=[[0], [0]], tail_tokens=[4, 4], jitter=False)
    dev = RT.Device(cfg, kp, vp)
    gb = RT.GroupedDecodeBatch(dev, ids, base, kvl, q_pos, q)
    other = M.Config(cfg.page_size, 16, 2, 64, cfg.num_pages, cfg.max_position, cfg.rope_theta)     # G = 8: R differs
    with pytest.raises(M.MepicError) as e:
        M.mepic_attn_decode_grouped(other, q=gb.q, k_pool=dev.k_pool, v_pool=dev.v_pool, plan=gb.plan, plan_host=gb.plan_host,
                                    kv_len=gb.kv_len, q_pos=gb.q_pos, rope_table=dev.rope, out=gb.out, workspace=gb.workspace,
                                    workspace_bytes=gb.ws_bytes, status=dev.status, batch=2, sm_scale=1.0)
    assert e.value.code == M.MEPIC_E_INVAL
    with pytest.raises(M.MepicError) as e:
        M.mepic_attn_decode_grouped(cfg, q=gb.q, k_pool=dev.k_pool, v_pool=dev.v_pool, plan=gb.plan, plan_host=gb.plan_host,
                                    kv_len=gb.kv_len, q_pos=gb.q_pos, rope_table=dev.rope, out=gb.out, workspace=gb.workspace,
                                    workspace_bytes=gb.ws_bytes - 16, status=dev.status, batch=2, sm_scale=1.0)
    assert e.value.code == M.MEPIC_E_INVAL


def test_more_than_32_requests():
    n_req = 70
    rng = np.random.default_rng(5)
    uses = [sorted(rng.choice(6, size=int(rng.integers(1, 4)), replace=False).tolist()) for _ in range(n_req)]
    tails = [int(x) for x in rng.integers(1, 50, size=n_req)]
    args = _shared_case(55, Hq=8, Hkv=2, D=128, P=16, n_req=n_req, chunk_pages=[7, 5, 9, 3, 4, 6], uses=uses,
                        tail_tokens=tails, jitter=False)
    _run(*args, 1.0 / np.sqrt(128), 1e4, sample=list(range(0, n_req, 7)))


def test_one_dominant_key_inside_a_shared_chunk():
    # A key ~80 nats above all others sits in a page three requests alias: every request's running maximum jumps when
    # that page is reached, whatever was accumulated before scales to nothing, and the output is that key's V row.
    # The big components sit in the slowest-rotating pair (63, 127 at D = 128): the score barely depends on positions.
    cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q = _shared_case(
        23, Hq=8, Hkv=2, D=128, P=16, n_req=4, chunk_pages=[20, 12], uses=[[1, 0], [0], [1, 0, 1], [1]],
        tail_tokens=[40, 7, 100, 300], jitter=False)
    big = f32_to_bf16_bits(np.array([30.0], dtype=np.float32))[0]
    q[:, :, 63] = big
    # chunk 0's shared pages follow a private page in every request that uses it; take its 10th shared page, slot 5
    r0 = 1
    page = page_ids[r0, 1 + 9]
    kp[page, :, 5, 63] = big
    dev, gb = _run(cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, 1.0 / np.sqrt(128), 1e4)
    got = bf16_bits_to_f64(RT.bf16_bits(gb.out))
    v_star = np.repeat(bf16_bits_to_f64(vp[page, :, 5, :]), 4, axis=0)
    for r in (0, 1, 2):                                   # the requests that alias chunk 0; request 3 does not
        assert (page_ids[r] == page).any()
        assert np.abs(got[r] - v_star).max() <= 2e-2, r
    assert not (page_ids[3] == page).any()


def test_plan_patched_through_a_decode_loop_stays_parity_green():
    """A serving loop: every request grows by one token per step and gains a page now and then.  The plan is built once
    and patched (mepic_decode_plan_patch: only the changed stretches are uploaded); after every page gain, and on some
    steps in between, the grouped result is compared with the fp64 oracle on the tables as they are then."""
    P, Hq, Hkv, D = 16, 8, 2, 128
    cfg, kp, vp, ids, base, kvl, q_pos, q = _shared_case(61, Hq=Hq, Hkv=Hkv, D=D, P=P, n_req=5, chunk_pages=[6, 4, 5],
                                                         uses=[[0, 1], [1, 0], [2], [0, 2, 1], [1]], tail_tokens=[16, 5, 32, 9, 1], jitter=False)
    rng = np.random.default_rng(62)
    B, stride0 = ids.shape
    steps, spare_per_req = 37, 4
    # the tokens to come: their K/V is already in the pool (random numbers instead of the NaN poison), in pages nobody uses yet
    for pool in (kp, vp):
        bad = pool == 0x7FC0
        pool[bad] = f32_to_bf16_bits(rng.standard_normal(int(bad.sum())).astype(np.float32))
    n0 = cfg.num_pages
    extra = lambda: f32_to_bf16_bits(rng.standard_normal((B * spare_per_req, Hkv, P, D)).astype(np.float32))
    kp, vp = np.concatenate([kp, extra()]), np.concatenate([vp, extra()])
    cfg = M.Config(P, Hq, Hkv, D, n0 + B * spare_per_req, cfg.max_position + (spare_per_req + 1) * P, 1e4)
    stride = stride0 + spare_per_req
    ids2 = np.zeros((B, stride), dtype=np.int32); base2 = np.zeros((B, stride), dtype=np.int32)
    ids2[:, :stride0] = np.maximum(ids, 0); base2[:, :stride0] = base
    dev = RT.Device(cfg, kp, vp)
    gb = RT.GroupedDecodeBatch(dev, ids2, base2, kvl, q_pos, q)
    kvl = kvl.copy()
    next_page, gains, uploaded = n0, 0, 0
    for step in range(steps):
        gained = False
        for r in range(B):
            if kvl[r] % P == 0:
                e = kvl[r] // P
                ids2[r, e] = next_page; next_page += 1
                base2[r, e] = base2[r, e - 1] + P
                gained = True; gains += 1
            kvl[r] += 1
        last = kvl - 1
        q_pos = (base2[np.arange(B), last // P] + last % P).astype(np.int32)
        if gained:
            uploaded += gb.patch(ids2, base2, kvl)
        gb.kv_len.copy_(torch.from_numpy(kvl)); gb.q_pos.copy_(torch.from_numpy(q_pos))
        out = gb.run(0.09); torch.cuda.synchronize()
        assert dev.read_status() == 0, step
        if gained or step % 7 == 0:
            got = RT.bf16_bits(out)
            for r in range(B):
                ne = -(-int(kvl[r]) // P)
                want = O.decode_attention_one(q[r], kp, vp, list(ids2[r, :ne]), list(base2[r, :ne]), int(kvl[r]), int(q_pos[r]), 0.09, 1e4)
                _check(got[r], want, f"step {step} request {r}")
    assert gains >= 2 * B and 0 < uploaded < gains * 4 * len(gb.plan_host)      # patches were made, and they were partial uploads
