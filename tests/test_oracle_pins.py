"""Pins for the CPU oracle: closed forms, invariants, library special cases, brute force.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong
sign or index, transposed operand, wrong head mapping) fails at least one.
None of these tests touches the CUDA library.
"""
import math
import os

import numpy as np
import pytest
import torch

from mepic_inputs import f32_to_bf16_bits, bf16_bits_to_f64, make_workload, make_custom
from oracle import mepic_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(rng, shape, std=1.0):
    return f32_to_bf16_bits((rng.standard_normal(shape) * std).astype(np.float32))


# ---------------------------------------------------------------- RoPE closed forms
def test_rope_is_orthogonal_and_additive():
    rng = np.random.default_rng(1)
    D, theta = 16, 1e4
    x = rng.standard_normal((5, D))
    for p in (0, 1, 7, 1234, 65535):
        y = O.rope_rotate(x, np.int64(p), theta)
        assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=0, atol=1e-12)
    # R(p) as a matrix: columns = images of basis vectors; R^T R = I; R(0) = I
    eye = np.eye(D)
    R = lambda p: O.rope_rotate(eye, np.int64(p), theta).T
    assert np.allclose(R(0), eye, atol=0)
    for a, b in ((3, 5), (100, 23), (4096, 8191)):
        assert np.allclose(R(a).T @ R(a), eye, atol=1e-12)
        assert np.allclose(R(a) @ R(b), R(a + b), atol=1e-10)


def test_rope_matches_complex_exponential_form():
    # Independent formulation: (x_i + j x_{i+D/2}) * exp(j * pos * theta^(-2i/D)).
    rng = np.random.default_rng(2)
    D, theta = 64, 5e5
    x = rng.standard_normal((7, D))
    pos = np.array([0, 1, 2, 17, 300, 8255, 65535])
    z = (x[:, :D // 2] + 1j * x[:, D // 2:]) * np.exp(
        1j * pos[:, None] * np.array([theta ** (-(2.0 * i) / D) for i in range(D // 2)])[None, :])
    want = np.concatenate([z.real, z.imag], axis=-1)
    got = O.rope_rotate(x, pos, theta)
    assert np.allclose(got, want, atol=1e-9)


def test_rope_first_pair_rotates_by_pos_radians():
    # i = 0 has inverse frequency 1: a unit vector on lane 0 at position p maps to (cos p, sin p).
    D = 8
    x = np.zeros(D); x[0] = 1.0
    y = O.rope_rotate(x, np.int64(3), 1e4)
    assert abs(y[0] - math.cos(3.0)) < 1e-15 and abs(y[D // 2] - math.sin(3.0)) < 1e-15
    # last pair has inverse frequency theta^(-(D-2)/D)
    x = np.zeros(D); x[D // 2 - 1] = 1.0
    y = O.rope_rotate(x, np.int64(5), 1e4)
    ang = 5.0 * 1e4 ** (-(D - 2) / D)
    assert abs(y[D // 2 - 1] - math.cos(ang)) < 1e-15 and abs(y[D - 1] - math.sin(ang)) < 1e-15


# ---------------------------------------------------------------- attention invariants
def _tiny_problem(seed=0, Hq=4, Hkv=2, D=8, P=4, n_pages=12, E=5, kv_len=18):
    rng = np.random.default_rng(seed)
    k_pool = _bits(rng, (n_pages, Hkv, P, D))
    v_pool = _bits(rng, (n_pages, Hkv, P, D))
    page_ids = list(rng.permutation(n_pages)[:E])
    pos_base = [e * P for e in range(E)]
    q = _bits(rng, (Hq, D))
    return q, k_pool, v_pool, page_ids, pos_base, kv_len


def test_relative_position_shift_invariance():
    q, kp, vp, ids, base, L = _tiny_problem(3)
    a = O.decode_attention_one(q, kp, vp, ids, base, L, base[-1] + 1, 0.35, 1e4)
    for shift in (1, 37, 4096):
        b = O.decode_attention_one(q, kp, vp, ids, [x + shift for x in base], L, base[-1] + 1 + shift, 0.35, 1e4)
        assert np.abs(a - b).max() < 1e-9
    # ...but moving only the keys (not q) must change the result
    c = O.decode_attention_one(q, kp, vp, ids, [x + 5 for x in base], L, base[-1] + 1, 0.35, 1e4)
    assert np.abs(a - c).max() > 1e-4


def test_equals_attention_over_contiguous_prerotated_k():
    # Build the standard pipeline by hand: contiguous K rotated BEFORE "caching", no page table.
    q, kp, vp, ids, base, L = _tiny_problem(4)
    theta, scale, q_pos = 1e4, 0.5, 23
    P, D = kp.shape[2], kp.shape[3]
    Kc = np.concatenate([bf16_bits_to_f64(kp[p]).transpose(1, 0, 2) for p in ids])[:L]   # [L, Hkv, D]
    Vc = np.concatenate([bf16_bits_to_f64(vp[p]).transpose(1, 0, 2) for p in ids])[:L]
    inv = np.array([theta ** (-(2.0 * i) / D) for i in range(D // 2)])
    def rot(x, p):
        zc = (x[..., :D // 2] + 1j * x[..., D // 2:]) * np.exp(1j * p * inv)
        return np.concatenate([zc.real, zc.imag], -1)
    Kr = np.stack([rot(Kc[t], base[t // P] + t % P) for t in range(L)])
    qf = rot(bf16_bits_to_f64(q), q_pos)
    want = np.zeros_like(qf)
    G = q.shape[0] // kp.shape[1]
    for h in range(q.shape[0]):
        s = np.array([scale * float(np.dot(qf[h], Kr[t, h // G])) for t in range(L)])
        w = np.exp(s - s.max()); w /= w.sum()
        want[h] = sum(w[t] * Vc[t, h // G] for t in range(L))
    got = O.decode_attention_one(q, kp, vp, ids, base, L, q_pos, scale, theta)
    assert np.abs(got - want).max() < 1e-12


def test_physical_page_permutation_leaves_output_unchanged():
    q, kp, vp, ids, base, L = _tiny_problem(5)
    a = O.decode_attention_one(q, kp, vp, ids, base, L, 19, 0.4, 1e4)
    perm = np.random.default_rng(9).permutation(kp.shape[0])      # new_id = perm[old_id]
    kp2 = np.empty_like(kp); vp2 = np.empty_like(vp)
    kp2[perm] = kp; vp2[perm] = vp
    b = O.decode_attention_one(q, kp2, vp2, [int(perm[p]) for p in ids], base, L, 19, 0.4, 1e4)
    assert np.array_equal(a, b)


def test_same_pages_at_two_offsets_only_positions_differ():
    # A chunk's shared pages read at two different position bases: outputs differ,
    # and each equals the contiguous computation at its own base.
    q, kp, vp, ids, base, L = _tiny_problem(6, E=4, kv_len=16)
    a = O.decode_attention_one(q, kp, vp, ids, [0, 4, 8, 12], 16, 15, 1.0, 1e4)
    b = O.decode_attention_one(q, kp, vp, ids, [0, 4, 40, 44], 16, 47, 1.0, 1e4)
    assert np.abs(a - b).max() > 1e-6


def test_zero_positions_reduce_to_library_sdpa():
    rng = np.random.default_rng(7)
    Hq, Hkv, D, P, E = 6, 2, 16, 4, 6
    kp = _bits(rng, (10, Hkv, P, D)); vp = _bits(rng, (10, Hkv, P, D))
    ids = [7, 2, 9, 0, 4, 5]; L = 22
    q = _bits(rng, (Hq, D))
    got = O.decode_attention_one(q, kp, vp, ids, [0] * E, L, 0, 0.25, 1e4)
    # all keys at position 0 would still be rotated by their in-page offset; use rotate=False arm
    got0 = O.decode_attention_one(q, kp, vp, ids, [0] * E, L, 0, 0.25, 1e4, rotate=False)
    Kc = torch.from_numpy(np.concatenate([bf16_bits_to_f64(kp[p]).transpose(1, 0, 2) for p in ids])[:L])
    Vc = torch.from_numpy(np.concatenate([bf16_bits_to_f64(vp[p]).transpose(1, 0, 2) for p in ids])[:L])
    qt = torch.from_numpy(bf16_bits_to_f64(q))                                    # [Hq, D]
    G = Hq // Hkv
    Kh = Kc.permute(1, 0, 2).repeat_interleave(G, dim=0)                          # [Hq, L, D]
    Vh = Vc.permute(1, 0, 2).repeat_interleave(G, dim=0)
    want = torch.nn.functional.scaled_dot_product_attention(qt[:, None, :], Kh, Vh, scale=0.25)[:, 0, :].numpy()
    assert np.abs(got0 - want).max() < 1e-12
    # with huge theta every frequency but the first vanishes; with pos identical for q and all
    # keys (pos_base chosen so that base+slot is constant is impossible) -> use P=1 pages instead
    kp1 = kp[:, :, :1, :].copy(); vp1 = vp[:, :, :1, :].copy()
    got1 = O.decode_attention_one(q, kp1, vp1, ids, [11] * E, E, 11, 0.25, 1e4)
    K1 = torch.from_numpy(np.stack([bf16_bits_to_f64(kp1[p])[:, 0, :] for p in ids]))   # [E, Hkv, D]
    V1 = torch.from_numpy(np.stack([bf16_bits_to_f64(vp1[p])[:, 0, :] for p in ids]))
    want1 = torch.nn.functional.scaled_dot_product_attention(
        qt[:, None, :], K1.permute(1, 0, 2).repeat_interleave(G, 0), V1.permute(1, 0, 2).repeat_interleave(G, 0),
        scale=0.25)[:, 0, :].numpy()
    assert np.abs(got1 - want1).max() < 1e-12      # equal positions: rotation cancels in every score
    assert np.abs(got - got0).max() > 1e-6         # and the rotation is not a no-op in general


def test_softmax_closed_forms():
    rng = np.random.default_rng(8)
    Hq, Hkv, D, P = 2, 1, 8, 4
    kp = _bits(rng, (3, Hkv, P, D)); vp = _bits(rng, (3, Hkv, P, D)); q = _bits(rng, (Hq, D))
    # one key: o = v exactly
    o = O.decode_attention_one(q, kp, vp, [2], [0], 1, 0, 0.7, 1e4)
    assert np.array_equal(o, np.broadcast_to(bf16_bits_to_f64(vp[2, 0, 0]), (Hq, D)))
    # identical un-rotated keys at identical positions cannot be built inside one page; use q = 0:
    # all scores 0 -> o = mean(v)
    o = O.decode_attention_one(np.zeros((Hq, D), np.uint16), kp, vp, [1, 0], [0, 4], 7, 6, 0.7, 1e4)
    Vc = np.concatenate([bf16_bits_to_f64(vp[1, 0]), bf16_bits_to_f64(vp[0, 0])])[:7]
    assert np.abs(o - Vc.mean(0)).max() < 1e-15
    # two keys: weight of key 0 is sigmoid(s0 - s1)
    theta = 1e4
    o = O.decode_attention_one(q, kp, vp, [0], [5], 2, 9, 0.7, theta)
    k0 = O.rope_rotate(bf16_bits_to_f64(kp[0, 0, 0]), np.int64(5), theta)
    k1 = O.rope_rotate(bf16_bits_to_f64(kp[0, 0, 1]), np.int64(6), theta)
    for h in range(Hq):
        qr = O.rope_rotate(bf16_bits_to_f64(q[h]), np.int64(9), theta)
        w0 = 1.0 / (1.0 + math.exp(-0.7 * (float(qr @ k0) - float(qr @ k1))))
        want = w0 * bf16_bits_to_f64(vp[0, 0, 0]) + (1 - w0) * bf16_bits_to_f64(vp[0, 0, 1])
        assert np.abs(o[h] - want).max() < 1e-13


# ---------------------------------------------------------------- brute force
def _brute_rotate(x, pos, theta):
    D = len(x); half = D // 2
    y = [0.0] * D
    for i in range(half):
        ang = pos * theta ** (-(2.0 * i) / D)
        R = [[math.cos(ang), -math.sin(ang)], [math.sin(ang), math.cos(ang)]]
        y[i] = R[0][0] * x[i] + R[0][1] * x[i + half]
        y[i + half] = R[1][0] * x[i] + R[1][1] * x[i + half]
    return y


def _brute_attention(q, K, V, scale):
    s = [scale * sum(a * b for a, b in zip(q, k)) for k in K]
    mx = max(s)
    w = [math.exp(x - mx) for x in s]
    z = sum(w)
    return [sum(w[t] * V[t][d] for t in range(len(K))) / z for d in range(len(V[0]))]


@pytest.mark.parametrize("seed,D,P,Hq,Hkv", [(0, 4, 2, 2, 1), (1, 8, 4, 4, 2), (2, 6, 3, 3, 3)])
def test_decode_matches_scalar_brute_force(seed, D, P, Hq, Hkv):
    rng = np.random.default_rng(seed)
    n_pages, E = 5, 3
    kp = _bits(rng, (n_pages, Hkv, P, D)); vp = _bits(rng, (n_pages, Hkv, P, D)); q = _bits(rng, (Hq, D))
    ids = [4, 1, 3]; base = [0, 10, 3]; L = 3 * P - 1; q_pos = 12; theta = 100.0; scale = 0.6
    got = O.decode_attention_one(q, kp, vp, ids, base, L, q_pos, scale, theta)
    kf, vf, qf = bf16_bits_to_f64(kp), bf16_bits_to_f64(vp), bf16_bits_to_f64(q)
    G = Hq // Hkv
    for h in range(Hq):
        K, V = [], []
        for t in range(L):
            pg, sl = ids[t // P], t % P
            K.append(_brute_rotate(list(kf[pg, h // G, sl]), base[t // P] + sl, theta))
            V.append(list(vf[pg, h // G, sl]))
        want = _brute_attention(_brute_rotate(list(qf[h]), q_pos, theta), K, V, scale)
        assert np.abs(got[h] - np.array(want)).max() < 1e-12


def test_prefill_matches_scalar_brute_force_and_commits_bits():
    rng = np.random.default_rng(11)
    D, P, Hq, Hkv, n_pages = 8, 4, 4, 2, 6
    kp = _bits(rng, (n_pages, Hkv, P, D)); vp = _bits(rng, (n_pages, Hkv, P, D))
    ids = [5, 0, 2, 3]; base = [0, 4, 8, 12]; L = 14
    q_slot = [0, 1, 2, 3, 12, 13]                    # first block + a 2-token question
    R = len(q_slot)
    qn = _bits(rng, (R, Hq, D)); kn = _bits(rng, (R, Hkv, D)); vn = _bits(rng, (R, Hkv, D))
    kp0, vp0 = kp.copy(), vp.copy()
    theta, scale = 50.0, 0.45
    got = O.prefill_attention_one(qn, kn, vn, q_slot, kp, vp, ids, base, L, scale, theta)
    # side effect: exactly the new rows' bits, nothing else
    exp_k, exp_v = kp0.copy(), vp0.copy()
    for i, s in enumerate(q_slot):
        exp_k[ids[s // P], :, s % P, :] = kn[i]; exp_v[ids[s // P], :, s % P, :] = vn[i]
    assert np.array_equal(kp, exp_k) and np.array_equal(vp, exp_v)
    assert not np.array_equal(kp, kp0)
    kf, vf, qf = bf16_bits_to_f64(kp), bf16_bits_to_f64(vp), bf16_bits_to_f64(qn)
    G = Hq // Hkv
    for i, s in enumerate(q_slot):
        for h in range(Hq):
            K, V = [], []
            for t in range(s + 1):                   # causal by logical slot, inclusive
                K.append(_brute_rotate(list(kf[ids[t // P], h // G, t % P]), base[t // P] + t % P, theta))
                V.append(list(vf[ids[t // P], h // G, t % P]))
            want = _brute_attention(_brute_rotate(list(qf[i, h]), base[s // P] + s % P, theta), K, V, scale)
            assert np.abs(got[i, h] - np.array(want)).max() < 1e-12


def test_prefill_rows_see_each_other_and_last_row_equals_decode():
    rng = np.random.default_rng(12)
    D, P, Hq, Hkv = 8, 4, 2, 1
    kp = _bits(rng, (4, Hkv, P, D)); vp = _bits(rng, (4, Hkv, P, D))
    ids = [1, 3, 0]; base = [0, 4, 8]; L = 11
    q_slot = [8, 9, 10]
    qn = _bits(rng, (3, Hq, D)); kn = _bits(rng, (3, Hkv, D)); vn = _bits(rng, (3, Hkv, D))
    out = O.prefill_attention_one(qn, kn, vn, q_slot, kp, vp, ids, base, L, 0.5, 1e4)
    dec = O.decode_attention_one(qn[2], kp, vp, ids, base, L, 10, 0.5, 1e4)   # pools now hold the new rows
    assert np.abs(out[2] - dec).max() < 1e-14
    # changing row 0's K changes row 1's output (it is visible to later rows) but not row 0's own slot-mates before it
    kn2 = kn.copy(); kn2[0] = _bits(rng, (Hkv, D))
    out2 = O.prefill_attention_one(qn, kn2, vn, q_slot, kp, vp, ids, base, L, 0.5, 1e4)
    assert np.abs(out2[1] - out[1]).max() > 1e-6


# ---------------------------------------------------------------- split-KV merge
def test_merge_of_any_partition_equals_unsplit():
    rng = np.random.default_rng(13)
    n, D = 37, 8
    q = rng.standard_normal(D); K = rng.standard_normal((n, D)) * 3; V = rng.standard_normal((n, D))
    s = 0.8 * (K @ q); w = np.exp(s - s.max()); want = (w / w.sum()) @ V
    for cuts in ([0, 37], [0, 1, 37], [0, 5, 6, 20, 37], list(range(38))):
        parts = [O.partial_attention(q, K[a:b], V[a:b], 0.8) for a, b in zip(cuts[:-1], cuts[1:])]
        m = np.array([p[0] for p in parts]); l = np.array([p[1] for p in parts]); o = np.stack([p[2] for p in parts])
        got = O.merge_partials(m, l, o)
        assert np.abs(got - want).max() < 1e-13


# ---------------------------------------------------------------- tables
def _read_golden():
    d = {}
    with open(os.path.join(GOLDEN, "hand_example_tables.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *rest = line.split()
            d[k] = rest
    return d


def test_hand_worked_example_tables():
    g = _read_golden()
    st = O.OracleStore(int(g["page_size"][0]), int(g["num_pages"][0]))
    A = list(range(100, 100 + int(g["chunk_A_tokens"][0])))
    B = list(range(900, 900 + int(g["chunk_B_tokens"][0])))
    ka, ra, sa = st.register_chunk(A)
    kb, rb, sb = st.register_chunk(B)
    assert (ra, rb) == (False, False)
    assert sa == [int(x) for x in g["chunk_A_shared"]] and sb == [int(x) for x in g["chunk_B_shared"]]
    segs = []
    for tok in g["segments"]:
        segs.append((O.KIND_CHUNK, {"CA": ka, "CB": kb}[tok]) if tok[0] == "C" else (O.KIND_PROMPT, int(tok[1:])))
    t = st.build_block_table(1, segs)
    assert t.page_ids == [int(x) for x in g["page_ids"]]
    assert t.pos_base == [int(x) for x in g["pos_base"]]
    assert t.kv_len == int(g["kv_len"][0]) and len(t.page_ids) == int(g["n_entries"][0])
    want = []
    for r in g["recompute_ranges"]:
        a, b = r.split("-"); want.extend(range(int(a), int(b) + 1))
    assert t.recompute_slots == want
    s = st.stats()
    assert s["pages_private_held"] == int(g["private_pages"][0]) and s["pages_shared_held"] == int(g["shared_pages"][0])
    # leading pad: the canonical form of A is 8 pads then the tokens
    assert st.canonical_chunk(A) == tuple([0] * 8 + A)


def test_chunks_at_offsets_32_and_35_become_block_aligned_and_share_pages():
    # Section 2.3's example (block size 16; the same chunk after 32 and after 35 prompt tokens would
    # straddle different blocks): with canonical padding both copies start on a block boundary and
    # alias the same shared pages.
    st = O.OracleStore(16, 64)
    C = list(range(1, 49))
    key, _, shared = st.register_chunk(C)
    t1 = st.build_block_table(1, [(O.KIND_PROMPT, 32), (O.KIND_CHUNK, key), (O.KIND_PROMPT, 3)])
    t2 = st.build_block_table(2, [(O.KIND_PROMPT, 35), (O.KIND_CHUNK, key), (O.KIND_PROMPT, 3)])
    assert t1.page_ids[3:5] == shared and t2.page_ids[4:6] == shared      # chunk starts at entry 2 / entry 3
    assert t1.pos_base[2] == 32 and t2.pos_base[3] == 48                  # both multiples of 16
    assert t1.page_ids[2] != t2.page_ids[2 + 1]                           # first block private to each
    assert t1.kv_len == 32 + 48 + 3 and t2.kv_len == 48 + 48 + 3


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_table_closed_form_counts_on_configs(cfg):
    scale = 1.0 if cfg == 1 else 0.25
    wl = make_workload(cfg, scale=scale)
    P = wl.page_size
    st = O.OracleStore(P, wl.num_pages)
    tables, keys_used = [], set()
    n_chunk_segs = 0
    for r in wl.decode_requests + wl.prefill_requests:
        segs = []
        for kind, val in r.segments:
            if kind == O.KIND_CHUNK:
                key, _, _ = st.register_chunk(wl.chunks[val]); keys_used.add(key); n_chunk_segs += 1
                segs.append((kind, key))
            else:
                segs.append((kind, val))
        tables.append((r, st.build_block_table(r.request_id, segs)))
    s = st.stats()
    ceil = lambda a: -(-a // P)
    exp_entries = 0; exp_private = 0
    for r, t in tables:
        e = sum(ceil(len(wl.chunks[v]) if k == O.KIND_CHUNK else v) for k, v in r.segments)
        assert len(t.page_ids) == e and t.pos_base == [i * P for i in range(e)]
        exp_entries += e
        exp_private += sum(1 if k == O.KIND_CHUNK else ceil(v) for k, v in r.segments)
    exp_shared = sum(len(k) // P - 1 for k in keys_used)
    assert s["unshared_equivalent_pages"] == exp_entries
    assert s["pages_private_held"] == exp_private and s["pages_shared_held"] == exp_shared
    assert s["dedup_hits"] == n_chunk_segs - len(keys_used)
    assert s["pages_free"] == wl.num_pages - exp_private - exp_shared
    # shared pages never appear as a private (first) page, private pages are globally unique
    shared_ids = {p for c in st.chunks.values() for p in c["shared"]}
    private_ids = [p for r in st.requests.values() for p in r["private"]]
    assert len(private_ids) == len(set(private_ids)) and not (set(private_ids) & shared_ids)
    for r, t in tables:
        e = 0
        for k, v in r.segments:
            n = ceil(len(wl.chunks[v]) if k == O.KIND_CHUNK else v)
            if k == O.KIND_CHUNK:
                assert (e * P) % P == 0 and t.page_ids[e] in private_ids
                assert all(p in shared_ids for p in t.page_ids[e + 1:e + n])
            e += n


def test_reject_leaves_nothing_allocated_and_release_restores_fifo_order():
    st = O.OracleStore(4, 6)
    key, _, shared = st.register_chunk(list(range(10)))          # 3 pages -> 2 shared: pages 0,1
    assert shared == [0, 1]
    before = list(st.free)
    with pytest.raises(O.Reject):
        # needs 1 + 4 = 5 > 4 free; the only idle chunk is the one the request itself uses: protected
        st.build_block_table(1, [(O.KIND_CHUNK, key), (O.KIND_PROMPT, 13)])
    assert list(st.free) == before and st.stats()["chunk_refs"] == 0 and not st.requests
    assert st.stats()["chunks_resident"] == 1 and st.stats()["chunks_evicted"] == 0
    t1 = st.build_block_table(1, [(O.KIND_CHUNK, key), (O.KIND_PROMPT, 5)])   # private 2 | 3,4
    assert t1.page_ids == [2, 0, 1, 3, 4] and list(st.free) == [5]
    with pytest.raises(O.Reject):
        st.register_chunk(list(range(50, 50 + 24)))              # 6 pages -> 5 shared > 1 free; the chunk in use cannot go
    assert list(st.free) == [5] and st.stats()["chunks_resident"] == 1
    t2 = st.build_block_table(2, [(O.KIND_PROMPT, 2)])
    assert t2.page_ids == [5]
    st.release(2); st.release(1)
    assert list(st.free) == [5, 2, 3, 4]                          # freed pages appended ascending per release
    assert st.stats()["chunk_refs"] == 0 and st.stats()["chunks_resident"] == 1
    # the chunk stays resident while nothing needs its pages: registering it again is a hit with the same pages
    _, hit, again = st.register_chunk(list(range(10)))
    assert hit and again == [0, 1]


def test_idle_chunks_are_reclaimed_least_recently_used_first_and_only_under_pressure():
    # Section 3.2.3 "Eviction Policy": zero-reference chunk objects go, whole, oldest use first; pages of live
    # requests and chunks in use never do; nothing is reclaimed while free pages suffice.
    st = O.OracleStore(4, 10)
    A, _, sa = st.register_chunk(list(range(100, 112)))          # 3 pages -> shared 0,1
    B, _, sb = st.register_chunk(list(range(200, 212)))          # shared 2,3
    C, _, sc = st.register_chunk(list(range(300, 312)))          # shared 4,5
    assert (sa, sb, sc) == ([0, 1], [2, 3], [4, 5])
    t = st.build_block_table(1, [(O.KIND_CHUNK, B)])             # B in use; private page 6; free 7,8,9
    assert t.page_ids == [6, 2, 3]
    st.register_chunk(list(range(100, 112)))                     # touch A: now C is the least recently used idle chunk
    # a prompt of 4 pages does not fit the 3 free pages: C (LRU, idle) goes, A (idle, newer) and B (in use) stay
    t2 = st.build_block_table(2, [(O.KIND_PROMPT, 16)])
    assert t2.page_ids == [7, 8, 9, 4] and list(st.free) == [5]
    s = st.stats()
    assert s["chunks_evicted"] == 1 and s["pages_evicted"] == 2 and s["chunks_resident"] == 2
    assert C not in st.chunks and A in st.chunks and B in st.chunks
    # next demand of 2 pages: A is the only idle chunk left
    t3 = st.build_block_table(3, [(O.KIND_PROMPT, 8)])
    assert t3.page_ids == [5, 0] and list(st.free) == [1] and A not in st.chunks
    # B is in use: a demand that would need its pages is rejected and changes nothing
    with pytest.raises(O.Reject):
        st.build_block_table(4, [(O.KIND_PROMPT, 8)])
    assert list(st.free) == [1] and B in st.chunks and st.stats()["chunks_evicted"] == 2
    # a reclaimed chunk registers again as a miss, with fresh pages
    st.release(3)                                                # frees 0, 5 -> free [1, 0, 5]
    _, hit, sa2 = st.register_chunk(list(range(100, 112)))
    assert not hit and sa2 == [1, 0]


def test_same_chunk_twice_in_one_request_and_one_page_chunk():
    st = O.OracleStore(4, 20)
    key, _, shared = st.register_chunk([7, 8, 9, 10, 11, 12, 13, 14])     # 2 pages, 1 shared
    one, _, none = st.register_chunk([5, 6])                                # 1 page, no shared
    assert none == []
    t = st.build_block_table(3, [(O.KIND_CHUNK, key), (O.KIND_CHUNK, one), (O.KIND_CHUNK, key)])
    assert t.page_ids[1] == t.page_ids[4] == shared[0]
    assert len({t.page_ids[0], t.page_ids[2], t.page_ids[3]}) == 3
    assert t.pos_base == [0, 4, 8, 12, 16] and t.kv_len == 20
    assert st.stats()["chunk_refs"] == 3
    # a chunk equal to another chunk's padded form is the same chunk (identity = padded tokens)
    k2, hit, _ = st.register_chunk([0, 0, 5, 6])
    assert hit and k2 == one


# ---------------------------------------------------------------- power of the tolerance
def test_negative_controls_exceed_tolerance_on_benchmark_statistics():
    """On inputs with the benchmark's statistics, dropping or mangling the rotation moves the
    output by more than the parity tolerance (max-abs 2e-2 or mean-abs 2e-3), so a kernel that
    ignored RoPE could not pass."""
    wl = make_custom(2, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, rope_theta=5e5, sm_scale=1.0,
                     q_std=1 / math.sqrt(128), n_pool_chunks=4, chunk_tokens=512, zipf_s=1.1,
                     decode_chunks_per_request=[4, 4], decode_question=64, salt=99)
    kp, vp = wl.kv_pool(); q = wl.decode_q()
    st = O.OracleStore(16, wl.num_pages)
    r = wl.decode_requests[0]
    segs = [(k, st.register_chunk(wl.chunks[v])[0]) if k == O.KIND_CHUNK else (k, v) for k, v in r.segments]
    t = st.build_block_table(0, segs)
    qp = t.kv_len - 1
    good = O.decode_attention_one(q[0], kp, vp, t.page_ids, t.pos_base, t.kv_len, qp, 1.0, 5e5)
    def exceeds(x):
        d = np.abs(x - good)
        return d.max() > 2e-2 or d.mean() > 2e-3
    no_rope = O.decode_attention_one(q[0], kp, vp, t.page_ids, t.pos_base, t.kv_len, qp, 1.0, 5e5, rotate=False)
    zero_base = O.decode_attention_one(q[0], kp, vp, t.page_ids, [0] * len(t.pos_base), t.kv_len, qp, 1.0, 5e5)
    wrong_qpos = O.decode_attention_one(q[0], kp, vp, t.page_ids, t.pos_base, t.kv_len, 0, 1.0, 5e5)
    assert exceeds(no_rope) and exceeds(zero_base) and exceeds(wrong_qpos)


def test_pairing_convention_matters_interleaved_differs_beyond_tolerance():
    """The paper gives no RoPE pairing; the specification fixes split-half (i, i + D/2).  An interleaved
    (2i, 2i+1) rotation of the same inputs is a different function: the tolerance tells them apart, so a kernel
    built on the other convention could not pass."""
    wl = make_custom(2, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, rope_theta=5e5, sm_scale=1.0,
                     q_std=1 / math.sqrt(128), n_pool_chunks=4, chunk_tokens=512, zipf_s=1.1,
                     decode_chunks_per_request=[4], decode_question=64, salt=7)
    kp, vp = wl.kv_pool(); q = wl.decode_q()
    st = O.OracleStore(16, wl.num_pages)
    r = wl.decode_requests[0]
    segs = [(k, st.register_chunk(wl.chunks[v])[0]) if k == O.KIND_CHUNK else (k, v) for k, v in r.segments]
    t = st.build_block_table(0, segs)
    good = O.decode_attention_one(q[0], kp, vp, t.page_ids, t.pos_base, t.kv_len, t.kv_len - 1, 1.0, 5e5)
    # interleaved pairing, written out independently with complex numbers on (x[2i], x[2i+1])
    D, P, L, theta = 128, 16, t.kv_len, 5e5
    inv = np.array([theta ** (-(2.0 * i) / D) for i in range(D // 2)])
    def rot_il(x, pos):
        z = (x[..., 0::2] + 1j * x[..., 1::2]) * np.exp(1j * np.asarray(pos, dtype=np.float64)[..., None] * inv)
        y = np.empty_like(x); y[..., 0::2] = z.real; y[..., 1::2] = z.imag
        return y
    K = bf16_bits_to_f64(O.gather_pages(kp, t.page_ids, L)); V = bf16_bits_to_f64(O.gather_pages(vp, t.page_ids, L))
    pos = O.slot_positions(t.pos_base, L, P)
    Kr = rot_il(K, pos[:, None] * np.ones((1, K.shape[1])))
    qr = rot_il(bf16_bits_to_f64(q[0]), np.full(q.shape[1], L - 1.0))
    other = np.empty_like(good)
    for h in range(q.shape[1]):
        s = Kr[:, h // 4, :] @ qr[h]
        w = np.exp(s - s.max()); w /= w.sum()
        other[h] = w @ V[:, h // 4, :]
    d = np.abs(other - good)
    assert d.max() > 2e-2 or d.mean() > 2e-3


# --------------------------------------------------------------------------- fp8 (e4m3) pages
def test_e4m3_codes_roundtrip_and_known_values():
    v = O.e4m3_values()
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF]) and v[0x7E] == 448.0 and v[0xFE] == -448.0
    assert v[0x38] == 1.0 and v[0x40] == 2.0 and v[0x01] == 2.0 ** -9 and v[0x08] == 2.0 ** -6 and v[0x00] == 0.0
    finite = [c for c in range(256) if not np.isnan(v[c]) and c != 0x80]            # -0 encodes as 0x80 too; skip it here
    assert list(O.e4m3_encode(v[finite].astype(np.float32))) == finite
    # halves go to the even mantissa; out-of-range saturates; half the smallest subnormal goes to zero
    x = np.array([1.0625, 1.1875, 1000.0, -1000.0, 2.0 ** -10, 3 * 2.0 ** -10, 464.0, 0.0], dtype=np.float32)
    assert list(O.e4m3_encode(x)) == [0x38, 0x3A, 0x7E, 0xFE, 0x00, 0x02, 0x7E, 0x00]


def test_e4m3_encode_is_nearest_value_by_brute_force():
    v = O.e4m3_values()
    pos = np.array([c for c in range(128) if not np.isnan(v[c])])
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(4000) * s for s in (1e-3, 0.05, 1.0, 30.0, 400.0)]).astype(np.float32)
    codes = O.e4m3_encode(x)
    for xi, ci in zip(x, codes):
        d = np.abs(v[pos] - min(abs(float(xi)), 448.0))
        best = pos[np.flatnonzero(d == d.min())]
        want = best[0] if len(best) == 1 else [c for c in best if c % 2 == 0][0]   # a tie: the even mantissa
        assert (ci & 0x7F) == want and (ci >> 7) == int(np.signbit(xi)), (xi, ci, want)


def test_quantize_pages_scale_and_error_bound():
    rng = np.random.default_rng(6)
    pool = f32_to_bf16_bits((rng.standard_normal((5, 2, 16, 64)) * rng.uniform(0.01, 20, size=(5, 2, 1, 1))).astype(np.float32))
    pool[3, 1] = 0                                                                  # an all-zero block
    codes, scale = O.quantize_pages(pool)
    x = bf16_bits_to_f64(pool)
    amax = np.abs(x).max(axis=(2, 3))
    assert np.array_equal(scale[amax > 0], (amax[amax > 0].astype(np.float32) / np.float32(448.0)))
    assert scale[3, 1] == 1.0 and not codes[3, 1].any()
    # every non-zero block uses the top code for its largest element
    assert all((codes[i, j] & 0x7F).max() == 0x7E for i in range(5) for j in range(2) if amax[i, j] > 0)
    back = O.dequantize_pages(codes, scale)
    # half a unit in the last place of a 3-bit mantissa, or half a subnormal step, in units of the block's scale;
    # plus the float32 rounding of x / scale
    bound = np.maximum(np.abs(x) * 2.0 ** -4, scale[:, :, None, None] * 2.0 ** -10) * (1 + 1e-6)
    assert (np.abs(back - x) <= bound).all()


def test_decode_over_value_pools_equals_decode_over_bf16_pools():
    # values that e4m3 represents exactly with scale 1: the fp8 route and the bf16 route must then agree to the last bit
    rng = np.random.default_rng(8)
    v = O.e4m3_values()
    codes_k = rng.integers(0, 0x78, size=(6, 2, 16, 64)).astype(np.uint8) | (rng.integers(0, 2, size=(6, 2, 16, 64)).astype(np.uint8) << 7)
    codes_v = rng.integers(0, 0x78, size=(6, 2, 16, 64)).astype(np.uint8)
    ones = np.ones((6, 2), dtype=np.float32)
    kf, vf = O.dequantize_pages(codes_k, ones), O.dequantize_pages(codes_v, ones)
    kb, vb = f32_to_bf16_bits(kf.astype(np.float32)), f32_to_bf16_bits(vf.astype(np.float32))
    assert np.array_equal(bf16_bits_to_f64(kb), kf)                                 # exactly representable in bf16 too
    q = f32_to_bf16_bits(rng.standard_normal((4, 64)).astype(np.float32))
    args = ([4, 1, 3, 0, 5], [0, 16, 40, 56, 72], 70, 85, 0.05, 1e4)
    assert np.array_equal(O.decode_attention_one(q, kf, vf, *args), O.decode_attention_one(q, kb, vb, *args))


def test_quantize_pages_nan_zero_and_infinity_rules_by_hand():
    """The codec's corner rules (the design notes' reading R24), with every expected byte worked out by hand from the
    format's definition (1-4-3, bias 7, 448 = 0x7E, NaN = 0x7F) rather than by calling the codec:
    a NaN element takes the NaN code and does not take part in the block's maximum; a block whose finite maximum
    is zero (all zero, all NaN, or a mix of both) has scale 1; -0 keeps its sign bit; an infinite element makes
    the scale infinite, after which finite elements encode to zero and the infinite ones (inf/inf) to the NaN code."""
    def bf16(x):
        return int(f32_to_bf16_bits(np.array([x], dtype=np.float32))[0])
    pool = np.zeros((5, 1, 16, 64), dtype=np.uint16)
    # block 0: largest finite |x| = 3.5 -> scale = 3.5 / 448 = 2^-7 exactly
    row = [3.5, float("nan"), -1.75, -0.0, 2.0 ** -7, 2.0 ** -16, 2.0 ** -17, 3.0 * 2.0 ** -17, 0.4375]
    for j, x in enumerate(row):
        pool[0, 0, 0, j] = bf16(x)
    pool[0, 0, 5, 9] = 0xFFC0                      # a NaN with its sign bit set
    # x / 2^-7:          448   NaN  -224  -0    1     2^-9   2^-10 (tie -> even = 0)   3 * 2^-10 (tie -> 2 steps)   56
    want0 = [0x7E, 0x7F, 0xF6, 0x80, 0x38, 0x01, 0x00, 0x02, 0x66]
    pool[1, 0] = 0x7FC0                            # block 1: nothing but NaN
    pool[2, 0, 3, 3] = 0x7FC0                      # block 2: zeros and one NaN
    pool[3, 0, 0, 0] = bf16(float("inf")); pool[3, 0, 0, 1] = bf16(-2.0); pool[3, 0, 0, 2] = bf16(float("-inf"))
    # block 4 stays all zero
    with np.errstate(invalid="ignore"):
        codes, scale = O.quantize_pages(pool)
    assert scale[0, 0] == np.float32(2.0 ** -7)
    assert list(codes[0, 0, 0, :9]) == want0 and codes[0, 0, 5, 9] == 0x7F
    rest = codes[0, 0].copy(); rest[0, :9] = 0; rest[5, 9] = 0
    assert not rest.any()
    assert scale[1, 0] == 1.0 and (codes[1, 0] == 0x7F).all()
    assert scale[2, 0] == 1.0 and codes[2, 0, 3, 3] == 0x7F and np.count_nonzero(codes[2, 0]) == 1
    assert np.isinf(scale[3, 0]) and list(codes[3, 0, 0, :3]) == [0x7F, 0x80, 0x7F] and not codes[3, 0, 1:].any()
    assert scale[4, 0] == 1.0 and not codes[4, 0].any()
    # the encoder alone: NaN of either sign -> 0x7F; the zeros keep their sign
    nan_neg = np.array([0xFFC00000], dtype=np.uint32).view(np.float32)[0]
    assert list(O.e4m3_encode(np.array([np.nan, nan_neg, 0.0, -0.0], dtype=np.float32))) == [0x7F, 0x7F, 0x00, 0x80]
    # what the attention reads back: value(code) * scale, NaN stays NaN
    with np.errstate(invalid="ignore"):
        back = O.dequantize_pages(codes, scale)
    assert list(back[0, 0, 0, [0, 2, 4, 8]]) == [3.5, -1.75, 2.0 ** -7, 0.4375] and np.isnan(back[0, 0, 0, 1])


def test_commit_into_8bit_pages_by_hand_and_against_the_whole_page_codec():
    """Commit rule for 8-bit pages (the design notes' reading R25), bytes worked out by hand: a call that writes a
    block's slot 0 sets the block's scale from the rows it writes; a later call that appends keeps the scale and
    saturates.  A commit of a whole page must equal the whole-page codec on the same values (two routes, one format)."""
    def bf16(x):
        return int(f32_to_bf16_bits(np.array([x], dtype=np.float32))[0])
    P, Hkv, D = 4, 2, 8
    kc = np.full((3, Hkv, P, D), 0x55, dtype=np.uint8); vc = kc.copy()
    ks = np.full((3, Hkv), 7.0, dtype=np.float32); vs = ks.copy()
    page_ids = [2, 0]                                   # logical slots 0-3 live on page 2, slots 4-7 on page 0
    k_new = np.zeros((3, Hkv, D), dtype=np.uint16); v_new = np.zeros((3, Hkv, D), dtype=np.uint16)
    # rows for slots 4 and 5 (page 0, in-page slots 0 and 1: the block starts here) and slot 2 (page 2, slot 2: an append)
    k_new[0, 0, :3] = [bf16(7.0), bf16(-3.5), bf16(0.875)]      # head 0: block maximum 7 -> scale 7/448 = 2^-6
    k_new[1, 0, 0] = bf16(1.75)
    k_new[0, 1, 0] = bf16(float("nan"))                          # head 1 sees only NaN and zeros: scale 1
    k_new[2, 0, :2] = [bf16(4000.0), bf16(-14.0)]                # the append: page 2 keeps scale 7
    v_new[0, 0, 0] = bf16(448.0)                                 # V head 0: scale 1
    O.commit_rows_fp8(kc, ks, vc, vs, page_ids, [4, 5, 2], k_new, v_new)
    assert ks[0, 0] == np.float32(2.0 ** -6) and ks[0, 1] == 1.0 and ks[2, 0] == 7.0 and ks[1, 0] == 7.0
    # x / 2^-6: 448 -> 0x7E ; -224 -> 0xF6 ; 56 -> 0x66 ; second row 112 = 1.75 * 2^6 -> e = 13, m = 6 -> 0x6E
    assert list(kc[0, 0, 0, :4]) == [0x7E, 0xF6, 0x66, 0x00] and list(kc[0, 0, 1, :2]) == [0x6E, 0x00]
    assert kc[0, 1, 0, 0] == 0x7F and not kc[0, 1, 0, 1:].any() and not kc[0, 1, 1].any()
    assert (kc[0, :, 2:] == 0x55).all() and (kc[1] == 0x55).all()           # slots and pages not written keep their bytes
    # the append under scale 7: 4000/7 = 571 saturates to 448 (0x7E); -14/7 = -2 -> 0xC0; other slots untouched
    assert list(kc[2, 0, 2, :3]) == [0x7E, 0xC0, 0x00] and (kc[2, 0, [0, 1, 3]] == 0x55).all()
    assert vs[0, 0] == 1.0 and vc[0, 0, 0, 0] == 0x7E and vs[2, 0] == 7.0
    # a whole page through the commit = the whole-page codec
    rng = np.random.default_rng(11)
    page = f32_to_bf16_bits((rng.standard_normal((1, Hkv, P, D)) * 3).astype(np.float32))
    want_c, want_s = O.quantize_pages(page)
    c2 = np.zeros((1, Hkv, P, D), dtype=np.uint8); s2 = np.zeros((1, Hkv), dtype=np.float32)
    rows = np.ascontiguousarray(np.transpose(page[0], (1, 0, 2)))            # [P, Hkv, D]
    O.commit_rows_fp8(c2, s2, c2.copy(), s2.copy(), [0], [0, 1, 2, 3], rows, rows)
    assert np.array_equal(c2, want_c) and np.array_equal(s2, want_s)


def test_prefill_over_value_pools_equals_prefill_over_bf16_pools():
    # values that e4m3 holds exactly with scale 1: the route through 8-bit pages and the bf16 route give the same
    # bits, including the rows committed by the call
    rng = np.random.default_rng(12)
    P, Hkv, Hq, D, L = 4, 2, 4, 8, 14
    codes = lambda shape: rng.integers(0, 0x70, size=shape).astype(np.uint8) | (rng.integers(0, 2, size=shape).astype(np.uint8) << 7)
    kc, vc = codes((5, Hkv, P, D)), codes((5, Hkv, P, D))
    ones = np.ones((5, Hkv), dtype=np.float32)
    page_ids, pos_base = [3, 0, 4, 1], [0, 4, 20, 24]
    slots = [0, 1, 2, 3, 12, 13]
    vals = O.e4m3_values()
    new_c = codes((len(slots), Hkv, D)); new_cv = codes((len(slots), Hkv, D))
    k_new = f32_to_bf16_bits(vals[new_c].astype(np.float32)); v_new = f32_to_bf16_bits(vals[new_cv].astype(np.float32))
    # keep every block's maximum at 448 so that the commit's fresh scale is exactly 1 as well
    k_new[0, :, 0] = f32_to_bf16_bits(np.array([448.0], dtype=np.float32))[0]; v_new[0, :, 0] = k_new[0, 0, 0]
    k_new[4, :, 0] = k_new[0, 0, 0]; v_new[4, :, 0] = k_new[0, 0, 0]
    q_new = f32_to_bf16_bits(rng.standard_normal((len(slots), Hq, D)).astype(np.float32))
    kb = f32_to_bf16_bits(vals[kc].astype(np.float32)); vb = f32_to_bf16_bits(vals[vc].astype(np.float32))
    want = O.prefill_attention_one(q_new, k_new, v_new, slots, kb, vb, page_ids, pos_base, L, 0.3, 1e4)
    ks, vs = ones.copy(), ones.copy()
    O.commit_rows_fp8(kc, ks, vc, vs, page_ids, slots, k_new, v_new)
    assert (ks[[3, 1]] == 1.0).all() and (vs[[3, 1]] == 1.0).all()
    got = O.prefill_attention_one(q_new, k_new, v_new, slots, O.dequantize_pages(kc, ks), O.dequantize_pages(vc, vs),
                                  page_ids, pos_base, L, 0.3, 1e4)
    assert np.array_equal(got, want)
    assert np.array_equal(O.dequantize_pages(kc, ks), bf16_bits_to_f64(kb))        # the committed pool is the same pool
