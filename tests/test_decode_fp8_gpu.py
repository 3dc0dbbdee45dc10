"""fp8 (e4m3) pages: the quantiser bit for bit against the oracle's codec, and the decode over 8-bit pools against
the fp64 oracle evaluated on the same codes and scales (tolerance of the bf16 decode: max-abs 2e-2, mean-abs 2e-3,
relative L2 1e-2).  Both sides take the rounding decision in fp32 from the same bf16 inputs, so codes and scales must
be identical, not close."""
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


@pytest.mark.parametrize("P,Hkv,D", [(16, 2, 128), (64, 3, 128), (16, 4, 64), (32, 1, 128)])
def test_quantiser_codes_and_scales_are_the_oracles(P, Hkv, D):
    rng = np.random.default_rng(P + Hkv + D)
    n = 9
    x = rng.standard_normal((n, Hkv, P, D)) * rng.choice([1e-3, 0.3, 1.0, 40.0, 3e4], size=(n, Hkv, 1, 1))
    x[2, 0] = 0.0                                           # an all-zero block
    x[4, Hkv - 1, 3, 5] = 1e30                              # one huge element: everything else lands in the subnormals or zero
    pool = f32_to_bf16_bits(x.astype(np.float32))
    pool[6, 0, 1, 2] = 0x7FC0                               # a NaN element: NaN code, and it must not set the scale
    cfg = M.Config(P, 2 * Hkv, Hkv, D, n, 1024, 1e4)
    dev = RT.Device(cfg, pool, pool[::-1].copy())
    fp = RT.Fp8Pools(dev, pages=np.array([0, 1, 2, 4, 5, 6, 8], dtype=np.int32))
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    want_k, scale_k = O.quantize_pages(pool)
    want_v, scale_v = O.quantize_pages(pool[::-1].copy())
    got_k, got_v = fp.k_codes.cpu().numpy(), fp.v_codes.cpu().numpy()
    listed = [0, 1, 2, 4, 5, 6, 8]
    assert want_k[6, 0, 1, 2] == 0x7F and np.isfinite(scale_k).all()
    for pg in listed:
        for h in range(Hkv):
            assert np.array_equal(got_k[pg, h], want_k[pg, h]) and fp.k_scales[pg, h].item() == scale_k[pg, h], (pg, h)
            assert np.array_equal(got_v[pg, h], want_v[pg, h]) and fp.v_scales[pg, h].item() == scale_v[pg, h], (pg, h)
    # pages that were not listed are untouched
    assert not got_k[3].any() and not got_k[7].any() and (fp.k_scales.cpu().numpy()[[3, 7]] == 1.0).all()


def test_quantiser_reports_a_bad_page():
    cfg = M.Config(16, 4, 2, 128, 4, 1024, 1e4)
    pool = np.zeros((4, 2, 16, 128), dtype=np.uint16)
    dev = RT.Device(cfg, pool, pool)
    RT.Fp8Pools(dev, pages=np.array([1, 9], dtype=np.int32))
    torch.cuda.synchronize()
    assert dev.read_status() & M.MEPIC_DEV_BAD_PAGE


def _run(cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm_scale, theta, sample=None, poison=None):
    dev = RT.Device(cfg, kp, vp)
    fp = RT.Fp8Pools(dev)
    if poison is not None:
        poison(fp)
    batch = RT.Fp8DecodeBatch(fp, page_ids, pos_base, kv_len, q_pos, q)
    out = batch.run(sm_scale)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    got = RT.bf16_bits(out).copy()
    # the sharing-aware path over the same 8-bit pools (mepic_attn_decode_grouped_fp8): same definition, same tolerance
    gout = RT.Fp8GroupedDecodeBatch(fp, page_ids, pos_base, kv_len, q_pos, q).run(sm_scale)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    ggot = RT.bf16_bits(gout)
    # the oracle works on the oracle's own codes and scales (identical to the device's, see the quantiser test)
    kc, ks = O.quantize_pages(kp); vc, vs = O.quantize_pages(vp)
    kf, vf = O.dequantize_pages(kc, ks), O.dequantize_pages(vc, vs)
    P = cfg.page_size
    for b in (range(len(kv_len)) if sample is None else sample):
        n = -(-int(kv_len[b]) // P)
        want = O.decode_attention_one(q[b], kf, vf, list(page_ids[b, :n]), list(pos_base[b, :n]), int(kv_len[b]),
                                      int(q_pos[b]), sm_scale, theta)
        _check(got[b], want, f"request {b}")
        _check(ggot[b], want, f"request {b}, grouped")
    return got, (kf, vf)


def _workload(idx, scale=1.0, sample=None):
    wl = make_workload(idx, scale=scale)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    return _run(cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, wl.decode_q(), wl.sm_scale, wl.rope_theta, sample)


@pytest.mark.parametrize("idx,scale", [(2, 0.25), (4, 0.25), (5, 0.1)])
def test_scaled_configs_all_elements(idx, scale):
    _workload(idx, scale)


@pytest.mark.parametrize("idx,sample", [(2, [0, 13, 31]), (4, [0, 7]), (5, [0, 1, 64, 127])])
def test_full_size_configs_sampled_requests(idx, sample):
    _workload(idx, 1.0, sample)


def _manual(seed, *, Hq, Hkv, P, kv_lens, jitter=False, theta=1e4, spread=True):
    rng = np.random.default_rng(seed)
    D, B = 128, len(kv_lens)
    ents = [-(-L // P) for L in kv_lens]
    num_pages = sum(ents) + 3
    perm = rng.permutation(num_pages)
    stride = max(ents) + 2
    page_ids = np.full((B, stride), -7, dtype=np.int32); pos_base = np.zeros((B, stride), dtype=np.int32)
    at = 0
    for b in range(B):
        page_ids[b, :ents[b]] = perm[at:at + ents[b]]; at += ents[b]
        base = np.arange(ents[b]) * P
        if jitter:
            base = base + np.cumsum(rng.integers(0, 40, size=ents[b]))
        pos_base[b, :ents[b]] = base
    kv_len = np.asarray(kv_lens, dtype=np.int32)
    last = kv_len - 1
    q_pos = (pos_base[np.arange(B), last // P] + last % P).astype(np.int32)
    cfg = M.Config(P, Hq, Hkv, D, num_pages, int(max(q_pos.max(), pos_base.max() + P)) + 1, theta)
    # blocks of very different magnitude, so that the per-block scales matter (V stays within +-few units: the
    # tolerance is absolute and the bf16 output rounding alone exceeds it for outputs of magnitude 4 and more)
    kmag = rng.choice([0.05, 1.0, 12.0], size=(num_pages, Hkv, 1, 1)) if spread else 1.0
    vmag = rng.choice([0.02, 0.25, 1.0], size=(num_pages, Hkv, 1, 1)) if spread else 1.0
    kp = f32_to_bf16_bits((rng.standard_normal((num_pages, Hkv, P, D)) * kmag).astype(np.float32))
    vp = f32_to_bf16_bits((rng.standard_normal((num_pages, Hkv, P, D)) * vmag).astype(np.float32))
    q = f32_to_bf16_bits((rng.standard_normal((B, Hq, D)) * 0.3).astype(np.float32))
    return cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q


@pytest.mark.parametrize("Hq,Hkv,P", [(8, 2, 16), (4, 4, 16), (2, 1, 32), (3, 1, 16), (10, 2, 16), (6, 1, 64), (7, 1, 16), (8, 1, 64)])
def test_group_sizes_page_sizes_ragged_lengths_and_block_scales(Hq, Hkv, P):
    lens = [1, 15, 16, 17, 5 * P + 3, 9 * P, 23 * P + P // 2 + 1, 700]
    args = _manual(40 + Hq + P, Hq=Hq, Hkv=Hkv, P=P, kv_lens=lens, jitter=True)
    # slots past kv_len in each request's last page hold the NaN code: they must be ignored
    def poison(fp):
        cfg, _, _, page_ids, _, kv_len = args[0], None, None, args[3], None, args[5]
        for b, L in enumerate(kv_len):
            tail = int(L) % cfg.page_size
            if tail:
                pg = int(page_ids[b, -(-int(L) // cfg.page_size) - 1])
                fp.k_codes[pg, :, tail:, :] = 0x7F; fp.v_codes[pg, :, tail:, :] = 0x7F
    _run(*args, 1.0 / np.sqrt(128), 1e4, poison=poison)


def test_quantisation_is_what_separates_it_from_the_bf16_decode():
    # the 8-bit result must sit near the bf16 result (it is the same attention over slightly perturbed K/V) yet not
    # on top of it: a kernel that silently read the bf16 pool, or ignored the scales, fails one of the two bounds
    args = _manual(77, Hq=8, Hkv=2, P=16, kv_lens=[900, 333], theta=5e5)
    cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q = args
    got, _ = _run(*args, 0.12, 5e5)
    full = np.stack([O.decode_attention_one(q[b], kp, vp, list(page_ids[b]), list(pos_base[b]), int(kv_len[b]), int(q_pos[b]), 0.12, 5e5)
                     for b in range(2)])
    rel = np.linalg.norm(bf16_bits_to_f64(got) - full) / np.linalg.norm(full)
    assert 5e-3 < rel < 0.15, rel


def test_head_dim_64_is_refused():
    cfg = M.Config(16, 4, 2, 64, 8, 1024, 1e4)
    pool = np.zeros((8, 2, 16, 64), dtype=np.uint16)
    dev = RT.Device(cfg, pool, pool)
    fp = RT.Fp8Pools(dev)                                   # the quantiser itself takes any head_dim
    ids = np.zeros((1, 2), dtype=np.int32)
    batch = RT.Fp8DecodeBatch(fp, ids, ids, np.array([20], dtype=np.int32), np.array([19], dtype=np.int32))
    with pytest.raises(M.MepicError) as e:
        batch.run(1.0)
    assert e.value.code == M.MEPIC_E_INVAL
