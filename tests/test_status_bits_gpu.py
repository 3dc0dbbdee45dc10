"""Device status bits that no parity case sets: MEPIC_DEV_BAD_POSITION in every attention kernel.

A position that the rope table does not cover (a q_pos or a block-table position base beyond max_position) must be
reported through the status word and replaced by a safe value: the call returns, the GPU is unharmed, and the next
call on clean inputs is parity-green again.  The table handed to the kernels is deliberately short here; nothing in
these tests reads outside any buffer.
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

MAX_ABS, MEAN_ABS = 2e-2, 2e-3
P, HQ, HKV, D, THETA = 16, 8, 2, 128, 1e4


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"


def _case(seed, kv_lens, max_position):
    rng = np.random.default_rng(seed)
    B = len(kv_lens)
    ents = [-(-L // P) for L in kv_lens]
    num_pages = sum(ents) + 1
    stride = max(ents)
    perm = rng.permutation(num_pages)
    ids = np.zeros((B, stride), dtype=np.int32); base = np.zeros((B, stride), dtype=np.int32)
    at = 0
    for b in range(B):
        ids[b, :ents[b]] = perm[at:at + ents[b]]; at += ents[b]
        base[b, :ents[b]] = np.arange(ents[b]) * P
    kvl = np.asarray(kv_lens, dtype=np.int32)
    q_pos = (kvl - 1).astype(np.int32)
    cfg = M.Config(P, HQ, HKV, D, num_pages, max_position, THETA)
    bits = lambda shape: f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return cfg, bits((num_pages, HKV, P, D)), bits((num_pages, HKV, P, D)), ids, base, kvl, q_pos, bits((B, HQ, D))


def _parity(out, q, kp, vp, ids, base, kvl, q_pos, sm):
    got = bf16_bits_to_f64(RT.bf16_bits(out))
    for b in range(len(kvl)):
        want = O.decode_attention_one(q[b], kp, vp, list(ids[b]), list(base[b]), int(kvl[b]), int(q_pos[b]), sm, THETA)
        d = np.abs(got[b] - want)
        assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (b, d.max(), d.mean())


@pytest.mark.parametrize("kind", ["decode", "fp8", "grouped"])
def test_decode_query_position_beyond_the_rope_table(kind):
    cfg, kp, vp, ids, base, kvl, q_pos, q = _case(1, [150, 90, 200], max_position=255)
    dev = RT.Device(cfg, kp, vp)
    sm = 1.0 / np.sqrt(D)
    far = q_pos.copy(); far[1] = 9000                       # 9000 - any tile base > 255: no table row for that angle
    if kind == "decode":
        mk = lambda qp: RT.DecodeBatch(dev, ids, base, kvl, qp, q)
    elif kind == "fp8":
        pools = RT.Fp8Pools(dev)
        mk = lambda qp: RT.Fp8DecodeBatch(pools, ids, base, kvl, qp, q)
    else:
        mk = lambda qp: RT.GroupedDecodeBatch(dev, ids, base, kvl, qp, q)
    out = mk(far).run(sm); torch.cuda.synchronize()
    assert dev.read_status() == M.MEPIC_DEV_BAD_POSITION     # reported, and nothing else went wrong
    got = bf16_bits_to_f64(RT.bf16_bits(out))
    assert np.isfinite(got).all()                            # the clamped angle gives some finite result
    # the other requests of the batch are unaffected
    if kind != "fp8":
        for b in (0, 2):
            want = O.decode_attention_one(q[b], kp, vp, list(ids[b]), list(base[b]), int(kvl[b]), int(q_pos[b]), sm, THETA)
            assert np.abs(got[b] - want).max() <= MAX_ABS
    dev.status.zero_()
    out = mk(q_pos).run(sm); torch.cuda.synchronize()        # and the next clean call is clean
    assert dev.read_status() == 0
    if kind != "fp8":
        _parity(out, q, kp, vp, ids, base, kvl, q_pos, sm)


def test_prefill_position_base_beyond_the_rope_table():
    cfg, kp, vp, ids, base, kvl, _, _ = _case(2, [200], max_position=255)
    rng = np.random.default_rng(3)
    bits = lambda shape: f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    slots = np.arange(184, 200, dtype=np.int32)
    qn, kn, vn = bits((16, HQ, D)), bits((16, HKV, D)), bits((16, HKV, D))
    ro = np.array([0, 16], dtype=np.int32)
    sm = 1.0 / np.sqrt(D)
    far = base.copy(); far[0, 5] = 100000                    # the keys of entry 5 get positions the table does not have
    dev = RT.Device(cfg, kp.copy(), vp.copy())
    out = RT.PrefillBatch(dev, ids, far, kvl, ro, slots, qn, kn, vn).run(sm); torch.cuda.synchronize()
    assert dev.read_status() == M.MEPIC_DEV_BAD_POSITION
    assert np.isfinite(bf16_bits_to_f64(RT.bf16_bits(out))).all()
    # a query row whose own position is out of range
    far2 = base.copy(); far2[0, 11] = 5000; far2[0, 12] = 5016
    dev.status.zero_()
    RT.PrefillBatch(dev, ids, far2, kvl, ro, slots, qn, kn, vn).run(sm); torch.cuda.synchronize()
    assert dev.read_status() == M.MEPIC_DEV_BAD_POSITION
    # clean inputs afterwards: parity with the oracle, pool committed bit for bit
    dev2 = RT.Device(cfg, kp.copy(), vp.copy())
    out = RT.PrefillBatch(dev2, ids, base, kvl, ro, slots, qn, kn, vn).run(sm); torch.cuda.synchronize()
    assert dev2.read_status() == 0
    okp, ovp = kp.copy(), vp.copy()
    want = O.prefill_attention_one(qn, kn, vn, list(slots), okp, ovp, list(ids[0]), list(base[0]), 200, sm, THETA)
    d = np.abs(bf16_bits_to_f64(RT.bf16_bits(out)) - want)
    assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS
    assert np.array_equal(RT.bf16_bits(dev2.k_pool), okp) and np.array_equal(RT.bf16_bits(dev2.v_pool), ovp)
