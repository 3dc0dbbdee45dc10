"""The kernels' give-up path, run once in the only harmless form: a bounded wait on a barrier that nothing completes.

Every on-chip wait of the kernels polls a limited number of times and then gives up.  Here the limit is made short
(`mepic_kernel_test_hooks`) and the first worker leaves out ONE staged copy, so the barrier that copy would complete
is a flag nobody sets; nothing is in flight on it.  Expected: the call returns, the status word carries
MEPIC_DEV_WAIT_EXPIRED, the GPU and the context are fine, and the same call without the hook is parity-green against
the oracle right afterwards.  Nothing here faults, traps or spins without a bound.
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
SPIN = 1 << 12          # polls; the built-in limit is 1 << 22


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    yield
    M.mepic_kernel_test_hooks(0, -1)


def _case(seed, kv_lens):
    rng = np.random.default_rng(seed)
    B = len(kv_lens)
    ents = [-(-L // P) for L in kv_lens]
    num_pages = sum(ents) + 1
    perm = rng.permutation(num_pages)
    ids = np.zeros((B, max(ents)), dtype=np.int32); base = np.zeros_like(ids)
    at = 0
    for b in range(B):
        ids[b, :ents[b]] = perm[at:at + ents[b]]; at += ents[b]
        base[b, :ents[b]] = np.arange(ents[b]) * P
    kvl = np.asarray(kv_lens, dtype=np.int32)
    cfg = M.Config(P, HQ, HKV, D, num_pages, int(max(kv_lens)) + P, THETA)
    bits = lambda shape: f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return cfg, bits((num_pages, HKV, P, D)), bits((num_pages, HKV, P, D)), ids, base, kvl, (kvl - 1).astype(np.int32), bits((B, HQ, D))


@pytest.mark.parametrize("kind", ["decode", "fp8", "grouped"])
def test_decode_wait_runs_out_status_is_set_and_the_next_call_is_clean(kind):
    # long enough that worker 0 (the first warp's piece of the tile line) has several tiles
    cfg, kp, vp, ids, base, kvl, q_pos, q = _case(1, [6000, 5000, 7000])
    dev = RT.Device(cfg, kp, vp)
    sm = 1.0 / np.sqrt(D)
    if kind == "decode":
        batch = RT.DecodeBatch(dev, ids, base, kvl, q_pos, q)
    elif kind == "fp8":
        batch = RT.Fp8DecodeBatch(RT.Fp8Pools(dev), ids, base, kvl, q_pos, q)
    else:
        batch = RT.GroupedDecodeBatch(dev, ids, base, kvl, q_pos, q)
    torch.cuda.synchronize(); dev.status.zero_()
    try:
        M.mepic_kernel_test_hooks(SPIN, 1)            # worker 0 never gets its second tile
        batch.run(sm)
        torch.cuda.synchronize()                      # the call comes back
    finally:
        M.mepic_kernel_test_hooks(0, -1)
    assert dev.read_status() == M.MEPIC_DEV_WAIT_EXPIRED
    dev.status.zero_()
    out = batch.run(sm); torch.cuda.synchronize()
    assert dev.read_status() == 0
    if kind != "fp8":
        got = bf16_bits_to_f64(RT.bf16_bits(out))
        for b in range(len(kvl)):
            want = O.decode_attention_one(q[b], kp, vp, list(ids[b]), list(base[b]), int(kvl[b]), int(q_pos[b]), sm, THETA)
            d = np.abs(got[b] - want)
            assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (b, d.max())


@pytest.mark.parametrize("fp8", [False, True])
def test_prefill_wait_runs_out_every_role_leaves_and_the_next_call_is_clean(fp8):
    # one work item, one CTA (a 16-byte workspace keeps the call from cutting the item into shares): 600 keys = 5 key tiles
    cfg, kp, vp, ids, base, kvl, _, _ = _case(2, [600])
    rng = np.random.default_rng(3)
    bits = lambda shape: f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    slots = np.arange(568, 600, dtype=np.int32)
    qn, kn, vn = bits((32, HQ, D)), bits((32, HKV, D)), bits((32, HKV, D))
    ro = np.array([0, 32], dtype=np.int32)
    sm = 1.0 / np.sqrt(D)
    dev = RT.Device(cfg, kp.copy(), vp.copy())
    if fp8:
        pools = RT.Fp8Pools(dev)
        pb = RT.Fp8PrefillBatch(pools, ids, base, kvl, ro, slots, qn, kn, vn)
    else:
        pb = RT.PrefillBatch(dev, ids, base, kvl, ro, slots, qn, kn, vn)
    pb.ws_bytes = 16
    for skip in (0, 2):                               # the very first key tile; one in the middle of the pipeline
        try:
            M.mepic_kernel_test_hooks(SPIN, skip)
            pb.run(sm)
            torch.cuda.synchronize()
        finally:
            M.mepic_kernel_test_hooks(0, -1)
        assert dev.read_status() == M.MEPIC_DEV_WAIT_EXPIRED, skip
        dev.status.zero_()
    out = pb.run(sm); torch.cuda.synchronize()
    assert dev.read_status() == 0
    if fp8:
        kc, ks = O.quantize_pages(kp); vc, vs = O.quantize_pages(vp)
        O.commit_rows_fp8(kc, ks, vc, vs, list(ids[0]), list(slots), kn, vn)
        want = O.prefill_attention_one(qn, kn, vn, list(slots), O.dequantize_pages(kc, ks), O.dequantize_pages(vc, vs),
                                       list(ids[0]), list(base[0]), 600, sm, THETA)
        d = np.abs(bf16_bits_to_f64(RT.bf16_bits(out)) - want)
        assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS
        assert np.array_equal(pools.k_codes.cpu().numpy(), kc) and np.array_equal(pools.k_scales.cpu().numpy(), ks)
        return
    okp, ovp = kp.copy(), vp.copy()
    want = O.prefill_attention_one(qn, kn, vn, list(slots), okp, ovp, list(ids[0]), list(base[0]), 600, sm, THETA)
    d = np.abs(bf16_bits_to_f64(RT.bf16_bits(out)) - want)
    assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS
    assert np.array_equal(RT.bf16_bits(dev.k_pool), okp) and np.array_equal(RT.bf16_bits(dev.v_pool), ovp)
