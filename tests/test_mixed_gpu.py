"""Config 5 as a serving step: the decode batch and the prefill requests enqueued on two streams over ONE pool.

Both calls must stay correct while they overlap on the GPU: separate workspaces, one shared K/V pool; the prefill
commit writes only private pages of the prefill requests, which no decode request reads.
"""
import numpy as np
import pytest
import torch

import paper_2512_16822_b200 as M
from paper_2512_16822_b200 import runtime as RT
from paper_2512_16822_b200.build import build_library
from mepic_inputs import make_workload, bf16_bits_to_f64
from oracle import mepic_oracle as O

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("scale", [0.1, 1.0])
def test_config5_decode_and_prefill_overlapping_on_two_streams(scale):
    build_library()
    wl = make_workload(5, scale=scale)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        dec = RT.build_tables(st, wl.chunks, wl.decode_requests)
        pre = RT.build_tables(st, wl.chunks, wl.prefill_requests)
        stats = st.stats()
    assert stats["pages_free"] >= 0
    dev = RT.Device(cfg, kp, vp)
    d_ids, d_base, d_len, d_qpos = RT.pack_tables(dec, wl.page_size)
    q = wl.decode_q()
    db = RT.DecodeBatch(dev, d_ids, d_base, d_len, d_qpos, q)
    p_ids, p_base, p_len, _ = RT.pack_tables(pre, wl.page_size)
    slots = [t.recompute_slots for t in pre]
    rows = [wl.prefill_rows(i, len(s)) for i, s in enumerate(slots)]
    ro = np.concatenate([[0], np.cumsum([len(s) for s in slots])]).astype(np.int32)
    pb = RT.PrefillBatch(dev, p_ids, p_base, p_len, ro, np.concatenate(slots).astype(np.int32),
                         np.concatenate([r.q_new for r in rows]), np.concatenate([r.k_new for r in rows]),
                         np.concatenate([r.v_new for r in rows]))
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(2):                      # twice: the second round overlaps with warm caches
        pb.run(wl.sm_scale, s2)
        db.run(wl.sm_scale, s1)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    # oracle: the prefill commit touches only the prefill requests' private pages; apply it, then check both
    ok, ov = kp.copy(), vp.copy()
    got_p = RT.bf16_bits(pb.out)
    for b, t in enumerate(pre):
        R = len(slots[b])
        sel = sorted(set([0, 15, 16, R // 2, R - 1]))
        want = O.prefill_attention_one(rows[b].q_new, rows[b].k_new, rows[b].v_new, list(slots[b]), ok, ov,
                                       list(t.page_ids), list(t.pos_base), t.kv_len, wl.sm_scale, wl.rope_theta, rows=sel)
        g = bf16_bits_to_f64(got_p[ro[b]:ro[b + 1]][sel])
        d = np.abs(g - want)
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, ("prefill", b, d.max(), d.mean())
    assert np.array_equal(RT.bf16_bits(dev.k_pool), ok) and np.array_equal(RT.bf16_bits(dev.v_pool), ov)
    got_d = RT.bf16_bits(db.out)
    sample = range(len(dec)) if len(dec) <= 16 else [0, 1, len(dec) // 2, len(dec) - 1]
    for b in sample:
        t = dec[b]
        want = O.decode_attention_one(q[b], ok, ov, list(t.page_ids), list(t.pos_base), t.kv_len, int(d_qpos[b]),
                                      wl.sm_scale, wl.rope_theta)
        d = np.abs(bf16_bits_to_f64(got_d[b]) - want)
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, ("decode", b, d.max(), d.mean())
