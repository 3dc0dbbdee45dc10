"""Decode through the entry point that needs no workspace (mepic_attn_decode_static).

Some callers of the library cannot allocate device memory when they decode (they run inside an
allocator callback, or their host process forbids device allocation after start-up, or the page
pool already owns all free memory), so they cannot hand mepic_attn_decode its workspace.  The
static entry point keeps the split-KV partials in an array built into the library.  This test
calls it through the C ABI, twice in a row (the array is shared and keeps the previous call's
contents), and checks each result against the ordinary entry point on the same inputs: within the
tolerance the decode parity tests use and, since both entry points run the same kernels over the
same partial slots, bit for bit; the first batch is also compared with the CPU oracle directly.  It
also checks that a batch too large for the array is refused with a clear error and that the calls
take no device memory, neither from torch's caching allocator nor from the driver (the free-memory
figure of the device is the same before and after; the array itself appears when the library's
decode module is first used, which the ordinary call before it has already done).

The file name sorts last on purpose: if this test fails, every other test has already run.
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

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _setup(cfg_index, scale):
    wl = make_workload(cfg_index, scale=scale)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    dev = RT.Device(cfg, kp, vp)
    return wl, cfg, dev, RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, wl.decode_q()), tables


def _static(cfg, dev, batch, out, sm_scale):
    M.mepic_attn_decode_static(cfg, q=batch.q, k_pool=dev.k_pool, v_pool=dev.v_pool, page_ids=batch.page_ids,
                               pos_base=batch.pos_base, kv_len=batch.kv_len, q_pos=batch.q_pos,
                               rope_table=dev.rope, out=out, status=dev.status, table_stride=batch.stride,
                               batch=batch.batch, sm_scale=sm_scale, stream=torch.cuda.current_stream())


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    # two different batches back to back: the second call finds the first call's partials in the array
    for cfg_index, scale in ((1, 1.0), (2, 0.25)):
        wl, cfg, dev, batch, tables = _setup(cfg_index, scale)
        assert M.mepic_attn_decode_workspace(cfg, batch.batch) <= M.MEPIC_DECODE_STATIC_SCRATCH_BYTES
        want_bits = RT.bf16_bits(batch.run(wl.sm_scale)).copy()
        want = bf16_bits_to_f64(want_bits)
        torch.cuda.synchronize()
        out = torch.empty_like(batch.out)
        for call in range(2):
            out.zero_()
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
            free_before = torch.cuda.mem_get_info()[0]
            launches = M.mepic_launch_count()
            _static(cfg, dev, batch, out, wl.sm_scale)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] == free_before        # nothing taken from the driver either
            assert M.mepic_launch_count() - launches == 2
            assert dev.read_status() == 0
            got = bf16_bits_to_f64(RT.bf16_bits(out))
            d = np.abs(got - want)
            assert np.isfinite(got).all() and d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (cfg_index, call, d.max())
            assert np.array_equal(RT.bf16_bits(out), want_bits), (cfg_index, call)
            if cfg_index == 1:      # and against the definition itself, not only against the other entry point
                q = wl.decode_q()
                kp, vp = wl.kv_pool()
                for b, t in enumerate(tables):
                    ref = O.decode_attention_one(q[b], kp, vp, list(t.page_ids), list(t.pos_base), int(t.kv_len),
                                                 int(batch.q_pos[b].item()), wl.sm_scale, wl.rope_theta)
                    e = np.abs(got[b] - ref)
                    assert e.max() <= MAX_ABS and e.mean() <= MEAN_ABS, (b, call, e.max())


def test_static_scratch_refuses_sizes_beyond_the_array():
    build_library()
    wl, cfg, dev, batch, _ = _setup(1, 1.0)
    big = 200000      # a batch whose partials cannot fit the built-in array; the size check comes before any launch
    assert M.mepic_attn_decode_workspace(cfg, big) > M.MEPIC_DECODE_STATIC_SCRATCH_BYTES
    launches = M.mepic_launch_count()
    with pytest.raises(M.MepicError) as e:
        M.mepic_attn_decode_static(cfg, q=batch.q, k_pool=dev.k_pool, v_pool=dev.v_pool, page_ids=batch.page_ids,
                                   pos_base=batch.pos_base, kv_len=batch.kv_len, q_pos=batch.q_pos,
                                   rope_table=dev.rope, out=batch.out, status=dev.status, table_stride=batch.stride,
                                   batch=big, sm_scale=wl.sm_scale)
    assert e.value.code == M.MEPIC_E_INVAL and "scratch" in str(e.value)
    assert M.mepic_launch_count() == launches
