"""Decode kernel (through the C ABI) against the fp64 oracle, element by element.

Tolerance (stated by the benchmark spec for bf16 inputs): max-abs <= 2e-2 and mean-abs
<= 2e-3 against the oracle.  Outputs here are small (|o| ~ 0.01-0.1), so the
tests also hold the kernel to a much tighter internal bar: relative L2 error
<= 1e-2 (bf16 output rounding alone gives ~2e-3).
"""
import numpy as np
import pytest
import torch

import paper_2512_16822_b200 as M
from paper_2512_16822_b200 import runtime as RT
from paper_2512_16822_b200.build import build_library
from mepic_inputs import make_workload, make_custom, f32_to_bf16_bits, bf16_bits_to_f64
from oracle import mepic_oracle as O

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_L2 = 2e-2, 2e-3, 1e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"


def _config_of(wl, num_pages=None, max_position=None):
    return M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim,
                    wl.num_pages if num_pages is None else num_pages,
                    wl.max_position if max_position is None else max_position, wl.rope_theta, wl.pad_token_id)


def _check(got_bits, want, what=""):
    got = bf16_bits_to_f64(got_bits)
    d = np.abs(got - want)
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert np.isfinite(got).all(), what
    assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (what, d.max(), d.mean())
    assert rel <= REL_L2, (what, rel)
    return d.max(), d.mean(), rel


def _run_decode(wl, sample=None, q_pos_override=None):
    """Build tables with the library, run the kernel, compare (sampled) requests with the oracle."""
    cfg = _config_of(wl)
    kp, vp = wl.kv_pool()
    q = wl.decode_q()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    if q_pos_override is not None:
        q_pos = q_pos_override(q_pos)
    dev = RT.Device(cfg, kp, vp)
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q)
    out = batch.run(wl.sm_scale)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    got = RT.bf16_bits(out)
    idx = range(len(tables)) if sample is None else sample
    worst = (0.0, 0.0, 0.0)
    for b in idx:
        t = tables[b]
        want = O.decode_attention_one(q[b], kp, vp, list(t.page_ids), list(t.pos_base), t.kv_len, int(q_pos[b]),
                                      wl.sm_scale, wl.rope_theta)
        worst = max(worst, _check(got[b], want, f"request {b}"))
    return worst


def test_config1_tiny_decode_all_elements():
    _run_decode(make_workload(1))


@pytest.mark.parametrize("cfg_index,scale", [(2, 0.25), (4, 0.25), (5, 0.1)])
def test_scaled_configs_all_elements(cfg_index, scale):
    _run_decode(make_workload(cfg_index, scale=scale))


@pytest.mark.parametrize("cfg_index,sample", [(2, [0, 3, 7, 11, 13, 18, 22, 26, 29, 31]), (4, [0, 2, 5, 7]),
                                               (5, [0, 1, 9, 23, 40, 64, 77, 90, 101, 113, 120, 127])])
def test_full_size_configs_sampled_requests(cfg_index, sample):
    # The full configuration in the launch shape the benchmark times; the oracle checks whole sampled requests.
    _run_decode(make_workload(cfg_index), sample=sample)


def _manual_case(seed, *, Hq, Hkv, D, P, kv_lens, pos_jitter=False, theta=1e4, scale=None, q_std=1.0, max_position=None):
    """Hand-built tables (random page ids, optional arbitrary position bases) - no store involved."""
    rng = np.random.default_rng(seed)
    B = len(kv_lens)
    ents = [-(-L // P) for L in kv_lens]
    num_pages = sum(ents) + 3
    perm = rng.permutation(num_pages)
    stride = max(ents) + 2
    page_ids = np.full((B, stride), -7, dtype=np.int32)           # poison beyond the used entries: must never be read
    pos_base = np.zeros((B, stride), dtype=np.int32)
    at = 0
    for b in range(B):
        page_ids[b, :ents[b]] = perm[at:at + ents[b]]; at += ents[b]
        base = np.arange(ents[b]) * P
        if pos_jitter:
            base = base + np.cumsum(rng.integers(0, 40, size=ents[b]))    # gaps between pages, still increasing
        pos_base[b, :ents[b]] = base
    kv_len = np.asarray(kv_lens, dtype=np.int32)
    last = kv_len - 1
    q_pos = (pos_base[np.arange(B), last // P] + last % P).astype(np.int32)
    maxpos = int(max(q_pos.max(), pos_base.max() + P)) + 1 if max_position is None else max_position
    cfg = M.Config(P, Hq, Hkv, D, num_pages, maxpos, theta)
    kp = f32_to_bf16_bits(rng.standard_normal((num_pages, Hkv, P, D)).astype(np.float32))
    vp = f32_to_bf16_bits(rng.standard_normal((num_pages, Hkv, P, D)).astype(np.float32))
    # slots past kv_len in each request's last page hold NaN bit patterns: they must be ignored
    for b in range(B):
        tail = kv_lens[b] % P
        if tail:
            pg = page_ids[b, ents[b] - 1]
            kp[pg, :, tail:, :] = 0x7FC0; vp[pg, :, tail:, :] = 0x7FC0
    q = f32_to_bf16_bits((rng.standard_normal((B, Hq, D)) * q_std).astype(np.float32))
    sm = (1.0 / np.sqrt(D)) if scale is None else scale
    return cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm, theta


def _run_manual(case):
    cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm, theta = case
    dev = RT.Device(cfg, kp, vp)
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q)
    out = batch.run(sm)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    got = RT.bf16_bits(out)
    for b in range(len(kv_len)):
        n = -(-int(kv_len[b]) // cfg.page_size)
        want = O.decode_attention_one(q[b], kp, vp, list(page_ids[b, :n]), list(pos_base[b, :n]), int(kv_len[b]),
                                      int(q_pos[b]), sm, theta)
        _check(got[b], want, f"request {b} kv_len {kv_len[b]}")
    return got


@pytest.mark.parametrize("Hq,Hkv,D,P", [
    (8, 2, 64, 16), (8, 2, 128, 16), (5, 1, 128, 16), (10, 2, 128, 32), (4, 4, 128, 16), (4, 2, 64, 64),
    (8, 1, 128, 16), (16, 2, 64, 16), (2, 2, 64, 16), (10, 2, 64, 16), (3, 1, 128, 16), (12, 2, 64, 32), (7, 1, 128, 16)])
def test_group_sizes_head_dims_page_sizes_ragged_lengths(Hq, Hkv, D, P):
    # lengths: one token, a page minus one, exact pages, several tiles plus ragged tails
    _run_manual(_manual_case(100 + Hq + D + P, Hq=Hq, Hkv=Hkv, D=D, P=P,
                             kv_lens=[1, P - 1, P, P + 1, 5 * P + 3, 777, 2049, 64]))


def test_arbitrary_position_bases_and_poisoned_tails():
    _run_manual(_manual_case(7, Hq=8, Hkv=2, D=128, P=16, kv_lens=[333, 1000, 17, 4096], pos_jitter=True, theta=5e5))


def test_query_position_before_the_keys_and_far_after():
    # rotation uses q_pos - base with either sign; q_pos is an input, not derived from kv_len
    case = list(_manual_case(8, Hq=8, Hkv=2, D=128, P=16, kv_lens=[200, 300], theta=5e5, max_position=5000))
    case[6] = np.array([0, 4999], dtype=np.int32)
    _run_manual(tuple(case))


def test_many_short_requests_more_units_than_workers_can_hold_one_each():
    rng = np.random.default_rng(3)
    _run_manual(_manual_case(9, Hq=4, Hkv=2, D=64, P=16, kv_lens=[int(x) for x in rng.integers(1, 90, size=300)]))


def test_shift_invariance_and_page_permutation_on_gpu():
    case = _manual_case(11, Hq=8, Hkv=2, D=128, P=16, kv_lens=[500, 123], theta=5e5, max_position=20000)
    a = _run_manual(case)
    cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm, theta = case
    b = _run_manual((cfg, kp, vp, page_ids, pos_base + 9000, kv_len, q_pos + 9000, q, sm, theta))
    da = bf16_bits_to_f64(a) - bf16_bits_to_f64(b)
    assert np.abs(da).max() <= 2e-3          # same result up to rounding of different table rows
    perm = np.random.default_rng(4).permutation(cfg.num_pages)
    kp2 = np.empty_like(kp); vp2 = np.empty_like(vp); kp2[perm] = kp; vp2[perm] = vp
    ids2 = np.where(page_ids >= 0, perm[np.clip(page_ids, 0, None)], page_ids).astype(np.int32)
    c = _run_manual((cfg, kp2, vp2, ids2, pos_base, kv_len, q_pos, q, sm, theta))
    assert np.array_equal(a, c)              # physical placement cannot change a single bit


def test_negative_controls_fail_the_tolerance():
    # The same check that passes for the kernel must FAIL for an oracle without rotation or with zeroed bases.
    wl = make_workload(2, scale=0.25)
    cfg = _config_of(wl)
    kp, vp = wl.kv_pool(); q = wl.decode_q()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    dev = RT.Device(cfg, kp, vp)
    out = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q).run(wl.sm_scale)
    torch.cuda.synchronize()
    got = bf16_bits_to_f64(RT.bf16_bits(out))[0]
    t = tables[0]
    def fails(want):
        d = np.abs(got - want)
        return d.max() > MAX_ABS or d.mean() > MEAN_ABS
    no_rope = O.decode_attention_one(q[0], kp, vp, list(t.page_ids), list(t.pos_base), t.kv_len, int(q_pos[0]),
                                     wl.sm_scale, wl.rope_theta, rotate=False)
    zero_base = O.decode_attention_one(q[0], kp, vp, list(t.page_ids), [0] * len(t.pos_base), t.kv_len,
                                       int(q_pos[0]), wl.sm_scale, wl.rope_theta)
    assert fails(no_rope) and fails(zero_base)


def test_bad_page_id_is_reported_not_faulted():
    case = list(_manual_case(12, Hq=8, Hkv=2, D=64, P=16, kv_lens=[100]))
    cfg, kp, vp, page_ids = case[0], case[1], case[2], case[3].copy()
    page_ids[0, 2] = cfg.num_pages + 5
    dev = RT.Device(cfg, kp, vp)
    RT.DecodeBatch(dev, page_ids, case[4], case[5], case[6], case[7]).run(case[8])
    torch.cuda.synchronize()
    assert dev.read_status() & M.MEPIC_DEV_BAD_PAGE


def test_argument_validation():
    case = _manual_case(13, Hq=8, Hkv=2, D=64, P=16, kv_lens=[40])
    cfg = case[0]
    dev = RT.Device(cfg, case[1], case[2])
    b = RT.DecodeBatch(dev, case[3], case[4], case[5], case[6], case[7])
    with pytest.raises(M.MepicError) as e:
        M.mepic_attn_decode(cfg, q=b.q, k_pool=dev.k_pool, v_pool=dev.v_pool, page_ids=b.page_ids, pos_base=b.pos_base,
                            kv_len=b.kv_len, q_pos=b.q_pos, rope_table=dev.rope, out=b.out, workspace=b.workspace,
                            workspace_bytes=16, status=dev.status, table_stride=b.stride, batch=1, sm_scale=1.0)
    assert e.value.code == M.MEPIC_E_INVAL
    with pytest.raises(M.MepicError) as e:
        M.mepic_attn_decode(cfg, q=None, k_pool=dev.k_pool, v_pool=dev.v_pool, page_ids=b.page_ids, pos_base=b.pos_base,
                            kv_len=b.kv_len, q_pos=b.q_pos, rope_table=dev.rope, out=b.out, workspace=b.workspace,
                            workspace_bytes=b.ws_bytes, status=dev.status, table_stride=b.stride, batch=1, sm_scale=1.0)
    assert e.value.code == M.MEPIC_E_INVAL


def test_decode_call_can_be_captured_in_a_cuda_graph_and_replayed():
    # The call only enqueues kernels on the caller's stream (tensor maps are encoded on the host and passed by value),
    # so a serving loop may capture it once and replay it with new q / tables written into the same buffers.
    wl = make_workload(1)
    cfg = _config_of(wl)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    dev = RT.Device(cfg, kp, vp)
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, wl.decode_q())
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        batch.run(wl.sm_scale, side)                      # first call outside capture (function attributes, entry points)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        batch.run(wl.sm_scale, torch.cuda.current_stream())
    rng = np.random.default_rng(3)
    for _ in range(2):
        q = f32_to_bf16_bits(rng.standard_normal((len(tables), wl.n_q_heads, wl.head_dim)).astype(np.float32))
        batch.q.view(torch.int16).copy_(torch.from_numpy(q.view(np.int16)))
        batch.out.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert dev.read_status() == 0
        got = RT.bf16_bits(batch.out)
        for b, t in enumerate(tables):
            want = O.decode_attention_one(q[b], kp, vp, list(t.page_ids), list(t.pos_base), t.kv_len, int(q_pos[b]),
                                          wl.sm_scale, wl.rope_theta)
            _check(got[b], want, f"request {b}")


def test_one_dominant_key_late_in_the_context_moves_the_reference_far():
    # One key whose score lies ~80 nats above all others, deep inside the context: the running maximum jumps when its
    # tile arrives (everything accumulated before is scaled to nothing) and the output is that key's V row.  The big
    # components sit in the slowest-rotating pair (63, 127 at D = 128), so their product barely depends on the positions.
    case = list(_manual_case(31, Hq=8, Hkv=2, D=128, P=16, kv_lens=[700, 2500], theta=1e4))
    cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm, theta = case
    big = f32_to_bf16_bits(np.array([30.0], dtype=np.float32))[0]
    q[:, :, 63] = big
    star = [450, 1777]
    for b, t in enumerate(star):
        kp[page_ids[b, t // 16], :, t % 16, 63] = big
    got = _run_manual(tuple(case))
    for b, t in enumerate(star):
        v_star = bf16_bits_to_f64(vp[page_ids[b, t // 16], :, t % 16, :])            # [Hkv, D]
        want = np.repeat(v_star, 4, axis=0)                                          # q head h reads kv head h // 4
        assert np.abs(bf16_bits_to_f64(got[b]) - want).max() <= 2e-2
