"""Seeded random shapes through the three attention entry points, each checked against the oracle element by element.

Group size 1..8, one to three kv heads, both head dims, page sizes 16/32/64, ragged lengths from one token to a few
thousand, arbitrary position bases; decode per request, decode grouped over hand-built shared chunks, prefill with random
sets of new rows (none, a few, all).  The fixed cases of the other files pin the corners; this one walks between them.
"""
import numpy as np
import pytest

import test_decode_gpu as TD
import test_decode_grouped_gpu as TG
import test_prefill_gpu as TP

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("i", range(24))
def test_random_case(i):
    TD.build_library()
    rng = np.random.default_rng([2512, i])
    G = int(rng.integers(1, 9)); Hkv = int(rng.integers(1, 4)); D = int(rng.choice([64, 128])); P = int(rng.choice([16, 32, 64]))
    Hq = G * Hkv
    # ---- decode, then the grouped call on the same (unshared) tables
    B = int(rng.integers(1, 12))
    kv_lens = [int(x) for x in rng.integers(1, int(rng.choice([40, 300, 2500])), size=B)]
    case = TD._manual_case(1000 + i, Hq=Hq, Hkv=Hkv, D=D, P=P, kv_lens=kv_lens, pos_jitter=bool(rng.integers(0, 2)),
                           theta=float(rng.choice([1e4, 5e5])))
    TD._run_manual(case)
    cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm, theta = case
    TG._run(cfg, kp, vp, page_ids, pos_base, kv_len, q_pos, q, sm, theta, also_plain=False)
    # ---- grouped decode over shared chunks
    n_req = int(rng.integers(2, 9)); n_ch = int(rng.integers(1, 4))
    chunk_pages = [int(x) for x in rng.integers(1, 12, size=n_ch)]
    uses = [[int(c) for c in rng.integers(0, n_ch, size=int(rng.integers(1, 4)))] for _ in range(n_req)]
    tails = [int(x) for x in rng.integers(1, 3 * P, size=n_req)]
    shared = TG._shared_case(2000 + i, Hq=Hq, Hkv=Hkv, D=D, P=P, n_req=n_req, chunk_pages=chunk_pages, uses=uses,
                             tail_tokens=tails, jitter=bool(rng.integers(0, 2)))
    TG._run(*shared, 1.0 / np.sqrt(D), 1e4, also_plain=False)
    # ---- prefill
    specs = []
    for _ in range(int(rng.integers(1, 4))):
        L = int(rng.integers(1, int(rng.choice([60, 400, 1500]))))
        k = int(rng.integers(0, min(L, 200) + 1))
        new = sorted(set(int(x) for x in rng.choice(L, size=k, replace=False))) if k else []
        if rng.integers(0, 2) and L - 1 not in new:
            new.append(L - 1)
        specs.append((L, sorted(new)))
    if sum(len(s) for _, s in specs) == 0:
        specs[0] = (specs[0][0], [0])
    pc = TP._manual(3000 + i, Hq=Hq, Hkv=Hkv, D=D, P=P, specs=specs, jitter=bool(rng.integers(0, 2)))
    TP._run_prefill(*pc, 1.0 / np.sqrt(D), 1e4)


@pytest.mark.parametrize("i", range(8))
def test_random_case_over_8bit_pages(i):
    import test_decode_fp8_gpu as TF
    TD.build_library()
    rng = np.random.default_rng([2512, 100 + i])
    G = int(rng.integers(1, 9)); Hkv = int(rng.integers(1, 4)); P = int(rng.choice([16, 32, 64]))
    lens = [int(x) for x in rng.integers(1, int(rng.choice([40, 300, 2500])), size=int(rng.integers(1, 10)))]
    args = TF._manual(500 + i, Hq=G * Hkv, Hkv=Hkv, P=P, kv_lens=lens, jitter=bool(rng.integers(0, 2)), spread=bool(rng.integers(0, 2)))
    TF._run(*args, 1.0 / np.sqrt(128), 1e4)
