"""Run one benchmark configuration through the public binding and print the device time.

    python -m paper_2512_16822_b200.cases decode  --config 2 [--scale 1.0] [--iters 10] [--unshared] [--grouped] [--fp8] [--graph]
    python -m paper_2512_16822_b200.cases prefill --config 3 [--scale 0.5] [--iters 4]
    python -m paper_2512_16822_b200.cases mixed   --config 5            # decode and prefill of one pool on two streams

A small driver for profiling (a fixed, short sequence of calls that a profiler can capture) and for trying the
library on the synthetic workloads.  Inputs come from ``mepic_inputs``; nothing here checks results (the tests do).
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _setup_unshared_decode(index: int, scale: float, fp8: bool = False):
    """The decode batch on a layout without chunk sharing: every request owns private copies of its chunks."""
    import torch
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
    from mepic_inputs import make_workload
    wl = make_workload(index, scale=scale)
    P = wl.page_size
    ents = [sum(-(-(len(wl.chunks[v]) if k == 0 else v) // P) for k, v in r.segments) for r in wl.decode_requests]
    lens = [sum((len(wl.chunks[v]) if k == 0 else v) for k, v in r.segments) for r in wl.decode_requests]
    num_pages = int(sum(ents))
    cfg = M.Config(P, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, num_pages, wl.max_position, wl.rope_theta, wl.pad_token_id)
    B, stride = len(ents), max(ents)
    page_ids = np.zeros((B, stride), dtype=np.int32); pos_base = np.zeros((B, stride), dtype=np.int32)
    perm = np.random.default_rng([0, wl.index, 99]).permutation(num_pages).astype(np.int32)
    at = 0
    for b, e in enumerate(ents):
        page_ids[b, :e] = perm[at:at + e]; at += e
        pos_base[b, :e] = np.arange(e) * P
    kv_len = np.asarray(lens, dtype=np.int32)
    dev = RT.Device(cfg)
    dev.k_pool.normal_(); dev.v_pool.normal_()
    if fp8:
        return wl, dev, RT.Fp8DecodeBatch(RT.Fp8Pools(dev), page_ids, pos_base, kv_len, kv_len - 1, wl.decode_q())
    return wl, dev, RT.DecodeBatch(dev, page_ids, pos_base, kv_len, kv_len - 1, wl.decode_q())


def _setup(index: int, scale: float, which: str, grouped: bool = False, fp8: bool = False):
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
    from mepic_inputs import make_workload
    wl = make_workload(index, scale=scale)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        dec = RT.build_tables(st, wl.chunks, wl.decode_requests) if wl.decode_requests else []
        pre = RT.build_tables(st, wl.chunks, wl.prefill_requests) if wl.prefill_requests else []
    dev = RT.Device(cfg, kp, vp)
    dbatch = pbatch = None
    if which in ("decode", "both"):
        if not dec:
            raise SystemExit(f"config {index} has no decode requests")
        page_ids, pos_base, kv_len, q_pos = RT.pack_tables(dec, wl.page_size)
        if fp8:
            return wl, dev, RT.Fp8DecodeBatch(RT.Fp8Pools(dev), page_ids, pos_base, kv_len, q_pos, wl.decode_q())
        kind = RT.GroupedDecodeBatch if grouped else RT.DecodeBatch
        dbatch = kind(dev, page_ids, pos_base, kv_len, q_pos, wl.decode_q())
        if which == "decode":
            return wl, dev, dbatch
    if not pre:
        raise SystemExit(f"config {index} has no prefill requests")
    page_ids, pos_base, kv_len, _ = RT.pack_tables(pre, wl.page_size)
    slots = [t.recompute_slots for t in pre]
    rows = [wl.prefill_rows(i, len(s)) for i, s in enumerate(slots)]
    ro = np.concatenate([[0], np.cumsum([len(s) for s in slots])]).astype(np.int32)
    pbatch = RT.PrefillBatch(dev, page_ids, pos_base, kv_len, ro, np.concatenate(slots).astype(np.int32),
                             np.concatenate([r.q_new for r in rows]), np.concatenate([r.k_new for r in rows]),
                             np.concatenate([r.v_new for r in rows]))
    return wl, dev, ((dbatch, pbatch) if which == "both" else pbatch)


def _mixed(index: int, scale: float) -> None:
    """A serving step of a config that has both kinds of request: the decode batch and the prefill requests over one
    pool, each call alone and then both enqueued on two streams (device time from the fork to the join)."""
    import torch
    wl, dev, (db, pb) = _setup(index, scale, "both")
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    main_s = torch.cuda.current_stream()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev.device)

    def both():
        fork = torch.cuda.Event(); fork.record(main_s)
        s1.wait_event(fork); s2.wait_event(fork)
        pb.run(wl.sm_scale, s2)
        db.run(wl.sm_scale, s1)
        j1, j2 = torch.cuda.Event(), torch.cuda.Event()
        j1.record(s1); j2.record(s2)
        main_s.wait_event(j1); main_s.wait_event(j2)

    for name, fn in (("decode alone", lambda: db.run(wl.sm_scale)), ("prefill alone", lambda: pb.run(wl.sm_scale)),
                     ("both, two streams", both)):
        times = []
        for it in range(8):
            flush.fill_(1); flush.view(torch.int64).sum()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                times.append(e0.elapsed_time(e1))
        print(f"mixed config {index} scale {scale}: {name}: {sorted(times)[len(times) // 2]:.4f} ms median, {min(times):.4f} min "
              f"(L2 flushed), device status {dev.read_status()}")


def main() -> None:
    import torch
    ap = argparse.ArgumentParser()
    ap.add_argument("which", choices=["decode", "prefill", "mixed"])
    ap.add_argument("--config", type=int, default=None)
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--iters", type=int, default=4)
    ap.add_argument("--unshared", action="store_true", help="decode only: no chunk sharing, one page per table entry")
    ap.add_argument("--grouped", action="store_true", help="decode only: the sharing-aware path (host plan + grouped kernel)")
    ap.add_argument("--graph", action="store_true", help="capture the call in a CUDA graph and time replays (no L2 flush: launch latency)")
    ap.add_argument("--fp8", action="store_true", help="decode only: 8-bit (e4m3) pages made from the bf16 pool by the library's quantiser")
    args = ap.parse_args()
    index = args.config if args.config is not None else {"decode": 2, "prefill": 3, "mixed": 5}[args.which]
    if args.which == "mixed":
        _mixed(index, args.scale)
        return
    if args.unshared and args.which == "decode":
        wl, dev, batch = _setup_unshared_decode(index, args.scale, args.fp8)
    else:
        wl, dev, batch = _setup(index, args.scale, args.which, args.grouped, args.fp8)
    for _ in range(max(args.iters - 1, 1)):
        batch.run(wl.sm_scale)
    torch.cuda.synchronize()
    if args.graph:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            batch.run(wl.sm_scale, torch.cuda.current_stream())
        for name, fn in (("direct calls", lambda: batch.run(wl.sm_scale)), ("graph replays", graph.replay)):
            for _ in range(5):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(200):
                fn()
            e1.record()
            torch.cuda.synchronize()
            print(f"{args.which} config {index}: {name}: {e0.elapsed_time(e1) / 200 * 1e3:.2f} us per call back to back, device status {dev.read_status()}")
        return
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev.device)
    times = []
    for _ in range(5):
        flush.fill_(1); flush.view(torch.int64).sum()                 # L2 flushed, dirty lines pushed out
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); batch.run(wl.sm_scale); e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    print(f"{args.which} config {index} scale {args.scale}: {min(times):.4f} ms min, {sorted(times)[2]:.4f} ms median "
          f"(L2 flushed), device status {dev.read_status()}")


if __name__ == "__main__":
    main()
