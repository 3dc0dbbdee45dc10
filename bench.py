#!/usr/bin/env python
"""Benchmark of the MEPIC hot path on B200: RoPE-fused paged-attention decode (HBM GB/s).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]

One "step" is one pass of the decode hot path over one batch: a call of
``mepic_attn_decode`` (split-KV kernel + merge kernel) on the configuration the
metric is quoted on (config 2, the Llama-3-8B-shaped decode layer).  ``value``
is the effective bandwidth = logical K/V bytes the batch must read / device
time, with every input already resident in HBM and the L2 flushed between
timed steps.  ``e2e`` is the same call with the step's inputs (q and the block
tables) coming from pinned host memory and the result read back, copies inside
the timed region; the K/V pool is the cache itself and stays resident.

Under torchrun every rank runs its own replica of the batch on its own GPU
(requests are independent: no data-path collective); the aggregate is all
ranks' bytes over the slowest rank's time.

``--impl reference`` times the CPU oracle, as it stands, on the host cores
(rank 0 only) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from mepic_inputs import make_workload  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one mepic_decode_splitkv launch (ncu, see profiles/);
# config 2: 356.9 MB read + 3.9 MB written (profiles/decode_splitkv_config2.md).
NCU_TRAFFIC_BYTES = {2: 360_870_000}


def kv_bytes_per_token(wl) -> int:
    """Algorithmic bytes per context token: K and V, all KV heads, bf16."""
    return 2 * wl.n_kv_heads * wl.head_dim * 2


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)", d
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)", {}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def wait_first_sample(self, timeout_s: float = 5.0):
        t0 = time.time()
        while self.proc is not None and not self.rows and time.time() - t0 < timeout_s:
            time.sleep(0.05)

    def mark(self):
        """Start of the region whose samples count."""
        self.t_begin = time.time()

    def stop(self) -> dict:
        t_end = time.time()
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, r in self.rows:
            if ts < getattr(self, "t_begin", 0.0) or ts > t_end + 0.2:
                continue
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
                for name, val in zip(names, r[4:8]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_decode_sample(wl, budget_s: float):
    """Time the oracle (tables + attention) on whole requests of ``wl`` until ~budget_s is spent."""
    from oracle import mepic_oracle as O
    kp, vp = wl.kv_pool()
    q = wl.decode_q()
    t0 = time.perf_counter()
    st = O.OracleStore(wl.page_size, wl.num_pages, wl.pad_token_id)
    tables = []
    for r in wl.decode_requests:
        segs = [(k, st.register_chunk(wl.chunks[v])[0]) if k == O.KIND_CHUNK else (k, v) for k, v in r.segments]
        tables.append(st.build_block_table(r.request_id, segs))
    t_tables = time.perf_counter() - t0
    done, tokens, t_attn = 0, 0, 0.0
    for b, t in enumerate(tables):
        t1 = time.perf_counter()
        O.decode_attention_one(q[b], kp, vp, t.page_ids, t.pos_base, t.kv_len, t.pos_base[(t.kv_len - 1) // wl.page_size]
                               + (t.kv_len - 1) % wl.page_size, wl.sm_scale, wl.rope_theta)
        t_attn += time.perf_counter() - t1
        done += 1; tokens += t.kv_len
        if t_attn >= budget_s:
            break
    return {"requests": done, "tokens": tokens, "seconds": t_attn, "tables_seconds": t_tables}


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info()]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args.config)
    bpt = kv_bytes_per_token(wl)
    # one step = one whole request of the batch through the oracle (a bounded sample of the workload)
    per_step = []
    total_tokens = 0
    from oracle import mepic_oracle as O
    kp, vp = wl.kv_pool(); q = wl.decode_q()
    st = O.OracleStore(wl.page_size, wl.num_pages, wl.pad_token_id)
    tables = []
    for r in wl.decode_requests:
        segs = [(k, st.register_chunk(wl.chunks[v])[0]) if k == O.KIND_CHUNK else (k, v) for k, v in r.segments]
        tables.append(st.build_block_table(r.request_id, segs))
    for i in range(args.warmup + args.steps):
        b = i % len(tables)
        t = tables[b]
        t1 = time.perf_counter()
        O.decode_attention_one(q[b], kp, vp, t.page_ids, t.pos_base, t.kv_len,
                               t.pos_base[(t.kv_len - 1) // wl.page_size] + (t.kv_len - 1) % wl.page_size,
                               wl.sm_scale, wl.rope_theta)
        dt = time.perf_counter() - t1
        if i >= args.warmup:
            per_step.append(dt); total_tokens += t.kv_len
    secs = sum(per_step)
    value = total_tokens * bpt / secs / 1e9
    cores = cpu_threads()
    sample = f"{args.steps} steps, each one whole request of the batch ({tables[0].kv_len} context tokens) in fp64"
    line = {"impl": "reference", "metric": "rope_fused_paged_decode_effective_hbm_bandwidth", "value": value, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / len(per_step),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config{args.config}:{wl.name}", "sample": sample},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


class L2Flush:
    """Evicts the 126 MB L2 between timed steps: writes a 512 MiB buffer, then reads a second one.

    The read pass pushes the dirty lines of the write pass out to HBM before the start event, so
    their write-back is not charged to the kernel being timed."""

    def __init__(self, device):
        import torch
        self.w = torch.empty(512 << 20, dtype=torch.uint8, device=device)
        self.r = torch.zeros(64 << 20, dtype=torch.int64, device=device)       # 512 MiB, summed without a widening copy
        self.acc = torch.zeros((), dtype=torch.int64, device=device)

    def __call__(self):
        import torch
        self.w.fill_(1)
        torch.sum(self.r, dim=0, out=self.acc)


def measure_grouped(args, wl, dev, page_ids, pos_base, kv_len, q_pos, q_bits, logical_bytes: int):
    """The same decode batch through mepic_attn_decode_grouped: requests that alias a page are scored against it
    together.  Rate = the logical bytes a per-request decode must read / time, so it can exceed the HBM roofline."""
    import torch
    from paper_2512_16822_b200 import runtime as RT
    t0 = time.perf_counter()
    batch = RT.GroupedDecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    setup_ms = 1e3 * (time.perf_counter() - t0)
    t0 = time.perf_counter()
    import paper_2512_16822_b200 as M
    M.mepic_decode_plan_build(dev.cfg, page_ids, pos_base, kv_len)
    plan_ms = 1e3 * (time.perf_counter() - t0)
    stream = torch.cuda.current_stream()
    flush = L2Flush(dev.device)
    for _ in range(3):
        batch.run(wl.sm_scale, stream)
    steps = max(5, min(args.steps, 50))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        flush()
        a.record(stream); batch.run(wl.sm_scale, stream); b.record(stream)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    ms = sum(a.elapsed_time(b) for a, b in evs) / steps
    entries = int(sum(-(-int(k) // wl.page_size) for k in kv_len))
    staged = int(batch.plan_host[12])
    page_bytes = wl.page_size * kv_bytes_per_token(wl)
    return {"value": logical_bytes / (ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms, "steps": steps,
            "table_entries": entries, "pages_staged": staged, "staged_bytes_per_step": staged * page_bytes,
            "staged_gbs": staged * page_bytes / (ms * 1e-3) / 1e9, "plan_build_ms": plan_ms, "plan_ints": int(len(batch.plan_host)),
            "note": "sharing-aware decode (host plan + mepic_attn_decode_grouped); value = logical bytes of the per-request "
                    "decode / time; L2 flushed between steps"}


def measure_fp8(args, wl, dev, page_ids, pos_base, kv_len, q_pos, q_bits):
    """The same decode batch over 8-bit (e4m3) copies of the pools (library quantiser, one scale per page and head)."""
    import torch
    from paper_2512_16822_b200 import runtime as RT
    pools = RT.Fp8Pools(dev)
    batch = RT.Fp8DecodeBatch(pools, page_ids, pos_base, kv_len, q_pos, q_bits)
    stream = torch.cuda.current_stream()
    flush = L2Flush(dev.device)
    for _ in range(3):
        batch.run(wl.sm_scale, stream)
    steps = max(5, min(args.steps, 50))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        flush()
        a.record(stream); batch.run(wl.sm_scale, stream); b.record(stream)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    ms = sum(a.elapsed_time(b) for a, b in evs) / steps
    tokens = int(kv_len.astype(np.int64).sum())
    bytes_per_token = kv_bytes_per_token(wl) // 2
    return {"ms_per_step": ms, "steps": steps, "context_tokens_per_s": tokens / (ms * 1e-3),
            "kv_bytes_per_token": bytes_per_token, "value": tokens * bytes_per_token / (ms * 1e-3) / 1e9, "unit": "GB/s",
            "note": "e4m3 pages + fp32 scale per (page, kv head): half the K/V bytes of bf16 per context token; "
                    "value = 8-bit bytes / time; L2 flushed between steps"}


def measure_unshared(args, wl, device_index: int):
    """The same decode batch on a layout WITHOUT chunk sharing: every request owns a private copy of each of its
    chunks (one page per block-table entry), so no page is read twice and nothing can be served from L2 because a
    neighbour touched it.  Separates kernel quality from the cache effect of sharing."""
    import torch
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
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
    q_pos = kv_len - 1
    dev = RT.Device(cfg, device=f"cuda:{device_index}")
    dev.k_pool.normal_(); dev.v_pool.normal_()             # values do not matter for timing; drawn on the device
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, wl.decode_q())
    stream = torch.cuda.current_stream()
    flush = L2Flush(dev.device)
    for _ in range(3):
        batch.run(wl.sm_scale, stream)
    steps = max(5, min(args.steps, 50))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        flush()
        a.record(stream); batch.run(wl.sm_scale, stream); b.record(stream)
    torch.cuda.synchronize()
    assert dev.read_status() == 0
    ms = sum(a.elapsed_time(b) for a, b in evs) / steps
    nbytes = int(kv_len.astype(np.int64).sum()) * kv_bytes_per_token(wl)
    return {"value": nbytes / (ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms, "pages_held": num_pages,
            "note": "no chunk sharing: logical bytes = unique bytes; L2 flushed between steps"}


def measure_prefill(args, device_index: int):
    """Config 3 (first-block recompute prefill): one step = one mepic_attn_prefill call (commit + attention)."""
    import torch
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
    wl = make_workload(3)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.prefill_requests)
    page_ids, pos_base, kv_len, _ = RT.pack_tables(tables, wl.page_size)
    q_slots = [t.recompute_slots for t in tables]
    rows = [wl.prefill_rows(i, len(t.recompute_slots)) for i, t in enumerate(tables)]
    row_offsets = np.concatenate([[0], np.cumsum([len(s) for s in q_slots])]).astype(np.int32)
    dev = RT.Device(cfg, kp, vp, device=f"cuda:{device_index}")
    pb = RT.PrefillBatch(dev, page_ids, pos_base, kv_len, row_offsets, np.concatenate(q_slots).astype(np.int32),
                         np.concatenate([r.q_new for r in rows]), np.concatenate([r.k_new for r in rows]),
                         np.concatenate([r.v_new for r in rows]))
    stream = torch.cuda.current_stream()
    # unmasked (row, key) pairs only: QK^T and PV, 2 flops per multiply-add
    pairs = sum(int((s.astype(np.int64) + 1).sum()) for s in q_slots)
    flops = 4 * wl.head_dim * wl.n_q_heads * pairs
    for _ in range(3):
        pb.run(wl.sm_scale, stream)
    torch.cuda.synchronize()
    assert dev.read_status() == 0, "device status word is not clean"
    steps = max(5, min(args.steps, 20))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record(stream); pb.run(wl.sm_scale, stream); b.record(stream)
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    mean_ms = sum(ms) / len(ms)
    _, _, peaks = measured_peaks()
    peak = float(peaks.get("bf16_tflops", 1590.0))
    achieved = flops / (mean_ms * 1e-3) / 1e12
    return {"workload": f"config3:{wl.name}", "metric": "first_block_recompute_prefill_tflops", "value": achieved,
            "unit": "TFLOP/s", "ms_per_step": mean_ms, "ms_min": min(ms), "steps": steps, "flops_per_step": flops,
            "rows": int(row_offsets[-1]), "kv_len": int(kv_len[0]), "dtype": "bf16 MMA, fp32 accumulate",
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": achieved / peak, "traffic": None,
                         "peak_source": "measured burst bf16 (MEASURED_PEAKS.json bf16_tflops)" if peaks else "fallback 1590",
                         "kernel": "mepic_prefill_attn (+ commit kernel: the C-ABI call is timed as a whole)"}}


def max_over_ranks(total_ms: float, world: int, device) -> float:
    """The slowest rank's time: every multi-GPU number is the job's bytes over this."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gbs(world: int, steps: int, bytes_per_rank_step: int, total_ms: float) -> float:
    """Whole-job throughput: all ranks' bytes (replicas, weak scaling) over the slowest rank's time."""
    return world * steps * bytes_per_rank_step / (total_ms * 1e-3) / 1e9


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
    from paper_2512_16822_b200.build import build_library

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the MEPIC kernels have no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    build_library()

    wl = make_workload(args.config)
    cfg = M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages, wl.max_position,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    q_bits = wl.decode_q()
    t0 = time.perf_counter()
    with M.Store(cfg) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
        stats = st.stats()
    table_build_ms = 1e3 * (time.perf_counter() - t0)
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    dev = RT.Device(cfg, kp, vp, device=f"cuda:{local_rank}")
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    logical_bytes = int(kv_len.astype(np.int64).sum()) * kv_bytes_per_token(wl)
    stream = torch.cuda.current_stream()
    l2_flush = L2Flush(dev.device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(steps, step_fn, flush):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in evs:
            if flush:
                l2_flush()
            a.record(stream); step_fn(); b.record(stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    step = lambda: batch.run(wl.sm_scale, stream)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert dev.read_status() == 0, "device status word is not clean"

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample()
        sampler.mark()
    launches0 = M.mepic_launch_count()
    barrier()
    ms = timed(args.steps, step, flush=True)
    barrier()
    launches = M.mepic_launch_count() - launches0
    ms_warm = timed(args.steps, step, flush=False)

    # end to end: the step's inputs come from pinned host memory, the result goes back to the host
    # one pinned mirror of the step's inputs (q + block tables + lengths + positions): one copy in, one copy out
    h_in, hv = batch.host_mirror()
    hv["q"].copy_(torch.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)))
    hv["page_ids"].copy_(torch.from_numpy(page_ids)); hv["pos_base"].copy_(torch.from_numpy(pos_base))
    hv["kv_len"].copy_(torch.from_numpy(kv_len)); hv["q_pos"].copy_(torch.from_numpy(q_pos))
    h_out = torch.empty(batch.out.shape, dtype=torch.bfloat16).pin_memory()
    h2d = int(h_in.numel())
    d2h = int(h_out.numel() * h_out.element_size())

    def e2e_step():
        batch.upload(h_in)
        batch.run(wl.sm_scale, stream)
        h_out.copy_(batch.out, non_blocking=True)

    for _ in range(3):
        e2e_step()
    barrier()
    ms_e2e = timed(args.steps, e2e_step, flush=True)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    assert dev.read_status() == 0, "device status word is not clean"

    def agg(xs):
        return max_over_ranks(sum(xs), world, dev.device)

    tot, tot_warm, tot_e2e = agg(ms), agg(ms_warm), agg(ms_e2e)
    prefill = unshared = grouped = fp8 = None
    if rank == 0 and world == 1 and not args.no_fp8 and wl.head_dim == 128:
        fp8 = measure_fp8(args, wl, dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    if rank == 0 and world == 1 and not args.no_grouped:
        grouped = measure_grouped(args, wl, dev, page_ids, pos_base, kv_len, q_pos, q_bits, logical_bytes)
    if rank == 0 and world == 1 and not args.no_prefill:
        prefill = measure_prefill(args, local_rank)
    if rank == 0 and world == 1 and not args.no_unshared:
        unshared = measure_unshared(args, wl, local_rank)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    gbs = lambda total_ms: aggregate_gbs(world, args.steps, logical_bytes, total_ms)
    peak, peak_src, _ = measured_peaks()
    per_launch_ms = sum(ms) / len(ms)
    achieved = logical_bytes / (per_launch_ms * 1e-3) / 1e9
    line = {
        "metric": "rope_fused_paged_decode_effective_hbm_bandwidth", "value": gbs(tot), "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": tot / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"config{args.config}:{wl.name}", "batch": len(tables), "n_q_heads": wl.n_q_heads,
                   "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim, "page_size": wl.page_size,
                   "kv_len_mean": float(kv_len.mean()), "logical_kv_bytes_per_step": logical_bytes,
                   "l2": "flushed between timed steps (512 MiB written, then 512 MiB of another buffer read so no dirty "
                         "line is left to write back inside the timed region); value_no_flush is the same loop without it",
                   "parallelism": "replicas" if world > 1 else "single"},
        "value_no_flush": gbs(tot_warm), "ms_per_step_no_flush": tot_warm / args.steps,
        "e2e": {"value": gbs(tot_e2e), "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": tot_e2e / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(args.config), "peak_source": peak_src,
                     "kernel": "mepic_decode_splitkv (+ its merge kernel: the C-ABI call is timed as a whole)",
                     "algorithmic_bytes_per_launch": logical_bytes, "frac_of_nominal_8TBs": achieved / 8000.0},
        "pages": {"held": stats["pages_shared_held"] + stats["pages_private_held"],
                  "shared": stats["pages_shared_held"], "private": stats["pages_private_held"],
                  "unshared_equivalent": stats["unshared_equivalent_pages"], "dedup_hits": stats["dedup_hits"]},
        "table_build_ms": table_build_ms,
        "prefill": prefill,
        "unshared_layout": unshared,
        "grouped_decode": grouped,
        "fp8_decode": fp8,
    }
    if not args.no_cpu_baseline and world == 1:
        s = oracle_decode_sample(wl, args.cpu_budget)
        line["cpu_baseline"] = {"value": s["tokens"] * kv_bytes_per_token(wl) / s["seconds"] / 1e9, "unit": "GB/s",
                                "cores": cpu_threads(), "kind": "oracle",
                                "sample": f"{s['requests']} whole requests ({s['tokens']} context tokens) of the same batch, "
                                          f"fp64 numpy, {s['seconds']:.1f} s; table build for the full batch {s['tables_seconds']*1e3:.1f} ms"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 4, 5])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the config-3 prefill measurement")
    ap.add_argument("--no-unshared", action="store_true", help="skip the decode run on the layout without sharing")
    ap.add_argument("--no-grouped", action="store_true", help="skip the sharing-aware (grouped) decode run")
    ap.add_argument("--no-fp8", action="store_true", help="skip the decode run over 8-bit pages")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
