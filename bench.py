#!/usr/bin/env python
"""Benchmark of the MEPIC hot path on B200: RoPE-fused paged-attention decode (HBM GB/s) and
first-block-recompute prefill (TFLOP/s), on the five synthetic configurations.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]
    python bench.py --leg prefill --config 3 --scale 0.5 --steps 2 --warmup 1     # one leg alone (profiling)

Headline.  One "step" is one pass of the decode hot path over one batch: a call of ``mepic_attn_decode``
(split-KV kernel + merge kernel) on the configuration the metric is quoted on (config 2, the Llama-3-8B-shaped
decode layer).  ``value`` is the effective bandwidth = logical K/V bytes the batch must read / device time, with
every input already resident in HBM and the L2 flushed between timed steps.  ``e2e`` is the same call with the
step's inputs (q and the block tables) coming from pinned host memory and the result read back, copies inside the
timed region; the K/V pool is the cache itself and stays resident.  Exactly K steps are timed for the headline; a
second, longer run of the same step (at least half a second of device time) gives the clock sampler something to
see and a median / minimum per step.

``configs`` holds the other configurations through the same C-ABI calls: decode on configs 1, 4 and 5 (shared and
unshared layout, end to end, error against an oracle sample, one negative control), prefill on configs 3 and 5,
and config 5 as one serving step (decode and prefill together).

Under torchrun every rank runs its own replica of the headline batch on its own GPU (requests are independent: no
data-path collective); the aggregate is all ranks' bytes over the slowest rank's time.

``--impl reference`` times the CPU oracle, as it stands, on the host cores (rank 0 only) on a bounded sample of
the same workload.
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
FALLBACK_BF16_TFLOPS = 1590.0
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
MAX_ABS, MEAN_ABS = 2e-2, 2e-3
METRIC = "rope_fused_paged_decode_effective_hbm_bandwidth"
L2_NOTE = ("flushed between timed steps (512 MiB written, then 512 MiB of another buffer read so no dirty line is "
           "left to write back inside the timed region); value_no_flush is the same loop without it")


def kv_bytes_per_token(wl) -> int:
    """Algorithmic bytes per context token: K and V, all KV heads, bf16."""
    return 2 * wl.n_kv_heads * wl.head_dim * 2


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)", d
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, an earlier measurement)", {}


def ncu_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of ``kernel`` on ``workload`` from the tracked ncu summary (profiles/traffic.json),
    with the capture it came from; None when there is no capture of that pair."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as f:
            for row in json.load(f)["captures"]:
                if row["kernel"] == kernel and row["workload"] == workload:
                    return row
    except Exception:
        pass
    return None


def config_dict(index: int, wl, kv_len, world: int) -> dict:
    """The ``config`` object of the JSON line; both arms print the same keys and values."""
    kv = np.asarray(kv_len, dtype=np.int64)
    return {"workload": f"config{index}:{wl.name}", "batch": int(len(kv)), "n_q_heads": wl.n_q_heads,
            "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim, "page_size": wl.page_size,
            "kv_len_mean": float(kv.mean()), "logical_kv_bytes_per_step": int(kv.sum()) * kv_bytes_per_token(wl),
            "l2": L2_NOTE, "parallelism": "replicas" if world > 1 else "single"}


# ---------------------------------------------------------------- clocks during the timed regions
class ClockSampler:
    """Samples SM clock and throttle reasons every few milliseconds through NVML (read-only queries) while the timed
    regions run; falls back to polling nvidia-smi.  Only samples taken inside a marked window count."""
    PERIOD_S = 0.002

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []              # (time, sm_mhz, sm_max_mhz, reasons bitmask or list)
        self.windows = []
        self._stop = threading.Event()
        self.thread = None
        self.how = None

    def _nvml_loop(self, nv, h):
        smax = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop.is_set():
            try:
                self.rows.append((time.time(), float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)), float(smax),
                                  int(get_reasons(h))))
            except Exception:
                pass
            time.sleep(self.PERIOD_S)

    def _smi_loop(self):
        fields = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                  "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={fields}", "--format=csv,noheader,nounits",
                                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        self._proc = proc
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in proc.stdout:
            r = [x.strip() for x in line.split(",")]
            try:
                self.rows.append((time.time(), float(r[0]), float(r[1]),
                                  [n for n, v in zip(names, r[2:6]) if v.lower().startswith("active")]))
            except Exception:
                continue

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            # the CUDA device of this rank, found in NVML by its PCI address (NVML's indices need not match CUDA's)
            h = None
            try:
                import torch
                pr = torch.cuda.get_device_properties(self.gpu)
                h = nv.nvmlDeviceGetHandleByPciBusId(f"{pr.pci_domain_id:08X}:{pr.pci_bus_id:02X}:{pr.pci_device_id:02X}.0".encode())
            except Exception:
                h = None
            if h is None:
                h = nv.nvmlDeviceGetHandleByIndex(self.gpu)
            nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
            self.how = "nvml, every 2 ms"
            self._nv = nv
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, h), daemon=True)
            self.thread.start()
            return
        except Exception:
            pass
        try:
            self.how = "nvidia-smi -lms 20"
            self.thread = threading.Thread(target=self._smi_loop, daemon=True)
            self.thread.start()
        except Exception:
            self.how = None

    def wait_first_sample(self, timeout_s: float = 5.0):
        t0 = time.time()
        while self.how and not self.rows and time.time() - t0 < timeout_s:
            time.sleep(0.01)

    def window(self, name: str):
        sampler = self

        class _W:
            def __enter__(self_w):
                self_w.t0 = time.time()

            def __exit__(self_w, *exc):
                sampler.windows.append((name, self_w.t0, time.time()))
        return _W()

    def stop(self) -> dict:
        self._stop.set()
        proc = getattr(self, "_proc", None)
        if proc is not None:
            proc.terminate()
        if self.how is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source available"], "samples": 0}
        bits = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "sw_power_cap": 0x4}
        sm, smax, reasons, per_window = [], [], set(), {}
        for ts, mhz, mx, rs in list(self.rows):
            for name, t0, t1 in self.windows:
                if t0 <= ts <= t1:
                    sm.append(mhz); smax.append(mx)
                    per_window[name] = per_window.get(name, 0) + 1
                    if isinstance(rs, int):
                        reasons.update(n for n, b in bits.items() if rs & b)
                    else:
                        reasons.update(rs)
                    break
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons), "samples": len(sm),
                "samples_per_region": per_window, "source": self.how}


# ---------------------------------------------------------------- the oracle legs (CPU)
def oracle_tables(wl, requests):
    from oracle import mepic_oracle as O
    st = O.OracleStore(wl.page_size, wl.num_pages, wl.pad_token_id)
    tables = []
    for r in requests:
        segs = [(k, st.register_chunk(wl.chunks[v])[0]) if k == O.KIND_CHUNK else (k, v) for k, v in r.segments]
        tables.append(st.build_block_table(r.request_id, segs))
    return tables


def oracle_decode_one(wl, kp, vp, q, t, b, **kw):
    from oracle import mepic_oracle as O
    last = t.kv_len - 1
    q_pos = t.pos_base[last // wl.page_size] + last % wl.page_size
    return O.decode_attention_one(q[b], kp, vp, t.page_ids, t.pos_base, t.kv_len, q_pos, wl.sm_scale, wl.rope_theta, **kw)


def oracle_decode_sample(wl, budget_s: float):
    """Time the oracle (tables + attention) on whole requests of ``wl`` until ~budget_s is spent."""
    kp, vp = wl.kv_pool()
    q = wl.decode_q()
    t0 = time.perf_counter()
    tables = oracle_tables(wl, wl.decode_requests)
    t_tables = time.perf_counter() - t0
    done, tokens, t_attn = 0, 0, 0.0
    for b, t in enumerate(tables):
        t1 = time.perf_counter()
        oracle_decode_one(wl, kp, vp, q, t, b)
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
    kp, vp = wl.kv_pool(); q = wl.decode_q()
    tables = oracle_tables(wl, wl.decode_requests)
    for i in range(args.warmup + args.steps):
        b = i % len(tables)
        t1 = time.perf_counter()
        oracle_decode_one(wl, kp, vp, q, tables[b], b)
        dt = time.perf_counter() - t1
        if i >= args.warmup:
            per_step.append(dt); total_tokens += tables[b].kv_len
    secs = sum(per_step)
    value = total_tokens * bpt / secs / 1e9
    cores = cpu_threads()
    sample = f"{args.steps} steps, each one whole request of the batch ({tables[0].kv_len} context tokens) in fp64"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / len(per_step),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(args.config, wl, [t.kv_len for t in tables], 1),
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------- GPU set-up shared by every leg
class L2Flush:
    """Evicts the 126 MB L2 between timed steps: writes a 512 MiB buffer, then reads a second one.

    The read pass pushes the dirty lines of the write pass out to HBM before the start event, so
    their write-back is not charged to the kernel being timed."""
    _cache = {}

    def __init__(self, device):
        import torch
        key = str(device)
        if key not in L2Flush._cache:
            L2Flush._cache[key] = (torch.empty(512 << 20, dtype=torch.uint8, device=device),
                                   torch.zeros(64 << 20, dtype=torch.int64, device=device),   # 512 MiB, summed in place
                                   torch.zeros((), dtype=torch.int64, device=device))
        self.w, self.r, self.acc = L2Flush._cache[key]

    def __call__(self):
        import torch
        self.w.fill_(1)
        torch.sum(self.r, dim=0, out=self.acc)


def time_steps(step_fn, steps: int, flush, stream):
    """CUDA events on the launching stream around each step; the flush runs outside the events."""
    import torch
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        if flush is not None:
            flush()
        a.record(stream); step_fn(); b.record(stream)
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def summary(ms):
    return {"ms_per_step": sum(ms) / len(ms), "ms_median": statistics.median(ms), "ms_min": min(ms), "steps": len(ms)}


def make_config(wl, num_pages=None):
    import paper_2512_16822_b200 as M
    return M.Config(wl.page_size, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages if num_pages is None else num_pages,
                    wl.max_position, wl.rope_theta, wl.pad_token_id)


def shared_layout(wl, device: str):
    """Store -> block tables of the workload's requests; pools filled from the workload's seeded K/V."""
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
    cfg = make_config(wl)
    t0 = time.perf_counter()
    with M.Store(cfg) as st:
        dec = RT.build_tables(st, wl.chunks, wl.decode_requests) if wl.decode_requests else []
        pre = RT.build_tables(st, wl.chunks, wl.prefill_requests) if wl.prefill_requests else []
        stats = st.stats()
    build_ms = 1e3 * (time.perf_counter() - t0)
    kp, vp = wl.kv_pool()
    dev = RT.Device(cfg, kp, vp, device=device)
    return {"cfg": cfg, "dev": dev, "decode_tables": dec, "prefill_tables": pre, "stats": stats, "table_build_ms": build_ms,
            "kp": kp, "vp": vp}


def unshared_layout(wl, device: str):
    """The decode batch on a layout WITHOUT chunk sharing: every request owns a private copy of each of its chunks
    (one page per block-table entry), so no page is read twice and nothing can be served from L2 because a
    neighbour touched it.  Separates kernel quality from the cache effect of sharing.  Pool values are drawn on the
    device (they do not matter for timing)."""
    from paper_2512_16822_b200 import runtime as RT
    P = wl.page_size
    ents = [sum(-(-(len(wl.chunks[v]) if k == 0 else v) // P) for k, v in r.segments) for r in wl.decode_requests]
    lens = [sum((len(wl.chunks[v]) if k == 0 else v) for k, v in r.segments) for r in wl.decode_requests]
    num_pages = int(sum(ents))
    cfg = make_config(wl, num_pages)
    B, stride = len(ents), max(ents)
    page_ids = np.zeros((B, stride), dtype=np.int32); pos_base = np.zeros((B, stride), dtype=np.int32)
    perm = np.random.default_rng([0, wl.index, 99]).permutation(num_pages).astype(np.int32)
    at = 0
    for b, e in enumerate(ents):
        page_ids[b, :e] = perm[at:at + e]; at += e
        pos_base[b, :e] = np.arange(e) * P
    kv_len = np.asarray(lens, dtype=np.int32)
    dev = RT.Device(cfg, device=device)
    dev.k_pool.normal_(); dev.v_pool.normal_()
    return dev, page_ids, pos_base, kv_len, (kv_len - 1).astype(np.int32)


def decode_batch(kind: str, dev, page_ids, pos_base, kv_len, q_pos, q_bits):
    from paper_2512_16822_b200 import runtime as RT
    if kind == "fp8":
        return RT.Fp8DecodeBatch(RT.Fp8Pools(dev), page_ids, pos_base, kv_len, q_pos, q_bits)
    if kind == "grouped":
        return RT.GroupedDecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    return RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q_bits)


def prefill_batch(wl, dev, tables):
    from paper_2512_16822_b200 import runtime as RT
    page_ids, pos_base, kv_len, _ = RT.pack_tables(tables, wl.page_size)
    q_slots = [np.asarray(t.recompute_slots) for t in tables]
    rows = [wl.prefill_rows(i, len(s)) for i, s in enumerate(q_slots)]
    row_offsets = np.concatenate([[0], np.cumsum([len(s) for s in q_slots])]).astype(np.int32)
    pb = RT.PrefillBatch(dev, page_ids, pos_base, kv_len, row_offsets, np.concatenate(q_slots).astype(np.int32),
                         np.concatenate([r.q_new for r in rows]), np.concatenate([r.k_new for r in rows]),
                         np.concatenate([r.v_new for r in rows]))
    # unmasked (row, key) pairs only: QK^T and PV, 2 flops per multiply-add
    pairs = sum(int((s.astype(np.int64) + 1).sum()) for s in q_slots)
    flops = 4 * wl.head_dim * wl.n_q_heads * pairs
    return pb, flops, q_slots, rows, (page_ids, pos_base, kv_len, row_offsets)


def rates_gbs(nbytes: int, ms: float, peak: float) -> dict:
    g = nbytes / (ms * 1e-3) / 1e9
    return {"value": g, "unit": "GB/s", "frac_of_measured": g / peak, "frac_of_nominal_8TBs": g / NOMINAL_HBM_GBS}


def error_figures(got, want) -> dict:
    d = np.abs(got - want)
    return {"max_abs": float(d.max()), "mean_abs": float(d.mean()),
            "rel_l2": float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))}


# ---------------------------------------------------------------- decode on one configuration
def decode_error(wl, lay, out_bits, sample) -> dict:
    """Measured error of the GPU result against the oracle on whole sampled requests, plus one negative control:
    the oracle without rotation must be further from the GPU result than the tolerance allows."""
    from mepic_inputs import bf16_bits_to_f64
    got = bf16_bits_to_f64(out_bits)
    q = wl.decode_q()
    tables = oracle_tables(wl, wl.decode_requests)
    g, w, nr = [], [], []
    for b in sample:
        g.append(got[b]); w.append(oracle_decode_one(wl, lay["kp"], lay["vp"], q, tables[b], b))
        nr.append(oracle_decode_one(wl, lay["kp"], lay["vp"], q, tables[b], b, rotate=False))
    g, w, nr = np.stack(g), np.stack(w), np.stack(nr)
    e = error_figures(g, w)
    neg = error_figures(g, nr)
    e.update({"sample": f"requests {list(sample)} of {len(tables)} against the fp64 oracle, all heads and dims",
              "within_tolerance": bool(e["max_abs"] <= MAX_ABS and e["mean_abs"] <= MEAN_ABS),
              "negative_control": {"what": "oracle with the rotation left out", "max_abs": neg["max_abs"],
                                   "mean_abs": neg["mean_abs"], "rel_l2": neg["rel_l2"],
                                   "fails_tolerance": bool(neg["max_abs"] > MAX_ABS or neg["mean_abs"] > MEAN_ABS)}})
    return e


def fp8_decode_error(wl, lay, pools, tabs, out, grouped_out, b: int = 0) -> dict:
    """8-bit pages: the oracle quantises the pages request ``b`` reads from the bf16 pool (the library's codes and scales
    for them must agree bit for bit) and evaluates the request on those codes and scales; error figures of the
    per-request and of the sharing-aware 8-bit decode against it."""
    import torch
    from mepic_inputs import bf16_bits_to_f64
    from oracle import mepic_oracle as O
    from paper_2512_16822_b200 import runtime as RT
    page_ids, pos_base, kv_len, q_pos = tabs
    n = -(-int(kv_len[b]) // wl.page_size)
    mine = np.unique(page_ids[b, :n])
    okc, oks = O.quantize_pages(lay["kp"][mine]); ovc, ovs = O.quantize_pages(lay["vp"][mine])
    sel = torch.from_numpy(mine.astype(np.int64)).to(pools.k_codes.device)
    same = bool(np.array_equal(pools.k_codes[sel].cpu().numpy(), okc) and np.array_equal(pools.k_scales[sel].cpu().numpy(), oks) and
                np.array_equal(pools.v_codes[sel].cpu().numpy(), ovc) and np.array_equal(pools.v_scales[sel].cpu().numpy(), ovs))
    local = {int(pg): i for i, pg in enumerate(mine)}
    ids = [local[int(pg)] for pg in page_ids[b, :n]]
    want = O.decode_attention_one(wl.decode_q()[b], O.dequantize_pages(okc, oks), O.dequantize_pages(ovc, ovs), ids, list(pos_base[b, :n]),
                                  int(kv_len[b]), int(q_pos[b]), wl.sm_scale, wl.rope_theta)
    e = error_figures(bf16_bits_to_f64(RT.bf16_bits(out))[b], want)
    g = error_figures(bf16_bits_to_f64(RT.bf16_bits(grouped_out))[b], want)
    e.update({"sample": f"request {b} against the fp64 oracle evaluated on the oracle's own codes and scales of the {len(mine)} pages it reads",
              "codes_and_scales_bit_exact": same,
              "within_tolerance": bool(same and e["max_abs"] <= MAX_ABS and e["mean_abs"] <= MEAN_ABS),
              "grouped": {**g, "within_tolerance": bool(g["max_abs"] <= MAX_ABS and g["mean_abs"] <= MEAN_ABS)}})
    return e


def decode_legs(index: int, args, device: str, peak: float, *, scale=1.0, kinds=("plain", "unshared", "e2e", "error")):
    """Decode of one configuration through mepic_attn_decode: shared layout (flushed / not), unshared layout, end to
    end, error figures.  Returns the per-config object."""
    import torch
    import paper_2512_16822_b200 as M
    from paper_2512_16822_b200 import runtime as RT
    wl = make_workload(index, scale=scale)
    lay = shared_layout(wl, device)
    dev = lay["dev"]
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(lay["decode_tables"], wl.page_size)
    q_bits = wl.decode_q()
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    stream = torch.cuda.current_stream()
    flush = L2Flush(dev.device)
    nbytes = int(kv_len.astype(np.int64).sum()) * kv_bytes_per_token(wl)
    steps = max(5, min(args.steps, 50))
    step = lambda: batch.run(wl.sm_scale, stream)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    assert dev.read_status() == 0, "device status word is not clean"
    out = {"workload": f"config{index}:{wl.name}", "batch": len(kv_len), "kv_len_mean": float(kv_len.mean()),
           "kv_len_max": int(kv_len.max()), "logical_kv_bytes_per_step": nbytes,
           "pages": {"held": lay["stats"]["pages_shared_held"] + lay["stats"]["pages_private_held"],
                     "unshared_equivalent": lay["stats"]["unshared_equivalent_pages"]},
           "table_build_ms": lay["table_build_ms"]}
    ms = time_steps(step, steps, flush, stream)
    d = summary(ms); d.update(rates_gbs(nbytes, d["ms_per_step"], peak))
    d["note"] = "shared layout: effective rate (logical bytes; repeats of shared pages may come from L2)"
    out["decode"] = d
    ms = time_steps(step, steps, None, stream)
    out["decode"]["ms_per_step_no_flush"] = sum(ms) / len(ms)
    if "e2e" in kinds:
        h_in, hv = batch.host_mirror()
        hv["q"].copy_(torch.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)))
        hv["page_ids"].copy_(torch.from_numpy(page_ids)); hv["pos_base"].copy_(torch.from_numpy(pos_base))
        hv["kv_len"].copy_(torch.from_numpy(kv_len)); hv["q_pos"].copy_(torch.from_numpy(q_pos))
        h_out = torch.empty(batch.out.shape, dtype=torch.bfloat16).pin_memory()

        def e2e_step():
            batch.upload(h_in)
            batch.run(wl.sm_scale, stream)
            h_out.copy_(batch.out, non_blocking=True)
        for _ in range(3):
            e2e_step()
        ms = time_steps(e2e_step, steps, flush, stream)
        d = summary(ms); d.update(rates_gbs(nbytes, d["ms_per_step"], peak))
        d.update({"h2d_bytes_per_step": int(h_in.numel()), "d2h_bytes_per_step": int(h_out.numel() * h_out.element_size())})
        out["e2e"] = d
    if "error" in kinds:
        batch.run(wl.sm_scale, stream); torch.cuda.synchronize()
        B = len(kv_len)
        sample = sorted({0, B // 2, B - 1}) if index != 4 else [0, B - 1]
        out["error"] = decode_error(wl, lay, RT.bf16_bits(batch.out), sample)
    assert dev.read_status() == 0, "device status word is not clean"
    del batch, dev, lay
    torch.cuda.empty_cache()
    if "unshared" in kinds:
        udev, uids, ubase, ukv, uqpos = unshared_layout(wl, device)
        ub = RT.DecodeBatch(udev, uids, ubase, ukv, uqpos, q_bits)
        ustep = lambda: ub.run(wl.sm_scale, stream)
        for _ in range(3):
            ustep()
        ms = time_steps(ustep, steps, flush, stream)
        assert udev.read_status() == 0
        d = summary(ms); d.update(rates_gbs(nbytes, d["ms_per_step"], peak))
        d.update({"pages_held": int(udev.cfg.num_pages),
                  "note": "no chunk sharing: logical bytes = unique bytes, every byte comes from DRAM; L2 flushed between steps"})
        out["unshared_layout"] = d
        del ub, udev
        torch.cuda.empty_cache()
    return out


# ---------------------------------------------------------------- prefill on one configuration
def prefill_error(wl, lay, pb, q_slots, rows, tabs, n_rows=12) -> dict:
    """Error of sampled rows of request 0 against the oracle, the committed pages bit for bit, and one negative
    control (oracle with every position base zeroed)."""
    from mepic_inputs import bf16_bits_to_f64
    from oracle import mepic_oracle as O
    from paper_2512_16822_b200 import runtime as RT
    page_ids, pos_base, kv_len, row_offsets = tabs
    R = len(q_slots[0])
    pick = sorted(set(np.linspace(0, R - 1, n_rows).astype(int).tolist()))
    okp, ovp = lay["kp"].copy(), lay["vp"].copy()
    ne = -(-int(kv_len[0]) // wl.page_size)
    args = (rows[0].q_new, rows[0].k_new, rows[0].v_new, list(q_slots[0]), okp, ovp, list(page_ids[0][:ne]))
    want = O.prefill_attention_one(*args, list(pos_base[0][:ne]), int(kv_len[0]), wl.sm_scale, wl.rope_theta, rows=pick)
    wrong = O.prefill_attention_one(*args, [0] * ne, int(kv_len[0]), wl.sm_scale, wl.rope_theta, rows=pick)
    got = bf16_bits_to_f64(RT.bf16_bits(pb.out[:R]))[pick]
    e = error_figures(got, want)
    neg = error_figures(got, wrong)
    touched = sorted({int(page_ids[0][s // wl.page_size]) for s in q_slots[0]})
    kbits, vbits = RT.bf16_bits(pb.dev.k_pool[touched]), RT.bf16_bits(pb.dev.v_pool[touched])
    e.update({"sample": f"{len(pick)} of the {R} rows of request 0 (first to last), all heads and dims, against the fp64 oracle",
              "within_tolerance": bool(e["max_abs"] <= MAX_ABS and e["mean_abs"] <= MEAN_ABS),
              "committed_pages_bit_exact": bool(np.array_equal(kbits, okp[touched]) and np.array_equal(vbits, ovp[touched])),
              "negative_control": {"what": "oracle with every position base set to zero", "max_abs": neg["max_abs"],
                                   "mean_abs": neg["mean_abs"], "rel_l2": neg["rel_l2"],
                                   "fails_tolerance": bool(neg["max_abs"] > MAX_ABS or neg["mean_abs"] > MEAN_ABS)}})
    return e


def prefill_error_fp8(wl, lay, pools, pb, q_slots, rows, tabs, n_rows=12) -> dict:
    """8-bit pages: the oracle quantises the pages request 0 reads from the bf16 pool, commits request 0's rows into
    them by its own rule (codes and scales of those pages must then equal the library's bit for bit) and evaluates
    sampled rows on those codes and scales."""
    import torch
    from mepic_inputs import bf16_bits_to_f64
    from oracle import mepic_oracle as O
    from paper_2512_16822_b200 import runtime as RT
    page_ids, pos_base, kv_len, row_offsets = tabs
    ne = -(-int(kv_len[0]) // wl.page_size)
    mine = np.unique(page_ids[0][:ne])
    okc, oks = O.quantize_pages(lay["kp"][mine]); ovc, ovs = O.quantize_pages(lay["vp"][mine])
    local = {int(pg): i for i, pg in enumerate(mine)}
    ids0 = [local[int(pg)] for pg in page_ids[0][:ne]]
    O.commit_rows_fp8(okc, oks, ovc, ovs, ids0, list(q_slots[0]), rows[0].k_new, rows[0].v_new)
    sel = torch.from_numpy(mine.astype(np.int64)).to(pools.k_codes.device)
    same = bool(np.array_equal(pools.k_codes[sel].cpu().numpy(), okc) and np.array_equal(pools.k_scales[sel].cpu().numpy(), oks) and
                np.array_equal(pools.v_codes[sel].cpu().numpy(), ovc) and np.array_equal(pools.v_scales[sel].cpu().numpy(), ovs))
    R = len(q_slots[0])
    pick = sorted(set(np.linspace(0, R - 1, n_rows).astype(int).tolist()))
    want = O.prefill_attention_one(rows[0].q_new, rows[0].k_new, rows[0].v_new, list(q_slots[0]), O.dequantize_pages(okc, oks),
                                   O.dequantize_pages(ovc, ovs), ids0, list(pos_base[0][:ne]), int(kv_len[0]), wl.sm_scale, wl.rope_theta, rows=pick)
    e = error_figures(bf16_bits_to_f64(RT.bf16_bits(pb.out[:R]))[pick], want)
    e.update({"sample": f"{len(pick)} of the {R} rows of request 0 (first to last), all heads and dims, against the fp64 oracle "
                        f"evaluated on the oracle's own codes and scales of the {len(mine)} pages the request reads",
              "committed_codes_and_scales_bit_exact": same,
              "within_tolerance": bool(same and e["max_abs"] <= MAX_ABS and e["mean_abs"] <= MEAN_ABS)})
    return e


def prefill_leg(index: int, args, device: str, *, scale=1.0, error=True, lay=None, fp8=False):
    """One step = one mepic_attn_prefill call (commit + attention) over the configuration's prefill requests.
    fp8: the same requests over 8-bit (e4m3) pools made from the workload's pool by the library's quantiser, the
    bf16 pools freed before the run (mepic_attn_prefill_fp8: commits codes, attends over codes)."""
    import torch
    from paper_2512_16822_b200 import runtime as RT
    wl = make_workload(index, scale=scale)
    lay = lay or shared_layout(wl, device)
    dev = lay["dev"]
    pb, flops, q_slots, rows, tabs = prefill_batch(wl, dev, lay["prefill_tables"])
    if fp8:
        pools = RT.Fp8Pools(dev)
        torch.cuda.synchronize()
        dev.k_pool = dev.v_pool = None                   # from here on the 8-bit pools are the only pools
        torch.cuda.empty_cache()
        pb8 = RT.Fp8PrefillBatch(pools, *tabs[:3], tabs[3], np.concatenate(q_slots).astype(np.int32),
                                 np.concatenate([r.q_new for r in rows]), np.concatenate([r.k_new for r in rows]),
                                 np.concatenate([r.v_new for r in rows]))
        del pb
        pb = pb8
        error8, error = error, False
    stream = torch.cuda.current_stream()
    for _ in range(3):
        pb.run(wl.sm_scale, stream)
    torch.cuda.synchronize()
    assert dev.read_status() == 0, "device status word is not clean"
    steps = max(5, min(args.steps, 20))
    ms = time_steps(lambda: pb.run(wl.sm_scale, stream), steps, None, stream)
    _, _, peaks = measured_peaks()
    burst = float(peaks.get("bf16_tflops", FALLBACK_BF16_TFLOPS))
    sustained = float(peaks.get("bf16_tflops_sustained", 0.0)) or None
    d = summary(ms)
    achieved = flops / (d["ms_per_step"] * 1e-3) / 1e12
    tr = ncu_traffic("mepic_prefill_attn", f"config{index}")
    d.update({"workload": f"config{index}:{wl.name}", "metric": "first_block_recompute_prefill_tflops", "value": achieved,
              "unit": "TFLOP/s", "flops_per_step": flops, "rows": int(tabs[3][-1]), "requests": len(q_slots),
              "kv_len": int(tabs[2][0]), "dtype": "bf16 MMA, fp32 accumulate",
              "l2": "not flushed: a step reads far more than L2 holds only through the shared pages; the bound is the tensor pipe",
              "roofline": {"bound": "tensor", "achieved": achieved, "peak": burst, "unit": "TFLOP/s",
                           "frac": achieved / burst, "frac_of_sustained": achieved / sustained if sustained else None,
                           "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                           "traffic": tr["dram_bytes_per_launch"] if tr else None, "traffic_source": tr,
                           "peak_source": "measured burst bf16 (MEASURED_PEAKS.json bf16_tflops)" if peaks else "fallback 1590",
                           "kernel": "mepic_prefill_attn (+ commit kernel: the C-ABI call is timed as a whole)"}})
    if fp8:
        bpt = kv_bytes_per_token(wl) // 2
        d.update({"metric": "first_block_recompute_prefill_tflops_8bit_pages",
                  "pages_per_GB": int(1e9 // (wl.page_size * bpt + 2 * wl.n_kv_heads * 4)),
                  "pages_per_GB_bf16": int(1e9 // (wl.page_size * kv_bytes_per_token(wl))),
                  "note": "e4m3 pages + one fp32 scale per (page, kv head); no bf16 copy of the pool on the device; "
                          "more shapes, appends and a NaN element in tests/test_fp8_end_to_end_gpu.py"})
        d["roofline"]["kernel"] = "mepic_prefill_attn, 8-bit pages (+ commit kernel: the C-ABI call is timed as a whole)"
        d["roofline"]["traffic"] = None; d["roofline"]["traffic_source"] = None
        if error8:
            d["error"] = prefill_error_fp8(wl, lay, pools, pb, q_slots, rows, tabs)
    if error:
        d["error"] = prefill_error(wl, lay, pb, q_slots, rows, tabs)
    return d, lay, pb


# ---------------------------------------------------------------- the other decode paths on the headline batch
def measure_variant(kind: str, args, wl, dev, tabs, q_bits, logical_bytes: int, peak: float, lay=None):
    """The headline batch through mepic_attn_decode_grouped ("grouped") or mepic_attn_decode_fp8 ("fp8")."""
    import torch
    import paper_2512_16822_b200 as M
    page_ids, pos_base, kv_len, q_pos = tabs
    batch = decode_batch(kind, dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    stream = torch.cuda.current_stream()
    flush = L2Flush(dev.device)
    for _ in range(3):
        batch.run(wl.sm_scale, stream)
    steps = max(5, min(args.steps, 50))
    ms = time_steps(lambda: batch.run(wl.sm_scale, stream), steps, flush, stream)
    assert dev.read_status() == 0
    d = summary(ms)
    tokens = int(kv_len.astype(np.int64).sum())
    if kind == "grouped":
        t0 = time.perf_counter()
        M.mepic_decode_plan_build(dev.cfg, page_ids, pos_base, kv_len)
        plan_ms = 1e3 * (time.perf_counter() - t0)
        staged = int(batch.plan_host[12])
        page_bytes = wl.page_size * kv_bytes_per_token(wl)
        d.update({"value": logical_bytes / (d["ms_per_step"] * 1e-3) / 1e9, "unit": "GB/s",
                  "table_entries": int(sum(-(-int(k) // wl.page_size) for k in kv_len)), "pages_staged": staged,
                  "staged_bytes_per_step": staged * page_bytes,
                  "staged_gbs": staged * page_bytes / (d["ms_per_step"] * 1e-3) / 1e9,
                  "staged_frac_of_measured": staged * page_bytes / (d["ms_per_step"] * 1e-3) / 1e9 / peak,
                  "plan_build_ms": plan_ms, "plan_ints": int(len(batch.plan_host)),
                  "note": "sharing-aware decode (host plan + mepic_attn_decode_grouped); value = logical bytes of the "
                          "per-request decode / time; staged = bytes the kernel actually brings on chip; L2 flushed between steps"})
    else:
        bpt = kv_bytes_per_token(wl) // 2
        d.update({"context_tokens_per_s": tokens / (d["ms_per_step"] * 1e-3), "kv_bytes_per_token": bpt,
                  "value": tokens * bpt / (d["ms_per_step"] * 1e-3) / 1e9, "unit": "GB/s",
                  "frac_of_measured": tokens * bpt / (d["ms_per_step"] * 1e-3) / 1e9 / peak,
                  "pages_per_GB": int(1e9 // (wl.page_size * bpt + 2 * wl.n_kv_heads * 4)),
                  "pages_per_GB_bf16": int(1e9 // (wl.page_size * kv_bytes_per_token(wl))),
                  "note": "e4m3 pages + fp32 scale per (page, kv head): half the K/V bytes of bf16 per context token; "
                          "value = 8-bit bytes / time; L2 flushed between steps"})
        # the sharing-aware path over the same 8-bit pools
        from paper_2512_16822_b200 import runtime as RT
        gb = RT.Fp8GroupedDecodeBatch(batch.pools, page_ids, pos_base, kv_len, q_pos, q_bits)
        for _ in range(3):
            gb.run(wl.sm_scale, stream)
        gms = summary(time_steps(lambda: gb.run(wl.sm_scale, stream), steps, flush, stream))
        assert dev.read_status() == 0
        staged = int(gb.plan_host[12]) * wl.page_size * bpt
        gms.update({"value": tokens * bpt / (gms["ms_per_step"] * 1e-3) / 1e9, "unit": "GB/s",
                    "staged_gbs": staged / (gms["ms_per_step"] * 1e-3) / 1e9,
                    "note": "mepic_attn_decode_grouped_fp8: value = 8-bit bytes of the per-request decode / time"})
        d["grouped"] = gms
        if lay is not None:
            d["error"] = fp8_decode_error(wl, lay, batch.pools, tabs, batch.out, gb.out)
        del gb
    del batch
    return d


def measure_decode_loop(args, device: str, index: int = 2, n_steps: int = 64):
    """A decode loop as a serving system runs it: n_steps consecutive steps of the batch, every request one token
    longer each step (page gains included), the step's inputs from pinned host memory, the result read back and
    waited for before the next step.  Once through mepic_attn_decode (q, lengths, positions every step; the block
    tables again whenever a request gained a page) and once through the sharing-aware path (the plan built once
    before the loop, patched with mepic_decode_plan_patch at every page gain, only the changed stretches uploaded).
    Wall-clock time per step: host work (table update, plan patch) counts."""
    import torch
    from paper_2512_16822_b200 import runtime as RT
    wl = make_workload(index)
    P = wl.page_size
    import paper_2512_16822_b200 as M
    B = len(wl.decode_requests)
    spare = -(-n_steps // P) + 1
    cfg0 = make_config(wl)
    with M.Store(cfg0) as st:
        tables = RT.build_tables(st, wl.chunks, wl.decode_requests)
    ids0, base0, kvl0, _ = RT.pack_tables(tables, P)
    stride = ids0.shape[1] + spare
    cfg = M.Config(P, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.num_pages + B * spare, wl.max_position + (spare + 1) * P,
                   wl.rope_theta, wl.pad_token_id)
    kp, vp = wl.kv_pool()
    pad = np.zeros((B * spare,) + kp.shape[1:], dtype=np.uint16)        # the pages the loop will hand out (values do not matter)
    dev = RT.Device(cfg, np.concatenate([kp, pad]), np.concatenate([vp, pad]), device=device)
    q_bits = wl.decode_q()
    stream = torch.cuda.current_stream()
    out = {}
    for path in ("per_request", "grouped"):
        ids = np.zeros((B, stride), dtype=np.int32); base = np.zeros((B, stride), dtype=np.int32)
        ids[:, :ids0.shape[1]] = ids0; base[:, :ids0.shape[1]] = base0
        kvl = kvl0.copy()
        q_pos = (kvl - 1).astype(np.int32)
        if path == "per_request":
            batch = RT.DecodeBatch(dev, ids, base, kvl, q_pos, q_bits)
            h_in, hv = batch.host_mirror()
            hv["q"].copy_(torch.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)))
            h_ids, h_base, h_kvl, h_qpos = hv["page_ids"].numpy(), hv["pos_base"].numpy(), hv["kv_len"].numpy(), hv["q_pos"].numpy()
            h_q = hv["q"].view(torch.bfloat16)
        else:
            batch = RT.GroupedDecodeBatch(dev, ids, base, kvl, q_pos, q_bits)
            h_q = torch.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)).view(torch.bfloat16).pin_memory()
            h_kvl_t = torch.empty(B, dtype=torch.int32).pin_memory(); h_qpos_t = torch.empty(B, dtype=torch.int32).pin_memory()
            h_kvl, h_qpos = h_kvl_t.numpy(), h_qpos_t.numpy()
        h_out = torch.empty(batch.out.shape, dtype=torch.bfloat16).pin_memory()
        next_page = wl.num_pages
        for rep in range(2):                       # the first pass warms up (and checks the status word); the second is timed
            ids[:, ids0.shape[1]:] = 0; kvl[:] = kvl0
            if rep == 1 and path == "grouped":
                batch = RT.GroupedDecodeBatch(dev, ids, base, kvl, (kvl - 1).astype(np.int32), q_bits)   # a fresh plan (built outside the timed loop)
            if path == "per_request":
                h_ids[:] = ids; h_base[:] = base
                batch.upload(h_in)
            next_page = wl.num_pages
            gains = uploaded = 0
            host_s = 0.0
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for step in range(n_steps):
                th = time.perf_counter()
                gained = False
                for r in range(B):
                    if kvl[r] % P == 0:
                        e = kvl[r] // P
                        ids[r, e] = next_page; next_page += 1
                        base[r, e] = base[r, e - 1] + P
                        gained = True; gains += 1
                    kvl[r] += 1
                h_kvl[:] = kvl; h_qpos[:] = kvl - 1
                if path == "per_request":
                    if gained:
                        h_ids[:] = ids; h_base[:] = base
                        host_s += time.perf_counter() - th
                        batch.upload(h_in); uploaded += int(h_in.numel())
                    else:
                        host_s += time.perf_counter() - th
                        batch.q.copy_(h_q, non_blocking=True); batch.kv_len.copy_(hv["kv_len"], non_blocking=True)
                        batch.q_pos.copy_(hv["q_pos"], non_blocking=True)
                        uploaded += int(h_q.numel() * 2 + 8 * B)
                else:
                    if gained:
                        uploaded += batch.patch(ids, base, kvl)
                    host_s += time.perf_counter() - th
                    batch.q.copy_(h_q, non_blocking=True); batch.kv_len.copy_(h_kvl_t, non_blocking=True)
                    batch.q_pos.copy_(h_qpos_t, non_blocking=True)
                    uploaded += int(h_q.numel() * 2 + 8 * B)
                batch.run(wl.sm_scale, stream)
                h_out.copy_(batch.out, non_blocking=True)
                stream.synchronize()
            wall = time.perf_counter() - t0
            assert dev.read_status() == 0, "device status word is not clean"
        tokens = int(kvl0.astype(np.int64).sum()) + B * (n_steps + 1) // 2
        out[path] = {"ms_per_step": 1e3 * wall / n_steps, "steps": n_steps, "page_gains": gains,
                     "host_ms_per_step": 1e3 * host_s / n_steps, "h2d_bytes_per_step": uploaded / n_steps,
                     "d2h_bytes_per_step": int(h_out.numel() * 2),
                     "value": tokens * kv_bytes_per_token(wl) / (wall / n_steps) / 1e9, "unit": "GB/s"}
        if path == "grouped":
            out[path]["plan_ints"] = int(len(batch.plan_host))
        del batch
    out["grouped_over_per_request"] = out["per_request"]["ms_per_step"] / out["grouped"]["ms_per_step"]
    out["note"] = (f"config {index}, {n_steps} consecutive decode steps, kv_len + 1 per step and request; wall clock per step with the "
                   "result awaited every step; value = mean logical K/V bytes per step / time; no L2 flush (a serving loop has none)")
    return out


def measure_mixed(args, device: str):
    """Config 5 as one serving step: its decode batch and its prefill requests over one pool, each call alone and
    both enqueued on two streams (device time from the fork to the join)."""
    import torch
    from paper_2512_16822_b200 import runtime as RT
    wl = make_workload(5)
    lay = shared_layout(wl, device)
    dev = lay["dev"]
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(lay["decode_tables"], wl.page_size)
    db = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, wl.decode_q())
    pb, flops, _, _, _ = prefill_batch(wl, dev, lay["prefill_tables"])
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    main_s = torch.cuda.current_stream()
    flush = L2Flush(dev.device)

    def both():
        fork = torch.cuda.Event(); fork.record(main_s)
        s1.wait_event(fork); s2.wait_event(fork)
        pb.run(wl.sm_scale, s2)
        db.run(wl.sm_scale, s1)
        j1, j2 = torch.cuda.Event(), torch.cuda.Event()
        j1.record(s1); j2.record(s2)
        main_s.wait_event(j1); main_s.wait_event(j2)

    # the same with the prefill enqueued first on a high-priority stream and the decode behind it on a low-priority one:
    # the decode's CTAs then move in as the prefill's last wave leaves SMs idle
    lo_p, hi_p = torch.cuda.Stream.priority_range() if hasattr(torch.cuda.Stream, "priority_range") else (0, -1)
    s_hi, s_lo = torch.cuda.Stream(priority=hi_p), torch.cuda.Stream(priority=lo_p)

    def prefill_first():
        fork = torch.cuda.Event(); fork.record(main_s)
        s_hi.wait_event(fork); s_lo.wait_event(fork)
        pb.run(wl.sm_scale, s_hi)
        db.run(wl.sm_scale, s_lo)
        j1, j2 = torch.cuda.Event(), torch.cuda.Event()
        j1.record(s_hi); j2.record(s_lo)
        main_s.wait_event(j1); main_s.wait_event(j2)

    out = {}
    steps = max(5, min(args.steps, 10))
    for name, fn in (("decode_alone", lambda: db.run(wl.sm_scale, main_s)), ("prefill_alone", lambda: pb.run(wl.sm_scale, main_s)),
                     ("together_two_streams", both), ("together_prefill_first_decode_low_priority", prefill_first)):
        for _ in range(2):
            fn()
        out[name] = summary(time_steps(fn, steps, flush, main_s))
    assert dev.read_status() == 0
    s = out["decode_alone"]["ms_median"] + out["prefill_alone"]["ms_median"]
    best = min(out["together_two_streams"]["ms_median"], out["together_prefill_first_decode_low_priority"]["ms_median"])
    out["together_over_sum"] = best / s
    out["note"] = "medians; L2 flushed before each measurement"
    return out


# ---------------------------------------------------------------- multi-rank plumbing
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


def run_leg(args):
    """One leg alone on (possibly scaled) inputs: a short, fixed sequence of calls for a profiler to capture."""
    import torch
    from paper_2512_16822_b200 import runtime as RT
    from paper_2512_16822_b200.build import build_library
    build_library()
    device = "cuda:0"
    peak, _, _ = measured_peaks()
    if args.leg in ("prefill", "prefill-fp8"):
        d, _, _ = prefill_leg(args.config if args.config in (3, 5) else 3, args, device, scale=args.scale, error=False,
                              fp8=args.leg == "prefill-fp8")
        print(json.dumps(d), flush=True)
        return
    if args.leg == "mixed":
        print(json.dumps(measure_mixed(args, device)), flush=True)
        return
    if args.leg == "loop":
        print(json.dumps(measure_decode_loop(args, device, args.config if args.config != 3 else 2)), flush=True)
        return
    wl = make_workload(args.config, scale=args.scale)
    stream = torch.cuda.current_stream()
    if args.leg == "unshared":
        dev, page_ids, pos_base, kv_len, q_pos = unshared_layout(wl, device)
        kind = "plain"
    else:
        lay = shared_layout(wl, device)
        dev = lay["dev"]
        page_ids, pos_base, kv_len, q_pos = RT.pack_tables(lay["decode_tables"], wl.page_size)
        kind = {"decode": "plain", "graph": "plain"}.get(args.leg, args.leg)
    if args.leg == "unshared-fp8":
        dev, page_ids, pos_base, kv_len, q_pos = unshared_layout(wl, device)
        kind = "fp8"
    batch = decode_batch(kind, dev, page_ids, pos_base, kv_len, q_pos, wl.decode_q())
    step = lambda: batch.run(wl.sm_scale, stream)
    for _ in range(max(args.warmup, 1)):
        step()
    torch.cuda.synchronize()
    nbytes = int(kv_len.astype(np.int64).sum()) * kv_bytes_per_token(wl) // (2 if kind == "fp8" else 1)
    if args.leg == "graph":
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            batch.run(wl.sm_scale, torch.cuda.current_stream())
        res = {}
        for name, fn in (("direct_calls_us", step), ("graph_replays_us", graph.replay)):
            for _ in range(5):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(200):
                fn()
            e1.record(); torch.cuda.synchronize()
            res[name] = e0.elapsed_time(e1) / 200 * 1e3
        res["note"] = "per call, back to back, no L2 flush: launch latency of a tiny batch"
        print(json.dumps(res), flush=True)
        return
    ms = time_steps(step, args.steps, L2Flush(dev.device), stream)
    d = summary(ms); d.update(rates_gbs(nbytes, d["ms_per_step"], peak))
    d.update({"leg": args.leg, "workload": f"config{args.config}:{wl.name}", "scale": args.scale, "status": dev.read_status()})
    print(json.dumps(d), flush=True)


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
    device = f"cuda:{local_rank}"

    wl = make_workload(args.config)
    lay = shared_layout(wl, device)
    cfg, dev, tables, stats = lay["cfg"], lay["dev"], lay["decode_tables"], lay["stats"]
    table_build_ms = lay["table_build_ms"]
    q_bits = wl.decode_q()
    page_ids, pos_base, kv_len, q_pos = RT.pack_tables(tables, wl.page_size)
    batch = RT.DecodeBatch(dev, page_ids, pos_base, kv_len, q_pos, q_bits)
    logical_bytes = int(kv_len.astype(np.int64).sum()) * kv_bytes_per_token(wl)
    stream = torch.cuda.current_stream()
    l2_flush = L2Flush(dev.device)
    warmup = max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step = lambda: batch.run(wl.sm_scale, stream)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    assert dev.read_status() == 0, "device status word is not clean"

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample()
    launches0 = M.mepic_launch_count()
    barrier()
    with sampler.window("headline"):
        ms = time_steps(step, args.steps, l2_flush, stream)
        barrier()
    launches = M.mepic_launch_count() - launches0
    ms_warm = time_steps(step, args.steps, None, stream)
    # the same step, for at least half a second of device time (flushed): enough samples of the clocks, and a
    # median / minimum that do not rest on a handful of launches
    n_long = int(min(max(0.5 / (1e-3 * sum(ms) / len(ms)), args.steps), 4000))
    with sampler.window("sustained"):
        ms_long = time_steps(step, n_long, l2_flush, stream)

    # end to end: one pinned mirror of the step's inputs (q + block tables + lengths + positions): one copy in,
    # the kernels, one copy out, all inside the timed region
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
    with sampler.window("e2e"):
        ms_e2e = time_steps(e2e_step, args.steps, l2_flush, stream)
        barrier()
    assert dev.read_status() == 0, "device status word is not clean"

    def agg(xs):
        return max_over_ranks(sum(xs), world, dev.device)

    tot, tot_warm, tot_e2e = agg(ms), agg(ms_warm), agg(ms_e2e)
    peak, peak_src, peaks = measured_peaks()
    extras = rank == 0 and world == 1
    error = grouped = fp8 = unshared = None
    configs = {}
    tabs = (page_ids, pos_base, kv_len, q_pos)
    if extras and not args.quick:
        B = len(kv_len)
        error = decode_error(wl, lay, RT.bf16_bits(batch.out), sorted({0, B // 2, B - 1}))
        if wl.head_dim == 128:
            with sampler.window("fp8"):
                fp8 = measure_variant("fp8", args, wl, dev, tabs, q_bits, logical_bytes, peak, lay=lay)
        with sampler.window("grouped"):
            grouped = measure_variant("grouped", args, wl, dev, tabs, q_bits, logical_bytes, peak)
    del batch
    if extras:
        # the same batch without sharing: every byte from DRAM
        udev, uids, ubase, ukv, uqpos = unshared_layout(wl, device)
        ub = RT.DecodeBatch(udev, uids, ubase, ukv, uqpos, q_bits)
        for _ in range(3):
            ub.run(wl.sm_scale, stream)
        with sampler.window("unshared"):
            ums = time_steps(lambda: ub.run(wl.sm_scale, stream), max(5, min(args.steps, 50)), l2_flush, stream)
        assert udev.read_status() == 0
        unshared = summary(ums); unshared.update(rates_gbs(logical_bytes, unshared["ms_per_step"], peak))
        unshared.update({"pages_held": int(udev.cfg.num_pages),
                         "note": "no chunk sharing: logical bytes = unique bytes, every byte comes from DRAM; L2 flushed between steps"})
        del ub, udev
        torch.cuda.empty_cache()
    if extras and not args.quick:
        del dev, lay
        torch.cuda.empty_cache()
        with sampler.window("other_configs"):
            for idx in (1, 4, 5):
                if idx != args.config:
                    configs[f"config{idx}"] = decode_legs(idx, args, device, peak)
            pre3, _, _ = prefill_leg(3, args, device)
            configs["config3"] = {"prefill": pre3}
            torch.cuda.empty_cache()
            configs["config3"]["prefill_8bit_pages"], _, _ = prefill_leg(3, args, device, fp8=True)
            torch.cuda.empty_cache()
            pre5, _, _ = prefill_leg(5, args, device)
            configs.setdefault("config5", {})["prefill"] = pre5
            torch.cuda.empty_cache()
            configs["config5"]["serving_step"] = measure_mixed(args, device)
            torch.cuda.empty_cache()
            loop = measure_decode_loop(args, device)
        if grouped is not None:
            grouped["e2e"] = loop
    clocks = sampler.stop() if rank == 0 else None
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    gbs = lambda total_ms: aggregate_gbs(world, args.steps, logical_bytes, total_ms)
    per_launch_ms = sum(ms) / len(ms)
    effective = logical_bytes / (per_launch_ms * 1e-3) / 1e9
    tr = ncu_traffic("mepic_decode_splitkv", f"config{args.config}")
    roofline = {"bound": "hbm", "peak": peak, "unit": "GB/s", "peak_source": peak_src,
                "kernel": "mepic_decode_splitkv (+ its merge kernel: the C-ABI call is timed as a whole)",
                "algorithmic_bytes_per_launch": logical_bytes,
                "traffic": tr["dram_bytes_per_launch"] if tr else None, "traffic_source": tr,
                "effective": {"achieved": effective, "frac": effective / peak, "frac_of_nominal_8TBs": effective / NOMINAL_HBM_GBS,
                              "what": "this line's value: logical bytes / time on the shared layout; includes L2 hits on shared pages"}}
    roofline["effective"]["traffic"] = roofline["traffic"]
    if unshared is not None:
        # the DRAM-honest figure: the same kernel and the same logical bytes on the layout where no byte can come from L2
        tru = ncu_traffic("mepic_decode_splitkv_unshared", f"config{args.config}")
        roofline.update({"traffic": tru["dram_bytes_per_launch"] if tru else None, "traffic_source": tru})
        roofline.update({"achieved": unshared["value"], "frac": unshared["value"] / peak,
                         "frac_of_nominal_8TBs": unshared["value"] / NOMINAL_HBM_GBS,
                         "what": "unshared layout of the same batch (unshared_layout.ms_per_step): every byte comes from DRAM"})
    else:
        roofline.update({"achieved": effective, "frac": effective / peak, "frac_of_nominal_8TBs": effective / NOMINAL_HBM_GBS,
                         "what": "shared layout (effective): the unshared-layout run is made at 1 GPU only"})
    line = {
        "metric": METRIC, "value": gbs(tot), "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": tot / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": config_dict(args.config, wl, kv_len, world),
        "value_no_flush": gbs(tot_warm), "ms_per_step_no_flush": tot_warm / args.steps,
        "sustained": dict(summary(ms_long), **rates_gbs(logical_bytes, sum(ms_long) / len(ms_long), peak)),
        "e2e": {"value": gbs(tot_e2e), "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": tot_e2e / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "pages": {"held": stats["pages_shared_held"] + stats["pages_private_held"],
                  "shared": stats["pages_shared_held"], "private": stats["pages_private_held"],
                  "unshared_equivalent": stats["unshared_equivalent_pages"], "dedup_hits": stats["dedup_hits"]},
        "table_build_ms": table_build_ms,
        "error": error,
        "prefill": configs.get("config3", {}).get("prefill"),
        "unshared_layout": unshared,
        "grouped_decode": grouped,
        "fp8_decode": fp8,
        "configs": configs,
        "targets": {"decode": ">= 70 % of HBM bandwidth", "prefill": ">= 50 % of dense bf16 peak",
                    "denominators": {"hbm_gbs_measured": peak, "hbm_gbs_nominal": NOMINAL_HBM_GBS,
                                     "bf16_tflops_burst": peaks.get("bf16_tflops"),
                                     "bf16_tflops_sustained": peaks.get("bf16_tflops_sustained"),
                                     "bf16_tflops_nominal": NOMINAL_BF16_TFLOPS}},
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
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="headline and unshared layout only: no other configs, no variants")
    ap.add_argument("--leg", default=None, choices=["decode", "unshared", "grouped", "fp8", "unshared-fp8", "prefill", "prefill-fp8", "mixed", "graph", "loop"],
                    help="run one leg alone (a short fixed sequence of calls, e.g. for a profiler) and print its line")
    ap.add_argument("--scale", type=float, default=1.0, help="with --leg: shrink the configuration (1.0 = as specified)")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.config == 3:
            raise SystemExit("--impl reference times the decode metric: --config 1, 2, 4 or 5")
        run_reference(args)
    elif args.leg:
        run_leg(args)
    else:
        if args.config == 3:
            raise SystemExit("the headline metric is a decode rate: --config 1, 2, 4 or 5 (config 3 is in `configs`)")
        run_ours(args)


if __name__ == "__main__":
    main()
