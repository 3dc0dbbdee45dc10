"""Device-side plumbing around the C ABI: torch tensors, streams, uploads.

Nothing here computes any part of the method; it allocates the buffers the ABI
asks the caller to own, moves host tables to the device and issues the calls.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import (Config, Segment, Store, MEPIC_SEG_CHUNK, MEPIC_SEG_PROMPT, mepic_attn_decode,
               mepic_decode_plan_build, mepic_decode_plan_patch, mepic_attn_decode_grouped, mepic_attn_decode_grouped_fp8, mepic_attn_decode_grouped_workspace,
               mepic_pages_quantize, mepic_attn_decode_fp8,
               mepic_attn_decode_workspace, mepic_attn_prefill, mepic_attn_prefill_fp8, mepic_attn_prefill_workspace,
               mepic_rope_table_fill)


@dataclass
class Table:
    request_id: int
    page_ids: np.ndarray
    pos_base: np.ndarray
    kv_len: int
    recompute_slots: np.ndarray


def build_tables(store: Store, chunks: Sequence[np.ndarray], requests) -> List[Table]:
    """Register each request's chunks, then build its block table, in request order.

    ``requests`` are objects with ``request_id`` and ``segments`` = [(kind, value)] where a chunk
    segment's value indexes ``chunks``.
    """
    out = []
    for r in requests:
        segs = []
        for kind, val in r.segments:
            if kind == MEPIC_SEG_CHUNK:
                cid, _, _, _ = store.chunk_register(chunks[val])
                segs.append(Segment(MEPIC_SEG_CHUNK, cid))
            else:
                segs.append(Segment(MEPIC_SEG_PROMPT, int(val)))
        pages, base, kv_len, slots = store.build_block_table(r.request_id, segs)
        out.append(Table(r.request_id, pages, base, kv_len, slots))
    return out


def pack_tables(tables: Sequence[Table], page_size: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Host arrays page_ids[B, stride], pos_base[B, stride], kv_len[B], q_pos[B].

    q_pos is the position of the request's last slot: the decode query is the newest token, whose
    K/V is already in the cache.
    """
    stride = max(len(t.page_ids) for t in tables)
    B = len(tables)
    page_ids = np.zeros((B, stride), dtype=np.int32)
    pos_base = np.zeros((B, stride), dtype=np.int32)
    kv_len = np.zeros(B, dtype=np.int32)
    for i, t in enumerate(tables):
        page_ids[i, :len(t.page_ids)] = t.page_ids
        pos_base[i, :len(t.pos_base)] = t.pos_base
        kv_len[i] = t.kv_len
    last = kv_len - 1
    q_pos = pos_base[np.arange(B), last // page_size] + last % page_size
    return page_ids, pos_base, kv_len, q_pos.astype(np.int32)


def bf16_tensor(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bit patterns -> torch.bfloat16 tensor on ``device`` (no value conversion)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Device:
    """The buffers one pool needs on a GPU: K/V pools, rope table, status word."""

    def __init__(self, cfg: Config, k_bits: Optional[np.ndarray] = None, v_bits: Optional[np.ndarray] = None,
                 device: str = "cuda:0", bf16_pools: bool = True):
        if not torch.cuda.is_available():
            raise RuntimeError("the MEPIC kernels need a CUDA device; there is no CPU path")
        self.cfg = cfg
        self.device = torch.device(device)
        shape = (cfg.num_pages, cfg.n_kv_heads, cfg.page_size, cfg.head_dim)
        if not bf16_pools:
            self.k_pool = self.v_pool = None           # a device whose only pools are 8-bit (see Fp8Pools)
        elif k_bits is not None:
            assert k_bits.shape == shape and v_bits.shape == shape
            self.k_pool = bf16_tensor(k_bits, self.device)
            self.v_pool = bf16_tensor(v_bits, self.device)
        else:
            self.k_pool = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
            self.v_pool = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
        self.rope = torch.from_numpy(mepic_rope_table_fill(cfg)).to(self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)

    def read_status(self) -> int:
        return int(self.status.item())


class DecodeBatch:
    """Device copies of one decode batch's tables plus output and workspace."""

    def __init__(self, dev: Device, page_ids: np.ndarray, pos_base: np.ndarray, kv_len: np.ndarray,
                 q_pos: np.ndarray, q_bits: Optional[np.ndarray] = None):
        cfg = dev.cfg
        self.dev = dev
        self.batch, self.stride = page_ids.shape
        d = dev.device
        # The per-step inputs (q and the tables) are views of ONE device buffer, so that a serving loop can bring a
        # step's inputs over with a single host-to-device copy from a pinned mirror (see host_mirror / upload).
        qshape = (self.batch, cfg.n_q_heads, cfg.head_dim)
        parts = [("q", qshape, torch.bfloat16), ("page_ids", (self.batch, self.stride), torch.int32),
                 ("pos_base", (self.batch, self.stride), torch.int32), ("kv_len", (self.batch,), torch.int32),
                 ("q_pos", (self.batch,), torch.int32)]
        self._layout, at = [], 0
        for name, shape, dt in parts:
            n = int(np.prod(shape)) * torch.empty((), dtype=dt).element_size()
            self._layout.append((name, shape, dt, at, n))
            at += -(-n // 256) * 256                                   # every view starts 256-byte aligned
        self.step_inputs = torch.empty(at, dtype=torch.uint8, device=d)
        for name, shape, dt, off, n in self._layout:
            setattr(self, name, self.step_inputs[off:off + n].view(dt).view(shape))
        self.page_ids.copy_(torch.from_numpy(np.ascontiguousarray(page_ids, dtype=np.int32)))
        self.pos_base.copy_(torch.from_numpy(np.ascontiguousarray(pos_base, dtype=np.int32)))
        self.kv_len.copy_(torch.from_numpy(np.ascontiguousarray(kv_len, dtype=np.int32)))
        self.q_pos.copy_(torch.from_numpy(np.ascontiguousarray(q_pos, dtype=np.int32)))
        if q_bits is not None:
            self.q.view(torch.int16).copy_(torch.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)))
        self.out = torch.empty(qshape, dtype=torch.bfloat16, device=d)
        self.ws_bytes = mepic_attn_decode_workspace(cfg, self.batch)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=d)

    def run(self, sm_scale: float, stream=None) -> torch.Tensor:
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        mepic_attn_decode(self.dev.cfg, q=self.q, k_pool=self.dev.k_pool, v_pool=self.dev.v_pool,
                          page_ids=self.page_ids, pos_base=self.pos_base, kv_len=self.kv_len, q_pos=self.q_pos,
                          rope_table=self.dev.rope, out=self.out, workspace=self.workspace,
                          workspace_bytes=self.ws_bytes, status=self.dev.status, table_stride=self.stride,
                          batch=self.batch, sm_scale=sm_scale, stream=s)
        return self.out

    def host_mirror(self):
        """Pinned host buffer with the layout of ``step_inputs`` and named views into it (q as int16 bit patterns)."""
        host = torch.empty(self.step_inputs.numel(), dtype=torch.uint8).pin_memory()
        views = {}
        for name, shape, dt, off, n in self._layout:
            hdt = torch.int16 if dt == torch.bfloat16 else dt
            views[name] = host[off:off + n].view(hdt).view(shape)
        return host, views

    def upload(self, host: torch.Tensor) -> None:
        """One asynchronous host-to-device copy of a whole step's inputs (on the current stream)."""
        self.step_inputs.copy_(host, non_blocking=True)


class Fp8Pools:
    """8-bit (e4m3) copies of a device's K/V pools with one scale per (page, kv head), made by the library's quantiser."""

    def __init__(self, dev: Device, pages: Optional[np.ndarray] = None):
        cfg = dev.cfg
        self.dev = dev
        d = dev.device
        shape = (cfg.num_pages, cfg.n_kv_heads, cfg.page_size, cfg.head_dim)
        self.k_codes = torch.zeros(shape, dtype=torch.uint8, device=d)
        self.v_codes = torch.zeros(shape, dtype=torch.uint8, device=d)
        self.k_scales = torch.ones((cfg.num_pages, cfg.n_kv_heads), dtype=torch.float32, device=d)
        self.v_scales = torch.ones((cfg.num_pages, cfg.n_kv_heads), dtype=torch.float32, device=d)
        if dev.k_pool is not None:                     # pools without a bf16 original start empty: prefill fills them
            self.quantize(np.arange(cfg.num_pages, dtype=np.int32) if pages is None else pages)

    def quantize(self, pages: np.ndarray, stream=None) -> None:
        lst = torch.from_numpy(np.ascontiguousarray(pages, dtype=np.int32)).to(self.dev.device)
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        for src, dst, sc in ((self.dev.k_pool, self.k_codes, self.k_scales), (self.dev.v_pool, self.v_codes, self.v_scales)):
            mepic_pages_quantize(self.dev.cfg, src_pool=src, dst_pool=dst, scales=sc, pages=lst, n_pages=int(lst.numel()),
                                 status=self.dev.status, stream=s)


class Fp8DecodeBatch(DecodeBatch):
    """A decode batch that reads the 8-bit pools."""

    def __init__(self, pools: Fp8Pools, page_ids, pos_base, kv_len, q_pos, q_bits=None):
        super().__init__(pools.dev, page_ids, pos_base, kv_len, q_pos, q_bits)
        self.pools = pools

    def run(self, sm_scale: float, stream=None) -> torch.Tensor:
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        mepic_attn_decode_fp8(self.dev.cfg, q=self.q, k_pool=self.pools.k_codes, v_pool=self.pools.v_codes,
                              k_scales=self.pools.k_scales, v_scales=self.pools.v_scales, page_ids=self.page_ids,
                              pos_base=self.pos_base, kv_len=self.kv_len, q_pos=self.q_pos, rope_table=self.dev.rope,
                              out=self.out, workspace=self.workspace, workspace_bytes=self.ws_bytes,
                              status=self.dev.status, table_stride=self.stride, batch=self.batch, sm_scale=sm_scale,
                              stream=s)
        return self.out


class GroupedDecodeBatch:
    """One decode batch run through the sharing-aware path: host plan + its device copy, output, workspace."""

    def __init__(self, dev: Device, page_ids: np.ndarray, pos_base: np.ndarray, kv_len: np.ndarray,
                 q_pos: np.ndarray, q_bits: Optional[np.ndarray] = None, n_sms: int = 0):
        cfg = dev.cfg
        self.dev = dev
        self.batch = page_ids.shape[0]
        d = dev.device
        with torch.cuda.device(d):
            built = mepic_decode_plan_build(cfg, page_ids, pos_base, kv_len, n_sms)
        # the host copy lives in page-locked memory: a patch uploads stretches of it without a staging copy
        self._plan_pinned = torch.empty(len(built), dtype=torch.int32).pin_memory()
        self.plan_host = self._plan_pinned.numpy()
        self.plan_host[:] = built
        self.plan = torch.from_numpy(built).to(d)
        self._uploaded = None
        self.kv_len = torch.from_numpy(np.ascontiguousarray(kv_len, dtype=np.int32)).to(d)
        self.q_pos = torch.from_numpy(np.ascontiguousarray(q_pos, dtype=np.int32)).to(d)
        qshape = (self.batch, cfg.n_q_heads, cfg.head_dim)
        self.q = bf16_tensor(q_bits, d) if q_bits is not None else torch.empty(qshape, dtype=torch.bfloat16, device=d)
        self.out = torch.empty(qshape, dtype=torch.bfloat16, device=d)
        self.ws_bytes = mepic_attn_decode_grouped_workspace(cfg, self.plan_host)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=d)

    def run(self, sm_scale: float, stream=None) -> torch.Tensor:
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        mepic_attn_decode_grouped(self.dev.cfg, q=self.q, k_pool=self.dev.k_pool, v_pool=self.dev.v_pool,
                                  plan=self.plan, plan_host=self.plan_host, kv_len=self.kv_len, q_pos=self.q_pos,
                                  rope_table=self.dev.rope, out=self.out, workspace=self.workspace,
                                  workspace_bytes=self.ws_bytes, status=self.dev.status, batch=self.batch,
                                  sm_scale=sm_scale, stream=s)
        return self.out

    def patch(self, page_ids: np.ndarray, pos_base: np.ndarray, kv_len: np.ndarray) -> int:
        """Requests gained pages: patch the host plan in place and upload only what changed (on the current stream).
        Returns the bytes uploaded.  kv_len itself is the caller's per-step input and is not touched here."""
        if self._uploaded is not None:
            self._uploaded.synchronize()              # the previous patch's copies have read the host buffer
        ranges = mepic_decode_plan_patch(self.dev.cfg, self.plan_host, page_ids, pos_base, kv_len)
        sent = 0
        for lo, n in ranges:
            self.plan[lo:lo + n].copy_(self._plan_pinned[lo:lo + n], non_blocking=True)
            sent += 4 * n
        if ranges:
            self._uploaded = torch.cuda.Event(); self._uploaded.record()
            need = mepic_attn_decode_grouped_workspace(self.dev.cfg, self.plan_host)
            if need > self.ws_bytes:                  # more partial slots than before: a larger workspace (rare)
                self.ws_bytes = need + need // 8
                self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.dev.device)
        return sent


class PrefillBatch:
    """Device copies of one prefill batch: new rows, their slots, tables, output, workspace."""

    def __init__(self, dev: Device, page_ids: np.ndarray, pos_base: np.ndarray, kv_len: np.ndarray,
                 row_offsets: np.ndarray, q_slot: np.ndarray, q_bits: np.ndarray, k_bits: np.ndarray,
                 v_bits: np.ndarray):
        cfg = dev.cfg
        self.dev = dev
        self.batch, self.stride = page_ids.shape
        d = dev.device
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(d)
        self.page_ids, self.pos_base, self.kv_len = i32(page_ids), i32(pos_base), i32(kv_len)
        self.row_offsets_host = np.ascontiguousarray(row_offsets, dtype=np.int32)
        self.row_offsets, self.q_slot = i32(row_offsets), i32(q_slot)
        self.q_new, self.k_new, self.v_new = bf16_tensor(q_bits, d), bf16_tensor(k_bits, d), bf16_tensor(v_bits, d)
        self.out = torch.empty(self.q_new.shape, dtype=torch.bfloat16, device=d)
        self.ws_bytes = mepic_attn_prefill_workspace(cfg, self.batch, self.row_offsets_host)
        self.workspace = torch.empty(max(self.ws_bytes, 16), dtype=torch.uint8, device=d)

    def run(self, sm_scale: float, stream=None) -> torch.Tensor:
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        mepic_attn_prefill(self.dev.cfg, q_new=self.q_new, k_new=self.k_new, v_new=self.v_new,
                           row_offsets=self.row_offsets, q_slot=self.q_slot, k_pool=self.dev.k_pool,
                           v_pool=self.dev.v_pool, page_ids=self.page_ids, pos_base=self.pos_base,
                           kv_len=self.kv_len, rope_table=self.dev.rope, out=self.out, workspace=self.workspace,
                           workspace_bytes=self.ws_bytes, status=self.dev.status,
                           row_offsets_host=self.row_offsets_host, table_stride=self.stride, batch=self.batch,
                           sm_scale=sm_scale, stream=s)
        return self.out

    def repeated(self) -> bool:
        """Whether the last call ran its repeat launch (first workspace word; synchronises the device)."""
        return int(self.workspace[:4].view(torch.int32).item()) != 0


class Fp8PrefillBatch(PrefillBatch):
    """A prefill batch that commits into, and attends over, the 8-bit pools."""

    def __init__(self, pools: Fp8Pools, page_ids, pos_base, kv_len, row_offsets, q_slot, q_bits, k_bits, v_bits):
        super().__init__(pools.dev, page_ids, pos_base, kv_len, row_offsets, q_slot, q_bits, k_bits, v_bits)
        self.pools = pools

    def run(self, sm_scale: float, stream=None) -> torch.Tensor:
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        mepic_attn_prefill_fp8(self.dev.cfg, q_new=self.q_new, k_new=self.k_new, v_new=self.v_new,
                               row_offsets=self.row_offsets, q_slot=self.q_slot, k_pool=self.pools.k_codes,
                               v_pool=self.pools.v_codes, k_scales=self.pools.k_scales, v_scales=self.pools.v_scales,
                               page_ids=self.page_ids, pos_base=self.pos_base, kv_len=self.kv_len,
                               rope_table=self.dev.rope, out=self.out, workspace=self.workspace,
                               workspace_bytes=self.ws_bytes, status=self.dev.status,
                               row_offsets_host=self.row_offsets_host, table_stride=self.stride, batch=self.batch,
                               sm_scale=sm_scale, stream=s)
        return self.out


class Fp8GroupedDecodeBatch(GroupedDecodeBatch):
    """The sharing-aware decode path over the 8-bit pools."""

    def __init__(self, pools: Fp8Pools, page_ids, pos_base, kv_len, q_pos, q_bits=None, n_sms: int = 0):
        super().__init__(pools.dev, page_ids, pos_base, kv_len, q_pos, q_bits, n_sms)
        self.pools = pools

    def run(self, sm_scale: float, stream=None) -> torch.Tensor:
        s = stream if stream is not None else torch.cuda.current_stream(self.dev.device)
        mepic_attn_decode_grouped_fp8(self.dev.cfg, q=self.q, k_pool=self.pools.k_codes, v_pool=self.pools.v_codes,
                                      k_scales=self.pools.k_scales, v_scales=self.pools.v_scales, plan=self.plan,
                                      plan_host=self.plan_host, kv_len=self.kv_len, q_pos=self.q_pos,
                                      rope_table=self.dev.rope, out=self.out, workspace=self.workspace,
                                      workspace_bytes=self.ws_bytes, status=self.dev.status, batch=self.batch,
                                      sm_scale=sm_scale, stream=s)
        return self.out
