"""Python binding of libmepic (the B200 hot path of MEPIC).

Argument marshalling only: every function here has the name of the C entry
point it forwards to (see ``include/mepic.h``) and does no part of the method
itself.  Device buffers are torch CUDA tensors (or anything with a
``data_ptr()``) that the caller allocates; host arrays are numpy.

The shared library is built in-tree by ``paper_2512_16822_b200.build``.  If it
is missing, importing this package raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import numpy as np

from .build import LIB_PATH, build_library

__all__ = [
    "MepicError", "Config", "Segment", "Store", "lib",
    "mepic_store_create", "mepic_store_destroy", "mepic_chunk_register", "mepic_build_block_table",
    "mepic_request_release", "mepic_chunk_mark_uncomputed", "mepic_store_stats", "mepic_store_attach_remote", "mepic_store_test_hooks", "mepic_kernel_test_hooks", "mepic_prefill_test_two_pass", "mepic_rope_table_floats", "mepic_rope_table_fill",
    "mepic_attn_decode_workspace", "mepic_attn_decode", "mepic_attn_decode_static",
    "mepic_pages_quantize", "mepic_attn_decode_fp8", "mepic_decode_plan_max_ints", "mepic_decode_plan_build", "mepic_decode_plan_patch", "mepic_attn_decode_grouped_workspace",
    "mepic_attn_decode_grouped", "mepic_attn_decode_grouped_fp8",
    "MEPIC_DECODE_STATIC_SCRATCH_BYTES", "mepic_attn_prefill_workspace",
    "mepic_attn_prefill", "mepic_attn_prefill_fp8", "mepic_last_error", "mepic_launch_count",
    "MEPIC_OK", "MEPIC_E_INVAL", "MEPIC_E_NOSPACE", "MEPIC_E_NOTFOUND", "MEPIC_E_CAPACITY",
    "MEPIC_E_CUDA", "MEPIC_E_EXISTS", "MEPIC_SEG_CHUNK", "MEPIC_SEG_PROMPT",
]

MEPIC_OK = 0
MEPIC_E_INVAL = -1
MEPIC_E_NOSPACE = -2
MEPIC_E_NOTFOUND = -3
MEPIC_E_CAPACITY = -4
MEPIC_E_CUDA = -5
MEPIC_E_EXISTS = -6
MEPIC_SEG_CHUNK = 0
MEPIC_SEG_PROMPT = 1
MEPIC_DECODE_STATIC_SCRATCH_BYTES = 8 << 20
MEPIC_DEV_BAD_PAGE = 0x1
MEPIC_DEV_WAIT_EXPIRED = 0x2
MEPIC_DEV_BAD_POSITION = 0x4
MEPIC_DEV_BAD_SLOT = 0x8
MEPIC_DEV_BAD_PLAN = 0x10


class MepicError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"mepic error {code}: {text}")
        self.code = code


class _ConfigC(C.Structure):
    _fields_ = [("page_size", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("num_pages", C.c_int32), ("pad_token_id", C.c_int32),
                ("max_position", C.c_int32), ("rope_theta", C.c_float)]


class _StatsC(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "pages_total", "pages_free", "pages_shared_held", "pages_private_held", "chunks_resident",
        "chunk_refs", "dedup_hits", "unshared_equivalent_pages", "live_requests", "chunks_evicted",
        "pages_evicted", "chunks_spilled", "chunks_fetched", "remote_chunks", "remote_pages")]


class _SegmentC(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_tokens", C.c_int32), ("chunk_id", C.c_uint64)]


class _DecodeArgsC(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
                ("page_ids", C.c_void_p), ("pos_base", C.c_void_p), ("kv_len", C.c_void_p),
                ("q_pos", C.c_void_p), ("rope_table", C.c_void_p), ("out", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("status", C.c_void_p),
                ("table_stride", C.c_int32), ("batch", C.c_int32), ("sm_scale", C.c_float)]


class _PrefillArgsC(C.Structure):
    _fields_ = [("q_new", C.c_void_p), ("k_new", C.c_void_p), ("v_new", C.c_void_p),
                ("row_offsets", C.c_void_p), ("q_slot", C.c_void_p), ("k_pool", C.c_void_p),
                ("v_pool", C.c_void_p), ("page_ids", C.c_void_p), ("pos_base", C.c_void_p),
                ("kv_len", C.c_void_p), ("rope_table", C.c_void_p), ("out", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("status", C.c_void_p),
                ("row_offsets_host", C.c_void_p), ("table_stride", C.c_int32), ("batch", C.c_int32),
                ("sm_scale", C.c_float)]


class _DecodeGroupedArgsC(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("plan", C.c_void_p),
                ("plan_host", C.c_void_p), ("kv_len", C.c_void_p), ("q_pos", C.c_void_p), ("rope_table", C.c_void_p),
                ("out", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("status", C.c_void_p), ("batch", C.c_int32), ("sm_scale", C.c_float)]


@dataclass(frozen=True)
class Config:
    page_size: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    num_pages: int
    max_position: int
    rope_theta: float
    pad_token_id: int = 0

    def c(self) -> _ConfigC:
        return _ConfigC(self.page_size, self.n_q_heads, self.n_kv_heads, self.head_dim, self.num_pages,
                        self.pad_token_id, self.max_position, self.rope_theta)


@dataclass(frozen=True)
class Segment:
    kind: int
    value: int      # chunk id (kind == MEPIC_SEG_CHUNK) or token count (MEPIC_SEG_PROMPT)


_LIB: Optional[C.CDLL] = None

_PROTOTYPES = {
    "mepic_last_error": (C.c_char_p, []),
    "mepic_launch_count": (C.c_int64, []),
    "mepic_store_create": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(C.c_void_p)]),
    "mepic_store_destroy": (None, [C.c_void_p]),
    "mepic_chunk_register": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_uint64),
                                         C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_void_p, C.c_int32,
                                         C.POINTER(C.c_int32)]),
    "mepic_build_block_table": (C.c_int32, [C.c_void_p, C.c_int64, C.POINTER(_SegmentC), C.c_int32,
                                            C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int32),
                                            C.POINTER(C.c_int32), C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]),
    "mepic_request_release": (C.c_int32, [C.c_void_p, C.c_int64]),
    "mepic_chunk_mark_uncomputed": (C.c_int32, [C.c_void_p, C.c_uint64]),
    "mepic_store_stats": (C.c_int32, [C.c_void_p, C.POINTER(_StatsC)]),
    "mepic_store_attach_remote": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_void_p]),
    "mepic_store_test_hooks": (C.c_int32, [C.c_void_p, C.c_uint64, C.c_int32]),
    "mepic_kernel_test_hooks": (C.c_int32, [C.c_int32, C.c_int32]),
    "mepic_prefill_test_two_pass": (C.c_int32, [C.c_int32]),
    "mepic_rope_table_floats": (C.c_size_t, [C.POINTER(_ConfigC)]),
    "mepic_rope_table_fill": (C.c_int32, [C.POINTER(_ConfigC), C.c_void_p]),
    "mepic_attn_decode_workspace": (C.c_size_t, [C.POINTER(_ConfigC), C.c_int32]),
    "mepic_attn_decode": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_DecodeArgsC), C.c_void_p]),
    "mepic_attn_decode_static": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_DecodeArgsC), C.c_void_p]),
    "mepic_pages_quantize": (C.c_int32, [C.POINTER(_ConfigC), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                         C.c_void_p, C.c_void_p]),
    "mepic_attn_decode_fp8": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_DecodeArgsC), C.c_void_p, C.c_void_p, C.c_void_p]),
    "mepic_decode_plan_max_ints": (C.c_size_t, [C.POINTER(_ConfigC), C.c_int32, C.c_int32, C.c_int32]),
    "mepic_decode_plan_build": (C.c_int32, [C.POINTER(_ConfigC), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                            C.c_int32, C.c_int32, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]),
    "mepic_decode_plan_patch": (C.c_int32, [C.POINTER(_ConfigC), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                            C.c_int32, C.c_void_p, C.POINTER(C.c_int32)]),
    "mepic_attn_decode_grouped_workspace": (C.c_size_t, [C.POINTER(_ConfigC), C.c_void_p]),
    "mepic_attn_decode_grouped": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_DecodeGroupedArgsC), C.c_void_p]),
    "mepic_attn_decode_grouped_fp8": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_DecodeGroupedArgsC), C.c_void_p, C.c_void_p, C.c_void_p]),
    "mepic_attn_prefill_workspace": (C.c_size_t, [C.POINTER(_ConfigC), C.c_int32, C.c_void_p]),
    "mepic_attn_prefill": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_PrefillArgsC), C.c_void_p]),
    "mepic_attn_prefill_fp8": (C.c_int32, [C.POINTER(_ConfigC), C.POINTER(_PrefillArgsC), C.c_void_p, C.c_void_p, C.c_void_p]),
}


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2512_16822_b200.build` "
                              "(the MEPIC kernels have no fallback path)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in _PROTOTYPES.items():
            if not hasattr(handle, name):
                continue          # reported by the symbol test, and by the call that needs it
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _LIB = handle
    return _LIB


def _check(code: int) -> None:
    if code != MEPIC_OK:
        raise MepicError(code, mepic_last_error())


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array / raw int; None stays NULL."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if isinstance(x, np.ndarray):
        return int(x.ctypes.data)
    raise TypeError(f"cannot take the address of {type(x)}")


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def mepic_last_error() -> str:
    return lib().mepic_last_error().decode()


def mepic_launch_count() -> int:
    return int(lib().mepic_launch_count())


# ------------------------------------------------------------------ scheduling path (host)
def mepic_store_create(cfg: Config) -> int:
    out = C.c_void_p()
    c = cfg.c()
    _check(lib().mepic_store_create(C.byref(c), C.byref(out)))
    return out.value


def mepic_store_destroy(store: int) -> None:
    lib().mepic_store_destroy(store)


def mepic_chunk_register(store: int, tokens: np.ndarray) -> Tuple[int, bool, int, np.ndarray]:
    """-> (chunk_id, was_resident, lead_pad, shared_pages int32[]); was_resident: 0 new, 1 resident, 2 from the remote tier."""
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    cid, res, lead, n = C.c_uint64(), C.c_int32(), C.c_int32(), C.c_int32()
    cap = max(int(tok.size), 1)          # a chunk never has more pages than tokens
    pages = np.empty(cap, dtype=np.int32)
    _check(lib().mepic_chunk_register(store, tok.ctypes.data, int(tok.size), C.byref(cid), C.byref(res),
                                      C.byref(lead), pages.ctypes.data, cap, C.byref(n)))
    return int(cid.value), int(res.value), int(lead.value), pages[:n.value].copy()


def mepic_build_block_table(store: int, request_id: int, segments: Sequence[Segment]
                            ) -> Tuple[np.ndarray, np.ndarray, int, np.ndarray]:
    """-> (page_ids int32[E], pos_base int32[E], kv_len, recompute_slots int32[])."""
    n = len(segments)
    segs = (_SegmentC * max(n, 1))()
    for i, s in enumerate(segments):
        segs[i].kind = int(s.kind)
        segs[i].n_tokens = int(s.value) if s.kind == MEPIC_SEG_PROMPT else 0
        segs[i].chunk_id = int(s.value) if s.kind == MEPIC_SEG_CHUNK else 0
    ne, kv, ns = C.c_int32(), C.c_int32(), C.c_int32()
    # size query: zero capacity reports the required counts and holds nothing
    code = lib().mepic_build_block_table(store, request_id, segs, n, None, None, 0, C.byref(ne), C.byref(kv),
                                         None, 0, C.byref(ns))
    if code not in (MEPIC_E_CAPACITY, MEPIC_OK):
        _check(code)
    pages = np.empty(max(ne.value, 1), dtype=np.int32)
    base = np.empty(max(ne.value, 1), dtype=np.int32)
    slots = np.empty(max(ns.value, 1), dtype=np.int32)
    _check(lib().mepic_build_block_table(store, request_id, segs, n, pages.ctypes.data, base.ctypes.data,
                                         pages.size, C.byref(ne), C.byref(kv), slots.ctypes.data, slots.size,
                                         C.byref(ns)))
    return pages[:ne.value], base[:ne.value], int(kv.value), slots[:ns.value]


def mepic_chunk_mark_uncomputed(store: int, chunk_id: int) -> None:
    _check(lib().mepic_chunk_mark_uncomputed(store, chunk_id))


def mepic_request_release(store: int, request_id: int) -> None:
    _check(lib().mepic_request_release(store, request_id))


def mepic_store_stats(store: int) -> dict:
    st = _StatsC()
    _check(lib().mepic_store_stats(store, C.byref(st)))
    return {name: int(getattr(st, name)) for name, _ in _StatsC._fields_}


def mepic_store_attach_remote(store: int, k_pool, v_pool, capacity_pages: int, stream=None) -> None:
    """Attach the remote tier.  numpy pools: host mode (plain memcpy); torch CUDA tensors: device mode."""
    on_host = isinstance(k_pool, np.ndarray)
    if on_host:
        assert k_pool.flags["C_CONTIGUOUS"] and v_pool.flags["C_CONTIGUOUS"]
        kp, vp, st = k_pool.ctypes.data, v_pool.ctypes.data, None
    else:
        kp, vp, st = _ptr(k_pool), _ptr(v_pool), _stream_ptr(stream)
    _check(lib().mepic_store_attach_remote(store, kp, vp, 1 if on_host else 0, int(capacity_pages), st))


def mepic_store_test_hooks(store: int, hash_mask: int = 0xFFFFFFFFFFFFFFFF, fail_copies: int = 0) -> None:
    _check(lib().mepic_store_test_hooks(store, hash_mask, fail_copies))


def mepic_kernel_test_hooks(spin_limit: int = 0, skip_tile: int = -1) -> None:
    _check(lib().mepic_kernel_test_hooks(spin_limit, skip_tile))


def mepic_prefill_test_two_pass(on: bool) -> None:
    _check(lib().mepic_prefill_test_two_pass(1 if on else 0))


class Store:
    """Owns one ``mepic_store_t`` handle (context manager; same calls as the C ABI)."""

    def __init__(self, cfg: Config):
        self.cfg = cfg
        self.handle = mepic_store_create(cfg)

    def chunk_register(self, tokens):
        return mepic_chunk_register(self.handle, tokens)

    def build_block_table(self, request_id, segments):
        return mepic_build_block_table(self.handle, request_id, segments)

    def chunk_mark_uncomputed(self, chunk_id):
        mepic_chunk_mark_uncomputed(self.handle, chunk_id)

    def request_release(self, request_id):
        mepic_request_release(self.handle, request_id)

    def stats(self):
        return mepic_store_stats(self.handle)

    def attach_remote(self, k_pool, v_pool, capacity_pages, stream=None):
        self._remote_pools = (k_pool, v_pool)          # the store keeps raw pointers: keep the arrays alive
        mepic_store_attach_remote(self.handle, k_pool, v_pool, capacity_pages, stream)

    def close(self):
        if self.handle:
            mepic_store_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ------------------------------------------------------------------ rope table (host set-up)
def mepic_rope_table_floats(cfg: Config) -> int:
    c = cfg.c()
    return int(lib().mepic_rope_table_floats(C.byref(c)))


def mepic_rope_table_fill(cfg: Config) -> np.ndarray:
    """-> float32 [max_position+1, head_dim/2, 2] = (cos, sin)."""
    n = mepic_rope_table_floats(cfg)
    if n == 0:
        raise MepicError(MEPIC_E_INVAL, mepic_last_error())
    out = np.empty(n, dtype=np.float32)
    c = cfg.c()
    _check(lib().mepic_rope_table_fill(C.byref(c), out.ctypes.data))
    return out.reshape(cfg.max_position + 1, cfg.head_dim // 2, 2)


# ------------------------------------------------------------------ attention (device)
def mepic_attn_decode_workspace(cfg: Config, batch: int) -> int:
    c = cfg.c()
    n = int(lib().mepic_attn_decode_workspace(C.byref(c), batch))
    if n == 0:
        raise MepicError(MEPIC_E_INVAL, mepic_last_error())
    return n


def mepic_attn_decode(cfg: Config, *, q, k_pool, v_pool, page_ids, pos_base, kv_len, q_pos, rope_table, out,
                      workspace, workspace_bytes: int, status, table_stride: int, batch: int,
                      sm_scale: float, stream=None) -> None:
    a = _DecodeArgsC(_ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_ids), _ptr(pos_base), _ptr(kv_len),
                     _ptr(q_pos), _ptr(rope_table), _ptr(out), _ptr(workspace), workspace_bytes, _ptr(status),
                     table_stride, batch, sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_decode(C.byref(c), C.byref(a), _stream_ptr(stream)))


def mepic_attn_decode_static(cfg: Config, *, q, k_pool, v_pool, page_ids, pos_base, kv_len, q_pos, rope_table, out,
                             status, table_stride: int, batch: int, sm_scale: float, stream=None) -> None:
    """Decode for callers that cannot allocate device memory: no workspace argument.

    The split-KV partials go to a fixed array inside the library (MEPIC_DECODE_STATIC_SCRATCH_BYTES
    per GPU) that all calls on a device share, so calls that overlap on the GPU race; sizes beyond
    the array are refused with MEPIC_E_INVAL.  Nothing is allocated by this call.
    """
    a = _DecodeArgsC(_ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_ids), _ptr(pos_base), _ptr(kv_len),
                     _ptr(q_pos), _ptr(rope_table), _ptr(out), None, 0, _ptr(status), table_stride, batch, sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_decode_static(C.byref(c), C.byref(a), _stream_ptr(stream)))


def mepic_pages_quantize(cfg: Config, *, src_pool, dst_pool, scales, pages, n_pages: int, status, stream=None) -> None:
    """bf16 pool -> e4m3 codes + one scale per (page, kv head) for the listed pages (all device tensors)."""
    c = cfg.c()
    _check(lib().mepic_pages_quantize(C.byref(c), _ptr(src_pool), _ptr(dst_pool), _ptr(scales), _ptr(pages), n_pages,
                                      _ptr(status), _stream_ptr(stream)))


def mepic_attn_decode_fp8(cfg: Config, *, q, k_pool, v_pool, k_scales, v_scales, page_ids, pos_base, kv_len, q_pos,
                          rope_table, out, workspace, workspace_bytes: int, status, table_stride: int, batch: int,
                          sm_scale: float, stream=None) -> None:
    a = _DecodeArgsC(_ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_ids), _ptr(pos_base), _ptr(kv_len),
                     _ptr(q_pos), _ptr(rope_table), _ptr(out), _ptr(workspace), workspace_bytes, _ptr(status),
                     table_stride, batch, sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_decode_fp8(C.byref(c), C.byref(a), _ptr(k_scales), _ptr(v_scales), _stream_ptr(stream)))


def mepic_decode_plan_max_ints(cfg: Config, batch: int, table_stride: int, n_sms: int = 0) -> int:
    c = cfg.c()
    n = int(lib().mepic_decode_plan_max_ints(C.byref(c), batch, table_stride, n_sms))
    if n == 0:
        raise MepicError(MEPIC_E_INVAL, mepic_last_error())
    return n


def mepic_decode_plan_build(cfg: Config, page_ids: np.ndarray, pos_base: np.ndarray, kv_len: np.ndarray,
                            n_sms: int = 0) -> np.ndarray:
    """Host block tables -> the grouped-decode plan (int32 array, opaque).  n_sms = 0: current device."""
    ids = np.ascontiguousarray(page_ids, dtype=np.int32)
    base = np.ascontiguousarray(pos_base, dtype=np.int32)
    lens = np.ascontiguousarray(kv_len, dtype=np.int32)
    batch, stride = ids.shape
    assert base.shape == ids.shape and lens.shape == (batch,)
    cap = mepic_decode_plan_max_ints(cfg, batch, stride, n_sms)
    out = np.empty(cap, dtype=np.int32)
    used = C.c_size_t(0)
    c = cfg.c()
    _check(lib().mepic_decode_plan_build(C.byref(c), ids.ctypes.data, base.ctypes.data, lens.ctypes.data, batch, stride,
                                         n_sms, out.ctypes.data, cap, C.byref(used)))
    return out[:used.value].copy()


def mepic_decode_plan_patch(cfg: Config, plan_host: np.ndarray, page_ids: np.ndarray, pos_base: np.ndarray,
                            kv_len: np.ndarray):
    """Patch ``plan_host`` in place after requests gained pages -> list of (first int, count) ranges that changed."""
    ids = np.ascontiguousarray(page_ids, dtype=np.int32)
    base = np.ascontiguousarray(pos_base, dtype=np.int32)
    lens = np.ascontiguousarray(kv_len, dtype=np.int32)
    batch, stride = ids.shape
    assert plan_host.dtype == np.int32 and plan_host.flags["C_CONTIGUOUS"]
    ranges = np.zeros(4, dtype=np.int64)
    n = C.c_int32(0)
    c = cfg.c()
    _check(lib().mepic_decode_plan_patch(C.byref(c), plan_host.ctypes.data, ids.ctypes.data, base.ctypes.data, lens.ctypes.data,
                                         batch, stride, ranges.ctypes.data, C.byref(n)))
    return [(int(ranges[2 * k]), int(ranges[2 * k + 1])) for k in range(n.value)]


def mepic_attn_decode_grouped_workspace(cfg: Config, plan_host: np.ndarray) -> int:
    c = cfg.c()
    n = int(lib().mepic_attn_decode_grouped_workspace(C.byref(c), plan_host.ctypes.data))
    if n == 0:
        raise MepicError(MEPIC_E_INVAL, mepic_last_error())
    return n


def mepic_attn_decode_grouped(cfg: Config, *, q, k_pool, v_pool, plan, plan_host: np.ndarray, kv_len, q_pos, rope_table,
                              out, workspace, workspace_bytes: int, status, batch: int, sm_scale: float,
                              stream=None) -> None:
    a = _DecodeGroupedArgsC(_ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(plan), plan_host.ctypes.data, _ptr(kv_len),
                            _ptr(q_pos), _ptr(rope_table), _ptr(out), _ptr(workspace), workspace_bytes, _ptr(status),
                            batch, sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_decode_grouped(C.byref(c), C.byref(a), _stream_ptr(stream)))


def mepic_attn_prefill_workspace(cfg: Config, batch: int, row_offsets_host: np.ndarray) -> int:
    c = cfg.c()
    ro = np.ascontiguousarray(row_offsets_host, dtype=np.int32)
    n = int(lib().mepic_attn_prefill_workspace(C.byref(c), batch, ro.ctypes.data))
    if n == 0:
        raise MepicError(MEPIC_E_INVAL, mepic_last_error())
    return n


def mepic_attn_prefill(cfg: Config, *, q_new, k_new, v_new, row_offsets, q_slot, k_pool, v_pool, page_ids,
                       pos_base, kv_len, rope_table, out, workspace, workspace_bytes: int, status,
                       row_offsets_host: np.ndarray, table_stride: int, batch: int, sm_scale: float,
                       stream=None) -> None:
    ro = np.ascontiguousarray(row_offsets_host, dtype=np.int32)
    a = _PrefillArgsC(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(row_offsets), _ptr(q_slot), _ptr(k_pool),
                      _ptr(v_pool), _ptr(page_ids), _ptr(pos_base), _ptr(kv_len), _ptr(rope_table), _ptr(out),
                      _ptr(workspace), workspace_bytes, _ptr(status), ro.ctypes.data, table_stride, batch,
                      sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_prefill(C.byref(c), C.byref(a), _stream_ptr(stream)))


def mepic_attn_prefill_fp8(cfg: Config, *, q_new, k_new, v_new, row_offsets, q_slot, k_pool, v_pool, k_scales, v_scales,
                           page_ids, pos_base, kv_len, rope_table, out, workspace, workspace_bytes: int, status,
                           row_offsets_host: np.ndarray, table_stride: int, batch: int, sm_scale: float,
                           stream=None) -> None:
    """Prefill over 8-bit pools: k_pool / v_pool are uint8 code pools, k_scales / v_scales their fp32 scales."""
    ro = np.ascontiguousarray(row_offsets_host, dtype=np.int32)
    a = _PrefillArgsC(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(row_offsets), _ptr(q_slot), _ptr(k_pool),
                      _ptr(v_pool), _ptr(page_ids), _ptr(pos_base), _ptr(kv_len), _ptr(rope_table), _ptr(out),
                      _ptr(workspace), workspace_bytes, _ptr(status), ro.ctypes.data, table_stride, batch,
                      sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_prefill_fp8(C.byref(c), C.byref(a), _ptr(k_scales), _ptr(v_scales), _stream_ptr(stream)))


def mepic_attn_decode_grouped_fp8(cfg: Config, *, q, k_pool, v_pool, k_scales, v_scales, plan, plan_host: np.ndarray, kv_len, q_pos,
                                  rope_table, out, workspace, workspace_bytes: int, status, batch: int, sm_scale: float,
                                  stream=None) -> None:
    """Sharing-aware decode over 8-bit pools: k_pool / v_pool are uint8 code pools, k_scales / v_scales their fp32 scales."""
    a = _DecodeGroupedArgsC(_ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(plan), plan_host.ctypes.data, _ptr(kv_len),
                            _ptr(q_pos), _ptr(rope_table), _ptr(out), _ptr(workspace), workspace_bytes, _ptr(status),
                            batch, sm_scale)
    c = cfg.c()
    _check(lib().mepic_attn_decode_grouped_fp8(C.byref(c), C.byref(a), _ptr(k_scales), _ptr(v_scales), _stream_ptr(stream)))
