"""CPU oracle for attention over a page-aligned, position-free chunk KV cache.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, fp64 statement of
what the MEPIC hot path computes.  The CUDA library never imports, links or
calls it, and it never imports the library; only the tests, the smoke check
and the CPU-baseline leg of the benchmark may use it.

What it states, and where the paper fixes it:

* Scheduling path (Section 3.2, Algorithm 1): chunk segments are padded at the
  front and prompt segments at the back so that every chunk starts on a KV
  block boundary; the last prompt segment is left unpadded (Section 3.2.1).
  A chunk's identity is its padded token sequence (Section 3.2.3, "KV Block
  Allocation"); its first KV block is private to each request and the
  remaining blocks are shared by every request that uses the chunk
  (Section 3.2.3, Section 3.3.1).  Under memory pressure zero-reference chunk
  objects are reclaimed whole, least recently used first, and only then; a
  request is rejected when free plus reclaimable blocks cannot supply its
  demand (Section 3.2.3 "Eviction Policy"; Algorithm 1, admission check).
* Computation path (Section 3.3): recomputed K/V rows are written straight
  into their assigned pages (Section 3.3.2); pages hold keys WITHOUT rotary
  position embedding, and the rotation is applied to K when the attention
  operator reads it (Section 3.3.3).  The result is therefore ordinary softmax
  attention with RoPE applied at each token's assigned position: that
  definition is what `decode_attention` and `prefill_attention` write out.

Readings taken where the paper is silent (each also listed in the design
notes): split-half ("rotate_half") RoPE pairing with inverse frequencies
theta**(-2i/D) and no frequency scaling; V is never rotated; a token's
position is its index in the padded logical sequence, i.e. block-table entry
e starts at position e*P; pad slots are ordinary attended tokens; causality
is by logical slot while rotation is by position; free pages are handed out
first-in-first-out starting from 0..num_pages-1, and released pages rejoin the
queue in ascending order.

Parity unpinned by the paper: the RoPE pairing convention and the physical
page-id assignment order (the paper gives neither); they are pinned only by
the specification above, which the oracle and the library implement
independently.
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

KIND_CHUNK = 0
KIND_PROMPT = 1


class Reject(Exception):
    """Algorithm 1's Reject: the pool cannot supply the blocks a call needs."""


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# Scheduling path (Section 3.2, Algorithm 1): integer work, exact.
# ----------------------------------------------------------------------------

@dataclass
class OracleTable:
    page_ids: List[int]
    pos_base: List[int]
    kv_len: int
    recompute_slots: List[int]


class OracleStore:
    """Page pool + chunk index, keyed by chunk CONTENT (no hash function)."""

    def __init__(self, page_size: int, num_pages: int, pad_token_id: int = 0):
        self.P = int(page_size)
        self.num_pages = int(num_pages)
        self.pad = int(pad_token_id)
        self.free = deque(range(self.num_pages))
        self.chunks: Dict[Tuple[int, ...], dict] = {}
        self.requests: Dict[int, dict] = {}
        self.dedup_hits = 0
        self.tick = 0
        self.chunks_evicted = 0
        self.pages_evicted = 0
        self.remote = None              # see attach_remote

    # Algorithm 1 "resolve HBM residency and remote availability" / Section 3.2.3 eviction: a second tier that
    # keeps the K/V of evicted chunks (here: copies of the page arrays) and gives them back on the next use.
    def attach_remote(self, k_pool: np.ndarray, v_pool: np.ndarray, capacity_pages: int) -> None:
        if self.remote is not None:
            raise ValueError("already attached")
        self.remote = {"k": k_pool, "v": v_pool, "cap": int(capacity_pages), "used": 0, "chunks": {}, "tick": 0,
                       "spilled": 0, "fetched": 0}

    def _spill(self, key, pages) -> None:
        r = self.remote
        r["tick"] += 1
        if key in r["chunks"]:
            r["chunks"][key]["last_use"] = r["tick"]        # shared pages never change once computed
            return
        if len(pages) > r["cap"]:
            return
        while r["cap"] - r["used"] < len(pages):            # the tier drops its own least recently used chunks
            victim = min(r["chunks"], key=lambda k: r["chunks"][k]["last_use"])
            r["used"] -= len(r["chunks"].pop(victim)["kv"])
        r["chunks"][key] = {"kv": [(r["k"][p].copy(), r["v"][p].copy()) for p in pages], "last_use": r["tick"]}
        r["used"] += len(pages)
        r["spilled"] += 1

    def _touch(self, key) -> None:
        self.tick += 1
        self.chunks[key]["last_use"] = self.tick

    # Section 3.2.3 "Eviction Policy" + Algorithm 1 admission check: under pressure, whole zero-reference chunk
    # objects are reclaimed, least recently used first; chunks the call is about to use are protected; if that
    # cannot cover the demand the call is rejected and nothing is reclaimed.
    def _make_room(self, need: int, protect=()) -> bool:
        if need <= len(self.free):
            return True
        cand = [(c["last_use"], k) for k, c in self.chunks.items()
                if c["refs"] == 0 and c["shared"] and k not in protect]
        if len(self.free) + sum(len(self.chunks[k]["shared"]) for _, k in cand) < need:
            return False
        for _, k in sorted(cand, key=lambda x: x[0]):
            if need <= len(self.free):
                break
            gone = self.chunks.pop(k)
            if self.remote is not None and not gone["uncomputed"]:
                self._spill(k, gone["shared"])
            pages = sorted(gone["shared"])
            self.free.extend(pages)
            self.chunks_evicted += 1
            self.pages_evicted += len(pages)
        return True

    # Section 3.2.1: leading pad so that the chunk fills whole blocks.
    def canonical_chunk(self, tokens: Sequence[int]) -> Tuple[int, ...]:
        n = len(tokens)
        lead = (-n) % self.P
        return tuple([self.pad] * lead + [int(t) for t in tokens])

    # Section 3.2.2 / 3.2.3: residency lookup, then allocation of the shareable blocks.
    def register_chunk(self, tokens: Sequence[int]):
        if len(tokens) == 0:
            raise ValueError("empty chunk")
        key = self.canonical_chunk(tokens)
        if key in self.chunks:
            self.dedup_hits += 1
            self._touch(key)
            return key, 1, list(self.chunks[key]["shared"])
        n_pages = len(key) // self.P
        n_shared = n_pages - 1          # first block is private per request
        if not self._make_room(n_shared):
            raise Reject("no space for shared pages")
        shared = [self.free.popleft() for _ in range(n_shared)]
        self.chunks[key] = {"shared": shared, "refs": 0, "n_pages": n_pages, "last_use": 0, "uncomputed": False}
        self._touch(key)
        r = self.remote
        if r is not None and shared and key in r["chunks"]:      # not in HBM, but a remote copy exists: bring it back
            r["tick"] += 1
            r["chunks"][key]["last_use"] = r["tick"]
            for p, (kpage, vpage) in zip(shared, r["chunks"][key]["kv"]):
                r["k"][p] = kpage
                r["v"][p] = vpage
            r["fetched"] += 1
            return key, 2, list(shared)
        return key, 0, list(shared)

    # Section 3.3.1: a newly encountered chunk (nobody has its K/V) is recomputed whole by the next request
    # that uses it; cached chunks recompute their first block only.
    def mark_uncomputed(self, key) -> None:
        c = self.chunks[key]
        if c["refs"] != 0:
            raise ValueError("chunk is aliased by live requests")
        c["uncomputed"] = True

    # Algorithm 1, last stage: walk the segments in order and assign blocks.
    def build_block_table(self, request_id: int, segments: Sequence[Tuple[int, object]]) -> OracleTable:
        if request_id in self.requests:
            raise ValueError("request already has a table")
        segs = [(k, v) for (k, v) in segments if not (k == KIND_PROMPT and int(v) == 0)]
        if not segs:
            raise ValueError("no tokens")
        need = 0
        for i, (kind, val) in enumerate(segs):
            if kind == KIND_CHUNK:
                if val not in self.chunks:
                    raise KeyError("chunk not registered")
                need += 1
            else:
                need += -(-int(val) // self.P)
        protect = {v for k, v in segs if k == KIND_CHUNK}
        if not self._make_room(need, protect):
            raise Reject("no space for private pages")     # nothing was allocated or reclaimed
        pages: List[int] = []
        private: List[int] = []
        recompute: List[int] = []
        used: List[Tuple[int, ...]] = []
        kv_len = 0
        for i, (kind, val) in enumerate(segs):
            start = len(pages) * self.P
            if kind == KIND_CHUNK:
                c = self.chunks[val]
                first = self.free.popleft()
                private.append(first)
                pages.append(first)
                pages.extend(c["shared"])
                n_rec = self.P * c["n_pages"] if c["uncomputed"] else self.P
                c["uncomputed"] = False
                recompute.extend(range(start, start + n_rec))
                c["refs"] += 1
                self._touch(val)
                used.append(val)
                kv_len = len(pages) * self.P
            else:
                n = int(val)
                n_pages = -(-n // self.P)
                for _ in range(n_pages):
                    pg = self.free.popleft()
                    private.append(pg)
                    pages.append(pg)
                last = (i == len(segs) - 1)
                seg_len = n if last else n_pages * self.P      # trailing pad unless final
                recompute.extend(range(start, start + seg_len))
                kv_len = start + seg_len
        pos_base = [e * self.P for e in range(len(pages))]
        self.requests[request_id] = {"private": private, "chunks": used, "entries": len(pages)}
        return OracleTable(pages, pos_base, kv_len, recompute)

    def release(self, request_id: int) -> None:
        r = self.requests.pop(request_id)
        for key in r["chunks"]:
            self.chunks[key]["refs"] -= 1
            self._touch(key)
        for pg in sorted(r["private"]):
            self.free.append(pg)

    def stats(self) -> dict:
        shared = sum(len(c["shared"]) for c in self.chunks.values())
        private = sum(len(r["private"]) for r in self.requests.values())
        return {
            "pages_total": self.num_pages,
            "pages_free": len(self.free),
            "pages_shared_held": shared,
            "pages_private_held": private,
            "chunks_resident": len(self.chunks),
            "chunk_refs": sum(c["refs"] for c in self.chunks.values()),
            "dedup_hits": self.dedup_hits,
            "unshared_equivalent_pages": sum(r["entries"] for r in self.requests.values()),
            "live_requests": len(self.requests),
            "chunks_evicted": self.chunks_evicted,
            "pages_evicted": self.pages_evicted,
            "chunks_spilled": self.remote["spilled"] if self.remote else 0,
            "chunks_fetched": self.remote["fetched"] if self.remote else 0,
            "remote_chunks": len(self.remote["chunks"]) if self.remote else 0,
            "remote_pages": self.remote["used"] if self.remote else 0,
        }


# ----------------------------------------------------------------------------
# Computation path (Section 3.3): fp64.
# ----------------------------------------------------------------------------

def rope_angles(pos: np.ndarray, head_dim: int, theta: float) -> np.ndarray:
    """phi[..., i] = pos * theta**(-2 i / D), i < D/2."""
    half = head_dim // 2
    inv_freq = np.float64(theta) ** (-2.0 * np.arange(half, dtype=np.float64) / head_dim)
    return np.asarray(pos, dtype=np.float64)[..., None] * inv_freq


def rope_rotate(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, split-half pairing (i, i + D/2), on the last axis.

    ``pos`` broadcasts against ``x.shape[:-1]``.
    """
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    half = d // 2
    phi = rope_angles(np.broadcast_to(np.asarray(pos), x.shape[:-1]), d, theta)
    c, s = np.cos(phi), np.sin(phi)
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, lo * s + hi * c], axis=-1)


def gather_pages(pool: np.ndarray, page_ids: Sequence[int], kv_len: int) -> np.ndarray:
    """pool ``[num_pages, Hkv, P, D]`` -> logical ``[kv_len, Hkv, D]`` (same dtype)."""
    P = pool.shape[2]
    n_entries = -(-kv_len // P)
    g = pool[np.asarray(page_ids[:n_entries], dtype=np.int64)]        # [E, Hkv, P, D]
    g = np.transpose(g, (0, 2, 1, 3)).reshape(n_entries * P, pool.shape[1], pool.shape[3])
    return g[:kv_len]


def slot_positions(pos_base: Sequence[int], kv_len: int, P: int) -> np.ndarray:
    t = np.arange(kv_len, dtype=np.int64)
    return np.asarray(pos_base, dtype=np.int64)[t // P] + t % P


def _softmax_rows(s: np.ndarray) -> np.ndarray:
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / e.sum(axis=-1, keepdims=True)


def decode_attention_one(q_bits: np.ndarray, k_pool: np.ndarray, v_pool: np.ndarray,
                         page_ids: Sequence[int], pos_base: Sequence[int], kv_len: int,
                         q_pos: int, sm_scale: float, theta: float,
                         rotate: bool = True) -> np.ndarray:
    """One request, one query token: ``q_bits`` uint16 ``[Hq, D]`` -> fp64 ``[Hq, D]``.

    Section 3.3.3 as a definition: gather the request's pages, rotate every K
    row at its assigned position and q at ``q_pos``, then dense softmax
    attention; q head h reads KV head h // (Hq / Hkv).
    """
    P = k_pool.shape[2]
    K = gather_pages(k_pool, page_ids, kv_len)                          # [L, Hkv, D]
    V = gather_pages(v_pool, page_ids, kv_len)
    # pools are bf16 bit patterns, or already values (float64: de-quantised fp8 pages)
    K = bf16_bits_to_f64(K) if K.dtype == np.uint16 else K.astype(np.float64)
    V = bf16_bits_to_f64(V) if V.dtype == np.uint16 else V.astype(np.float64)
    q = bf16_bits_to_f64(q_bits)                                        # [Hq, D]
    if rotate:
        pos = slot_positions(pos_base, kv_len, P)
        K = rope_rotate(K, pos[:, None], theta)
        q = rope_rotate(q, np.int64(q_pos), theta)
    Hq, Hkv = q.shape[0], K.shape[1]
    G = Hq // Hkv
    out = np.empty_like(q)
    for h in range(Hq):
        kh = h // G
        s = sm_scale * (K[:, kh, :] @ q[h])                             # [L]
        p = _softmax_rows(s[None, :])[0]
        out[h] = p @ V[:, kh, :]
    return out


def decode_attention(q_bits: np.ndarray, k_pool: np.ndarray, v_pool: np.ndarray,
                     tables: Sequence[OracleTable], q_pos: Sequence[int],
                     sm_scale: float, theta: float) -> np.ndarray:
    """Batch of decode requests: ``q_bits`` uint16 ``[B, Hq, D]`` -> fp64 ``[B, Hq, D]``."""
    return np.stack([
        decode_attention_one(q_bits[b], k_pool, v_pool, t.page_ids, t.pos_base, t.kv_len,
                             q_pos[b], sm_scale, theta)
        for b, t in enumerate(tables)])


def commit_rows(k_pool: np.ndarray, v_pool: np.ndarray, page_ids: Sequence[int],
                q_slot: Sequence[int], k_new: np.ndarray, v_new: np.ndarray) -> None:
    """Section 3.3.2: write the new rows' bits, un-rotated, at (page, slot). In place."""
    P = k_pool.shape[2]
    for i, slot in enumerate(q_slot):
        pg = page_ids[slot // P]
        k_pool[pg, :, slot % P, :] = k_new[i]
        v_pool[pg, :, slot % P, :] = v_new[i]


def prefill_attention_one(q_new: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                          q_slot: Sequence[int], k_pool: np.ndarray, v_pool: np.ndarray,
                          page_ids: Sequence[int], pos_base: Sequence[int], kv_len: int,
                          sm_scale: float, theta: float,
                          rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Selective-recompute prefill for one request (Sections 3.3.1-3.3.3).

    Commits ``k_new/v_new`` (uint16 ``[R, Hkv, D]``) into the pools IN PLACE
    (bf16 pools; for float64 value pools see the comment below), then lets every new row i attend, causally by logical slot, over slots
    ``0..q_slot[i]`` of the paged context with K rotated at its position and
    the row's q rotated at the position of its own slot.  Returns fp64
    ``[R, Hq, D]`` (or only the listed ``rows``).
    """
    P = k_pool.shape[2]
    if k_pool.dtype == np.uint16:
        commit_rows(k_pool, v_pool, page_ids, q_slot, k_new, v_new)
        K = bf16_bits_to_f64(gather_pages(k_pool, page_ids, kv_len))
        V = bf16_bits_to_f64(gather_pages(v_pool, page_ids, kv_len))
    else:
        # value pools (float64: de-quantised 8-bit pages).  The commit into 8-bit pages is a separate step with
        # its own rule (commit_rows_fp8); the caller has made it and de-quantised, so the new rows are already in.
        K = gather_pages(k_pool, page_ids, kv_len).astype(np.float64)
        V = gather_pages(v_pool, page_ids, kv_len).astype(np.float64)
    pos = slot_positions(pos_base, kv_len, P)
    K = rope_rotate(K, pos[:, None], theta)
    sel = list(range(len(q_slot))) if rows is None else list(rows)
    Hq, Hkv = q_new.shape[1], K.shape[1]
    G = Hq // Hkv
    out = np.empty((len(sel), Hq, q_new.shape[2]), dtype=np.float64)
    for j, i in enumerate(sel):
        slot = int(q_slot[i])
        q = rope_rotate(bf16_bits_to_f64(q_new[i]), np.int64(pos[slot]), theta)   # [Hq, D]
        for h in range(Hq):
            kh = h // G
            s = sm_scale * (K[:slot + 1, kh, :] @ q[h])
            p = _softmax_rows(s[None, :])[0]
            out[j, h] = p @ V[:slot + 1, kh, :]
    return out


# --------------------------------------------------------------------------- fp8 (e4m3) pages
# The paper's related-work section names KV-cache quantisation as complementary and fixes no format.  This build's
# reading: OCP 8-bit floating point E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities; the
# all-ones exponent with all-ones mantissa is NaN; largest finite value 448), one scale per (page, kv head) and pool:
#     scale = max|x| / 448 over the block's non-NaN elements (1 if that maximum is zero), code = E4M3(x / scale) rounded to nearest, ties to even,
#     saturating; x~ = value(code) * scale.   All of it in float32, as the device does it.
E4M3_MAX = 448.0


def e4m3_values() -> np.ndarray:
    """The value of each of the 256 codes, from the format's definition (NaN for 0x7f and 0xff)."""
    out = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 0xF and m == 0x7:
            out[code] = np.nan
        elif e == 0:
            out[code] = sign * (m / 8.0) * 2.0 ** -6              # subnormal
        else:
            out[code] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """float32 -> code: round to nearest representable value, ties to the even mantissa, saturate at +-448."""
    x = np.asarray(x, dtype=np.float32)
    a = np.where(np.isnan(x), 0.0, np.abs(x)).astype(np.float64)        # NaN gets its code at the end
    sign = (np.signbit(x)).astype(np.uint8) << 7
    a = np.minimum(a, E4M3_MAX)
    # exponent of the binade; values below the smallest normal (2^-6) use the subnormal step 2^-9
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, -6, 8)
    step = 2.0 ** (e - 3)
    q = np.rint(a / step)                 # numpy rounds halves to even; a/step is exact (a has at most 24 bits)
    val = q * step                        # may have carried into the next binade: still representable
    val = np.minimum(val, E4M3_MAX)
    # value -> code
    with np.errstate(divide="ignore"):
        e2 = np.floor(np.log2(np.where(val > 0, val, 1.0)))
    e2 = np.clip(e2, -6, 8)
    normal = val >= 2.0 ** -6
    mant = np.where(normal, val / 2.0 ** e2 - 1.0, val / 2.0 ** -6) * 8.0
    code = np.where(normal, ((e2 + 7).astype(np.int64) << 3), 0) | np.rint(mant).astype(np.int64)
    code = code.astype(np.uint8) | sign
    return np.where(np.isnan(x), np.uint8(0x7F), code).astype(np.uint8)


def quantize_pages(pool_bits: np.ndarray):
    """bf16 pool ``[N, Hkv, P, D]`` -> (codes uint8 same shape, scales float32 ``[N, Hkv]``)."""
    x = bf16_bits_to_f64(pool_bits).astype(np.float32)                 # bf16 is exact in float32
    amax = np.where(np.isnan(x), np.float32(0), np.abs(x)).max(axis=(2, 3))       # NaN elements do not set the scale
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    y = (x / scale[:, :, None, None]).astype(np.float32)
    return e4m3_encode(y), scale


def dequantize_pages(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """-> float64 pool of the values the attention reads: value(code) * scale (the product in float64)."""
    return e4m3_values()[codes] * scale.astype(np.float64)[:, :, None, None]


def commit_rows_fp8(k_codes: np.ndarray, k_scale: np.ndarray, v_codes: np.ndarray, v_scale: np.ndarray,
                    page_ids: Sequence[int], q_slot: Sequence[int], k_new: np.ndarray, v_new: np.ndarray) -> None:
    """Section 3.3.2 for 8-bit pages: write the new rows (bf16 bits ``[R, Hkv, D]``) into the code pools. In place.

    The paper commits recomputed K/V straight into the assigned pages and names quantisation only as something that
    can be combined with it, so the rule for a page whose scale is a property of the whole (page, kv head) block is
    this build's reading: pages fill from slot 0 upwards, so a call whose rows for a block include the block's slot 0
    STARTS that block and sets its scale from the rows it writes there (largest non-NaN magnitude / 448, 1 if that is
    zero, as for whole pages); a call whose rows for a block do not include slot 0 APPENDS to it: the block keeps its
    scale and the new codes saturate at +-448 times that scale.  Codes are E4M3(x / scale), all in float32.
    """
    P = k_codes.shape[2]
    by_page: Dict[int, List[Tuple[int, int]]] = {}
    for i, slot in enumerate(q_slot):
        by_page.setdefault(int(page_ids[int(slot) // P]), []).append((int(slot) % P, i))
    for codes, scale, new in ((k_codes, k_scale, k_new), (v_codes, v_scale, v_new)):
        x = bf16_bits_to_f64(new).astype(np.float32)                                  # [R, Hkv, D]
        for pg, rows in by_page.items():
            idx = [i for _, i in rows]
            if any(s == 0 for s, _ in rows):
                amax = np.where(np.isnan(x[idx]), np.float32(0), np.abs(x[idx])).max(axis=(0, 2))      # per kv head
                scale[pg] = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
            with np.errstate(invalid="ignore", over="ignore"):
                y = (x[idx] / scale[pg][None, :, None]).astype(np.float32)
            c = e4m3_encode(y)
            for (s, _), ci in zip(rows, c):
                codes[pg, :, s, :] = ci


def merge_partials(m: np.ndarray, l: np.ndarray, o: np.ndarray) -> np.ndarray:
    """Combine split-KV partial results.

    Split s covers a subset of the keys and carries its running maximum
    ``m[s]``, its sum of ``exp(score - m[s])`` as ``l[s]`` and the matching
    un-normalised weighted sum of V as ``o[s]``.  The combination
    ``m* = max m``, ``l* = sum l e^{m-m*}``, ``o* = sum o e^{m-m*} / l*`` equals
    attention over the union of the subsets (standard log-sum-exp algebra; the
    paper has no counterpart, the split is this implementation's).
    """
    m = np.asarray(m, dtype=np.float64)
    w = np.exp(m - m.max(axis=0, keepdims=True))
    l_star = (np.asarray(l, dtype=np.float64) * w).sum(axis=0)
    return (np.asarray(o, dtype=np.float64) * w[..., None]).sum(axis=0) / l_star[..., None]


def partial_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, sm_scale: float):
    """(m, l, o) of one key subset, for ``merge_partials``: q ``[D]``, K/V ``[n, D]``."""
    s = sm_scale * (K @ q)
    m = s.max()
    e = np.exp(s - m)
    return m, e.sum(), e @ V
