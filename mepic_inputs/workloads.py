"""Seeded synthetic workloads shaped like RAG / agent prompts.

Each workload is a pool of reusable document chunks (token-id arrays), a list
of requests (each an ordered list of segments: references to pool chunks and
request-private prompt pieces), a page pool of random bf16 K/V, and random
query / new-row tensors.  The five named configurations stand in for the
retrieval-augmented QA prompts the paper evaluates on (1.4k-2.2k tokens,
61-98 % of them reusable chunk tokens, Table 1) and for its 2-16 chunk
long-prompt sweep; no item of those datasets is used or reproduced.

Nothing here builds a page table, rotates a vector or computes attention:
this module only draws random numbers and lays out request structure.
Every array is a pure function of ``(0, config_index)`` through
``numpy.random.default_rng``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

from .bf16 import f32_to_bf16_bits

CONFIG_NAMES = {
    1: "tiny_decode",
    2: "llama3_8b_decode",
    3: "first_block_prefill",
    4: "long_prompt_decode",
    5: "mixed_serving",
}

# Segment kinds, shared vocabulary with the C ABI (0 = chunk, 1 = prompt).
KIND_CHUNK = 0
KIND_PROMPT = 1


@dataclass
class Request:
    """One request: ordered segments, each ``(kind, value)``.

    ``(KIND_CHUNK, i)`` refers to ``Workload.chunks[i]``; ``(KIND_PROMPT, n)``
    is a request-private prompt piece of ``n`` tokens.
    """
    request_id: int
    segments: List[Tuple[int, int]]


@dataclass
class PrefillRows:
    """Un-rotated bf16 bit patterns of the rows a prefill call recomputes."""
    q_new: np.ndarray   # uint16 [R, Hq, D]
    k_new: np.ndarray   # uint16 [R, Hkv, D]
    v_new: np.ndarray   # uint16 [R, Hkv, D]


@dataclass
class Workload:
    index: int
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int
    rope_theta: float
    sm_scale: float
    q_std: float
    pad_token_id: int
    num_pages: int
    max_position: int
    chunks: List[np.ndarray]
    decode_requests: List[Request]
    prefill_requests: List[Request] = field(default_factory=list)
    seed_words: Tuple[int, ...] = (0, 0)

    # ---- random tensors (drawn on demand; large ones are never cached) ----
    def _rng(self, stream: int, sub: int = 0) -> np.random.Generator:
        return np.random.default_rng(list(self.seed_words) + [stream, sub])

    def kv_pool(self, num_pages: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
        """bf16 bits ``[num_pages, Hkv, P, D]`` for K and for V, ~N(0,1).

        Filled per physical page, independent of any page table, so that two
        requests aliasing one page see the same K/V by construction.
        """
        n = self.num_pages if num_pages is None else num_pages
        shape = (n, self.n_kv_heads, self.page_size, self.head_dim)
        k = np.empty(shape, dtype=np.uint16)
        v = np.empty(shape, dtype=np.uint16)
        rng = self._rng(1)
        slab = max(1, (1 << 24) // int(np.prod(shape[1:])))
        for lo in range(0, n, slab):
            hi = min(n, lo + slab)
            k[lo:hi] = f32_to_bf16_bits(rng.standard_normal((hi - lo,) + shape[1:], dtype=np.float32))
            v[lo:hi] = f32_to_bf16_bits(rng.standard_normal((hi - lo,) + shape[1:], dtype=np.float32))
        return k, v

    def decode_q(self) -> np.ndarray:
        """bf16 bits ``[B, Hq, D]``: one un-rotated query token per decode request."""
        rng = self._rng(2)
        q = rng.standard_normal((len(self.decode_requests), self.n_q_heads, self.head_dim),
                                dtype=np.float32) * np.float32(self.q_std)
        return f32_to_bf16_bits(q)

    def prefill_rows(self, request_index: int, n_rows: int) -> PrefillRows:
        """New-row Q/K/V for prefill request ``request_index`` (``n_rows`` rows)."""
        rng = self._rng(3, request_index)
        q = rng.standard_normal((n_rows, self.n_q_heads, self.head_dim), dtype=np.float32)
        q *= np.float32(self.q_std)
        k = rng.standard_normal((n_rows, self.n_kv_heads, self.head_dim), dtype=np.float32)
        v = rng.standard_normal((n_rows, self.n_kv_heads, self.head_dim), dtype=np.float32)
        return PrefillRows(f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v))

    def chunk_tokens(self, i: int) -> np.ndarray:
        return self.chunks[i]


def _ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def _zipf_weights(n: int, s: float) -> np.ndarray:
    w = 1.0 / np.arange(1, n + 1, dtype=np.float64) ** s
    return w / w.sum()


def _pool_capacity(chunks: Sequence[np.ndarray], requests: Sequence[Request], page: int) -> int:
    """Enough pages for every chunk's shareable part plus every private page."""
    cap = sum(max(_ceil_div(len(c), page) - 1, 0) for c in chunks)
    for r in requests:
        for kind, val in r.segments:
            cap += 1 if kind == KIND_CHUNK else _ceil_div(val, page)
    return cap


def make_custom(index: int, *, n_q_heads: int, n_kv_heads: int, head_dim: int, page_size: int,
                rope_theta: float, sm_scale: float, q_std: float,
                n_pool_chunks: int, chunk_tokens, zipf_s: Optional[float],
                decode_chunks_per_request: Sequence[int] = (), decode_question: int = 0,
                prefill_chunks_per_request: Sequence[int] = (), prefill_question: int = 0,
                extra_pages: int = 0, name: Optional[str] = None, salt: int = 0) -> Workload:
    """Build a workload from explicit shape parameters.

    ``chunk_tokens`` is an int (every pool chunk that long) or a sequence with
    one length per pool chunk (lengths need not be page multiples).  A request
    draws its chunks without replacement, rank-k probability proportional to
    ``k**-zipf_s`` (uniform when ``zipf_s`` is None), independently of other
    requests; a non-zero question length appends one final prompt segment.
    """
    seed_words = (0, index) if salt == 0 else (0, index, salt)
    rng = np.random.default_rng(list(seed_words))
    lens = [int(chunk_tokens)] * n_pool_chunks if np.isscalar(chunk_tokens) else [int(x) for x in chunk_tokens]
    assert len(lens) == n_pool_chunks
    chunks = [rng.integers(1, 32000, size=n, dtype=np.int32) for n in lens]
    weights = None if zipf_s is None else _zipf_weights(n_pool_chunks, zipf_s)

    def draw(n_chunks: int, question: int, rid: int) -> Request:
        ids = rng.choice(n_pool_chunks, size=n_chunks, replace=False, p=weights)
        segs = [(KIND_CHUNK, int(i)) for i in ids]
        if question > 0:
            segs.append((KIND_PROMPT, int(question)))
        return Request(rid, segs)

    dec = [draw(n, decode_question, rid) for rid, n in enumerate(decode_chunks_per_request)]
    pre = [draw(n, prefill_question, 100000 + rid) for rid, n in enumerate(prefill_chunks_per_request)]
    num_pages = _pool_capacity(chunks, dec + pre, page_size) + extra_pages

    def kv_len_bound(r: Request) -> int:
        return sum(_ceil_div(len(chunks[v]) if k == KIND_CHUNK else v, page_size) * page_size
                   for k, v in r.segments)

    max_position = max([kv_len_bound(r) for r in dec + pre] + [page_size])
    return Workload(index=index, name=name or CONFIG_NAMES.get(index, f"custom{index}"),
                    n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                    page_size=page_size, rope_theta=float(rope_theta), sm_scale=float(sm_scale),
                    q_std=float(q_std), pad_token_id=0, num_pages=num_pages,
                    max_position=max_position, chunks=chunks, decode_requests=dec,
                    prefill_requests=pre, seed_words=seed_words)


def _lognormal_chunk_counts(index: int, n: int) -> List[int]:
    """Context lengths ~ lognormal(ln 4096, 0.8) clipped to [512, 32768], in 512-token chunks."""
    rng = np.random.default_rng([0, index, 7])
    lengths = np.clip(np.exp(rng.normal(np.log(4096.0), 0.8, size=n)), 512.0, 32768.0)
    return [int(min(max(round(x / 512.0), 1), 64)) for x in lengths]


def make_workload(index: int, *, scale: float = 1.0) -> Workload:
    """One of the five benchmark configurations (1-based ``index``).

    ``scale`` < 1 shrinks batch sizes and chunk counts proportionally for test
    cases that the CPU oracle must finish in seconds; ``scale == 1`` is the
    configuration as specified.
    """
    def s(n: int, lo: int = 1) -> int:
        return max(lo, int(round(n * scale)))

    inv_sqrt_128 = 1.0 / np.sqrt(128.0)
    if index == 1:
        return make_custom(1, n_q_heads=8, n_kv_heads=2, head_dim=64, page_size=16, rope_theta=1e4,
                           sm_scale=0.125, q_std=1.0, n_pool_chunks=3, chunk_tokens=128, zipf_s=None,
                           decode_chunks_per_request=[2] * 4, decode_question=32)
    if index == 2:
        # Q arrives pre-scaled by 1/sqrt(D); the softmax scale is therefore 1.
        return make_custom(2, n_q_heads=32, n_kv_heads=8, head_dim=128, page_size=16, rope_theta=5e5,
                           sm_scale=1.0, q_std=inv_sqrt_128, n_pool_chunks=s(64, 4), chunk_tokens=512,
                           zipf_s=1.1, decode_chunks_per_request=[s(16, 2)] * s(32, 2), decode_question=64)
    if index == 3:
        return make_custom(3, n_q_heads=32, n_kv_heads=8, head_dim=128, page_size=16, rope_theta=5e5,
                           sm_scale=1.0, q_std=inv_sqrt_128, n_pool_chunks=s(128, 4), chunk_tokens=512,
                           zipf_s=1.1, prefill_chunks_per_request=[s(32, 2)] * s(8, 1), prefill_question=256)
    if index == 4:
        return make_custom(4, n_q_heads=32, n_kv_heads=8, head_dim=128, page_size=64, rope_theta=5e5,
                           sm_scale=1.0, q_std=inv_sqrt_128, n_pool_chunks=s(48, 4), chunk_tokens=2048,
                           zipf_s=1.2, decode_chunks_per_request=[s(32, 2)] * s(8, 1), decode_question=0)
    if index == 5:
        counts = _lognormal_chunk_counts(5, s(128, 2))
        if scale < 1.0:
            counts = [max(1, int(round(c * scale))) for c in counts]
        return make_custom(5, n_q_heads=40, n_kv_heads=8, head_dim=128, page_size=16, rope_theta=5e5,
                           sm_scale=float(inv_sqrt_128), q_std=1.0, n_pool_chunks=s(256, 8), chunk_tokens=512,
                           zipf_s=1.0, decode_chunks_per_request=counts, decode_question=64,
                           prefill_chunks_per_request=[s(16, 2)] * s(4, 1), prefill_question=s(1792, 64))
    raise ValueError(f"unknown configuration index {index}")
