"""Seeded synthetic inputs for the paged decode-attention path.

This module only *draws* inputs: request lengths, a scattered page placement, N(0,1) tensors
rounded to bf16, and the rotary cos/sin table that the path takes as an argument.  It holds none of
the method's arithmetic (no rotation, no softmax, no cache indexing beyond laying the synthetic
cache out) and is the one module that both the CPU oracle's tests and the CUDA path's tests load.

bf16 tensors are carried as ``numpy.uint16`` bit patterns.

Recipe: ``numpy.random.default_rng(seed)`` draws, in this order, the context lengths, the page
permutation and (last) the peak mask.  The tensors K pages, V pages, q, k_new, v_new (ids 0..4) are
drawn chunk by chunk from ``default_rng([seed, id, chunk])`` as fp32 standard normals and rounded to
nearest-even bf16.  Only the pages a request references are
filled; every other page of the pool, every slot at or past the append position of a request's last
page, and the page that unused block-table entries point at hold the NaN pattern 0x7FC0, so any read
outside a request's valid tokens poisons the result.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

BF16_NAN = np.uint16(0x7FC0)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to nearest-even bf16 and return the 16-bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


_CHUNK = 1 << 22


def _normal_bf16(seed: int, tensor_id: int, shape) -> np.ndarray:
    """N(0,1) fp32 draws rounded to bf16.

    The tensor is cut into chunks of 2**22 elements; chunk c is drawn from its own generator
    ``default_rng([seed, tensor_id, c])``, so the result does not depend on how many threads fill it.
    """
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)

    def fill(c: int) -> None:
        lo = c * _CHUNK
        hi = min(n, lo + _CHUNK)
        g = np.random.default_rng([seed, tensor_id, c])
        out[lo:hi] = f32_to_bf16_bits(g.standard_normal(hi - lo, dtype=np.float32))

    n_chunks = (n + _CHUNK - 1) // _CHUNK
    workers = min(n_chunks, len(os.sched_getaffinity(0)), 32)
    if workers <= 1:
        for c in range(n_chunks):
            fill(c)
    else:
        with ThreadPoolExecutor(workers) as ex:
            list(ex.map(fill, range(n_chunks)))
    return out.reshape(shape)


def rope_table(max_position: int, d: int, base: float):
    """cos/sin of p * base**(-2i/d), evaluated in fp64 and rounded once to fp32: [max_position, d/2]."""
    i = np.arange(d // 2, dtype=np.float64)
    inv_freq = np.power(float(base), -2.0 * i / d)
    ang = np.arange(max_position, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


@dataclass
class DecodeWorkload:
    name: str
    seed: int
    B: int
    Hq: int
    Hkv: int
    d: int
    page_size: int
    num_pages: int
    rope_base: float
    context_lens: np.ndarray          # int32 [B]; tokens cached before this step; <0 = inactive row
    block_table: np.ndarray           # int32 [B, max_pages_per_seq]
    k_cache: np.ndarray               # uint16 [num_pages, page_size, Hkv, d]
    v_cache: np.ndarray               # uint16 [num_pages, page_size, Hkv, d]
    q: np.ndarray                     # uint16 [B, Hq, d]   (un-rotated)
    k_new: np.ndarray                 # uint16 [B, Hkv, d]  (un-rotated)
    v_new: np.ndarray                 # uint16 [B, Hkv, d]
    rope_cos: np.ndarray              # float32 [max_position, d/2]
    rope_sin: np.ndarray              # float32 [max_position, d/2]
    poison_page: int
    extra: dict = field(default_factory=dict)
    window: int = 0                   # > 0: the step uses sliding-window attention of this length

    @property
    def max_pages_per_seq(self) -> int:
        return int(self.block_table.shape[1])

    @property
    def max_position(self) -> int:
        return int(self.rope_cos.shape[0])

    @property
    def max_context_len(self) -> int:
        """Largest number of tokens any request attends over in this step (cached + the new one)."""
        act = self.context_lens[self.context_lens >= 0]
        return int(act.max()) + 1 if act.size else 1

    @property
    def attended_tokens(self) -> int:
        act = self.context_lens[self.context_lens >= 0].astype(np.int64) + 1
        if self.window > 0:
            act = np.minimum(act, self.window)
        return int(act.sum())

    @property
    def kv_bytes(self) -> int:
        """K and V bytes of all attended tokens, all KV heads (the algorithmic read of the step)."""
        return self.attended_tokens * self.Hkv * self.d * 2 * 2


def make_workload(name: str, seed: int, B: int, Hq: int, Hkv: int, d: int, page_size: int,
                  num_pages: int, context_lens=None, len_range=None, rope_base: float = 10000.0,
                  peak_fraction: float = 0.0, peak_scale: float = 8.0,
                  inactive_rows=(), max_pages_per_seq: int | None = None) -> DecodeWorkload:
    """Draw one decode step's inputs.

    ``context_lens`` fixes the lengths; otherwise they are integers uniform in ``len_range``
    (both ends inclusive), drawn first.  ``inactive_rows`` get context_lens = -1 afterwards (their
    draws still happen so the other rows do not depend on them).
    """
    rng = np.random.default_rng(seed)
    if context_lens is None:
        lo, hi = len_range
        lens = rng.integers(lo, hi + 1, size=B).astype(np.int32)
    else:
        lens = np.asarray(context_lens, dtype=np.int32).copy()
        assert lens.shape == (B,)
    ps = page_size
    pages_per_req = (lens.astype(np.int64) + 1 + ps - 1) // ps      # room for the appended token
    n_used = int(pages_per_req.sum())
    assert n_used + 1 <= num_pages, "pool too small for the requests plus one poison page"
    perm = rng.permutation(num_pages).astype(np.int32)
    used = perm[:n_used]
    poison_page = int(perm[n_used])
    mp = int(pages_per_req.max()) if max_pages_per_seq is None else int(max_pages_per_seq)
    assert mp >= int(pages_per_req.max())
    block_table = np.full((B, mp), poison_page, dtype=np.int32)
    off = 0
    for b in range(B):
        n = int(pages_per_req[b])
        block_table[b, :n] = used[off:off + n]
        off += n

    k_cache = np.full((num_pages, ps, Hkv, d), BF16_NAN, dtype=np.uint16)
    v_cache = np.full((num_pages, ps, Hkv, d), BF16_NAN, dtype=np.uint16)
    k_cache[used] = _normal_bf16(seed, 0, (n_used, ps, Hkv, d))
    v_cache[used] = _normal_bf16(seed, 1, (n_used, ps, Hkv, d))
    q = _normal_bf16(seed, 2, (B, Hq, d))
    k_new = _normal_bf16(seed, 3, (B, Hkv, d))
    v_new = _normal_bf16(seed, 4, (B, Hkv, d))

    extra = {}
    if peak_fraction > 0.0:
        # One Bernoulli draw per (request, cached position); a hit scales that token's K row of
        # every KV head.  A power-of-two scale keeps the values exact in bf16.
        lmax = int(lens.max())
        mask = rng.random((B, lmax)) < peak_fraction
        n_hits = 0
        for b in range(B):
            pos = np.nonzero(mask[b, :int(lens[b])])[0]
            n_hits += pos.size
            pg = block_table[b, pos // ps]
            sl = pos % ps
            rows = bf16_bits_to_f32(k_cache[pg, sl]) * np.float32(peak_scale)
            k_cache[pg, sl] = f32_to_bf16_bits(rows)
        extra["peaked_positions"] = n_hits

    # Slots at or past the append position hold NaN until the path writes the new token.
    for b in range(B):
        L = int(lens[b])
        last = int(pages_per_req[b]) - 1
        first_bad = L - last * ps
        pg = block_table[b, last]
        k_cache[pg, first_bad:] = BF16_NAN
        v_cache[pg, first_bad:] = BF16_NAN

    for b in inactive_rows:
        lens[b] = -1

    max_position = int(lens.max()) + 1 if (lens >= 0).any() else 1
    cos, sin = rope_table(max_position, d, rope_base)
    return DecodeWorkload(name=name, seed=seed, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps,
                          num_pages=num_pages, rope_base=rope_base, context_lens=lens,
                          block_table=block_table, k_cache=k_cache, v_cache=v_cache, q=q,
                          k_new=k_new, v_new=v_new, rope_cos=cos, rope_sin=sin,
                          poison_page=poison_page, extra=extra)


def make_projection_inputs(seed: int, B: int, H: int, Hq: int, Hkv: int, d: int):
    """Hidden states x [B,H] ~ N(0,1) and QKV weights W [(Hq+2Hkv)*d, H] ~ N(0, 1/H), both bf16 bits
    (so that the projected features are ~N(0,1) like the q/k/v tensors of the other workloads)."""
    x = _normal_bf16(seed, 10, (B, H))
    n = (Hq + 2 * Hkv) * d
    w = bf16_bits_to_f32(_normal_bf16(seed, 11, (n, H))) * np.float32(1.0 / math.sqrt(H))
    return x, f32_to_bf16_bits(w)


GRAPH_SWEEP_BATCHES = (1, 8, 32, 128, 256)


def tiny() -> DecodeWorkload:
    """Batch 1, 8 query / 2 KV heads, head_dim 64, 512 cached tokens, append lands on a new page."""
    return make_workload("tiny", 1, B=1, Hq=8, Hkv=2, d=64, page_size=16, num_pages=64,
                         context_lens=[512], rope_base=10000.0)


def single_request() -> DecodeWorkload:
    """Batch 1, 32 query / 8 KV heads, head_dim 128, 4096 cached tokens, 4096-page pool."""
    return make_workload("single_request", 2, B=1, Hq=32, Hkv=8, d=128, page_size=16,
                         num_pages=4096, context_lens=[4096], rope_base=500000.0)


def continuous_batching() -> DecodeWorkload:
    """Batch 64, lengths uniform in [128, 8192], 32 query / 8 KV heads, 40000-page shared pool."""
    return make_workload("continuous_batching", 3, B=64, Hq=32, Hkv=8, d=128, page_size=16,
                         num_pages=40000, len_range=(128, 8192), rope_base=500000.0)


def long_context() -> DecodeWorkload:
    """Batch 4, 131072 cached tokens each, 64 query / 8 KV heads, 1% of K rows scaled by 8."""
    return make_workload("long_context", 4, B=4, Hq=64, Hkv=8, d=128, page_size=16,
                         num_pages=40000, context_lens=[131072] * 4, rope_base=500000.0,
                         peak_fraction=0.01, peak_scale=8.0)


def graph_sweep(batch: int) -> DecodeWorkload:
    """One bucket of the serving sweep: 28 query / 4 KV heads, page_size 32, lengths in [512, 2048]."""
    i = GRAPH_SWEEP_BATCHES.index(batch)
    pool = max(64, int(math.ceil(1.25 * 65 * batch)))
    return make_workload(f"graph_sweep_b{batch}", 50 + i, B=batch, Hq=28, Hkv=4, d=128,
                         page_size=32, num_pages=pool, len_range=(512, 2048), rope_base=1000000.0)


def gqa_group16() -> DecodeWorkload:
    """High-ratio GQA (32 query : 2 KV heads, the shape the paper reports its generated kernel
    collapsing on): batch 16, lengths uniform in [2048, 8192], head_dim 128, page_size 16."""
    return make_workload("gqa_group16", 60, B=16, Hq=32, Hkv=2, d=128, page_size=16, num_pages=10000,
                         len_range=(2048, 8192), rope_base=10000.0)


def sliding_window_4k() -> DecodeWorkload:
    """Sliding-window decode (window 4096, the variant the paper wires in for one model family):
    batch 32, lengths uniform in [4096, 12288], 32 query / 8 KV heads, head_dim 128, page_size 16."""
    w = make_workload("sliding_window_4k", 61, B=32, Hq=32, Hkv=8, d=128, page_size=16, num_pages=26000,
                      len_range=(4096, 12288), rope_base=1000000.0)
    w.window = 4096
    return w


def qwen3_like_b32() -> DecodeWorkload:
    """A layer shaped like the paper's Qwen3 family: 32 query / 8 KV heads, head_dim 128, per-head Q/K
    RMSNorm before the rotation; batch 32, lengths uniform in [512, 2048].  ``extra['rope_variants']``
    names the prelude options (norm weights 1 + 0.1 N(0,1), seeded)."""
    w = make_workload("qwen3_like_b32", 76, B=32, Hq=32, Hkv=8, d=128, page_size=16, num_pages=32 * 132 + 8,
                      len_range=(512, 2048), rope_base=1000000.0)
    g = np.random.default_rng([76, 20])
    w.extra["rope_variants"] = dict(
        q_norm_weight=f32_to_bf16_bits((1 + 0.1 * g.standard_normal(128)).astype(np.float32)),
        k_norm_weight=f32_to_bf16_bits((1 + 0.1 * g.standard_normal(128)).astype(np.float32)), norm_eps=1e-6)
    return w


def glm4_like_b32() -> DecodeWorkload:
    """A layer shaped like the paper's GLM-4 family: 32 query / 2 KV heads (the 32:2 ratio), head_dim
    128, rotary embedding on the first 64 elements only, interleaved pairs; batch 32, lengths uniform
    in [512, 2048].  The rope tables are [max_position, 32]."""
    w = make_workload("glm4_like_b32", 77, B=32, Hq=32, Hkv=2, d=128, page_size=16, num_pages=32 * 132 + 8,
                      len_range=(512, 2048), rope_base=1000000.0)
    w.rope_cos, w.rope_sin = rope_table(w.max_position, 64, w.rope_base)
    w.extra["rope_variants"] = dict(rotary_dim=64, interleaved=True)
    return w


NAMED = {
    "tiny": tiny,
    "single_request": single_request,
    "continuous_batching": continuous_batching,
    "long_context": long_context,
    **{f"graph_sweep_b{b}": (lambda b=b: graph_sweep(b)) for b in GRAPH_SWEEP_BATCHES},
    "gqa_group16": gqa_group16,
    "sliding_window_4k": sliding_window_4k,
    "qwen3_like_b32": qwen3_like_b32,
    "glm4_like_b32": glm4_like_b32,
}
