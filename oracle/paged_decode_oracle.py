"""CPU oracle for single-token decode attention over a paged KV cache.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu-baseline leg may import this module; the
product path never does, and this module imports nothing from the CUDA path.  It is deliberately
plain and slow: fp64 numpy, one request and one head at a time, no tiling, no online softmax, no
splitting in the main routine.

What it follows.  The paper describes the path in prose only (Method, "Principle-Driven LLM Kernel
Generator", families (iii) and (iv); the runtime paragraph on the KV append; the multi-request
paragraph on the block-granular paged cache): a standalone RoPE kernel, a scatter kernel that writes
the new K/V vectors into the cache, and an online-softmax attention over the paged cache whose
cross-CTA partial results are merged.  The append paragraph fixes the semantics: writing the new
token and then attending over the length advanced by one is the same as a fused append-attention.
Online softmax and the log-sum-exp merge are exact re-associations of ``softmax(q K^T / sqrt(d)) V``,
so the oracle for attention is that definition written out.

Readings taken where the paper is silent (all listed in the design notes):
  * rotate-half pairing (x_i, x_{i+d/2}); cos/sin are inputs (fp32 table indexed by position);
  * the rotated value stored to the cache and to q is the round-to-nearest-even bf16 of the real
    number a*c - b*s (resp. b*c + a*s); evaluated here as two exact fp64 products, one fp64
    subtraction/addition and one *direct* fp64 -> bf16 rounding;
  * the new token's position is context_lens[b]; the query attends over positions 0..context_lens[b];
  * query head hq reads KV head hq // (Hq // Hkv); scale 1/sqrt(d); no mask other than the length;
  * split partials are normalised per split, with a natural-log log-sum-exp; an empty split has
    lse = -inf and a zero vector; a row with context_lens[b] < 0 is inactive (no write, zero output).

bf16 tensors are numpy uint16 bit patterns.  Every function is pinned by tests/test_oracle_pins.py
(brute force, closed forms, exact rational arithmetic, invariants); none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------------------------
# bf16 <-> fp64
# --------------------------------------------------------------------------------------------


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns as fp64 (bf16 is the top half of an fp32)."""
    u32 = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def f64_to_bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round fp64 directly to the nearest bf16, ties to even; returns uint16 bit patterns.

    bf16 has 8 significant bits, exponents like fp32 (normal from 2^-126, subnormal quantum 2^-133),
    largest finite value (2 - 2^-7) * 2^127.  The rounding is done on the real value in one step:
    scale by a power of two so that one unit is the bf16 quantum at x's magnitude, round to the
    nearest integer with ties to even (``numpy.rint``), scale back.  Both scalings are exact.
    """
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros(x.shape, dtype=np.uint16)
    sign = np.signbit(x)
    ax = np.abs(x)
    nan = np.isnan(x)
    finite = np.isfinite(x)
    with np.errstate(over="ignore", invalid="ignore"):
        _, e = np.frexp(np.where(finite, ax, 1.0))       # ax = m * 2^e, 0.5 <= m < 1
        e = np.maximum(e, -125)                          # below 2^-126 the quantum stays 2^-133
        # quantum = 2^(e-8): 8 significant bits for a value in [2^(e-1), 2^e)
        n = np.rint(np.ldexp(ax, 8 - e))                 # integer in [0, 256]
        r = np.ldexp(n, e - 8)                           # the rounded magnitude, exact in fp64
    big = r >= np.ldexp(1.0, 128)
    r32 = np.where(finite & ~big, r, 0.0).astype(np.float32)   # exact: r is a bf16 value
    bits = (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    bits = np.where(finite & big, np.uint16(0x7F80), bits)
    bits = np.where(np.isinf(x), np.uint16(0x7F80), bits)
    bits = np.where(sign, bits | np.uint16(0x8000), bits)
    bits = np.where(nan, np.uint16(0x7FC0), bits)
    out[...] = bits
    return out


# --------------------------------------------------------------------------------------------
# A1: rotary position embedding of the new q and k
# --------------------------------------------------------------------------------------------


def rope_rotate_f64(x: np.ndarray, cos_row: np.ndarray, sin_row: np.ndarray) -> np.ndarray:
    """Rotate-half RoPE of vectors x[..., d] (fp64) by angles given as cos/sin[d/2]; fp64 result.

    For i < d/2 the pair (x_i, x_{i+d/2}) becomes (x_i c_i - x_{i+d/2} s_i, x_{i+d/2} c_i + x_i s_i).
    """
    d = x.shape[-1]
    h = d // 2
    a = x[..., :h]
    b = x[..., h:]
    c = np.asarray(cos_row, dtype=np.float64)
    s = np.asarray(sin_row, dtype=np.float64)
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def rope_rotate_bf16(x_bits: np.ndarray, cos_row: np.ndarray, sin_row: np.ndarray) -> np.ndarray:
    """bf16 in, bf16 out: exact products, one fp64 add, one direct rounding to bf16."""
    return f64_to_bf16_rne(rope_rotate_f64(bf16_to_f64(x_bits), cos_row, sin_row))


# --------------------------------------------------------------------------------------------
# A1 + A2: rotate the new q/k and append the new k/v through the block table
# --------------------------------------------------------------------------------------------


def oracle_rope_kv_append(q, k_new, v_new, k_cache, v_cache, block_table, context_lens,
                          rope_cos, rope_sin, page_size):
    """Returns (q_rot, k_cache_after, v_cache_after); the inputs are not modified.

    q [B,Hq,d], k_new/v_new [B,Hkv,d], caches [num_pages, page_size, Hkv, d] (uint16 bf16 bits),
    block_table int32 [B, max_pages], context_lens int32 [B], rope_cos/sin fp32 [max_position, d/2].
    For an active row b with p = context_lens[b]: q[b] and k_new[b] are rotated by row p of the
    table; the rotated k and the untouched v go to page block_table[b, p // page_size], slot
    p % page_size, for every KV head.  Rows with context_lens[b] < 0 are left alone.
    """
    q_rot = np.array(q, dtype=np.uint16, copy=True)
    k_out = np.array(k_cache, dtype=np.uint16, copy=True)
    v_out = np.array(v_cache, dtype=np.uint16, copy=True)
    B = q_rot.shape[0]
    for b in range(B):
        p = int(context_lens[b])
        if p < 0:
            continue
        q_rot[b] = rope_rotate_bf16(q[b], rope_cos[p], rope_sin[p])
        k_rot = rope_rotate_bf16(k_new[b], rope_cos[p], rope_sin[p])
        page = int(block_table[b, p // page_size])
        slot = p % page_size
        k_out[page, slot] = k_rot
        v_out[page, slot] = v_new[b]
    return q_rot, k_out, v_out


# --------------------------------------------------------------------------------------------
# Prelude variants of A1: per-head RMSNorm, partial rotary, interleaved pairing
# --------------------------------------------------------------------------------------------


def rms_norm_bf16(x_bits: np.ndarray, weight_bits: np.ndarray, eps: float) -> np.ndarray:
    """Per-vector RMSNorm of bf16 vectors x[..., d] with a bf16 weight[d]; bf16 bits out.

    y = bf16( bf16( x / sqrt(mean(x^2) + eps) ) * w ): normalise in high precision, round to the
    model dtype, scale by the weight, round again (the attention-prelude family names the norm only
    as "per-head Q/K RMSNorm"; this is the usual decoder implementation).  The mean of squares is the
    exactly rounded sum (math.fsum) divided by d; eps is the fp32 value given.
    """
    import math
    x = bf16_to_f64(x_bits)
    w = bf16_to_f64(weight_bits)
    d = x.shape[-1]
    flat = x.reshape(-1, d)
    out = np.empty(flat.shape, dtype=np.uint16)
    eps64 = float(np.float32(eps))
    for r in range(flat.shape[0]):
        ss = math.fsum(float(v) * float(v) for v in flat[r])
        inv = 1.0 / math.sqrt(ss / d + eps64)
        y1 = f64_to_bf16_rne(flat[r] * inv)
        out[r] = f64_to_bf16_rne(bf16_to_f64(y1) * w)
    return out.reshape(x.shape)


def rope_rotate_variant_bf16(x_bits, cos_row, sin_row, rotary_dim=None, interleaved=False):
    """Rotation of the first rotary_dim elements of x[..., d] (bf16 bits), the rest passed through.

    Half-split pairing: (x_i, x_{i+R/2}); interleaved: (x_{2i}, x_{2i+1}); i < R/2, angle i.
    Same exact-then-round arithmetic as rope_rotate_bf16.
    """
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    d = x_bits.shape[-1]
    R = d if not rotary_dim else int(rotary_dim)
    out = x_bits.copy()
    x = bf16_to_f64(x_bits)
    c = np.asarray(cos_row, dtype=np.float64)[:R // 2]
    s = np.asarray(sin_row, dtype=np.float64)[:R // 2]
    if interleaved:
        a = x[..., 0:R:2]
        b = x[..., 1:R:2]
        out[..., 0:R:2] = f64_to_bf16_rne(a * c - b * s)
        out[..., 1:R:2] = f64_to_bf16_rne(b * c + a * s)
    else:
        a = x[..., :R // 2]
        b = x[..., R // 2:R]
        out[..., :R // 2] = f64_to_bf16_rne(a * c - b * s)
        out[..., R // 2:R] = f64_to_bf16_rne(b * c + a * s)
    return out


def oracle_rope_kv_append_ex(q, k_new, v_new, k_cache, v_cache, block_table, context_lens,
                             rope_cos, rope_sin, page_size, rotary_dim=None, interleaved=False,
                             q_norm_weight=None, k_norm_weight=None, norm_eps=0.0):
    """oracle_rope_kv_append with the prelude variants: optional RMSNorm of q / k head vectors first,
    then the (partial, half-split or interleaved) rotation, then the append.  v is never touched."""
    q_rot = np.array(q, dtype=np.uint16, copy=True)
    k_out = np.array(k_cache, dtype=np.uint16, copy=True)
    v_out = np.array(v_cache, dtype=np.uint16, copy=True)
    for b in range(q_rot.shape[0]):
        p = int(context_lens[b])
        if p < 0:
            continue
        qb = q[b] if q_norm_weight is None else rms_norm_bf16(q[b], q_norm_weight, norm_eps)
        kb = k_new[b] if k_norm_weight is None else rms_norm_bf16(k_new[b], k_norm_weight, norm_eps)
        q_rot[b] = rope_rotate_variant_bf16(qb, rope_cos[p], rope_sin[p], rotary_dim, interleaved)
        k_rot = rope_rotate_variant_bf16(kb, rope_cos[p], rope_sin[p], rotary_dim, interleaved)
        page = int(block_table[b, p // page_size])
        slot = p % page_size
        k_out[page, slot] = k_rot
        v_out[page, slot] = v_new[b]
    return q_rot, k_out, v_out


# --------------------------------------------------------------------------------------------
# Attention-prelude fusion (kernel family (i)): QKV projection feeding A1/A2
# --------------------------------------------------------------------------------------------


def oracle_qkv_projection(x_bits, w_qkv_bits, Hq, Hkv, d):
    """x [B,H] bf16, W_qkv [(Hq+2Hkv)*d, H] bf16 ([N,K] layout: one output feature per row, rows
    ordered q heads, k heads, v heads).  y = x W^T in fp64, rounded once to bf16.

    Returns (q [B,Hq,d], k_new [B,Hkv,d], v_new [B,Hkv,d]) as bf16 bits.  (The paper's family (i)
    fuses "QKV projection + RoPE"; its template GEMV stores weights [N,K]; no bias is mentioned.)
    """
    x = bf16_to_f64(x_bits)
    w = bf16_to_f64(w_qkv_bits)
    y = f64_to_bf16_rne(x @ w.T)
    B = x.shape[0]
    q = y[:, :Hq * d].reshape(B, Hq, d)
    k = y[:, Hq * d:(Hq + Hkv) * d].reshape(B, Hkv, d)
    v = y[:, (Hq + Hkv) * d:].reshape(B, Hkv, d)
    return q, k, v


def oracle_qkv_rope_kv_append(x_bits, w_qkv_bits, k_cache, v_cache, block_table, context_lens,
                              rope_cos, rope_sin, page_size, Hq, Hkv, d):
    """Projection, then the plain A1 + A2 on its bf16 results.  Returns (q_rot, k_cache, v_cache)."""
    q, k_new, v_new = oracle_qkv_projection(x_bits, w_qkv_bits, Hq, Hkv, d)
    return oracle_rope_kv_append(q, k_new, v_new, k_cache, v_cache, block_table, context_lens,
                                 rope_cos, rope_sin, page_size)


def oracle_oproj_residual_rmsnorm(attn_out_bits, w_o_bits, residual_bits, norm_weight_bits, eps):
    """Output projection + residual add + post-RMSNorm (kernel family (v)).

    h = bf16(residual + attn_out W_o^T) with the sum in fp64 and one rounding; normed =
    rms_norm_bf16(h, weight, eps).  attn_out [B,K], W_o [N,K], residual [B,N], weight [N]: bf16 bits.
    Returns (h bits, normed bits).
    """
    a = bf16_to_f64(attn_out_bits)
    w = bf16_to_f64(w_o_bits)
    h = f64_to_bf16_rne(bf16_to_f64(residual_bits) + a @ w.T)
    return h, rms_norm_bf16(h, norm_weight_bits, eps)


# --------------------------------------------------------------------------------------------
# A4 + A5 as one definition: softmax(q K^T * scale) V per query head over the gathered pages
# --------------------------------------------------------------------------------------------


def gather_kv(cache, block_table_row, n_tokens, page_size, kv_head):
    """Dense fp64 [n_tokens, d] of one request's one KV head, logical order, via the block table."""
    d = cache.shape[-1]
    out = np.empty((n_tokens, d), dtype=np.float64)
    for t0 in range(0, n_tokens, page_size):
        page = int(block_table_row[t0 // page_size])
        n = min(page_size, n_tokens - t0)
        out[t0:t0 + n] = bf16_to_f64(cache[page, :n, kv_head, :])
    return out


def oracle_paged_decode_attn(q_rot, k_cache, v_cache, block_table, context_lens, page_size,
                             new_tokens=1, softmax_scale=None, return_lse=False, window=0):
    """out fp64 [B,Hq,d] (and lse fp64 [B,Hq], natural log, of the scaled scores).

    Row b attends over positions 0 .. n_b - 1 with n_b = context_lens[b] + new_tokens, or, with a
    sliding window (window > 0; the variant the paper's per-model adaptations mention), over its last
    `window` positions max(0, n_b - window) .. n_b - 1 only.  Inactive rows (context_lens[b] < 0)
    and rows with nothing to attend give a zero vector and lse = -inf.
    """
    q_rot = np.asarray(q_rot, dtype=np.uint16)
    B, Hq, d = q_rot.shape
    Hkv = k_cache.shape[2]
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(float(d)) if softmax_scale is None or softmax_scale <= 0 else float(softmax_scale)
    out = np.zeros((B, Hq, d), dtype=np.float64)
    lse = np.full((B, Hq), -np.inf, dtype=np.float64)
    for b in range(B):
        if int(context_lens[b]) < 0:
            continue
        n = int(context_lens[b]) + int(new_tokens)
        if n <= 0:
            continue
        lo = max(0, n - int(window)) if window and window > 0 else 0
        for h in range(Hkv):
            K = gather_kv(k_cache, block_table[b], n, page_size, h)[lo:]
            V = gather_kv(v_cache, block_table[b], n, page_size, h)[lo:]
            for g in range(G):
                hq = h * G + g
                qv = bf16_to_f64(q_rot[b, hq])
                s = (K @ qv) * scale
                m = s.max()
                w = np.exp(s - m)
                z = w.sum()
                out[b, hq] = (w @ V) / z
                lse[b, hq] = m + np.log(z)
    if return_lse:
        return out, lse
    return out


# --------------------------------------------------------------------------------------------
# A4 / A5 separately: per-split partial results and their log-sum-exp merge
# --------------------------------------------------------------------------------------------


def oracle_split_partials(q_rot, k_cache, v_cache, block_table, context_lens, page_size,
                          split_starts, new_tokens=1, softmax_scale=None):
    """Partial attention over token ranges.

    ``split_starts[b]`` is an increasing list [t_0=0, t_1, ..., t_S]; split s of row b covers tokens
    t_s <= t < min(t_{s+1}, n_b).  Returns (partial_o fp64 [B,Hq,S,d], partial_lse fp64 [B,Hq,S]):
    each split's own softmax-weighted mean of V and the natural-log log-sum-exp of its scaled
    scores; an empty split has a zero vector and lse = -inf.
    """
    q_rot = np.asarray(q_rot, dtype=np.uint16)
    B, Hq, d = q_rot.shape
    Hkv = k_cache.shape[2]
    G = Hq // Hkv
    S = len(split_starts[0]) - 1
    scale = 1.0 / np.sqrt(float(d)) if softmax_scale is None or softmax_scale <= 0 else float(softmax_scale)
    po = np.zeros((B, Hq, S, d), dtype=np.float64)
    pl = np.full((B, Hq, S), -np.inf, dtype=np.float64)
    for b in range(B):
        if int(context_lens[b]) < 0:
            continue
        n = int(context_lens[b]) + int(new_tokens)
        for h in range(Hkv):
            K = gather_kv(k_cache, block_table[b], n, page_size, h)
            V = gather_kv(v_cache, block_table[b], n, page_size, h)
            for g in range(G):
                hq = h * G + g
                qv = bf16_to_f64(q_rot[b, hq])
                for s_i in range(S):
                    lo = int(split_starts[b][s_i])
                    hi = min(int(split_starts[b][s_i + 1]), n)
                    if hi <= lo:
                        continue
                    s = (K[lo:hi] @ qv) * scale
                    m = s.max()
                    w = np.exp(s - m)
                    z = w.sum()
                    po[b, hq, s_i] = (w @ V[lo:hi]) / z
                    pl[b, hq, s_i] = m + np.log(z)
    return po, pl


def oracle_splitkv_merge(partial_o, partial_lse):
    """Combine per-split results: out = sum_s w_s O_s / sum_s w_s with w_s = exp(lse_s - max lse).

    Splits with lse = -inf carry no weight; if every split of a row is empty the output is zero.
    Returns (out fp64 [B,Hq,d], lse fp64 [B,Hq]).
    """
    po = np.asarray(partial_o, dtype=np.float64)
    pl = np.asarray(partial_lse, dtype=np.float64)
    B, Hq, S, d = po.shape
    out = np.zeros((B, Hq, d), dtype=np.float64)
    lse = np.full((B, Hq), -np.inf, dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            M = pl[b, h].max()
            if not np.isfinite(M):
                continue
            w = np.exp(pl[b, h] - M)           # exp(-inf) = 0 for empty splits
            z = w.sum()
            out[b, h] = (w[:, None] * po[b, h]).sum(axis=0) / z
            lse[b, h] = M + np.log(z)
    return out, lse


def oracle_decode_step(w, softmax_scale=None, window=0):
    """Whole step on a workload object (fields as in the seeded generator): append, then attend.

    Returns (q_rot bits, k_cache_after bits, v_cache_after bits, out fp64).
    """
    q_rot, k_after, v_after = oracle_rope_kv_append(
        w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens,
        w.rope_cos, w.rope_sin, w.page_size)
    out = oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens,
                                   w.page_size, new_tokens=1, softmax_scale=softmax_scale, window=window)
    return q_rot, k_after, v_after, out
