"""Pins for the CPU oracle: each test checks it against something the mathematics fixes
(brute force, closed forms, exact rational arithmetic, invariants, a library routine), never against
its own formula retyped."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import paged_decode_oracle as O
from paper_2606_07665_b200 import workloads as W


# ---------------------------------------------------------------------------------------------
# helpers that are independent of the oracle's code
# ---------------------------------------------------------------------------------------------

def bf16_value(bits: int) -> Fraction:
    """Exact rational value of a finite bf16 pattern, from the format definition."""
    sign = -1 if bits & 0x8000 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    v = Fraction((1 << 7) + m, 1 << 7)
    return sign * (v * Fraction(2) ** (e - 127))


def fraction_to_bf16(x: Fraction) -> int:
    """Nearest-even bf16 pattern of an exact rational (finite range), by searching the neighbours."""
    sign = 0x8000 if x < 0 else 0
    ax = abs(x)
    lo, hi = 0, 0x7F80                      # patterns are monotone in value on [0, inf)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if bf16_value(mid) <= ax:
            lo = mid
        else:
            hi = mid
    v_lo = bf16_value(lo)
    v_hi = bf16_value(hi) if hi < 0x7F80 else Fraction(2) ** 128
    if ax - v_lo < v_hi - ax:
        r = lo
    elif ax - v_lo > v_hi - ax:
        r = hi
    else:
        r = lo if lo % 2 == 0 else hi
    return sign | r


def tiny_case(seed=0, B=2, Hq=6, Hkv=2, d=8, ps=4, lens=(9, 3), pool=16, **kw):
    return W.make_workload("t", seed, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps, num_pages=pool,
                           context_lens=list(lens), rope_base=100.0, **kw)


# ---------------------------------------------------------------------------------------------
# fp64 -> bf16 rounding
# ---------------------------------------------------------------------------------------------

def test_bf16_widening_matches_format_definition():
    pats = np.arange(0, 0x7F80, 37, dtype=np.uint16)
    got = O.bf16_to_f64(pats)
    for p, g in zip(pats.tolist(), got.tolist()):
        assert Fraction(g) == bf16_value(p)
    assert O.bf16_to_f64(np.array([0x3F80, 0xBF80, 0x4000], np.uint16)).tolist() == [1.0, -1.0, 2.0]


def test_bf16_rne_exhaustive_ties_and_neighbours():
    pats = np.arange(0, 0x7F7F, dtype=np.uint16)          # every finite pattern with a finite successor
    v = O.bf16_to_f64(pats)
    v_next = O.bf16_to_f64(pats + np.uint16(1))
    # representable values map to themselves
    assert np.array_equal(O.f64_to_bf16_rne(v), pats)
    assert np.array_equal(O.f64_to_bf16_rne(-v), pats | np.uint16(0x8000))
    mid = (v + v_next) / 2.0                                # exact in fp64
    even = np.where(pats % 2 == 0, pats, pats + np.uint16(1))
    assert np.array_equal(O.f64_to_bf16_rne(mid), even)
    assert np.array_equal(O.f64_to_bf16_rne(-mid), even | np.uint16(0x8000))
    assert np.array_equal(O.f64_to_bf16_rne(np.nextafter(mid, np.inf)), pats + np.uint16(1))
    assert np.array_equal(O.f64_to_bf16_rne(np.nextafter(mid, -np.inf)), pats)


def test_bf16_rne_overflow_and_specials():
    big = float(O.bf16_to_f64(np.array([0x7F7F], np.uint16))[0])
    half_ulp = 2.0 ** 119
    got = O.f64_to_bf16_rne(np.array([big + half_ulp, np.nextafter(big + half_ulp, 0), np.inf, -np.inf,
                                      -0.0, 2.0 ** -140]))
    assert got.tolist() == [0x7F80, 0x7F7F, 0x7F80, 0xFF80, 0x8000, 0x0000]
    assert O.f64_to_bf16_rne(np.array([np.nan]))[0] & 0x7FFF > 0x7F80


def test_bf16_rne_avoids_double_rounding_through_fp32():
    # 1 + 2^-8 + 2^-30 is above the bf16 tie 1 + 2^-8; rounding to fp32 first lands on the tie and
    # then rounds to even (down).  The direct rounding must go up.
    x = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert O.f64_to_bf16_rne(np.array([x]))[0] == 0x3F81
    via_f32 = W.f32_to_bf16_bits(np.array([x], dtype=np.float64).astype(np.float32))[0]
    assert via_f32 == 0x3F80


def test_bf16_rne_matches_torch_on_fp32_representable_values():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    x32 = (rng.standard_normal(200000) * np.exp(rng.uniform(-30, 30, 200000))).astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.f64_to_bf16_rne(x32.astype(np.float64)), want)


def test_bf16_rne_against_rationals_random():
    rng = np.random.default_rng(6)
    x = rng.standard_normal(300) * np.exp(rng.uniform(-95, 88, 300))
    got = O.f64_to_bf16_rne(x)
    for xi, g in zip(x.tolist(), got.tolist()):
        assert g == fraction_to_bf16(Fraction(xi))


# ---------------------------------------------------------------------------------------------
# RoPE
# ---------------------------------------------------------------------------------------------

def test_rope_hand_example_pairs_first_and_second_half():
    # d=4: pair (x0,x2) turned by 90 degrees, pair (x1,x3) by 0 degrees.
    x = np.array([1.0, 2.0, 3.0, 4.0])
    got = O.rope_rotate_f64(x, np.array([0.0, 1.0]), np.array([1.0, 0.0]))
    assert got.tolist() == [-3.0, 2.0, 1.0, 4.0]


def test_rope_equals_complex_multiplication():
    rng = np.random.default_rng(7)
    d = 16
    x = rng.standard_normal((5, d))
    th = rng.uniform(-3, 3, d // 2)
    z = (x[:, :d // 2] + 1j * x[:, d // 2:]) * np.exp(1j * th)
    got = O.rope_rotate_f64(x, np.cos(th), np.sin(th))
    assert np.allclose(got[:, :d // 2], z.real, rtol=0, atol=1e-15)
    assert np.allclose(got[:, d // 2:], z.imag, rtol=0, atol=1e-15)


def test_rope_preserves_norms():
    w = W.single_request()
    cos, sin = w.rope_cos.astype(np.float64), w.rope_sin.astype(np.float64)
    x = O.bf16_to_f64(w.q[0])
    for p in (1, 17, 4095, 4096):
        # fp32 table entries: c^2+s^2 differs from 1 by ~1e-7, so compare against the scaled norm
        r = O.rope_rotate_f64(x, cos[p], sin[p])
        h = w.d // 2
        pair_before = (x[:, :h] ** 2 + x[:, h:] ** 2) * (cos[p] ** 2 + sin[p] ** 2)
        pair_after = r[:, :h] ** 2 + r[:, h:] ** 2
        assert np.allclose(pair_after, pair_before, rtol=1e-14, atol=0)
    th = np.random.default_rng(1).uniform(-3, 3, w.d // 2)
    r = O.rope_rotate_f64(x, np.cos(th), np.sin(th))
    assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-15 * 8, atol=0)


def test_rope_relative_position_property():
    d, base = 32, 10000.0
    rng = np.random.default_rng(8)
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    inv = base ** (-2.0 * np.arange(d // 2) / d)

    def R(x, p):
        return O.rope_rotate_f64(x, np.cos(p * inv), np.sin(p * inv))

    for m, n in ((5, 3), (100, 37), (7, 7)):
        assert abs(R(q, m) @ R(k, n) - R(q, m - n) @ k) < 1e-12


def test_rope_position_zero_is_identity_on_bits():
    w = tiny_case(lens=(0, 5))
    q_rot, k_after, _ = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                w.block_table, w.context_lens, w.rope_cos,
                                                w.rope_sin, w.page_size)
    assert np.array_equal(q_rot[0], w.q[0])
    assert np.array_equal(k_after[w.block_table[0, 0], 0], w.k_new[0])
    assert not np.array_equal(q_rot[1], w.q[1])


def test_rope_bf16_matches_exact_rational_arithmetic():
    rng = np.random.default_rng(9)
    d = 8
    for trial in range(60):
        x = W.f32_to_bf16_bits(rng.standard_normal(d).astype(np.float32) * np.float32(2.0 ** rng.integers(-3, 4)))
        p = int(rng.integers(1, 100000))
        inv = 500000.0 ** (-2.0 * np.arange(d // 2) / d)
        c = np.cos(p * inv).astype(np.float32)
        s = np.sin(p * inv).astype(np.float32)
        got = O.rope_rotate_bf16(x, c, s)
        for i in range(d // 2):
            a, b = bf16_value(int(x[i])), bf16_value(int(x[i + d // 2]))
            ci, si = Fraction(float(c[i])), Fraction(float(s[i]))
            assert int(got[i]) == fraction_to_bf16(a * ci - b * si)
            assert int(got[i + d // 2]) == fraction_to_bf16(b * ci + a * si)


def test_rope_bf16_near_tie_is_rounded_from_the_exact_value():
    # a*c - b*s with a = 1 + 2^-7 (odd last bit), c = 1, b*s = -2^-8 - tiny => exact value just
    # above the tie between 0x3F81 and 0x3F82; an fp32 evaluation would lose the tiny term.
    a = np.array([0x3F81, 0x3F80], np.uint16)              # x = (1+2^-7, 1.0), d = 2
    c = np.array([1.0], np.float32)
    s = np.array([-(2.0 ** -8) * (1 + 2.0 ** -20)], np.float32)
    got = O.rope_rotate_bf16(a, c, s)
    exact = bf16_value(0x3F81) * 1 - bf16_value(0x3F80) * Fraction(float(s[0]))
    assert int(got[0]) == fraction_to_bf16(exact) == 0x3F82


# ---------------------------------------------------------------------------------------------
# append / indexing
# ---------------------------------------------------------------------------------------------

def test_append_changes_only_the_target_slots():
    w = tiny_case(lens=(8, 3, 0), B=3, ps=4, inactive_rows=())   # row 0 appends at a page boundary
    q_rot, k_after, v_after = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                      w.block_table, w.context_lens, w.rope_cos,
                                                      w.rope_sin, w.page_size)
    dk = k_after != w.k_cache
    dv = v_after != w.v_cache
    expect = np.zeros(w.k_cache.shape[:2], dtype=bool)
    for b, L in enumerate(w.context_lens.tolist()):
        expect[w.block_table[b, L // w.page_size], L % w.page_size] = True
    # all target slots held NaN before, so every element of a target slot changes
    assert np.array_equal(dk.all(axis=(2, 3)), expect) and np.array_equal(dk.any(axis=(2, 3)), expect)
    assert np.array_equal(dv.all(axis=(2, 3)), expect) and np.array_equal(dv.any(axis=(2, 3)), expect)
    for b, L in enumerate(w.context_lens.tolist()):
        pg, sl = w.block_table[b, L // w.page_size], L % w.page_size
        assert np.array_equal(v_after[pg, sl], w.v_new[b])
    assert w.context_lens[0] % w.page_size == 0 and w.block_table[0, 2] != w.poison_page


def test_append_skips_inactive_rows():
    w = tiny_case(lens=(8, 3), inactive_rows=(1,))
    q_rot, k_after, v_after = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                      w.block_table, w.context_lens, w.rope_cos,
                                                      w.rope_sin, w.page_size)
    assert np.array_equal(q_rot[1], w.q[1])
    changed_pages = np.unique(np.nonzero(k_after != w.k_cache)[0])
    assert changed_pages.tolist() == [int(w.block_table[0, 2])]
    out = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, w.page_size)
    assert np.all(out[1] == 0.0) and np.isfinite(out[0]).all()


# ---------------------------------------------------------------------------------------------
# attention
# ---------------------------------------------------------------------------------------------

def brute_force_attention(w, q_rot, k_cache, v_cache, new_tokens=1):
    """Pure-Python loops, written from the definition with explicit paged indexing."""
    G = w.Hq // w.Hkv
    out = np.zeros((w.B, w.Hq, w.d))
    for b in range(w.B):
        n = int(w.context_lens[b]) + new_tokens
        for hq in range(w.Hq):
            h = hq // G
            qv = [float(x) for x in W.bf16_bits_to_f32(q_rot[b, hq])]
            scores = []
            for t in range(n):
                page = int(w.block_table[b, t // w.page_size])
                krow = W.bf16_bits_to_f32(k_cache[page, t % w.page_size, h])
                scores.append(math.fsum(qv[j] * float(krow[j]) for j in range(w.d)) / math.sqrt(w.d))
            mx = max(scores)
            ws = [math.exp(s - mx) for s in scores]
            z = math.fsum(ws)
            for j in range(w.d):
                acc = []
                for t in range(n):
                    page = int(w.block_table[b, t // w.page_size])
                    acc.append(ws[t] * float(W.bf16_bits_to_f32(v_cache[page, t % w.page_size, h, j:j + 1])[0]))
                out[b, hq, j] = math.fsum(acc) / z
    return out


@pytest.mark.parametrize("cfg", [dict(), dict(Hq=4, Hkv=4, d=4, ps=2, lens=(5, 1)),
                                 dict(Hq=6, Hkv=1, d=6, ps=8, lens=(15, 16))])
def test_attention_matches_brute_force(cfg):
    w = tiny_case(seed=11, **cfg)
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    ref = brute_force_attention(w, q_rot, k_after, v_after)
    assert np.abs(out - ref).max() < 1e-14
    assert np.isfinite(out).all()          # NaN-poisoned slots and pages never reach the output


def test_single_token_context_returns_v_exactly():
    w = tiny_case(lens=(0, 0))
    _, _, _, out = O.oracle_decode_step(w)
    G = w.Hq // w.Hkv
    for b in range(w.B):
        for hq in range(w.Hq):
            assert np.array_equal(out[b, hq], O.bf16_to_f64(w.v_new[b, hq // G]))


def test_identical_keys_and_zero_query_give_mean_of_v():
    w = tiny_case(seed=12, lens=(10, 6))
    q_rot, k_after, v_after = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                      w.block_table, w.context_lens, w.rope_cos,
                                                      w.rope_sin, w.page_size)
    k_same = k_after.copy()
    k_same[:] = k_after[w.block_table[0, 0], 0, 0][None, None, None, :]
    out = O.oracle_paged_decode_attn(q_rot, k_same, v_after, w.block_table, w.context_lens, w.page_size)
    out0 = O.oracle_paged_decode_attn(np.zeros_like(q_rot), k_after, v_after, w.block_table,
                                      w.context_lens, w.page_size)
    G = w.Hq // w.Hkv
    for b in range(w.B):
        n = int(w.context_lens[b]) + 1
        for hq in range(w.Hq):
            rows = [O.bf16_to_f64(v_after[w.block_table[b, t // w.page_size], t % w.page_size, hq // G])
                    for t in range(n)]
            mean = np.mean(rows, axis=0)
            assert np.allclose(out[b, hq], mean, rtol=0, atol=1e-15)
            assert np.allclose(out0[b, hq], mean, rtol=0, atol=1e-15)


def test_physical_page_permutation_leaves_output_bit_identical():
    w = tiny_case(seed=13, lens=(13, 7), pool=20)
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    perm = np.random.default_rng(3).permutation(w.num_pages)
    k2 = np.empty_like(k_after)
    v2 = np.empty_like(v_after)
    k2[perm] = k_after
    v2[perm] = v_after
    bt2 = perm[w.block_table].astype(np.int32)
    out2 = O.oracle_paged_decode_attn(q_rot, k2, v2, bt2, w.context_lens, w.page_size)
    assert np.array_equal(out, out2)


def test_dominant_key_returns_its_value_exactly():
    w = tiny_case(seed=14, B=1, Hq=2, Hkv=2, d=8, lens=(11,))
    q_rot, k_after, v_after = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                      w.block_table, w.context_lens, w.rope_cos,
                                                      w.rope_sin, w.page_size)
    t_star = 6
    pg, sl = w.block_table[0, t_star // w.page_size], t_star % w.page_size
    qf = W.bf16_bits_to_f32(q_rot[0])
    k_after[pg, sl] = W.f32_to_bf16_bits(qf * np.float32(2.0 ** 12))    # score ~ 4096*|q|^2/sqrt(8)
    out = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, w.page_size)
    for h in range(2):
        assert np.array_equal(out[0, h], O.bf16_to_f64(v_after[pg, sl, h]))


def test_two_key_closed_form_pins_the_scale():
    # d = 4, q = (2,0,0,0), k0 = (1,0,0,0), k1 = 0: scores (2/sqrt(4), 0) = (1, 0)
    d, ps = 4, 2
    one, two = 0x3F80, 0x4000
    q = np.zeros((1, 1, d), np.uint16); q[0, 0, 0] = two
    k = np.zeros((3, ps, 1, d), np.uint16); k[2, 0, 0, 0] = one
    v = np.zeros((3, ps, 1, d), np.uint16); v[2, 0, 0, :] = one; v[2, 1, 0, :] = two
    bt = np.array([[2]], np.int32)
    out, lse = O.oracle_paged_decode_attn(q, k, v, bt, np.array([2], np.int32), ps, new_tokens=0,
                                          return_lse=True)
    e = math.e
    assert np.allclose(out[0, 0], (e * 1.0 + 2.0) / (e + 1.0), rtol=1e-15, atol=0)
    assert abs(lse[0, 0] - math.log(e + 1.0)) < 1e-15
    out2 = O.oracle_paged_decode_attn(q, k, v, bt, np.array([2], np.int32), ps, new_tokens=0,
                                      softmax_scale=1.0)
    assert np.allclose(out2[0, 0], (e * e + 2.0) / (e * e + 1.0), rtol=1e-15, atol=0)


def test_query_heads_read_their_own_kv_head():
    w = tiny_case(seed=15, Hq=6, Hkv=3, lens=(5, 9))
    q_rot, k_after, v_after = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                      w.block_table, w.context_lens, w.rope_cos,
                                                      w.rope_sin, w.page_size)
    for h in range(w.Hkv):
        v_after[:, :, h, :] = W.f32_to_bf16_bits(np.array([float(h + 1)], np.float32))[0]
    out = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, w.page_size)
    for hq in range(w.Hq):
        assert np.allclose(out[:, hq], float(hq // 2 + 1), rtol=1e-15, atol=0)


def test_matches_torch_sdpa_on_gathered_dense_kv():
    torch = pytest.importorskip("torch")
    w = W.make_workload("t", 21, B=3, Hq=8, Hkv=2, d=64, page_size=16, num_pages=40,
                        context_lens=[100, 37, 16], rope_base=10000.0)
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    G = w.Hq // w.Hkv
    for b in range(w.B):
        n = int(w.context_lens[b]) + 1
        pages = w.block_table[b, :(n + w.page_size - 1) // w.page_size]
        K = W.bf16_bits_to_f32(k_after[pages]).reshape(-1, w.Hkv, w.d)[:n].astype(np.float64)
        V = W.bf16_bits_to_f32(v_after[pages]).reshape(-1, w.Hkv, w.d)[:n].astype(np.float64)
        Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(G, dim=0)      # [Hq, n, d]
        Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(G, dim=0)
        Qt = torch.from_numpy(W.bf16_bits_to_f32(q_rot[b]).astype(np.float64))[:, None, :]
        ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt)[:, 0, :].numpy()
        assert np.abs(out[b] - ref).max() < 1e-13


def test_append_then_attend_equals_dense_attention_over_concatenation():
    # the equivalence the paper states: separate append + attention over length+1 == fused call
    w = tiny_case(seed=16, Hq=4, Hkv=2, d=8, lens=(7, 12))
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    G = w.Hq // w.Hkv
    for b in range(w.B):
        L = int(w.context_lens[b])
        p = L
        for hq in range(w.Hq):
            h = hq // G
            K_old = np.array([O.bf16_to_f64(w.k_cache[w.block_table[b, t // w.page_size], t % w.page_size, h])
                              for t in range(L)])
            V_old = np.array([O.bf16_to_f64(w.v_cache[w.block_table[b, t // w.page_size], t % w.page_size, h])
                              for t in range(L)])
            k_rot = O.bf16_to_f64(O.rope_rotate_bf16(w.k_new[b, h], w.rope_cos[p], w.rope_sin[p]))
            K = np.vstack([K_old, k_rot[None]])
            V = np.vstack([V_old, O.bf16_to_f64(w.v_new[b, h])[None]])
            s = K @ O.bf16_to_f64(q_rot[b, hq]) / math.sqrt(w.d)
            pw = np.exp(s - s.max())
            assert np.allclose(out[b, hq], pw @ V / pw.sum(), rtol=0, atol=1e-14)


# ---------------------------------------------------------------------------------------------
# split partials + merge
# ---------------------------------------------------------------------------------------------

def test_merge_of_any_partition_equals_unsplit():
    w = tiny_case(seed=17, lens=(29, 11), ps=4, pool=24)
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    _, lse = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens,
                                        w.page_size, return_lse=True)
    rng = np.random.default_rng(4)
    for trial in range(5):
        S = int(rng.integers(1, 7))
        starts = []
        for b in range(w.B):
            cuts = np.sort(rng.integers(0, 36, size=S - 1)).tolist()      # may repeat or exceed the length
            starts.append([0] + cuts + [64])
        po, pl = O.oracle_split_partials(q_rot, k_after, v_after, w.block_table, w.context_lens,
                                         w.page_size, starts)
        merged, mlse = O.oracle_splitkv_merge(po, pl)
        assert np.abs(merged - out).max() < 1e-13
        assert np.abs(mlse - lse).max() < 1e-13
    po, pl = O.oracle_split_partials(q_rot, k_after, v_after, w.block_table, w.context_lens,
                                     w.page_size, [[0, 64]] * w.B)
    merged, _ = O.oracle_splitkv_merge(po, pl)
    assert np.array_equal(merged, po[:, :, 0]) and np.array_equal(merged, out)


def test_merge_closed_form_and_empty_rows():
    po = np.zeros((1, 2, 3, 2)); pl = np.full((1, 2, 3), -np.inf)
    po[0, 0, 0] = [1.0, 2.0]; pl[0, 0, 0] = math.log(3.0)       # weight 3
    po[0, 0, 2] = [5.0, -2.0]; pl[0, 0, 2] = math.log(1.0)      # weight 1; split 1 empty
    out, lse = O.oracle_splitkv_merge(po, pl)
    assert np.allclose(out[0, 0], [(3 * 1 + 5) / 4, (3 * 2 - 2) / 4], rtol=1e-15)
    assert abs(lse[0, 0] - math.log(4.0)) < 1e-15
    assert np.all(out[0, 1] == 0.0) and lse[0, 1] == -np.inf


def test_peaked_workload_matches_brute_force():
    w = W.make_workload("p", 23, B=1, Hq=2, Hkv=1, d=8, page_size=4, num_pages=40,
                        context_lens=[120], rope_base=100.0, peak_fraction=0.2, peak_scale=8.0)
    assert w.extra["peaked_positions"] > 5
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    assert np.abs(out - brute_force_attention(w, q_rot, k_after, v_after)).max() < 1e-14


def test_sliding_window_pins():
    w = tiny_case(seed=18, lens=(29, 11), ps=4, pool=24)
    q_rot, k_after, v_after, full = O.oracle_decode_step(w)
    # a window at least as long as the context changes nothing
    assert np.array_equal(O.oracle_decode_step(w, window=30)[3], full)
    assert np.array_equal(O.oracle_decode_step(w, window=1000)[3], full)
    # a window of one token returns the newest v exactly
    one = O.oracle_decode_step(w, window=1)[3]
    G = w.Hq // w.Hkv
    for b in range(w.B):
        for hq in range(w.Hq):
            assert np.array_equal(one[b, hq], O.bf16_to_f64(w.v_new[b, hq // G]))
    # brute force over the last 7 tokens, written with explicit indexing
    win = O.oracle_decode_step(w, window=7)[3]
    for b in range(w.B):
        n = int(w.context_lens[b]) + 1
        for hq in range(w.Hq):
            h = hq // G
            toks = list(range(max(0, n - 7), n))
            qv = O.bf16_to_f64(q_rot[b, hq])
            sc = [float(O.bf16_to_f64(k_after[w.block_table[b, t // 4], t % 4, h]) @ qv) / math.sqrt(w.d) for t in toks]
            mx = max(sc)
            ws = [math.exp(x - mx) for x in sc]
            ref = sum(wt * O.bf16_to_f64(v_after[w.block_table[b, t // 4], t % 4, h]) for wt, t in zip(ws, toks)) / sum(ws)
            assert np.abs(win[b, hq] - ref).max() < 1e-14
    # tokens before the window may hold anything
    k_bad, v_bad = k_after.copy(), v_after.copy()
    for t in range(0, 30 - 7):
        k_bad[w.block_table[0, t // 4], t % 4] = 0x7FC0
        v_bad[w.block_table[0, t // 4], t % 4] = 0x7FC0
    again = O.oracle_paged_decode_attn(q_rot, k_bad, v_bad, w.block_table, w.context_lens, w.page_size, window=7)
    assert np.array_equal(again[0], win[0])


def test_rope_variants_reduce_to_the_plain_rotation():
    rng = np.random.default_rng(31)
    d = 16
    x = W.f32_to_bf16_bits(rng.standard_normal((5, d)).astype(np.float32))
    th = rng.uniform(-3, 3, d // 2)
    c, s = np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)
    # full rotary dim, half-split: identical bits to the plain routine
    assert np.array_equal(O.rope_rotate_variant_bf16(x, c, s), O.rope_rotate_bf16(x, c, s))
    # interleaved == plain rotation of the de-interleaved vector, re-interleaved
    deint = np.concatenate([x[:, 0::2], x[:, 1::2]], axis=-1)
    plain = O.rope_rotate_bf16(deint, c, s)
    want = np.empty_like(x)
    want[:, 0::2] = plain[:, :d // 2]
    want[:, 1::2] = plain[:, d // 2:]
    assert np.array_equal(O.rope_rotate_variant_bf16(x, c, s, interleaved=True), want)
    # partial rotary: tail untouched, head == plain rotation of the head slice with the first angles
    R = 8
    got = O.rope_rotate_variant_bf16(x, c, s, rotary_dim=R)
    assert np.array_equal(got[:, R:], x[:, R:])
    assert np.array_equal(got[:, :R], O.rope_rotate_bf16(x[:, :R], c[:R // 2], s[:R // 2]))
    gi = O.rope_rotate_variant_bf16(x, c, s, rotary_dim=R, interleaved=True)
    assert np.array_equal(gi[:, R:], x[:, R:])
    # hand example, interleaved, d = 4: pairs (x0,x1) by 90 degrees, (x2,x3) by 0
    hx = W.f32_to_bf16_bits(np.array([1.0, 2.0, 3.0, 4.0], np.float32))
    hv = O.rope_rotate_variant_bf16(hx, np.array([0.0, 1.0], np.float32), np.array([1.0, 0.0], np.float32),
                                    interleaved=True)
    assert W.bf16_bits_to_f32(hv).tolist() == [-2.0, 1.0, 3.0, 4.0]


def test_rms_norm_pins():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(32)
    d = 64
    x = W.f32_to_bf16_bits(rng.standard_normal((7, d)).astype(np.float32) * 3)
    ones = np.full(d, 0x3F80, np.uint16)
    w = W.f32_to_bf16_bits((1 + 0.1 * rng.standard_normal(d)).astype(np.float32))
    # hand example: x = (3, 4), unit weight, eps = 0: rms = sqrt(12.5)
    hx = W.f32_to_bf16_bits(np.array([3.0, 4.0], np.float32))
    hy = O.rms_norm_bf16(hx, np.array([0x3F80, 0x3F80], np.uint16), 0.0)
    assert hy.tolist() == O.f64_to_bf16_rne(np.array([3.0, 4.0]) / math.sqrt(12.5)).tolist()
    # unit weight: the result is within one bf16 rounding of torch's fp64 rms_norm (library routine)
    y = O.bf16_to_f64(O.rms_norm_bf16(x, ones, 1e-6))
    ref = torch.nn.functional.rms_norm(torch.from_numpy(O.bf16_to_f64(x)), (d,), eps=float(np.float32(1e-6))).numpy()
    assert np.abs(y - ref).max() <= 2.0 ** -8 * np.abs(ref).max()
    assert np.array_equal(O.f64_to_bf16_rne(ref), O.rms_norm_bf16(x, ones, 1e-6))
    # scaling the input by a power of two changes nothing when eps = 0
    x4 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(x) * np.float32(4.0))
    assert np.array_equal(O.rms_norm_bf16(x4, w, 0.0), O.rms_norm_bf16(x, w, 0.0))
    # the weight is applied after rounding the normalised value to bf16
    y1 = O.rms_norm_bf16(x, ones, 1e-6)
    want = O.f64_to_bf16_rne(O.bf16_to_f64(y1) * O.bf16_to_f64(w))
    assert np.array_equal(O.rms_norm_bf16(x, w, 1e-6), want)
    # mean of squares of the unit-weight output is ~1
    assert np.allclose(np.mean(y ** 2, axis=-1), 1.0, atol=2e-3)


def test_append_ex_defaults_equal_plain_append_and_norm_feeds_rotation():
    w = tiny_case(seed=33, Hq=4, Hkv=2, d=8, lens=(9, 3))
    plain = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table,
                                    w.context_lens, w.rope_cos, w.rope_sin, w.page_size)
    ex = O.oracle_rope_kv_append_ex(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table,
                                    w.context_lens, w.rope_cos, w.rope_sin, w.page_size)
    for a, b in zip(plain, ex):
        assert np.array_equal(a, b)
    wt = W.f32_to_bf16_bits(np.linspace(0.5, 1.5, 8).astype(np.float32))
    q_rot, k_after, v_after = O.oracle_rope_kv_append_ex(
        w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.rope_cos,
        w.rope_sin, w.page_size, q_norm_weight=wt, k_norm_weight=wt, norm_eps=1e-6)
    p = int(w.context_lens[0])
    want_q = O.rope_rotate_bf16(O.rms_norm_bf16(w.q[0], wt, 1e-6), w.rope_cos[p], w.rope_sin[p])
    assert np.array_equal(q_rot[0], want_q)
    assert np.array_equal(v_after, plain[2])          # v is never normalised


def test_qkv_projection_pins():
    rng = np.random.default_rng(41)
    Hq, Hkv, d, H, B = 4, 2, 8, 24, 3
    N = (Hq + 2 * Hkv) * d
    x = W.f32_to_bf16_bits(rng.standard_normal((B, H)).astype(np.float32))
    wq = W.f32_to_bf16_bits((rng.standard_normal((N, H)) / np.sqrt(H)).astype(np.float32))
    q, k, v = O.oracle_qkv_projection(x, wq, Hq, Hkv, d)
    assert q.shape == (B, Hq, d) and k.shape == (B, Hkv, d) and v.shape == (B, Hkv, d)
    # brute force with exact rationals: feature n of row b is sum_j x[b,j] * W[n,j], rounded once
    for b, n in ((0, 0), (1, Hq * d + 3), (2, N - 1), (1, 17)):
        acc = sum(bf16_value(int(x[b, j])) * bf16_value(int(wq[n, j])) for j in range(H))
        want = fraction_to_bf16(acc)
        flat = np.concatenate([q[b].ravel(), k[b].ravel(), v[b].ravel()])
        assert int(flat[n]) == want
    # selection weights: row n of W is a unit vector -> feature n copies an input element exactly
    sel = np.zeros((N, H), np.uint16)
    for n in range(N):
        sel[n, n % H] = 0x3F80
    q2, k2, v2 = O.oracle_qkv_projection(x, sel, Hq, Hkv, d)
    flat = np.concatenate([q2.reshape(B, -1), k2.reshape(B, -1), v2.reshape(B, -1)], axis=1)
    assert np.array_equal(flat, x[:, np.arange(N) % H])
    # the fused routine is the projection followed by the plain rotation + append
    w = tiny_case(seed=42, Hq=Hq, Hkv=Hkv, d=d, lens=(9, 3, 0), B=3)
    q_rot, k_after, v_after = O.oracle_qkv_rope_kv_append(x, wq, w.k_cache, w.v_cache, w.block_table,
                                                          w.context_lens, w.rope_cos, w.rope_sin,
                                                          w.page_size, Hq, Hkv, d)
    ref = O.oracle_rope_kv_append(q, k, v, w.k_cache, w.v_cache, w.block_table, w.context_lens,
                                  w.rope_cos, w.rope_sin, w.page_size)
    for a, bb in zip((q_rot, k_after, v_after), ref):
        assert np.array_equal(a, bb)


def test_oproj_residual_rmsnorm_pins():
    rng = np.random.default_rng(43)
    B, K, N = 3, 16, 8
    a = W.f32_to_bf16_bits(rng.standard_normal((B, K)).astype(np.float32))
    wo = W.f32_to_bf16_bits((rng.standard_normal((N, K)) / 4).astype(np.float32))
    res = W.f32_to_bf16_bits(rng.standard_normal((B, N)).astype(np.float32))
    nw = W.f32_to_bf16_bits((1 + 0.1 * rng.standard_normal(N)).astype(np.float32))
    h, normed = O.oracle_oproj_residual_rmsnorm(a, wo, res, nw, 1e-5)
    for b in range(B):
        for n in range(N):
            acc = bf16_value(int(res[b, n])) + sum(bf16_value(int(a[b, k])) * bf16_value(int(wo[n, k]))
                                                   for k in range(K))
            assert int(h[b, n]) == fraction_to_bf16(acc)            # residual + product, rounded once
    assert np.array_equal(normed, O.rms_norm_bf16(h, nw, 1e-5))
    # zero weights: h is the residual, bit for bit
    h0, _ = O.oracle_oproj_residual_rmsnorm(a, np.zeros_like(wo), res, nw, 1e-5)
    assert np.array_equal(h0, res)


def test_tiny_workload_oracle_result_is_frozen():
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = open(os.path.join(here, "tiny_oracle.txt")).read().splitlines()
    now = mod.summary().splitlines()
    assert len(stored) == len(now)
    for a, b in zip(stored, now):
        if a.startswith("out_head"):
            va = np.array([float(x) for x in a.split()[1:]])
            vb = np.array([float(x) for x in b.split()[1:]])
            assert np.allclose(va, vb, rtol=1e-12, atol=0), (a, b)
        else:
            assert a == b


# ---------------------------------------------------------------------------------------------
# Structural properties of softmax attention that hold for any inputs (they pin the oracle against
# the mathematics, not against another implementation)
# ---------------------------------------------------------------------------------------------

def _dense_case(seed, n_tokens=23, Hq=4, Hkv=2, d=8, ps=4):
    """One request whose cache is filled by the generator; returns bits ready for the attention oracle."""
    w = tiny_case(seed=seed, B=1, Hq=Hq, Hkv=Hkv, d=d, ps=ps, lens=(n_tokens,), pool=2 * (n_tokens // ps + 2))
    q_rot, k_after, v_after = O.oracle_rope_kv_append(w.q, w.k_new, w.v_new, w.k_cache, w.v_cache,
                                                      w.block_table, w.context_lens, w.rope_cos,
                                                      w.rope_sin, w.page_size)
    return w, q_rot, k_after, v_after


def test_output_is_a_convex_combination_of_the_values():
    # every output coordinate lies between the smallest and the largest value of that coordinate
    # among the attended tokens of the head's KV head, and equals neither unless all are equal
    w, q_rot, k, v = _dense_case(21)
    out = O.oracle_paged_decode_attn(q_rot, k, v, w.block_table, w.context_lens, w.page_size)
    n = int(w.context_lens[0]) + 1
    G = w.Hq // w.Hkv
    for hq in range(w.Hq):
        vals = O.gather_kv(v, w.block_table[0], n, w.page_size, hq // G)
        assert (out[0, hq] > vals.min(axis=0)).all() and (out[0, hq] < vals.max(axis=0)).all()


def test_token_order_inside_the_cache_does_not_matter():
    # attention is a sum over tokens: storing the same (k, v) pairs in a different token order gives
    # the same output up to fp64 summation order
    w, q_rot, k, v = _dense_case(22)
    out = O.oracle_paged_decode_attn(q_rot, k, v, w.block_table, w.context_lens, w.page_size)
    n = int(w.context_lens[0]) + 1
    perm = np.random.default_rng(5).permutation(n)
    k2, v2 = k.copy(), v.copy()
    ps = w.page_size
    for new_t, old_t in enumerate(perm):
        po, so = w.block_table[0, old_t // ps], old_t % ps
        pn, sn = w.block_table[0, new_t // ps], new_t % ps
        k2[pn, sn], v2[pn, sn] = k[po, so], v[po, so]
    out2 = O.oracle_paged_decode_attn(q_rot, k2, v2, w.block_table, w.context_lens, w.page_size)
    assert np.allclose(out, out2, rtol=1e-13, atol=1e-15)


def test_duplicating_every_token_changes_nothing_but_the_lse():
    # softmax over a multiset with every element twice has the same weights ratio: the output is
    # unchanged and the log-sum-exp grows by exactly ln 2
    w, q_rot, k, v = _dense_case(23, n_tokens=11)
    n = int(w.context_lens[0]) + 1
    out, lse = O.oracle_paged_decode_attn(q_rot, k, v, w.block_table, w.context_lens, w.page_size,
                                          return_lse=True)
    ps = w.page_size
    pages2 = (2 * n + ps - 1) // ps
    k2 = np.zeros((pages2, ps) + k.shape[2:], k.dtype)
    v2 = np.zeros_like(k2)
    for t in range(2 * n):
        src = t % n
        k2[t // ps, t % ps] = k[w.block_table[0, src // ps], src % ps]
        v2[t // ps, t % ps] = v[w.block_table[0, src // ps], src % ps]
    bt2 = np.arange(pages2, dtype=np.int32)[None, :]
    out2, lse2 = O.oracle_paged_decode_attn(q_rot, k2, v2, bt2, np.array([2 * n], np.int32), ps,
                                            new_tokens=0, return_lse=True)
    assert np.allclose(out, out2, rtol=1e-13, atol=1e-15)
    assert np.allclose(lse2 - lse, math.log(2.0), rtol=0, atol=1e-13)


def test_scaling_q_by_a_power_of_two_equals_scaling_the_softmax_scale():
    # scores are bilinear in q: doubling q (exact in bf16) is the same as doubling softmax_scale
    w, q_rot, k, v = _dense_case(24)
    q2 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(q_rot) * np.float32(2.0))
    d = w.d
    a = O.oracle_paged_decode_attn(q2, k, v, w.block_table, w.context_lens, w.page_size)
    b = O.oracle_paged_decode_attn(q_rot, k, v, w.block_table, w.context_lens, w.page_size,
                                   softmax_scale=2.0 / math.sqrt(d))
    assert np.allclose(a, b, rtol=1e-13, atol=1e-15)
