"""GPU parity of the attention-prelude fusion (QKV projection + RoPE + KV append in one launch).

The projection accumulates in fp32 in an order of its own, so its bf16 results may differ from the
correctly rounded fp64 ones by one unit in the last place now and then; everything downstream of
those results is exact.  The test therefore demands that almost all stored values equal the oracle's
bit for bit and that the rest are within one bf16 step of the pair's magnitude, that nothing outside
the target slots changes, and that attention over the resulting cache matches the oracle's."""
import numpy as np
import pytest

from oracle import paged_decode_oracle as O
from paper_2606_07665_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _close_bf16(got_bits, ref_bits, what):
    got = W.bf16_bits_to_f32(got_bits).astype(np.float64)
    ref = W.bf16_bits_to_f32(ref_bits).astype(np.float64)
    assert np.isfinite(got).all(), what
    exact = float(np.mean(got_bits == ref_bits))
    d = ref.shape[-1]
    mag = np.sqrt(ref[..., :d // 2] ** 2 + ref[..., d // 2:] ** 2)
    mag = np.concatenate([mag, mag], axis=-1)
    assert (np.abs(got - ref) <= 2.0 ** -6 * mag + 1e-30).all(), (what, float(np.abs(got - ref).max()))
    assert exact >= 0.97, (what, exact)
    return exact


@pytest.mark.parametrize("B,H,Hq,Hkv,d,ps", [
    (1, 256, 8, 2, 128, 16),
    (5, 320, 4, 4, 128, 16),          # K not a multiple of the 256-wide stage: zero-filled tail
    (8, 1024, 8, 2, 64, 16),
    (12, 512, 28, 4, 128, 32),        # batch tile of 16 with empty rows
    (16, 512, 8, 2, 128, 16),         # largest batch on the warp-MMA kernel
    (17, 320, 8, 2, 128, 16),         # smallest batch on the tcgen05 kernel; K not a multiple of its 256-wide stage
    (31, 768, 8, 2, 128, 16),
    (40, 256, 4, 2, 64, 16),          # head_dim 64: two overlapping 24-pair tiles per head
    (4, 4096, 32, 8, 128, 16),        # 8B-class layer: 6144 x 4096 weights
    (33, 256, 4, 2, 128, 16),
    (96, 512, 8, 2, 128, 16),         # widest batch tile that still takes 256-wide stages
    (100, 512, 8, 2, 64, 16),         # 104-row tile, 128-wide stages
    (128, 1024, 8, 2, 128, 32),       # exactly one 128-row tile
    (200, 320, 4, 4, 128, 16),        # two tiles of 104 rows, K not a multiple of the stage width
    (64, 4096, 32, 8, 128, 16),       # 8B-class layer, batched
])
def test_qkv_prelude_matches_oracle(B, H, Hq, Hkv, d, ps):
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    rng = np.random.default_rng(B * 1000 + H)
    lens = rng.integers(0, 300, size=B).tolist()
    inactive = (B - 1,) if B > 2 else ()
    w = W.make_workload("prelude", 80 + B, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps,
                        num_pages=B * (300 // ps + 2) + 4, context_lens=lens, rope_base=10000.0,
                        inactive_rows=inactive)
    x, wq = W.make_projection_inputs(90 + B, B, H, Hq, Hkv, d)
    q_ref, k_ref, v_ref = O.oracle_qkv_rope_kv_append(x, wq, w.k_cache, w.v_cache, w.block_table,
                                                      w.context_lens, w.rope_cos, w.rope_sin, ps, Hq, Hkv, d)
    st = runner.DecodeStep(w, num_splits=2)
    x_dev = torch.from_numpy(x.view(np.int16)).cuda()
    w_dev = torch.from_numpy(wq.view(np.int16)).cuda()
    st.q_rot.fill_(0x7FC0)
    ac.ac_qkv_rope_kv_append(x_dev, w_dev, H, st.q_rot, st.k_cache, st.v_cache, st.stride_page,
                             st.stride_token, st.stride_head, st.block_table, w.max_pages_per_seq,
                             st.context_lens, st.rope_cos, st.rope_sin, w.max_position, B, Hq, Hkv, d, ps,
                             w.num_pages, st.status_flag)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    active = w.context_lens >= 0
    q_gpu = runner.bits_of(st.q_rot)
    _close_bf16(q_gpu[active], q_ref[active], "q")
    assert (q_gpu[~active] == 0x7FC0).all()                      # inactive rows are not written
    k_gpu, v_gpu = st.cache_bits()
    target = np.zeros(k_ref.shape[:2], dtype=bool)
    for b in np.nonzero(active)[0]:
        L = int(w.context_lens[b])
        target[w.block_table[b, L // ps], L % ps] = True
    assert np.array_equal(k_gpu[~target], w.k_cache[~target])    # nothing else moved
    assert np.array_equal(v_gpu[~target], w.v_cache[~target])
    _close_bf16(k_gpu[target], k_ref[target], "k")
    ev = _close_bf16(v_gpu[target], v_ref[target], "v")
    # attention over what the kernel produced, against the oracle over the same bits
    out_ref = O.oracle_paged_decode_attn(q_gpu, k_gpu, v_gpu, w.block_table, w.context_lens, ps)
    st.attention()
    torch.cuda.synchronize()
    err = np.abs(st.out_f64() - out_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    print(f"[prelude] B={B} H={H}: exact fraction of v = {ev:.4f}")


@pytest.mark.parametrize("kw", [
    dict(rotary_dim=64),                                       # partial rotary, half-split: partners in sister CTAs
    dict(interleaved=True),
    dict(rotary_dim=32, interleaved=True),
    dict(norm=True),                                           # per-head Q/K RMSNorm, then full rotary
    dict(norm=True, rotary_dim=64, interleaved=True),          # Qwen3- and GLM-4-style options together
    dict(norm="q_only", rotary_dim=64),
])
@pytest.mark.parametrize("B,d", [(5, 128), (16, 64), (40, 128), (100, 64), (200, 128)])
def test_qkv_prelude_variants_bit_exact_when_the_projection_is_exact(kw, B, d):
    """ac_qkv_rope_kv_append_ex: small-integer x and W make the projection exact, so q and both pools must
    equal the oracle's chain (projection -> RMSNorm -> partial / interleaved rotation -> append) bit for
    bit, on the warp-MMA kernel (up to 16 rows) and on the tcgen05 kernel (one ragged tile of 40 or 104
    rows, two tiles of 104)."""
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    kw = dict(kw)
    norm = kw.pop("norm", False)
    rotary_dim = min(kw.get("rotary_dim", 0), d)
    interleaved = kw.get("interleaved", False)
    H, Hq, Hkv, ps = 320, 6, 2, 16
    rng = np.random.default_rng(777 + B + d)
    lens = rng.integers(0, 400, size=B).tolist()
    w = W.make_workload("prelude_var", 400 + B, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps,
                        num_pages=B * (400 // ps + 2) + 4, context_lens=lens, rope_base=10000.0,
                        inactive_rows=(1,))
    R = rotary_dim or d
    w.rope_cos, w.rope_sin = W.rope_table(w.max_position, R, w.rope_base)
    x = W.f32_to_bf16_bits(rng.integers(-2, 3, size=(B, H)).astype(np.float32))
    wq = W.f32_to_bf16_bits(rng.integers(-2, 3, size=((Hq + 2 * Hkv) * d, H)).astype(np.float32))
    qw = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(d)).astype(np.float32)) if norm else None
    kw_bits = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(d)).astype(np.float32)) if norm is True else None
    q0, k0, v0 = O.oracle_qkv_projection(x, wq, Hq, Hkv, d)
    q_ref, k_ref, v_ref = O.oracle_rope_kv_append_ex(q0, k0, v0, w.k_cache, w.v_cache, w.block_table,
                                                     w.context_lens, w.rope_cos, w.rope_sin, ps,
                                                     rotary_dim=rotary_dim or None, interleaved=interleaved,
                                                     q_norm_weight=qw, k_norm_weight=kw_bits, norm_eps=1e-6)
    st = runner.DecodeStep(w, num_splits=1)
    dev = lambda a: None if a is None else torch.from_numpy(a.view(np.int16)).cuda()
    st.q_rot.fill_(0x7FC0)
    ac.ac_qkv_rope_kv_append_ex(dev(x), dev(wq), H, st.q_rot, st.k_cache, st.v_cache, st.stride_page,
                                st.stride_token, st.stride_head, st.block_table, w.max_pages_per_seq,
                                st.context_lens, st.rope_cos, st.rope_sin, w.max_position, B, Hq, Hkv, d, ps,
                                w.num_pages, st.status_flag, rotary_dim=rotary_dim, interleaved=interleaved,
                                q_norm_weight=dev(qw), k_norm_weight=dev(kw_bits), norm_eps=1e-6)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    active = w.context_lens >= 0
    q_gpu = runner.bits_of(st.q_rot)
    assert np.array_equal(q_gpu[active], q_ref[active]), "q differs"
    assert (q_gpu[~active] == 0x7FC0).all()
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_ref), "K pool differs"
    assert np.array_equal(v_gpu, v_ref), "V pool differs"
    out_ref = O.oracle_paged_decode_attn(q_ref, k_ref, v_ref, w.block_table, w.context_lens, ps)
    st.attention()
    torch.cuda.synchronize()
    err = np.abs(st.out_f64() - out_ref)
    scale = max(1.0, float(np.abs(out_ref).max()))         # integer projections make outputs of size ~50
    assert err.max() <= 2e-2 * scale and err.mean() <= 2e-3 * scale


def test_qkv_prelude_variants_on_random_inputs():
    """N(0,1) inputs, Qwen3-like options (Q/K RMSNorm) on an 8-row batch of a 2048-hidden layer: the
    fp32 projection may be one bf16 step off now and then, and the norm spreads such a step over the
    head vector, so q and the appended k are held to the oracle within two bf16 steps of the pair's
    magnitude; v is not touched by the options."""
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    B, H, Hq, Hkv, d, ps = 8, 2048, 16, 4, 128, 16
    rng = np.random.default_rng(991)
    lens = rng.integers(0, 300, size=B).tolist()
    w = W.make_workload("prelude_var_n", 500, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps, num_pages=B * 21 + 4,
                        context_lens=lens, rope_base=1000000.0)
    x, wq = W.make_projection_inputs(501, B, H, Hq, Hkv, d)
    qw = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(d)).astype(np.float32))
    kw_bits = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(d)).astype(np.float32))
    q0, k0, v0 = O.oracle_qkv_projection(x, wq, Hq, Hkv, d)
    q_ref, k_ref, v_ref = O.oracle_rope_kv_append_ex(q0, k0, v0, w.k_cache, w.v_cache, w.block_table,
                                                     w.context_lens, w.rope_cos, w.rope_sin, ps,
                                                     q_norm_weight=qw, k_norm_weight=kw_bits, norm_eps=1e-6)
    st = runner.DecodeStep(w, num_splits=1)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda()
    ac.ac_qkv_rope_kv_append_ex(dev(x), dev(wq), H, st.q_rot, st.k_cache, st.v_cache, st.stride_page,
                                st.stride_token, st.stride_head, st.block_table, w.max_pages_per_seq,
                                st.context_lens, st.rope_cos, st.rope_sin, w.max_position, B, Hq, Hkv, d, ps,
                                w.num_pages, st.status_flag, q_norm_weight=dev(qw), k_norm_weight=dev(kw_bits),
                                norm_eps=1e-6)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    q_gpu = runner.bits_of(st.q_rot)
    k_gpu, v_gpu = st.cache_bits()
    target = np.zeros(k_ref.shape[:2], dtype=bool)
    for b in range(B):
        L = int(w.context_lens[b])
        target[w.block_table[b, L // ps], L % ps] = True

    def close(got_bits, ref_bits, what):
        got = W.bf16_bits_to_f32(got_bits).astype(np.float64)
        ref = W.bf16_bits_to_f32(ref_bits).astype(np.float64)
        mag = np.sqrt(ref[..., :d // 2] ** 2 + ref[..., d // 2:] ** 2)
        mag = np.concatenate([mag, mag], axis=-1)
        assert (np.abs(got - ref) <= 2.0 ** -5 * mag + 2.0 ** -7).all(), (what, float(np.abs(got - ref).max()))
        assert float(np.mean(got_bits == ref_bits)) >= 0.9, what

    close(q_gpu, q_ref, "q")
    close(k_gpu[target], k_ref[target], "k")
    assert np.array_equal(k_gpu[~target], w.k_cache[~target]) and np.array_equal(v_gpu[~target], w.v_cache[~target])
    _close_bf16(v_gpu[target], v_ref[target], "v")


@pytest.mark.parametrize("variant", [False, True])
@pytest.mark.parametrize("B", [6, 40])
def test_qkv_prelude_flags_rows_it_cannot_store(B, variant):
    """A row whose page id lies outside the pool, and one whose position lies outside the rope table: the
    projection launch sets both status bits, writes neither q nor the cache for them, and serves the
    other rows exactly -- plain and with the prelude variants, on the warp-MMA kernel (6 rows) and on
    the tcgen05 kernel (40 rows)."""
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    H, Hq, Hkv, d, ps = 256, 4, 2, 128, 16
    rng = np.random.default_rng(31 + B)
    lens = rng.integers(20, 300, size=B).tolist()
    w = W.make_workload("prelude_flags", 600 + B, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps,
                        num_pages=B * 21 + 4, context_lens=lens, rope_base=10000.0)
    x = W.f32_to_bf16_bits(rng.integers(-2, 3, size=(B, H)).astype(np.float32))
    wq = W.f32_to_bf16_bits(rng.integers(-2, 3, size=((Hq + 2 * Hkv) * d, H)).astype(np.float32))
    opts = dict(rotary_dim=64, interleaved=True) if variant else {}
    if variant:
        w.rope_cos, w.rope_sin = W.rope_table(w.max_position, 64, w.rope_base)
    q0, k0, v0 = O.oracle_qkv_projection(x, wq, Hq, Hkv, d)
    bad_page, bad_pos = 1, 3
    ok_rows = [b for b in range(B) if b not in (bad_page, bad_pos)]
    lens_ok = w.context_lens.copy()
    lens_ok[[bad_page, bad_pos]] = -1                      # the oracle skips the two rows
    q_ref, k_ref, v_ref = O.oracle_rope_kv_append_ex(q0, k0, v0, w.k_cache, w.v_cache, w.block_table, lens_ok,
                                                     w.rope_cos, w.rope_sin, ps, rotary_dim=opts.get("rotary_dim"),
                                                     interleaved=opts.get("interleaved", False))
    st = runner.DecodeStep(w, num_splits=1)
    bt = w.block_table.copy()
    bt[bad_page, lens[bad_page] // ps] = 1_000_000
    st.block_table.copy_(torch.from_numpy(bt))
    lens_dev = w.context_lens.copy()
    lens_dev[bad_pos] = w.max_position + 3
    st.context_lens.copy_(torch.from_numpy(lens_dev))
    st.q_rot.fill_(0x7FC0)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda()
    ac.ac_qkv_rope_kv_append_ex(dev(x), dev(wq), H, st.q_rot, st.k_cache, st.v_cache, st.stride_page,
                                st.stride_token, st.stride_head, st.block_table, w.max_pages_per_seq,
                                st.context_lens, st.rope_cos, st.rope_sin, w.max_position, B, Hq, Hkv, d, ps,
                                w.num_pages, st.status_flag, **opts)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 3
    q_gpu = runner.bits_of(st.q_rot)
    assert np.array_equal(q_gpu[ok_rows], q_ref[ok_rows])
    assert (q_gpu[bad_pos] == 0x7FC0).all()                # q of the row with the bad page id is still valid
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_ref) and np.array_equal(v_gpu, v_ref)


@pytest.mark.parametrize("B", [8, 100])
def test_qkv_prelude_bit_exact_when_the_projection_is_exact(B):
    """Small-integer x and W make every dot product an integer that fp32 and fp64 both hold exactly, so
    the projected bf16 features equal the oracle's and the rotation that follows can be held to the
    oracle bit for bit -- on the warp-MMA kernel (B = 8) and on the tcgen05 kernel (B = 100), whose
    epilogue rotates in fp32 and falls back to fp64 for the values it cannot prove (about one in a
    thousand of the 128 000 rotations here)."""
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    H, Hq, Hkv, d, ps = 256, 8, 2, 128, 16
    rng = np.random.default_rng(4242 + B)
    lens = rng.integers(0, 1500, size=B).tolist()
    w = W.make_workload("prelude_exact", 300 + B, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps,
                        num_pages=B * (1500 // ps + 2) + 4, context_lens=lens, rope_base=10000.0)
    x = W.f32_to_bf16_bits(rng.integers(-2, 3, size=(B, H)).astype(np.float32))
    wq = W.f32_to_bf16_bits(rng.integers(-2, 3, size=((Hq + 2 * Hkv) * d, H)).astype(np.float32))
    q_ref, k_ref, v_ref = O.oracle_qkv_rope_kv_append(x, wq, w.k_cache, w.v_cache, w.block_table,
                                                      w.context_lens, w.rope_cos, w.rope_sin, ps, Hq, Hkv, d)
    st = runner.DecodeStep(w, num_splits=1)
    ac.ac_qkv_rope_kv_append(torch.from_numpy(x.view(np.int16)).cuda(), torch.from_numpy(wq.view(np.int16)).cuda(),
                             H, st.q_rot, st.k_cache, st.v_cache, st.stride_page, st.stride_token,
                             st.stride_head, st.block_table, w.max_pages_per_seq, st.context_lens,
                             st.rope_cos, st.rope_sin, w.max_position, B, Hq, Hkv, d, ps, w.num_pages,
                             st.status_flag)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    assert np.array_equal(runner.bits_of(st.q_rot), q_ref)
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_ref)
    assert np.array_equal(v_gpu, v_ref)


@pytest.mark.parametrize("B,K,N", [(1, 256, 64), (5, 320, 96), (8, 1024, 512), (13, 512, 256), (31, 768, 128),
                                   (40, 256, 64), (4, 4096, 4096), (33, 128, 64), (100, 512, 192), (128, 1024, 256),
                                   (200, 320, 128), (40, 256, 96), (64, 4096, 4096), (16, 512, 128), (17, 320, 96),
                                   (96, 1024, 256)])
def test_oproj_residual_rmsnorm_matches_oracle(B, K, N):
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    rng = np.random.default_rng(B * 7 + K + N)
    a = W.f32_to_bf16_bits((rng.standard_normal((B, K)) * 0.3).astype(np.float32))
    wo = W.f32_to_bf16_bits((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    res = W.f32_to_bf16_bits(rng.standard_normal((B, N)).astype(np.float32))
    nw = W.f32_to_bf16_bits((1 + 0.1 * rng.standard_normal(N)).astype(np.float32))
    h_ref, normed_ref = O.oracle_oproj_residual_rmsnorm(a, wo, res, nw, 1e-5)
    dev = lambda x: torch.from_numpy(x.view(np.int16)).cuda()
    a_d, w_d, r_d, n_d = dev(a), dev(wo), dev(res), dev(nw)
    h_d = torch.full((B, N), 0x7FC0, dtype=torch.int16, device="cuda")
    y_d = torch.full((B, N), 0x7FC0, dtype=torch.int16, device="cuda")
    ac.ac_oproj_residual_rmsnorm(a_d, w_d, K, N, r_d, h_d, n_d, 1e-5, y_d, B)
    torch.cuda.synchronize()
    h = runner.bits_of(h_d)
    y = runner.bits_of(y_d)
    hf, hr = W.bf16_bits_to_f32(h).astype(np.float64), W.bf16_bits_to_f32(h_ref).astype(np.float64)
    assert np.isfinite(hf).all()
    # at most one bf16 step; where residual and projection cancel, the fp32 accumulation error of
    # the projection (relative to ITS magnitude, ~1) shows in the small sum
    assert (np.abs(hf - hr) <= 2.0 ** -7 * np.abs(hr) + 3e-5).all()
    assert np.mean(h == h_ref) >= 0.97
    # the norm is exact given the h the kernel produced
    assert np.array_equal(y, O.rms_norm_bf16(h, nw, 1e-5))
    # and close to the oracle's end-to-end result
    yf, yr = W.bf16_bits_to_f32(y).astype(np.float64), W.bf16_bits_to_f32(normed_ref).astype(np.float64)
    assert np.abs(yf - yr).max() <= 2.0 ** -6 * np.abs(yr).max()
    # in place on the residual stream
    ac.ac_oproj_residual_rmsnorm(a_d, w_d, K, N, r_d, r_d, n_d, 1e-5, y_d, B)
    torch.cuda.synchronize()
    assert np.array_equal(runner.bits_of(r_d), h)


def test_attention_block_chain_matches_oracle_chain():
    """Projection -> attention -> output projection, the three launches back to back on one stream,
    against the same chain in the oracle.  One-ulp differences of the bf16 projections propagate, so
    the end results are compared with a tolerance relative to their scale."""
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    B, H, Hq, Hkv, d, ps = 6, 1024, 8, 2, 128, 16
    rng = np.random.default_rng(77)
    lens = rng.integers(0, 900, size=B).tolist()
    w = W.make_workload("block", 78, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps, num_pages=B * 60 + 4,
                        context_lens=lens, rope_base=10000.0)
    hidden, wq = W.make_projection_inputs(79, B, H, Hq, Hkv, d)
    wo = W.f32_to_bf16_bits((rng.standard_normal((H, Hq * d)) / np.sqrt(Hq * d)).astype(np.float32))
    nw = W.f32_to_bf16_bits((1 + 0.1 * rng.standard_normal(H)).astype(np.float32))
    # oracle chain
    q_rot, k_after, v_after = O.oracle_qkv_rope_kv_append(hidden, wq, w.k_cache, w.v_cache, w.block_table,
                                                          w.context_lens, w.rope_cos, w.rope_sin, ps, Hq, Hkv, d)
    attn = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, ps)
    attn_bits = O.f64_to_bf16_rne(attn).reshape(B, Hq * d)
    h_ref, y_ref = O.oracle_oproj_residual_rmsnorm(attn_bits, wo, hidden, nw, 1e-5)
    blk = runner.AttentionBlockStep(w, hidden, wq, wo, nw, 1e-5, num_splits=2)
    blk.step()
    torch.cuda.synchronize()
    assert int(blk.step_.status_flag.item()) == 0
    for got_t, ref in ((blk.residual_out, h_ref), (blk.normed_out, y_ref)):
        got = W.bf16_bits_to_f32(runner.bits_of(got_t)).astype(np.float64)
        want = W.bf16_bits_to_f32(ref).astype(np.float64)
        rms = np.sqrt(np.mean(want ** 2))
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= 3e-2 * rms
        assert np.abs(got - want).mean() <= 2e-3 * rms
    # captured as one graph and replayed: same bits as the eager chain
    first = runner.bits_of(blk.normed_out).copy()
    blk2 = runner.AttentionBlockStep(w, hidden, wq, wo, nw, 1e-5, num_splits=2)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        blk2.step(side)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    fresh = runner.DecodeStep(w)
    blk2.step_.k_cache.copy_(fresh.k_cache); blk2.step_.v_cache.copy_(fresh.v_cache)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        blk2.step(side)
    blk2.step_.k_cache.copy_(fresh.k_cache); blk2.step_.v_cache.copy_(fresh.v_cache)
    blk2.normed_out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert np.array_equal(runner.bits_of(blk2.normed_out), first)
