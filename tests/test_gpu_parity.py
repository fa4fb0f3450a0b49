"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Cache writes and rotated q are compared bit for bit; attention outputs within the stated
tolerances (max abs <= 2e-2, mean abs <= 2e-3, plus a scale-aware bound)."""
import numpy as np
import pytest

from oracle import paged_decode_oracle as O
from paper_2606_07665_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS = 2e-2
MEAN_ABS = 2e-3
# Scale-aware bound per output element, from the kernel's arithmetic: the final rounding to bf16
# costs at most half a bf16 spacing, 2^-8 * |ref|; rounding the softmax weights to bf16 before the
# P.V product perturbs each weight by at most 2^-8 relative with random sign, which moves an output
# by a few times 2^-8/sqrt(3) * rms of its row in the worst element; fp32 accumulation is far below.
ROUND_REL = 2.0 ** -8
ROW_RMS_REL = 1e-2


@pytest.fixture(scope="module")
def rt():
    import torch
    from paper_2606_07665_b200 import binding, build, runner
    build.build()
    binding.ac_init(0)
    torch.cuda.set_device(0)
    return runner


def check_out(got, ref, what=""):
    """got, ref: [..., d]; rows are the last axis."""
    err = np.abs(got - ref)
    assert np.isfinite(got).all(), what
    assert err.max() <= MAX_ABS, (what, err.max())
    assert err.mean() <= MEAN_ABS, (what, err.mean())
    row_rms = np.sqrt(np.mean(ref ** 2, axis=-1, keepdims=True))
    bound = ROUND_REL * np.abs(ref) + ROW_RMS_REL * row_rms
    worst = float((err / np.maximum(bound, 1e-30)).max()) if err.size else 0.0
    assert (err <= bound).all(), (what, "worst err/bound", worst)
    return worst


def run_and_compare(rt, w, num_splits=None, layout="token_major", check_cache=True, fused=True,
                    window=0):
    """fused: False = three launches (RoPE+append, attention, merge); True = merge inside the
    attention kernel; "step" = the single-launch fused step."""
    import torch
    q_rot, k_after, v_after, out_ref = O.oracle_decode_step(w, window=window)
    st = rt.DecodeStep(w, num_splits=num_splits, layout=layout, fused_merge=bool(fused),
                       fused_step=(fused == "step"), window=window)
    st.step()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    if check_cache:
        assert np.array_equal(rt.bits_of(st.q_rot), q_rot), "rotated q differs"
        k_gpu, v_gpu = st.cache_bits()
        assert np.array_equal(k_gpu, k_after), "K pool differs"
        assert np.array_equal(v_gpu, v_after), "V pool differs"
    worst = check_out(st.out_f64(), out_ref, f"{w.name} S={st.num_splits} {layout} fused={fused}")
    print(f"[parity] {w.name} S={st.num_splits} {layout} fused={fused}: worst err/bound = {worst:.3f}")
    return st, out_ref


def small(seed, **kw):
    base = dict(B=3, Hq=8, Hkv=2, d=128, page_size=16, num_pages=96, context_lens=[200, 37, 333],
                rope_base=10000.0)
    base.update(kw)
    return W.make_workload("small", seed, **base)


# ---------------------------------------------------------------------------------------------
# RoPE + append: bit-exact
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kw", [
    dict(),
    dict(d=64, Hq=6, Hkv=3, context_lens=[15, 16, 17]),                     # around a page boundary
    dict(context_lens=[0, 1, 31], page_size=32, num_pages=16),
    dict(B=5, Hq=28, Hkv=4, page_size=32, num_pages=64, context_lens=[100, 64, 0, 255, 31], inactive_rows=(1, 3)),
    dict(B=2, Hq=32, Hkv=2, context_lens=[500, 77], rope_base=500000.0),
])
@pytest.mark.parametrize("fused", [True, "step"])
def test_rope_append_bit_exact(rt, kw, fused):
    run_and_compare(rt, small(31, **kw), fused=fused)


def test_rope_append_bit_exact_with_far_position_angles(rt):
    # Short contexts keep the pool small; table row p is replaced by the row of a far position
    # (100000..131071, base 500000: tiny sines, many near-cancellations).  Both sides read this table.
    rng = np.random.default_rng(7)
    w = W.make_workload("rope_far", 32, B=64, Hq=32, Hkv=8, d=128, page_size=16, num_pages=400,
                        context_lens=rng.integers(0, 60, size=64).tolist(), rope_base=500000.0)
    cos, sin = W.rope_table(131072, 128, 500000.0)
    far = rng.integers(100000, 131072, size=w.max_position)
    w.rope_cos = np.ascontiguousarray(cos[far])
    w.rope_sin = np.ascontiguousarray(sin[far])
    run_and_compare(rt, w)
    run_and_compare(rt, w, fused="step")


def test_rope_constructed_near_tie(rt):
    # x = (1 + 2^-7, 1), c = 1, s = -(2^-8)(1 + 2^-20): exact result just above a bf16 tie
    import torch
    w = small(33, B=1, Hq=2, Hkv=2, d=64, context_lens=[5], num_pages=8)
    w.q[:] = 0x3F80
    w.q[0, :, :32] = 0x3F81
    w.k_new[:] = w.q[0]
    w.rope_cos[:] = 1.0
    w.rope_sin[:] = np.float32(-(2.0 ** -8) * (1 + 2.0 ** -20))
    for fused in (True, "step"):
        st, _ = run_and_compare(rt, w, fused=fused)
        assert (rt.bits_of(st.q_rot)[0, :, :32] == 0x3F82).all()


@pytest.mark.parametrize("kw", [
    dict(rotary_dim=64),                                       # partial rotary, half-split
    dict(interleaved=True),
    dict(rotary_dim=32, interleaved=True),
    dict(norm=True),                                           # per-head Q/K RMSNorm, then full rotary
    dict(norm=True, rotary_dim=64, interleaved=True),
    dict(norm="q_only"),
    dict(),                                                    # options present but plain
])
@pytest.mark.parametrize("path", ["kernel", "step"])
@pytest.mark.parametrize("d", [128, 64])
def test_rope_prelude_variants_bit_exact_and_feed_attention(rt, kw, d, path):
    # path "kernel": the stand-alone variant kernel followed by attention; "step": the same variants
    # applied inside the single-launch step (ac_decode_step_fused_ex with rope options)
    import torch
    kw = dict(kw)
    norm = kw.pop("norm", False)
    rotary_dim = min(kw.get("rotary_dim", 0), d)
    interleaved = kw.get("interleaved", False)
    w = small(37, B=4, Hq=12, Hkv=3, d=d, context_lens=[200, 0, 37, 333], num_pages=64, inactive_rows=(2,))
    R = rotary_dim or d
    w.rope_cos, w.rope_sin = W.rope_table(w.max_position, R, w.rope_base)      # [max_position, R/2]
    rng = np.random.default_rng(3)
    qw = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(d)).astype(np.float32)) if norm else None
    kw_bits = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(d)).astype(np.float32)) if norm is True else None
    q_rot, k_after, v_after = O.oracle_rope_kv_append_ex(
        w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.rope_cos, w.rope_sin,
        w.page_size, rotary_dim=rotary_dim or None, interleaved=interleaved, q_norm_weight=qw,
        k_norm_weight=kw_bits, norm_eps=1e-6)
    out_ref = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, w.page_size)
    st = rt.DecodeStep(w, num_splits=2, fused_step=(path == "step"))
    dev = lambda a: None if a is None else torch.from_numpy(a.view(np.int16)).cuda()
    if path == "step":
        st.q_rot.fill_(0x7FC0)
        st.decode_step_fused(rotary_dim=rotary_dim, interleaved=interleaved, q_norm_weight=dev(qw),
                             k_norm_weight=dev(kw_bits), norm_eps=1e-6)
        torch.cuda.synchronize()
        st.q_rot[2] = st.q_in[2]                      # the inactive row's q is not written by the step
    else:
        st.rope_kv_append_ex(rotary_dim=rotary_dim, interleaved=interleaved, q_norm_weight=dev(qw),
                             k_norm_weight=dev(kw_bits), norm_eps=1e-6)
        st.attention()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    assert np.array_equal(rt.bits_of(st.q_rot), q_rot), "q after norm/rotation differs"
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_after) and np.array_equal(v_gpu, v_after)
    check_out(st.out_f64(), out_ref, f"prelude variant {kw} norm={norm} d={d}")


@pytest.mark.parametrize("window,splits", [(100, 1), (333, 3)])
def test_fused_step_variants_with_a_sliding_window(rt, window, splits):
    # the prelude variants and the sliding window together in the single-launch step
    import torch
    w = small(58, B=3, Hq=12, Hkv=3, d=128, context_lens=[700, 45, 333], num_pages=96)
    w.rope_cos, w.rope_sin = W.rope_table(w.max_position, 64, w.rope_base)
    rng = np.random.default_rng(4)
    qw = W.f32_to_bf16_bits((1 + 0.2 * rng.standard_normal(w.d)).astype(np.float32))
    q_rot, k_after, v_after = O.oracle_rope_kv_append_ex(
        w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.rope_cos, w.rope_sin,
        w.page_size, rotary_dim=64, interleaved=True, q_norm_weight=qw, k_norm_weight=qw, norm_eps=1e-6)
    out_ref = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, w.page_size,
                                         window=window)
    st = rt.DecodeStep(w, num_splits=splits, fused_step=True, window=window)
    nw = torch.from_numpy(qw.view(np.int16)).cuda()
    st.decode_step_fused(rotary_dim=64, interleaved=True, q_norm_weight=nw, k_norm_weight=nw, norm_eps=1e-6)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    assert np.array_equal(rt.bits_of(st.q_rot), q_rot)
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_after) and np.array_equal(v_gpu, v_after)
    check_out(st.out_f64(), out_ref, f"variants + window {window}")


def test_append_flags_out_of_range_and_writes_nothing(rt):
    import torch
    w = small(34, B=2, context_lens=[40, 50], num_pages=32)
    st = rt.DecodeStep(w)
    bt = w.block_table.copy()
    bt[0, 40 // 16] = 10_000                  # page id outside the pool
    st.block_table.copy_(torch.from_numpy(bt))
    lens = w.context_lens.copy()
    lens[1] = w.max_position + 5               # position outside the rope table
    st.context_lens.copy_(torch.from_numpy(lens))
    before_k, before_v = st.cache_bits()
    st.rope_kv_append()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 3
    after_k, after_v = st.cache_bits()
    assert np.array_equal(before_k, after_k) and np.array_equal(before_v, after_v)


# ---------------------------------------------------------------------------------------------
# attention: small shapes spanning several tiles, ragged tails, every group size and layout
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kw", [
    dict(),
    dict(Hq=4, Hkv=4),                                                       # G = 1
    dict(Hq=28, Hkv=4, page_size=32, num_pages=48),                          # G = 7
    dict(Hq=16, Hkv=2),                                                      # G = 8
    dict(Hq=32, Hkv=2),                                                      # G = 16 (two row blocks)
    dict(Hq=24, Hkv=2, d=64),                                                # G = 12, d = 64
    dict(d=64, Hq=8, Hkv=2, page_size=64, num_pages=24),
    dict(context_lens=[0, 15, 16], num_pages=16),                            # one token; tile edges
    dict(context_lens=[63, 64, 65]),
    dict(B=4, context_lens=[1000, 3, 511, 700], num_pages=200, inactive_rows=(2,)),
])
@pytest.mark.parametrize("splits,fused", [(1, True), (3, True), (3, False), (1, "step"), (3, "step")])
def test_attention_small(rt, kw, splits, fused):
    run_and_compare(rt, small(41, **kw), num_splits=splits, fused=fused)


@pytest.mark.parametrize("splits", [1, 2, 5, 16])
def test_attention_split_sweep_and_partials(rt, splits):
    import torch
    w = small(42, B=2, context_lens=[900, 257], num_pages=128)
    run_and_compare(rt, w, num_splits=splits, fused=True)
    st, out_ref = run_and_compare(rt, w, num_splits=splits, fused=False)
    if splits > 1:
        # the workspace format is part of the ABI: compare each split's partial with the oracle's
        q_rot, k_after, v_after, _ = O.oracle_decode_step(w)
        starts = [[s * st.split_tokens for s in range(splits + 1)]] * w.B
        po_ref, pl_ref = O.oracle_split_partials(q_rot, k_after, v_after, w.block_table, w.context_lens,
                                                 w.page_size, starts)
        po, pl = st.partials()
        empty = ~np.isfinite(pl_ref)
        assert np.array_equal(np.isneginf(pl), empty)
        assert np.abs(pl[~empty] - pl_ref[~empty]).max() < 2e-2
        assert np.abs(po[~empty] - po_ref[~empty]).max() < 2e-2


def test_merge_kernel_alone_against_oracle(rt):
    import torch
    from paper_2606_07665_b200 import binding as ac
    rng = np.random.default_rng(5)
    B, Hq, S, d = 3, 5, 7, 128
    po = rng.standard_normal((B, Hq, S, d)).astype(np.float32)
    pl = (rng.standard_normal((B, Hq, S)) * 5).astype(np.float32)
    pl[0, 0, :] = -np.inf                          # a row with nothing to merge
    pl[1, 2, 3] = -np.inf
    po[1, 2, 3] = np.nan                           # partial of an empty split must not be read
    pl[2, 1, :] = [-np.inf] * 6 + [1.5]
    ws = torch.from_numpy(np.concatenate([po.ravel(), pl.ravel()])).cuda()
    lens = torch.tensor([5, 5, 5], dtype=torch.int32).cuda()
    out = torch.full((B, Hq, d), 0x7FC0, dtype=torch.int16).cuda()
    ac.ac_splitkv_merge(ws, S, lens, out, B, Hq, d)
    torch.cuda.synchronize()
    ref, _ = O.oracle_splitkv_merge(np.where(np.isnan(po), 0.0, po), pl)
    got = W.bf16_bits_to_f32(rt.bits_of(out)).astype(np.float64)
    assert np.abs(got - ref).max() <= 2.0 ** -8 * max(1.0, np.abs(ref).max())
    assert (rt.bits_of(out)[0, 0] == 0).all()
    lens[1] = -1
    ac.ac_splitkv_merge(ws, S, lens, out, B, Hq, d)
    torch.cuda.synchronize()
    assert (rt.bits_of(out)[1] == 0).all()


@pytest.mark.parametrize("splits,fused", [(1, True), (4, True), (4, False), (1, "step"), (4, "step")])
def test_attention_head_major_layout(rt, splits, fused):
    run_and_compare(rt, small(43, Hq=16, Hkv=4, context_lens=[300, 45, 129]), num_splits=splits,
                    layout="head_major", fused=fused)


def test_single_token_context_returns_v_bits(rt):
    import torch
    w = small(44, context_lens=[0, 0, 0], num_pages=8)
    st, _ = run_and_compare(rt, w, num_splits=1)
    G = w.Hq // w.Hkv
    got = rt.bits_of(st.out)
    for hq in range(w.Hq):
        assert np.array_equal(got[:, hq], w.v_new[:, hq // G])


def test_page_permutation_gives_bit_identical_output(rt):
    import torch
    w = small(45, context_lens=[700, 123, 64], num_pages=128)
    st1, _ = run_and_compare(rt, w, num_splits=3)
    out1 = rt.bits_of(st1.out).copy()
    perm = np.random.default_rng(9).permutation(w.num_pages)
    w2 = W.make_workload("small", 45, B=3, Hq=8, Hkv=2, d=128, page_size=16, num_pages=128,
                         context_lens=[700, 123, 64], rope_base=10000.0)
    k2 = np.empty_like(w2.k_cache); v2 = np.empty_like(w2.v_cache)
    k2[perm] = w2.k_cache; v2[perm] = w2.v_cache
    w2.k_cache, w2.v_cache = k2, v2
    w2.block_table = perm[w2.block_table].astype(np.int32)
    st2 = rt.DecodeStep(w2, num_splits=3)
    st2.step()
    torch.cuda.synchronize()
    assert np.array_equal(out1, rt.bits_of(st2.out))


def test_attention_without_new_token_and_deterministic(rt):
    import torch
    w = small(46, context_lens=[310, 48, 129], num_pages=64)
    q_rot, k_after, v_after, _ = O.oracle_decode_step(w)
    ref = O.oracle_paged_decode_attn(q_rot, w.k_cache, w.v_cache, w.block_table, w.context_lens,
                                     w.page_size, new_tokens=0)
    st = rt.DecodeStep(w, num_splits=2)
    q_dev = torch.from_numpy(q_rot.view(np.int16)).cuda()
    st.attention(new_tokens=0, q=q_dev)
    st.merge()
    torch.cuda.synchronize()
    check_out(st.out_f64(), ref, "new_tokens=0")
    first = rt.bits_of(st.out).copy()
    for _ in range(3):
        st.attention(new_tokens=0, q=q_dev)
        st.merge()
    torch.cuda.synchronize()
    assert np.array_equal(first, rt.bits_of(st.out))


def test_graph_replay_equals_eager_and_tracks_updated_lengths(rt):
    import torch

    def make():
        w = small(47, B=4, Hq=28, Hkv=4, page_size=32, num_pages=96, context_lens=[600, 31, 32, 257],
                  inactive_rows=(1,))
        w.rope_cos, w.rope_sin = W.rope_table(w.max_position + 4, w.d, w.rope_base)   # room to advance
        return w

    w = make()
    st, out_ref = run_and_compare(rt, w, num_splits=2)
    eager = rt.bits_of(st.out).copy()
    k_eager, v_eager = st.cache_bits()
    st2 = rt.DecodeStep(w, num_splits=2, max_context_len=w.max_context_len + 4)
    graph = st2.capture()
    # capture ran one eager warm-up step on the same buffers; restore the caches and replay
    fresh = rt.DecodeStep(w, num_splits=2)
    st2.k_cache.copy_(fresh.k_cache); st2.v_cache.copy_(fresh.v_cache); st2.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    check_out(st2.out_f64(), out_ref, "graph replay")
    k2, v2 = st2.cache_bits()
    assert np.array_equal(k2, k_eager) and np.array_equal(v2, v_eager)
    # identical launch configuration replayed eagerly gives identical bits
    st2.k_cache.copy_(fresh.k_cache); st2.v_cache.copy_(fresh.v_cache)
    st2.step()
    torch.cuda.synchronize()
    eager2 = rt.bits_of(st2.out).copy()
    st2.k_cache.copy_(fresh.k_cache); st2.v_cache.copy_(fresh.v_cache); st2.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert np.array_equal(rt.bits_of(st2.out), eager2)
    # same graph, device-side lengths advanced by one token per active row: still matches the oracle
    w_next = make()
    _, k_after, v_after, _ = O.oracle_decode_step(w_next)
    w_next.k_cache, w_next.v_cache = k_after, v_after
    w_next.context_lens = np.where(w_next.context_lens >= 0, w_next.context_lens + 1, -1).astype(np.int32)
    _, _, _, out_next = O.oracle_decode_step(w_next)
    st2.context_lens.copy_(torch.from_numpy(w_next.context_lens))
    graph.replay()
    torch.cuda.synchronize()
    assert int(st2.status_flag.item()) == 0
    check_out(st2.out_f64(), out_next, "replay with advanced lengths")


def test_fused_step_flags_out_of_range_and_writes_nothing(rt):
    import torch
    w = small(35, B=3, context_lens=[40, 50, 60], num_pages=32)
    st = rt.DecodeStep(w, num_splits=2, fused_step=True)
    bt = w.block_table.copy()
    bt[0, 40 // 16] = 10_000                  # page id outside the pool
    st.block_table.copy_(torch.from_numpy(bt))
    lens = w.context_lens.copy()
    lens[1] = w.max_position + 5               # position outside the rope table (and the block table)
    st.context_lens.copy_(torch.from_numpy(lens))
    before_k, before_v = st.cache_bits()
    st.step()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) & 3 == 3
    after_k, after_v = st.cache_bits()
    # only row 2 appended
    changed = np.unique(np.nonzero(after_k != before_k)[0]).tolist()
    assert changed == [int(w.block_table[2, 60 // 16])]
    q_rot, k_ref, v_ref, out_ref = O.oracle_decode_step(w)
    check_out(st.out_f64()[2], out_ref[2], "row untouched by the bad rows")


def test_fused_step_graph_replay_advances(rt):
    import torch
    w = small(36, B=3, Hq=28, Hkv=4, page_size=32, num_pages=96, context_lens=[600, 31, 257])
    w.rope_cos, w.rope_sin = W.rope_table(w.max_position + 4, w.d, w.rope_base)
    _, k1, v1, out1 = O.oracle_decode_step(w)
    st = rt.DecodeStep(w, num_splits=2, fused_step=True, max_context_len=w.max_context_len + 4)
    graph = st.capture()
    fresh = rt.DecodeStep(w, num_splits=2)
    st.k_cache.copy_(fresh.k_cache); st.v_cache.copy_(fresh.v_cache); st.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    check_out(st.out_f64(), out1, "fused step replay")
    kg, vg = st.cache_bits()
    assert np.array_equal(kg, k1) and np.array_equal(vg, v1)
    w2 = small(36, B=3, Hq=28, Hkv=4, page_size=32, num_pages=96, context_lens=[600, 31, 257])
    w2.rope_cos, w2.rope_sin = w.rope_cos, w.rope_sin
    w2.k_cache, w2.v_cache = k1, v1
    w2.context_lens = (w2.context_lens + 1).astype(np.int32)
    _, k2, v2, out2 = O.oracle_decode_step(w2)
    st.context_lens.copy_(torch.from_numpy(w2.context_lens))
    graph.replay()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    check_out(st.out_f64(), out2, "fused step replay, advanced lengths")
    kg, vg = st.cache_bits()
    assert np.array_equal(kg, k2) and np.array_equal(vg, v2)


def test_fused_step_flags_a_row_it_cannot_append(rt):
    # Two ways the single-launch step can find no tile for the new token's slot: the block-table row
    # is full (position / page_size == max_pages_per_seq), or max_context_len is too small for the
    # row (its slot lies beyond the last split).  Both must set the position bit, leave both pools and
    # q_rot_out untouched, and keep the fused merge's counters consistent for the next launch.
    import torch
    w = small(38, B=3, context_lens=[47, 50, 60], num_pages=32)            # 47 + 1 tokens fill 3 pages
    w.rope_cos, w.rope_sin = W.rope_table(128, w.d, w.rope_base)
    for case in ("full_row", "short_bucket"):
        if case == "full_row":
            st = rt.DecodeStep(w, num_splits=2, fused_step=True)
            lens = w.context_lens.copy()
            lens[1] = w.max_pages_per_seq * w.page_size                      # first slot past the row
            bad_row = 1
        else:
            st = rt.DecodeStep(w, num_splits=1, fused_step=True, max_context_len=64)
            assert st.split_tokens == 64
            lens = w.context_lens.copy()
            lens[0] = 64                                                     # 65 tokens, 64 covered
            bad_row = 0
        st.context_lens.copy_(torch.from_numpy(lens))
        st.q_rot.fill_(0x7FC0)
        before_k, before_v = st.cache_bits()
        st.step()
        torch.cuda.synchronize()
        assert int(st.status_flag.item()) == 2, case
        after_k, after_v = st.cache_bits()
        good = [b for b in range(w.B) if b != bad_row]
        changed = sorted(set(np.nonzero(after_k != before_k)[0].tolist()))
        assert changed == sorted(int(w.block_table[b, lens[b] // 16]) for b in good), case
        assert (rt.bits_of(st.q_rot)[bad_row] == 0x7FC0).all(), case
        # the three-call path flags the full row the same way
        if case == "full_row":
            st3 = rt.DecodeStep(w, num_splits=2, fused_merge=False)
            st3.context_lens.copy_(torch.from_numpy(lens))
            st3.rope_kv_append()
            torch.cuda.synchronize()
            assert int(st3.status_flag.item()) == 2
        # the other rows are served, and the workspace is fit for another launch
        w_ok = small(38, B=3, context_lens=[47, 50, 60], num_pages=32)
        w_ok.rope_cos, w_ok.rope_sin = w.rope_cos, w.rope_sin
        _, _, _, out_ref = O.oracle_decode_step(w_ok)
        for b in good:
            check_out(st.out_f64()[b], out_ref[b], f"{case}: row {b}")
        if st.num_splits > 1:
            n = st.B * st.Hq * st.num_splits * (st.d + 1)
            counters = st.workspace.view(torch.int32)[n:n + st.B * st.Hkv]
            assert int(counters.abs().sum().item()) == 0, case


def _chained_steps_case(n_steps, seed):
    """A small batch with room in its block table and rope table for n_steps more tokens, per-step
    q/k_new/v_new, and the oracle stepped through the same sequence."""
    rng = np.random.default_rng(seed)
    lens0 = np.array([200, 37, 333], dtype=np.int32)
    B, Hq, Hkv, d, ps = 3, 8, 2, 128, 16
    pages_needed = [(int(n) + n_steps + ps) // ps for n in lens0]
    w = W.make_workload("chain", seed, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps, num_pages=160,
                        context_lens=lens0.tolist(), rope_base=10000.0, max_pages_per_seq=max(pages_needed))
    # pages for the tokens to come: unused pages of the pool (they hold NaN until written)
    taken = set(int(x) for x in w.block_table.ravel())
    spare = [pg for pg in range(w.num_pages) if pg not in taken]
    for b in range(B):
        have = (int(lens0[b]) + ps) // ps
        for j in range(have, pages_needed[b]):
            w.block_table[b, j] = spare.pop()
    w.rope_cos, w.rope_sin = W.rope_table(int(lens0.max()) + n_steps + 1, d, w.rope_base)
    qs = W.f32_to_bf16_bits(rng.standard_normal((n_steps, B, Hq, d), dtype=np.float32))
    ks = W.f32_to_bf16_bits(rng.standard_normal((n_steps, B, Hkv, d), dtype=np.float32))
    vs = W.f32_to_bf16_bits(rng.standard_normal((n_steps, B, Hkv, d), dtype=np.float32))
    k_cache, v_cache = w.k_cache, w.v_cache
    out_ref = None
    for i in range(n_steps):
        lens = (lens0 + i).astype(np.int32)
        q_rot, k_cache, v_cache = O.oracle_rope_kv_append(qs[i], ks[i], vs[i], k_cache, v_cache,
                                                          w.block_table, lens, w.rope_cos, w.rope_sin, ps)
        if i == n_steps - 1:
            out_ref = O.oracle_paged_decode_attn(q_rot, k_cache, v_cache, w.block_table, lens, ps)
    return w, lens0, qs, ks, vs, k_cache, v_cache, out_ref


@pytest.mark.parametrize("mode", ["per_step_length_buffers", "lengths_advanced_by_a_kernel"])
def test_chained_fused_steps_in_one_graph(rt, mode):
    # 120 single-launch steps of the same requests inside ONE captured graph.  Every kernel of the
    # chain may start under the tail of the one before it and reads context_lens, the block table and
    # the older cache tiles before it synchronises, so a step must never see a slot that the step two
    # back has not finished writing.  per_step_length_buffers: nothing at all between the launches
    # (step i reads its own context_lens buffer).  lengths_advanced_by_a_kernel: an ordinary kernel
    # between the launches advances the one context_lens buffer and another rewrites the block table
    # (unused entries hold different garbage at every step).  The final pools must equal the oracle's
    # bit for bit and the last step's output must match it.
    import torch
    from paper_2606_07665_b200 import binding as ac
    n_steps = 120
    w, lens0, qs, ks, vs, k_ref, v_ref, out_ref = _chained_steps_case(n_steps, 91)
    st = rt.DecodeStep(w, num_splits=2, fused_step=True, max_context_len=int(lens0.max()) + n_steps + 1)
    dev = st.device
    q_d = torch.from_numpy(qs.view(np.int16)).to(dev)
    k_d = torch.from_numpy(ks.view(np.int16)).to(dev)
    v_d = torch.from_numpy(vs.view(np.int16)).to(dev)
    lens_steps = torch.from_numpy(np.stack([lens0 + i for i in range(n_steps)]).astype(np.int32)).to(dev)
    ps = w.page_size
    tables = np.repeat(w.block_table[None], n_steps, axis=0).copy()
    for i in range(n_steps):
        for b in range(w.B):
            used = (int(lens0[b]) + i) // ps + 1
            tables[i, b, used:] = 1_000_000 + i              # never read: outside the pool on purpose
    tables_d = torch.from_numpy(tables).to(dev)
    one = torch.ones(1, dtype=torch.int32, device=dev)

    def enqueue(stream):
        if mode == "lengths_advanced_by_a_kernel":
            st.context_lens.copy_(lens_steps[0])
        for i in range(n_steps):
            if mode == "lengths_advanced_by_a_kernel":
                st.block_table.copy_(tables_d[i])
                lens_buf, table = st.context_lens, st.block_table
            else:
                lens_buf, table = lens_steps[i], tables_d[i]
            ac.ac_decode_step_fused_ex(q_d[i], st.q_rot, k_d[i], v_d[i], st.k_cache, st.v_cache,
                                       st.stride_page, st.stride_token, st.stride_head, table,
                                       w.max_pages_per_seq, lens_buf, st.rope_cos, st.rope_sin,
                                       w.max_position, 0.0, st.num_splits, st.workspace, st.workspace_bytes,
                                       st.out, st.B, st.Hq, st.Hkv, st.d, st.ps, st.num_pages,
                                       st.max_context_len, st.status_flag, stream)
            if mode == "lengths_advanced_by_a_kernel":
                st.context_lens.add_(one)

    fresh_k, fresh_v = st.k_cache.clone(), st.v_cache.clone()
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        enqueue(side)                                        # warm-up outside capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue(side)
    for rep in range(3):
        st.k_cache.copy_(fresh_k)
        st.v_cache.copy_(fresh_v)
        st.out.fill_(0x7FC0)
        graph.replay()
        torch.cuda.synchronize()
        assert int(st.status_flag.item()) == 0
        k_gpu, v_gpu = st.cache_bits()
        assert np.array_equal(k_gpu, k_ref), f"K pool differs after the chain ({mode}, replay {rep})"
        assert np.array_equal(v_gpu, v_ref), f"V pool differs after the chain ({mode}, replay {rep})"
        check_out(st.out_f64(), out_ref, f"last step of the chain ({mode}, replay {rep})")


@pytest.mark.parametrize("fused", [False, True, "step"])
@pytest.mark.parametrize("window,splits", [(1, 1), (7, 1), (16, 2), (100, 1), (100, 3), (333, 2), (5000, 2)])
def test_sliding_window(rt, window, splits, fused):
    # windows that start inside a tile, on a tile edge, before the first token, and rows shorter than
    # the window; everything before the window is poisoned to prove it is neither read nor weighted
    w = small(51, B=4, Hq=16, Hkv=2, context_lens=[900, 5, 333, 99], num_pages=160, inactive_rows=(1,))
    for b in range(w.B):
        n = int(w.context_lens[b]) + 1
        if n <= 0:
            continue
        for t in range(0, max(0, n - window)):
            pg, sl = w.block_table[b, t // w.page_size], t % w.page_size
            w.k_cache[pg, sl] = 0x7FC0
            w.v_cache[pg, sl] = 0x7FC0
    run_and_compare(rt, w, num_splits=splits, fused=fused, window=window)


@pytest.mark.parametrize("fused", [False, True, "step"])
@pytest.mark.parametrize("kw,splits,window", [
    # Grids of at most one CTA per SM (148 on the target) whose splits are longer than 192 tokens run
    # twelve-warp CTAs: without a merge, with the merge inside a cluster (2 .. 16 splits), with a window,
    # with 16 query heads per KV head, head_dim 64, a ragged batch with an inactive row
    (dict(B=2, Hq=32, Hkv=8, context_lens=[3000, 1500], num_pages=300), 1, 0),
    (dict(B=2, Hq=32, Hkv=8, context_lens=[3000, 1500], num_pages=300), 4, 0),
    (dict(B=2, Hq=32, Hkv=8, context_lens=[3000, 1500], num_pages=300), 9, 0),
    (dict(B=3, Hq=32, Hkv=2, d=64, context_lens=[2500, 700, 1300], num_pages=300), 5, 0),
    (dict(B=4, Hq=28, Hkv=4, page_size=32, context_lens=[2047, 0, 900, 411], num_pages=120, inactive_rows=(1,)), 3, 0),
    (dict(B=2, Hq=14, Hkv=2, context_lens=[2600, 1000], num_pages=240), 2, 1000),
    (dict(B=1, Hq=8, Hkv=8, context_lens=[4095], num_pages=260), 13, 0),
])
def test_grids_of_one_cta_per_sm(rt, kw, splits, window, fused):
    w = small(61, **kw)
    assert w.B * w.Hkv * splits <= 148
    st, _ = run_and_compare(rt, w, num_splits=splits, fused=fused, window=window)
    assert st.split_tokens > 192


@pytest.mark.parametrize("fused", [True, "step"])
@pytest.mark.parametrize("kw", [
    dict(B=2, Hq=16, Hkv=1, d=128, page_size=16, context_lens=[700, 33], num_pages=64),            # multi-query
    dict(B=2, Hq=4, Hkv=4, d=64, page_size=256, context_lens=[1000, 255], num_pages=8),            # largest page
    dict(B=3, Hq=8, Hkv=2, d=128, page_size=64, context_lens=[63, 64, 4000], num_pages=72),
    dict(B=1, Hq=64, Hkv=4, d=64, page_size=16, context_lens=[129], num_pages=12),                 # group of 16, d = 64
])
def test_extreme_shapes(rt, kw, fused):
    run_and_compare(rt, small(52, **kw), fused=fused)
    run_and_compare(rt, small(52, **kw), fused=fused, num_splits=1, check_cache=False)


@pytest.mark.parametrize("fused", [True, "step"])
def test_many_short_requests(rt, fused):
    # 1500 rows of 0..40 tokens: grid rows far beyond one wave, most tiles ragged, some rows inactive
    rng = np.random.default_rng(12)
    lens = rng.integers(0, 41, size=1500).tolist()
    w = W.make_workload("many", 53, B=1500, Hq=8, Hkv=2, d=64, page_size=16, num_pages=4700,
                        context_lens=lens, rope_base=10000.0, inactive_rows=(3, 700, 1499))
    run_and_compare(rt, w, fused=fused)


@pytest.mark.parametrize("fused", [True, "step"])
def test_one_very_long_request(rt, fused):
    # 400k tokens for one KV head: many splits, positions far into the rope table, > 2^24 cache elements
    import torch
    w = W.make_workload("verylong", 54, B=1, Hq=4, Hkv=1, d=128, page_size=32, num_pages=12600,
                        context_lens=[400_000], rope_base=1000000.0)
    st = rt.DecodeStep(w, fused_merge=True, fused_step=(fused == "step"))
    st.step()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0 and st.num_splits > 8
    q_rot, k_after, v_after, out_ref = O.oracle_decode_step(w)
    assert np.array_equal(rt.bits_of(st.q_rot), q_rot)
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_after) and np.array_equal(v_gpu, v_after)
    check_out(st.out_f64(), out_ref, "400k-token request")


@pytest.mark.parametrize("fused", [False, True, "step"])
def test_batch_of_only_inactive_rows(rt, fused):
    # a bucket that is all padding: nothing is written to the cache, every output row is +0
    import torch
    w = small(56, B=3, context_lens=[40, 50, 60], num_pages=32, inactive_rows=(0, 1, 2))
    st = rt.DecodeStep(w, num_splits=2, fused_merge=bool(fused), fused_step=(fused == "step"))
    before_k, before_v = st.cache_bits()
    st.out.fill_(0x7FC0)
    st.step()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    after_k, after_v = st.cache_bits()
    assert np.array_equal(before_k, after_k) and np.array_equal(before_v, after_v)
    assert (rt.bits_of(st.out) == 0).all()


@pytest.mark.parametrize("kw,splits", [
    (dict(B=4, Hq=8, Hkv=2, context_lens=[200, 37, 333, 0], num_pages=96), 3),     # gathered by one kernel
    (dict(B=4, Hq=8, Hkv=2, context_lens=[200, 37, 333, 0], num_pages=96), 1),
    (dict(B=3, Hq=8, Hkv=2, context_lens=[200, 37, 333], num_pages=96), 2),        # sizes not 16-byte multiples
    (dict(B=1, Hq=8, Hkv=2, context_lens=[77], num_pages=16), 2),
])
@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_from_host_buffers(rt, kw, splits, pinned):
    # pinned: inputs gathered by one kernel, result stored straight into the host buffer by the
    # attention kernel; pageable: one copy per buffer in, one copy out.  Same results either way.
    import torch
    from paper_2606_07665_b200 import binding as ac
    w = small(57, **kw)
    q_rot, k_after, v_after, out_ref = O.oracle_decode_step(w)
    st = rt.DecodeStep(w, num_splits=splits)

    def pin(a):
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
        return t.pin_memory() if pinned else t.clone()

    h_q, h_k, h_v, h_bt, h_len = pin(w.q), pin(w.k_new), pin(w.v_new), pin(w.block_table), pin(w.context_lens)
    h_out = torch.full((w.B, w.Hq, w.d), 0x7FC0, dtype=torch.int16)
    h_out = h_out.pin_memory() if pinned else h_out
    # device staging buffers start with garbage: everything must come from the host buffers
    for t in (st.q_in, st.k_new, st.v_new):
        t.fill_(0x7FC0)
    st.block_table.fill_(-7)
    st.context_lens.fill_(-1)
    st.workspace.view(torch.int32).fill_(123456)              # the call clears its own counters
    for rep in range(2):
        ac.ac_decode_step_host(h_q, h_k, h_v, h_bt, h_len, h_out, st.q_in, st.k_new, st.v_new, st.block_table,
                               st.context_lens, st.out, st.k_cache, st.v_cache, st.stride_page, st.stride_token,
                               st.stride_head, w.max_pages_per_seq, st.rope_cos, st.rope_sin, w.max_position,
                               0.0, st.num_splits, st.workspace if st.num_splits > 1 else None,
                               st.workspace_bytes, st.B, st.Hq, st.Hkv, st.d, st.ps, st.num_pages,
                               st.max_context_len, st.status_flag)
        torch.cuda.synchronize()
        assert int(st.status_flag.item()) == 0
        got = W.bf16_bits_to_f32(h_out.numpy().view(np.uint16)).astype(np.float64)
        check_out(got, out_ref, f"host step rep {rep}")
        assert np.array_equal(rt.bits_of(st.out), h_out.numpy().view(np.uint16))    # device copy holds the same bits
        k_gpu, v_gpu = st.cache_bits()
        assert np.array_equal(k_gpu, k_after) and np.array_equal(v_gpu, v_after)


def test_peaked_scores(rt):
    w = W.make_workload("peaked", 48, B=2, Hq=16, Hkv=2, d=128, page_size=16, num_pages=300,
                        context_lens=[2000, 1500], rope_base=500000.0, peak_fraction=0.01)
    run_and_compare(rt, w, num_splits=4)
    run_and_compare(rt, w, num_splits=1, check_cache=False)


# ---------------------------------------------------------------------------------------------
# the five benchmark workloads, in the launch configuration the benchmark uses (planned splits)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("fused", [True, "step"])
def test_workload_tiny(rt, fused):
    run_and_compare(rt, W.tiny(), fused=fused)


@pytest.mark.parametrize("fused", [True, "step"])
def test_workload_single_request(rt, fused):
    run_and_compare(rt, W.single_request(), fused=fused)


@pytest.mark.parametrize("fused", [True, "step"])
@pytest.mark.parametrize("batch", W.GRAPH_SWEEP_BATCHES)
def test_workload_graph_sweep(rt, batch, fused):
    import torch
    w = W.graph_sweep(batch)
    st, out_ref = run_and_compare(rt, w, fused=fused)
    graph = st.capture()
    graph.replay()
    torch.cuda.synchronize()
    check_out(st.out_f64(), out_ref, "graph replay")


@pytest.mark.parametrize("fused", [True, False, "step"])
def test_workload_continuous_batching(rt, fused):
    run_and_compare(rt, W.continuous_batching(), fused=fused)


@pytest.mark.parametrize("splits", [1, 2])
def test_longest_first_row_order_with_ties_and_inactive_rows(rt, splits):
    # 100 requests x 4 KV heads = 400+ CTAs: more than fit on the GPU at once, so the kernel serves
    # requests in order of decreasing length.  Many equal lengths and some inactive rows: every row
    # must still be served exactly once.
    rng = np.random.default_rng(11)
    lens = rng.choice([0, 15, 16, 100, 100, 100, 333, 700], size=100).tolist()
    w = W.make_workload("lpt", 50, B=100, Hq=8, Hkv=4, d=64, page_size=16, num_pages=2600,
                        context_lens=lens, rope_base=10000.0, inactive_rows=(0, 17, 99))
    st, _ = run_and_compare(rt, w, num_splits=splits)
    assert (rt.bits_of(st.out)[[0, 17, 99]] == 0).all()


@pytest.mark.parametrize("fused", [False, True, "step"])
def test_caller_supplied_row_order(rt, fused):
    # any permutation of the rows gives the same result; the runner's default for large batches is
    # "longest first", here also a random one and the identity, on a grid several waves deep
    import torch
    rng = np.random.default_rng(13)
    lens = rng.integers(0, 600, size=200).tolist()
    w = W.make_workload("order", 55, B=200, Hq=8, Hkv=4, d=64, page_size=16, num_pages=8000,
                        context_lens=lens, rope_base=10000.0, inactive_rows=(5, 150))
    q_rot, k_after, v_after, out_ref = O.oracle_decode_step(w)
    outs = []
    for order in ("auto", rng.permutation(200).astype(np.int32), None):
        st = rt.DecodeStep(w, num_splits=2, fused_merge=bool(fused), fused_step=(fused == "step"),
                           row_order=order)
        assert (st.row_order is not None) == (order is not None)
        st.step()
        torch.cuda.synchronize()
        assert int(st.status_flag.item()) == 0
        check_out(st.out_f64(), out_ref, "row order")
        k_gpu, v_gpu = st.cache_bits()
        assert np.array_equal(k_gpu, k_after) and np.array_equal(v_gpu, v_after)
        outs.append(rt.bits_of(st.out).copy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


def test_fused_merge_repeated_launches_and_row_without_tokens(rt):
    # The arrival counters reset themselves: many launches on one workspace stay correct, also when a
    # row has no tokens at all (its output is +0) and when most splits of a short row are empty.
    import torch
    w = small(49, B=4, Hq=16, Hkv=2, context_lens=[1500, 10, 700, 64], num_pages=200, inactive_rows=(3,))
    q_rot, k_after, v_after, out_ref = O.oracle_decode_step(w)
    st = rt.DecodeStep(w, num_splits=6, fused_merge=True)
    st.rope_kv_append()
    for i in range(20):
        st.out.fill_(0x7FC0)
        st.attention()
        torch.cuda.synchronize()
        check_out(st.out_f64(), out_ref, f"fused launch {i}")
    assert (rt.bits_of(st.out)[3] == 0).all()
    n = st.B * st.Hq * st.num_splits * (st.d + 1)
    counters = st.workspace.view(torch.int32)[n:n + st.B * st.Hkv]
    assert int(counters.abs().sum().item()) == 0


@pytest.mark.parametrize("fused", [True, "step"])
def test_workload_gqa_group16(rt, fused):
    run_and_compare(rt, W.gqa_group16(), fused=fused)


@pytest.mark.parametrize("fused", [True, "step"])
def test_workload_sliding_window_4k(rt, fused):
    w = W.sliding_window_4k()
    run_and_compare(rt, w, fused=fused, window=w.window)


@pytest.mark.parametrize("name", ["qwen3_like_b32", "glm4_like_b32"])
def test_workload_model_variants(rt, name):
    # the two model-shaped workloads of the benchmark: the single-launch step with the options the
    # workload names (Q/K RMSNorm; 32:2 GQA with partial, interleaved rotary) against the oracle's chain
    import torch
    w = W.NAMED[name]()
    opts = w.extra["rope_variants"]
    q_rot, k_after, v_after = O.oracle_rope_kv_append_ex(
        w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.rope_cos, w.rope_sin,
        w.page_size, rotary_dim=opts.get("rotary_dim"), interleaved=opts.get("interleaved", False),
        q_norm_weight=opts.get("q_norm_weight"), k_norm_weight=opts.get("k_norm_weight"),
        norm_eps=opts.get("norm_eps", 0.0))
    out_ref = O.oracle_paged_decode_attn(q_rot, k_after, v_after, w.block_table, w.context_lens, w.page_size)
    st = rt.DecodeStep(w, fused_step=True, rope_variants="workload")
    st.step()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    assert np.array_equal(rt.bits_of(st.q_rot), q_rot), "q after norm/rotation differs"
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_after) and np.array_equal(v_gpu, v_after)
    check_out(st.out_f64(), out_ref, name)


_LONG_CONTEXT_ORACLE = {}


def long_context_oracle():
    """The oracle's whole step on the long-context workload, computed once per test session.

    Append and rotation by the oracle's own routine on the whole pools; attention by the oracle's own
    routine on every one of the B x Hkv (request, KV head) pairs, each call seeing only that pair's
    pages and head (views of the oracle's appended pools), the pairs spread over a thread pool.
    Returns (workload, q_rot bits, K pool after, V pool after, out fp64 [B,Hq,d])."""
    if not _LONG_CONTEXT_ORACLE:
        import os
        from concurrent.futures import ThreadPoolExecutor
        w = W.long_context()
        q_rot, k_after, v_after = O.oracle_rope_kv_append(
            w.q, w.k_new, w.v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.rope_cos,
            w.rope_sin, w.page_size)
        G = w.Hq // w.Hkv
        out = np.zeros((w.B, w.Hq, w.d), dtype=np.float64)

        def one(pair):
            b, h = pair
            used = w.block_table[b, :(int(w.context_lens[b]) + w.page_size) // w.page_size]
            remap = np.arange(used.size, dtype=np.int32)[None, :]
            kc = k_after[used, :, h:h + 1, :]            # this pair's pages and head only
            vc = v_after[used, :, h:h + 1, :]
            out[b, h * G:(h + 1) * G] = O.oracle_paged_decode_attn(
                q_rot[b:b + 1, h * G:(h + 1) * G], kc, vc, remap, w.context_lens[b:b + 1], w.page_size)[0]

        pairs = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
        with ThreadPoolExecutor(min(len(pairs), len(os.sched_getaffinity(0)))) as ex:
            list(ex.map(one, pairs))
        _LONG_CONTEXT_ORACLE["v"] = (w, q_rot, k_after, v_after, out)
    return _LONG_CONTEXT_ORACLE["v"]


@pytest.mark.parametrize("fused", [False, True, "step"])
def test_workload_long_context_all_heads(rt, fused):
    # the headline workload in the launch configuration the benchmark times (planned splits), every
    # one of its 4 x 64 output heads against the oracle, and both pools bit for bit
    import torch
    w, q_rot, k_after, v_after, out_ref = long_context_oracle()
    st = rt.DecodeStep(w, fused_merge=bool(fused), fused_step=(fused == "step"))
    st.step()
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    assert st.num_splits > 1
    assert np.array_equal(rt.bits_of(st.q_rot), q_rot), "rotated q differs"
    k_gpu, v_gpu = st.cache_bits()
    assert np.array_equal(k_gpu, k_after), "K pool differs"
    assert np.array_equal(v_gpu, v_after), "V pool differs"
    worst = check_out(st.out_f64(), out_ref, f"long_context S={st.num_splits} fused={fused}")
    print(f"[parity] long_context all heads S={st.num_splits} fused={fused}: worst err/bound = {worst:.3f}")


# ---------------------------------------------------------------------------------------------
# Seeded random configurations: shapes, lengths, page sizes, layouts, splits, windows and launch
# flavours drawn together, so that combinations nobody wrote down by hand are exercised as well.
# ---------------------------------------------------------------------------------------------

def _random_case(seed):
    rng = np.random.default_rng(9000 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 4, 8]))
    G = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 12, 16]))
    ps = int(rng.choice([16, 32, 48, 64, 128]))
    B = int(rng.integers(1, 10))
    top = int(rng.choice([40, 300, 1500, 5000]))
    lens = rng.integers(0, top + 1, size=B)
    # sprinkle the boundaries: empty cache, one token, exact page and tile multiples
    for b in range(B):
        r = rng.random()
        if r < 0.08:
            lens[b] = 0
        elif r < 0.16:
            lens[b] = ps * int(rng.integers(1, 4)) - int(rng.integers(0, 2))
        elif r < 0.24:
            lens[b] = 16 * int(rng.integers(1, 9)) - 1
    inactive = tuple(int(b) for b in range(B) if rng.random() < 0.12)
    if len(inactive) == B:
        inactive = inactive[1:]
    pages = int(sum((int(n) + 1 + ps - 1) // ps for n in lens)) + int(rng.integers(2, 40))
    w = W.make_workload(f"random{seed}", 9000 + seed, B=B, Hq=G * Hkv, Hkv=Hkv, d=d, page_size=ps,
                        num_pages=pages, context_lens=lens.tolist(), rope_base=float(rng.choice([1e4, 5e5])),
                        inactive_rows=inactive, peak_fraction=float(rng.choice([0.0, 0.02])))
    max_len = int(lens.max()) + 1
    splits = None if rng.random() < 0.3 else int(rng.integers(1, max(2, min(9, max_len // 64 + 2))))
    layout = str(rng.choice(["token_major", "head_major"]))
    fused = [False, True, "step"][int(rng.integers(0, 3))]
    window = 0 if rng.random() < 0.6 else int(rng.integers(1, max_len + 40))
    return w, splits, layout, fused, window


@pytest.mark.parametrize("seed", range(40))
def test_random_configurations_match_oracle(rt, seed):
    w, splits, layout, fused, window = _random_case(seed)
    run_and_compare(rt, w, num_splits=splits, layout=layout, fused=fused, window=window,
                    check_cache=True)


def test_hbm_read_probe_runs_and_validates(rt):
    import torch
    from paper_2606_07665_b200 import binding as ac
    buf = torch.full((1 << 20,), 0x01010101, dtype=torch.int32, device="cuda")
    sink = torch.zeros(2, dtype=torch.int64, device="cuda")
    ac.ac_hbm_read_probe(buf, buf.numel() * 4, sink)
    ac.ac_hbm_read_probe(buf, 16 * 3 + 5, sink)               # ragged tail is ignored
    torch.cuda.synchronize()
    assert int(sink[0].item()) == 0 and int(buf.sum().item()) == (1 << 20) * 0x01010101
    assert ac.lib().ac_hbm_read_probe(None, 1024, None, None) == 1
    assert ac.lib().ac_hbm_read_probe(buf.data_ptr() + 4, 1024, None, None) == 4
    assert ac.lib().ac_hbm_read_probe(buf.data_ptr(), 8, None, None) == 2


def test_maximum_batch(rt):
    """B = 65535, the largest batch the ABI accepts (grid.y limit): every row gets its own CTA."""
    B = 65535
    rng = np.random.default_rng(B)
    lens = rng.integers(0, 21, size=B).tolist()
    w = W.make_workload("max_batch", B, B=B, Hq=2, Hkv=1, d=64, page_size=16,
                        num_pages=sum((n + 16) // 16 for n in lens) + 8, context_lens=lens, rope_base=10000.0)
    run_and_compare(rt, w, fused="step")
