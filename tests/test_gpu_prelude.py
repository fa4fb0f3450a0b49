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
    (31, 768, 8, 2, 128, 16),         # batch tile of 32
    (40, 256, 4, 2, 64, 16),          # two batch tiles
    (4, 4096, 32, 8, 128, 16),        # 8B-class layer: 6144 x 4096 weights
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
