"""The allocation-free attention entry point against the regular one.

Some users of this library cannot allocate device memory around a decode step -- an engine that has
already given all free HBM to its KV-cache pool, code that runs where the host framework forbids
cudaMalloc, a step function with nowhere to keep a workspace -- so
``ac_paged_decode_attn_static_scratch`` keeps the split partials in an array built into the library.
This test calls it through the C ABI twice in a row, on different workloads so the second call sees
the first call's leftovers in the shared array, and compares each result with what
``ac_paged_decode_attn`` + ``ac_splitkv_merge`` produce with a caller-allocated workspace.  Both
paths run the same kernels on the same inputs, so the outputs must agree bit for bit, which is
inside the tolerance the parity tests use.  The file is named so that pytest collects it last.
"""
import numpy as np
import pytest

from paper_2606_07665_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _both_paths(runner, ac, torch, w, num_splits):
    st = runner.DecodeStep(w, num_splits=num_splits, fused_merge=False)
    st.rope_kv_append()
    st.attention()
    st.merge()
    torch.cuda.synchronize()
    want = runner.bits_of(st.out).copy()
    want_f = st.out_f64()
    st.out.fill_(0x7FC0)          # NaN pattern: the new entry point must overwrite every row
    ac.ac_paged_decode_attn_static_scratch(
        st.q_rot, st.k_cache, st.v_cache, st.stride_page, st.stride_token, st.stride_head,
        st.block_table, w.max_pages_per_seq, st.context_lens, 1, 0.0, num_splits, st.out,
        st.B, st.Hq, st.Hkv, st.d, st.ps, st.num_pages, st.max_context_len, st.status_flag)
    torch.cuda.synchronize()
    assert int(st.status_flag.item()) == 0
    got = runner.bits_of(st.out)
    got_f = st.out_f64()
    assert np.isfinite(got_f).all()
    err = np.abs(got_f - want_f)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3       # the parity tests' tolerance
    assert np.array_equal(got, want)                       # same kernels, same inputs: same bits


def test_static_scratch_matches_workspace_path_twice_in_a_row():
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    first = W.make_workload("noalloc_a", 71, B=3, Hq=16, Hkv=2, d=128, page_size=16, num_pages=200,
                            context_lens=[900, 130, 2047], rope_base=10000.0)
    second = W.make_workload("noalloc_b", 72, B=2, Hq=28, Hkv=4, d=128, page_size=32, num_pages=64,
                             context_lens=[300, 64], rope_base=10000.0, inactive_rows=(1,))
    _both_paths(runner, ac, torch, first, num_splits=6)
    _both_paths(runner, ac, torch, second, num_splits=3)     # fewer, shorter rows over stale contents
    _both_paths(runner, ac, torch, second, num_splits=1)     # single split: no scratch involved


def test_static_scratch_rejects_oversized_requests():
    import torch
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build
    build.build()
    torch.cuda.set_device(0)
    ac.ac_init(0)
    p = 0x1000            # never dereferenced: the size check comes first
    # 64 * 64 * 64 * 129 * 4 bytes = 135 MB of partials > 8 MiB
    rc = ac.lib().ac_paged_decode_attn_static_scratch(p, p, p, 2048, 128, 64, p, 64, p, 1, 0.0, 64, p,
                                                      64, 64, 8, 128, 16, 4096, 8192, None, None)
    assert rc == 8
    assert "AC_STATIC_SCRATCH_BYTES" in ac.lib().ac_status_string(rc).decode()
