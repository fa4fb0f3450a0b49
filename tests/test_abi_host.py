"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared symbol,
the pure planning helpers behave, and argument validation rejects bad calls without launching."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ac():
    from paper_2606_07665_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ac.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ac_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(ac):
    names = declared_functions()
    assert "ac_paged_decode_attn" in names and "ac_rope_kv_append" in names and "ac_splitkv_merge" in names
    lib = ctypes.CDLL(ac.lib_path())
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ac.EXPORTS) == names


def test_status_strings(ac):
    for code in range(0, 8):
        s = ac.lib().ac_status_string(code).decode()
        assert s and s != "unknown status"
    assert ac.lib().ac_status_string(99).decode() == "unknown status"


def test_split_tokens_and_workspace(ac):
    assert ac.ac_split_tokens(4097, 1) == 4160          # multiple of 64 covering the context
    assert ac.ac_split_tokens(4097, 4) == 1088
    assert ac.ac_split_tokens(1, 8) == 64
    for n, s in ((513, 3), (131073, 64), (8192, 7), (2049, 2)):
        st = ac.ac_split_tokens(n, s)
        assert st % 64 == 0 and st * s >= n and (st - 64) * s < n
    assert ac.ac_workspace_bytes(4, 64, 128, 1) == 0
    assert ac.ac_workspace_bytes(4, 64, 128, 16) == 4 * 64 * 16 * 129 * 4


@pytest.mark.parametrize("B,Hq,Hkv,d,ps,maxlen", [
    (1, 8, 2, 64, 16, 513), (1, 32, 8, 128, 16, 4097), (64, 32, 8, 128, 16, 7979),
    (4, 64, 8, 128, 16, 131073), (1, 28, 4, 128, 32, 2049), (256, 28, 4, 128, 32, 2049)])
def test_plan_properties(ac, B, Hq, Hkv, d, ps, maxlen):
    S, st, wb = ac.ac_decode_plan(B, Hq, Hkv, d, ps, maxlen, 148)
    assert S >= 1 and st % 64 == 0
    assert st == ac.ac_split_tokens(maxlen, S)
    assert st * S >= maxlen and st * (S - 1) < maxlen          # no split is empty for the longest row
    assert wb == ac.ac_workspace_bytes(B, Hq, d, S)
    if S > 1:                                                     # splits stay long enough to amortise set-up:
        in_cluster = S <= 16 and B * Hkv * S <= 148              # 128 tokens where the merge is the cheap
        assert st >= (128 if in_cluster else 256)                 # one inside a cluster, 256 otherwise
    if B * Hkv >= 148 * 2 and maxlen <= 4096:
        assert S == 1                                             # already enough CTAs without splitting
    if B * Hkv < 148 and maxlen >= 512:
        assert S > 1                                              # small batches are split across SMs


def test_plan_fills_one_wave_for_very_long_contexts(ac):
    # few requests, very long contexts: the most splits of at least 8192 tokens that still fit one wave
    # of two CTAs per SM -- the shape the launch runs with four warps per CTA
    for B, Hkv, maxlen, want in [(4, 8, 131073, 9), (2, 8, 131073, 16), (8, 8, 131073, 4), (1, 8, 1000000, 37)]:
        S, st, _ = ac.ac_decode_plan(B, 8 * Hkv, Hkv, 128, 16, maxlen, 148)
        assert S == want, (B, Hkv, maxlen, S)
        assert st >= 8192 and 148 < B * Hkv * S <= 296 and st * (S - 1) < maxlen


def test_plan_for_lengths(ac):
    import numpy as np
    # every row at the maximum: the same plan as without lengths
    for B, Hq, Hkv, d, ps, maxlen in [(1, 32, 8, 128, 16, 4097), (8, 28, 4, 128, 32, 2049), (4, 64, 8, 128, 16, 131073),
                                      (64, 32, 8, 128, 16, 8193), (256, 28, 4, 128, 32, 2049)]:
        assert ac.ac_decode_plan_for_lengths([maxlen] * B, Hq, Hkv, d, ps, maxlen, 148) == \
            ac.ac_decode_plan(B, Hq, Hkv, d, ps, maxlen, 148)
    # a ragged batch: splits beyond a row's end cost nothing, so the plan may split finer -- never coarser --
    # and still leaves no split empty for the longest row
    rng = np.random.default_rng(5)
    for B, Hkv in [(32, 4), (16, 2), (8, 4), (48, 2)]:
        lens = rng.integers(513, 2050, size=B).tolist()
        maxlen = max(lens)
        S0, _, _ = ac.ac_decode_plan(B, 4 * Hkv, Hkv, 128, 16, maxlen, 148)
        S1, st1, wb1 = ac.ac_decode_plan_for_lengths(lens, 4 * Hkv, Hkv, 128, 16, maxlen, 148)
        assert S1 >= S0
        assert st1 == ac.ac_split_tokens(maxlen, S1) and st1 * (S1 - 1) < maxlen
        assert wb1 == ac.ac_workspace_bytes(B, 4 * Hkv, 128, S1)
        pieces = sum(-(-n // st1) for n in lens) * Hkv
        assert S1 == 1 or st1 >= 128
        assert S1 == S0 or pieces <= 2 * 148                      # the finer plan still fits one wave
    # inactive rows launch nothing: they count neither as pairs nor as bytes.  (The grid they widen does
    # decide which kernel flavour a launch gets -- twelve-warp CTAs and the cluster merge need a grid of
    # at most one CTA per SM -- so the comparison is between two grids of the same kind.)
    lens = [2000, 1800] + [0, -1] * 15
    assert ac.ac_decode_plan_for_lengths(lens, 32, 8, 128, 16, 2000, 148)[0] == \
        ac.ac_decode_plan_for_lengths(lens + [0] * 16, 32, 8, 128, 16, 2000, 148)[0]
    assert ac.ac_decode_plan_for_lengths(lens, 32, 8, 128, 16, 2000, 148)[0] > \
        ac.ac_decode_plan_for_lengths([2000] * 32, 32, 8, 128, 16, 2000, 148)[0]
    # the graph-sweep bucket of 32 requests: 128 (request, KV head) pairs fit the GPU at one twelve-warp
    # CTA per SM, which streams fast enough that no split (and no merge) is the cheapest plan
    from paper_2606_07665_b200 import workloads as W
    w = W.graph_sweep(32)
    counts = [int(n) + 1 for n in w.context_lens]
    assert ac.ac_decode_plan_for_lengths(counts, w.Hq, w.Hkv, w.d, w.page_size, w.max_context_len, 148)[0] == 1
    L = ac.lib()
    ns, st, wb = ctypes.c_int(), ctypes.c_int(), ctypes.c_size_t()
    assert L.ac_decode_plan_for_lengths(None, 4, 8, 2, 64, 16, 512, 148, ctypes.byref(ns), ctypes.byref(st),
                                        ctypes.byref(wb)) == 1


def test_plan_rejects_bad_shapes(ac):
    L = ac.lib()
    ns, st, wb = ctypes.c_int(), ctypes.c_int(), ctypes.c_size_t()
    args = (ctypes.byref(ns), ctypes.byref(st), ctypes.byref(wb))
    assert L.ac_decode_plan(1, 8, 2, 64, 16, 512, 148, None, None, None) == 1
    assert L.ac_decode_plan(0, 8, 2, 64, 16, 512, 148, *args) == 2
    assert L.ac_decode_plan(1, 8, 3, 64, 16, 512, 148, *args) == 2        # Hq % Hkv
    assert L.ac_decode_plan(1, 8, 2, 96, 16, 512, 148, *args) == 3        # head_dim
    assert L.ac_decode_plan(1, 8, 2, 64, 24, 512, 148, *args) == 3        # page size
    assert L.ac_decode_plan(1, 34, 2, 64, 16, 512, 148, *args) == 3       # group of 17
    assert L.ac_decode_plan(1, 8, 2, 64, 16, 0, 148, *args) == 2


def test_kernel_calls_validate_before_touching_the_device(ac):
    # No GPU here: every one of these must return a validation status, never reach a launch.
    L = ac.lib()
    p = 0x1000            # fake, aligned, never dereferenced on the host
    common_tail = (1, 8, 2, 64, 16, 64)
    assert L.ac_rope_kv_append(None, p, p, p, p, p, 2048, 128, 64, p, 33, p, p, p, 513,
                               *common_tail, None, None) == 1
    assert L.ac_rope_kv_append(p, p, p, p, p, p, 2048, 128, 64, p, 33, p, p, p, 513,
                               1, 8, 2, 80, 16, 64, None, None) == 3
    assert L.ac_rope_kv_append(p, p, p, p, p + 2, p, 2048, 128, 64, p, 33, p, p, p, 513,
                               *common_tail, None, None) == 4
    assert L.ac_rope_kv_append(p, p, p, p, p, p, 2048, 100, 64, p, 33, p, p, p, 513,
                               *common_tail, None, None) == 4          # stride not a multiple of 8
    assert L.ac_rope_kv_append(p, p, p, p, p, p, 2048, 128, 32, p, 33, p, p, p, 513,
                               *common_tail, None, None) == 2          # head stride < head_dim
    attn_tail = (1, 8, 2, 64, 16, 64, 513)
    assert L.ac_paged_decode_attn(p, p, None, 2048, 128, 64, p, 33, p, 1, 0.0, 1, None, 0, p,
                                  *attn_tail, None, None) == 1
    assert L.ac_paged_decode_attn(p, p, p, 2048, 128, 64, p, 33, p, 1, 0.0, 4, None, 0, p,
                                  *attn_tail, None, None) == 5         # splits without workspace
    assert L.ac_paged_decode_attn(p, p, p, 2048, 128, 64, p, 33, p, 1, 0.0, 4, p, 100, p,
                                  *attn_tail, None, None) == 5         # workspace too small
    assert L.ac_paged_decode_attn(p, p, p, 2048, 128, 64, p, 33, p, 2, 0.0, 1, None, 0, p,
                                  *attn_tail, None, None) == 3         # new_tokens not in {0,1}
    assert L.ac_paged_decode_attn(p, p, p, 2048, 128, 64, p, 33, p, 1, 0.0, 1, None, 0, None,
                                  *attn_tail, None, None) == 1         # single split needs out
    assert L.ac_splitkv_merge(None, 4, None, p, 1, 8, 64, None) == 1
    assert L.ac_splitkv_merge(p, 0, None, p, 1, 8, 64, None) == 2
    assert L.ac_splitkv_merge(p, 4, None, p, 1, 8, 96, None) == 3
    # valid arguments but no initialised device: refused, still nothing launched
    import torch
    if not torch.cuda.is_available():
        r = L.ac_splitkv_merge(p, 4, None, p, 1, 8, 64, None)
        assert r in (6, 7)


def test_binding_fails_loudly_without_the_library(tmp_path, monkeypatch):
    from paper_2606_07665_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="missing"):
        binding.lib()
