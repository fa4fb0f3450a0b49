"""ctypes binding of libac.so: the same entry points as include/ac.h, argument marshalling only.

Tensor arguments are torch CUDA tensors (their ``data_ptr()`` is passed through) or plain integer
addresses; ``stream`` is a ``torch.cuda.Stream``, a raw ``cudaStream_t`` integer, or None for torch's
current stream.  A non-zero status raises ``AcError``.  Nothing here computes anything: if the shared
library has not been built, loading it raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_float, c_int, c_int64, c_size_t, c_void_p, POINTER

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libac.so")
_lib = None

STATUS_NAMES = {0: "AC_OK", 1: "AC_ERR_NULL", 2: "AC_ERR_SHAPE", 3: "AC_ERR_UNSUPPORTED",
                4: "AC_ERR_ALIGN", 5: "AC_ERR_WORKSPACE", 6: "AC_ERR_CUDA", 7: "AC_ERR_NOT_INIT",
                8: "AC_ERR_SCRATCH_LIMIT"}
AC_FLAG_PAGE_OOB = 1
AC_FLAG_POSITION_OOB = 2
AC_FLAG_WAIT_TIMEOUT = 4

EXPORTS = ("ac_init", "ac_status_string", "ac_last_cuda_error", "ac_sm_count", "ac_decode_plan",
           "ac_decode_plan_for_lengths",
           "ac_split_tokens", "ac_workspace_bytes", "ac_rope_kv_append", "ac_paged_decode_attn",
           "ac_splitkv_merge", "ac_decode_step_host", "ac_paged_decode_attn_static_scratch",
           "ac_fused_workspace_bytes", "ac_fused_workspace_reset", "ac_paged_decode_attn_fused_merge",
           "ac_decode_step_fused", "ac_paged_decode_attn_ex", "ac_decode_step_fused_ex",
           "ac_rope_kv_append_ex", "ac_qkv_rope_kv_append", "ac_oproj_residual_rmsnorm",
           "ac_hbm_read_probe", "ac_qkv_rope_kv_append_ex")
AC_STATIC_SCRATCH_BYTES = 8 << 20


class AcAttnOptions(ctypes.Structure):
    """Mirror of ac_attn_options."""
    _fields_ = [("window", c_int), ("fused_merge", c_int), ("row_order", c_void_p), ("rope", c_void_p),
                ("reserved", c_int * 2)]


class AcRopeOptions(ctypes.Structure):
    """Mirror of ac_rope_options."""
    _fields_ = [("rotary_dim", c_int), ("interleaved", c_int), ("q_norm_weight", c_void_p),
                ("k_norm_weight", c_void_p), ("norm_eps", c_float), ("reserved", c_int * 4)]


class AcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().ac_status_string(status).decode()
        extra = f" (cuda error {lib().ac_last_cuda_error()})" if status == 6 else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}: {msg}{extra}")


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """The loaded shared library; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_2606_07665_b200.build`")
        L = ctypes.CDLL(_LIB_PATH)
        L.ac_init.argtypes = [c_int]
        L.ac_init.restype = c_int
        L.ac_status_string.argtypes = [c_int]
        L.ac_status_string.restype = c_char_p
        L.ac_last_cuda_error.argtypes = []
        L.ac_last_cuda_error.restype = c_int
        L.ac_sm_count.argtypes = []
        L.ac_sm_count.restype = c_int
        L.ac_decode_plan.argtypes = [c_int] * 7 + [POINTER(c_int), POINTER(c_int), POINTER(c_size_t)]
        L.ac_decode_plan.restype = c_int
        L.ac_decode_plan_for_lengths.argtypes = ([c_void_p] + [c_int] * 7 +
                                                 [POINTER(c_int), POINTER(c_int), POINTER(c_size_t)])
        L.ac_decode_plan_for_lengths.restype = c_int
        L.ac_split_tokens.argtypes = [c_int, c_int]
        L.ac_split_tokens.restype = c_int
        L.ac_workspace_bytes.argtypes = [c_int] * 4
        L.ac_workspace_bytes.restype = c_size_t
        L.ac_rope_kv_append.argtypes = ([c_void_p] * 6 + [c_int64] * 3 + [c_void_p, c_int, c_void_p,
                                        c_void_p, c_void_p, c_int] + [c_int] * 6 + [c_void_p, c_void_p])
        L.ac_rope_kv_append.restype = c_int
        L.ac_rope_kv_append_ex.argtypes = L.ac_rope_kv_append.argtypes + [POINTER(AcRopeOptions)]
        L.ac_rope_kv_append_ex.restype = c_int
        L.ac_qkv_rope_kv_append.argtypes = ([c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p] +
                                            [c_int64] * 3 + [c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                            c_int] + [c_int] * 6 + [c_void_p, c_void_p])
        L.ac_qkv_rope_kv_append.restype = c_int
        L.ac_qkv_rope_kv_append_ex.argtypes = L.ac_qkv_rope_kv_append.argtypes + [POINTER(AcRopeOptions)]
        L.ac_qkv_rope_kv_append_ex.restype = c_int
        L.ac_oproj_residual_rmsnorm.argtypes = [c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p,
                                                c_float, c_void_p, c_int, c_void_p]
        L.ac_oproj_residual_rmsnorm.restype = c_int
        L.ac_paged_decode_attn.argtypes = ([c_void_p] * 3 + [c_int64] * 3 + [c_void_p, c_int, c_void_p,
                                           c_int, c_float, c_int, c_void_p, c_size_t, c_void_p] +
                                           [c_int] * 7 + [c_void_p, c_void_p])
        L.ac_paged_decode_attn.restype = c_int
        L.ac_paged_decode_attn_fused_merge.argtypes = L.ac_paged_decode_attn.argtypes
        L.ac_paged_decode_attn_fused_merge.restype = c_int
        L.ac_fused_workspace_bytes.argtypes = [c_int] * 5
        L.ac_fused_workspace_bytes.restype = c_size_t
        L.ac_fused_workspace_reset.argtypes = [c_void_p, c_size_t] + [c_int] * 5 + [c_void_p]
        L.ac_fused_workspace_reset.restype = c_int
        L.ac_decode_step_fused.argtypes = ([c_void_p] * 6 + [c_int64] * 3 + [c_void_p, c_int, c_void_p,
                                           c_void_p, c_void_p, c_int, c_float, c_int, c_void_p, c_size_t,
                                           c_void_p] + [c_int] * 7 + [c_void_p, c_void_p])
        L.ac_decode_step_fused.restype = c_int
        L.ac_paged_decode_attn_ex.argtypes = L.ac_paged_decode_attn.argtypes + [POINTER(AcAttnOptions)]
        L.ac_paged_decode_attn_ex.restype = c_int
        L.ac_decode_step_fused_ex.argtypes = L.ac_decode_step_fused.argtypes + [POINTER(AcAttnOptions)]
        L.ac_decode_step_fused_ex.restype = c_int
        L.ac_splitkv_merge.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p]
        L.ac_splitkv_merge.restype = c_int
        L.ac_decode_step_host.argtypes = ([c_void_p] * 6 + [c_void_p] * 6 + [c_void_p] * 2 + [c_int64] * 3 +
                                          [c_int, c_void_p, c_void_p, c_int, c_float, c_int, c_void_p,
                                           c_size_t] + [c_int] * 7 + [c_void_p, c_void_p])
        L.ac_decode_step_host.restype = c_int
        L.ac_paged_decode_attn_static_scratch.argtypes = ([c_void_p] * 3 + [c_int64] * 3 + [c_void_p, c_int,
                                                          c_void_p, c_int, c_float, c_int, c_void_p] +
                                                          [c_int] * 7 + [c_void_p, c_void_p])
        L.ac_paged_decode_attn_static_scratch.restype = c_int
        L.ac_hbm_read_probe.argtypes = [c_void_p, c_size_t, c_void_p, c_void_p]
        L.ac_hbm_read_probe.restype = c_int
        _lib = L
    return _lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str) -> None:
    if status != 0:
        raise AcError(status, where)


def ac_init(device: int = -1) -> None:
    _check(lib().ac_init(device), "ac_init")


def ac_sm_count() -> int:
    return lib().ac_sm_count()


def ac_split_tokens(max_context_len: int, num_splits: int) -> int:
    return lib().ac_split_tokens(max_context_len, num_splits)


def ac_workspace_bytes(B: int, Hq: int, d: int, num_splits: int) -> int:
    return lib().ac_workspace_bytes(B, Hq, d, num_splits)


def ac_decode_plan(B, Hq, Hkv, d, page_size, max_context_len, sm_count=0):
    """Returns (num_splits, split_tokens, workspace_bytes)."""
    ns, st, wb = c_int(0), c_int(0), c_size_t(0)
    _check(lib().ac_decode_plan(B, Hq, Hkv, d, page_size, max_context_len, sm_count,
                                ctypes.byref(ns), ctypes.byref(st), ctypes.byref(wb)), "ac_decode_plan")
    return ns.value, st.value, wb.value


def ac_decode_plan_for_lengths(token_counts, Hq, Hkv, d, page_size, max_context_len, sm_count=0):
    """token_counts: host sequence of B ints (tokens each row attends over; <= 0 = inactive row).
    Returns (num_splits, split_tokens, workspace_bytes)."""
    counts = (ctypes.c_int32 * len(token_counts))(*[int(t) for t in token_counts])
    ns, st, wb = c_int(0), c_int(0), c_size_t(0)
    _check(lib().ac_decode_plan_for_lengths(ctypes.cast(counts, c_void_p), len(token_counts), Hq, Hkv, d,
                                            page_size, max_context_len, sm_count, ctypes.byref(ns),
                                            ctypes.byref(st), ctypes.byref(wb)),
           "ac_decode_plan_for_lengths")
    return ns.value, st.value, wb.value


def ac_rope_kv_append(q_in, q_out, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                      stride_head, block_table, max_pages_per_seq, context_lens, rope_cos, rope_sin,
                      max_position, B, Hq, Hkv, d, page_size, num_pages, status_flag=None, stream=None):
    _check(lib().ac_rope_kv_append(_ptr(q_in), _ptr(q_out), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                   _ptr(v_cache), stride_page, stride_token, stride_head,
                                   _ptr(block_table), max_pages_per_seq, _ptr(context_lens),
                                   _ptr(rope_cos), _ptr(rope_sin), max_position, B, Hq, Hkv, d,
                                   page_size, num_pages, _ptr(status_flag), _stream(stream)),
           "ac_rope_kv_append")


def ac_rope_kv_append_ex(q_in, q_out, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                         stride_head, block_table, max_pages_per_seq, context_lens, rope_cos, rope_sin,
                         max_position, B, Hq, Hkv, d, page_size, num_pages, status_flag=None, stream=None,
                         rotary_dim=0, interleaved=False, q_norm_weight=None, k_norm_weight=None,
                         norm_eps=0.0):
    opt = _rope_options(rotary_dim, interleaved, q_norm_weight, k_norm_weight, norm_eps)
    _check(lib().ac_rope_kv_append_ex(_ptr(q_in), _ptr(q_out), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                      _ptr(v_cache), stride_page, stride_token, stride_head,
                                      _ptr(block_table), max_pages_per_seq, _ptr(context_lens),
                                      _ptr(rope_cos), _ptr(rope_sin), max_position, B, Hq, Hkv, d,
                                      page_size, num_pages, _ptr(status_flag), _stream(stream),
                                      ctypes.byref(opt)), "ac_rope_kv_append_ex")


def ac_qkv_rope_kv_append(x, w_qkv, H, q_out, k_cache, v_cache, stride_page, stride_token, stride_head,
                          block_table, max_pages_per_seq, context_lens, rope_cos, rope_sin, max_position,
                          B, Hq, Hkv, d, page_size, num_pages, status_flag=None, stream=None):
    _check(lib().ac_qkv_rope_kv_append(_ptr(x), _ptr(w_qkv), H, _ptr(q_out), _ptr(k_cache), _ptr(v_cache),
                                       stride_page, stride_token, stride_head, _ptr(block_table),
                                       max_pages_per_seq, _ptr(context_lens), _ptr(rope_cos),
                                       _ptr(rope_sin), max_position, B, Hq, Hkv, d, page_size, num_pages,
                                       _ptr(status_flag), _stream(stream)), "ac_qkv_rope_kv_append")


def ac_qkv_rope_kv_append_ex(x, w_qkv, H, q_out, k_cache, v_cache, stride_page, stride_token, stride_head,
                             block_table, max_pages_per_seq, context_lens, rope_cos, rope_sin, max_position,
                             B, Hq, Hkv, d, page_size, num_pages, status_flag=None, stream=None,
                             rotary_dim=0, interleaved=False, q_norm_weight=None, k_norm_weight=None,
                             norm_eps=0.0):
    opt = _rope_options(rotary_dim, interleaved, q_norm_weight, k_norm_weight, norm_eps)
    _check(lib().ac_qkv_rope_kv_append_ex(_ptr(x), _ptr(w_qkv), H, _ptr(q_out), _ptr(k_cache), _ptr(v_cache),
                                          stride_page, stride_token, stride_head, _ptr(block_table),
                                          max_pages_per_seq, _ptr(context_lens), _ptr(rope_cos),
                                          _ptr(rope_sin), max_position, B, Hq, Hkv, d, page_size, num_pages,
                                          _ptr(status_flag), _stream(stream), ctypes.byref(opt)),
           "ac_qkv_rope_kv_append_ex")


def ac_oproj_residual_rmsnorm(attn_out, w_o, K, N, residual_in, residual_out, norm_weight, norm_eps,
                              normed_out, B, stream=None):
    _check(lib().ac_oproj_residual_rmsnorm(_ptr(attn_out), _ptr(w_o), K, N, _ptr(residual_in),
                                           _ptr(residual_out), _ptr(norm_weight), norm_eps,
                                           _ptr(normed_out), B, _stream(stream)),
           "ac_oproj_residual_rmsnorm")


def ac_paged_decode_attn(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head, block_table,
                         max_pages_per_seq, context_lens, new_tokens, softmax_scale, num_splits,
                         workspace, workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages,
                         max_context_len, status_flag=None, stream=None):
    _check(lib().ac_paged_decode_attn(_ptr(q_rot), _ptr(k_cache), _ptr(v_cache), stride_page,
                                      stride_token, stride_head, _ptr(block_table), max_pages_per_seq,
                                      _ptr(context_lens), new_tokens, softmax_scale, num_splits,
                                      _ptr(workspace), workspace_bytes, _ptr(out), B, Hq, Hkv, d,
                                      page_size, num_pages, max_context_len, _ptr(status_flag),
                                      _stream(stream)), "ac_paged_decode_attn")


def ac_fused_workspace_bytes(B: int, Hq: int, Hkv: int, d: int, num_splits: int) -> int:
    return lib().ac_fused_workspace_bytes(B, Hq, Hkv, d, num_splits)


def ac_fused_workspace_reset(workspace, workspace_bytes, B, Hq, Hkv, d, num_splits, stream=None):
    _check(lib().ac_fused_workspace_reset(_ptr(workspace), workspace_bytes, B, Hq, Hkv, d, num_splits,
                                          _stream(stream)), "ac_fused_workspace_reset")


def ac_paged_decode_attn_fused_merge(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head,
                                     block_table, max_pages_per_seq, context_lens, new_tokens,
                                     softmax_scale, num_splits, workspace, workspace_bytes, out, B, Hq,
                                     Hkv, d, page_size, num_pages, max_context_len, status_flag=None,
                                     stream=None):
    _check(lib().ac_paged_decode_attn_fused_merge(
        _ptr(q_rot), _ptr(k_cache), _ptr(v_cache), stride_page, stride_token, stride_head,
        _ptr(block_table), max_pages_per_seq, _ptr(context_lens), new_tokens, softmax_scale, num_splits,
        _ptr(workspace), workspace_bytes, _ptr(out), B, Hq, Hkv, d, page_size, num_pages,
        max_context_len, _ptr(status_flag), _stream(stream)), "ac_paged_decode_attn_fused_merge")


def ac_decode_step_fused(q_in, q_rot_out, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                         stride_head, block_table, max_pages_per_seq, context_lens, rope_cos, rope_sin,
                         max_position, softmax_scale, num_splits, workspace, workspace_bytes, out, B, Hq,
                         Hkv, d, page_size, num_pages, max_context_len, status_flag=None, stream=None):
    _check(lib().ac_decode_step_fused(
        _ptr(q_in), _ptr(q_rot_out), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), stride_page,
        stride_token, stride_head, _ptr(block_table), max_pages_per_seq, _ptr(context_lens),
        _ptr(rope_cos), _ptr(rope_sin), max_position, softmax_scale, num_splits, _ptr(workspace),
        workspace_bytes, _ptr(out), B, Hq, Hkv, d, page_size, num_pages, max_context_len,
        _ptr(status_flag), _stream(stream)), "ac_decode_step_fused")


def _rope_options(rotary_dim=0, interleaved=False, q_norm_weight=None, k_norm_weight=None, norm_eps=0.0):
    opt = AcRopeOptions()
    opt.rotary_dim = int(rotary_dim)
    opt.interleaved = 1 if interleaved else 0
    opt.q_norm_weight = _ptr(q_norm_weight)
    opt.k_norm_weight = _ptr(k_norm_weight)
    opt.norm_eps = float(norm_eps)
    return opt


def _options(window: int = 0, fused_merge: bool = False, row_order=None, rope=None):
    """rope: an AcRopeOptions instance (kept alive by the returned structure) or None."""
    opt = AcAttnOptions()
    opt.window = int(window)
    opt.fused_merge = 1 if fused_merge else 0
    opt.row_order = _ptr(row_order)
    opt.rope = ctypes.addressof(rope) if rope is not None else None
    opt._keep = rope
    return opt


def ac_paged_decode_attn_ex(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head, block_table,
                            max_pages_per_seq, context_lens, new_tokens, softmax_scale, num_splits,
                            workspace, workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages,
                            max_context_len, status_flag=None, stream=None, window=0, fused_merge=False,
                            row_order=None):
    _check(lib().ac_paged_decode_attn_ex(
        _ptr(q_rot), _ptr(k_cache), _ptr(v_cache), stride_page, stride_token, stride_head,
        _ptr(block_table), max_pages_per_seq, _ptr(context_lens), new_tokens, softmax_scale, num_splits,
        _ptr(workspace), workspace_bytes, _ptr(out), B, Hq, Hkv, d, page_size, num_pages,
        max_context_len, _ptr(status_flag), _stream(stream),
        ctypes.byref(_options(window, fused_merge, row_order))), "ac_paged_decode_attn_ex")


def ac_decode_step_fused_ex(q_in, q_rot_out, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                            stride_head, block_table, max_pages_per_seq, context_lens, rope_cos, rope_sin,
                            max_position, softmax_scale, num_splits, workspace, workspace_bytes, out, B,
                            Hq, Hkv, d, page_size, num_pages, max_context_len, status_flag=None,
                            stream=None, window=0, row_order=None, rotary_dim=0, interleaved=False,
                            q_norm_weight=None, k_norm_weight=None, norm_eps=0.0):
    """The rope keywords are those of ac_rope_kv_append_ex (all default = the plain rotation)."""
    variants = rotary_dim or interleaved or q_norm_weight is not None or k_norm_weight is not None
    rope = _rope_options(rotary_dim, interleaved, q_norm_weight, k_norm_weight, norm_eps) if variants else None
    opt = _options(window, False, row_order, rope)
    _check(lib().ac_decode_step_fused_ex(
        _ptr(q_in), _ptr(q_rot_out), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), stride_page,
        stride_token, stride_head, _ptr(block_table), max_pages_per_seq, _ptr(context_lens),
        _ptr(rope_cos), _ptr(rope_sin), max_position, softmax_scale, num_splits, _ptr(workspace),
        workspace_bytes, _ptr(out), B, Hq, Hkv, d, page_size, num_pages, max_context_len,
        _ptr(status_flag), _stream(stream), ctypes.byref(opt)), "ac_decode_step_fused_ex")


def ac_splitkv_merge(workspace, num_splits, context_lens, out, B, Hq, d, stream=None):
    _check(lib().ac_splitkv_merge(_ptr(workspace), num_splits, _ptr(context_lens), _ptr(out), B, Hq, d,
                                  _stream(stream)), "ac_splitkv_merge")


def ac_decode_step_host(q_host, k_new_host, v_new_host, block_table_host, context_lens_host, out_host,
                        q, k_new, v_new, block_table, context_lens, out, k_cache, v_cache, stride_page,
                        stride_token, stride_head, max_pages_per_seq, rope_cos, rope_sin, max_position,
                        softmax_scale, num_splits, workspace, workspace_bytes, B, Hq, Hkv, d, page_size,
                        num_pages, max_context_len, status_flag=None, stream=None):
    _check(lib().ac_decode_step_host(_ptr(q_host), _ptr(k_new_host), _ptr(v_new_host),
                                     _ptr(block_table_host), _ptr(context_lens_host), _ptr(out_host),
                                     _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(block_table),
                                     _ptr(context_lens), _ptr(out), _ptr(k_cache), _ptr(v_cache),
                                     stride_page, stride_token, stride_head, max_pages_per_seq,
                                     _ptr(rope_cos), _ptr(rope_sin), max_position, softmax_scale,
                                     num_splits, _ptr(workspace), workspace_bytes, B, Hq, Hkv, d,
                                     page_size, num_pages, max_context_len, _ptr(status_flag),
                                     _stream(stream)), "ac_decode_step_host")


def ac_paged_decode_attn_static_scratch(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head,
                                        block_table, max_pages_per_seq, context_lens, new_tokens,
                                        softmax_scale, num_splits, out, B, Hq, Hkv, d, page_size,
                                        num_pages, max_context_len, status_flag=None, stream=None):
    """Attention + merge with the split partials in the library's built-in array (no workspace
    argument, no allocation anywhere in the call); see include/ac.h for the size limit and rules."""
    _check(lib().ac_paged_decode_attn_static_scratch(
        _ptr(q_rot), _ptr(k_cache), _ptr(v_cache), stride_page, stride_token, stride_head,
        _ptr(block_table), max_pages_per_seq, _ptr(context_lens), new_tokens, softmax_scale, num_splits,
        _ptr(out), B, Hq, Hkv, d, page_size, num_pages, max_context_len, _ptr(status_flag),
        _stream(stream)), "ac_paged_decode_attn_static_scratch")


def ac_hbm_read_probe(buffer, nbytes, sink=None, stream=None):
    """Enqueues one read-only pass over ``buffer`` (calibration; the caller times it)."""
    _check(lib().ac_hbm_read_probe(_ptr(buffer), nbytes, _ptr(sink), _stream(stream)), "ac_hbm_read_probe")
