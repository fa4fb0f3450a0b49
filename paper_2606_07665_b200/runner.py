"""Device-side staging of a workload and the launch sequence of one decode step.

Only plumbing: torch tensors for device memory, the split plan from the library, and the three
C-ABI calls in order.  Every arithmetic step runs inside libac's kernels.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as ac


def _dev_u16(a: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> device int16 tensor (same bits)."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device)


def bits_of(t: torch.Tensor) -> np.ndarray:
    """Device int16 tensor -> host uint16 bit patterns."""
    return t.detach().cpu().numpy().view(np.uint16)


class DecodeStep:
    """Holds one workload on the device and enqueues RoPE+append -> attention -> merge.

    ``layout`` is "token_major" ([page, slot, head, d], the default) or "head_major"
    ([page, head, slot, d]); the kernels see only the strides.
    """

    def __init__(self, w, device="cuda:0", num_splits: int | None = None, layout: str = "token_major",
                 max_context_len: int | None = None, fused_merge: bool = True,
                 fused_step: bool = False, window: int = 0, row_order="auto", rope_variants=None):
        self.w = w
        # prelude variants the single-launch step applies (rotary_dim, interleaved, q_norm_weight,
        # k_norm_weight, norm_eps); None = the plain rotation
        if isinstance(rope_variants, str) and rope_variants == "workload":
            # the options the workload itself names, norm weights moved to the device
            self.rope_variants = {
                k: (torch.from_numpy(np.ascontiguousarray(v).view(np.int16)).to(device) if isinstance(v, np.ndarray) else v)
                for k, v in w.extra.get("rope_variants", {}).items()}
        else:
            self.rope_variants = dict(rope_variants) if rope_variants else {}
        self.window = int(window) if window else int(getattr(w, "window", 0))   # > 0: sliding window
        self.fused_step = bool(fused_step)             # one launch: RoPE + append + attention + merge
        self.fused_merge = bool(fused_merge) or self.fused_step
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        ac.ac_init(self.device.index if self.device.index is not None else -1)
        self.B, self.Hq, self.Hkv, self.d, self.ps = w.B, w.Hq, w.Hkv, w.d, w.page_size
        self.num_pages = w.num_pages
        self.layout = layout
        kc, vc = w.k_cache, w.v_cache
        if layout == "head_major":
            kc = np.ascontiguousarray(kc.transpose(0, 2, 1, 3))
            vc = np.ascontiguousarray(vc.transpose(0, 2, 1, 3))
            self.stride_page = self.Hkv * self.ps * self.d
            self.stride_head = self.ps * self.d
            self.stride_token = self.d
        elif layout == "token_major":
            self.stride_page = self.ps * self.Hkv * self.d
            self.stride_token = self.Hkv * self.d
            self.stride_head = self.d
        else:
            raise ValueError(layout)
        self.k_cache = _dev_u16(kc, self.device)
        self.v_cache = _dev_u16(vc, self.device)
        self.q_in = _dev_u16(w.q, self.device)
        self.q_rot = self.q_in.clone()          # rows the kernel skips (inactive) keep their input
        self.k_new = _dev_u16(w.k_new, self.device)
        self.v_new = _dev_u16(w.v_new, self.device)
        self.block_table = torch.from_numpy(w.block_table).to(self.device)
        self.context_lens = torch.from_numpy(w.context_lens).to(self.device)
        self.rope_cos = torch.from_numpy(w.rope_cos).to(self.device)
        self.rope_sin = torch.from_numpy(w.rope_sin).to(self.device)
        # Scheduling hint: requests by decreasing length (what a scheduler that knows the lengths
        # hands over with the block table).  "auto": wherever the grid is more than one wave deep -- the
        # kernel would otherwise rank the requests itself in every CTA (up to 128 rows, ~1 us) or keep
        # index order (more rows); decided in set_splits, once the grid is known.
        self._row_order_auto = isinstance(row_order, str) and row_order == "auto"
        if self._row_order_auto:
            row_order = None
        self.row_order = None if row_order is None else torch.from_numpy(np.asarray(row_order, np.int32)).to(self.device)
        self.out = torch.zeros((self.B, self.Hq, self.d), dtype=torch.int16, device=self.device)
        self.status_flag = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.max_context_len = int(max_context_len) if max_context_len else w.max_context_len
        self.set_splits(num_splits)

    def set_splits(self, num_splits: int | None) -> None:
        span = self.max_context_len
        if self.window > 0:
            span = min(span, self.window + 63)         # tokens a row can attend over, as the kernel counts
        if num_splits is None:
            # the lengths are on the host (the scheduler built context_lens from them): plan with them
            counts = [min(int(n) + 1, span) if n >= 0 else 0 for n in self.w.context_lens]
            num_splits, _, _ = ac.ac_decode_plan_for_lengths(counts, self.Hq, self.Hkv, self.d, self.ps,
                                                             span, ac.ac_sm_count())
        self.num_splits = int(num_splits)
        self.split_tokens = ac.ac_split_tokens(span, self.num_splits)
        if self._row_order_auto:
            deep = self.B > 1 and self.B * self.Hkv * self.num_splits > 2 * (ac.ac_sm_count() or 148)
            order = np.argsort(-self.w.context_lens.astype(np.int64), kind="stable").astype(np.int32)
            self.row_order = torch.from_numpy(order).to(self.device) if deep else None
        # sized for either merge flavour: partials, then the fused path's arrival counters
        self.workspace_bytes = ac.ac_fused_workspace_bytes(self.B, self.Hq, self.Hkv, self.d,
                                                           self.num_splits)
        self.workspace = (torch.empty(max(self.workspace_bytes, 16) // 4, dtype=torch.float32,
                                      device=self.device))
        ac.ac_fused_workspace_reset(self.workspace, self.workspace_bytes, self.B, self.Hq, self.Hkv,
                                    self.d, self.num_splits)

    # -- the three calls -----------------------------------------------------------------------
    def rope_kv_append_ex(self, stream=None, rotary_dim=0, interleaved=False, q_norm_weight=None,
                          k_norm_weight=None, norm_eps=0.0) -> None:
        """Prelude variants; norm weights are device int16 tensors holding bf16 bits."""
        ac.ac_rope_kv_append_ex(self.q_in, self.q_rot, self.k_new, self.v_new, self.k_cache, self.v_cache,
                                self.stride_page, self.stride_token, self.stride_head, self.block_table,
                                self.w.max_pages_per_seq, self.context_lens, self.rope_cos, self.rope_sin,
                                self.w.max_position, self.B, self.Hq, self.Hkv, self.d, self.ps,
                                self.num_pages, self.status_flag, stream, rotary_dim=rotary_dim,
                                interleaved=interleaved, q_norm_weight=q_norm_weight,
                                k_norm_weight=k_norm_weight, norm_eps=norm_eps)

    def rope_kv_append(self, stream=None) -> None:
        ac.ac_rope_kv_append(self.q_in, self.q_rot, self.k_new, self.v_new, self.k_cache, self.v_cache,
                             self.stride_page, self.stride_token, self.stride_head, self.block_table,
                             self.w.max_pages_per_seq, self.context_lens, self.rope_cos, self.rope_sin,
                             self.w.max_position, self.B, self.Hq, self.Hkv, self.d, self.ps,
                             self.num_pages, self.status_flag, stream)

    def attention(self, stream=None, new_tokens: int = 1, q=None) -> None:
        if self.window > 0 or self.row_order is not None:
            ac.ac_paged_decode_attn_ex(self.q_rot if q is None else q, self.k_cache, self.v_cache,
                                       self.stride_page, self.stride_token, self.stride_head,
                                       self.block_table, self.w.max_pages_per_seq, self.context_lens,
                                       new_tokens, 0.0, self.num_splits,
                                       self.workspace if self.num_splits > 1 else None,
                                       self.workspace_bytes, self.out, self.B, self.Hq, self.Hkv, self.d,
                                       self.ps, self.num_pages, self.max_context_len, self.status_flag,
                                       stream, window=self.window, fused_merge=self.fused_merge,
                                       row_order=self.row_order)
            return
        fn = ac.ac_paged_decode_attn_fused_merge if self.fused_merge else ac.ac_paged_decode_attn
        fn(self.q_rot if q is None else q, self.k_cache, self.v_cache,
                                self.stride_page, self.stride_token, self.stride_head, self.block_table,
                                self.w.max_pages_per_seq, self.context_lens, new_tokens, 0.0,
                                self.num_splits, self.workspace if self.num_splits > 1 else None,
                                self.workspace_bytes, self.out, self.B, self.Hq, self.Hkv, self.d,
                                self.ps, self.num_pages, self.max_context_len, self.status_flag, stream)

    def merge(self, stream=None) -> None:
        if self.num_splits > 1 and not self.fused_merge:
            ac.ac_splitkv_merge(self.workspace, self.num_splits, self.context_lens, self.out, self.B,
                                self.Hq, self.d, stream)

    def decode_step_fused(self, stream=None, **rope_variants) -> None:
        """rope_variants: rotary_dim, interleaved, q_norm_weight, k_norm_weight, norm_eps (prelude
        variants applied inside the step; norm weights are device int16 tensors holding bf16 bits)."""
        ac.ac_decode_step_fused_ex(self.q_in, self.q_rot, self.k_new, self.v_new, self.k_cache,
                                   self.v_cache, self.stride_page, self.stride_token, self.stride_head,
                                   self.block_table, self.w.max_pages_per_seq, self.context_lens,
                                   self.rope_cos, self.rope_sin, self.w.max_position, 0.0, self.num_splits,
                                   self.workspace if self.num_splits > 1 else None, self.workspace_bytes,
                                   self.out, self.B, self.Hq, self.Hkv, self.d, self.ps, self.num_pages,
                                   self.max_context_len, self.status_flag, stream, window=self.window,
                                   row_order=self.row_order, **{**self.rope_variants, **rope_variants})

    def step(self, stream=None) -> None:
        if self.fused_step:
            self.decode_step_fused(stream)
            return
        self.rope_kv_append(stream)
        self.attention(stream)
        self.merge(stream)

    @property
    def launches_per_step(self) -> int:
        if self.fused_step:
            return 1
        return 3 if (self.num_splits > 1 and not self.fused_merge) else 2

    def capture(self) -> torch.cuda.CUDAGraph:
        """Record one step into a CUDA graph (one graph per batch-size bucket in a serving loop)."""
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.step(side)                      # warm-up outside capture
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            self.step(side)
        return graph

    # -- results -------------------------------------------------------------------------------
    def cache_bits(self):
        k, v = bits_of(self.k_cache), bits_of(self.v_cache)
        if self.layout == "head_major":
            k = k.reshape(self.num_pages, self.Hkv, self.ps, self.d).transpose(0, 2, 1, 3)
            v = v.reshape(self.num_pages, self.Hkv, self.ps, self.d).transpose(0, 2, 1, 3)
        return k, v

    def out_f64(self) -> np.ndarray:
        b = bits_of(self.out)
        return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)

    def partials(self):
        n = self.B * self.Hq * self.num_splits
        ws = self.workspace.detach().cpu().numpy()
        po = ws[:n * self.d].reshape(self.B, self.Hq, self.num_splits, self.d)
        pl = ws[n * self.d:n * self.d + n].reshape(self.B, self.Hq, self.num_splits)
        return po, pl


class AttentionBlockStep:
    """The attention block of one decoder layer for one decode step, as three launches in a row:
    QKV projection + RoPE + KV append, paged decode attention with the merge fused in, output
    projection + residual + RMSNorm.  ``hidden`` [B,H], ``w_qkv`` [(Hq+2Hkv)*d, H], ``w_o`` [H, Hq*d],
    ``norm_weight`` [H] are uint16 arrays of bf16 bits; ``hidden`` is both the projection's input and
    the residual stream."""

    def __init__(self, w, hidden, w_qkv, w_o, norm_weight, norm_eps=1e-5, device="cuda:0",
                 num_splits: int | None = None):
        self.step_ = DecodeStep(w, device=device, num_splits=num_splits, fused_merge=True)
        st = self.step_
        self.H = int(hidden.shape[1])
        self.norm_eps = float(norm_eps)
        self.hidden = _dev_u16(hidden, st.device)
        self.w_qkv = _dev_u16(w_qkv, st.device)
        self.w_o = _dev_u16(w_o, st.device)
        self.norm_weight = _dev_u16(norm_weight, st.device)
        self.residual_out = torch.empty_like(self.hidden)
        self.normed_out = torch.empty_like(self.hidden)

    def step(self, stream=None) -> None:
        st = self.step_
        ac.ac_qkv_rope_kv_append(self.hidden, self.w_qkv, self.H, st.q_rot, st.k_cache, st.v_cache,
                                 st.stride_page, st.stride_token, st.stride_head, st.block_table,
                                 st.w.max_pages_per_seq, st.context_lens, st.rope_cos, st.rope_sin,
                                 st.w.max_position, st.B, st.Hq, st.Hkv, st.d, st.ps, st.num_pages,
                                 st.status_flag, stream)
        st.attention(stream)
        ac.ac_oproj_residual_rmsnorm(st.out, self.w_o, st.Hq * st.d, self.H, self.hidden,
                                     self.residual_out, self.norm_weight, self.norm_eps, self.normed_out,
                                     st.B, stream)
