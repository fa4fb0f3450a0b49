#!/usr/bin/env python
"""Benchmark of the paged decode-attention step (RoPE + KV append -> split-KV attention -> merge).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of synthetic requests.  The headline
workload is ``long_context`` (the largest single-GPU configuration: 4 requests x 131072 cached
tokens, 2.1 GB of K/V read per step, far larger than L2, so no cache flush is needed between steps).
``value`` is achieved KV-read bandwidth = algorithmic K/V bytes of the step / device time per step,
with all inputs resident in HBM.  ``e2e`` is the same metric through ``ac_decode_step_host`` with the
step's inputs in pinned host memory and the result read back to the host inside the timed region.
The other workloads are reported under ``workloads``: us per call measured inside a captured CUDA
graph that chains calls over enough replicas of the workload that every call finds its K/V cold in
L2 (how a serving loop runs the kernels: one graph per batch-size bucket covering the whole step),
plus the time of a call that is its own graph launch with L2 flushed before it.  With N > 1 every rank runs an independent
replica on its own GPU (the path has no exchange step); value is the sum over ranks.

Timing: the block of K = ``--steps`` steps is repeated until about one second of device time has
been timed (``timed_blocks`` blocks, each between its own pair of CUDA events, no host
synchronisation in between) and the MEDIAN block is reported, so that the clock sampler sees the GPU
under sustained load even when K steps take a few milliseconds; ``us_x_sm_mhz`` = us per step x
median SM clock makes runs at different clocks comparable.

``--impl reference`` times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2606_07665_b200 import workloads as W  # noqa: E402

METRIC = "paged decode-attention KV-read bandwidth (us per call in ms_per_step)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0          # datasheet figure, for context only (the roofline uses the measured copy peak)
L2_FLUSH_BYTES = 512 << 20
# the five configurations the benchmark spec names (the serving sweep counts once per bucket)
BASELINE_CONFIGS = ("tiny", "single_request", "continuous_batching", "long_context") + tuple(
    f"graph_sweep_b{b}" for b in W.GRAPH_SWEEP_BATCHES)


# ---------------------------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------------------------

def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def ncu_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu summary (profiles/dram_traffic.json), or None."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            return json.load(f)[kernel][workload]["dram_bytes_per_launch"]
    except Exception:
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            try:
                power.append(float(parts[2]))
            except ValueError:
                pass
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        # "under load": samples taken while the board drew more than half of its highest reading
        busy = [c for c, w in zip(sm, power) if power and w >= 0.5 * max(power)] if len(power) == len(sm) else sm
        return {"sm_mhz": statistics.median(busy) if busy else (statistics.median(sm) if sm else None),
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "samples_under_load": len(busy),
                "power_w_max": max(power) if power else None, "reasons": sorted(reasons)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    return rank, local, world


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (reported baseline; also the --impl reference arm)
# ---------------------------------------------------------------------------------------------

def oracle_rows(w, budget_s: float = 1.5):
    """The oracle timed on workload ``w`` twice: BLAS limited to one thread, and as it stands (all the
    threads BLAS takes).  Each row: GB/s of K/V covered, threads, and what the sample was."""
    rows = []
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        threadpool_limits = None
    for label in ("1 thread", "all cores"):
        if label == "1 thread":
            if threadpool_limits is None:
                continue
            with threadpool_limits(limits=1):
                b, t, desc = oracle_sample_seconds(w, budget_s)
            threads = 1
        else:
            b, t, desc = oracle_sample_seconds(w, budget_s)
            threads = cpu_threads_used()
        rows.append({"threads": threads, "value": round(b / t / 1e9, 4), "unit": UNIT, "kind": "oracle",
                     "seconds": round(t, 3), "sample": desc})
    return rows


def oracle_sample_seconds(w, budget_s: float = 12.0):
    """Times the oracle on (request, KV head) pairs of ``w`` until about ``budget_s`` of CPU work.

    Each sampled pair runs the oracle's own routines on views restricted to that request and KV
    head: rotation + append of the new token, then attention of the group's query heads over all
    cached pages.  Returns (KV bytes covered, seconds, description).
    """
    from oracle import paged_decode_oracle as O
    G = w.Hq // w.Hkv
    pairs = [(b, h) for b in range(w.B) for h in range(w.Hkv) if w.context_lens[b] >= 0]
    rng = np.random.default_rng(0)
    rng.shuffle(pairs)
    t_total, bytes_total, n_done = 0.0, 0, 0
    for b, h in pairs:
        used = w.block_table[b, :(int(w.context_lens[b]) + w.page_size) // w.page_size]
        remap = np.arange(used.size, dtype=np.int32)[None, :]
        kc = w.k_cache[used][:, :, h:h + 1, :]           # the sample's own pages (copy = gather cost excluded)
        vc = w.v_cache[used][:, :, h:h + 1, :]
        t0 = time.perf_counter()
        q_rot, k_after, v_after = O.oracle_rope_kv_append(
            w.q[b:b + 1, h * G:(h + 1) * G], w.k_new[b:b + 1, h:h + 1], w.v_new[b:b + 1, h:h + 1], kc, vc,
            remap, w.context_lens[b:b + 1], w.rope_cos, w.rope_sin, w.page_size)
        O.oracle_paged_decode_attn(q_rot, k_after, v_after, remap, w.context_lens[b:b + 1], w.page_size)
        t_total += time.perf_counter() - t0
        bytes_total += (int(w.context_lens[b]) + 1) * w.d * 2 * 2
        n_done += 1
        if t_total >= budget_s:
            break
    desc = (f"{n_done} of {len(pairs)} (request, KV head) pairs of {w.name}: rotation+append and "
            f"attention of the {G} query heads of each pair, fp64 numpy")
    return bytes_total, t_total, desc


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def cpu_threads_used() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    w = W.NAMED[args.workload]()
    per_step_budget = max(1.0, min(15.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample_seconds(w, per_step_budget)
    tot_b, tot_t, desc = 0, 0.0, ""
    for _ in range(args.steps):
        b, t, desc = oracle_sample_seconds(w, per_step_budget)
        tot_b += b
        tot_t += t
    gbs = tot_b / tot_t / 1e9
    cores = cpu_threads_used()
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": w.kv_bytes / (gbs * 1e9) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "head_dim": w.d,
                   "page_size": w.page_size, "seed": w.seed,
                   "note": "ms_per_step is the sample's rate extrapolated to the whole step"},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                         "cpu_model": cpu_model(), "host_cores": len(os.sched_getaffinity(0))},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# replicas: the path has no exchange step, so N GPUs run N independent copies of the workload
# ---------------------------------------------------------------------------------------------

def max_over_ranks(values, world, device="cpu"):
    """Element-wise maximum of per-rank timings (every rank gets the result)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(kv_bytes_per_rank, ms_slowest_rank, world):
    """Whole-job GB/s: every rank moves kv_bytes_per_rank per step; the step ends with the slowest."""
    return world * kv_bytes_per_rank / (ms_slowest_rank * 1e-3) / 1e9


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------

TIMED_REGION_MS = 1000.0          # repeat the K-step block until about this much device time is timed


def blocks_for(ms_per_block: float, target_ms: float | None = None) -> int:
    target_ms = TIMED_REGION_MS if target_ms is None else target_ms
    return int(max(1, min(2000, -(-target_ms // max(ms_per_block, 1e-3)))))


def time_headline(st, steps, warmup, torch):
    """Blocks of K steps back to back, each block between its own pair of CUDA events on the launching
    stream, repeated until about a second has been timed; returns the median block.

    With the single-launch fused step the step IS the dominant kernel, so its average launch
    duration is the block time / K (no event is recorded between launches: an event node between
    two kernels would undo the programmatic overlap of their tail and ramp).  With separate launches
    an event pair around every attention launch gives that kernel's own duration.
    Returns (ms per step, ms per attention launch, number of blocks timed).
    """
    stream = torch.cuda.current_stream()
    w0 = torch.cuda.Event(enable_timing=True)
    w1 = torch.cuda.Event(enable_timing=True)
    w0.record(stream)
    for _ in range(warmup):
        st.step(stream)
    w1.record(stream)
    torch.cuda.synchronize()
    n_blocks = blocks_for(w0.elapsed_time(w1) / max(1, warmup) * steps)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_blocks + 1)]
    if st.fused_step:
        marks[0].record(stream)
        for blk in range(n_blocks):
            for _ in range(steps):
                st.decode_step_fused(stream)
            marks[blk + 1].record(stream)
        torch.cuda.synchronize()
        per_step = statistics.median(marks[i].elapsed_time(marks[i + 1]) for i in range(n_blocks)) / steps
        return per_step, per_step, n_blocks
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps * n_blocks)]
    marks[0].record(stream)
    for blk in range(n_blocks):
        for i in range(steps):
            st.rope_kv_append(stream)
            ev[blk * steps + i][0].record(stream)
            st.attention(stream)
            ev[blk * steps + i][1].record(stream)
            st.merge(stream)
        marks[blk + 1].record(stream)
    torch.cuda.synchronize()
    block_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(n_blocks)]
    mid = sorted(range(n_blocks), key=lambda i: block_ms[i])[n_blocks // 2]          # the median block
    attn_ms = [a.elapsed_time(b) for a, b in ev[mid * steps:(mid + 1) * steps]]
    return block_ms[mid] / steps, sum(attn_ms) / len(attn_ms), n_blocks


def time_e2e(st, steps, warmup, torch):
    from paper_2606_07665_b200 import binding as ac
    w = st.w

    def pinned(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else a).pin_memory()

    h_q, h_k, h_v = pinned(w.q), pinned(w.k_new), pinned(w.v_new)
    h_bt, h_len = pinned(w.block_table), pinned(w.context_lens)
    h_out = torch.empty((w.B, w.Hq, w.d), dtype=torch.int16).pin_memory()
    q_stage = torch.empty_like(st.q_in)
    stream = torch.cuda.current_stream()

    def one():
        ac.ac_decode_step_host(h_q, h_k, h_v, h_bt, h_len, h_out, q_stage, st.k_new, st.v_new,
                               st.block_table, st.context_lens, st.out, st.k_cache, st.v_cache,
                               st.stride_page, st.stride_token, st.stride_head, w.max_pages_per_seq,
                               st.rope_cos, st.rope_sin, w.max_position, 0.0, st.num_splits,
                               st.workspace if st.num_splits > 1 else None, st.workspace_bytes,
                               st.B, st.Hq, st.Hkv, st.d, st.ps, st.num_pages, st.max_context_len,
                               st.status_flag, stream)

    w0 = torch.cuda.Event(enable_timing=True)
    w1 = torch.cuda.Event(enable_timing=True)
    w0.record(stream)
    for _ in range(warmup):
        one()
    w1.record(stream)
    torch.cuda.synchronize()
    n_blocks = blocks_for(w0.elapsed_time(w1) / max(1, warmup) * steps, 0.3 * TIMED_REGION_MS)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_blocks + 1)]
    marks[0].record(stream)
    for blk in range(n_blocks):
        for _ in range(steps):
            one()
        marks[blk + 1].record(stream)
    torch.cuda.synchronize()
    h2d = sum(t.numel() * t.element_size() for t in (h_q, h_k, h_v, h_bt, h_len))
    d2h = h_out.numel() * h_out.element_size()
    ms = statistics.median(marks[i].elapsed_time(marks[i + 1]) for i in range(n_blocks)) / steps
    return ms, h2d, d2h


L2_BYTES = 126 << 20


def time_in_graph(make_step, kv_bytes, torch, replays=20):
    """GPU time of one call when it runs inside a larger captured graph (how a serving loop runs it).

    R replicas of the workload (separate device buffers, R x K/V bytes >= 4 x L2, so every call finds
    its K/V cold in L2) are stepped one after the other inside ONE captured graph; a chain of at
    least 8 calls even for workloads that exceed L2 on their own.  The graph is replayed `replays`
    times between one pair of events: us per call = elapsed / (replays x calls in the graph).
    Host launch overhead is paid once per replay, not once per call.
    """
    n_rep = max(1, min(40, -(-4 * L2_BYTES // kv_bytes)))
    steps = [make_step() for _ in range(n_rep)]
    rounds = max(1, -(-8 // n_rep))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for st in steps:
            st.step(side)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(rounds):
            for st in steps:
                st.step(side)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(replays):
        graph.replay()
    t1.record(stream)
    torch.cuda.synchronize()
    calls = replays * rounds * n_rep
    us = t0.elapsed_time(t1) * 1e3 / calls
    info = {"replicas": n_rep, "calls_per_graph": rounds * n_rep, "num_splits": steps[0].num_splits,
            "launches_per_call": steps[0].launches_per_step, "status_flag": int(steps[0].status_flag.item())}
    del graph, steps
    return us, info


def time_prelude_fusion(torch, device, batches=(1, 8, 32, 128, 256), replicas=12, replays=20):
    """Attention-prelude fusion (QKV projection + RoPE + KV append, one launch) on an 8B-class layer:
    hidden 4096, 32 query / 8 KV heads, head_dim 128 -> 6144 x 4096 bf16 weights (50.3 MB), streamed
    from HBM once per call.  `replicas` separate copies of the weights are cycled inside one captured
    graph so that every call finds them cold in L2.  Reports us per call and weight GB/s."""
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import runner
    H, Hq, Hkv, d, ps = 4096, 32, 8, 128, 16
    rows = []
    for B in batches:
        lens = np.random.default_rng(B).integers(100, 2000, size=B).tolist()
        w = W.make_workload("prelude", 70, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps, num_pages=B * 130 + 8,
                            context_lens=lens, rope_base=500000.0)
        x, wq = W.make_projection_inputs(71, B, H, Hq, Hkv, d)
        st = runner.DecodeStep(w, device=device)
        xs = [torch.from_numpy(x.view(np.int16)).to(device) for _ in range(replicas)]
        ws = [torch.from_numpy(wq.view(np.int16)).to(device) for _ in range(replicas)]

        def call(i, stream):
            ac.ac_qkv_rope_kv_append(xs[i], ws[i], H, st.q_rot, st.k_cache, st.v_cache, st.stride_page,
                                     st.stride_token, st.stride_head, st.block_table, w.max_pages_per_seq,
                                     st.context_lens, st.rope_cos, st.rope_sin, w.max_position, B, Hq, Hkv,
                                     d, ps, w.num_pages, st.status_flag, stream)

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(replicas):
                call(i, side)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(replicas):
                call(i, side)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(replays):
            graph.replay()
        t1.record()
        torch.cuda.synchronize()
        us = t0.elapsed_time(t1) * 1e3 / (replays * replicas)
        wbytes = wq.size * 2
        rows.append({"kernel": "ac_qkv_rope_kv_append", "B": B, "weight_mb": round(wbytes / 1e6, 1),
                     "us_per_call": round(us, 2), "weight_gbs": round(wbytes / us / 1e3, 1),
                     "status_flag": int(st.status_flag.item())})
        del graph
        if B <= 128:
            # the same launch with per-head Q/K RMSNorm folded into its epilogue (the CTAs of a head as a cluster)
            nw = torch.from_numpy(W.f32_to_bf16_bits(np.ones(d, dtype=np.float32)).view(np.int16)).to(device)

            def call_ex(i, stream):
                ac.ac_qkv_rope_kv_append_ex(xs[i], ws[i], H, st.q_rot, st.k_cache, st.v_cache, st.stride_page,
                                            st.stride_token, st.stride_head, st.block_table, w.max_pages_per_seq,
                                            st.context_lens, st.rope_cos, st.rope_sin, w.max_position, B, Hq,
                                            Hkv, d, ps, w.num_pages, st.status_flag, stream,
                                            q_norm_weight=nw, k_norm_weight=nw, norm_eps=1e-6)

            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for i in range(replicas):
                    call_ex(i, side)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(replicas):
                    call_ex(i, side)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            t0.record()
            for _ in range(replays):
                graph.replay()
            t1.record()
            torch.cuda.synchronize()
            us = t0.elapsed_time(t1) * 1e3 / (replays * replicas)
            rows.append({"kernel": "ac_qkv_rope_kv_append_ex (Q/K RMSNorm)", "B": B,
                         "weight_mb": round(wbytes / 1e6, 1), "us_per_call": round(us, 2),
                         "weight_gbs": round(wbytes / us / 1e3, 1), "status_flag": int(st.status_flag.item())})
            del graph
        del xs, ws

        # output projection + residual + RMSNorm on the same layer: W_o [4096, 4096] (33.6 MB)
        K, N = Hq * d, H
        rng = np.random.default_rng(72)
        wo = W.f32_to_bf16_bits((rng.standard_normal((N, K), dtype=np.float32) / np.float32(np.sqrt(K))))
        a = W.f32_to_bf16_bits(rng.standard_normal((B, K), dtype=np.float32) * np.float32(0.3))
        res = W.f32_to_bf16_bits(rng.standard_normal((B, N), dtype=np.float32))
        nw = W.f32_to_bf16_bits(np.ones(N, dtype=np.float32))
        dev = lambda t: torch.from_numpy(t.view(np.int16)).to(device)
        wos = [dev(wo) for _ in range(replicas)]
        a_d, r_d, n_d = dev(a), dev(res), dev(nw)
        h_d, y_d = torch.empty_like(r_d), torch.empty_like(r_d)

        def ocall(i, stream):
            ac.ac_oproj_residual_rmsnorm(a_d, wos[i], K, N, r_d, h_d, n_d, 1e-5, y_d, B, stream)

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(replicas):
                ocall(i, side)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(replicas):
                ocall(i, side)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        t0.record()
        for _ in range(replays):
            graph.replay()
        t1.record()
        torch.cuda.synchronize()
        us = t0.elapsed_time(t1) * 1e3 / (replays * replicas)
        rows.append({"kernel": "ac_oproj_residual_rmsnorm", "B": B, "weight_mb": round(wo.size * 2 / 1e6, 1),
                     "us_per_call": round(us, 2), "weight_gbs": round(wo.size * 2 / us / 1e3, 1)})
        del graph, wos, st
        torch.cuda.empty_cache()
    return rows


def time_attention_block(torch, device, batches=(1, 8, 32), replicas=8, replays=20):
    """The whole attention block of an 8B-class layer for one decode step -- QKV projection + RoPE +
    append, paged attention (contexts uniform in [512, 2048]), output projection + residual + RMSNorm
    -- as the chain of launches a serving graph would hold, cycled over `replicas` separate copies of
    weights and caches inside one captured graph (84 MB of weights + the K/V per copy, cold in L2)."""
    from paper_2606_07665_b200 import runner
    H, Hq, Hkv, d, ps = 4096, 32, 8, 128, 16
    rows = []
    for B in batches:
        lens = np.random.default_rng(100 + B).integers(512, 2049, size=B).tolist()
        w = W.make_workload("block", 73, B=B, Hq=Hq, Hkv=Hkv, d=d, page_size=ps, num_pages=B * 132 + 8,
                            context_lens=lens, rope_base=500000.0)
        hidden, wq = W.make_projection_inputs(74, B, H, Hq, Hkv, d)
        rng = np.random.default_rng(75)
        wo = W.f32_to_bf16_bits(rng.standard_normal((H, Hq * d), dtype=np.float32) / np.float32(np.sqrt(Hq * d)))
        nw = W.f32_to_bf16_bits(np.ones(H, dtype=np.float32))
        blocks = [runner.AttentionBlockStep(w, hidden, wq, wo, nw, 1e-5, device=device) for _ in range(replicas)]
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for blk in blocks:
                blk.step(side)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for blk in blocks:
                blk.step(side)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(replays):
            graph.replay()
        t1.record()
        torch.cuda.synchronize()
        us = t0.elapsed_time(t1) * 1e3 / (replays * replicas)
        moved = wq.size * 2 + wo.size * 2 + w.kv_bytes
        rows.append({"B": B, "us_per_block": round(us, 2), "bytes_mb": round(moved / 1e6, 1),
                     "gbs": round(moved / us / 1e3, 1), "num_splits": blocks[0].step_.num_splits,
                     "launches": 4, "status_flag": int(blocks[0].step_.status_flag.item())})
        del graph, blocks
        torch.cuda.empty_cache()
    return rows


def time_read_stream(torch, device, nbytes=4 << 30, reps=10):
    """GB/s of a plain coalesced read-only pass over a 4 GiB device buffer (the library's probe kernel,
    16-byte streaming loads, nothing written): best and median of `reps` passes after three warm-ups.
    Context for the roofline fractions, whose denominator is a copy (read + write) measurement."""
    from paper_2606_07665_b200 import binding as ac
    buf = torch.empty(nbytes // 4, dtype=torch.int32, device=device)
    buf.fill_(0x01010101)
    sink = torch.zeros(2, dtype=torch.int64, device=device)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        ac.ac_hbm_read_probe(buf, nbytes, sink, stream)
    torch.cuda.synchronize()
    times = []
    for _ in range(reps):
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ac.ac_hbm_read_probe(buf, nbytes, sink, stream)
        b.record(stream)
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    del buf
    torch.cuda.empty_cache()
    return {"best_gbs": round(nbytes / min(times) / 1e6, 1), "median_gbs": round(nbytes / statistics.median(times) / 1e6, 1),
            "bytes": nbytes, "kernel": "hbm_read_probe_kernel"}


def time_rope_variants(torch, device, batch=256, reps=50):
    """us per call of ac_rope_kv_append_ex with the prelude variants switched on (per-head Q/K RMSNorm,
    partial rotary, interleaved pairing) on a graph-sweep-shaped batch, one launch per event pair."""
    from paper_2606_07665_b200 import runner
    w = W.graph_sweep(batch)
    R = 64
    w.rope_cos, w.rope_sin = W.rope_table(w.max_position, R, w.rope_base)
    st = runner.DecodeStep(w, device=device, fused_merge=False)
    rng = np.random.default_rng(5)
    nw = torch.from_numpy(W.f32_to_bf16_bits((1 + 0.1 * rng.standard_normal(w.d)).astype(np.float32)).view(np.int16)).to(device)
    stream = torch.cuda.current_stream()
    rows = []
    for label, kw in (("qk_norm+partial_rotary_64+interleaved", dict(rotary_dim=R, interleaved=True, q_norm_weight=nw, k_norm_weight=nw, norm_eps=1e-6)),
                      ("partial_rotary_64", dict(rotary_dim=R))):
        for _ in range(3):
            st.rope_kv_append_ex(stream, **kw)
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            st.rope_kv_append_ex(stream, **kw)
            b.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b) * 1e3)
        rows.append({"kernel": "rope_kv_append_ex_kernel", "variant": label, "B": batch,
                     "us_per_call_own_launch": round(statistics.median(times), 2),
                     "status_flag": int(st.status_flag.item())})
    return rows


def time_model_variants(torch, device, peak):
    """The single-launch step with the prelude variants two of the paper's model families need, in-graph
    and K/V cold like the other workloads: a Qwen3-like layer (32 query / 8 KV heads, per-head Q/K
    RMSNorm) and a GLM-4-like one (32 query / 2 KV heads, rotary on 64 of 128 elements, interleaved
    pairs), batch 32, contexts uniform in [512, 2048]."""
    from paper_2606_07665_b200 import runner
    rows = []
    for name in ("qwen3_like_b32", "glm4_like_b32"):
        w = W.NAMED[name]()
        us, info = time_in_graph(lambda: runner.DecodeStep(w, device=device, fused_step=True, rope_variants="workload"),
                                 w.kv_bytes, torch)
        rows.append({"workload": name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "kv_mb": round(w.kv_bytes / 1e6, 1),
                     "variants": sorted(w.extra["rope_variants"]),
                     "num_splits": info["num_splits"], "us_per_call": round(us, 2),
                     "kv_gbs": round(w.kv_bytes / us / 1e3, 1),
                     "frac_of_hbm_peak": round(w.kv_bytes / us / 1e3 / peak, 4),
                     "entry_point": "ac_decode_step_fused_ex + ac_attn_options.rope",
                     "status_flag": info["status_flag"]})
    return rows


def time_warm_replays(st, torch, reps=50):
    """us per call when the same captured step is replayed back to back with nothing else touching the
    GPU: K/V of workloads that fit in L2 stay resident there (the warm figure next to the cold ones)."""
    graph = st.capture()
    for _ in range(5):
        graph.replay()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(reps):
        graph.replay()
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / reps


def time_kernels_alone(w, device, runner, torch, reps=10):
    """Median us of each kernel of the three-call path on its own (one event pair per launch, the
    launches of a kind back to back with a synchronise in between): ac_rope_kv_append,
    ac_paged_decode_attn (partials only) and ac_splitkv_merge."""
    st = runner.DecodeStep(w, device=device, fused_step=False, fused_merge=False)
    stream = torch.cuda.current_stream()
    out = {}
    for name, call in (("ac_rope_kv_append", st.rope_kv_append), ("ac_paged_decode_attn", st.attention),
                       ("ac_splitkv_merge", st.merge)):
        call()
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            call()
            b.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b) * 1e3)
        out[name + "_us"] = round(statistics.median(times), 2)
    out["num_splits"] = st.num_splits
    out["note"] = "each call timed alone between events, own launch (host launch path included)"
    del st
    return out


def time_single_graph_call(st, torch, reps=30):
    """us per call when every call is its own graph launch (host launch overhead included), L2
    flushed between calls: write a buffer 4x L2, then read it so its dirty lines are written back."""
    graph = st.capture()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    junk = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=st.device)
    sink = torch.zeros(1, dtype=torch.int64, device=st.device)
    times = []
    for i in range(reps):
        junk.fill_(i & 0xFF)
        sink += junk.view(torch.int64).sum()
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        graph.replay()
        b.record(stream)
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b) * 1e3)
    return statistics.median(times)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2606_07665_b200 import binding as ac
    from paper_2606_07665_b200 import build, runner

    rank, local, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    build.build()
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))
    ac.ac_init(local)
    peak, peak_kind = measured_peak()

    if args.rope_variants_only:
        if rank == 0:
            print(json.dumps({"rope_variants": time_rope_variants(torch, device, reps=5)}))
        return
    if args.prelude_only:
        if rank == 0:
            print(json.dumps({"prelude_fusion": time_prelude_fusion(torch, device, batches=(args.prelude_batch,),
                                                                   replicas=4,
                                                                   replays=3)}))
        return
    w = W.NAMED[args.workload]()
    st = runner.DecodeStep(w, device=device, fused_step=not args.three_launches,
                           fused_merge=not args.separate_merge)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    ms_step, ms_attn, timed_blocks = time_headline(st, args.steps, args.warmup, torch)
    barrier()
    ms_e2e, h2d, d2h = time_e2e(st, args.steps, args.warmup, torch)
    barrier()
    clocks = sampler.stop() if rank == 0 else None       # sampled over both timed regions
    flag = int(st.status_flag.item())
    launches_per_step = st.launches_per_step
    timed_num_splits = st.num_splits

    ms_step, ms_attn, ms_e2e = max_over_ranks([ms_step, ms_attn, ms_e2e], world, device)

    if rank == 0:
        kv = w.kv_bytes
        value = aggregate_throughput(kv, ms_step, world)
        e2e_value = aggregate_throughput(kv, ms_e2e, world)
        attn_gbs = kv / (ms_attn * 1e-3) / 1e9
        others = []
        if not args.only_headline:
            del st
            torch.cuda.empty_cache()
            for name in ("tiny", "single_request", "continuous_batching") + tuple(
                    f"graph_sweep_b{b}" for b in W.GRAPH_SWEEP_BATCHES) + ("gqa_group16",
                                                                            "sliding_window_4k"):
                ww = W.NAMED[name]()
                us, info = time_in_graph(lambda: runner.DecodeStep(ww, device=device, fused_step=not args.three_launches),
                                         ww.kv_bytes, torch)
                s2 = runner.DecodeStep(ww, device=device, fused_step=not args.three_launches)
                alone_us = time_single_graph_call(s2, torch)
                warm_us = time_warm_replays(s2, torch)
                others.append({
                    "workload": name, "B": ww.B, "kv_mb": round(ww.kv_bytes / 1e6, 3),
                    "num_splits": info["num_splits"], "us_per_call": round(us, 2),
                    "kv_gbs": round(ww.kv_bytes / us / 1e3, 1),
                    "frac_of_hbm_peak": round(ww.kv_bytes / us / 1e3 / peak, 4),
                    "frac_of_nominal_8000": round(ww.kv_bytes / us / 1e3 / NOMINAL_HBM_GBS, 4),
                    "how": (f"{info['calls_per_graph']} calls on {info['replicas']} replicas inside one "
                            "captured graph, K/V cold in L2 at every call"),
                    "us_per_call_own_graph_launch_l2_flushed": round(alone_us, 2),
                    "us_per_call_own_graph_launch_warm": round(warm_us, 2),
                    "fits_in_l2": bool(ww.kv_bytes < L2_BYTES),
                    "status_flag": info["status_flag"],
                    "cpu_baseline": oracle_rows(ww) if name in BASELINE_CONFIGS else None})
                del s2, ww
                torch.cuda.empty_cache()
            kernels_alone = time_kernels_alone(w, device, runner, torch)
            read_stream = time_read_stream(torch, device)
            rope_variants = time_rope_variants(torch, device)
            model_variants = time_model_variants(torch, device, peak)
            prelude = time_prelude_fusion(torch, device)
            for r in prelude:
                r["frac_of_hbm_peak"] = round(r["weight_gbs"] / peak, 4)
            block = time_attention_block(torch, device)
            for r in block:
                r["frac_of_hbm_peak"] = round(r["gbs"] / peak, 4)
            cpu_bytes, cpu_s, cpu_desc = oracle_sample_seconds(w, 12.0)
            cpu = {"value": cpu_bytes / cpu_s / 1e9, "unit": UNIT, "cores": cpu_threads_used(),
                   "kind": "oracle", "sample": cpu_desc, "cpu_model": cpu_model(),
                   "host_cores": len(os.sched_getaffinity(0)),
                   "rows": oracle_rows(w, 4.0)}
        else:
            cpu = None
            prelude = []
            block = []
            kernels_alone = None
            read_stream = None
            rope_variants = []
            model_variants = []
        sm_mhz = clocks.get("sm_mhz") if clocks else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "timed_blocks": timed_blocks,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "head_dim": w.d,
                       "page_size": w.page_size, "context_len": int(w.context_lens.max()),
                       "num_pages": w.num_pages, "seed": w.seed, "num_splits": timed_num_splits,
                       "kv_bytes_per_step": kv, "l2": "inputs larger than L2 (no flush)",
                       "timing": f"median of {timed_blocks} blocks of {args.steps} steps, ~{TIMED_REGION_MS / 1e3:.0f} s timed",
                       "launches_per_step": launches_per_step,
                       "entry_point": "ac_rope_kv_append + ac_paged_decode_attn_fused_merge"
                       if args.three_launches else "ac_decode_step_fused",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "us_per_call": ms_step * 1e3,
            "us_x_sm_mhz": ms_step * 1e3 * sm_mhz if sm_mhz else None,
            "frac_of_hbm_peak": value / world / peak,
            "frac_of_nominal_8000": value / world / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": attn_gbs, "peak": peak, "unit": "GB/s",
                         "frac": attn_gbs / peak, "peak_kind": peak_kind,
                         "kernel": "paged_decode_attn_kernel" + ("" if args.three_launches else " (fused step)"),
                         "traffic": ncu_traffic("paged_decode_attn_kernel", w.name),
                         "read_only_stream": read_stream,
                         "frac_of_read_only_stream": (attn_gbs / read_stream["best_gbs"]) if read_stream else None},
            "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
            "gpu_launches": args.steps * launches_per_step * timed_blocks,
            "clocks": clocks, "status_flag": flag, "workloads": others,
            "kernels_alone": kernels_alone, "prelude_fusion": prelude, "attention_block": block,
            "rope_variants": rope_variants, "model_variants": model_variants,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="long_context", choices=sorted(W.NAMED))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--three-launches", action="store_true",
                    help="time ac_rope_kv_append + ac_paged_decode_attn_fused_merge instead of the "
                         "single-launch ac_decode_step_fused")
    ap.add_argument("--separate-merge", action="store_true",
                    help="with --three-launches: use ac_paged_decode_attn + ac_splitkv_merge (three "
                         "kernels) instead of the merge fused into the attention kernel")
    ap.add_argument("--prelude-batch", type=int, default=8,
                    help="batch rows for --prelude-only (above 32 the tcgen05 projection kernel runs)")
    ap.add_argument("--prelude-only", action="store_true",
                    help="time only the projection fusions (ac_qkv_rope_kv_append, ac_oproj_residual_rmsnorm) "
                         "at batch 8 and print their rows; used for profiling those kernels")
    ap.add_argument("--rope-variants-only", action="store_true",
                    help="time only ac_rope_kv_append_ex with the prelude variants on (profiling that kernel)")
    ap.add_argument("--timed-ms", type=float, default=None,
                    help="device time to fill with repeated K-step blocks (default 1000; profiling runs pass a small value)")
    ap.add_argument("--only-headline", action="store_true",
                    help="skip the other workloads and the CPU baseline")
    args = ap.parse_args()
    if args.timed_ms is not None:
        global TIMED_REGION_MS
        TIMED_REGION_MS = max(0.0, args.timed_ms)
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 1000 if args.steps is None else args.steps
        args.warmup = 10 if args.warmup is None else max(3, args.warmup)
        run_ours(args)


if __name__ == "__main__":
    main()
