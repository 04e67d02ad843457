#!/usr/bin/env python
"""Benchmark of the paged decode attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--also a,b] [--chunk C]
    python bench.py --impl reference ...      # times the fp64 CPU oracle instead

One "step" = kv_append -> paged_decode_attention (-> paged_decode_reduce) over
one synthetic decode batch, by default as the single fused launch
``paged_decode_step`` (``--path separate`` times the three calls). ``value`` is KV GB/s: algorithmic KV
bytes of the batch (every valid K and V element once) divided by the step time, inputs
resident in HBM. Timing protocol: W warm-up steps, then K steps, each preceded by an L2 flush (a 512 MB
buffer, four times the L2, is streamed through it by a read-only kernel outside the step's event pair,
which leaves the L2 full of clean lines of that buffer; overwriting the buffer instead leaves it full of
DIRTY lines whose write-back to HBM is then charged to the timed step -- ``--flush write`` times that,
and the headline record carries both figures) and timed by its own pair of CUDA events on the launching
stream; the step time is the MEDIAN of the K. The same K steps run back to back without
flushes are reported beside it. Prints ONE JSON line on rank 0: the headline workload (llama8b) at the
top level and, at one GPU, the other graded configurations under ``also``, each with its own clock
record and a parity flag from the oracle pass that is also its CPU baseline (a batch with a shared
prefix also carries the same step through the shared-prefix cascade, under ``cascade``). With N > 1 (torchrun) every
rank runs its own independent batch (sequences shard with no collective), the step time is the max over
ranks and the value sums the ranks' bytes.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_06068_b200 import workloads as W  # noqa: E402

METRIC = "paged decode attention KV GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 512 << 20          # four times the 126 MB L2
READ_PROBE_BYTES = 4 << 30          # the read-only streaming probe sums this many bytes per pass
# chunk_tokens each workload is timed with (longctx is fixed by its definition)
DEFAULT_CHUNK = {"tiny": 0, "llama8b": 0, "longctx": 2048, "chat70b": 0, "prefix_fp8": 0,
                 "scenario_c": 2048}
# shared prefix length of the workloads that have one (for --mode cascade)
PREFIX_TOKENS = {"prefix_fp8": 2048, "scenario_c": 32768}
# what runs beside the headline workload in the default invocation (one GPU)
DEFAULT_ALSO = ["longctx", "chat70b", "prefix_fp8"]
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel of the decode step,
# from the ncu captures summarised under profiles/ (None: not captured). Captures taken on a batch cut
# to about 1 GB are scaled to the full batch by the KV bytes (traffic grows with them).
NCU_TRAFFIC_BYTES = {
    "llama8b": 620_500_000,       # profiles/attention_tma_llama8b_ncu.md
    "longctx": 2_707_000_000,     # profiles/attention_tma_split_fused_longctx_ncu.md (2 of 8 sequences captured, x 4.576)
    "chat70b": 1_470_800_000,     # profiles/attention_persist_chat70b_ncu.md
    "prefix_fp8": 157_800_000,    # profiles/attention_tma_e4m3_prefix_fp8_ncu.md
}
TOL = {"bf16": (5e-3, 1e-2), "e4m3": (2e-2, 2e-2)}


def prefix_chunk_tokens(w, prefix, sms=148):
    """Chunk size for the cascade's prefix launch: its units are (128-row block of batch x group rows, kv
    head, chunk), each a CTA with a fixed cost of several microseconds, so: at most one CTA per SM, and
    chunks of at least 1024 tokens (measured: scenario_c 2048 -> 53.7 us per step, 512 -> 74 us, 4096 -> 66 us;
    prefix_fp8 1024 -> 66 us, 512 -> 70 us). Rounded up to a power of two."""
    rows = w.batch * (w.num_q_heads // w.num_kv_heads)
    per_chunk = -(-rows // 128) * w.num_kv_heads
    n_chunks = max(sms // per_chunk, 1)
    chunk = max(-(-prefix // n_chunks), 1024)
    return 1 << (chunk - 1).bit_length()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, index):
        self.index, self.samples, self.reasons = index, [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.002)   # several samples even inside a timed region of a few ms

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons)}


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def make(name, rank, batch=None):
    from paper_2605_06068_b200.sharding import rank_seed
    seed = rank_seed(W.BASE_SEED + list(W.WORKLOADS).index(name), rank)
    if batch and name != "tiny":
        return W.WORKLOADS[name](seed=seed, batch=batch)
    return W.WORKLOADS[name](seed=seed)


def oracle_pass(w, n_threads=0):
    """One oracle evaluation of the whole batch; returns (seconds, out fp64 [B,Hq,D])."""
    import oracle
    k, v = w.k_cache, w.v_cache
    if w.kv_dtype == "bf16":
        k, v = k.copy(), v.copy()
        oracle.kv_append(w.k_new, w.v_new, k, v, w.block_table, w.seq_lens)
    t0 = time.perf_counter()
    out, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale, w.k_scale,
                                           w.v_scale, n_threads=n_threads)
    return time.perf_counter() - t0, out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = make(args.workload, 0, args.batch)
    cores = oracle.hardware_threads()
    for _ in range(min(args.warmup, 1)):
        oracle_pass(w)
    times = [oracle_pass(w)[0] for _ in range(args.steps)]
    t = float(np.median(times))
    val = w.kv_bytes / t / 1e9
    sample = f"full {w.name} batch ({w.total_tokens} tokens), one fp64 pass per step, median of {args.steps}"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(w, 0, 1),
            "tokens_per_s": w.batch / t,
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def unique_kv_bytes(w):
    """Bytes of DISTINCT KV a pass touches: a page that several rows of the block table share (a common
    prefix) counts once. Equals ``w.kv_bytes`` when no page is shared."""
    P = w.page_size
    valid = {}
    for b in range(w.batch):
        L = int(max(w.seq_lens[b], 0))
        for i in range((L + P - 1) // P):
            pg = int(w.block_table[b, i])
            valid[pg] = max(valid.get(pg, 0), min(P, L - i * P))
    n = sum(valid.values()) * w.num_kv_heads * w.head_dim * 2 * w.elem_bytes
    if w.kv_dtype == "e4m3":
        n += len(valid) * w.num_kv_heads * 2 * 4
    return int(n)


FLUSH_NOTE = {"read": "streamed through the L2 by a read-only kernel, which leaves it holding clean lines of "
                      "that buffer",
              "write": "overwritten, which leaves the L2 full of dirty lines whose write-back overlaps the step",
              "none": "NOT done: steps run back to back"}


def config_of(w, chunk, world, flush="read"):
    unique = unique_kv_bytes(w)
    return {"workload": w.name, "batch_per_gpu": w.batch, "num_q_heads": w.num_q_heads,
            "num_kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "page_size": w.page_size,
            "kv_dtype": w.kv_dtype, "total_tokens_per_gpu": w.total_tokens,
            "kv_bytes_per_gpu": w.kv_bytes, "unique_kv_bytes_per_gpu": unique, "chunk_tokens": chunk,
            "l2": f"L2 flushed before every timed step ({L2_FLUSH_BYTES >> 20} MB {FLUSH_NOTE[flush]}, outside "
                  f"the step's event pair); a step reads {unique / 1e6:.0f} MB of distinct KV, L2 is 126 MB",
            "timing": "median of per-step CUDA-event pairs",
            "parallelism": f"dp{world} (independent batches, no collective)"}


def read_ceiling(dev, stream, reps=8):
    """GB/s of the library's read-only streaming probe over READ_PROBE_BYTES (best of ``reps`` passes;
    the buffer is 32 times the L2, so every pass comes from HBM)."""
    import torch
    from paper_2605_06068_b200 import binding as pda
    buf = torch.empty(READ_PROBE_BYTES // 4, dtype=torch.int32, device=dev)
    buf.fill_(1)
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    for _ in range(2):
        pda.debug_read_probe(buf, sink)
    best = float("inf")
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        pda.debug_read_probe(buf, sink)
        e1.record(stream)
        e1.synchronize()
        best = min(best, e0.elapsed_time(e1))
    del buf
    torch.cuda.empty_cache()
    return READ_PROBE_BYTES / (best * 1e-3) / 1e9


def run_workload(name, args, ctx, headline, mode=None):
    """Times one workload on this rank's GPU; returns the rank-0 record (None on other ranks)."""
    import torch
    import torch.distributed as dist
    from paper_2605_06068_b200 import binding as pda
    from paper_2605_06068_b200.sharding import aggregate

    world, rank, dev, stream = ctx["world"], ctx["rank"], ctx["dev"], ctx["stream"]
    w = make(name, rank, args.batch)
    chunk = DEFAULT_CHUNK[w.name] if args.chunk is None or not headline else args.chunk
    mode = mode or (args.mode if headline else "decode")
    if args.chunk is None and mode == "verify" and chunk:
        chunk *= 2   # a multi-query unit costs more to start than a decode unit: larger chunks (4096 for longctx)
    to16 = lambda a: torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    q = to16(w.q)
    if w.kv_dtype == "bf16":
        k_cache, v_cache, k_new, v_new = to16(w.k_cache), to16(w.v_cache), to16(w.k_new), to16(w.v_new)
        k_scale = v_scale = None
    else:
        k_cache, v_cache = torch.from_numpy(w.k_cache).to(dev), torch.from_numpy(w.v_cache).to(dev)
        k_scale, v_scale = torch.from_numpy(w.k_scale).to(dev), torch.from_numpy(w.v_scale).to(dev)
        k_new = v_new = None
    bt = torch.from_numpy(w.block_table).to(dev)
    sl = torch.from_numpy(w.seq_lens).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = torch.empty_like(q)
    part_o = part_lse = None
    if chunk:
        mc = pda.max_chunks(int(w.seq_lens.max()), chunk)
        part_o = torch.empty((w.batch, w.num_q_heads, mc, w.head_dim), dtype=torch.float32, device=dev)
        part_lse = torch.empty((w.batch, w.num_q_heads, mc), dtype=torch.float32, device=dev)
    fused = args.path == "fused"
    workspace = pda.new_workspace(w.batch, w.num_kv_heads, dev)
    flags = {"tma": 0, "generic": pda.PDA_FLAG_FORCE_GENERIC}[args.kernel]
    launches_per_step = 1 if fused else (1 if k_new is not None else 0) + 1 + (1 if chunk else 0)

    if mode == "cascade":
        prefix = PREFIX_TOKENS[w.name]
        # (suffix chunks of 512 tokens: prefix_fp8 59.7 us per step against 66.0 with 256 and 61.9 with 1024;
        # scenario_c's suffixes are shorter than either)
        pchunk, schunk = args.prefix_chunk or prefix_chunk_tokens(w, prefix), (chunk or 512)
        mc = (prefix + pchunk - 1) // pchunk + pda.max_chunks(int(w.seq_lens.max()) - prefix + 1, schunk)
        part_o = torch.empty((w.batch, w.num_q_heads, mc, w.head_dim), dtype=torch.float32, device=dev)
        part_lse = torch.empty((w.batch, w.num_q_heads, mc), dtype=torch.float32, device=dev)
        launches_per_step = 3 + (1 if k_new is not None else 0)
    if mode == "verify":
        T = args.verify_tokens
        g = torch.Generator(device=dev).manual_seed(1)
        vq = torch.randn((w.batch, T, w.num_q_heads, w.head_dim), generator=g, device=dev).to(torch.bfloat16)
        vk = torch.randn((w.batch, T, w.num_kv_heads, w.head_dim), generator=g, device=dev).to(torch.bfloat16)
        vv = torch.randn((w.batch, T, w.num_kv_heads, w.head_dim), generator=g, device=dev).to(torch.bfloat16)
        vout = torch.empty_like(vq)
        vpo = vpl = None
        if chunk:
            mc = pda.max_chunks(int(w.seq_lens.max()), chunk)
            vpo = torch.empty((w.batch, T, w.num_q_heads, mc, w.head_dim), dtype=torch.float32, device=dev)
            vpl = torch.empty((w.batch, T, w.num_q_heads, mc), dtype=torch.float32, device=dev)
        launches_per_step = 2 + (1 if chunk else 0)

    def step(ev=None):
        """One step; ``ev``: a pair of events recorded round the dominant launch."""
        if mode == "cascade":
            if k_new is not None:
                pda.kv_append(k_new, v_new, k_cache, v_cache, bt, sl, status=status)
            if ev:
                ev[0].record(stream)
            pda.paged_prefix_decode_attention(q, k_cache, v_cache, bt, sl, float(w.scale), prefix, pchunk,
                                              schunk, part_o, part_lse, out=out, k_scale=k_scale,
                                              v_scale=v_scale, status=status)
            if ev:
                ev[1].record(stream)
            return
        if mode == "verify":
            if w.kv_dtype == "bf16":
                pda.kv_append_tokens(vk, vv, k_cache, v_cache, bt, sl, status=status)
            else:
                pda.kv_append_tokens_fp8(vk, vv, k_cache, v_cache, k_scale, v_scale, bt, sl, status=status)
            if ev:
                ev[0].record(stream)
            pda.paged_verify_attention(vq, k_cache, v_cache, bt, sl, float(w.scale), chunk_tokens=chunk,
                                       out=vout, part_o=vpo, part_lse=vpl, k_scale=k_scale, v_scale=v_scale,
                                       status=status)
            if ev:
                ev[1].record(stream)
            return
        if fused:   # append + attention + reduce in one launch
            if ev:
                ev[0].record(stream)
            pda.paged_decode_step(q, k_new, v_new, k_cache, v_cache, bt, sl, float(w.scale),
                                  chunk_tokens=chunk, out=out, part_o=part_o, part_lse=part_lse,
                                  workspace=workspace, k_scale=k_scale, v_scale=v_scale, status=status)
            if ev:
                ev[1].record(stream)
            return
        if k_new is not None:
            pda.kv_append(k_new, v_new, k_cache, v_cache, bt, sl, status=status)
        if ev:
            ev[0].record(stream)
        pda.paged_decode_attention(q, k_cache, v_cache, bt, sl, float(w.scale), chunk_tokens=chunk,
                                   out=out, part_o=part_o, part_lse=part_lse, k_scale=k_scale,
                                   v_scale=v_scale, flags=flags, status=status)
        if ev:
            ev[1].record(stream)
        if chunk:
            pda.paged_decode_reduce(part_o, part_lse, sl, chunk, out=out)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    new_event = lambda: torch.cuda.Event(enable_timing=True)
    K = args.steps
    one_launch = fused and mode == "decode"    # the step IS the dominant launch: one event pair serves both
    flush_buf, flush_sink = ctx["flush_buf"], ctx["flush_sink"]

    def flush(i, how=None):
        how = how or args.flush
        if how == "read":
            pda.debug_read_probe(flush_buf, flush_sink)   # evicts the KV (and everything else) from L2
        elif how == "write":
            flush_buf.fill_(i)                            # the same, but leaves dirty lines behind

    # ---- device-resident timing: every step after an L2 flush, timed by its own event pair -------------
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    step_ev = [(new_event(), new_event()) for _ in range(K)]
    kern_ev = step_ev if one_launch else [(new_event(), new_event()) for _ in range(K)]
    sampler = ClockSampler(physical_gpu_index(ctx["local"]))
    with sampler:
        for i in range(K):
            flush(i)
            if one_launch:
                step(step_ev[i])
            else:
                step_ev[i][0].record(stream)
                step(kern_ev[i])
                step_ev[i][1].record(stream)
        barrier()
    step_times = [a.elapsed_time(b) for a, b in step_ev]
    kern_times = [a.elapsed_time(b) for a, b in kern_ev]
    ms_step, ms_attn = float(np.median(step_times)), float(np.median(kern_times))
    if int(status.item()) != 0:
        raise RuntimeError(f"device status {int(status.item())}: {pda.status_string(int(status.item()))}")

    # ---- the flushed step once more without per-step events: K x (flush + step) minus K x flush, one event
    # pair each. An event pair resolves about 2 us and puts a gap before the launch it brackets; the
    # difference of the two totals does neither (it is printed beside the median, not instead of it).
    ms_by_diff = None
    if args.flush != "none":
        def total(with_step):
            a, b = new_event(), new_event()
            barrier()
            a.record(stream)
            for i in range(K):
                flush(i)
                if with_step:
                    step()
            b.record(stream)
            barrier()
            return a.elapsed_time(b) / K
        ms_by_diff = total(True) - total(False)

    # ---- headline only: the other flush, for the record (median of K, same event placement) -------------
    ms_other_flush = None
    if headline and args.flush != "none":
        other = "write" if args.flush == "read" else "read"
        evs = [(new_event(), new_event()) for _ in range(K)]
        for i in range(K):
            flush(i, other)
            evs[i][0].record(stream)
            step()
            evs[i][1].record(stream)
        barrier()
        ms_other_flush = (other, float(np.median([a.elapsed_time(b) for a, b in evs])))

    # ---- the same K steps back to back, no flush (what a serving loop sees when nothing else runs) -------
    t_start, t_end = new_event(), new_event()
    barrier()
    t_start.record(stream)
    for _ in range(K):
        step()
    t_end.record(stream)
    barrier()
    ms_b2b = t_start.elapsed_time(t_end) / K
    if int(status.item()) != 0:
        raise RuntimeError(f"device status {int(status.item())}: {pda.status_string(int(status.item()))}")

    # ---- the same step captured once in a CUDA graph and replayed (no host launch work) ----------------
    ms_graph = 0.0
    if not args.no_graph:
        cap = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        cap.wait_stream(stream)
        with torch.cuda.stream(cap):
            with torch.cuda.graph(graph, stream=cap):
                step()   # the binding launches on the current stream, which is `cap` here
        barrier()
        for _ in range(3):
            graph.replay()
        barrier()
        g0, g1 = new_event(), new_event()
        g0.record()
        for _ in range(K):
            graph.replay()
        g1.record()
        barrier()
        ms_graph = g0.elapsed_time(g1) / K
        del graph

    gpu_out = (vout if mode == "verify" else out).float().cpu().numpy().astype(np.float64)

    # ---- end to end from pinned host buffers (bf16 workloads) ------------------------------------------
    e2e = None
    if k_new is not None and mode == "decode":
        pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
        hq, hk, hv, hbt, hsl = pin(w.q), pin(w.k_new), pin(w.v_new), pin(w.block_table), pin(w.seq_lens)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k_new), torch.empty_like(v_new)
        dbt, dsl = torch.empty_like(bt), torch.empty_like(sl)
        out_host = torch.empty(w.q.shape, dtype=torch.int16).pin_memory()

        def host_step(in_place):
            # in place (1): q, k_new, v_new are read from, and the result is written to, the pinned host
            # buffers by the kernel itself; (2): block_table and seq_lens too, so the step is one launch;
            # staged (0): everything copied through device buffers around the launch
            st = (None, None, None) if in_place else (dq, dk, dv)
            tb = (None, None) if in_place == 2 else (dbt, dsl)
            pda.paged_decode_step_host(hq, hk, hv, hbt, hsl, st[0], st[1], st[2], tb[0], tb[1], k_cache, v_cache,
                                       float(w.scale), chunk, part_o, part_lse,
                                       None if in_place else out, out_host,
                                       workspace=workspace if fused else None, status=status, stream=stream)

        def time_host(in_place):
            for _ in range(max(args.warmup, 3)):
                host_step(in_place)
            barrier()
            times = []
            for i in range(K):
                flush(i)
                e0, e1 = new_event(), new_event()
                e0.record(stream)
                host_step(in_place)
                e1.record(stream)
                e1.synchronize()          # the caller reads the result before the next step
                times.append(e0.elapsed_time(e1))
            barrier()
            return float(np.median(times))
        ms_modes = {"staged: inputs and result copied through device buffers": time_host(0),
                    "in place: the kernel reads q, k_new, v_new from and writes out to pinned host memory over "
                    "the bus; block_table and seq_lens are copied": time_host(1),
                    "all in place: the kernel also reads block_table and seq_lens from pinned host memory; the "
                    "step is one launch": time_host(2)}
        # (split-KV launches re-read q once per chunk: over the bus that can cost more than one copy)
        best_mode = min(ms_modes, key=ms_modes.get)
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hbt, hsl))
        d2h = out_host.numel() * out_host.element_size()
        e2e = (ms_modes[best_mode], h2d, d2h, best_mode, list(ms_modes.values()))

    # ---- aggregate over ranks --------------------------------------------------------------------------
    (ms_step, ms_attn, ms_e2e, ms_graph, ms_b2b), (kv_bytes_all, batch_all) = aggregate(
        [ms_step, ms_attn, e2e[0] if e2e else 0.0, ms_graph, ms_b2b], [float(w.kv_bytes), float(w.batch)],
        device=dev)
    del k_cache, v_cache, part_o, part_lse
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    peak, peak_kind = ctx["peak"]
    unique = unique_kv_bytes(w)
    shared = unique < 0.999 * w.kv_bytes          # pages shared between sequences: HBM sees them once
    hbm_bytes = unique if shared else w.kv_bytes
    value = kv_bytes_all / (ms_step * 1e-3) / 1e9
    achieved = hbm_bytes / (ms_attn * 1e-3) / 1e9      # per GPU, dominant kernel alone
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "traffic": NCU_TRAFFIC_BYTES.get(w.name) if mode == "decode" and not args.batch else None,
                "algorithmic_bytes": hbm_bytes,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}
    if shared:
        roofline["bytes_kind"] = ("distinct KV bytes (shared pages once): what must come from HBM after an "
                                  "L2 flush; the logical figure counts every sequence's reads")
        roofline["logical_gbs"] = w.kv_bytes / (ms_attn * 1e-3) / 1e9
        roofline["logical_bytes"] = w.kv_bytes
    if ctx.get("read_ceiling"):
        roofline["read_ceiling_gbs"] = ctx["read_ceiling"]
        roofline["frac_of_read_ceiling"] = achieved / ctx["read_ceiling"]
    rec = {
        "value": value, "unit": "GB/s", "ms_per_step": ms_step, "attention_ms": ms_attn,
        "back_to_back_ms_per_step": ms_b2b,
        "step_ms_min_max": [float(min(step_times)), float(max(step_times))],
        "config": config_of(w, chunk, world, args.flush),
        "tokens_per_s": batch_all / (ms_step * 1e-3),
        "path": f"{args.path}/{args.kernel}" if mode == "decode" else mode,
        "pct_of_nominal_hbm_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
        "roofline": roofline,
        "gpu_launches": launches_per_step * K,
        "clocks": sampler.summary(),
        "dtype": "bf16" if w.kv_dtype == "bf16" else "e4m3",
    }
    if ms_by_diff is not None:
        rec["ms_per_step_by_difference"] = ms_by_diff
    if ms_other_flush:
        rec["ms_per_step_after_" + ms_other_flush[0] + "_flush"] = ms_other_flush[1]
    if ms_graph > 0:
        rec["cuda_graph_replay"] = {"ms_per_step": ms_graph, "value": kv_bytes_all / (ms_graph * 1e-3) / 1e9,
                                    "unit": "GB/s", "note": "replays back to back, no flush"}
    if e2e:
        rec["e2e"] = {"value": kv_bytes_all / (ms_e2e * 1e-3) / 1e9, "unit": "GB/s",
                      "ms_per_step": ms_e2e, "h2d_bytes_per_step": e2e[1],
                      "d2h_bytes_per_step": e2e[2],
                      "mode": e2e[3], "staged_ms_per_step": e2e[4][0], "in_place_ms_per_step": e2e[4][1],
                      "all_in_place_ms_per_step": e2e[4][2]}
    if world == 1 and not args.no_cpu_baseline and mode in ("decode", "cascade"):  # (the cascade's result is the same)
        # The oracle as it stands, timed on the host cores on this very batch; its result is also what
        # the GPU output of the timed steps is checked against, element by element (no throughput is
        # reported for a workload that fails).
        import oracle
        passes = [oracle_pass(w) for _ in range(2 if headline else 1)]
        t, ref = min(p[0] for p in passes), passes[0][1]
        atol, rtol = TOL[w.kv_dtype]
        err = np.abs(gpu_out - ref)
        worst = float((err / (atol + rtol * np.abs(ref))).max())
        ok = bool(np.isfinite(gpu_out).all() and worst <= 1.0)
        rec["cpu_baseline"] = {
            "value": w.kv_bytes / t / 1e9, "unit": "GB/s", "cores": oracle.hardware_threads(),
            "kind": "oracle", "tokens_per_s": w.batch / t,
            "sample": f"full {w.name} batch ({w.total_tokens} tokens), best of {len(passes)} fp64 passes"}
        rec["parity"] = {"ok": ok, "max_err_over_tol": worst, "against": "the oracle pass timed as cpu_baseline",
                         "rule": f"|gpu - ref| <= {atol} + {rtol} |ref| on every output element"}
        if not ok:
            for key in ("value", "tokens_per_s", "pct_of_nominal_hbm_8TBs", "roofline", "e2e", "cuda_graph_replay"):
                rec[key] = None
    return rec


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2605_06068_b200 import binding as pda
    from paper_2605_06068_b200 import build as pda_build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        pda_build.build()
    if world > 1:
        dist.barrier()
    pda.lib()
    dev = torch.device("cuda", local)
    ctx = {"world": world, "rank": rank, "local": local, "dev": dev, "stream": torch.cuda.current_stream(),
           "peak": measured_peak(),
           "flush_buf": torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev),
           "flush_sink": torch.zeros(1, dtype=torch.int32, device=dev)}
    if not args.no_read_probe:
        ctx["read_ceiling"] = read_ceiling(dev, ctx["stream"])

    head = run_workload(args.workload, args, ctx, headline=True)
    also = {}
    names = DEFAULT_ALSO if args.also is None else [n for n in args.also.split(",") if n]
    if world == 1 and args.mode == "decode" and (args.also is not None or args.workload == "llama8b") \
            and not args.batch:
        for name in names:
            if name != args.workload:
                also[name] = run_workload(name, args, ctx, headline=False)
                if name in PREFIX_TOKENS and rank == 0:
                    # a batch with a shared prefix: the same step through paged_prefix_decode_attention (the
                    # prefix read once for the whole batch) beside the plain decode step
                    c = run_workload(name, args, ctx, headline=False, mode="cascade")
                    also[name]["cascade"] = {k: c[k] for k in ("ms_per_step", "attention_ms", "back_to_back_ms_per_step",
                                                               "value", "clocks", "parity", "gpu_launches") if k in c}
    if rank == 0:
        if head.get("parity") and not head["parity"]["ok"]:
            raise RuntimeError(f"parity check failed on {args.workload}: {head['parity']}")
        line = {"metric": METRIC, "value": head.pop("value"), "unit": head.pop("unit"), "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": head.pop("ms_per_step"),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": head.pop("dtype"),
                "data": "synthetic"}
        line.update(head)
        if also:
            line["also"] = also
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b", choices=list(W.WORKLOADS))
    ap.add_argument("--also", default=None,
                    help="comma-separated workloads timed after the headline one and reported under \"also\" "
                         "(default with llama8b at one GPU: longctx,chat70b,prefix_fp8; \"\" for none)")
    ap.add_argument("--batch", type=int, default=None,
                    help="cut (or grow) the workload's batch, e.g. for a profiler capture of about 1 GB")
    ap.add_argument("--chunk", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    ap.add_argument("--no-read-probe", action="store_true", help="skip the read-only streaming probe")
    ap.add_argument("--flush", default="read", choices=["read", "write", "none"],
                    help="L2 flush before every timed step: a 512 MB buffer read (leaves clean lines), "
                         "overwritten (leaves dirty lines: their write-back then overlaps the step), or none")
    ap.add_argument("--mode", default="decode", choices=["decode", "cascade", "verify"],
                    help="cascade: paged_prefix_decode_attention on a shared-prefix workload; "
                         "verify: kv_append_tokens + paged_verify_attention with --verify-tokens queries")
    ap.add_argument("--prefix-chunk", type=int, default=None,
                    help="cascade: tokens per prefix chunk (default: prefix_chunk_tokens())")
    ap.add_argument("--verify-tokens", type=int, default=16)
    ap.add_argument("--path", default="fused", choices=["fused", "separate"],
                    help="fused: one paged_decode_step launch; separate: kv_append, attention, reduce")
    ap.add_argument("--kernel", default="tma", choices=["tma", "generic"],
                    help="attention kernel of the separate path")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
