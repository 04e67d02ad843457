#!/usr/bin/env python
"""Benchmark of the paged decode attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--chunk C]
    python bench.py --impl reference ...      # times the fp64 CPU oracle instead

One "step" = kv_append -> paged_decode_attention (-> paged_decode_reduce) over
one synthetic decode batch, by default as the single fused launch
``paged_decode_step`` (``--path separate`` times the three calls). ``value`` is KV GB/s: algorithmic KV bytes of the
batch (every valid K and V element once) divided by the step time, inputs
resident in HBM. Prints ONE JSON line on rank 0. With N > 1 (torchrun) every
rank runs its own independent batch (sequences shard with no collective), the
step time is the max over ranks and the value sums the ranks' bytes.
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
# chunk_tokens each workload is timed with (longctx is fixed by its definition)
DEFAULT_CHUNK = {"tiny": 0, "llama8b": 0, "longctx": 2048, "chat70b": 0, "prefix_fp8": 0,
                 "scenario_c": 2048}
# shared prefix length of the workloads that have one (for --mode cascade)
PREFIX_TOKENS = {"prefix_fp8": 2048, "scenario_c": 32768}
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, from the ncu
# capture summarised under profiles/ (None: not captured for that workload)
NCU_TRAFFIC_BYTES = {"llama8b": 621_190_000}  # profiles/attention_tma_llama8b_ncu.md


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


def make(name, rank):
    from paper_2605_06068_b200.sharding import rank_seed
    seed = rank_seed(W.BASE_SEED + list(W.WORKLOADS).index(name), rank)
    return W.WORKLOADS[name](seed=seed)


def oracle_pass(w, n_threads=0):
    """One oracle evaluation of the whole batch; returns seconds."""
    import oracle
    k, v = w.k_cache, w.v_cache
    if w.kv_dtype == "bf16":
        k, v = k.copy(), v.copy()
        oracle.kv_append(w.k_new, w.v_new, k, v, w.block_table, w.seq_lens)
    t0 = time.perf_counter()
    oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale, w.k_scale,
                                  w.v_scale, n_threads=n_threads)
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = make(args.workload, 0)
    cores = oracle.hardware_threads()
    for _ in range(min(args.warmup, 1)):
        oracle_pass(w)
    times = [oracle_pass(w) for _ in range(args.steps)]
    t = float(np.mean(times))
    val = w.kv_bytes / t / 1e9
    sample = f"full {w.name} batch ({w.total_tokens} tokens), one fp64 pass per step"
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


def l2_note(w):
    """How the timed iterations stand to the 126 MB L2: the distinct KV bytes a step reads."""
    used = np.unique(w.block_table[w.block_table >= 0]).size
    elem = 1 if w.kv_dtype == "e4m3" else 2
    unique = 2 * used * w.num_kv_heads * w.page_size * w.head_dim * elem
    if unique > 126e6:
        return f"inputs larger than L2 (a step reads {unique / 1e6:.0f} MB of distinct KV; L2 is 126 MB)"
    return (f"working set fits in L2 ({unique / 1e6:.1f} MB of distinct KV) and is not flushed between "
            "iterations: a launch-latency figure, not a bandwidth figure")


def config_of(w, chunk, world):
    return {"workload": w.name, "batch_per_gpu": w.batch, "num_q_heads": w.num_q_heads,
            "num_kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "page_size": w.page_size,
            "kv_dtype": w.kv_dtype, "total_tokens_per_gpu": w.total_tokens,
            "kv_bytes_per_gpu": w.kv_bytes, "chunk_tokens": chunk,
            "l2": l2_note(w),
            "parallelism": f"dp{world} (independent batches, no collective)"}


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

    w = make(args.workload, rank)
    chunk = DEFAULT_CHUNK[w.name] if args.chunk is None else args.chunk
    if args.chunk is None and args.mode == "verify" and chunk:
        chunk *= 2   # a multi-query unit costs more to start than a decode unit: larger chunks (4096 for longctx)
    dev = torch.device("cuda", local)
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
    stream = torch.cuda.current_stream()
    fused = args.path == "fused"
    workspace = pda.new_workspace(w.batch, w.num_kv_heads, dev)
    flags = {"tma": 0, "generic": pda.PDA_FLAG_FORCE_GENERIC}[args.kernel]
    launches_per_step = 1 if fused else (1 if k_new is not None else 0) + 1 + (1 if chunk else 0)

    mode = args.mode
    if mode == "cascade":
        prefix = PREFIX_TOKENS[w.name]
        pchunk, schunk = args.prefix_chunk, (chunk or 256)
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

    # ---- device-resident timing -------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local))
    with sampler:
        t_start.record(stream)
        for i in range(args.steps):
            step(evs[i])
        t_end.record(stream)
        barrier()
    ms_step = t_start.elapsed_time(t_end) / args.steps
    ms_attn = float(np.mean([a.elapsed_time(b) for a, b in evs]))
    if int(status.item()) != 0:
        raise RuntimeError(f"device status {int(status.item())}: {pda.status_string(int(status.item()))}")

    # ---- the same step captured once in a CUDA graph and replayed (no host launch work) --------
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
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(args.steps):
            graph.replay()
        g1.record()
        barrier()
        ms_graph = g0.elapsed_time(g1) / args.steps

    # ---- end to end from pinned host buffers (bf16 workloads) --------------------------------
    e2e = None
    if k_new is not None and mode == "decode":
        pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
        hq, hk, hv, hbt, hsl = pin(w.q), pin(w.k_new), pin(w.v_new), pin(w.block_table), pin(w.seq_lens)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k_new), torch.empty_like(v_new)
        dbt, dsl = torch.empty_like(bt), torch.empty_like(sl)
        out_host = torch.empty(w.q.shape, dtype=torch.int16).pin_memory()

        def host_step(in_place):
            # in place: q, k_new, v_new are read from, and the result is written to, the pinned host
            # buffers by the kernel itself; staged: copied through device buffers around it
            st = (None, None, None) if in_place else (dq, dk, dv)
            pda.paged_decode_step_host(hq, hk, hv, hbt, hsl, st[0], st[1], st[2], dbt, dsl, k_cache, v_cache,
                                       float(w.scale), chunk, part_o, part_lse,
                                       None if in_place else out, out_host,
                                       workspace=workspace if fused else None, status=status, stream=stream)

        def time_host(in_place):
            for _ in range(max(args.warmup, 3)):
                host_step(in_place)
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                host_step(in_place)
                stream.synchronize()      # the caller reads the result before the next step
            e1.record(stream)
            barrier()
            return e0.elapsed_time(e1) / args.steps
        ms_e2e_staged = time_host(False)
        ms_e2e_in_place = time_host(True)
        # (split-KV launches re-read q once per chunk: over the bus that can cost more than one copy)
        ms_e2e = min(ms_e2e_in_place, ms_e2e_staged)
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hbt, hsl))
        d2h = out_host.numel() * out_host.element_size()
        e2e = (ms_e2e, h2d, d2h, ms_e2e_staged, ms_e2e_in_place)

    # ---- aggregate over ranks ----------------------------------------------------------------
    from paper_2605_06068_b200.sharding import aggregate
    (ms_step, ms_attn, ms_e2e, ms_graph), (kv_bytes_all, batch_all) = aggregate(
        [ms_step, ms_attn, e2e[0] if e2e else 0.0, ms_graph], [float(w.kv_bytes), float(w.batch)],
        device=dev)

    if rank == 0:
        peak, peak_kind = measured_peak()
        value = kv_bytes_all / (ms_step * 1e-3) / 1e9
        achieved = w.kv_bytes / (ms_attn * 1e-3) / 1e9      # per GPU, dominant kernel alone
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.kv_dtype == "bf16" else "e4m3",
            "data": "synthetic", "config": config_of(w, chunk, world),
            "tokens_per_s": batch_all / (ms_step * 1e-3),
            "path": f"{args.path}/{args.kernel}" if mode == "decode" else mode,
            "pct_of_nominal_hbm_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "attention_ms": ms_attn,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": NCU_TRAFFIC_BYTES.get(w.name),
                         "algorithmic_bytes": w.kv_bytes,
                         "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": sampler.summary(),
        }
        if ms_graph > 0:
            line["cuda_graph_replay"] = {"ms_per_step": ms_graph,
                                         "value": kv_bytes_all / (ms_graph * 1e-3) / 1e9, "unit": "GB/s"}
        if e2e:
            line["e2e"] = {"value": kv_bytes_all / (ms_e2e * 1e-3) / 1e9, "unit": "GB/s",
                           "ms_per_step": ms_e2e, "h2d_bytes_per_step": e2e[1],
                           "d2h_bytes_per_step": e2e[2],
                           "mode": ("in place: the kernel reads q, k_new, v_new from and writes out to pinned "
                                    "host memory over the bus; block_table and seq_lens are copied")
                                   if e2e[4] <= e2e[3] else "staged: inputs and result copied through device buffers",
                           "staged_ms_per_step": e2e[3], "in_place_ms_per_step": e2e[4]}
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            t = min(oracle_pass(w) for _ in range(2))
            line["cpu_baseline"] = {
                "value": w.kv_bytes / t / 1e9, "unit": "GB/s", "cores": oracle.hardware_threads(),
                "kind": "oracle", "tokens_per_s": w.batch / t,
                "sample": f"full {w.name} batch ({w.total_tokens} tokens), best of 2 fp64 passes"}
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
    ap.add_argument("--chunk", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    ap.add_argument("--mode", default="decode", choices=["decode", "cascade", "verify"],
                    help="cascade: paged_prefix_decode_attention on a shared-prefix workload; "
                         "verify: kv_append_tokens + paged_verify_attention with --verify-tokens queries")
    ap.add_argument("--prefix-chunk", type=int, default=512)
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
