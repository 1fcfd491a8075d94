#!/usr/bin/env python
"""Benchmark of the paged decode-attention hot path (plan -> run -> combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path over one batch: the split-KV partial
kernel and the LSE combine kernel (launched with a programmatic dependency on
it; --fuse merges inside the partial kernel instead) over every sequence of
the workload.  The default workload is the single long sequence
(batch 1, 32 query / 8 KV heads, head_dim 128, page 16, 32,768 tokens); the
metric is KV-read GB/s = logical K+V bytes of the batch / time per step.

Timing: CUDA events on the launching stream around exactly K steps (replayed
as CUDA graphs of up to 256 steps each so host launch cost stays out of a
20-microsecond step), after W warm-up steps, with a barrier and a device
synchronise on both sides, maximum over ranks.  Successive steps read
different physical copies of the pools (distinct memory, differently shuffled
block tables) that together exceed 1 GiB, so no step finds its K/V in L2.
SM clocks and throttle reasons are sampled through NVML during the timed
region.  With --gpus N (launched by torchrun, one rank per GPU) every rank
runs its own sequences; nothing is exchanged (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode-attn KV-read GB/s"
UNIT = "GB/s"
GRAPH_STEPS = 256
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the partial kernel, from the
# ncu capture summarised under profiles/ (null until a capture of that workload exists).
NCU_TRAFFIC_BYTES = {
    "long_32k": 134_300_000 + 3_362_000,          # profiles/decode_attn_mma_kernel_long_32k.md
    "sweep_8192x64": 2_148_308_000 + 4_320_000,   # profiles/decode_attn_mma_kernel_sweep_8192x64.md
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8192)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="long_32k",
                    help="long_32k | short_chat | shared_prefix | sweep_<context>x<batch> | tiny")
    ap.add_argument("--split", default="auto", choices=["auto", "deterministic"])
    ap.add_argument("--chunk-tokens", type=int, default=0)
    ap.add_argument("--max-splits", type=int, default=0, help="most splits of one sequence (0: the library default)")
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "mma", "umma"])
    ap.add_argument("--fuse", action="store_true",
                    help="merge inside the partial kernel (one launch per step) instead of the combine kernel")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host")
    ap.add_argument("--partial-only", action="store_true",
                    help="diagnostic: time the partial kernel alone (results are not merged)")
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--skip-cpu", action="store_true", help="leave out the cpu_baseline leg")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--probe", action="store_true", help="also time the gather-only probe")
    ap.add_argument("--copies", type=int, default=0, help="pool copies to rotate over (0: enough for 1 GiB)")
    ap.add_argument("--alias-after", type=int, default=0,
                    help="sweep cells too large for memory: sequences i >= K reuse the pages of sequence i mod K")
    ap.add_argument("--in-dtype", default="bf16", choices=["bf16", "fp16"], help="type of q, K and V")
    ap.add_argument("--page-size", type=int, default=16, choices=[16, 32, 64, 128, 256], help="tokens per KV page")
    ap.add_argument("--q-heads", type=int, default=32, choices=[8, 16, 24, 32, 40, 48, 56, 64, 72, 96, 128],
                    help="query heads over the 8 KV heads of a sweep cell (groups of 1 to 16)")
    ap.add_argument("--prefix-aware", action="store_true",
                    help="shared_prefix workload: tell the planner about the common prefix (attended once per block of sequences)")
    ap.add_argument("--mask-fraction", type=float, default=None,
                    help="RUN mask (Alg. 1 step 2): this fraction of the rows, picked by a seeded hash, reads no KV")
    return ap.parse_args()


IN_DTYPE = "bf16"     # set from --in-dtype
PAGE_SIZE = 16        # set from --page-size
Q_HEADS = 32          # set from --q-heads (sweep cells)


def make_workload(name, device, table_seed=None, seed_shift=0, alias_after=None):
    from paper_2609_37062_b200 import workloads as wl
    w = _make_workload_bf16(name, device, table_seed, seed_shift, alias_after)
    return wl.as_fp16(w) if IN_DTYPE == "fp16" else w


def _make_workload_bf16(name, device, table_seed=None, seed_shift=0, alias_after=None):
    from paper_2609_37062_b200 import workloads as wl
    if name == "tiny":
        return wl.config_tiny(device=device)
    if name == "long_32k":
        return wl.config_long(device=device, seed=1 + seed_shift, table_seed=table_seed, page_size=PAGE_SIZE)
    if name == "short_chat":
        return wl.config_short_chat(device=device, seed=2 + seed_shift, table_seed=table_seed, page_size=PAGE_SIZE)
    if name == "shared_prefix":
        return wl.config_shared_prefix(device=device, seed=3 + seed_shift, table_seed=table_seed,
                                       page_size=PAGE_SIZE)
    if name.startswith("sweep_"):
        ctx, batch = name[len("sweep_"):].split("x")
        return wl.config_sweep_cell(int(ctx), int(batch), device=device, seed=4 + seed_shift, table_seed=table_seed,
                                    alias_after=alias_after, page_size=PAGE_SIZE, num_q_heads=Q_HEADS)
    raise SystemExit(f"unknown workload {name}")


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Reads SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
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

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80, "sync_boost": 0x10, "applications_clocks_setting": 0x2}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.nv:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def time_oracle(w_host, budget_s=12.0):
    """The fp64 CPU oracle as it stands, on this machine's cores, over the whole batch."""
    import oracle
    inp = oracle.PagedInputs.from_workload(w_host)
    t0 = time.perf_counter()
    oracle.paged_decode_attention(inp)
    first = time.perf_counter() - t0
    reps, total = 1, first
    while total < budget_s and reps < 50:
        t0 = time.perf_counter()
        oracle.paged_decode_attention(inp)
        total += time.perf_counter() - t0
        reps += 1
    return total / reps, reps, oracle.max_threads()


def oracle_sample(name):
    """A bounded sample of the workload for the CPU leg: whole batch when small, else a few sequences."""
    import dataclasses
    from paper_2609_37062_b200 import workloads as wl
    w = make_workload(name, "cpu") if not name.startswith("sweep_") else None
    if w is not None and w.logical_tokens <= 600_000:
        return w, "whole batch", 1.0
    if w is None:
        ctx, batch = (int(x) for x in name[len("sweep_"):].split("x"))
        keep = min(batch, max(1, 262144 // ctx))
        w = wl.config_sweep_cell(ctx, keep, num_q_heads=Q_HEADS)
        return w, f"{keep} of {batch} sequences, extrapolated per token", 1.0
    return w, "whole batch", 1.0


def run_reference(args):
    """The oracle as it stands on this machine's cores: W warm-up and exactly K timed steps, each step a
    bounded sample of the workload sized so that the whole run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2609_37062_b200 import workloads as wl
    w, sample, _ = oracle_sample(args.workload)
    inp = oracle.PagedInputs.from_workload(w)
    t0 = time.perf_counter()
    oracle.paged_decode_attention(inp)
    t_full = time.perf_counter() - t0
    budget_s = 150.0
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    if (steps + warmup) * t_full > budget_s:
        frac = budget_s / ((steps + warmup) * t_full)
        if w.batch > 1:
            keep = max(1, int(w.batch * frac))
            lens = [int(x) for x in w.seq_lens[:keep]]
            sample = f"{keep} of {w.batch} sequences per step"
        else:
            per = max(16, int(int(w.seq_lens[0]) * frac) // 16 * 16)
            lens = [per]
            sample = f"the first {per} of {int(w.seq_lens[0])} tokens per step"
        w = wl.make_workload(w.name, lens, w.num_q_heads, w.num_kv_heads, w.head_dim, seed=7)
        inp = oracle.PagedInputs.from_workload(w)
    for _ in range(warmup):
        oracle.paged_decode_attention(inp)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.paged_decode_attention(inp)
    dt = (time.perf_counter() - t0) / steps
    gbs = w.logical_kv_bytes / dt / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": sample, "tokens": w.logical_tokens},
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    args = parse_args()
    global IN_DTYPE, PAGE_SIZE, Q_HEADS
    IN_DTYPE = args.in_dtype
    PAGE_SIZE = args.page_size
    Q_HEADS = args.q_heads
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2609_37062_b200 import binding as da

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode-attention path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs: R physical copies of the workload, this rank's own sequences
    alias = args.alias_after or None
    first = make_workload(args.workload, dev, table_seed=1000 * rank, seed_shift=100 * rank, alias_after=alias)
    kv_bytes = first.logical_kv_bytes
    unique_bytes = first.unique_kv_bytes
    copies = args.copies or max(2, -(-(1 << 30) // max(unique_bytes, 1)) + 1)
    copies = min(copies, 64)
    pools = [first]
    for i in range(1, copies):
        pools.append(make_workload(args.workload, dev, table_seed=1000 * rank + i, seed_shift=100 * rank, alias_after=alias))

    kernel = {"auto": da.DA_KERNEL_AUTO, "simt": da.DA_KERNEL_SIMT, "mma": da.DA_KERNEL_MMA_TMA,
              "umma": da.DA_KERNEL_UMMA_PREFIX}[args.kernel]
    policy = da.make_policy(
        split_mode=da.DA_SPLIT_DETERMINISTIC if args.split == "deterministic" else da.DA_SPLIT_AUTO,
        chunk_tokens=args.chunk_tokens, max_splits=args.max_splits, kernel=kernel, fuse_combine=1 if args.fuse else 0,
        ctas_per_sm=args.ctas_per_sm,
        shared_prefix_tokens=first.shared_prefix_tokens if args.prefix_aware else 0)
    shape = da.shape_of_workload(first)
    lens_host = first.seq_lens.cpu().numpy()            # the planner takes the lengths from host memory
    t0 = time.perf_counter()
    plan = da.decode_attn_plan(shape, policy, lens_host)
    plan_us = (time.perf_counter() - t0) * 1e6
    info = plan.info()
    t0 = time.perf_counter()
    for _ in range(50):                      # steady state: buffers come from the library's cache
        da.decode_attn_plan(shape, policy, lens_host).destroy()
    replan_us = (time.perf_counter() - t0) * 1e6 / 50
    out = torch.empty((first.batch, first.num_q_heads, first.head_dim), dtype=torch.float32, device=dev)
    lse = torch.empty((first.batch, first.num_q_heads), dtype=torch.float32, device=dev)
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=dev)
    launches_per_step = 1 if (policy.fuse_combine or info.n_slots == 0) else 2
    if info.kernel == da.DA_KERNEL_UMMA_PREFIX:
        launches_per_step += 1      # the tcgen05 prefix kernel, then the kernel for what follows the prefix

    run_mask = None
    masked_bytes = 0
    if args.mask_fraction is not None:
        g = torch.Generator().manual_seed(12345)
        n_mask = int(round(args.mask_fraction * first.batch))
        keep = torch.ones(first.batch, dtype=torch.uint8)
        keep[torch.randperm(first.batch, generator=g)[:n_mask]] = 0
        run_mask = keep.to(dev)
        masked_bytes = int((first.seq_lens.cpu().long() * (1 - keep.long())).sum().item()) * first.kv_bytes_per_token

    def step(i, combine=True):
        w = pools[i % copies]
        da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws,
                           plan.workspace_bytes, run_mask=run_mask)
        if combine and not policy.fuse_combine and not args.partial_only:
            da.decode_attn_combine(plan, ws, out, lse)

    def make_runner(n_steps, first_index, combine=True):
        """n_steps consecutive steps starting at rotation index first_index, as one callable."""
        if args.no_graph:
            return lambda: [step(first_index + j, combine) for j in range(n_steps)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for j in range(n_steps):
                step(first_index + j, combine)
        return g.replay

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for i in range(max(args.warmup, 3)):
            step(i)
        stream.synchronize()
        st = da.decode_attn_last_device_status(plan)
        if st != da.DA_OK:
            raise SystemExit(f"device status after warm-up: {da.decode_attn_strerror(st)}")
        chunk = min(GRAPH_STEPS, args.steps)
        full, rem = divmod(args.steps, chunk)
        run_chunk = make_runner(chunk, 0)
        run_rem = make_runner(rem, 0) if rem else None
        run_chunk()                      # graph warm-up (uploads the graph), untimed
        stream.synchronize()

        sampler = ClockSampler(physical_gpu_index(local_rank))
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sampler.start()
        ev0.record(stream)
        for _ in range(full):
            run_chunk()
        if run_rem:
            run_rem()
        ev1.record(stream)
        stream.synchronize()
        clocks = sampler.stop()
        barrier()
        ms = ev0.elapsed_time(ev1)
        st = da.decode_attn_last_device_status(plan, stream)
        if st != da.DA_OK:
            raise SystemExit(f"device status after the timed region: {da.decode_attn_strerror(st)}")

        # the dominant kernel by itself: the same replays without the combine launch
        kernel_only_us = None
        if not policy.fuse_combine and not args.partial_only and info.n_slots > 0:
            n_ko = min(chunk, 2048)
            run_ko = make_runner(n_ko, 0, combine=False)
            run_ko()
            stream.synchronize()
            k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            k0.record(stream)
            run_ko()
            k1.record(stream)
            stream.synchronize()
            kernel_only_us = k0.elapsed_time(k1) * 1e3 / n_ko

        probe_us = None
        if args.probe and info.kernel == da.DA_KERNEL_MMA_TMA:
            chk = torch.empty(int(info.n_units), dtype=torch.int32, device=dev)
            for i in range(3):
                w = pools[i % copies]
                da.decode_attn_gather_probe(plan, w.k_pool, w.v_pool, w.block_table, chk)
            n_probe = min(args.steps, 512)
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            p0.record(stream)
            for i in range(n_probe):
                w = pools[i % copies]
                da.decode_attn_gather_probe(plan, w.k_pool, w.v_pool, w.block_table, chk)
            p1.record(stream)
            stream.synchronize()
            probe_us = p0.elapsed_time(p1) * 1e3 / n_probe

    from paper_2609_37062_b200 import sharding
    ms = sharding.max_over_ranks(ms, dev)
    sec_per_step = ms * 1e-3 / args.steps
    value = world * kv_bytes / sec_per_step / 1e9

    # ---- end to end from host buffers through the C ABI (copies inside the timed region)
    e2e = None
    e2e_resident = None
    if not args.skip_e2e:
        hw = make_workload(args.workload, "cpu", table_seed=1000 * rank, seed_shift=100 * rank)
        pin = lambda t: t.contiguous().pin_memory()
        hq, hk, hv, hbt, hsl = pin(hw.q_bits), pin(hw.k_pool), pin(hw.v_pool), pin(hw.block_table), pin(hw.seq_lens)
        hout = torch.empty((hw.batch, hw.num_q_heads, hw.head_dim), dtype=torch.float32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hbt, hsl))
        d2h = hout.numel() * 4
        n_e2e = max(3, min(args.steps, int(2.0 / max(h2d / 20e9, 1e-4))))
        for _ in range(2):
            da.decode_attn_host_step(shape, policy, hq, hk, hv, hbt, hsl, hout)
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            da.decode_attn_host_step(shape, policy, hq, hk, hv, hbt, hsl, hout)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = sharding.max_over_ranks(dt, dev)
        e2e = {"value": world * kv_bytes * n_e2e / dt / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": dt / n_e2e * 1e3,
               "what": "decode_attn_host_step: q, both pools, block table and lengths copied from pinned host "
                       "memory, plan, run, merge, out copied back, every step"}
        da.decode_attn_host_release()
        # the same with the pools resident (what a serving engine does): only q, table, lengths move
        w0 = pools[0]
        n_res = min(args.steps, 2000)
        with torch.cuda.stream(stream):
            def resident_step():
                w0.q_bits.copy_(hq, non_blocking=True)
                w0.block_table.copy_(hbt, non_blocking=True)
                w0.seq_lens.copy_(hsl, non_blocking=True)
                pl = da.decode_attn_plan(shape, policy, hsl)
                da.decode_attn_run(pl, w0.q_bits, w0.k_pool, w0.v_pool, w0.block_table, w0.seq_lens, out, lse, ws,
                                   plan.workspace_bytes)
                if not policy.fuse_combine:
                    da.decode_attn_combine(pl, ws, out, lse)
                hout.copy_(out, non_blocking=True)
                stream.synchronize()
                pl.destroy()
            for _ in range(3):
                resident_step()
            barrier()
            t0 = time.perf_counter()
            for _ in range(n_res):
                resident_step()
            dt = time.perf_counter() - t0
        e2e_resident = {"value": world * kv_bytes * n_res / dt / 1e9, "unit": UNIT,
                        "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in (hq, hbt, hsl)),
                        "d2h_bytes_per_step": d2h, "steps": n_res, "ms_per_step": dt / n_res * 1e3,
                        "what": "pools resident in HBM; q, block table, lengths from pinned host memory, plan, run, "
                                "merge, out back to host, synchronised every step"}

    # ---- the oracle on this machine's cores (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        w_cpu, sample, _ = oracle_sample(args.workload)
        sec, reps, cores = time_oracle(w_cpu)
        cpu = {"value": w_cpu.logical_kv_bytes / sec / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"{sample}; {w_cpu.logical_tokens} tokens, {reps} runs, {sec * 1e3:.1f} ms each"}

    if rank == 0:
        peak, peak_kind = peak_hbm()
        # With a shared-prefix plan a prefix page is fetched once for the whole batch: the bytes the
        # step has to move are the unique ones.
        prefix_plan = int(policy.shared_prefix_tokens) > 0
        algo_bytes = unique_bytes if prefix_plan else kv_bytes
        achieved = algo_bytes / sec_per_step / 1e9
        kname = {da.DA_KERNEL_SIMT: "decode_attn_simt_kernel", da.DA_KERNEL_MMA_TMA: "decode_attn_mma_kernel",
                 da.DA_KERNEL_UMMA_PREFIX: "decode_attn_umma_prefix_kernel + decode_attn_mma_kernel"}[info.kernel]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": sec_per_step * 1e3, "us_per_step": sec_per_step * 1e6,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": f"{IN_DTYPE} in, f32 accumulate",
            "data": "synthetic",
            "config": {"workload": args.workload, "batch": first.batch, "num_q_heads": first.num_q_heads,
                       "num_kv_heads": first.num_kv_heads, "head_dim": first.head_dim, "page_size": first.page_size,
                       "tokens": first.logical_tokens, "logical_kv_bytes": kv_bytes, "unique_kv_bytes": unique_bytes,
                       "split": args.split, "chunk_tokens": info.chunk_tokens, "units": info.n_units,
                       "max_splits": info.max_splits_used, "kernel": kname, "ctas_per_sm": info.ctas_per_sm,
                       "fused_combine": bool(policy.fuse_combine), "cuda_graph": not args.no_graph,
                       "shared_prefix_tokens": int(policy.shared_prefix_tokens), "alias_after": args.alias_after,
                       "l2": f"rotating over {copies} physical pool copies ({copies * unique_bytes / 2**30:.2f} GiB)",
                       "first_plan_us": plan_us, "plan_us": replan_us, "parallelism": f"dp{world} (sequences sharded, no collective)"},
            "pct_of_8tbs": value / world / 8000.0 * 100.0,
            "pct_of_measured_hbm": value / world / peak * 100.0,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": (achieved / peak) if achieved else None, "peak_kind": f"of {peak_kind}",
                         "kernel": kname, "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                         "algorithmic_bytes_per_launch": algo_bytes,
                         "how": ("unique" if prefix_plan else "logical") +
                                " K+V bytes of the batch / (event time of the timed region / steps): the "
                                "step's combine launch and launch gaps are charged to the partial kernel",
                         "kernel_only": None if kernel_only_us is None else
                         {"us_per_launch": kernel_only_us, "achieved": algo_bytes / kernel_only_us / 1e3,
                          "frac": algo_bytes / kernel_only_us / 1e3 / peak,
                          "how": "the same graph replays without the combine launch (results are not merged)"}},
            "gpu_launches": args.steps * launches_per_step,
            "clocks": clocks,
            "e2e": e2e,
            "e2e_resident_kv": e2e_resident,
            "cpu_baseline": cpu,
        }
        if run_mask is not None:
            line["run_mask"] = {"masked_fraction": args.mask_fraction, "masked_kv_bytes": masked_bytes,
                                "read_kv_bytes": kv_bytes - masked_bytes,
                                "read_GB/s": (kv_bytes - masked_bytes) / sec_per_step / 1e9}
        if probe_us is not None:
            line["gather_probe"] = {"us": probe_us, "GB/s": kv_bytes / probe_us / 1e3}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
