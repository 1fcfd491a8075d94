#!/usr/bin/env python
"""Benchmark of the paged decode-attention hot path (plan -> run -> combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--shard seq|kv] [--impl reference]

A step is one pass of the whole path over one batch: the split-KV partial
kernel and the LSE combine kernel (launched with a programmatic dependency on
it; --fuse merges inside the partial kernel instead) over every sequence of
the workload.  The default workload is the single long sequence
(batch 1, 32 query / 8 KV heads, head_dim 128, page 16, 32,768 tokens); the
metric is KV-read GB/s = logical K+V bytes of the batch / time per step.

Timing: the timed region is exactly K steps, replayed as CUDA graphs (of up
to 256 steps each) so that host launch cost stays out of a 20-microsecond
step.  After W (>= 3) warm-up steps the region is run R times back to back
(R >= 30), each run bracketed by its own pair of CUDA events on the launching
stream; `ms_per_step` is the MEDIAN region / K, the fastest region is
reported beside it, the maximum over ranks is taken, and a barrier and a
device synchronise stand on both sides of the whole measurement.  Successive
steps read different physical copies of the pools (distinct memory,
differently shuffled block tables) that together exceed 1 GiB, and the number
of copies divides K so that consecutive regions keep rotating; where it cannot
(a K with no suitable divisor) an L2-sized buffer is overwritten between
regions, outside the events.  SM clocks and throttle reasons are sampled
through NVML during every timed measurement.

--gpus N > 1: when not already under torchrun the script starts N ranks
itself (python -m torch.distributed.run, one per GPU, NCCL).  --shard seq
(default): every rank runs its own sequences and nothing is exchanged (weak
scaling).  --shard kv: one long sequence is cut by KV range over the ranks;
every rank attends its range, one all-gather moves (out, lse) and the
library's shard merge finishes the step (strong scaling).

The default single-GPU run also times a fixed list of the other workload
configurations with the same method and prints them under `configs`
(short_chat and the few-shot batch with the oracle's time beside them, five
sweep cells in both split modes, the RUN-mask series, gather-only probes);
--sweep times all 20 cells of the length x batch sweep instead.  --append
puts the own-layer KV write into the step, as a launch of its own or fused
into the attention launch.  `python -m paper_2609_37062_b200.report` turns
the JSON line into tables.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
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
L2_BYTES = 126 << 20
MIN_REPEATS = 30

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the partial kernel.  These are NOT
# measured by this run: they are typed in from the ncu captures summarised under profiles/ and have
# to be refreshed whenever those are (null where no capture of that workload exists).
NCU_TRAFFIC_BYTES = {
    "long_32k": (134_301_000 + 3_876_000, "profiles/decode_attn_mma_kernel_long_32k.md"),
    "sweep_8192x64": (2_148_316_000 + 4_489_000, "profiles/decode_attn_mma_kernel_sweep_8192x64.md"),
}


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2048)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--repeats", type=int, default=0, help="timed regions of K steps (0: 30, more for very short regions)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="long_32k",
                    help="long_32k | short_chat | shared_prefix | sweep_<context>x<batch> | tiny")
    ap.add_argument("--shard", default="seq", choices=["seq", "kv"],
                    help="multi-GPU sharding: by sequence (no exchange) or one long sequence by KV range (one all-gather)")
    ap.add_argument("--context", type=int, default=0, help="--shard kv: tokens of the sequence (0: 32768)")
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
    ap.add_argument("--no-extras", action="store_true", help="leave out the list of other configurations")
    ap.add_argument("--extras", action="store_true", help="time the list of other configurations whatever the workload")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the list: every cell of the length x batch sweep (512..131072 x 1..256) in both split modes")
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
    ap.add_argument("--append", default="none", choices=["none", "separate", "fused"],
                    help="own-layer KV write in the step: a launch of its own before the attention launch, or fused into it")
    ap.add_argument("--dry-spawn", action="store_true",
                    help="start the ranks, join them in a gloo group on the CPU, print how many there are and exit")
    return ap.parse_args(argv)


IN_DTYPE = "bf16"     # set from --in-dtype
PAGE_SIZE = 16        # set from --page-size
Q_HEADS = 32          # set from --q-heads (sweep cells)


# ------------------------------------------------------------------------------------ launching ranks

def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_command(n_ranks: int, argv) -> list:
    """The command that starts `n_ranks` copies of this script, one per GPU, under torch's launcher."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]


def maybe_spawn(args, argv) -> bool:
    """`--gpus N` outside a launcher: become the launcher.  Returns True if this process only launched."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ or args.impl == "reference":
        return False
    env = dict(os.environ)
    # the communicator's own lines (rank count, transport) stay visible - on stderr, so that stdout
    # carries the one JSON line and nothing else
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    rc = subprocess.call(spawn_command(args.gpus, argv), env=env)
    if rc != 0:
        raise SystemExit(rc)
    return True


def dry_spawn():
    """Joins the launched ranks on the CPU (gloo) and reports how many there are: the launch path
    of `--gpus N` without a GPU."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        t = torch.ones(1, dtype=torch.int64)
        dist.all_reduce(t)
        counted = int(t.item())
        dist.destroy_process_group()
    else:
        counted = 1
    if rank == 0:
        print(json.dumps({"spawned_ranks": counted, "world_size": world, "backend": "gloo"}))


# ------------------------------------------------------------------------------------ inputs

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


def pick_copies(unique_bytes: int, steps: int, want: int = 0):
    """How many physical copies of the pools the steps rotate over: enough for 1 GiB, and a divisor
    of the region's step count so that back-to-back regions keep rotating.  Returns (copies,
    rotation_closed); when no divisor is in reach the caller flushes L2 between regions."""
    need = max(2, -(-(1 << 30) // max(unique_bytes, 1)) + 1)
    if want:
        return want, steps % want == 0
    for c in range(need, min(64, 2 * need + 8) + 1):
        if c > need and c * unique_bytes > (12 << 30):
            break
        if steps % c == 0:
            return c, True
    return min(need, 64), False


class ClockSampler:
    """Reads SM clock and throttle reasons through NVML while a timed measurement runs."""

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
        while True:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            if self._stop.is_set():
                break
            time.sleep(0.001)

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


# ------------------------------------------------------------------------------------ the timed measurement

class Bench:
    """Device, stream and rank context shared by every measurement of a run."""

    def __init__(self, torch, da, dev, local_rank, world, rank):
        self.torch, self.da, self.dev = torch, da, dev
        self.local_rank, self.world, self.rank = local_rank, world, rank
        self.stream = torch.cuda.Stream(device=dev)
        self._flush = None

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def flush_l2(self):
        if self._flush is None:
            self._flush = self.torch.empty(2 * L2_BYTES, dtype=self.torch.uint8, device=self.dev)
        self._flush.fill_(1)

    def time_regions(self, step_fn, steps, warmup, repeats=0, rotation_closed=True, no_graph=False, period=0):
        """Median / fastest time of a region of `steps` calls of step_fn(i) (i = rotation index),
        over back-to-back regions, each with its own event pair on the launching stream."""
        torch = self.torch
        with torch.cuda.stream(self.stream):
            for i in range(max(warmup, 3)):
                step_fn(i)
            self.stream.synchronize()
            chunk = min(GRAPH_STEPS, steps)
            full, rem = divmod(steps, chunk)

            def runner(n, first):
                if no_graph:
                    return lambda: [step_fn(first + j) for j in range(n)]
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for j in range(n):
                        step_fn(first + j)
                return g.replay

            # Rotation indices continue through the region: chunk c starts at index c * chunk.
            # step_fn looks at the index modulo `period` (its number of pool copies) only, so
            # chunks whose first index agrees modulo the period share one captured graph.
            graphs = {}

            def chunk_runner(c):
                first = c * chunk
                key = first % period if period else first
                if key not in graphs:
                    graphs[key] = runner(chunk, key)
                return graphs[key]

            chunk_runs = [chunk_runner(c) for c in range(full)]
            run_rem = runner(rem, (full * chunk) % period if period else full * chunk) if rem else None

            def region():
                for run in chunk_runs:
                    run()
                if run_rem:
                    run_rem()

            region()                                     # graph warm-up (uploads the graphs), untimed
            self.stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            region()
            e1.record(self.stream)
            self.stream.synchronize()
            est_ms = max(e0.elapsed_time(e1), 1e-3)
            if repeats <= 0:
                # at least 30 regions; very short ones are repeated until about 50 ms have been timed
                repeats = int(min(200, max(MIN_REPEATS, 50.0 / est_ms)))
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(repeats)]
            sampler = ClockSampler(physical_gpu_index(self.local_rank))
            self.barrier()
            sampler.start()
            for a, b in evs:
                if not rotation_closed:
                    self.flush_l2()
                a.record(self.stream)
                region()
                b.record(self.stream)
            self.stream.synchronize()
            clocks = sampler.stop()
            self.barrier()
        times = sorted(a.elapsed_time(b) for a, b in evs)
        return {"median_ms": statistics.median(times), "min_ms": times[0], "max_ms": times[-1], "repeats": repeats,
                "clocks": clocks}


def workload_copies(name, dev, rank, steps, want=0, alias=None, cap_bytes=14 << 30):
    first = make_workload(name, dev, table_seed=1000 * rank, seed_shift=100 * rank, alias_after=alias)
    copies, closed = pick_copies(first.unique_kv_bytes, steps, want)
    while copies > 2 and copies * first.unique_kv_bytes > cap_bytes:
        copies -= 1
        closed = steps % copies == 0
    pools = [first]
    for i in range(1, copies):
        pools.append(make_workload(name, dev, table_seed=1000 * rank + i, seed_shift=100 * rank, alias_after=alias))
    return pools, closed


def make_mask(torch, w, fraction, dev):
    g = torch.Generator().manual_seed(12345)
    n_mask = int(round(fraction * w.batch))
    keep = torch.ones(w.batch, dtype=torch.uint8)
    keep[torch.randperm(w.batch, generator=g)[:n_mask]] = 0
    masked_bytes = int((w.seq_lens.cpu().long() * (1 - keep.long())).sum().item()) * w.kv_bytes_per_token
    return keep.to(dev), masked_bytes


def time_config(bench, name, steps, warmup, split="auto", prefix_aware=False, mask_fractions=None, probe=False,
                replan=False, alias=None, pools_closed=None):
    """One entry (or, with mask fractions, several) of the `configs` list: the same timing method
    as the headline on another workload.  Frees the workload before returning (unless the caller
    passed the pools in)."""
    torch, da = bench.torch, bench.da
    pools, closed = pools_closed or workload_copies(name, bench.dev, bench.rank, steps, alias=alias)
    w0 = pools[0]
    copies = len(pools)
    policy = da.make_policy(
        split_mode=da.DA_SPLIT_DETERMINISTIC if split == "deterministic" else da.DA_SPLIT_AUTO,
        shared_prefix_tokens=w0.shared_prefix_tokens if prefix_aware else 0)
    shape = da.shape_of_workload(w0)
    lens_host = w0.seq_lens.cpu().numpy()
    plan = da.decode_attn_plan(shape, policy, lens_host)
    info = plan.info()
    out = torch.empty((w0.batch, w0.num_q_heads, w0.head_dim), dtype=torch.float32, device=bench.dev)
    lse = torch.empty((w0.batch, w0.num_q_heads), dtype=torch.float32, device=bench.dev)
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=bench.dev)
    peak, _ = peak_hbm()
    entries = []
    for frac in (mask_fractions if mask_fractions is not None else [None]):
        run_mask, masked_bytes = (None, 0) if frac is None else make_mask(torch, w0, frac, bench.dev)

        def step(i):
            w = pools[i % copies]
            da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws,
                               plan.workspace_bytes, run_mask=run_mask)
            da.decode_attn_combine(plan, ws, out, lse)

        t = bench.time_regions(step, steps, warmup, rotation_closed=closed, period=copies)
        st = da.decode_attn_last_device_status(plan, bench.stream)
        if st != da.DA_OK:
            raise SystemExit(f"{name}: device status {da.decode_attn_strerror(st)}")
        us, us_min = t["median_ms"] * 1e3 / steps, t["min_ms"] * 1e3 / steps
        kv = w0.logical_kv_bytes
        e = {"workload": name, "split": split, "us_per_step": us, "us_per_step_min": us_min, "steps": steps,
             "repeats": t["repeats"], "logical_kv_bytes": kv, "unique_kv_bytes": w0.unique_kv_bytes,
             "GB/s": kv / us / 1e3, "pct_of_8tbs": kv / us / 1e3 / 80.0, "pct_of_measured_hbm": kv / us / 1e3 / peak * 100,
             "units": info.n_units, "chunk_tokens": info.chunk_tokens, "max_splits": info.max_splits_used,
             "copies": copies, "clocks": t["clocks"]}
        if alias:
            e["alias_after"] = alias
        if prefix_aware:
            e["shared_prefix_tokens"] = int(policy.shared_prefix_tokens)
            e["unique_GB/s"] = w0.unique_kv_bytes / us / 1e3
            e["unique_pct_of_measured_hbm"] = w0.unique_kv_bytes / us / 1e3 / peak * 100
        if frac is not None:
            e["masked_fraction"] = frac
            e["read_kv_bytes"] = kv - masked_bytes
        entries.append(e)
    if probe and info.kernel == da.DA_KERNEL_MMA_TMA:
        chk = torch.empty(int(info.n_units), dtype=torch.int32, device=bench.dev)

        def probe_step(i):
            w = pools[i % copies]
            da.decode_attn_gather_probe(plan, w.k_pool, w.v_pool, w.block_table, chk)

        t = bench.time_regions(probe_step, steps, warmup, rotation_closed=closed, period=copies)
        us = t["median_ms"] * 1e3 / steps
        entries[0]["gather_probe"] = {"us_per_step": us, "GB/s": w0.logical_kv_bytes / us / 1e3,
                                      "what": "the same loads through the same tensor maps and page lookups, no attention arithmetic"}
    if replan:
        entries[0]["replan"] = time_replans(da, shape, policy, lens_host)
    plan.destroy()
    del pools, out, lse, ws
    torch.cuda.empty_cache()
    return entries


def time_replans(da, shape, policy, lens_host, n=200):
    """Host time of re-planning a step: plan + destroy per step (buffers come from the library's
    cache), and the in-place refresh of a capacity plan a serving loop would use, each timed call
    by call."""
    import numpy as np
    for _ in range(10):
        da.decode_attn_plan(shape, policy, lens_host).destroy()
    ts = []
    for _ in range(n):
        t0 = time.perf_counter()
        da.decode_attn_plan(shape, policy, lens_host).destroy()
        ts.append((time.perf_counter() - t0) * 1e6)
    ts.sort()
    res = {"plan_destroy_us_median": ts[len(ts) // 2], "plan_destroy_us_p90": ts[int(len(ts) * 0.9)], "calls": n}
    if int(policy.shared_prefix_tokens) == 0:
        total = int(np.asarray(lens_host).sum())
        cap = da.make_policy(split_mode=policy.split_mode, chunk_tokens=policy.chunk_tokens, max_splits=policy.max_splits,
                             kernel=policy.kernel, fuse_combine=policy.fuse_combine,
                             capacity_batch=max(int(shape.batch), 1), capacity_tokens=max(total, 16))
        plan = da.decode_attn_plan(shape, cap, lens_host)
        import torch
        s = torch.cuda.current_stream()
        for _ in range(10):
            da.decode_attn_plan_update(plan, lens_host, stream=s)
        us = []
        for _ in range(n):
            t0 = time.perf_counter()
            da.decode_attn_plan_update(plan, lens_host, stream=s)
            us.append((time.perf_counter() - t0) * 1e6)
        s.synchronize()
        plan.destroy()
        us.sort()
        res["plan_update_us_median"] = us[len(us) // 2]
        res["plan_update_us_p90"] = us[int(len(us) * 0.9)]
    return res


def sweep_configs(bench, steps, warmup):
    """Every cell of the length x batch sweep in both split modes.  The 128 GiB cell does not fit:
    its sequences i >= 64 reuse the pages of sequence i mod 64 (it is partly served by L2)."""
    out = []
    for ctx in (512, 2048, 8192, 32768, 131072):
        for batch in (1, 8, 64, 256):
            name = f"sweep_{ctx}x{batch}"
            alias = 64 if ctx * batch * 4096 > (100 << 30) else None
            pc = workload_copies(name, bench.dev, bench.rank, steps, alias=alias, cap_bytes=70 << 30)
            for split in ("auto", "deterministic"):
                out += time_config(bench, name, steps, warmup, split=split, alias=alias, pools_closed=pc)
            del pc
            bench.torch.cuda.empty_cache()
    return out


def oracle_beside(entry, name, skip):
    """The oracle as it stands on this machine's cores, on the same workload (a reported baseline)."""
    if skip:
        return
    sec, reps, cores = time_oracle(make_workload(name, "cpu"), budget_s=2.0)
    entry["cpu_baseline"] = {"ms_per_step": sec * 1e3, "value": entry["logical_kv_bytes"] / sec / 1e9, "unit": UNIT,
                             "cores": cores, "kind": "oracle", "sample": f"whole batch, {reps} runs"}


def extra_configs(bench, steps, warmup, skip_cpu=False):
    """The other workload configurations, timed like the headline (median of repeated regions)."""
    out = []
    out += time_config(bench, "short_chat", steps, warmup, replan=True)
    oracle_beside(out[-1], "short_chat", skip_cpu)
    out += time_config(bench, "shared_prefix", steps, warmup)
    oracle_beside(out[-1], "shared_prefix", skip_cpu)
    out += time_config(bench, "shared_prefix", steps, warmup, prefix_aware=True)
    for cell, probe in (("sweep_512x256", False), ("sweep_2048x1", False), ("sweep_8192x64", True),
                        ("sweep_32768x8", False), ("sweep_131072x1", False)):
        for split in ("auto", "deterministic"):
            out += time_config(bench, cell, steps, warmup, split=split, probe=probe and split == "auto")
    out += time_config(bench, "sweep_1024x256", steps, warmup,
                       mask_fractions=[0.0, 1 / 16, 1 / 8, 3 / 16, 1 / 4, 3 / 8, 1 / 2, 9 / 16, 1.0])
    return out


# ------------------------------------------------------------------------------------ CPU legs

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


def workload_keys(name, w):
    """The keys of `config` that name the workload; the same in both arms."""
    return {"workload": name, "batch": int(w.batch), "num_q_heads": int(w.num_q_heads),
            "num_kv_heads": int(w.num_kv_heads), "head_dim": int(w.head_dim), "page_size": int(w.page_size),
            "tokens": int(w.logical_kv_bytes) // (int(w.num_kv_heads) * int(w.head_dim) * 4),
            "logical_kv_bytes": int(w.logical_kv_bytes), "unique_kv_bytes": int(w.unique_kv_bytes)}


def run_reference(args):
    """The oracle as it stands on this machine's cores: W warm-up and exactly K timed steps, each step a
    bounded sample of the workload sized so that the whole run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2609_37062_b200 import workloads as wl
    # torch's launcher sets OMP_NUM_THREADS=1 for its ranks; the oracle takes the machine's cores all the same
    threads = (os.cpu_count() or 1) if os.environ.get("TORCHELASTIC_RUN_ID") else oracle.max_threads()
    w, sample, _ = oracle_sample(args.workload)
    full_keys = workload_keys(args.workload, w)
    if sample != "whole batch":                           # a sweep cell: the whole cell's size, without generating it
        ctx, batch = (int(x) for x in args.workload[len("sweep_"):].split("x"))
        nbytes = ctx * batch * int(w.num_kv_heads) * int(w.head_dim) * 4
        full_keys.update(batch=batch, tokens=ctx * batch, logical_kv_bytes=nbytes, unique_kv_bytes=nbytes)
    inp = oracle.PagedInputs.from_workload(w)
    t0 = time.perf_counter()
    oracle.paged_decode_attention(inp, num_threads=threads)
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
        oracle.paged_decode_attention(inp, num_threads=threads)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.paged_decode_attention(inp, num_threads=threads)
    dt = (time.perf_counter() - t0) / steps
    gbs = w.logical_kv_bytes / dt / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(full_keys, sample=sample, sample_tokens=w.logical_tokens),
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ KV-range sharding

def run_kv_shard(args, bench):
    """One long sequence cut by KV range over the ranks (context parallel): every rank attends its
    token range with plan / run / combine, one all-gather (NCCL) moves every rank's (out, lse) -
    a few KB - into local buffers, and decode_attn_merge_shards merges them in rank order.  No
    kernel of the library reads another GPU's memory."""
    import torch.distributed as dist
    torch, da = bench.torch, bench.da
    from paper_2609_37062_b200 import sharding, workloads as wl
    world, rank, dev = bench.world, bench.rank, bench.dev
    context = args.context or 32768
    steps = args.steps
    # every rank generates the same sequence (same seeds) and keeps its own range of it: the local
    # block table points at the pages of tokens [begin, end) only
    copies, closed = pick_copies(context * 4096 // world, steps, args.copies)
    fulls = [wl.config_long(device=dev, context=context, seed=1, table_seed=i) for i in range(copies)]
    shape_full = da.shape_of_workload(fulls[0])
    locals_ = []
    for w in fulls:
        bt, lens = sharding.shard_kv_tables(w.block_table, w.seq_lens, w.page_size, world, rank)
        locals_.append((bt.to(dev), lens.to(dev), lens))
    lens_host = locals_[0][2].numpy()
    shape = da.make_shape(1, fulls[0].num_q_heads, fulls[0].num_kv_heads, fulls[0].head_dim, fulls[0].page_size,
                          locals_[0][0].shape[1], fulls[0].num_pages, fulls[0].strides)
    policy = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC if args.split == "deterministic" else da.DA_SPLIT_AUTO)
    plan = da.decode_attn_plan(shape, policy, lens_host)
    out_local = torch.empty((1, shape.num_q_heads, shape.head_dim), dtype=torch.float32, device=dev)
    lse_local = torch.empty((1, shape.num_q_heads), dtype=torch.float32, device=dev)
    outs = torch.empty((world,) + tuple(out_local.shape), dtype=torch.float32, device=dev)
    lses = torch.empty((world,) + tuple(lse_local.shape), dtype=torch.float32, device=dev)
    out = torch.empty_like(out_local)
    lse = torch.empty_like(lse_local)
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=dev)

    def local_step(i):
        w = fulls[i % copies]
        bt, lens_dev, _ = locals_[i % copies]
        da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, bt, lens_dev, out_local, lse_local, ws, plan.workspace_bytes)
        da.decode_attn_combine(plan, ws, out_local, lse_local)

    def full_step(i):
        local_step(i)
        if world > 1:
            dist.all_gather_into_tensor(outs, out_local)
            dist.all_gather_into_tensor(lses, lse_local)
        else:
            outs.copy_(out_local.unsqueeze(0))
            lses.copy_(lse_local.unsqueeze(0))
        da.decode_attn_merge_shards(shape_full, world, outs, lses, out, lse)

    # collectives inside a captured graph need a communicator that supports it; fall back to host launches
    no_graph = args.no_graph
    try:
        t_full = bench.time_regions(full_step, steps, args.warmup, args.repeats, closed, no_graph, copies)
    except Exception:
        if no_graph:
            raise
        no_graph = True
        torch.cuda.synchronize()
        t_full = bench.time_regions(full_step, steps, args.warmup, args.repeats, closed, True, copies)
    t_local = bench.time_regions(local_step, steps, args.warmup, args.repeats, closed, no_graph, copies)
    ms = sharding.max_over_ranks(t_full["median_ms"], dev)
    ms_min = sharding.max_over_ranks(t_full["min_ms"], dev)
    ms_local = sharding.max_over_ranks(t_local["median_ms"], dev)
    kv_bytes = context * fulls[0].kv_bytes_per_token
    if rank == 0:
        peak, peak_kind = peak_hbm()
        sec = ms * 1e-3 / steps
        value = kv_bytes / sec / 1e9
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
                "warmup": max(args.warmup, 3), "repeats": t_full["repeats"], "ms_per_step": sec * 1e3,
                "us_per_step": sec * 1e6, "us_per_step_min": ms_min * 1e3 / steps, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": f"{IN_DTYPE} in, f32 accumulate", "data": "synthetic",
                "config": {"workload": f"long_{context}_kv_sharded", "tokens": context, "logical_kv_bytes": kv_bytes,
                           "tokens_per_rank": int(lens_host[0]), "split": args.split, "cuda_graph": not no_graph,
                           "l2": f"rotating over {copies} physical pool copies" + ("" if closed else ", L2 flushed between regions"),
                           "parallelism": f"cp{world} (one sequence cut by KV range; one all-gather of out and lse, then the shard merge)"},
                "exchange": {"us_per_step_local_attention": ms_local * 1e3 / steps,
                             "us_per_step_gather_and_merge": (ms - ms_local) * 1e3 / steps,
                             "share_of_step": (ms - ms_local) / ms if ms > 0 else None,
                             "bytes_gathered_per_rank": int(outs.numel() * 4 + lses.numel() * 4)},
                "roofline": {"bound": "hbm", "achieved": value / world, "peak": peak, "unit": "GB/s",
                             "frac": value / world / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                             "traffic_source": None, "kernel": "decode_attn_mma_kernel",
                             "how": "this rank's share of the K+V bytes / the whole step, exchange and merge included"},
                "gpu_launches": steps * t_full["repeats"] * 3, "clocks": t_full["clocks"], "e2e": None, "cpu_baseline": None}
        return line
    return None


# ------------------------------------------------------------------------------------ main

def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    args = parse_args(argv)
    global IN_DTYPE, PAGE_SIZE, Q_HEADS
    IN_DTYPE = args.in_dtype
    PAGE_SIZE = args.page_size
    Q_HEADS = args.q_heads
    if maybe_spawn(args, argv):
        return
    if args.dry_spawn:
        dry_spawn()
        return
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2609_37062_b200 import binding as da
    from paper_2609_37062_b200 import sharding

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
    bench = Bench(torch, da, dev, local_rank, world, rank)
    stream = bench.stream
    if args.shard == "kv":
        line = run_kv_shard(args, bench)
        if world > 1:
            dist.destroy_process_group()
        if line is not None:
            print(json.dumps(line), flush=True)
        return

    # ---- inputs: R physical copies of the workload, this rank's own sequences
    alias = args.alias_after or None
    pools, closed = workload_copies(args.workload, dev, rank, args.steps, args.copies, alias, cap_bytes=150 << 30)
    first, copies = pools[0], len(pools)
    kv_bytes = first.logical_kv_bytes
    unique_bytes = first.unique_kv_bytes
    wl_keys = workload_keys(args.workload, first)

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
    replan = time_replans(da, shape, policy, lens_host)
    out = torch.empty((first.batch, first.num_q_heads, first.head_dim), dtype=torch.float32, device=dev)
    lse = torch.empty((first.batch, first.num_q_heads), dtype=torch.float32, device=dev)
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=dev)
    launches_per_step = 1 if (policy.fuse_combine or info.n_slots == 0) else 2
    if info.kernel == da.DA_KERNEL_UMMA_PREFIX:
        launches_per_step += 1      # the tcgen05 prefix kernel, then the kernel for what follows the prefix

    run_mask, masked_bytes = None, 0
    if args.mask_fraction is not None:
        run_mask, masked_bytes = make_mask(torch, first, args.mask_fraction, dev)

    new_k = new_v = None
    if args.append != "none":
        from paper_2609_37062_b200 import workloads as wl
        n_new = first.batch * first.num_kv_heads * first.head_dim
        new_k = wl.normal_bf16_bits(wl.stream_key(77, wl.TENSOR_NEW_K, 0), 0, n_new, dev).view(first.batch, first.num_kv_heads, -1)
        new_v = wl.normal_bf16_bits(wl.stream_key(77, wl.TENSOR_NEW_V, 0), 0, n_new, dev).view(first.batch, first.num_kv_heads, -1)
        launches_per_step += 1 if args.append == "separate" else 0

    def step(i, combine=True):
        w = pools[i % copies]
        if args.append == "separate":
            da.decode_attn_append_kv(shape, new_k, new_v, w.block_table, w.seq_lens, w.k_pool, w.v_pool)
        da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws,
                           plan.workspace_bytes, run_mask=run_mask,
                           new_k=new_k if args.append == "fused" else None, new_v=new_v if args.append == "fused" else None)
        if combine and not policy.fuse_combine and not args.partial_only:
            da.decode_attn_combine(plan, ws, out, lse)

    timed = bench.time_regions(step, args.steps, args.warmup, args.repeats, closed, args.no_graph, copies)
    st = da.decode_attn_last_device_status(plan, stream)
    if st != da.DA_OK:
        raise SystemExit(f"device status after the timed region: {da.decode_attn_strerror(st)}")

    # the dominant kernel by itself: the same regions without the combine launch
    kernel_only_us = None
    if not policy.fuse_combine and not args.partial_only and info.n_slots > 0:
        t_ko = bench.time_regions(lambda i: step(i, combine=False), args.steps, 3, args.repeats, closed, args.no_graph, copies)
        kernel_only_us = t_ko["median_ms"] * 1e3 / args.steps

    probe_us = None
    if (args.probe or (args.workload == "long_32k" and not args.no_extras)) and info.kernel == da.DA_KERNEL_MMA_TMA:
        chk = torch.empty(int(info.n_units), dtype=torch.int32, device=dev)

        def probe_step(i):
            w = pools[i % copies]
            da.decode_attn_gather_probe(plan, w.k_pool, w.v_pool, w.block_table, chk)

        t_pr = bench.time_regions(probe_step, args.steps, 3, args.repeats, closed, args.no_graph, copies)
        probe_us = t_pr["median_ms"] * 1e3 / args.steps

    ms = sharding.max_over_ranks(timed["median_ms"], dev)
    ms_min = sharding.max_over_ranks(timed["min_ms"], dev)
    sec_per_step = ms * 1e-3 / args.steps
    value = world * kv_bytes / sec_per_step / 1e9
    clocks = timed["clocks"]

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
        bench.barrier()
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
            bench.barrier()
            t0 = time.perf_counter()
            for _ in range(n_res):
                resident_step()
            dt = time.perf_counter() - t0
        e2e_resident = {"value": world * kv_bytes * n_res / dt / 1e9, "unit": UNIT,
                        "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in (hq, hbt, hsl)),
                        "d2h_bytes_per_step": d2h, "steps": n_res, "ms_per_step": dt / n_res * 1e3,
                        "what": "pools resident in HBM; q, block table, lengths from pinned host memory, plan, run, "
                                "merge, out back to host, synchronised every step"}
        del hq, hk, hv, hbt, hsl, hout, hw

    # ---- the other configurations, same method (single-GPU default run)
    configs = None
    want_extras = args.extras or args.sweep or (args.workload == "long_32k" and not args.no_extras and args.mask_fraction is None and
                                  args.split == "auto" and not args.fuse and not args.partial_only)
    if want_extras and world == 1:
        plan.destroy()
        del pools, first
        torch.cuda.empty_cache()
        k_extra, w_extra = min(args.steps, 64), min(max(args.warmup, 3), 8)
        configs = sweep_configs(bench, k_extra, w_extra) if args.sweep else extra_configs(bench, k_extra, w_extra, args.skip_cpu)

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
        traffic, traffic_src = NCU_TRAFFIC_BYTES.get(args.workload, (None, None))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "repeats": timed["repeats"], "ms_per_step": sec_per_step * 1e3,
            "us_per_step": sec_per_step * 1e6, "us_per_step_min": ms_min * 1e3 / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": f"{IN_DTYPE} in, f32 accumulate",
            "data": "synthetic",
            "config": {**wl_keys,
                       "split": args.split, "chunk_tokens": info.chunk_tokens, "units": info.n_units,
                       "max_splits": info.max_splits_used, "kernel": kname, "ctas_per_sm": info.ctas_per_sm,
                       "fused_combine": bool(policy.fuse_combine), "cuda_graph": not args.no_graph,
                       "shared_prefix_tokens": int(policy.shared_prefix_tokens), "alias_after": args.alias_after,
                       "kv_append": args.append,
                       "l2": f"rotating over {copies} physical pool copies ({copies * unique_bytes / 2**30:.2f} GiB)" +
                             ("" if closed else ", L2 flushed between regions"),
                       "timing": f"median of {timed['repeats']} back-to-back regions of {args.steps} graph-replayed steps, "
                                 "each between its own CUDA events; min beside it",
                       "first_plan_us": plan_us, "plan_us": replan["plan_destroy_us_median"], "replan": replan,
                       "parallelism": f"dp{world} (sequences sharded, no collective)"},
            "pct_of_8tbs": value / world / 8000.0 * 100.0,
            "pct_of_measured_hbm": value / world / peak * 100.0,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": (achieved / peak) if achieved else None, "peak_kind": f"of {peak_kind}",
                         "kernel": kname, "traffic": traffic,
                         "traffic_source": None if traffic is None else
                         f"typed in from the ncu capture summarised in {traffic_src}; not measured by this run",
                         "algorithmic_bytes_per_launch": algo_bytes,
                         "how": ("unique" if prefix_plan else "logical") +
                                " K+V bytes of the batch / (median event time of a region / steps): the "
                                "step's combine launch and launch gaps are charged to the partial kernel",
                         "kernel_only": None if kernel_only_us is None else
                         {"us_per_launch": kernel_only_us, "achieved": algo_bytes / kernel_only_us / 1e3,
                          "frac": algo_bytes / kernel_only_us / 1e3 / peak,
                          "how": "the same regions without the combine launch (results are not merged)"}},
            "gpu_launches": args.steps * launches_per_step * timed["repeats"],
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
            line["gather_probe"] = {"us_per_step": probe_us, "GB/s": kv_bytes / probe_us / 1e3,
                                    "what": "the same loads through the same tensor maps and page lookups, no attention "
                                            "arithmetic: the ceiling for this access pattern"}
        if configs is not None:
            line["configs"] = configs
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)          # the last thing on stdout


if __name__ == "__main__":
    main()
