"""Step timeline of graph-replayed decode-attention steps, from a trace build of the library.

    python -m paper_2609_37062_b200.timeline [--context 32768] [--batch 1] [--steps 20] [--fuse]

Builds the library with -DDA_TRACE (build.build_trace), captures K steps of
run + combine in one CUDA graph - every step with its own stamp buffer and its
own physical copy of the pools - replays the graph back to back and reads the
last replay.  For every step it prints, relative to the moment the partial
kernel's dependency wait is over (minimum / median / maximum over blocks):
block entry, the producer's first page ids and first copy, the first stage
landing, the end of the streaming loop and of the unit, the combine kernel's
entry, release, loads, sums and end, and the same points of the next step.
%globaltimer ticks are 256 ns on B200, so single figures carry that grain;
the medians over steps and blocks are what to read.  The traced build is a
few tenths of a microsecond slower per step than the product library.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import sys


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--context", type=int, default=32768)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--copies", type=int, default=10)
    ap.add_argument("--fuse", action="store_true")
    ap.add_argument("--split", default="auto", choices=["auto", "deterministic"])
    ap.add_argument("--workload", default="sweep", choices=["sweep", "short_chat", "few_shot_suffixes"],
                    help="sweep: --batch sequences of --context tokens; short_chat: the 64-sequence chat mix; "
                         "few_shot_suffixes: the 256 private suffixes (16..256 tokens) of the few-shot batch, by themselves")
    ap.add_argument("--units", action="store_true",
                    help="also print, in SM clock cycles turned into microseconds at --mhz, what a block's first four units "
                         "spend waiting for their first stage, streaming and finishing, and how the second unit's finish divides")
    ap.add_argument("--mhz", type=float, default=1965.0)
    args = ap.parse_args(argv)

    from . import build as da_build
    os.environ["DECODE_ATTN_LIB"] = da_build.build_trace()
    import numpy as np
    import torch
    from . import binding as da
    from . import workloads as wl

    lib = da._lib
    lib.decode_attn_trace_set_buffer.argtypes = [ctypes.c_void_p]
    K, copies = args.steps, args.copies
    if args.workload == "short_chat":
        pools = [wl.config_short_chat(device="cuda", table_seed=i) for i in range(copies)]
    elif args.workload == "few_shot_suffixes":
        lens = [x - 1536 for x in wl.lengths_shared_prefix(256, 3)]
        pools = [wl.make_workload("few_shot_suffixes", lens, 32, 8, 128, seed=3, device="cuda", table_seed=i) for i in range(copies)]
    else:
        pools = [wl.config_sweep_cell(args.context, args.batch, device="cuda", table_seed=i) for i in range(copies)]
    w = pools[0]
    policy = da.make_policy(fuse_combine=int(args.fuse),
                            split_mode=da.DA_SPLIT_DETERMINISTIC if args.split == "deterministic" else da.DA_SPLIT_AUTO)
    plan = da.decode_attn_plan(da.shape_of_workload(w), policy, w.seq_lens)
    info = plan.info()
    if info.kernel != da.DA_KERNEL_MMA_TMA:
        raise SystemExit("the timeline covers plans of the tensor-core kernel")
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.batch, w.num_q_heads), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    n = int(info.grid)
    rows = n + 8192                                   # the combine blocks' stamps follow the partial kernel's rows
    trace = torch.zeros((K, rows, 32), dtype=torch.int64, device="cuda")

    def step(i, traced):
        p = pools[i % copies]
        lib.decode_attn_trace_set_buffer(trace[i].data_ptr() if traced else None)
        da.decode_attn_run(plan, p.q_bits, p.k_pool, p.v_pool, p.block_table, p.seq_lens, out, lse, ws, plan.workspace_bytes)
        if not args.fuse:
            da.decode_attn_combine(plan, ws, out, lse)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for i in range(5):
            step(i, False)
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(K):
                step(i, True)
        for _ in range(3):
            g.replay()
        s.synchronize()
        trace.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            g.replay()                                # back to back: the last one is read
        e0.record(s)
        g.replay()
        e1.record(s)
        s.synchronize()
    lib.decode_attn_trace_set_buffer(None)
    what = f"{args.context} tokens x {args.batch}" if args.workload == "sweep" else args.workload
    print(f"{what} ({args.split}): {info.n_units} units on {n} blocks; "
          f"region of {K} steps: {e0.elapsed_time(e1) * 1e3 / K:.2f} us per step (traced build)")
    t = trace.cpu().numpy().astype(np.float64)
    P, C = t[:, :n, :], t[:, n:4096, :]          # (rows from 4096 on hold the cycle stamps of the blocks' merges)

    def rng(a):
        a = a[a > 0]
        return (a.min(), float(np.median(a)), a.max()) if a.size else (np.nan,) * 3

    names = [("partial: block entry", "P", 0), ("partial: dependency wait over", "P", 7),
             ("partial: producer past the wait", "P", 8), ("partial: first page ids in hand", "P", 9),
             ("partial: first copy issued", "P", 2), ("partial: first stage landed", "P", 3),
             ("partial: first unit's streaming loop done", "P", 4), ("partial: first unit finished", "P", 6),
             ("partial: last unit finished", "P", 5),
             ("combine: block entry", "C", 0), ("combine: dependency wait over", "C", 1),
             ("combine: loads landed", "C", 3), ("combine: sums done", "C", 5), ("combine: done", "C", 2)]
    per_step = [{nm: rng((P if src == "P" else C)[i, :, slot]) for nm, src, slot in names} for i in range(K)]
    acc = {}
    for i in range(2, K - 1):
        zero = per_step[i]["partial: dependency wait over"][0]
        for nm, _, _ in names:
            acc.setdefault(nm, []).append([x - zero for x in per_step[i][nm]])
        for nm in ("partial: dependency wait over", "partial: first copy issued", "partial: first stage landed"):
            acc.setdefault("next " + nm, []).append([x - zero for x in per_step[i + 1][nm]])
    print("us after the earliest end of the step's dependency wait: min / median / max over blocks (medians over steps)")
    for nm, v in acc.items():
        a = np.array(v)
        if np.isnan(a).all():
            continue
        print(f"{nm:46s} {np.nanmedian(a[:, 0]) / 1e3:7.2f} {np.nanmedian(a[:, 1]) / 1e3:7.2f} {np.nanmedian(a[:, 2]) / 1e3:7.2f}")
    period = [per_step[i + 1]["partial: dependency wait over"][0] - per_step[i]["partial: dependency wait over"][0]
              for i in range(2, K - 1)]
    print(f"step period (end of wait to end of wait): median {np.median(period) / 1e3:.2f} us")
    if args.units:
        c = P[2:]                                     # steps 2.., every block

        def med(a, ok):
            a = a[ok]
            return float(np.median(a)) / args.mhz if a.size else float("nan")

        print(f"per unit, SM cycles at {args.mhz:.0f} MHz, medians over blocks and steps (us):")
        for k in range(4):
            c0, c1, c2, c3 = (c[:, :, 10 + 4 * k + j] for j in range(4))
            ok = (c0 > 0) & (c1 > 0) & (c2 > 0) & (c3 > 0)
            if not ok.any():
                continue
            line = (f"  unit {k}: waits for its first stage {med(c1 - c0, ok):.2f}, streams {med(c2 - c1, ok):.2f}, "
                    f"finishes {med(c3 - c2, ok):.2f}")
            if k > 0:
                prev = c[:, :, 13 + 4 * (k - 1)]
                line += f" (taken up {med(c0 - prev, ok & (prev > 0)):.2f} after the unit before was finished)"
            print(line)
        c2, c3 = c[:, :, 16], c[:, :, 17]
        a, b2, cc, d = (c[:, :, 26 + j] for j in range(4))
        ok = (c2 > 0) & (a > 0) & (b2 > 0) & (cc > 0) & (d > 0) & (c3 > 0)
        if ok.any():
            print(f"  the second unit's finish: next unit's loads asked for, sums shuffled {med(a - c2, ok):.2f} | vote barrier "
                  f"{med(b2 - a, ok):.2f} | low parts added, states into the scratch {med(cc - b2, ok):.2f} | barrier "
                  f"{med(d - cc, ok):.2f} | merge of the four warps' states and the record {med(c3 - d, ok):.2f}")
        f = t[2:, 4096:4096 + n, :]                   # stamps inside the merge of a block's last unit
        f0, f1, f2, f3 = (f[:, :, j] for j in range(4))
        ok = (f0 > 0) & (f1 > f0) & (f2 > f1) & (f3 > f2)
        if ok.any():
            print(f"  inside that merge (a block's last unit): maximum over the warps {med(f1 - f0, ok):.2f} | weights and sums "
                  f"{med(f2 - f1, ok):.2f} | stores {med(f3 - f2, ok):.2f}")


if __name__ == "__main__":
    main()
