"""Markdown tables from bench.py's JSON line(s).

    python bench.py --steps 20 --warmup 5 > line.json
    python -m paper_2609_37062_b200.report line.json [more.json ...]

Prints the headline, the per-configuration list (`configs`), the RUN-mask
series with the time a linear saving would give, and the sweep cells side by
side in both split modes - the tables of the design document are made this
way, from the benchmark's own output.
"""
from __future__ import annotations

import json
import sys


def _lines(path):
    with open(path) as f:
        for ln in f:
            ln = ln.strip()
            if ln.startswith("{"):
                yield json.loads(ln)


def _clk(c):
    c = c or {}
    r = ",".join(c.get("reasons") or []) or "none"
    return f"{c.get('sm_mhz')} MHz, {r}"


def headline(d):
    cfg, rf = d["config"], d["roofline"]
    print(f"### {cfg['workload']} ({d['n_gpus']} GPU, {d['steps']} steps per region, {d.get('repeats', 1)} regions)\n")
    print("| quantity | value |\n|---|---|")
    print(f"| us per step, median of regions (fastest region) | {d['us_per_step']:.2f} ({d.get('us_per_step_min', float('nan')):.2f}) |")
    print(f"| KV-read GB/s | {d['value']:.0f} |")
    print(f"| % of 8 TB/s / of the measured copy bandwidth | {d['pct_of_8tbs']:.1f} / {d['pct_of_measured_hbm']:.1f} |")
    ko = rf.get("kernel_only")
    if ko:
        print(f"| partial kernel alone, us per launch (fraction of measured) | {ko['us_per_launch']:.2f} ({ko['frac']:.3f}) |")
    if d.get("gather_probe"):
        g = d["gather_probe"]
        print(f"| gather-only probe, us (GB/s) | {g['us_per_step']:.2f} ({g['GB/s']:.0f}) |")
    rp = cfg.get("replan") or {}
    if rp:
        print(f"| re-plan (plan + destroy) us, median / p90 | {rp['plan_destroy_us_median']:.1f} / {rp['plan_destroy_us_p90']:.1f} |")
        if "plan_update_us_median" in rp:
            print(f"| in-place refresh (plan_update) us, median / p90 | {rp['plan_update_us_median']:.1f} / {rp['plan_update_us_p90']:.1f} |")
    if d.get("e2e"):
        print(f"| end to end from host buffers, GB/s (ms per step) | {d['e2e']['value']:.1f} ({d['e2e']['ms_per_step']:.2f}) |")
    if d.get("e2e_resident_kv"):
        e = d["e2e_resident_kv"]
        print(f"| pools resident, inputs from host, GB/s (us per step) | {e['value']:.0f} ({e['ms_per_step'] * 1e3:.0f}) |")
    if d.get("cpu_baseline"):
        c = d["cpu_baseline"]
        print(f"| oracle on {c['cores']} host cores, GB/s | {c['value']:.2f} |")
    if d.get("exchange"):
        x = d["exchange"]
        print(f"| local attention / gather + merge, us per step | {x['us_per_step_local_attention']:.2f} / {x['us_per_step_gather_and_merge']:.2f} |")
    print(f"| clocks during the timed regions | {_clk(d.get('clocks'))} |\n")


def configs(d):
    cs = d.get("configs") or []
    plain = [c for c in cs if "masked_fraction" not in c and not c["workload"].startswith("sweep_")]
    sweep = [c for c in cs if "masked_fraction" not in c and c["workload"].startswith("sweep_")]
    mask = [c for c in cs if "masked_fraction" in c]
    if plain:
        print("| workload | plan | us/step (fastest) | logical GB/s | % of 8 TB/s | unique GB/s | % of measured (unique) | units | clocks |")
        print("|---|---|---|---|---|---|---|---|---|")
        for c in plain:
            plan = c["split"] + (f", shared prefix {c['shared_prefix_tokens']}" if c.get("shared_prefix_tokens") else "")
            uq = c["unique_kv_bytes"] / c["us_per_step"] / 1e3
            peak = c["GB/s"] / (c["pct_of_measured_hbm"] / 100.0)
            print(f"| {c['workload']} | {plan} | {c['us_per_step']:.2f} ({c['us_per_step_min']:.2f}) | {c['GB/s']:.0f} | "
                  f"{c['pct_of_8tbs']:.1f} | {uq:.0f} | {uq / peak * 100:.1f} | {c['units']} | {_clk(c['clocks'])} |")
            if c.get("cpu_baseline"):
                o = c["cpu_baseline"]
                print(f"| | oracle on {o['cores']} host cores | {o['ms_per_step']:.1f} ms per step | {o['value']:.2f} | | | | | |")
            if c.get("replan"):
                r = c["replan"]
                print(f"| | re-plan us median / p90 | {r['plan_destroy_us_median']:.1f} / {r['plan_destroy_us_p90']:.1f}"
                      f" (refresh {r.get('plan_update_us_median', float('nan')):.1f} / {r.get('plan_update_us_p90', float('nan')):.1f}) | | | | | | |")
        print()
    if sweep:
        cells = {}
        for c in sweep:
            cells.setdefault(c["workload"], {})[c["split"]] = c
        print("| context x batch | KV bytes | AUTO us (fastest) | GB/s | % of 8 TB/s | % of measured | DETERMINISTIC us (fastest) | GB/s | % of 8 TB/s | DET / AUTO | probe GB/s |")
        print("|---|---|---|---|---|---|---|---|---|---|---|")
        for name, m in cells.items():
            a, t = m.get("auto"), m.get("deterministic")
            ref = a or t
            kv = ref["logical_kv_bytes"]
            size = f"{kv / 2**30:.3g} GiB" if kv >= 2**30 else f"{kv / 2**20:.0f} MiB"
            cell = name[len("sweep_"):].replace("x", " x ") + (f" (aliased, K = {ref['alias_after']})" if ref.get("alias_after") else "")

            def cols(c):
                return (f"{c['us_per_step']:.1f} ({c['us_per_step_min']:.1f}) | {c['GB/s']:.0f} | {c['pct_of_8tbs']:.1f}") if c else "- | - | -"
            ratio = f"{t['us_per_step'] / a['us_per_step']:.2f}" if a and t else "-"
            probe = f"{a['gather_probe']['GB/s']:.0f}" if a and a.get("gather_probe") else ""
            print(f"| {cell} | {size} | {cols(a)} | {a['pct_of_measured_hbm']:.1f} | {cols(t)} | {ratio} | {probe} |" if a else
                  f"| {cell} | {size} | - | - | - | - | {cols(t)} | - | |")
        print()
    if mask:
        t0 = next((c["us_per_step"] for c in mask if c["masked_fraction"] == 0.0), None)
        t1 = next((c["us_per_step"] for c in mask if c["masked_fraction"] == 1.0), None)
        print(f"RUN mask on {mask[0]['workload']} ({mask[0]['units']} units):\n")
        print("| masked fraction s | us/step (fastest) | KV bytes read (MB) | linear: (1 - s) (t(0) - t(1)) + t(1) | ratio | clocks |")
        print("|---|---|---|---|---|---|")
        for c in mask:
            s = c["masked_fraction"]
            lin = (1 - s) * (t0 - t1) + t1 if t0 is not None and t1 is not None else float("nan")
            print(f"| {s:.4g} | {c['us_per_step']:.1f} ({c['us_per_step_min']:.1f}) | {c['read_kv_bytes'] / 1e6:.0f} | {lin:.1f} | "
                  f"{c['us_per_step'] / lin:.3f} | {_clk(c['clocks'])} |")
        print()


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    if not argv:
        raise SystemExit(__doc__)
    for path in argv:
        for d in _lines(path):
            if d.get("impl") == "reference":
                print(f"reference arm (the oracle): {d['value']:.2f} GB/s, {d['ms_per_step']:.1f} ms per step, "
                      f"{d['cpu_baseline']['cores']} cores, sample: {d['cpu_baseline']['sample']}\n")
                continue
            headline(d)
            configs(d)


if __name__ == "__main__":
    main()
