"""Turn the JSON line of bench.py into the markdown tables quoted in the documentation.

    python bench.py > bench.json
    python -m paper_2609_33051_b200.report bench.json

Formatting only: every figure printed here is read from the benchmark's output.
"""
from __future__ import annotations

import json
import sys


def _f(x, nd=2):
    return "-" if x is None else f"{x:.{nd}f}"


def headline(d: dict) -> str:
    k, r, c = d["kernels"], d["roofline"], d["clocks"]
    fr = d.get("full_read_baseline") or {}
    lines = [
        f"workload: {d['config']['workload']}, {d['config']['layers']} logical layers on n_phys = {d['details']['n_phys']} slots "
        f"({d['details']['device_bytes'] / 1e9:.1f} GB); steps {d['steps']}, warm-up {d['warmup']}",
        f"value: {d['value'] / 1e6:.3f} M {d['unit']} ({d['ms_per_step']:.2f} ms per window over all layers); "
        f"SM clock median {c['sm_mhz']} of {c['sm_max_mhz']} MHz, reasons {c['reasons']}",
        f"decode ({k['decode']['kernel']}): {k['decode']['in_window_us']:.1f} us per launch in the window = "
        f"{k['decode']['in_window_gbs']:.0f} GB/s = {k['decode']['frac_of_measured']:.3f} of measured, "
        f"{k['decode']['frac_of_8TBs_nominal']:.3f} of 8 TB/s; back to back {k['decode']['back_to_back_us']:.1f} us "
        f"({k['decode']['back_to_back_frac_of_measured']:.3f}); share of the window {k['decode_share_of_window']:.2f}",
        f"flush ({k['update']['kernel']}): {k['update']['back_to_back_us']:.1f} us = {k['update']['back_to_back_gbs']:.0f} GB/s = "
        f"{k['update']['frac_of_measured']:.3f} of measured, {k['update']['frac_of_8TBs_nominal']:.3f} of 8 TB/s",
        f"roofline: {r['kernel']} {r['achieved']:.0f} / {r['peak']:.0f} GB/s = {r['frac']:.3f} ({r['peak_source']}); "
        f"ncu DRAM traffic per launch {(_f(r['traffic'] / 1e6, 1) + ' MB') if r.get('traffic') else '-'} vs algorithmic "
        f"{r['algorithmic_bytes_per_launch'] / 1e6:.1f} MB",
    ]
    if fr:
        lines.append(f"full-read window: {fr['value'] / 1e6:.3f} M ({fr['sketch_speedup']:.2f}x slower than the sketch path); "
                     f"unbuffered standard decode: {fr['standard']['value'] / 1e6:.3f} M ({fr['standard']['sketch_speedup']:.2f}x); "
                     f"sketch write adds {100 * fr['sketch_write_overhead']:.1f} % to the flush")
    if d.get("graph_replay") and "value" in d["graph_replay"]:
        lines.append(f"CUDA-graph replay of the window: {d['graph_replay']['value'] / 1e6:.3f} M")
    if d.get("sustained"):
        s = d["sustained"]
        bins = ", ".join(f"{mhz} MHz: {b['ms_per_step']:.1f} ms x {b['steps']}" for mhz, b in s["by_sm_mhz"].items())
        lines.append(f"sustained {s['seconds']:.1f} s: {s['value'] / 1e6:.3f} M; per-step time by SM clock: {bins}")
    if d.get("e2e"):
        e = d["e2e"]
        lines.append(f"end to end with host token tensors: {e['value'] / 1e6:.3f} M ({e['h2d_bytes_per_step'] / 1e9:.1f} GB up, "
                     f"{e['d2h_bytes_per_step'] / 1e9:.1f} GB down per step)")
    if d.get("cpu_baseline"):
        cb = d["cpu_baseline"]
        lines.append(f"CPU oracle: {cb['value']:.0f} {cb['unit']} on {cb['cores']} core ({cb['sample']})")
    return "\n".join("- " + ln for ln in lines)


def table(rows) -> str:
    out = ["| workload | map / storage | n_phys | M tokens/s/layer | decode us (in window) | of measured | of 8 TB/s | flush kernel | flush us | "
           "of measured | + sketch (+ map) on the flush | sketch vs full read | SM MHz | reasons |",
           "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for s in rows:
        name = s["workload"].split(":")[0]
        shape = s["workload"].split(":")[1].strip()
        var = ("fixed" if s["coefficient_map"].startswith("fixed") else "state-dep. P=4" if "P = 4" in s["coefficient_map"] else "state-dep. exact") \
            + " / " + s["sketch_storage"] + (" / erase vectors" if s.get("erase_factors") else "")
        out.append(f"| {name} ({shape}) | {var} | {s['n_phys']} | {s['value'] / 1e6:.2f} | {s['decode_in_window_us']:.1f} | "
                   f"{s['decode_frac_of_measured']:.2f} | {s['decode_frac_of_8TBs_nominal']:.2f} | {s['update_kernel']} | {s['update_us']:.0f} | "
                   f"{s['update_frac_of_measured']:.2f} | {100 * s['sketch_and_map_overhead_on_flush']:.0f} % | "
                   f"{s['full_read']['sketch_speedup']:.2f}x | {s['clocks']['sm_mhz']:.0f} | {','.join(s['clocks']['reasons']) or '-'} |")
    return "\n".join(out)


def main(path: str) -> None:
    with open(path) as f:
        d = json.loads(f.read().strip().splitlines()[-1])
    print("### Headline\n")
    print(headline(d))
    if d.get("sweep"):
        print("\n### Layer workloads and the large-batch sweep (one record per point, each with its own clock samples)\n")
        print(table(d["sweep"]))
    if d.get("variants"):
        print("\n### The paper's own configuration of the method: state-dependent coefficient map, bfloat16 sketch storage\n")
        print(table(d["variants"]))


if __name__ == "__main__":
    main(sys.argv[1])
