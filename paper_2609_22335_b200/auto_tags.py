"""Intensity tags of the tile classes from one profiling pass (paper Section 3.2.2, "Profile Metadata").

The paper obtains each kernel's (tau_TC, tau_ALU, tau_MEM) by running it in isolation under hardware
counters and quantising three utilisation fractions to 0..15: tensor-core throughput, CUDA-core FP32
throughput, DRAM throughput, each as a fraction of its peak.  Here the unit is a tile class, and one
profiling pass is one frame of the workload in the serial run mode under ncu -- every node of the
tile program is then an ordinary kernel, alone on the GPU, one CTA per tile:

    python -m paper_2609_22335_b200.auto_tags command --config cfg2        # prints the ncu command line
    ncu ... python -m paper_2609_22335_b200.auto_tags run --config cfg2    # what that command profiles
    python -m paper_2609_22335_b200.auto_tags derive --config cfg2 --csv launches.csv --program program.json

`run` also writes the tile program (node -> class, tiles) next to the CSV so that `derive` needs no GPU.
The tags are per TILE: a node kernel of G tiles runs on min(G, SMs) SMs, so the tensor and FMA pipe
figures are taken per active SM (ncu's "pct_of_peak_sustained_active"), and the DRAM figure is the
kernel's DRAM throughput scaled to what it would be with a tile on every SM.  A class's tag is the
tile-weighted mean over its nodes, quantised as tau = min(15, round(15 u)).
"""
from __future__ import annotations

import argparse
import csv
import json
import sys

METRICS = ("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
           "sm__pipe_fma_cycles_active.avg.pct_of_peak_sustained_active",
           "dram__throughput.avg.pct_of_peak_sustained_elapsed")
KERNEL = "vla_node_kernel"
N_CLASSES = 8
TAU_MAX = 15


def quantise(u: float) -> int:
    """Utilisation fraction -> 4-bit tag (Section 3.2.2)."""
    return max(0, min(TAU_MAX, int(round(TAU_MAX * u))))


def ncu_command(config: str, csv_path: str = "auto_tags_launches.csv") -> str:
    return ("ncu --metrics " + ",".join(METRICS) + " --clock-control none -k regex:" + KERNEL +
            f" --csv --log-file {csv_path} python -m paper_2609_22335_b200.auto_tags run --config {config}")


def read_launches(path: str):
    """ncu --csv log -> list of launches in launch order: {"grid": int, metric: value, ...} for KERNEL only."""
    rows = []
    with open(path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    by_id = {}
    order = []
    for r in csv.DictReader(lines):
        if KERNEL not in r["Kernel Name"]:
            continue
        i = int(r["ID"])
        if i not in by_id:
            by_id[i] = {"grid": int(r["Grid Size"].strip("()").split(",")[0])}
            order.append(i)
        try:
            by_id[i][r["Metric Name"]] = float(r["Metric Value"].replace(",", ""))
        except ValueError:
            by_id[i][r["Metric Name"]] = 0.0
    for i in order:
        rows.append(by_id[i])
    return rows


def derive(launches, program, n_sms: int):
    """Launches of ONE frame in program order (the last len(program) node kernels of the run) -> per-class tags.

    program: list of {"cls": int, "n_tiles": int} per node.  Returns (tags [8][3], per-class detail)."""
    n = len(program)
    if len(launches) < n:
        raise ValueError(f"{len(launches)} profiled launches for a program of {n} nodes")
    frame = launches[-n:]
    acc = [[0.0, 0.0, 0.0, 0.0] for _ in range(N_CLASSES)]           # weighted sums of u_TC, u_ALU, u_MEM and the weight
    for node, l in zip(program, frame):
        if l["grid"] != node["n_tiles"]:
            raise ValueError(f"launch grid {l['grid']} does not match node tiles {node['n_tiles']}: wrong launch window")
        active_sms = min(node["n_tiles"], n_sms)
        u_tc = l.get(METRICS[0], 0.0) / 100.0
        u_alu = l.get(METRICS[1], 0.0) / 100.0
        u_mem = min(1.0, l.get(METRICS[2], 0.0) / 100.0 * n_sms / active_sms)
        a = acc[node["cls"]]
        wgt = float(node["n_tiles"])
        a[0] += wgt * u_tc; a[1] += wgt * u_alu; a[2] += wgt * u_mem; a[3] += wgt
    tags, detail = [], {}
    for c in range(N_CLASSES):
        a = acc[c]
        if a[3] == 0:
            tags.append(None)
            continue
        u = [a[0] / a[3], a[1] / a[3], a[2] / a[3]]
        tags.append([quantise(x) for x in u])
        detail[c] = {"u_tc": u[0], "u_alu": u[1], "u_mem": u[2], "tiles": a[3]}
    return tags, detail


def relative_tags(detail):
    """The same measurements on a relative scale: per pipeline, the class that uses it most gets 15.

    Tiles that run alone on an SM and are bound by latency use a few per cent of every pipeline, so the paper's
    absolute rule quantises them all to 0 or 1 and the Phase-2 score cannot tell the classes apart; the relative
    scale keeps their order.  Returns tags [8][3] with None for classes without measurements."""
    keys = ("u_tc", "u_alu", "u_mem")
    top = [max((d[k] for d in detail.values()), default=0.0) for k in keys]
    out = []
    for c in range(N_CLASSES):
        d = detail.get(c, detail.get(str(c)))
        out.append(None if d is None else [quantise(d[k] / t) if t > 0 else 0 for k, t in zip(keys, top)])
    return out


def _run(config: str, program_path: str):
    """One frame of one request stream in the serial mode (what the ncu command profiles)."""
    import torch
    from vla_synth.configs import get_config
    from vla_synth.gen import make_weights, frame_inputs
    from . import Engine
    m = get_config(config)
    eng = Engine(m, mode="serial", n_streams=1)
    try:
        eng.load_weights(make_weights(m, seed=0, cache=False))
        prog = eng.program_info()
        eng.run([[frame_inputs(m, 0, 0, seed=0)]])
        sms = torch.cuda.get_device_properties(eng.device).multi_processor_count
    finally:
        eng.close()
    with open(program_path, "w") as f:
        json.dump({"config": config, "n_sms": sms, "nodes": [{"cls": n["cls"], "n_tiles": n["n_tiles"], "name": n["name"]} for n in prog]}, f)


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("what", choices=["command", "run", "derive"])
    ap.add_argument("--config", default="cfg2")
    ap.add_argument("--csv", default="auto_tags_launches.csv")
    ap.add_argument("--program", default="auto_tags_program.json")
    ap.add_argument("--relative", action="store_true", help="scale every pipeline so that its heaviest class gets 15")
    a = ap.parse_args(argv)
    if a.what == "command":
        print(ncu_command(a.config, a.csv))
    elif a.what == "run":
        _run(a.config, a.program)
    else:
        prog = json.load(open(a.program))
        tags, detail = derive(read_launches(a.csv), prog["nodes"], prog["n_sms"])
        out = {"config": prog["config"], "tags": relative_tags(detail) if a.relative else tags, "absolute_tags": tags,
               "scale": "relative" if a.relative else "absolute", "detail": detail}
        json.dump(out, sys.stdout, indent=1)
        print()


if __name__ == "__main__":
    main()
