"""Turns Nsight Compute output into the short text summaries kept under profiles/ and keeps
profiles/traffic.json (DRAM bytes per launch of every profiled kernel, read by bench.py) in step with them.

    python -m paper_2609_32114_b200.ncu_summary report REP.ncu-rep WORKLOAD "TITLE" "COMMAND" > profiles/NAME.md
    python -m paper_2609_32114_b200.ncu_summary traffic            # rebuild profiles/traffic.json from profiles/*.md

`report` reads the .ncu-rep with `ncu -i ... --page raw --csv` (works without a GPU) and prints one block per
captured launch.  Every summary starts with a line `workload: NAME`, which is how `traffic` files its figures.
"""
from __future__ import annotations

import csv
import glob
import io
import json
import os
import re
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PROFILES = os.path.join(ROOT, "profiles")

KEYS = [
    ("gpu__time_duration.sum", "duration"),
    ("launch__grid_size", "grid"), ("launch__block_size", "block"),
    ("launch__registers_per_thread", "registers/thread"),
    ("launch__shared_mem_per_block_dynamic", "dynamic smem/block"),
    ("launch__waves_per_multiprocessor", "waves/SM"),
    ("sm__warps_active.avg.pct_of_peak_sustained_active", "achieved occupancy (% of peak warps)"),
    ("dram__bytes_read.sum", "DRAM read"), ("dram__bytes_write.sum", "DRAM write"),
    ("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "DRAM throughput (% of peak)"),
    ("lts__t_bytes.sum", "L2 traffic"),
    ("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active", "tensor pipe active (% of peak)"),
    ("sm__inst_executed.avg.per_cycle_active", "IPC (per SM, active cycles)"),
    ("smsp__inst_executed.sum", "warp instructions"),
    ("sm__cycles_active.avg", "SM active cycles (avg)"),
    ("l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum", "shared-memory bank conflicts"),
]


def report(rep: str, workload: str, title: str, cmd: str) -> str:
    raw = subprocess.run(["ncu", "-i", rep, "--page", "raw", "--csv"], capture_output=True, text=True, check=True).stdout
    rows = list(csv.reader(io.StringIO(raw)))
    hdr, units = rows[0], rows[1]
    stall = [h for h in hdr if "issue_stalled" in h and "per_issue_active" in h and "not_issued" not in h]
    out = [f"# {title}", "", f"workload: {workload}", "",
           "Command (runs committed files only; on a B200 through the pool's runner):", "", f"    {cmd}", ""]
    for r in rows[2:]:
        out.append(f"## {r[hdr.index('Kernel Name')]}")
        for k, label in KEYS:
            if k in hdr:
                i = hdr.index(k)
                out.append(f"- {label}: {r[i]} {units[i]}")
        st = sorted(((float(r[hdr.index(h)]), h) for h in stall), reverse=True)[:6]
        out.append("- top warp stalls (cycles per issued instruction): " + ", ".join(
            f"{h.split('issue_stalled_')[1].split('_per_issue')[0]} {v:.2f}" for v, h in st))
        out.append("")
    return "\n".join(out)


_UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def kernel_key(name: str) -> str:
    """Short kernel name used by bench.py: tc_prep, tc_chain, decode, simt_prefill, plan."""
    for key in ("tc_prep", "tc_chain", "tc_fix", "decode", "simt_prefill", "plan"):
        if key in name:
            return key
    return name.split("(")[0].split("::")[-1]


def traffic() -> dict:
    """{workload: {kernel: {"dram_read": B, "dram_write": B, "launches": n, "source": file}}}; several captured
    launches of one kernel in one file are averaged."""
    table: dict = {}
    for path in sorted(glob.glob(os.path.join(PROFILES, "*.md"))):
        text = open(path).read()
        m = re.search(r"^workload:\s*(\S+)", text, flags=re.M)
        if not m:
            continue
        wl = m.group(1)
        for block in text.split("\n## ")[1:]:
            rd = re.search(r"- DRAM read: ([0-9.]+) (\w+)", block)
            wr = re.search(r"- DRAM write: ([0-9.]+) (\w+)", block)
            if not rd or not wr:
                continue
            k = kernel_key(block.splitlines()[0])
            e = table.setdefault(wl, {}).setdefault(k, {"dram_read": 0.0, "dram_write": 0.0, "launches": 0,
                                                        "source": os.path.basename(path)})
            if e["source"] != os.path.basename(path):
                continue                                   # first file (alphabetical) that covers this kernel wins
            e["dram_read"] += float(rd.group(1)) * _UNIT[rd.group(2)]
            e["dram_write"] += float(wr.group(1)) * _UNIT[wr.group(2)]
            e["launches"] += 1
    for wl in table.values():
        for e in wl.values():
            e["dram_read"] /= e["launches"]
            e["dram_write"] /= e["launches"]
    return table


def main(argv) -> int:
    if len(argv) >= 2 and argv[1] == "report" and len(argv) == 6:
        print(report(argv[2], argv[3], argv[4], argv[5]))
        return 0
    if len(argv) >= 2 and argv[1] == "traffic":
        t = traffic()
        with open(os.path.join(PROFILES, "traffic.json"), "w") as f:
            json.dump(t, f, indent=1, sort_keys=True)
            f.write("\n")
        print(json.dumps(t, indent=1, sort_keys=True))
        return 0
    sys.stderr.write(__doc__)
    return 2


if __name__ == "__main__":
    sys.exit(main(sys.argv))
