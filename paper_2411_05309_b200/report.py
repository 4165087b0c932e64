"""Turn the JSON line of ``bench.py`` into the markdown table the README shows.

    python bench.py > line.json
    python -m paper_2411_05309_b200.report line.json

One row per configuration of ``per_config`` (or the single record of a ``--workload`` run): time per
step, effective and migration GB/s, the roofline fraction with the direction that bounds the launch,
faults, the device scratch the workload holds beside its pool, end-to-end GB/s, the CPU oracle on the
host cores, and the same run with its scratch bounded where the line has one.
"""
from __future__ import annotations

import json
import sys


def _mib(nbytes: float) -> str:
    if not nbytes:
        return "none"
    return f"{nbytes / 2 ** 30:.1f} GiB" if nbytes >= 2 ** 30 else f"{nbytes / 2 ** 20:.1f} MiB"


def _row(cfg: str, r: dict) -> str:
    m, roof, sc = r["migration"], r["roofline"], r["scratch"]
    mig = f"{m['in_gbs']:.1f} in" + (f" + {m['out_gbs']:.1f} out" if m["out_gbs"] > 0.05 else "")
    if m.get("direct_gbs", 0.0) > 0.05:
        mig += f" + {m['direct_gbs']:.1f} read in place"
    frac = f"{roof['frac']:.3f}"
    if "frac_compulsory" in roof:
        frac += f" by faults, {roof['frac_compulsory']:.3f} of the compulsory floor"
    if roof.get("in_place"):
        frac += (f" (rows in place page by page; scattered reads over this table reach "
                 f"{roof['in_place']['scattered_read_peak_gbs']:.1f} GB/s)")
    cpu = r.get("cpu_baseline")
    cpu_s = "-"
    if cpu:
        cpu_s = f"{cpu['value']:.2f} on {cpu['cores']}"
        if "one_thread" in cpu:
            cpu_s += f" ({cpu['one_thread']['value']:.2f} on 1)"
    bounded = sc.get("bounded_to_an_eighth_of_the_pool")
    b_s = "-"
    if bounded:
        n = bounded["faults"]
        b_s = f"{_mib(bounded['limit_bytes'])}: {bounded['ms_per_step']:.0f} ms, " + (f"{n / 1e3:.0f} K faults" if n >= 10000 else f"{n} faults")
    ms = r["ms_per_step"]
    t = f"{ms:.2f} ms" if ms < 1000 else f"{ms / 1e3:.3f} s"
    return (f"| {cfg} {r['config']['workload'].split(':')[0].split(',')[0].split(' ', 1)[-1]} | {t} | {r['value']:.2f} | {mig} | {frac} | "
            f"{m['faults']:.0f} of {r['config']['pages']} pages | {_mib(sc['bytes'])} | {r['e2e']['value']:.2f} | {cpu_s} | {b_s} |")


def policies(line: dict) -> str:
    """cfg 5 under the other two policies, when the line has them."""
    recs = line.get("per_config") or {str(line["config"]["cfg"]): line}
    roof = recs.get("5", {}).get("roofline", {})
    out = []
    for key, name in (("counted_scattered", "the counted policy with rows read as their lookups come up"),
                      ("online", "the online policy (no count beforehand)"),
                      ("always_migrate", "the paper's policy (every first touch fetches)")):
        r = roof.get(key)
        if r:
            out.append(f"cfg 5 under {name}: {r['ms_per_step']:.1f} ms, {r['value']:.2f} GB/s, {r['faults']} faults, "
                       f"{r['bytes_in'] / 1e9:.2f} GB paged in + {r.get('bytes_direct', 0) / 1e9:.2f} GB read in place, "
                       f"roofline.frac {r['roofline']['frac']:.3f}.")
    return "\n".join(out)


def table(line: dict) -> str:
    recs = line.get("per_config") or {str(line["config"]["cfg"]): line}
    link = line.get("link_peak", {})
    out = []
    if link:
        out.append(f"Host link in this run: pinned copy {link['ce_h2d_gbs']:.1f} GB/s in, {link['ce_d2h_gbs']:.1f} out; "
                   f"loads issued by SMs {link['sm_h2d_gbs']:.1f}, stores {link['sm_d2h_gbs']:.1f}, both at once "
                   f"{link['sm_duplex_gbs']:.1f}.")
        out.append("")
    out.append("| configuration | time per step (cold pool) | effective GB/s | migration GB/s | roofline.frac (of the pinned-copy "
               "peak) | faults | scratch beside the pool | end-to-end GB/s | CPU oracle GB/s on host cores | scratch bounded to "
               "1/8 of the pool |")
    out.append("|---|---|---|---|---|---|---|---|---|---|")
    for cfg in sorted(recs, key=int):
        out.append(_row(cfg, recs[cfg]))
    return "\n".join(out)


def main(argv=None) -> int:
    argv = sys.argv[1:] if argv is None else argv
    text = open(argv[0]).read() if argv else sys.stdin.read()
    line = json.loads([l for l in text.splitlines() if l.startswith("{")][-1])
    print(table(line))
    extra = policies(line)
    if extra:
        print()
        print(extra)
    return 0


if __name__ == "__main__":
    sys.exit(main())
