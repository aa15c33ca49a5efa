"""Per-phase timeline of the persistent stack kernel on the benchmark's verify step.

    python -m paper_2607_04244_b200.timeline [--layers N] [--no-lm-head]
    python -m paper_2607_04244_b200.timeline --ablation-table

Builds the instrumented twin of the library (-DQL_TIMELINE: thread 0 of every thread block stamps
the phases of every fused operation with globaltimer), runs the benchmark step a few times and
prints, per kind of operation, where the time of one recorded step went.  The stamps cost a few
stores per operation; the regular library has none of them.

--ablation-table uses the regular library instead: it times the step with CUDA events while parts
of the kernel are switched off one at a time (the kernel's ablation switches; the outputs are then
garbage and are not looked at), which shows what each part costs without any stamp in the way.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def med_pos(v, present):
    v = v[present > 0]
    return float(np.median(v)) if v.size else float("nan")


def max_pos(v, present):
    v = v[present > 0]
    return float(v.max()) if v.size else float("nan")


ABLATIONS = (
    (0, "complete kernel"),
    (16, "rows published without the release fence"),
    (256, "watcher without its acquire fence"),
    (64, "no row epilogue (rows are published, nothing is stored)"),
    (32, "no accumulator exchange between the unpack groups"),
    (8, "split tiles not exchanged between thread blocks"),
    (2, "X operand not loaded or converted"),
    (2 | 4, "same, and the row scales 1/rms not awaited"),
    (1, "no weight copies, no unpacking, no MMAs"),
    (1 | 2 | 4, "no chunks, no X"),
    (1 | 2 | 4 | 8 | 32 | 64, "synchronisation skeleton only (dependency waits, barriers, publishing)"),
)


def ablation_table(args):
    import torch
    import paper_2607_04244_b200 as ql
    ql.load()
    import bench
    step = bench.VerifyStep(ql, torch, 16, 128, n_layers=args.layers, lm_head=not args.no_lm_head)
    n_ops = 4 * args.layers + (0 if args.no_lm_head else 1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    for mask, what in ABLATIONS:
        ql.ql_debug_set_ablate(mask)
        for _ in range(3):
            step.run()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            step.run()
        e1.record()
        torch.cuda.synchronize()
        rows.append((mask, what, e0.elapsed_time(e1) / args.steps))
    ql.ql_debug_set_ablate(0)
    step.run()
    torch.cuda.synchronize()
    assert ql.ql_device_status(step.ws) == ql.QL_OK
    full = rows[0][2]
    print(f"{n_ops} fused operations per step, {args.steps} steps per row, CUDA events")
    print(f"{'mask':>5s}  {'ms/step':>8s}  {'saved':>7s}  {'us/op':>6s}  what is switched off")
    for mask, what, ms in rows:
        print(f"{mask:5d}  {ms:8.3f}  {full - ms:7.3f}  {ms * 1e3 / n_ops:6.2f}  {what}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--ablation-table", action="store_true", help="time the step with parts of the kernel switched off (regular library)")
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--layers", type=int, default=36)
    ap.add_argument("--no-lm-head", action="store_true")
    ap.add_argument("--ablate", type=int, default=0, help="ablation mask of the stack kernel (timing experiments)")
    ap.add_argument("--json", default=None, help="also write the per-kind medians to this file")
    args = ap.parse_args()
    if args.ablation_table:
        return ablation_table(args)
    import torch
    from paper_2607_04244_b200 import build
    import paper_2607_04244_b200 as ql
    ql.load(build.build_library(timeline=True))
    assert ql.ql_debug_timeline_enabled()
    if args.ablate:
        ql.ql_debug_set_ablate(args.ablate)
    import bench
    step = bench.VerifyStep(ql, torch, 16, 128, n_layers=args.layers, lm_head=not args.no_lm_head)
    n_ops = 4 * args.layers + (0 if args.no_lm_head else 1)
    ncta = 160
    n_stamps = ncta * n_ops * 16
    buf = torch.zeros((n_stamps + 2 * ncta * 4 * 8 + ncta * n_ops,), dtype=torch.int64, device="cuda")
    for _ in range(3):
        step.run()
    torch.cuda.synchronize()
    ql.ql_debug_set_timeline(buf)
    step.run()
    torch.cuda.synchronize()
    ql.ql_debug_set_timeline(None)
    assert ql.ql_device_status(step.ws) == ql.QL_OK
    sm_mhz = torch.cuda.clock_rate() if hasattr(torch.cuda, "clock_rate") else 1965
    raw = buf.cpu().numpy()
    cyc = raw[n_stamps:n_stamps + ncta * 32].reshape(ncta, 4, 8).astype(np.float64)
    cyi = raw[n_stamps + ncta * 32:n_stamps + ncta * 64].reshape(ncta, 4, 8).astype(np.float64)
    gw = raw[n_stamps + ncta * 64:].reshape(ncta, n_ops).astype(np.float64)       # watcher saw the predecessor complete (ns)
    t = raw[:n_stamps].reshape(ncta, n_ops, 16).astype(np.float64)
    used = t[:, 0, 0] > 0
    cyc, cyi, t, gw = cyc[used], cyi[used], t[used], gw[used]
    gpub = t[:, :, 15].copy()                                # last row of the last segment published (ns)
    g0 = gpub[gpub > 0].min()
    gpub = np.where(gpub > 0, (gpub - g0) / 1e3, np.nan)
    gw = np.where(gw > 0, (gw - g0) / 1e3, np.nan)
    # SM cycles -> microseconds, relative to each thread block's own first stamp
    t = np.where(t > 0, (t - t[:, :1, :1]) / float(sm_mhz), np.nan)
    kinds = ["qkv", "o", "gate+up", "down"]
    names = [kinds[j % 4] for j in range(4 * args.layers)] + ([] if args.no_lm_head else ["lm_head"])
    end = np.nanmax(gpub, axis=0)                          # operation j published by every thread block
    mean = lambda v: float(np.nanmean(v)) if np.isfinite(v).any() else float("nan")
    vmax = lambda v: float(np.nanmax(v)) if np.isfinite(v).any() else float("nan")
    rows = {}
    for j in range(1 if n_ops > 1 else 0, n_ops):
        e = t[:, j, :]
        d = {
            "period (last publish to last publish)": end[j] - (end[j - 1] if j else 0.0),
            "watcher sees the predecessor complete, after its last publish (mean over thread blocks)": mean(gw[:, j]) - (end[j - 1] if j else 0.0),
            "same, last thread block": vmax(gw[:, j]) - (end[j - 1] if j else 0.0),
            "first chunk unpacked before X (mean)": mean(e[:, 1] - e[:, 0]),
            "waiting for the predecessor inside X duty (mean)": mean(e[:, 2] - e[:, 1]),
            "watcher sees it -> unpack threads notice (mean)": mean(e[:, 2] - e[:, 7]),
            "X build after the dependency (mean)": mean(e[:, 3] - e[:, 2]),
            "X build (max)": vmax(e[:, 3] - e[:, 2]),
            "last segment: chunks drained after X built (mean)": mean(e[:, 8] - e[:, 3]),
            "last segment: chunks drained after X built (max)": vmax(e[:, 8] - e[:, 3]),
            "last segment: accumulator exchange (mean)": mean(e[:, 9] - e[:, 8]),
            "owners of split tiles: exchange -> polling starts (mean)": mean(e[:, 10] - e[:, 9]),
            "owners of split tiles: exchange -> polling starts (max)": vmax(e[:, 10] - e[:, 9]),
            "owners: poll and add the contributors' rows (mean)": mean(e[:, 11] - e[:, 10]),
            "finishers: epilogue until stores issued (mean)": mean(e[:, 12] - e[:, 11]),
            "finishers: fence + publish (mean)": mean(e[:, 14] - e[:, 12]),
            "contributors: exchange -> partial sent (mean)": mean(np.where(np.isnan(e[:, 11]), e[:, 14] - e[:, 9], np.nan)),
            "operation entered -> last stamp (mean)": mean(e[:, 14] - e[:, 0]),
            "last thread block done after the mean one (global timer)": vmax(gpub[:, j]) - mean(gpub[:, j]),
        }
        rows.setdefault(names[j], []).append(d)
    total = end[-1]
    print(f"recorded step: {total:.1f} us from the first stamp to the last publish, {n_ops} fused operations, {t.shape[0]} thread blocks")
    out = {}
    for kind, lst in rows.items():
        print(f"\n{kind}  ({len(lst)} operations), mean over operations, microseconds")
        out[kind] = {}
        for key in lst[0]:
            v = float(np.nanmean([d[key] for d in lst]))
            out[kind][key] = v
            print(f"  {key:90s} {v:8.2f}")
    # cycle accounting of the unpack loop: per chunk of a group, averaged over groups and thread blocks
    chunks = cyc[:, :, 6].sum()
    names_c = ["wait for the ring stage", "wait for a free A buffer", "unpack + tcgen05.st issue", "tcgen05.wait::st",
               "wait for the MMAs of the chunk two back", "tcgen05.ld + scale-accumulate"]
    print(f"\nunpack loop, SM cycles per chunk of one group (4 groups work in parallel; {int(chunks)} group-chunks in the step)")
    out["unpack_cycles_per_group_chunk"] = {}
    for i, nm in enumerate(names_c):
        v = float(cyc[:, :, i].sum() / chunks)
        out["unpack_cycles_per_group_chunk"][nm] = v
        print(f"  {nm:66s} {v:8.0f}")
    halves = cyi[:, :, 3].sum()
    print("\nMMA issuers, SM cycles per half-chunk (4 MMAs + commit)")
    for i, nm in enumerate(["wait for the A buffer to be filled", "wait for X (first half of an operation)", "issue 4 MMAs + commit"]):
        print(f"  {nm:66s} {cyi[:, :, i].sum() / halves:8.0f}")
    if args.json:
        import json
        json.dump({"total_us": float(total), "kinds": out}, open(args.json, "w"), indent=1)


if __name__ == "__main__":
    main()
