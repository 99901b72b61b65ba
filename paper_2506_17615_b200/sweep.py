"""Message-size sweep of the simulated quantized AllReduce (config 4 of the benchmark definition).

    python -m paper_2506_17615_b200.sweep [--out sweep.jsonl] [--quick]

For every point (N in {4, 8, 16}, block in {128, 256, 512}, uniform(-1,1) and N(0,1), per-rank
messages from 16 KB to 256 MB in powers of two) it times, with CUDA events and inputs resident in
device memory, the single-launch (chain-fused) schedule, the launch-per-step schedule and the
unquantized bf16 ring, and prints one JSON line per point: GB/s of bf16 input reduced and the
fraction of the HBM roofline, each schedule against the bytes it must move: 4*n*N for the single
launch (inputs once, outputs once; its hop messages stay in registers), n*N*(6+8/B) for the
launch-per-step schedule, n*(8N-4) for the bf16 ring, over the measured copy bandwidth.  Inputs
rotate over several resident sets so that consecutive iterations do not find their inputs in L2.
"""
import argparse
import json
import os
import sys

import torch

import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import workloads as wl


def hbm_peak_gbs():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    try:
        with open(os.path.join(root, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def time_ms(fn, iters, warmup=3):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(iters):
        fn(i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / iters


def run_point(n_ranks, nbytes, block, dist, peak):
    w = wl.sweep_point(n_ranks, nbytes, block, dist)
    count = w.count
    if count % (n_ranks * block):
        return None
    in_bytes = 2 * count * n_ranks
    sets = 1 if in_bytes > 1_000_000_000 else min(16, max(2, -(-378_000_000 // (2 * in_bytes))))
    base = wl.make_inputs(w, device="cuda")
    ins, outs = [], []
    for s in range(sets):
        x = base if s == 0 else base.roll(s * 4096, dims=1).contiguous()    # same values, other addresses
        ins.append([x[r] for r in range(n_ranks)])
        o = torch.empty_like(x)
        outs.append([o[r] for r in range(n_ranks)])
    stream = torch.cuda.current_stream().cuda_stream
    wb = eq.allreduce_sim_workspace_bytes(n_ranks, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    wbp = eq.allreduce_sim_pipelined_workspace_bytes(n_ranks, count, block, False)
    wsp = torch.empty(wbp, dtype=torch.uint8, device="cuda")
    wb16 = eq.allreduce_sim_bf16_workspace_bytes(n_ranks, count)
    ws16 = torch.empty(wb16, dtype=torch.uint8, device="cuda")
    iters = max(5, min(200, int(2e9 // max(in_bytes, 1))))
    t_pipe = time_ms(lambda i: eq.allreduce_sim_pipelined(ins[i % sets], outs[i % sets], n_ranks, count, block,
                                                          wsp, wbp, False, stream), iters)
    t_steps = time_ms(lambda i: eq.allreduce_sim(ins[i % sets], outs[i % sets], n_ranks, count, block,
                                                 ws, wb, False, stream), iters)
    t_bf16 = time_ms(lambda i: eq.allreduce_sim_bf16(ins[i % sets], outs[i % sets], n_ranks, count,
                                                     ws16, wb16, stream), iters)
    alg = count * n_ranks * (6 + 8 / block)
    fused = 4 * count * n_ranks
    alg16 = count * (8 * n_ranks - 4)
    gbs = lambda nbytes_, ms: nbytes_ / (ms * 1e-3) / 1e9
    return {"nranks": n_ranks, "bytes_per_rank": nbytes, "block": block, "dist": dist, "iters": iters, "sets": sets,
            "pipelined": {"ms": t_pipe, "gbs_in": gbs(in_bytes, t_pipe), "frac": gbs(fused, t_pipe) / peak},
            "by_steps": {"ms": t_steps, "gbs_in": gbs(in_bytes, t_steps), "frac": gbs(alg, t_steps) / peak},
            "bf16_sim": {"ms": t_bf16, "gbs_in": gbs(in_bytes, t_bf16), "frac": gbs(alg16, t_bf16) / peak}}


def summarize(path):
    """Markdown summary of a sweep file written with --out."""
    rows = [json.loads(line) for line in open(path)]
    peak = rows[0]["peak_gbs"]
    out = ["# Message-size sweep (config 4): GB/s of bf16 input reduced and fraction of the HBM roofline",
           "",
           "Command: `python -m paper_2506_17615_b200.sweep --out sweep.jsonl` on one B200 (CUDA events, inputs resident,",
           "several input/output sets in rotation), then `--summarize sweep.jsonl`. Fraction = bytes the schedule must move",
           "(single launch, chain-fused: 4*n*N; launch per step: n*N*(6+8/B); bf16 comparator: n*(8N-4)) over time,",
           f"divided by the {rows[0]['peak_source']} HBM copy bandwidth {peak:.1f} GB/s.",
           f"{len(rows)} points; the table lists N(0,1) data (uniform(-1,1) is within a few percent).",
           "",
           "| N | block | bytes per rank | single launch GB/s (frac) | launch per step GB/s (frac) | bf16 ring per step GB/s (frac) |",
           "|---|---|---|---|---|---|"]
    shown = (1 << 14, 1 << 17, 1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 27, 1 << 28)
    for r in rows:
        if r["dist"] != "normal" or r["bytes_per_rank"] not in shown:
            continue
        p, st, b, sz = r["pipelined"], r["by_steps"], r["bf16_sim"], r["bytes_per_rank"]
        size = f"{sz >> 20} MB" if sz >= 1 << 20 else f"{sz >> 10} KB"
        out.append(f"| {r['nranks']} | {r['block']} | {size} | {p['gbs_in']:.0f} ({p['frac']:.3f}) | "
                   f"{st['gbs_in']:.0f} ({st['frac']:.3f}) | {b['gbs_in']:.0f} ({b['frac']:.3f}) |")
    big = [r for r in rows if r["bytes_per_rank"] >= 64 << 20]
    if big:
        lo = lambda key: min(r[key]["frac"] for r in big)
        hi = lambda key: max(r[key]["frac"] for r in big)
        out += ["",
                f"All {len(big)} points with at least 64 MB per rank: single launch {lo('pipelined'):.3f} - {hi('pipelined'):.3f} of the "
                f"measured peak ({lo('pipelined') * peak / 8000:.3f} - {hi('pipelined') * peak / 8000:.3f} of the nominal 8 TB/s); "
                f"launch per step {lo('by_steps'):.3f} - {hi('by_steps'):.3f} of measured "
                f"({lo('by_steps') * peak / 8000:.3f} - {hi('by_steps') * peak / 8000:.3f} of nominal). Below about 2 MB per rank "
                "every schedule is launch- and latency-bound (the paper sees the same below 2 MiB, Section 4); the single-launch "
                "schedule needs one launch instead of N+1 there."]
    return "\n".join(out) + "\n"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--quick", action="store_true", help="block 256 and N(0,1) only")
    ap.add_argument("--summarize", default=None, metavar="FILE", help="print a markdown summary of a sweep file and exit")
    args = ap.parse_args()
    if args.summarize:
        print(summarize(args.summarize), end="")
        return 0
    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device")
    peak, src = hbm_peak_gbs()
    out = open(args.out, "w") if args.out else None
    blocks = (256,) if args.quick else (128, 256, 512)
    dists = ("normal",) if args.quick else ("uniform", "normal")
    for n_ranks in (4, 8, 16):
        for block in blocks:
            for dist in dists:
                for p in range(14, 29):
                    rec = run_point(n_ranks, 1 << p, block, dist, peak)
                    if rec is None:
                        continue
                    rec["peak_gbs"], rec["peak_source"] = peak, src
                    line = json.dumps(rec)
                    print(line, flush=True)
                    if out:
                        out.write(line + "\n")
                        out.flush()
                    torch.cuda.empty_cache()
    if out:
        out.close()


if __name__ == "__main__":
    sys.exit(main())
