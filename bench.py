#!/usr/bin/env python
"""Benchmark of the simulated quantized AllReduce (EQuARX hot path) on B200.

One "step" is one pass of the whole hot path -- ring step 0 (quantize), N-1
dequantize-add-requantize steps and the all-gather dequantize -- over one
batch of synthetic bf16 tensors, through the C ABI.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]

Prints ONE JSON line.  `value` is GB/s of bf16 input reduced (2 * count *
nranks bytes per step) with inputs resident in device memory, for the
single-launch (chain-fused) schedule; `by_steps` is the same work as one launch
per ring step, whose hop messages do travel through memory.  Each schedule
carries its own roofline: bytes it must move / CUDA-event time / measured HBM
peak.  `e2e` is the same metric through equarx_allreduce_sim_host: pinned host
buffers, the copies inside the timed region.  A train of K steps is timed
between CUDA events; trains are repeated until at least MIN_TIMED_SECONDS of
GPU time has been measured and the median train is reported.

With --gpus N > 1 (under torchrun) every rank runs an independent replica on
its own GPU (the path has no inter-GPU exchange): weak scaling, no collective
on the data path; NCCL carries the barrier and the max only.
`--impl reference` times the CPU oracle on a bounded sample instead.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "q-AllReduce GB/s (bf16 in) & % of HBM roofline on 1 B200, N simulated ranks"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
MIN_TIMED_SECONDS = 0.5
L2_BYTES = 126_000_000

# DRAM traffic measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum per launch, divided
# by the elements the launch processes: count*nranks for the whole AllReduce, count for one ring
# step), from the captures summarised under profiles/.  Traffic grows in proportion to the elements
# processed, so a full launch of another size is this figure times its elements.  Hop launches: the
# outgoing message stays in L2 while a step's messages (count * (1 + 4/block) bytes over all ranks)
# fit the part of L2 that keeps them, about 20 MB; above that it is written back and read again
# from DRAM.
NCU_TRAFFIC = {
    "chain_fused_kernel": {"bytes_per_element": 4.0, "profile": "profiles/chain_fused_kernel_c2_c3.md",
                           # read + written while the kernel runs, as captured (the rest of the outputs is still
                           # dirty in L2 when the kernel ends and is written back during the next launch)
                           "captured": {"C2_gemma3_12b_prefill2048": 125.85e6 + 68.15e6,
                                        "C3_gemma3_27b_prefill8192": 704.66e6 + 651.57e6}},
    "rs_step_hop_small": {"bytes_per_element": 3.06, "profile": "profiles/rs_step_kernel_c2_full.md"},
    "rs_step_hop_large": {"bytes_per_element": 3.95, "profile": "profiles/rs_step_kernel_c2_full.md"},
}
HOP_MESSAGES_STAY_IN_L2_BYTES = 20_000_000


def workload_by_name(name):
    """C1 | C2 | C3 | C5, or a point of the message-size sweep: sweep:<nranks>:<bytes per rank>:<block>:<dist>."""
    from paper_2506_17615_b200 import workloads as wl
    if name.startswith("sweep:"):
        _, n, nbytes, block, dist = name.split(":")
        return wl.sweep_point(int(n), int(nbytes), int(block), dist)
    table = {"C1": wl.C1, "C2": wl.C2, "C3": wl.C3, "C5": wl.C5}
    if name not in table:
        raise SystemExit(f"unknown workload {name}; choose from {sorted(table)} or sweep:N:bytes:block:dist")
    return table[name]


def input_sets(w):
    """How many input/output sets the timed steps rotate through, so that no step finds its
    inputs in L2; at least three, so that a launch allowed to overlap the tail of its predecessors
    (the `overlapped` leg) never shares a tensor with a launch that may still be running."""
    in_bytes = 2 * w.count * w.nranks
    return min(64, max(3, -(-3 * L2_BYTES // (2 * in_bytes))))


def base_config(w, world):
    """The workload description; identical for both arms of the bench."""
    sets = input_sets(w)
    in_bytes = 2 * w.count * w.nranks
    return {"workload": w.name, "nranks": w.nranks, "count_per_rank": w.count, "block": w.block, "dist": w.dist,
            "bytes_per_rank": 2 * w.count, "payload": "int8 codes + fp32 block scales", "io": "bf16",
            "parallelism": f"replicas x{world}" if world > 1 else "1 GPU",
            "l2": f"{sets} input/output set(s) used in rotation ({sets * 2 * in_bytes / 1e6:.0f} MB working set "
                  f"against a 126 MB L2); no explicit flush"}


def ring_schedule_bytes(n_ranks, count, block):
    """Minimum bytes the ring schedule moves: N bf16 reads, every hop message written and read
    once (N messages of count*(1+4/block) bytes each way), N bf16 writes: n*N*(6 + 8/B)."""
    wire = count * (1.0 + 4.0 / block)
    return 2.0 * count * n_ranks + 2.0 * n_ranks * wire + 2.0 * count * n_ranks


def chain_fused_bytes(n_ranks, count):
    """Bytes the single-launch chain-fused form must move: every input read once, every output
    written once (its hop messages never leave the registers): 4*n*N."""
    return 4.0 * count * n_ranks


def launch_bytes(kind, n_ranks, count, block):
    wire = count * (1.0 + 4.0 / block)
    if kind == "quantize_blocks":
        return 2.0 * count + wire
    if kind == "rs_step_dequant_add_requant":
        return 2.0 * count + 2.0 * wire
    return wire + 2.0 * count * n_ranks          # ag_dequant


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json: 6650 GB/s, an earlier B200 copy measurement)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the GPU works."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_id), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.perf_counter(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, windows):
        """windows: list of (t0, t1) host intervals during which the GPU was busy."""
        def parse(line):
            p = [s.strip() for s in line.split(",")]
            return float(p[0]), float(p[1]), p[3:7]
        rows = []
        for t, line in self.samples:
            if any(a <= t <= b for a, b in windows):
                try:
                    rows.append(parse(line))
                except Exception:
                    pass
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0,
                    "total_samples": len(self.samples)}
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = sorted({names[i] for _, _, fl in rows for i, v in enumerate(fl) if v.lower().startswith("active")})
        return {"sm_mhz": statistics.median(r[0] for r in rows), "sm_max_mhz": max(r[1] for r in rows),
                "reasons": reasons, "samples": len(rows), "total_samples": len(self.samples)}


def _gcd(a, b):
    while b:
        a, b = b, a % b
    return a


def _lcm(a, b):
    return a // _gcd(a, b) * b


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2506_17615_b200 import workloads as wl
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = workload_by_name(args.workload)
    unit = _lcm(w.hidden, w.nranks * w.block) if w.hidden else w.nranks * w.block   # whole token rows
    # calibrate on the smallest sample, then size a step so that the run ends in ~2 minutes
    x = wl.as_u16(wl.make_inputs(w, count=unit))
    t0 = time.perf_counter()
    oracle.allreduce(x, w.block)
    rate = unit * w.nranks / max(time.perf_counter() - t0, 1e-6)          # element-events per second
    budget = 120.0 / (args.steps + args.warmup)
    mult = max(1, min(w.count // unit, int(rate * budget / (unit * w.nranks))))
    count = unit * mult
    x = wl.as_u16(wl.make_inputs(w, count=count))
    for _ in range(args.warmup):
        oracle.allreduce(x, w.block)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.allreduce(x, w.block)
    dt = (time.perf_counter() - t0) / args.steps
    value = 2.0 * count * w.nranks / dt / 1e9
    sample = (f"first {count} of {w.count} elements per rank of {w.name} ({count * w.nranks} element-hops per "
              f"step), single thread")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": base_config(w, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline_and_parity(w, x_dev, out_dev):
    """The oracle on a bounded sample of the bench workload, on the host's cores, and, from the same
    oracle run, the parity verdict of the GPU outputs `out_dev` for the inputs `x_dev` ([N, count]).

    The sample is the whole workload when the oracle finishes it in about half a minute; else a set
    of whole blocks drawn from every shard (blocks are independent, so they form a smaller AllReduce
    whose outputs must equal the full problem's outputs at those blocks)."""
    import numpy as np
    import torch
    import oracle
    from paper_2506_17615_b200 import workloads as wl
    n, count, block = w.nranks, w.count, w.block
    max_events = 600_000_000                       # ~60 M element-hops per second on one core
    if count * n <= max_events:
        x = wl.as_u16(x_dev)
        got = wl.as_u16(out_dev)
        part = "the full workload"
    else:
        shard = count // n
        bps = shard // block
        m = max(1, min(bps, max_events // (n * n * block)))
        g = torch.Generator().manual_seed(12345)
        idx = []
        for k in range(n):
            pick = torch.randperm(bps, generator=g)[:m].sort().values
            idx.append((k * shard + pick[:, None] * block + torch.arange(block)[None, :]).reshape(-1))
        idx = torch.cat(idx).to(x_dev.device)
        x = wl.as_u16(x_dev[:, idx])
        got = wl.as_u16(out_dev[:, idx])
        part = f"{m} of {bps} blocks of every shard ({n * m * block} of {count} elements per rank)"
    oracle.allreduce(x[:, :n * block], block)      # loads the library
    reps, t_total, res = 0, 0.0, None
    while t_total < 10.0 and reps < 20:
        t0 = time.perf_counter()
        res = oracle.allreduce(x, block)
        t_total += time.perf_counter() - t0
        reps += 1
    dt = t_total / reps
    bad = int(np.count_nonzero(got != res["out"]))
    base = {"value": 2.0 * x.shape[1] * n / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{part} of {w.name}, {reps} passes, {dt:.3f} s per pass, single thread",
            "host_cores": os.cpu_count()}
    parity = {"against": "oracle", "checked_words": int(got.size), "of_words": n * count, "mismatches": bad,
              "verdict": "bit-exact" if bad == 0 else "MISMATCH", "sample": part}
    return base, parity


def max_over_ranks(ms, world, device):
    """Slowest rank's time: the job is as fast as its slowest replica."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    if dist.get_backend() == "gloo":
        device = torch.device("cpu")
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_rank_step, ms_step, world):
    """Whole-job GB/s: every replica reduces bytes_per_rank_step in ms_step (max over ranks)."""
    return world * bytes_per_rank_step / (ms_step * 1e-3) / 1e9


def roofline_entry(kernel, bytes_per_launch, ms_per_launch, peak, peak_src, traffic, traffic_src, model):
    achieved = bytes_per_launch / (ms_per_launch * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_src,
            "bytes_per_launch": bytes_per_launch, "bytes_model": model, "peak_source": peak_src,
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}


def run_ring(args):
    """--ring: the ring with one rank per GPU (equarx_ring_allreduce through PeerRing): every process
    is one rank, messages go into the neighbours' mailboxes over peer memory.  The number of ranks is
    the number of processes; each rank holds the workload's per-rank tensor.  Not exercised on more
    than one GPU: every device-side wait is bounded, so a rank that cannot reach its peers reports
    a time-out instead of hanging."""
    import torch
    import torch.distributed as dist
    from paper_2506_17615_b200 import workloads as wl
    from paper_2506_17615_b200.ring import PeerRing, RingTimeout
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    # the process group carries IPC handles, barriers and the max only; no multimem/NVLS is used anywhere
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    base = workload_by_name(args.workload)
    unit = _lcm(base.hidden, world * base.block) if base.hidden else world * base.block
    count = max(unit, base.count // unit * unit)
    w = wl.Workload(base.name + f"_ring{world}", world, count, base.block, base.dist, base.hidden, base.seed)
    x = wl.make_rank(w, rank, device=dev)
    out = torch.empty_like(x)
    ring = PeerRing(count, w.block)
    stream = torch.cuda.current_stream().cuda_stream
    timeout_ns = 2_000_000_000

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    failure = None
    try:
        for _ in range(args.warmup):
            ring.allreduce(x, out, timeout_ns, stream)
            ring.check()
        trains, total = [], 0.0
        while len(trains) < 3 or (total < args.min_seconds * 1e3 and len(trains) < 400):
            barrier()
            ev0.record()
            for _ in range(args.steps):
                ring.allreduce(x, out, timeout_ns, stream)
            ev1.record()
            torch.cuda.synchronize()
            ring.check()
            barrier()
            ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
            trains.append(ms)
            total += ms
        ms_step = statistics.median(trains) / args.steps
    except RingTimeout as exc:
        failure = str(exc)
        ms_step = float("nan")
    if rank == 0:
        peak, peak_src = hbm_peak()
        in_bytes = 2 * count * world
        wire = count * (1.0 + 4.0 / w.block) / world            # one shard's message
        # per rank: N local shard reads, N-1 messages stored to the right neighbour and N to everybody's
        # all-gather slot, as many read, N shard writes
        link_bytes = (world - 1) * wire + (world - 1) * wire     # crossing NVLink, per rank and direction
        line = {"metric": METRIC, "value": in_bytes / (ms_step * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {**base_config(w, 1), "parallelism": f"ring, one rank per GPU x{world}"},
                "schedule": "equarx_ring_allreduce, ranks_here=1 (peer mailboxes, per-tile flags)",
                "nvlink_bytes_per_rank_and_direction": link_bytes, "gpu_launches": args.steps,
                "failure": failure, "note": "not exercised on more than one GPU"}
        print(json.dumps(line))
    if failure is None:
        ring.close()
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the flavours and the bf16 comparator")
    ap.add_argument("--ring", action="store_true",
                    help="one rank of a real ring per process/GPU instead of independent replicas (opt-in)")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="GPU time to measure per schedule (trains of --steps steps are repeated); "
                         "0 for profiling runs: three trains only")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.steps < 1:
        args.steps = 1
    if args.impl == "reference":
        run_reference(args)
        return
    if args.ring:
        run_ring(args)
        return

    import torch
    import paper_2506_17615_b200 as eq
    from paper_2506_17615_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        try:
            dist.init_process_group("nccl", device_id=dev)
            dist.barrier()
        except Exception as exc:      # the data path has no collective: any backend can carry the barrier
            print(f"bench: NCCL unavailable ({exc!r}); using gloo for the barrier and the max", file=sys.stderr)
            if dist.is_initialized():
                dist.destroy_process_group()
            dist.init_process_group("gloo")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # started first: nvidia-smi needs a moment before its first sample
    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler(f"GPU-{props.uuid}" if hasattr(props, "uuid") else local)

    w = workload_by_name(args.workload)
    N, count, block = w.nranks, w.count, w.block
    in_bytes = 2 * count * N
    sets = input_sets(w)
    xs, os_, ins, outs = [], [], [], []
    for s in range(sets):
        src = wl.Workload(w.name, N, count, block, w.dist, w.hidden, seed=w.seed + s)
        x = wl.make_inputs(src, device=dev)
        o = torch.empty_like(x)
        xs.append(x)
        os_.append(o)
        ins.append([x[r] for r in range(N)])
        outs.append([o[r] for r in range(N)])
    checksum = int(xs[0].view(torch.int16).to(torch.int64).bitwise_and(0xFFFF).sum().item())
    wb = eq.allreduce_sim_workspace_bytes(N, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device=dev)
    wbp = eq.allreduce_sim_pipelined_workspace_bytes(N, count, block, False)
    wsp = torch.empty(wbp, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def step_fused(i):           # the headline: the whole AllReduce as one chain-fused launch
        eq.allreduce_sim_pipelined(ins[i % sets], outs[i % sets], N, count, block, wsp, wbp, False, stream)

    def step_by_steps(i):        # one launch per ring step (N+1 launches)
        eq.allreduce_sim(ins[i % sets], outs[i % sets], N, count, block, ws, wb, False, stream)

    windows = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(step_fn, steps, min_seconds=None, max_trains=400):
        """Trains of exactly `steps` steps between CUDA events on the launching stream, each bracketed
        by a barrier + synchronize on both sides and reduced to the max over ranks; repeated until
        min_seconds of GPU time has been measured.  Returns (median ms per step, trains)."""
        if min_seconds is None:
            min_seconds = args.min_seconds
        min_seconds = min(min_seconds, args.min_seconds)
        for i in range(args.warmup):
            step_fn(i)
        trains, total = [], 0.0
        h0 = time.perf_counter()
        while len(trains) < 3 or (total < min_seconds * 1e3 and len(trains) < max_trains):
            barrier()
            ev0.record()
            for i in range(steps):
                step_fn(i)
            ev1.record()
            torch.cuda.synchronize()
            barrier()
            ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
            trains.append(ms)
            total += ms
        windows.append((h0, time.perf_counter()))
        return statistics.median(trains) / steps, len(trains)

    peak, peak_src = hbm_peak()

    # ---- headline: the chain-fused single launch; a timed train is exactly K launches of one kernel
    ms_step, trains = timed(step_fused, args.steps)
    value = aggregate_value(in_bytes, ms_step, world)
    t = NCU_TRAFFIC["chain_fused_kernel"]
    roofline = roofline_entry(
        "chain_fused_kernel", chain_fused_bytes(N, count), ms_step, peak, peak_src,
        t["captured"].get(w.name, t["bytes_per_element"] * count * N),
        f"ncu, {t['profile']}" + (", this workload, inside the kernel" if w.name in t["captured"] else ", scaled by elements"),
        "4*count*nranks: every bf16 input read once, every bf16 output written once; hop messages stay in registers")
    roofline["ring_schedule_bytes_per_launch"] = ring_schedule_bytes(N, count, block)
    roofline["note"] = ("frac counts only bytes this kernel moves through HBM; against the ring schedule's "
                        "count*nranks*(6+8/block) bytes the same time would read "
                        f"{ring_schedule_bytes(N, count, block) / (ms_step * 1e-3) / 1e9 / peak:.3f} of peak, "
                        "which is not a fraction of anything this kernel does")

    # ---- the same work as one launch per ring step: the hop messages go through memory
    ms_steps, trains_steps = timed(step_by_steps, args.steps)
    # per-kernel durations: trains of launches between CUDA events, in stream order.  Launch 0
    # (quantize) and launch N (all-gather) are idempotent and are repeated 4 times per train so
    # that the events' own overhead is amortised; launches 1..N-1 (the hops) form one train.
    ktrains = [("quantize_blocks", 0, 0, 4, 4)]
    if N > 1:
        ktrains.append(("rs_step_dequant_add_requant", 1, N - 1, 1, N - 1))
    ktrains.append(("ag_dequant", N, N, 4, 4))
    reps = max(5, min(50, args.steps))
    evs = {t_[0]: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(reps)] for t_ in ktrains}
    h0 = time.perf_counter()
    passes = 0
    while passes < 3 or (time.perf_counter() - h0 < args.min_seconds and passes < 2000):   # also gives the clock sampler load
        for i in range(reps):
            for name, first, last, repeat, _ in ktrains:
                a, b = evs[name][i]
                a.record()
                for _ in range(repeat):
                    eq.allreduce_sim_range(ins[i % sets], outs[i % sets], N, count, block, ws, wb, False,
                                           first, last, stream)
                b.record()
        torch.cuda.synchronize()
        passes += 1
    windows.append((h0, time.perf_counter()))
    kernels = {}
    train_ms = {t_[0]: sum(a.elapsed_time(b) for a, b in evs[t_[0]]) for t_ in ktrains}     # last pass
    per_step_ms = {}
    for name, first, last, repeat, launches in ktrains:
        avg_ms = train_ms[name] / (reps * launches)
        per_step = last - first + 1
        per_step_ms[name] = avg_ms * per_step
        kernels[name] = {"launches_per_step": per_step, "avg_us": avg_ms * 1e3,
                         "algorithmic_gbs": launch_bytes(name, N, count, block) / (avg_ms * 1e-3) / 1e9}
    for name in kernels:
        kernels[name]["share"] = per_step_ms[name] / sum(per_step_ms.values())
        kernels[name]["frac"] = kernels[name]["algorithmic_gbs"] / peak
    hop = NCU_TRAFFIC["rs_step_hop_small" if count * (1 + 4.0 / block) <= HOP_MESSAGES_STAY_IN_L2_BYTES
                      else "rs_step_hop_large"]
    by_steps = {"value": aggregate_value(in_bytes, ms_steps, world), "unit": UNIT, "ms_per_step": ms_steps,
                "trains": trains_steps, "gpu_launches_per_step": N + 1,
                "roofline": roofline_entry(
                    "rs_step_kernel x N + ag_dequant_kernel (whole step)", ring_schedule_bytes(N, count, block),
                    ms_steps, peak, peak_src, None, "not captured for the whole step",
                    "count*nranks*(6+8/block): N bf16 reads, every hop message written and read once, N bf16 writes"),
                "kernels": kernels,
                "hop_traffic_bytes_per_launch": hop["bytes_per_element"] * count,
                "hop_traffic_source": f"ncu, {hop['profile']}, scaled by elements"}

    flavours, bf16_sim, ratios, ring_local, graph_replay, overlapped = {}, None, None, None, None, None
    if not args.no_extras:
        # ---- the other flavours (semi-loop ring, stage selection, FP8), same workload, single launch
        wbf = eq.allreduce_sim_flavour_workspace_bytes(N, count, block, 7 if N % 2 == 0 else 6, False)
        wsf = torch.empty(wbf, dtype=torch.uint8, device=dev)
        names = {0: "full_loop_unquantized", 2: "full_loop_rs_only", 4: "full_loop_ag_only", 6: "full_loop_rs_ag",
                 1: "semi_loop_unquantized", 3: "semi_loop_rs_only", 5: "semi_loop_ag_only", 7: "semi_loop_rs_ag",
                 6 | 8: "full_loop_rs_ag_fp8_e4m3", 6 | 16: "full_loop_rs_ag_fp8_e5m2"}
        for fl, name in sorted(names.items()):
            if (fl & 1) and N % 2:
                continue
            ms_f, _ = timed(lambda i, fl=fl: eq.allreduce_sim_flavour(ins[i % sets], outs[i % sets], N, count, block,
                                                                      fl, wsf, wbf, False, stream),
                            max(5, min(50, args.steps)), min_seconds=0.1)
            flavours[name] = {"ms_per_step": ms_f, "value": aggregate_value(in_bytes, ms_f, world), "unit": UNIT}
        del wsf

        # ---- the ring with one rank per device, all ranks hosted by this GPU (mailboxes + per-tile flags)
        from paper_2506_17615_b200.ring import LocalRing
        lring = LocalRing(N, count, block, dev)

        def step_ring(i):
            lring.allreduce(ins[i % sets], outs[i % sets], 0, stream)

        ms_r, _ = timed(step_ring, max(5, min(50, args.steps)), min_seconds=0.2)
        lring.check()
        wire = count * (1.0 + 4.0 / block)
        ring_bytes = 4.0 * count * N + 2.0 * (N - 1) * wire + 2.0 * N * wire
        ring_local = {"ms_per_step": ms_r, "value": aggregate_value(in_bytes, ms_r, world), "unit": UNIT,
                      "schedule": "equarx_ring_allreduce, all ranks hosted by one cooperative launch",
                      "bytes_per_launch": ring_bytes,
                      "bytes_model": "inputs and outputs once; N-1 reduce-scatter messages per shard written and read "
                                     "once; the all-gather message of every shard written to and read from N mailboxes",
                      "frac": ring_bytes / (ms_r * 1e-3) / 1e9 / peak}
        del lring

        # ---- the single launch when consecutive calls are independent (they are here: each step has its own
        # tensors): equarx_allreduce_sim_pipelined_unordered starts while its predecessor is still finishing
        def step_unordered(i):
            eq.allreduce_sim_pipelined_unordered(ins[i % sets], outs[i % sets], N, count, block, stream)

        ms_u, _ = timed(step_unordered, args.steps, min_seconds=0.3)
        overlapped = {"ms_per_step": ms_u, "value": aggregate_value(in_bytes, ms_u, world), "unit": UNIT,
                      "schedule": "equarx_allreduce_sim_pipelined_unordered: same kernel, not ordered after the "
                                  "stream's unfinished earlier work (the steps use disjoint tensors)",
                      "achieved": chain_fused_bytes(N, count) / (ms_u * 1e-3) / 1e9,
                      "frac": chain_fused_bytes(N, count) / (ms_u * 1e-3) / 1e9 / peak,
                      "note": "above 1.0 of the measured copy bandwidth is possible here: the copy the peak was measured "
                              "with pays the launch boundaries that this mode overlaps"}

        # ---- both schedules recorded once per input set by stream capture and replayed as CUDA graphs
        # (removes the host-call and launch overhead that bounds small messages)
        graph_replay = {}
        for gname, fn in (("single_launch", step_fused), ("by_steps", step_by_steps)):
            graphs = []
            side = torch.cuda.Stream(dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for s_ in range(sets):
                    g_ = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g_, stream=side):
                        capture_stream = torch.cuda.current_stream().cuda_stream
                        if gname == "single_launch":
                            eq.allreduce_sim_pipelined(ins[s_], outs[s_], N, count, block, wsp, wbp, False, capture_stream)
                        else:
                            eq.allreduce_sim(ins[s_], outs[s_], N, count, block, ws, wb, False, capture_stream)
                    graphs.append(g_)
            torch.cuda.current_stream().wait_stream(side)
            ms_g, _ = timed(lambda i: graphs[i % sets].replay(), args.steps, min_seconds=0.2)
            graph_replay[gname] = {"ms_per_step": ms_g, "value": aggregate_value(in_bytes, ms_g, world), "unit": UNIT}
            del graphs

        # ---- unquantized comparator on the same GPU, same inputs, one launch per ring step
        wb16 = eq.allreduce_sim_bf16_workspace_bytes(N, count)
        ws16 = torch.empty(wb16, dtype=torch.uint8, device=dev)
        ms16, _ = timed(lambda i: eq.allreduce_sim_bf16(ins[i % sets], outs[i % sets], N, count, ws16, wb16, stream),
                        args.steps, min_seconds=0.2)
        bf16_sim = {"value": aggregate_value(in_bytes, ms16, world), "unit": UNIT, "ms_per_step": ms16,
                    "schedule": "one launch per ring step",
                    "algorithmic_bytes_per_step": count * (8 * N - 4),
                    "frac_of_measured_peak": count * (8 * N - 4) / (ms16 * 1e-3) / 1e9 / peak}
        del ws16
        # like for like: the same schedule form on both sides of each ratio
        ratios = {"single_launch_quantized_over_single_launch_bf16":
                      flavours["full_loop_unquantized"]["ms_per_step"] / ms_step,
                  "per_step_quantized_over_per_step_bf16": ms16 / ms_steps}

    # ---- end to end through the C ABI's host-buffer entry: every step uploads its N input tensors
    # from pinned host memory, reduces them and downloads the N outputs.  Two streams and two staging
    # buffers, used alternately, so that one step's upload overlaps the previous step's download.
    e2e = None
    if not args.no_e2e:
        h_in = [torch.empty((N, count), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        for i, h in enumerate(h_in):
            h.copy_(xs[i % sets])
        h_out = [torch.empty((N, count), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        sb = eq.allreduce_sim_host_staging_bytes(N, count)
        stage = [torch.empty(sb, dtype=torch.uint8, device=dev) for _ in range(2)]
        side = [torch.cuda.Stream(dev) for _ in range(2)]

        def host_step(i):
            eq.allreduce_sim_host([h_in[i % 2][r] for r in range(N)], [h_out[i % 2][r] for r in range(N)], N, count,
                                  block, stage[i % 2], sb, side[i % 2].cuda_stream)

        e_steps = max(3, min(10, args.steps))
        for i in range(3):
            host_step(i)
        barrier()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream()
        h0 = time.perf_counter()
        t0.record(cur)
        for s_ in side:
            s_.wait_event(t0)
        for i in range(e_steps):
            host_step(i)
        for s_ in side:
            cur.wait_stream(s_)
        t1.record(cur)
        torch.cuda.synchronize()
        windows.append((h0, time.perf_counter()))
        barrier()
        ms_e = max_over_ranks(t0.elapsed_time(t1), world, dev) / e_steps
        e2e = {"value": aggregate_value(in_bytes, ms_e, world), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
               "d2h_bytes_per_step": in_bytes, "ms_per_step": ms_e, "steps": e_steps,
               "api": "equarx_allreduce_sim_host (C ABI, host pointers); two streams and staging buffers in rotation"}
        del h_in, h_out, stage

    sampler.stop()
    clocks = sampler.summary(windows)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "trains": trains, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": base_config(w, world),
            "e2e": e2e, "gpu_launches": args.steps, "clocks": clocks,
            "roofline": roofline,
            "schedule": "chain-fused single launch (equarx_allreduce_sim_pipelined, keep_trace=0)",
            "by_steps": by_steps, "ring_on_one_gpu": ring_local, "graph_replay": graph_replay, "overlapped": overlapped, "flavours": flavours, "bf16_sim": bf16_sim,
            "speedup_vs_bf16": ratios, "input_checksum": checksum,
            "pdl_between_step_launches": os.environ.get("EQUARX_PDL", "1") != "0",
        }
        if world == 1 and not args.no_cpu_baseline:
            # the outputs of the last chain-fused step on set 0 are recomputed so that the parity verdict
            # belongs to the kernel that was timed
            step_fused(0)
            torch.cuda.synchronize()
            line["cpu_baseline"], line["parity"] = cpu_baseline_and_parity(w, xs[0], os_[0])
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
