#!/usr/bin/env python
"""Benchmark of the simulated quantized AllReduce (EQuARX hot path) on B200.

One "step" is one pass of the whole hot path -- ring step 0 (quantize), N-1
dequantize-add-requantize steps and the all-gather dequantize -- over one
batch of synthetic bf16 tensors, through the C ABI (equarx_allreduce_sim).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--impl ours|reference]

Prints ONE JSON line.  `value` is GB/s of bf16 input reduced (2 * count *
nranks bytes per step) with inputs resident in device memory; `e2e` is the
same metric with pinned host buffers and the copies inside the timed region.
With --gpus N > 1 (under torchrun) every rank runs an independent replica
on its own GPU (the path has no inter-GPU exchange): weak scaling, no
collective on the data path; NCCL is used for the barrier and the max only.
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

# DRAM traffic of one dequantize-add-requantize launch per element of a rank's shard,
# from the ncu capture summarised in profiles/ (dram__bytes_read.sum + dram__bytes_write.sum
# divided by the elements per rank; cold L2, so both inputs come from DRAM and the outgoing
# message stays in L2).
DAR_TRAFFIC_BYTES_PER_ELEMENT = 3.017
# DRAM traffic of one pipelined launch per element of every rank (ncu, profiles/): the N inputs
# are read once and the N outputs written once; hop messages never leave L2.
PIPELINED_TRAFFIC_BYTES_PER_RANK_ELEMENT = 4.0


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


def base_config(w):
    """The workload description shared by both arms of the bench."""
    return {"workload": w.name, "nranks": w.nranks, "count_per_rank": w.count, "block": w.block, "dist": w.dist,
            "bytes_per_rank": 2 * w.count, "payload": "int8 codes + fp32 block scales", "io": "bf16"}


def algorithmic_bytes(n_ranks, count, block):
    """Minimum bytes the schedule moves: N bf16 reads, every hop message written and read
    once (N messages of count*(1+4/block) bytes each way), N bf16 writes."""
    wire = count * (1.0 + 4.0 / block)
    return 2.0 * count * n_ranks + 2.0 * n_ranks * wire + 2.0 * count * n_ranks


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
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


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


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2506_17615_b200 import workloads as wl
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
    sample = f"first {count} of {w.count} elements per rank of {w.name} ({count * w.nranks} element-hops per step)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": dict(base_config(w), sample_count_per_rank=count),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def _gcd(a, b):
    while b:
        a, b = b, a % b
    return a


def _lcm(a, b):
    return a // _gcd(a, b) * b


def cpu_baseline(w):
    """The oracle on a bounded sample of the bench workload, on this machine's host cores."""
    import oracle
    from paper_2506_17615_b200 import workloads as wl
    count = w.count
    # ~60 M element-hops per second on one core: keep the sample near 10-30 s
    max_events = 600_000_000
    if count * w.nranks > max_events:
        unit = _lcm(w.hidden, w.nranks * w.block) if w.hidden else w.nranks * w.block
        count = max(unit, max_events // w.nranks // unit * unit)
    x = wl.as_u16(wl.make_inputs(w, count=count))
    oracle.allreduce(x[:, :w.nranks * w.block], w.block)      # loads the library
    reps, t_total = 0, 0.0
    while t_total < 10.0 and reps < 20:
        t0 = time.perf_counter()
        oracle.allreduce(x, w.block)
        t_total += time.perf_counter() - t0
        reps += 1
    dt = t_total / reps
    part = "the full workload" if count == w.count else f"the first {count} of {w.count} elements per rank"
    return {"value": 2.0 * count * w.nranks / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{part} of {w.name}, {reps} passes, {dt:.3f} s per pass, single thread",
            "host_cores": os.cpu_count()}


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
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
    # inputs of consecutive steps differ, so no step finds its inputs in the 126 MB L2
    sets = 1 if in_bytes > 1_000_000_000 else min(64, max(2, -(-378_000_000 // (2 * in_bytes))))
    ins, outs = [], []
    for s in range(sets):
        src = wl.Workload(w.name, N, count, block, w.dist, w.hidden, seed=w.seed + s)
        x = wl.make_inputs(src, device=dev)
        ins.append([x[r] for r in range(N)])
        o = torch.empty_like(x)
        outs.append([o[r] for r in range(N)])
    wb = eq.allreduce_sim_workspace_bytes(N, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device=dev)
    wbp = eq.allreduce_sim_pipelined_workspace_bytes(N, count, block, False)
    wsp = torch.empty(wbp, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def step_pipelined(i):       # the headline: one deep-pipelined launch per step
        eq.allreduce_sim_pipelined(ins[i % sets], outs[i % sets], N, count, block, wsp, wbp, False, stream)

    def step_by_steps(i):        # one launch per ring step (N+1 launches)
        eq.allreduce_sim(ins[i % sets], outs[i % sets], N, count, block, ws, wb, False, stream)

    windows = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(step_fn, steps):
        for i in range(args.warmup):
            step_fn(i)
        barrier()
        h0 = time.perf_counter()
        ev0.record()
        for i in range(steps):
            step_fn(i)
        ev1.record()
        torch.cuda.synchronize()
        windows.append((h0, time.perf_counter()))
        barrier()
        return max_over_ranks(ev0.elapsed_time(ev1), world, dev) / steps

    peak, peak_src = hbm_peak()
    alg_bytes = algorithmic_bytes(N, count, block)

    # ---- headline: the pipelined schedule; the timed region is exactly K launches of one kernel
    ms_step = timed(step_pipelined, args.steps)
    value = aggregate_value(in_bytes, ms_step, world)
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    traffic = PIPELINED_TRAFFIC_BYTES_PER_RANK_ELEMENT * count * N
    roofline = {"bound": "hbm", "kernel": "pipelined_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": alg_bytes,
                "dram_gbs": traffic / (ms_step * 1e-3) / 1e9, "dram_frac": traffic / (ms_step * 1e-3) / 1e9 / peak,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "note": "hop messages are written through to L2 and consumed at once from the SM's L1/L2, so DRAM "
                        "traffic (inputs + outputs) is below the algorithmic bytes and frac can exceed 1"}

    # ---- the same work as one launch per ring step
    ms_steps = timed(step_by_steps, args.steps)
    # per-kernel durations: trains of launches between CUDA events, in stream order.  Launch 0
    # (quantize) and launch N (all-gather) are idempotent and are repeated 4 times per train so
    # that the events' own overhead is amortised; launches 1..N-1 (the hops) form one train.
    trains = [("quantize_blocks", 0, 0, 4, 4)]
    if N > 1:
        trains.append(("rs_step_dequant_add_requant", 1, N - 1, 1, N - 1))
    trains.append(("ag_dequant", N, N, 4, 4))
    reps = max(5, min(50, args.steps))
    evs = {t[0]: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                  for _ in range(reps)] for t in trains}
    h0 = time.perf_counter()
    passes = 0
    while passes < 3 or (time.perf_counter() - h0 < 0.5 and passes < 2000):   # also gives the clock sampler load
        for i in range(reps):
            for name, first, last, repeat, _ in trains:
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
    train_ms = {t[0]: sum(a.elapsed_time(b) for a, b in evs[t[0]]) for t in trains}     # last pass
    per_step_ms = {}
    for name, first, last, repeat, launches in trains:
        avg_ms = train_ms[name] / (reps * launches)
        per_step = last - first + 1
        per_step_ms[name] = avg_ms * per_step
        kernels[name] = {"launches_per_step": per_step, "avg_us": avg_ms * 1e3,
                         "algorithmic_gbs": launch_bytes(name, N, count, block) / (avg_ms * 1e-3) / 1e9}
    for name in kernels:
        kernels[name]["share"] = per_step_ms[name] / sum(per_step_ms.values())
        kernels[name]["frac"] = kernels[name]["algorithmic_gbs"] / peak
    steps_gbs = alg_bytes / (ms_steps * 1e-3) / 1e9
    by_steps = {"value": aggregate_value(in_bytes, ms_steps, world), "unit": UNIT, "ms_per_step": ms_steps,
                "gpu_launches_per_step": N + 1, "algorithmic_gbs": steps_gbs, "frac": steps_gbs / peak,
                "frac_of_nominal_8TBs": steps_gbs / NOMINAL_HBM_GBS, "kernels": kernels,
                "hop_traffic_bytes_per_launch": DAR_TRAFFIC_BYTES_PER_ELEMENT * count}

    # ---- the other flavours (semi-loop ring, stage selection), same workload, pipelined form
    flavours = {}
    wbf = eq.allreduce_sim_flavour_workspace_bytes(N, count, block, 7 if N % 2 == 0 else 6, False)
    wsf = torch.empty(wbf, dtype=torch.uint8, device=dev)
    names = {0: "full_loop_unquantized", 2: "full_loop_rs_only", 4: "full_loop_ag_only", 6: "full_loop_rs_ag",
             1: "semi_loop_unquantized", 3: "semi_loop_rs_only", 5: "semi_loop_ag_only", 7: "semi_loop_rs_ag",
             6 | 8: "full_loop_rs_ag_fp8_e4m3", 6 | 16: "full_loop_rs_ag_fp8_e5m2"}
    for fl, name in sorted(names.items()):
        if (fl & 1) and N % 2:
            continue
        ms_f = timed(lambda i, fl=fl: eq.allreduce_sim_flavour(ins[i % sets], outs[i % sets], N, count, block, fl,
                                                               wsf, wbf, False, stream), max(5, min(200, args.steps)))
        flavours[name] = {"ms_per_step": ms_f, "value": aggregate_value(in_bytes, ms_f, world), "unit": UNIT}
    del wsf

    # unquantized comparator on the same GPU, same inputs
    wb16 = eq.allreduce_sim_bf16_workspace_bytes(N, count)
    ws16 = torch.empty(wb16, dtype=torch.uint8, device=dev)
    for i in range(args.warmup):
        eq.allreduce_sim_bf16(ins[i % sets], outs[i % sets], N, count, ws16, wb16, stream)
    torch.cuda.synchronize()
    h0 = time.perf_counter()
    ev0.record()
    for i in range(args.steps):
        eq.allreduce_sim_bf16(ins[i % sets], outs[i % sets], N, count, ws16, wb16, stream)
    ev1.record()
    torch.cuda.synchronize()
    windows.append((h0, time.perf_counter()))
    ms16 = max_over_ranks(ev0.elapsed_time(ev1), world, dev) / args.steps
    bf16_sim = {"value": in_bytes / (ms16 * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms16,
                "algorithmic_bytes_per_step": count * (8 * N - 4),
                "frac_of_measured_peak": count * (8 * N - 4) / (ms16 * 1e-3) / 1e9 / peak}
    del ws16

    # end to end through the host-buffer front end: every step uploads its N input tensors from
    # pinned host memory, runs the AllReduce and downloads the N outputs; copies of neighbouring
    # steps overlap with the kernels (three streams, two device buffer sets)
    e2e = None
    if not args.no_e2e:
        from paper_2506_17615_b200.host_api import HostPipeline
        h_in = [torch.empty((N, count), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        for i, h in enumerate(h_in):
            h.copy_(torch.stack(ins[i % sets]).cpu())
        h_out = [torch.empty((N, count), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        pipe = HostPipeline(N, count, block, dev)
        e_steps = max(3, min(20, args.steps))
        for i in range(3):
            pipe.submit(h_in[i % 2], h_out[i % 2])
        pipe.wait()
        barrier()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        pipe.h2d.wait_event(t0)
        for i in range(e_steps):
            pipe.submit(h_in[i % 2], h_out[i % 2])
        torch.cuda.current_stream().wait_stream(pipe.d2h)
        torch.cuda.current_stream().wait_stream(pipe.comp)
        t1.record()
        torch.cuda.synchronize()
        barrier()
        ms_e = max_over_ranks(t0.elapsed_time(t1), world, dev) / e_steps
        e2e = {"value": aggregate_value(in_bytes, ms_e, world), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
               "d2h_bytes_per_step": in_bytes, "ms_per_step": ms_e, "steps": e_steps,
               "api": "paper_2506_17615_b200.host_api.HostPipeline.submit (copies overlapped across steps)"}
        del h_in, h_out, pipe

    sampler.stop()
    clocks = sampler.summary(windows)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {**base_config(w), "parallelism": f"replicas x{world}" if world > 1 else "1 GPU",
                       "l2": f"{sets} input/output sets used in rotation ({sets * 2 * in_bytes / 1e6:.0f} MB "
                             f"working set against a 126 MB L2); no explicit flush",
                       "pdl_between_step_launches": os.environ.get("EQUARX_PDL", "1") != "0"},
            "e2e": e2e, "gpu_launches": args.steps, "clocks": clocks,
            "roofline": roofline, "schedule": "pipelined (equarx_allreduce_sim_pipelined, 1 launch per step)",
            "by_steps": by_steps, "flavours": flavours, "bf16_sim": bf16_sim,
            "speedup_vs_bf16_sim": value / world / bf16_sim["value"],
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
