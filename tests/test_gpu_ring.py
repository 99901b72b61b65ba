"""The ring with one rank per device (equarx_ring_allreduce), run on ONE GPU: all ranks are hosted by a
single cooperative launch and exchange their messages through per-rank mailboxes and per-tile flags,
exactly as ranks on different GPUs would.  Every message (from the mailboxes) and every output word
is compared with the CPU oracle.  A wait that nothing satisfies must come back as a status, not hang."""
import multiprocessing as mp

import numpy as np
import pytest
import torch

import oracle
import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import binding, workloads as wl
from paper_2506_17615_b200.ring import CudaIpcMemory, LocalRing, RingLayout, RingTimeout

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def guard_mailboxes(gu, ring):
    """Replace the ring's mailboxes by zeroed buffers with canary bands on both sides (once per ring)."""
    if getattr(ring, "_guards", None) is None:
        ring._guards = [gu.Guarded(ring.layout.mailbox_bytes) for _ in range(ring.layout.nranks)]
        for g in ring._guards:
            g.u8.zero_()
        ring.mailboxes = [g.u8 for g in ring._guards]
    return ring._guards


def run_and_compare(gu, ring, x, in_place=False):
    n, count = x.shape
    block = ring.layout.block
    guards = guard_mailboxes(gu, ring)
    res = oracle.allreduce(wl.as_u16(x), block, trace=True)
    xd = x.cuda()
    if in_place:
        bufs = [gu.Guarded(2 * count) for _ in range(n)]
        for r in range(n):
            bufs[r].view(torch.bfloat16).copy_(xd[r])
        ins = outs = bufs
    else:
        ins = [xd[r] for r in range(n)]
        outs = [gu.Guarded(2 * count) for _ in range(n)]
    ring.allreduce(ins, outs, stream=gu.stream_handle())
    ring.check()
    for o in outs + guards:
        o.check()
    out = torch.stack([o.view(torch.bfloat16) for o in outs])
    gu.assert_same_words(out, res["out"], "ring outputs")
    scales, codes = ring.trace()
    assert np.array_equal(codes, res["codes"]), "messages in the mailboxes: codes"
    assert np.array_equal(scales.view(np.uint32), res["scales"].view(np.uint32)), "messages in the mailboxes: scales"
    # every rank received the same all-gather messages, and every flag carries the call's epoch
    lay = ring.layout
    boxes = [m.cpu().numpy() for m in ring.mailboxes]
    for q in range(1, n):
        a0 = boxes[0][(n - 1) * lay.slot_bytes:lay.flags_offset]
        assert np.array_equal(boxes[q][(n - 1) * lay.slot_bytes:lay.flags_offset], a0)
    for b in boxes:
        flags = b[lay.flags_offset:lay.flags_offset + 4 * lay.slots * lay.tiles].view(np.uint32)
        assert (flags == ring.epoch).all()


@pytest.mark.parametrize("nranks", (1, 2, 3, 5, 8, 16, 64))
@pytest.mark.parametrize("block", (64, 128, 256, 512))
def test_ring_matches_oracle(gu, nranks, block):
    bps = 5 if block >= 256 else 37                          # ragged against the 512-element tile
    w = wl.Workload("t", nranks, nranks * bps * block, block, "normal", seed=40 + nranks)
    ring = LocalRing(nranks, w.count, block)
    run_and_compare(gu, ring, wl.make_inputs(w))


def test_ring_config1_and_repeated_calls_on_the_same_mailboxes(gu):
    """Epochs: three calls on different data reuse the mailboxes without clearing anything."""
    w = wl.C1
    ring = LocalRing(w.nranks, w.count, w.block)
    for seed in (0, 1, 2):
        x = wl.make_inputs(wl.Workload(w.name, w.nranks, w.count, w.block, w.dist, seed=seed))
        run_and_compare(gu, ring, x, in_place=(seed == 1))
    assert ring.epoch == 3


def test_ring_on_stress_blocks_and_activation_shapes(gu):
    x = wl.make_inputs(wl.C5, count=64 * 256 * 6)
    run_and_compare(gu, LocalRing(64, x.shape[1], 256), x)
    x = wl.make_inputs(wl.C2, count=32 * wl.C2.hidden)
    run_and_compare(gu, LocalRing(8, x.shape[1], 256), x)


def test_ring_config2_full_size_outputs(gu):
    """Config 2 at full size: every output word against the oracle (many tiles per warp, all SMs busy)."""
    w = wl.C2
    x = wl.make_inputs(w, device="cuda")
    ring = LocalRing(w.nranks, w.count, w.block)
    out = torch.empty_like(x)
    ring.allreduce([x[r] for r in range(w.nranks)], [out[r] for r in range(w.nranks)], stream=gu.stream_handle())
    ring.check()
    exp = oracle.allreduce(wl.as_u16(x), w.block)["out"]
    gu.assert_same_words(out, exp, "ring, config 2")


def test_a_message_that_never_arrives_is_reported_not_waited_for_forever(gu):
    """Rank 1 of a two-rank ring is launched alone: nothing ever writes its mailbox.  Its first wait
    runs out after the time limit, the kernel returns, the status names rank, step and tile, and the
    device is fully usable afterwards."""
    n, block = 2, 256
    count = n * block * 4
    lay = RingLayout(n, count, block)
    x = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=9)).cuda()
    out = torch.zeros_like(x)
    boxes = [torch.zeros(lay.mailbox_bytes, dtype=torch.uint8, device="cuda") for _ in range(n)]
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    eq.ring_allreduce([x[1]], [out[1]], 1, 1, n, count, block, boxes, 1, 20_000_000, status, gu.stream_handle())
    t1.record()
    torch.cuda.synchronize()
    assert status.cpu().tolist()[:3] == [1, 1, 1]            # {epoch of the failed call, rank, step}
    assert 15.0 < t0.elapsed_time(t1) < 2000.0               # about the 20 ms limit, and it did end
    # rank 1 did send its step-0 message to rank 0 before it gave up
    flags0 = boxes[0].cpu().numpy()[lay.flags_offset:lay.flags_offset + 4 * lay.tiles].view(np.uint32)
    assert (flags0 == 1).all()
    # nothing is left behind: the whole ring runs right after
    ring = LocalRing(n, count, block)
    run_and_compare(gu, ring, x.cpu())
    with pytest.raises(RingTimeout):
        from paper_2506_17615_b200.ring import _raise_on_status
        _raise_on_status(status.cpu().tolist(), n, 1)


def _ipc_child(handle, nbytes, q):
    try:
        mem = CudaIpcMemory()
        ptr = mem.open(handle)
        (err,) = mem.rt.cudaMemset(ptr, 0x3C, nbytes)
        (err2,) = mem.rt.cudaDeviceSynchronize()
        mem.close(ptr)
        q.put(("ok", int(err), int(err2)))
    except Exception as exc:                                 # pragma: no cover - reported to the parent
        q.put(("error", repr(exc), 0))


def test_mailbox_handles_map_the_same_memory_in_another_process():
    """The plumbing PeerRing relies on: a mailbox allocated here, exported as a CUDA IPC handle,
    opened by a second process (same GPU), written there and read back here.  Plain memsets only."""
    mem = CudaIpcMemory()
    nbytes = 1 << 20
    ptr = mem.alloc_zeroed(nbytes)
    try:
        handle = mem.export(ptr)
        assert len(handle) == 64
        ctx = mp.get_context("spawn")
        q = ctx.Queue()
        p = ctx.Process(target=_ipc_child, args=(handle, nbytes, q))
        p.start()
        verdict = q.get(timeout=180)
        p.join(timeout=60)
        assert verdict == ("ok", 0, 0), verdict
        host = np.zeros(nbytes, np.uint8)
        (err,) = mem.rt.cudaMemcpy(host.ctypes.data, ptr, nbytes, mem.rt.cudaMemcpyKind.cudaMemcpyDeviceToHost)
        assert int(err) == 0 and (host == 0x3C).all()
    finally:
        mem.free(ptr)


def test_bench_ring_mode_with_a_single_rank():
    """bench.py --ring runs PeerRing end to end (mailbox allocation, IPC export, the process group, the
    launch with ranks_here = 1, status read-back, close); with one process the ring has one rank."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env["MASTER_PORT"] = str(29600 + os.getpid() % 300)
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--ring", "--workload", "C1", "--steps", "3",
                          "--min-seconds", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["failure"] is None and line["value"] > 0 and line["config"]["nranks"] == 1
    assert "ranks_here=1" in line["schedule"]


def _mailbox_owner(nboxes, nbytes, handles_q, done_evt):
    """A second process that owns mailboxes: allocates them, hands out their IPC handles, frees them at the end."""
    mem = CudaIpcMemory()
    ptrs = [mem.alloc_zeroed(nbytes) for _ in range(nboxes)]
    handles_q.put([mem.export(p) for p in ptrs])
    done_evt.wait(timeout=300)
    for p in ptrs:
        mem.free(p)


def test_ring_through_mailboxes_owned_by_another_process(gu):
    """Half of the mailboxes live in allocations of ANOTHER process, mapped here through CUDA IPC, as a peer
    GPU's mailbox would be.  All ranks still run in one cooperative launch of this process (no kernel waits
    on another launch); records, flags and acquire loads go through the IPC mappings."""
    n, block = 4, 256
    count = n * block * 9
    lay = RingLayout(n, count, block)
    ctx = mp.get_context("spawn")
    handles_q, done = ctx.Queue(), ctx.Event()
    owner = ctx.Process(target=_mailbox_owner, args=(2, lay.mailbox_bytes, handles_q, done))
    owner.start()
    mem = CudaIpcMemory()
    mapped = []
    try:
        handles = handles_q.get(timeout=180)
        mapped = [mem.open(h) for h in handles]
        local = [torch.zeros(lay.mailbox_bytes, dtype=torch.uint8, device="cuda") for _ in range(2)]
        boxes = [mapped[0], local[0], mapped[1], local[1]]           # ranks 0 and 2 receive in the other process's memory
        x = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=55))
        xd = x.cuda()
        outs = [gu.Guarded(2 * count) for _ in range(n)]
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        for epoch in (1, 2):
            eq.ring_allreduce([xd[r] for r in range(n)], outs, 0, n, n, count, block, boxes, epoch, 0, status,
                              gu.stream_handle())
            torch.cuda.synchronize()
            assert status.cpu().tolist()[0] == 0
        exp = oracle.allreduce(wl.as_u16(x), block)["out"]
        for o in outs:
            o.check()
        gu.assert_same_words(torch.stack([o.view(torch.bfloat16) for o in outs]), exp, "ring over IPC-mapped mailboxes")
    finally:
        for p in mapped:
            mem.close(p)
        done.set()
        owner.join(timeout=60)
    assert owner.exitcode == 0
