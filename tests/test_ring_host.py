"""Host logic of the ring with one rank per device: mailbox addressing, the send/receive maps
of Section 3 (Fig. 1), argument validation of equarx_ring_allreduce (no GPU is touched), and the
set-up of PeerRing among two gloo processes on CPU with a stand-in for device memory."""
import os

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import binding
from paper_2506_17615_b200.ring import PeerRing, RingLayout, RingTimeout, _raise_on_status

A = 0x7000_0000_0000
MB = 1 << 20


@pytest.mark.parametrize("n", (1, 2, 3, 4, 8, 64))
def test_ring_maps(n):
    lay = RingLayout(n, n * 256 * 3, 256)
    for r in range(n):
        assert lay.left(lay.right(r)) == r
        # what a rank receives at step s+1 is the shard it sends on at step s+1 (after adding its own part)
        for s in range(n - 1):
            assert lay.shard_sent(lay.right(r), s + 1) == lay.shard_sent(r, s)
        assert lay.shard_sent(r, n - 1) == r                 # the last step finishes the rank's own shard
        assert sorted(lay.shard_sent(r, s) for s in range(n)) == list(range(n))
    # every reduce-scatter event sits in exactly one (rank, slot); the chain of shard k runs k+1, k+2, ..., k
    seen = set()
    for k in range(n):
        for j in range(n - 1):
            rank, slot = lay.event_location(k, j)
            assert rank == (k + 2 + j) % n and slot == j
            seen.add((rank, slot))
        assert lay.event_location(k, n - 1) == (k, n - 1 + k)
    assert len(seen) == n * (n - 1)


@pytest.mark.parametrize("n,count,block", [(1, 64, 64), (2, 2 * 640, 128), (4, 65536, 256), (8, 2048 * 3840, 256),
                                           (64, 1 << 24, 512)])
def test_mailbox_size_matches_the_library(n, count, block):
    lay = RingLayout(n, count, block)
    assert eq.ring_mailbox_bytes(n, count, block) == lay.mailbox_bytes
    assert lay.mailbox_bytes % 256 == 0
    assert lay.flags_offset == (2 * n - 1) * lay.tiles * 544
    assert eq.ring_mailbox_bytes(n, count + 1, block) == 0


def test_trace_is_read_from_the_right_slots():
    n, block = 3, 128
    lay = RingLayout(n, n * 640, block)                      # shard 640: 2 tiles, the second ragged; 5 blocks
    boxes = [np.zeros(lay.mailbox_bytes, np.uint8) for _ in range(n)]
    for k in range(n):
        for j in range(n):
            rank, slot = lay.event_location(k, j)
            rec = boxes[rank][slot * lay.slot_bytes:(slot + 1) * lay.slot_bytes].reshape(2, 544)
            for t in range(2):
                hdr = np.zeros(8, np.float32)
                hdr[:4] = [1000 * k + 100 * j + 4 * t + i for i in range(4)]
                rec[t, :32] = hdr.view(np.uint8)
                rec[t, 32:] = np.full(512, 10 * k + j, np.int8).view(np.uint8)
    # the all-gather message is in every rank's mailbox; event_location names the owner's copy
    scales, codes = lay.trace(boxes)
    assert scales.shape == (3, 3, 5) and codes.shape == (3, 3, 640)
    for k in range(n):
        for j in range(n):
            assert list(scales[k, j]) == [1000 * k + 100 * j + i for i in range(5)]
            assert (codes[k, j] == 10 * k + j).all()


def status_of(**kw):
    try:
        eq.ring_allreduce(**kw)
    except eq.EquarxError as e:
        return e.status
    return 0


def test_ring_entry_rejects_bad_arguments_before_any_cuda_call():
    n, count, block = 4, 65536, 256
    boxes = [A + (100 + q) * 16 * MB for q in range(n)]
    ok = dict(in_bf16=[A], out_bf16=[A + 16 * MB], rank_first=1, ranks_here=1, nranks=n, count=count, block=block,
              mailboxes=boxes, epoch=1, timeout_ns=0, status=A + 64 * MB)
    assert status_of(**{**ok, "nranks": 65}) == binding.ERR_NRANKS
    assert status_of(**{**ok, "rank_first": 4}) == binding.ERR_NRANKS
    assert status_of(**{**ok, "ranks_here": 0}) == binding.ERR_NRANKS
    assert status_of(**{**ok, "rank_first": 3, "ranks_here": 2, "in_bf16": [A, A + MB], "out_bf16": [A + 2 * MB, A + 3 * MB]}) \
        == binding.ERR_NRANKS
    assert status_of(**{**ok, "block": 100}) == binding.ERR_BLOCK
    assert status_of(**{**ok, "count": count + 256}) == binding.ERR_COUNT
    assert status_of(**{**ok, "epoch": 0}) == binding.ERR_COUNT
    assert status_of(**{**ok, "status": 0}) == binding.ERR_NULL
    assert status_of(**{**ok, "in_bf16": [0]}) == binding.ERR_NULL
    assert status_of(**{**ok, "mailboxes": boxes[:3] + [0]}) == binding.ERR_NULL
    assert status_of(**{**ok, "status": A + 64 * MB + 4}) == binding.ERR_ALIGN
    assert status_of(**{**ok, "out_bf16": [A + 16 * MB + 16]}) == binding.ERR_ALIGN
    assert status_of(**{**ok, "mailboxes": [boxes[0] + 8] + boxes[1:]}) == binding.ERR_ALIGN
    assert status_of(**{**ok, "out_bf16": [A + 64]}) == binding.ERR_ALIAS                   # partial overlap with the input
    assert status_of(**{**ok, "mailboxes": [A] + boxes[1:]}) == binding.ERR_ALIAS           # a mailbox on the input
    assert status_of(**{**ok, "mailboxes": [boxes[1] + 4096] + boxes[1:]}) == binding.ERR_ALIAS
    assert eq.last_cuda_error() == 0


def test_status_words_become_an_exception():
    _raise_on_status([0, 0, 0, 0], 4, epoch=5)
    _raise_on_status([4, 2, 3, 17], 4, epoch=5)              # an earlier call failed, this one did not
    with pytest.raises(RingTimeout) as e:
        _raise_on_status([5, 2, 3, 17], 4, epoch=5)
    assert (e.value.rank, e.value.step, e.value.tile) == (2, 3, 17) and "ring step 3" in str(e.value)
    with pytest.raises(RingTimeout) as e:
        _raise_on_status([9, 0, 4 + 2, 5], 4, epoch=9)
    assert "all-gather message of shard 2" in str(e.value)


class FakeMemory:
    """Stands in for device memory and CUDA IPC: 'pointers' are integers that encode the owner."""

    def __init__(self, rank, log):
        self.rank, self.log = rank, log

    def alloc_zeroed(self, nbytes):
        self.log.append(("alloc", nbytes))
        return 0x1000_0000 * (self.rank + 1)

    def export(self, ptr):
        return ptr.to_bytes(8, "little") + bytes(56)

    def open(self, handle):
        owner_ptr = int.from_bytes(handle[:8], "little")
        self.log.append(("open", owner_ptr))
        return owner_ptr + 0x100 * (self.rank + 1)          # a peer mapping has its own address in this process

    def close(self, ptr):
        self.log.append(("close", ptr))

    def free(self, ptr):
        self.log.append(("free", ptr))


def _peer_worker(rank, world, port, q, fail_rank):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log, calls = [], []
    status = [0, 0, 0, 0]

    def launch(ins, outs, rank_first, ranks_here, nranks, count, block, mailboxes, epoch, timeout_ns, st, stream):
        calls.append(dict(rank_first=rank_first, ranks_here=ranks_here, nranks=nranks, mailboxes=list(mailboxes),
                          epoch=epoch, timeout_ns=timeout_ns))
        if rank == fail_rank and epoch == 2:               # the kernel would have written this after a time-out
            st[:] = [epoch, rank, 1, 0]

    ring = PeerRing(2 * 256 * 3, 256, memory=FakeMemory(rank, log), launch=launch, status=status)
    ring.allreduce("x", "out")
    ring.check()
    ring.allreduce("x", "out", timeout_ns=5_000_000)
    failed = None
    try:
        ring.check()
    except RingTimeout as e:
        failed = (e.rank, e.step, e.tile)
    boxes = list(ring.mailboxes)
    ring.close()
    q.put((rank, log, calls, boxes, failed))
    dist.destroy_process_group()


def test_peer_ring_setup_between_two_gloo_processes():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31000 + os.getpid() % 2000
    procs = [ctx.Process(target=_peer_worker, args=(r, 2, port, q, 1)) for r in range(2)]
    for p in procs:
        p.start()
    got = {}
    for _ in procs:
        rank, log, calls, boxes, failed = q.get(timeout=180)
        got[rank] = (log, calls, boxes, failed)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    lay = RingLayout(2, 2 * 256 * 3, 256)
    for rank in (0, 1):
        log, calls, boxes, failed = got[rank]
        own, peer = 0x1000_0000 * (rank + 1), 0x1000_0000 * (2 - rank)
        assert log[0] == ("alloc", lay.mailbox_bytes)
        assert ("open", peer) in log and ("open", own) not in log          # the own mailbox is not re-mapped
        mapped = peer + 0x100 * (rank + 1)
        assert boxes[rank] == own and boxes[1 - rank] == mapped
        assert [c["epoch"] for c in calls] == [1, 2]
        assert all(c["rank_first"] == rank and c["ranks_here"] == 1 and c["nranks"] == 2 for c in calls)
        assert calls[1]["timeout_ns"] == 5_000_000 and calls[0]["mailboxes"] == boxes
        assert log[-2:] == [("close", mapped), ("free", own)]              # unmap peers, then free the own one
        assert failed == ((1, 1, 0) if rank == 1 else None)               # only the rank whose wait ran out raises


def _protocol_worker(rank, world, port, q, block, bps):
    """One rank of the ring as a CPU process: the schedule and slot maps of RingLayout drive real
    sends and receives (gloo); the arithmetic of every step is the oracle's per-step functions."""
    import torch
    import oracle
    from paper_2506_17615_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    count = world * bps * block
    lay = RingLayout(world, count, block)
    x = wl.as_u16(wl.make_rank(wl.Workload("t", world, count, block, "normal", seed=77), rank))
    shard = lay.shard
    slots = {}                                           # the mailbox: slot -> (codes, scales)

    def exchange(dst, src, codes, scales):
        """send one message to dst while receiving one from src (deadlock-free pairing)"""
        out_c, out_s = torch.from_numpy(codes.copy()), torch.from_numpy(scales.copy())
        in_c, in_s = torch.empty_like(out_c), torch.empty_like(out_s)
        reqs = [dist.isend(out_c, dst), dist.isend(out_s, dst), dist.irecv(in_c, src), dist.irecv(in_s, src)]
        for r_ in reqs:
            r_.wait()
        return in_c.numpy(), in_s.numpy()

    for s in range(world):
        k = lay.shard_sent(rank, s)
        mine = x[k * shard:(k + 1) * shard]
        if s == 0:
            codes, scales = oracle.quantize_blocks(mine, block)
        else:
            c_in, s_in = slots[lay.recv_slot(s)]
            codes, scales = oracle.rs_step(c_in, s_in, mine, block)
        if s + 1 < world:
            slots[lay.recv_slot(s + 1)] = exchange(lay.right(rank), lay.left(rank), codes, scales)
        else:
            assert k == rank                             # the reduced shard is the rank's own
            slots[lay.gather_slot(k)] = (codes, scales)
    # all-gather: every rank gets every reduced shard's message
    for step in range(1, world):
        dst, src = (rank + step) % world, (rank - step) % world
        slots[lay.gather_slot(src)] = exchange(dst, src, *slots[lay.gather_slot(rank)])
    out = np.concatenate([oracle.ag_dequant(*slots[lay.gather_slot(k)], block) for k in range(world)])
    q.put((rank, out))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", (2, 3))
def test_ring_schedule_among_cpu_processes_equals_the_oracle_allreduce(world):
    """The send/receive maps and mailbox slots, exercised by real message passing between processes,
    reproduce the single-process oracle's AllReduce bit for bit on every rank."""
    import oracle
    from paper_2506_17615_b200 import workloads as wl
    block, bps = 64, 3
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33000 + os.getpid() % 2000 + world
    procs = [ctx.Process(target=_protocol_worker, args=(r, world, port, q, block, bps)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=240) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    x = wl.as_u16(wl.make_inputs(wl.Workload("t", world, world * bps * block, block, "normal", seed=77)))
    exp = oracle.allreduce(x, block)["out"]
    for r in range(world):
        assert np.array_equal(got[r], exp[r]), f"rank {r}"
