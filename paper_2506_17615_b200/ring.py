"""Host side of the quantized ring AllReduce with one rank per device (equarx_ring_allreduce).

Plumbing only: where a message lives in a mailbox, who sends what to whom at which ring step
(Section 3, Fig. 1), allocating and zeroing mailboxes, exchanging their CUDA IPC handles between
the processes of a job, the epoch counter and reading the status words back.  Every arithmetic
step runs in the library's kernel.

  LocalRing  all ranks on one GPU (one cooperative launch): how the ring is run and checked on a
             single device.
  PeerRing   one rank per process and GPU; the mailboxes of all ranks are mapped into every
             process through CUDA IPC handles exchanged over torch.distributed.
"""
from dataclasses import dataclass

RECORD_BYTES, RECORD_HEADER, TILE_ELEMS = 544, 32, 512


class RingTimeout(RuntimeError):
    """A rank waited longer than the time limit for a message (the kernel returned; nothing hung)."""

    def __init__(self, rank, step, tile, nranks):
        self.rank, self.step, self.tile = rank, step, tile
        what = f"ring step {step}" if step < nranks else f"the all-gather message of shard {step - nranks}"
        super().__init__(f"rank {rank} gave up waiting for tile {tile} of {what}")


@dataclass(frozen=True)
class RingLayout:
    """Addresses inside a mailbox and the ring's send/receive maps."""
    nranks: int
    count: int
    block: int

    def __post_init__(self):
        if self.nranks < 1 or self.count <= 0 or self.count % (self.nranks * self.block):
            raise ValueError("count must be a positive multiple of nranks * block")

    @property
    def shard(self):
        return self.count // self.nranks

    @property
    def tiles(self):
        return -(-self.shard // TILE_ELEMS)

    @property
    def slots(self):
        return 2 * self.nranks - 1

    @property
    def slot_bytes(self):
        return self.tiles * RECORD_BYTES

    @property
    def flags_offset(self):
        return self.slots * self.slot_bytes

    @property
    def mailbox_bytes(self):
        raw = self.flags_offset + 4 * self.slots * self.tiles
        return -(-raw // 256) * 256

    # ---- who sends what (rank r sends to r+1; at step s it sends shard (r-1-s) mod N; shard k ends on rank k)
    def right(self, rank):
        return (rank + 1) % self.nranks

    def left(self, rank):
        return (rank - 1) % self.nranks

    def shard_sent(self, rank, step):
        return (rank - 1 - step) % self.nranks

    def recv_slot(self, step):
        """Slot of a rank's mailbox that holds the message it receives at ring step `step` >= 1."""
        if not 1 <= step <= self.nranks - 1:
            raise ValueError("messages are received at steps 1 .. nranks-1")
        return step - 1

    def gather_slot(self, shard):
        return self.nranks - 1 + shard

    def event_location(self, shard, event):
        """(rank, slot) where event `event` of `shard` can be read after a call: events 0..N-2 are
        the reduce-scatter messages in chain order, event N-1 the all-gather message (any rank)."""
        n = self.nranks
        if event == n - 1:
            return shard, self.gather_slot(shard)
        sender = (shard + 1 + event) % n
        assert self.shard_sent(sender, event) == shard
        return self.right(sender), self.recv_slot(event + 1)

    def flag_index(self, slot, tile):
        return slot * self.tiles + tile

    def trace(self, mailboxes):
        """mailboxes: one uint8 numpy array per rank (a host copy).  Returns (scales float32
        [N shards, N events, blocks per shard], codes int8 [N, N, shard]) in the oracle's order."""
        import numpy as np
        n, bps, per_tile = self.nranks, self.shard // self.block, TILE_ELEMS // self.block
        scales = np.zeros((n, n, bps), np.float32)
        codes = np.zeros((n, n, self.shard), np.int8)
        for k in range(n):
            for j in range(n):
                rank, slot = self.event_location(k, j)
                rec = np.asarray(mailboxes[rank][slot * self.slot_bytes:(slot + 1) * self.slot_bytes])
                rec = rec.reshape(self.tiles, RECORD_BYTES)
                hdr = np.ascontiguousarray(rec[:, :RECORD_HEADER]).view(np.float32)
                scales[k, j] = hdr[:, :per_tile].reshape(-1)[:bps]
                codes[k, j] = np.ascontiguousarray(rec[:, RECORD_HEADER:]).view(np.int8).reshape(-1)[:self.shard]
        return scales, codes


def _raise_on_status(words, nranks, epoch):
    """A failed call stamps the status with its epoch; any other first word means the call completed."""
    code, rank, step, tile = (int(w) & 0xFFFFFFFF for w in words)
    if epoch > 0 and code == epoch:
        raise RingTimeout(rank, step, tile, nranks)


class LocalRing:
    """The whole ring on the current GPU: N ranks hosted by one cooperative launch."""

    def __init__(self, nranks, count, block, device=None):
        import torch
        from . import binding
        self._b = binding
        self.layout = RingLayout(nranks, count, block)
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        nbytes = binding.ring_mailbox_bytes(nranks, count, block)
        if nbytes != self.layout.mailbox_bytes:
            raise RuntimeError("mailbox layout of the binding and the library disagree")
        self.mailboxes = [torch.zeros(nbytes, dtype=torch.uint8, device=self.device) for _ in range(nranks)]
        self.status = torch.zeros(4, dtype=torch.int32, device=self.device)
        self.epoch = 0

    def allreduce(self, ins, outs, timeout_ns=0, stream=0):
        """ins, outs: N bf16 device tensors.  Asynchronous; check() synchronises and raises on a time-out."""
        lay = self.layout
        self.epoch += 1
        self._b.ring_allreduce(ins, outs, 0, lay.nranks, lay.nranks, lay.count, lay.block, self.mailboxes,
                               self.epoch, timeout_ns, self.status, stream)

    def check(self):
        import torch
        torch.cuda.synchronize(self.device)
        _raise_on_status(self.status.cpu().tolist(), self.layout.nranks, self.epoch)

    def trace(self):
        return self.layout.trace([m.cpu().numpy() for m in self.mailboxes])


class CudaIpcMemory:
    """Device allocations that other processes can map: plain cudaMalloc, CUDA IPC handles."""

    def __init__(self):
        from cuda.bindings import runtime as rt
        self.rt = rt

    def _ok(self, err, what):
        if int(err) != 0:
            raise RuntimeError(f"{what} failed with CUDA error {int(err)}")

    def alloc_zeroed(self, nbytes):
        err, ptr = self.rt.cudaMalloc(nbytes)
        self._ok(err, "cudaMalloc")
        (err,) = self.rt.cudaMemset(ptr, 0, nbytes)
        self._ok(err, "cudaMemset")
        (err,) = self.rt.cudaDeviceSynchronize()
        self._ok(err, "cudaDeviceSynchronize")
        return int(ptr)

    def free(self, ptr):
        (err,) = self.rt.cudaFree(ptr)
        self._ok(err, "cudaFree")

    def export(self, ptr):
        err, handle = self.rt.cudaIpcGetMemHandle(ptr)
        self._ok(err, "cudaIpcGetMemHandle")
        return bytes(handle.reserved)

    def open(self, handle_bytes):
        handle = self.rt.cudaIpcMemHandle_t()
        handle.reserved = handle_bytes
        err, ptr = self.rt.cudaIpcOpenMemHandle(handle, self.rt.cudaIpcMemLazyEnablePeerAccess)
        self._ok(err, "cudaIpcOpenMemHandle")
        return int(ptr)

    def close(self, ptr):
        (err,) = self.rt.cudaIpcCloseMemHandle(ptr)
        self._ok(err, "cudaIpcCloseMemHandle")


class PeerRing:
    """One rank of the ring per process and GPU.

    `group` is a torch.distributed process group (or None for the default one) whose rank order is
    the ring order; it carries the mailbox handles at set-up and nothing afterwards.  `memory`
    provides alloc_zeroed / export / open / close / free (default: CudaIpcMemory); `launch` is the
    library call (default: binding.ring_allreduce).  Both are parameters so that the host logic can
    run among CPU processes.  Not exercised on more than one GPU.
    """

    def __init__(self, count, block, group=None, memory=None, launch=None, status=None):
        import torch.distributed as dist
        self.rank, nranks = dist.get_rank(group), dist.get_world_size(group)
        self.layout = RingLayout(nranks, count, block)
        self.memory = CudaIpcMemory() if memory is None else memory
        if launch is None:
            from . import binding
            launch = binding.ring_allreduce
        self._launch = launch
        self.own = self.memory.alloc_zeroed(self.layout.mailbox_bytes)
        handles = [None] * nranks
        dist.all_gather_object(handles, self.memory.export(self.own), group=group)
        # every rank stores into its right neighbour's mailbox and, at the last step, into everybody's
        self.mailboxes = [self.own if q == self.rank else self.memory.open(handles[q]) for q in range(nranks)]
        dist.barrier(group=group)            # nobody sends before every mailbox is mapped and zeroed
        if status is None:
            import torch
            status = torch.zeros(4, dtype=torch.int32, device="cuda")
        self.status = status
        self.epoch = 0
        self.group = group

    def allreduce(self, x, out, timeout_ns=0, stream=0):
        """x, out: this rank's bf16 tensors (count elements).  All ranks call it the same number of times."""
        lay = self.layout
        self.epoch += 1
        self._launch([x], [out], self.rank, 1, lay.nranks, lay.count, lay.block, self.mailboxes, self.epoch,
                     timeout_ns, self.status, stream)

    def check(self):
        """Synchronise this rank's device and raise RingTimeout if one of its waits ran out."""
        if hasattr(self.status, "cpu"):
            import torch
            torch.cuda.synchronize()
            words = self.status.cpu().tolist()
        else:
            words = list(self.status)
        _raise_on_status(words, self.layout.nranks, self.epoch)

    def close(self):
        """Between calls only: no kernel of any rank may still be using the mailboxes."""
        import torch.distributed as dist
        dist.barrier(group=self.group)
        for q, ptr in enumerate(self.mailboxes):
            if q != self.rank:
                self.memory.close(ptr)
        dist.barrier(group=self.group)       # peers have unmapped this rank's mailbox
        self.memory.free(self.own)
        self.mailboxes = []
