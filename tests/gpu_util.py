"""Helpers for the GPU parity tests: guarded device buffers, running the
library through its binding, and oracle comparisons on sampled blocks."""
import numpy as np
import torch

import oracle
import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import workloads as wl

GUARD = 256        # bytes of canary before and after every guarded buffer
CANARY = 0xA5


class Guarded:
    """A device buffer of `nbytes` with canary bands on both sides (in place of a
    memory checker: the bands are verified after the kernels ran)."""

    def __init__(self, nbytes, device="cuda"):
        pad = (nbytes + 255) // 256 * 256
        self.raw = torch.full((GUARD + pad + GUARD,), CANARY, dtype=torch.uint8, device=device)
        self.nbytes = nbytes
        self.u8 = self.raw[GUARD:GUARD + nbytes]

    def view(self, dtype):
        return self.u8.view(dtype)

    def data_ptr(self):
        return self.u8.data_ptr()

    def check(self):
        assert bool((self.raw[:GUARD] == CANARY).all()), "write before the buffer"
        assert bool((self.raw[GUARD + self.nbytes:GUARD + self.nbytes + GUARD] == CANARY).all()), \
            "write past the buffer"


def stream_handle():
    return torch.cuda.current_stream().cuda_stream


def to_dev_bf16(words_u16):
    return torch.from_numpy(np.ascontiguousarray(words_u16).view(np.int16)).cuda().view(torch.bfloat16)


def run_sim(x_dev, block, keep_trace=False, in_place=False, variant="steps"):
    """x_dev: bf16 CUDA tensor [N, count].  Returns (out [N, count] bf16, workspace Guarded).
    variant: "steps" = equarx_allreduce_sim, "pipelined" = equarx_allreduce_sim_pipelined."""
    n_ranks, count = x_dev.shape
    size_fn = {"steps": eq.allreduce_sim_workspace_bytes,
               "pipelined": eq.allreduce_sim_pipelined_workspace_bytes}[variant]
    wb = size_fn(n_ranks, count, block, keep_trace)
    assert wb > 0
    ws = Guarded(wb)
    if in_place:
        bufs = [Guarded(2 * count) for _ in range(n_ranks)]
        for r in range(n_ranks):
            bufs[r].view(torch.bfloat16).copy_(x_dev[r])
        ins = outs = bufs
    else:
        ins = [x_dev[r] for r in range(n_ranks)]
        outs = [Guarded(2 * count) for _ in range(n_ranks)]
    fn = {"steps": eq.allreduce_sim, "pipelined": eq.allreduce_sim_pipelined}[variant]
    fn(ins, outs, n_ranks, count, block, ws, wb, keep_trace, stream_handle())
    torch.cuda.synchronize()
    ws.check()
    for o in outs:
        o.check()
    out = torch.stack([o.view(torch.bfloat16) for o in outs])
    return out, ws


def assert_same_words(dev_bf16, words_u16, what):
    got = wl.as_u16(dev_bf16)
    exp = np.asarray(words_u16)
    if not np.array_equal(got, exp):
        bad = np.nonzero(got.ravel() != exp.ravel())[0]
        raise AssertionError(f"{what}: {bad.size} of {exp.size} bf16 words differ, first at {bad[0]}: "
                             f"got {got.ravel()[bad[0]]:#06x} expected {exp.ravel()[bad[0]]:#06x}")


def sample_blocks(n_ranks, bps, per_shard, seed):
    rng = np.random.default_rng(seed)
    m = min(per_shard, bps)
    picks = [np.sort(rng.choice(bps, size=m, replace=False)) for _ in range(n_ranks)]
    for p in picks:                 # always include the first and the last block of a shard
        p[0], p[-1] = 0, bps - 1
    return picks


def gather_blocks(t_dev, picks, block):
    """t_dev [N, count] -> [N, N*m*block]: the sampled blocks of every shard, in shard order.
    Because blocks are independent this is itself a valid, smaller AllReduce problem."""
    n_ranks, count = t_dev.shape
    shard = count // n_ranks
    idx = []
    for k, p in enumerate(picks):
        base = k * shard + torch.from_numpy(p.astype(np.int64))[:, None] * block + torch.arange(block)[None, :]
        idx.append(base.reshape(-1))
    idx = torch.cat(idx).to(t_dev.device)
    return t_dev[:, idx]


def oracle_out_on_samples(x_dev, picks, block):
    sub = gather_blocks(x_dev, picks, block)
    res = oracle.allreduce(wl.as_u16(sub), block)
    return res["out"]
