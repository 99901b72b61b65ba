"""Seeded synthetic inputs for the simulated quantized AllReduce.

This module only draws random bf16 tensors; it holds none of the method's
arithmetic and is the one module that both the CUDA tests/bench and the CPU
oracle's tests take their inputs from.  The tensors stand in for the paper's
workloads (Section 4: a (4096, 4096) N(0,1) tensor; Section 5: Gemma 3
prefill activations, two AllReduces per layer over [tokens x hidden] partial
sums), which are not available offline.

Every rank's values come from ``torch.Generator`` seeded with
``seed * 1_000_003 + rank``; structure that all ranks share (outlier
channels, block types, spike positions) comes from a generator seeded with
``seed``.  Values are rounded to bf16 by torch.  The stream depends on the
device the generator lives on, so a comparison must hand the *same* tensor to
both sides.
"""
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    nranks: int
    count: int          # bf16 elements per rank
    block: int
    dist: str
    hidden: int = 0     # row length for the activation-shaped workloads
    seed: int = 0

    @property
    def bytes_per_rank(self):
        return 2 * self.count


# The five configurations of the benchmark definition.
C1 = Workload("C1_small_normal", 4, 65_536, 256, "normal")
C2 = Workload("C2_gemma3_12b_prefill2048", 8, 2048 * 3840, 256, "normal_outlier50", hidden=3840)
C3 = Workload("C3_gemma3_27b_prefill8192", 8, 8192 * 5376, 256, "student3_outlier100", hidden=5376)
C5 = Workload("C5_stress_mixed_blocks", 64, 1 << 24, 256, "mixed_blocks")


def sweep_point(nranks, bytes_per_rank, block, dist, seed=0):
    """One point of the message-size sweep (16 KB .. 256 MB per rank)."""
    return Workload(f"C4_sweep_N{nranks}_{bytes_per_rank}B_b{block}_{dist}", nranks,
                    bytes_per_rank // 2, block, dist, seed=seed)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _outlier_channels(hidden, frac, seed):
    g = _gen("cpu", seed)
    k = int(round(frac * hidden))
    return torch.randperm(hidden, generator=g)[:k]


def _mixed_block_layout(nblocks, block, seed):
    """Block type (0 zero, 1 spike, 2 subnormal, 3 cancelling) and spike slot per block."""
    g = _gen("cpu", seed)
    types = torch.randint(0, 4, (nblocks,), generator=g)
    spike = torch.randint(0, block, (nblocks,), generator=g)
    return types, spike


def make_rank(w: Workload, rank: int, device="cpu", count=None):
    """bf16 tensor [count] of rank ``rank`` for workload ``w`` (count overrides w.count)."""
    n = w.count if count is None else count
    dev = torch.device(device)
    g = _gen(dev, w.seed * 1_000_003 + rank)
    if w.dist == "normal":
        x = torch.randn(n, generator=g, device=dev)
    elif w.dist == "uniform":
        x = torch.rand(n, generator=g, device=dev) * 2.0 - 1.0
    elif w.dist == "normal_outlier50":
        x = torch.randn(n // w.hidden, w.hidden, generator=g, device=dev)
        ch = _outlier_channels(w.hidden, 0.01, w.seed).to(dev)
        x[:, ch] *= 50.0
        x = x.reshape(-1)
    elif w.dist == "student3_outlier100":
        rows = n // w.hidden
        z = torch.randn(rows, w.hidden, generator=g, device=dev)
        chi2 = torch.zeros_like(z)
        for _ in range(3):
            chi2 += torch.randn(rows, w.hidden, generator=g, device=dev) ** 2
        x = 0.5 * z / torch.sqrt(chi2 / 3.0)
        del z, chi2
        ch = _outlier_channels(w.hidden, 0.005, w.seed).to(dev)
        x[:, ch] *= 100.0
        x = x.reshape(-1)
    elif w.dist == "mixed_blocks":
        nb = n // w.block
        types, spike = _mixed_block_layout(nb, w.block, w.seed)
        types, spike = types.to(dev), spike.to(dev)
        x = torch.zeros(nb, w.block, device=dev)
        # type 1: small noise plus one spike at bf16(6e4) = 59904, same slot on every rank
        noise = torch.randn(nb, w.block, generator=g, device=dev) * 1e-3
        m1 = types == 1
        x[m1] = noise[m1]
        rows = torch.nonzero(m1).squeeze(1)
        x[rows, spike[rows]] = 59904.0
        # type 2: bf16-subnormal magnitudes k * 2^-133, k in [1, 127], random sign
        k = torch.randint(1, 128, (nb, w.block), generator=g, device=dev).float()
        sgn = torch.randint(0, 2, (nb, w.block), generator=g, device=dev).float() * 2.0 - 1.0
        sub = (k * sgn).double() * (2.0 ** -133)
        m2 = types == 2
        # type 3: (-1)^rank * u with u shared by all ranks, so the exact sum cancels
        gu = _gen(dev, w.seed * 1_000_003 + 999_983)
        u = torch.randn(nb, w.block, generator=gu, device=dev)
        m3 = types == 3
        x[m3] = u[m3] * (1.0 if rank % 2 == 0 else -1.0)
        xb = x.to(torch.bfloat16)
        # subnormals are written through float64 -> bf16 so that no fp32 flush mode can touch them
        xb[m2] = sub[m2].to(torch.bfloat16)
        return xb.reshape(-1)
    else:
        raise ValueError(f"unknown distribution {w.dist!r}")
    return x.to(torch.bfloat16)


def make_inputs(w: Workload, device="cpu", count=None):
    """bf16 tensor [nranks, count]."""
    return torch.stack([make_rank(w, r, device, count) for r in range(w.nranks)])


def as_u16(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its raw words (host copy)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
