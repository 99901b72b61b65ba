"""Oracle pins for the other flavours (Sections 3.3, 3.4): semi-loop ring and stage selection."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2506_17615_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FLAVOURS = [(s, r, a) for s in (False, True) for r in (False, True) for a in (False, True)]


def to_f64(words):
    return torch.from_numpy(np.ascontiguousarray(words).view(np.int16)).view(torch.bfloat16).double().numpy()


def words_of(values):
    return torch.tensor(values, dtype=torch.float64).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def printed_mse():
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", "paper_mse.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                out[line[0]] = float(line[1])
    return out


def test_printed_mse_of_semi_loop_and_ag_only():
    """Section 4.1 prints 0.001 (semi-loop, both stages) and 0.0003 (full-loop, all-gather only)
    against the BF16 AllReduce: block 64, 8 devices, N(0,1)."""
    p = printed_mse()
    w = wl.Workload("mse", 8, 1 << 20, 64, "normal", seed=0)
    x = wl.as_u16(wl.make_inputs(w))
    base = to_f64(oracle.allreduce_bf16(x)[0])

    def mse(**kw):
        d = to_f64(oracle.allreduce_variant(x, 64, **kw)["out"][0]) - base
        return float(np.mean(d * d))

    semi = mse(semi_loop=True, quant_rs=True, quant_ag=True)
    ag_only = mse(semi_loop=False, quant_rs=False, quant_ag=True)
    full = mse(semi_loop=False, quant_rs=True, quant_ag=True)
    assert 0.85 * p["semi_loop_rs_ag"] <= semi <= 1.15 * p["semi_loop_rs_ag"], semi
    assert 0.85 * p["full_loop_ag_only"] <= ag_only <= 1.2 * p["full_loop_ag_only"], ag_only
    assert ag_only < semi < full          # the order of the three flavours in Fig. 7


def test_full_loop_variant_equals_the_ring_loop():
    x = wl.as_u16(wl.make_inputs(wl.C1, count=4 * 256 * 3))
    a = oracle.allreduce(x, 256, trace=True)
    b = oracle.allreduce_variant(x, 256, False, True, True, trace=True)
    for key in ("out", "codes", "scales"):
        assert np.array_equal(a[key], b[key]), key
    assert np.array_equal(oracle.allreduce_variant(x, 256, False, False, False)["out"], oracle.allreduce_bf16(x))


def test_two_ranks_semi_loop_is_the_full_loop():
    """With two ranks both rings are the single hop 1 -> 0 (and 0 -> 1)."""
    x = wl.as_u16(wl.make_inputs(wl.Workload("t", 2, 2 * 64 * 5, 64, "normal", seed=4)))
    for _, qr, qa in FLAVOURS[:4]:
        f = oracle.allreduce_variant(x, 64, False, qr, qa, trace=True)
        s = oracle.allreduce_variant(x, 64, True, qr, qa, trace=True)
        for key in ("out", "codes", "scales"):
            assert np.array_equal(f[key], s[key]), (qr, qa, key)


@pytest.mark.parametrize("semi,qr,qa", FLAVOURS)
def test_exact_integers_give_the_plain_sum(semi, qr, qa):
    """Small integers with a 127 planted on the first sender(s) of every block: all scales are 1,
    bf16 holds every partial sum, so every flavour must return the integer AllReduce."""
    rng = np.random.default_rng(5)
    N, B, bps = 6, 64, 2
    shard = B * bps
    x = rng.integers(-9, 10, size=(N, N * shard)).astype(np.float64)
    for k in range(N):
        firsts = [(k + N // 2) % N, (k + N // 2 + 1) % N] if semi else [(k + 1) % N]
        for b in range(bps):
            pos = k * shard + b * B + 2 * np.arange(len(firsts))
            x[:, pos] = 0.0
            for f, p in zip(firsts, pos):
                x[f, p] = 127.0
    total = x.sum(axis=0)
    assert np.abs(total).max() <= 127
    res = oracle.allreduce_variant(words_of(x), B, semi, qr, qa, trace=True)
    for r in range(N):
        assert np.array_equal(to_f64(res["out"][r]), total)
    used = res["scales"][res["scales"] != 0]
    assert np.all(used == np.float32(1.0))
    n_events = (N - 1 if qr else 0) + (1 if qa else 0)
    assert used.size == n_events * N * bps


def test_semi_loop_chain_order_from_scales():
    """Rank r holds the constant 2^r: the scale of a hop names the ranks summed so far.
    Chain A runs k+N/2, k+N/2-1, ..., k+1; chain B runs k+N/2+1, ..., k+N-1; the owner adds B, then A."""
    N, B = 8, 64
    x = np.zeros((N, N * B))
    for r in range(N):
        x[r, :] = 2.0 ** r
    res = oracle.allreduce_variant(words_of(x), B, True, True, True, trace=True)
    h = N // 2
    for k in range(N):
        run = 0.0
        for j in range(h):                                    # events 0..h-1: chain A
            run += 2.0 ** ((k + h - j) % N)
            assert res["scales"][k, j, 0] == np.float32(run) / np.float32(127.0), (k, j)
        run = 0.0
        for j in range(h - 1):                                # events h..N-2: chain B
            run += 2.0 ** ((k + h + 1 + j) % N)
            assert res["scales"][k, h + j, 0] == np.float32(run) / np.float32(127.0), (k, j)
        assert res["scales"][k, N - 1, 0] == np.float32(255.0) / np.float32(127.0)
    assert np.all(to_f64(res["out"]) == 255.0)


def test_all_gather_only_is_quantize_then_dequantize_of_the_bf16_ring():
    x = wl.as_u16(wl.make_inputs(wl.Workload("t", 4, 4 * 128 * 3, 128, "normal", seed=8)))
    ring = oracle.allreduce_bf16(x)
    codes, scales = oracle.quantize_blocks(ring[0], 128)
    expect = oracle.ag_dequant(codes, scales, 128)
    got = oracle.allreduce_variant(x, 128, False, False, True)["out"]
    for r in range(4):
        assert np.array_equal(got[r], expect)


def test_reduce_scatter_only_keeps_the_owner_sum_unquantized():
    """RS-only: the last hop's fp32 sum is only rounded to bf16, so it is closer to the exact sum
    than the fully quantized result, and its error obeys the hop bound without the last event."""
    w = wl.Workload("t", 8, 8 * 64 * 64, 64, "normal", seed=12)
    x = wl.as_u16(wl.make_inputs(w))
    exact = to_f64(x).sum(axis=0)
    rs = oracle.allreduce_variant(x, 64, False, True, False, trace=True)
    both = oracle.allreduce_variant(x, 64, False, True, True, trace=True)
    assert np.array_equal(rs["codes"][:, :7], both["codes"][:, :7])          # same hops
    assert not rs["scales"][:, 7].any()                                      # no all-gather event
    err_rs = np.abs(to_f64(rs["out"][0]) - exact)
    half_steps = np.repeat(rs["scales"][:, :7].astype(np.float64).sum(axis=1).reshape(-1), 64) * (0.5 + 2.0 ** -14)
    assert np.all(err_rs <= half_steps + 2.0 ** -7.9 * np.abs(to_f64(rs["out"][0])))
    assert np.mean(err_rs ** 2) < np.mean((to_f64(both["out"][0]) - exact) ** 2)


def test_variant_argument_errors():
    x = np.zeros((3, 3 * 64), np.uint16)
    with pytest.raises(oracle.OracleError):
        oracle.allreduce_variant(x, 64, semi_loop=True)        # odd number of ranks
