"""Oracle pins: hand-worked blocks, closed forms and special cases.

Expected values come from tests/golden/hand_blocks.txt (worked by hand from
the quantization rule of Section 3.2 and the hop of Section 3.1) or from
plain mathematics; none comes from the oracle itself.
"""
import numpy as np
import pytest
import torch

import oracle
from conftest import load_golden

GOLD = load_golden("hand_blocks.txt")


def bf16_words(values):
    t = torch.tensor([float(v) for v in values], dtype=torch.float64).to(torch.bfloat16)
    assert torch.equal(t.double(), torch.tensor([float(v) for v in values], dtype=torch.float64)), \
        "golden inputs must be exact bf16 values"
    return t.view(torch.int16).numpy().view(np.uint16)


def words(hexes):
    return np.array([int(h, 16) for h in hexes], dtype=np.uint16)


def f32_from_words(hexes):
    return np.array([int(h, 16) for h in hexes], dtype=np.uint32).view(np.float32)


def ints(vals):
    return np.array([int(v) for v in vals], dtype=np.int8)


def test_hand_chain_a_b():
    g = GOLD["chain_a_b"]
    a, b = bf16_words(g["a"]), bf16_words(g["b"])
    c0, s0 = oracle.quantize_blocks(a, 4)
    assert s0.view(np.uint32)[0] == int(g["event0_scale"][0], 16)
    assert np.array_equal(c0, ints(g["event0_codes"]))
    c1, s1 = oracle.rs_step(c0, s0, b, 4)
    assert s1.view(np.uint32)[0] == int(g["event1_scale"][0], 16)
    assert np.array_equal(c1, ints(g["event1_codes"]))
    out = oracle.ag_dequant(c1, s1, 4)
    assert np.array_equal(out, words(g["out_bf16"]))
    # the same chain through the ring simulation: N = 2, shard 0 runs rank 1 -> rank 0
    # and shard 1 runs rank 0 -> rank 1, so put a/b crosswise
    x = np.stack([np.concatenate([b, a]), np.concatenate([a, b])])
    res = oracle.allreduce(x, 4, trace=True)
    for k in range(2):
        assert res["scales"][k, 0, 0].view(np.uint32) == int(g["event0_scale"][0], 16)
        assert res["scales"][k, 1, 0].view(np.uint32) == int(g["event1_scale"][0], 16)
        assert np.array_equal(res["codes"][k, 0], ints(g["event0_codes"]))
        assert np.array_equal(res["codes"][k, 1], ints(g["event1_codes"]))
        for r in range(2):
            assert np.array_equal(res["out"][r, 4 * k:4 * k + 4], words(g["out_bf16"]))


def test_hand_chain_intermediate_sum():
    """acc of the worked chain, seen through a second hop with a zero local shard."""
    g = GOLD["chain_a_b"]
    a, b = bf16_words(g["a"]), bf16_words(g["b"])
    c0, s0 = oracle.quantize_blocks(a, 4)
    acc = f32_from_words(g["acc_f32"]).astype(np.float64)
    # requantizing acc by hand: amax = 3, codes = rne(acc * fl(127/3))
    inv = np.float32(127.0) / np.float32(3.0)
    expect = np.rint((acc.astype(np.float32) * inv).astype(np.float32)).astype(np.int8)
    c1, _ = oracle.rs_step(c0, s0, b, 4)
    assert np.array_equal(c1, expect)


@pytest.mark.parametrize("case", ["ties", "spike", "reciprocal_of_amax"])
def test_hand_value_blocks(case):
    g = GOLD[case]
    x = bf16_words(g["x"])
    codes, scales = oracle.quantize_blocks(x, len(x))
    assert scales.view(np.uint32)[0] == int(g["scale"][0], 16)
    assert np.array_equal(codes, ints(g["codes"]))


@pytest.mark.parametrize("case", ["bf16_max", "flush_edge_kept", "flush_edge_dropped"])
def test_hand_word_blocks(case):
    g = GOLD[case]
    x = words(g["x_words"])
    codes, scales = oracle.quantize_blocks(x, len(x))
    assert scales.view(np.uint32)[0] == int(g["scale"][0], 16)
    assert np.array_equal(codes, ints(g["codes"]))
    if "out_bf16" in g:
        assert np.array_equal(oracle.ag_dequant(codes, scales, len(x)), words(g["out_bf16"]))


def test_zero_blocks_give_zero_scale_and_exact_zeros():
    x = np.zeros((4, 4 * 64), np.uint16)
    x[1, 5] = 0x8000     # a negative zero is still a zero block
    res = oracle.allreduce(x, 64, trace=True)
    assert not res["scales"].view(np.uint32).any()
    assert not res["codes"].any()
    assert not res["out"].any()


def test_single_rank_is_one_quantization_round_trip():
    """N = 1: one event per block, out = bf16(code * scale), error within half a step."""
    rng = np.random.default_rng(1)
    xf = torch.tensor(rng.standard_normal(4096) * 3.0).to(torch.bfloat16)
    x = xf.view(torch.int16).numpy().view(np.uint16)[None, :]
    B = 128
    res = oracle.allreduce(x, B, trace=True)
    assert res["scales"].shape == (1, 1, 4096 // B)
    xv = xf.double().numpy().reshape(-1, B)
    amax = np.abs(xv).max(axis=1)
    scale = res["scales"][0, 0].astype(np.float64)
    # the scale is amax/127 rounded once to fp32
    assert np.all(np.abs(scale - amax / 127.0) <= amax / 127.0 * 2.0 ** -24)
    out = torch.from_numpy(res["out"][0].view(np.int16)).view(torch.bfloat16).double().numpy()
    err = np.abs(out.reshape(-1, B) - xv)
    # half a quantization step, plus the final bf16 rounding (2^-9 relative)
    assert np.all(err <= scale[:, None] * (0.5 + 2.0 ** -14) + np.abs(out.reshape(-1, B)) * 2.0 ** -8)
    # the block maximum maps to +-127 and comes back within one bf16 rounding
    codes = res["codes"][0, 0].reshape(-1, B)
    assert np.all(np.abs(codes).max(axis=1) == 127)


def test_exact_integer_chain_equals_plain_sum():
    """Integer inputs whose partial sums stay within +-127, with 127 planted at
    the head of every block chain: every scale is exactly 1, every
    quantization exact, so the result is the textbook integer AllReduce."""
    rng = np.random.default_rng(7)
    N, B, bps = 5, 64, 3
    shard = B * bps
    count = N * shard
    x = rng.integers(-12, 13, size=(N, count)).astype(np.float64)
    for k in range(N):
        first = (k + 1) % N
        for b in range(bps):
            pos = k * shard + b * B + int(rng.integers(0, B))
            x[:, pos] = 0.0
            x[first, pos] = 127.0
    total = x.sum(axis=0)
    assert np.abs(total).max() <= 127
    xw = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    res = oracle.allreduce(xw, B, trace=True, exact=True)
    assert np.all(res["scales"] == np.float32(1.0))
    out = torch.from_numpy(res["out"].view(np.int16)).view(torch.bfloat16).double().numpy()
    for r in range(N):
        assert np.array_equal(out[r], total)
    assert np.array_equal(res["exact_sum"], total)
    # event j of shard k carries the running integer sum over ranks k+1 .. k+1+j
    for k in range(N):
        run = np.zeros(shard)
        for j in range(N):
            run += x[(k + 1 + j) % N, k * shard:(k + 1) * shard]
            assert np.array_equal(res["codes"][k, j].astype(np.float64), run)


def test_bf16_ring_baseline_on_exact_integers():
    rng = np.random.default_rng(3)
    x = rng.integers(-15, 16, size=(4, 4 * 32)).astype(np.float64)
    xw = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    out = oracle.allreduce_bf16(xw)
    o = torch.from_numpy(out.view(np.int16)).view(torch.bfloat16).double().numpy()
    for r in range(4):
        assert np.array_equal(o[r], x.sum(axis=0))


def test_bf16_ring_baseline_rounds_every_hop():
    """1 + 2^-8 is not a bf16 value: each hop's rounding (ties to even) is visible."""
    one, tiny = 1.0, 2.0 ** -8
    N = 3
    # shard 0 chain runs rank 1 -> 2 -> 0: (tiny + tiny) + one = 1 + 2^-7 exactly representable;
    # shard 1 chain runs rank 2 -> 0 -> 1: (one + tiny) -> tie -> 1.0, then + tiny -> tie -> 1.0
    x = np.zeros((N, N), np.float64)
    x[1, 0], x[2, 0], x[0, 0] = tiny, tiny, one
    x[2, 1], x[0, 1], x[1, 1] = one, tiny, tiny
    xw = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    out = oracle.allreduce_bf16(xw)
    o = torch.from_numpy(out.view(np.int16)).view(torch.bfloat16).double().numpy()
    assert o[0, 0] == 1.0 + 2.0 ** -7
    assert o[0, 1] == 1.0


def test_argument_errors():
    x = np.zeros((2, 64), np.uint16)
    with pytest.raises(oracle.OracleError):
        oracle.allreduce(x, 64)            # count not a multiple of nranks * block
    with pytest.raises(oracle.OracleError):
        oracle.allreduce(x, 0)
    bad = np.zeros((2, 128), np.uint16)
    bad[0, 3] = 0x7F80                     # +inf
    with pytest.raises(oracle.OracleError) as e:
        oracle.allreduce(bad, 64)
    assert e.value.status == 9
