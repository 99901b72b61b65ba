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


# ---------------------------------------------------------------- FP8 payloads
from conftest import load_golden            # noqa: E402
from exact_fp import chain_allreduce         # noqa: E402

FP8_GOLD = load_golden("hand_blocks_fp8.txt")


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_fp8_hand_worked_block(fmt):
    g = FP8_GOLD[fmt]
    x = words_of([float(v) for v in g["x"]])[None, :]
    res = oracle.allreduce_variant(x, 8, False, True, True, trace=True, payload=fmt)
    assert res["scales"][0, 0, 0].view(np.uint32) == int(g["scale"][0], 16)
    assert [int(c) & 0xFF for c in res["codes"][0, 0]] == [int(c, 16) for c in g["codes"]]
    assert np.array_equal(to_f64(res["out"][0]), np.array([float(v) for v in g["out"]]))


def _fp8_value(byte, fmt):
    p, emin, bias = (4, -6, 7) if fmt == "e4m3" else (3, -14, 15)
    field, mant = (byte & 0x7F) >> (p - 1), byte & ((1 << (p - 1)) - 1)
    a = mant * 2.0 ** (emin - (p - 1)) if field == 0 else (1 + mant / 2 ** (p - 1)) * 2.0 ** (field - bias)
    return -a if byte & 0x80 else a


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("kind", ["normal", "wide", "tiny"])
@pytest.mark.parametrize("nranks,block,bps", [(1, 4, 2), (2, 3, 1), (3, 5, 2), (4, 8, 1)])
def test_fp8_brute_force_exact_rational(fmt, kind, nranks, block, bps):
    from test_oracle_pins_chain import rand_bf16
    from exact_fp import f32_word
    rng = np.random.default_rng(hash((fmt, kind, nranks, block)) % (2 ** 32))
    x = rand_bf16(rng, (nranks, nranks * block * bps), kind)
    res = oracle.allreduce_variant(x, block, False, True, True, trace=True, payload=fmt)
    out, events = chain_allreduce([[int(w) for w in row] for row in x], block, payload=fmt)
    for r in range(nranks):
        # FP8 has a negative zero code and the rational model has no signed zero: compare -0 as 0
        assert [0 if int(w) == 0x8000 else int(w) for w in res["out"][r]] == out
    for (k, b, j), (scale, vals) in events.items():
        assert int(res["scales"][k, j, b].view(np.uint32)) == f32_word(scale)
        got = [_fp8_value(int(c) & 0xFF, fmt) for c in res["codes"][k, j, b * block:(b + 1) * block]]
        assert got == [float(v) for v in vals]


@pytest.mark.parametrize("fmt,top", [("e4m3", 448.0), ("e5m2", 57344.0)])
def test_fp8_invariants(fmt, top):
    """Every non-zero event has a code of magnitude FMAX; outputs identical on all ranks;
    scaling all inputs by a power of two scales scales and outputs and leaves the codes alone."""
    x = wl.as_u16(wl.make_inputs(wl.Workload("t", 4, 4 * 64 * 6, 64, "normal", seed=3)))
    res = oracle.allreduce_variant(x, 64, False, True, True, trace=True, payload=fmt)
    vals = np.vectorize(lambda c: _fp8_value(int(c) & 0xFF, fmt))(res["codes"]).reshape(4, 4, -1, 64)
    assert np.all(np.abs(vals).max(axis=3) == top)
    for r in range(1, 4):
        assert np.array_equal(res["out"][0], res["out"][r])
    y = torch.tensor(to_f64(x) * 2.0 ** 7).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    res2 = oracle.allreduce_variant(y, 64, False, True, True, trace=True, payload=fmt)
    assert np.array_equal(res2["codes"], res["codes"])
    assert np.array_equal(res2["scales"], res["scales"] * np.float32(128.0))
    assert np.array_equal(to_f64(res2["out"]), to_f64(res["out"]) * 128.0)


def test_fp8_error_is_larger_than_int8_and_ordered():
    """With 3 and 2 mantissa bits the FP8 payloads are coarser than int8 on N(0,1) data."""
    x = wl.as_u16(wl.make_inputs(wl.Workload("t", 8, 8 * 64 * 256, 64, "normal", seed=0)))
    exact = to_f64(x).sum(axis=0)
    mse = {}
    for fmt in ("int8", "e4m3", "e5m2"):
        d = to_f64(oracle.allreduce_variant(x, 64, False, True, True, payload=fmt)["out"][0]) - exact
        mse[fmt] = float(np.mean(d * d))
    assert mse["int8"] < mse["e4m3"] < mse["e5m2"]


# ---------------------------------------------------------------- adder tree, bit for bit
def _fp8_or_int(c, payload):
    return float(int(c)) if payload == "int8" else _fp8_value(int(c) & 0xFF, payload)


@pytest.mark.parametrize("payload", ["int8", "e4m3", "e5m2"])
@pytest.mark.parametrize("kind", ["normal", "wide", "halves", "tiny"])
@pytest.mark.parametrize("semi,qr,qa", FLAVOURS)
@pytest.mark.parametrize("nranks,block,bps", [(2, 4, 1), (4, 3, 2), (6, 5, 1), (8, 2, 1)])
def test_adder_tree_exact_rational(payload, kind, semi, qr, qa, nranks, block, bps):
    """Fig. 4 / Fig. 5 evaluated with rationals and one explicit rounding per IEEE operation
    (tests/exact_fp.py, written from the figures) must give the oracle's scales, codes and outputs
    bit for bit: in particular the semi-loop owner, which adds chain B's message to its own shard,
    then chain A's, each by one fused multiply-add, and stays in fp32 in between."""
    if payload != "int8" and not (qr or qa):
        pytest.skip("nothing is quantized: the payload does not matter")
    from test_oracle_pins_chain import rand_bf16
    from exact_fp import f32_word, tree_allreduce
    rng = np.random.default_rng(hash((payload, kind, semi, qr, qa, nranks, block)) % (2 ** 32))
    x = rand_bf16(rng, (nranks, nranks * block * bps), kind)
    res = oracle.allreduce_variant(x, block, semi, qr, qa, trace=True, payload=payload)
    out, events = tree_allreduce([[int(w) for w in row] for row in x], block, semi, qr, qa, payload)
    for r in range(nranks):
        assert [0 if int(w) == 0x8000 else int(w) for w in res["out"][r]] == out
    assert len(events) == ((nranks - 1 if qr else 0) + (1 if qa else 0)) * nranks * bps
    for (k, b, j), (scale, vals) in events.items():
        assert int(res["scales"][k, j, b].view(np.uint32)) == f32_word(scale), (k, b, j)
        got = [_fp8_or_int(c, payload) for c in res["codes"][k, j, b * block:(b + 1) * block]]
        assert got == [float(v) for v in vals], (k, b, j)


# ---------------------------------------------------------------- randomized shapes (hypothesis)
from hypothesis import HealthCheck, given, settings, strategies as st   # noqa: E402


@settings(max_examples=60, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(half=st.integers(1, 4), block=st.integers(1, 6), bps=st.integers(1, 2),
       flavour=st.integers(0, 7), payload=st.sampled_from(["int8", "e4m3", "e5m2"]),
       kind=st.sampled_from(["normal", "wide", "halves", "tiny"]), seed=st.integers(0, 2 ** 31 - 1))
def test_random_shapes_against_the_exact_rational_tree(half, block, bps, flavour, payload, kind, seed):
    """Any even rank count up to 8, any block length, every flavour and payload: the oracle equals the
    rational evaluation of the adder chain / tree bit for bit."""
    from test_oracle_pins_chain import rand_bf16
    from exact_fp import f32_word, tree_allreduce
    semi, qr, qa = bool(flavour & 1), bool(flavour & 2), bool(flavour & 4)
    nranks = 2 * half
    x = rand_bf16(np.random.default_rng(seed), (nranks, nranks * block * bps), kind)
    res = oracle.allreduce_variant(x, block, semi, qr, qa, trace=True, payload=payload)
    out, events = tree_allreduce([[int(w) for w in row] for row in x], block, semi, qr, qa, payload)
    for r in range(nranks):
        assert [0 if int(w) == 0x8000 else int(w) for w in res["out"][r]] == out
    for (k, b, j), (scale, vals) in events.items():
        assert int(res["scales"][k, j, b].view(np.uint32)) == f32_word(scale)
        got = [_fp8_or_int(c, payload) for c in res["codes"][k, j, b * block:(b + 1) * block]]
        assert got == [float(v) for v in vals]
