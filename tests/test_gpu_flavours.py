"""GPU parity of the other flavours (semi-loop ring; quantize reduce-scatter only, all-gather
only, both, none) against the oracle's adder chains: outputs 0 ulp, quantized events bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

FLAVOURS = list(range(8))


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def decode(flavour):
    return bool(flavour & eq.FLAVOUR_SEMI_LOOP), bool(flavour & eq.FLAVOUR_QUANT_RS), bool(flavour & eq.FLAVOUR_QUANT_AG)


def payload_of(flavour):
    return "e4m3" if flavour & eq.FLAVOUR_E4M3 else "e5m2" if flavour & eq.FLAVOUR_E5M2 else "int8"


def run_flavour(gu, xd, block, flavour, keep_trace):
    n, count = xd.shape
    wb = eq.allreduce_sim_flavour_workspace_bytes(n, count, block, flavour, keep_trace)
    assert wb > 0
    ws = gu.Guarded(wb)
    outs = [gu.Guarded(2 * count) for _ in range(n)]
    eq.allreduce_sim_flavour([xd[r] for r in range(n)], outs, n, count, block, flavour, ws, wb, keep_trace,
                             gu.stream_handle())
    torch.cuda.synchronize()
    ws.check()
    for o in outs:
        o.check()
    return torch.stack([o.view(torch.bfloat16) for o in outs]), ws


def compare(gu, x, block, flavour):
    semi, qr, qa = decode(flavour)
    n, count = x.shape
    res = oracle.allreduce_variant(wl.as_u16(x), block, semi, qr, qa, trace=True, payload=payload_of(flavour))
    out, ws = run_flavour(gu, x.cuda(), block, flavour, True)
    gu.assert_same_words(out, res["out"], f"flavour {flavour} outputs")
    sc, co = eq.trace_views(ws.u8[binding.FLAVOUR_FIFO_BYTES:], n, count, block, keep_trace=True)
    assert np.array_equal(co.cpu().numpy().reshape(res["codes"].shape), res["codes"]), f"flavour {flavour} codes"
    assert np.array_equal(sc.cpu().numpy().view(np.uint32).reshape(res["scales"].shape),
                          res["scales"].view(np.uint32)), f"flavour {flavour} scales"
    out2, _ = run_flavour(gu, x.cuda(), block, flavour, False)
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))


@pytest.mark.parametrize("flavour", FLAVOURS)
@pytest.mark.parametrize("nranks", (2, 4, 6, 8, 16, 64))
@pytest.mark.parametrize("block", (64, 256, 512))
def test_flavours_match_oracle(gu, flavour, nranks, block):
    bps = 5 if block >= 256 else 19          # ragged against the 512-element tile
    w = wl.Workload("t", nranks, nranks * bps * block, block, "normal", seed=nranks + flavour)
    compare(gu, wl.make_inputs(w), block, flavour)


@pytest.mark.parametrize("flavour", (0, 2, 4, 6))
@pytest.mark.parametrize("nranks", (1, 3, 5))
def test_full_loop_flavours_odd_rank_counts(gu, flavour, nranks):
    w = wl.Workload("t", nranks, nranks * 128 * 9, 128, "normal", seed=nranks)
    compare(gu, wl.make_inputs(w), 128, flavour)


@pytest.mark.parametrize("flavour", FLAVOURS)
def test_flavours_on_stress_blocks(gu, flavour):
    compare(gu, wl.make_inputs(wl.C5, count=64 * 256 * 6), 256, flavour)


def test_both_quantized_is_the_pipelined_schedule_and_none_is_the_bf16_ring(gu):
    x = wl.make_inputs(wl.Workload("t", 8, 8 * 256 * 21, 256, "normal", seed=2)).cuda()
    ref, _ = gu.run_sim(x, 256, variant="pipelined")
    got, _ = run_flavour(gu, x, 256, eq.FLAVOUR_QUANT_RS | eq.FLAVOUR_QUANT_AG, False)
    assert torch.equal(ref.view(torch.int16), got.view(torch.int16))
    n, count = x.shape
    wb = eq.allreduce_sim_bf16_workspace_bytes(n, count)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    ring = torch.empty_like(x)
    eq.allreduce_sim_bf16([x[r] for r in range(n)], [ring[r] for r in range(n)], n, count, ws, wb, gu.stream_handle())
    torch.cuda.synchronize()
    got0, _ = run_flavour(gu, x, 256, 0, False)
    assert torch.equal(ring.view(torch.int16), got0.view(torch.int16))


@pytest.mark.parametrize("flavour", (1, 3, 7))
def test_semi_loop_full_size_every_word(gu, flavour):
    """Config 2 at full size through the semi-loop flavours: every output word against the oracle."""
    w = wl.C2
    semi, qr, qa = decode(flavour)
    x = wl.make_inputs(w, device="cuda")
    out, _ = run_flavour(gu, x, w.block, flavour, False)
    exp = oracle.allreduce_variant(wl.as_u16(x), w.block, semi, qr, qa)["out"]
    gu.assert_same_words(out, exp, f"flavour {flavour}, config 2")


def test_flavour_argument_errors(gu):
    x = torch.zeros((3, 3 * 64), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(x)
    ws = torch.empty(binding.FLAVOUR_FIFO_BYTES, dtype=torch.uint8, device="cuda")
    args = ([x[r] for r in range(3)], [out[r] for r in range(3)], 3, 3 * 64, 64)
    with pytest.raises(eq.EquarxError) as e:
        eq.allreduce_sim_flavour(*args, 32, ws, ws.numel())
    assert e.value.status == binding.ERR_FLAVOUR
    with pytest.raises(eq.EquarxError) as e:
        eq.allreduce_sim_flavour(*args, eq.FLAVOUR_SEMI_LOOP, ws, ws.numel())      # odd rank count
    assert e.value.status == binding.ERR_NRANKS
    assert eq.allreduce_sim_flavour_workspace_bytes(3, 3 * 64, 64, 1) == 0
    assert eq.allreduce_sim_flavour_workspace_bytes(4, 4 * 64, 64, 1) == binding.PIPELINE_MIN_WORKSPACE_BYTES
    assert eq.allreduce_sim_flavour_workspace_bytes(4, 4 * 64, 64, 1, True) > binding.FLAVOUR_FIFO_BYTES


FP8_FLAVOURS = [sched | fmt for fmt in (eq.FLAVOUR_E4M3, eq.FLAVOUR_E5M2) for sched in (2, 3, 4, 5, 6, 7)]


@pytest.mark.parametrize("flavour", FP8_FLAVOURS)
@pytest.mark.parametrize("nranks,block", [(2, 64), (4, 512), (8, 256), (16, 128)])
def test_fp8_flavours_match_oracle(gu, flavour, nranks, block):
    bps = 5 if block >= 256 else 19
    w = wl.Workload("t", nranks, nranks * bps * block, block, "normal", seed=nranks + flavour)
    compare(gu, wl.make_inputs(w), block, flavour)


@pytest.mark.parametrize("flavour", (6 | eq.FLAVOUR_E4M3, 6 | eq.FLAVOUR_E5M2, 7 | eq.FLAVOUR_E4M3))
@pytest.mark.parametrize("kind", ("wide", "tiny", "huge", "halves", "zeros"))
def test_fp8_value_ranges(gu, flavour, kind):
    """40-binade data, data around the flush thresholds and FP8 subnormals, near the bf16 maximum,
    exact ties, signed zeros."""
    from test_gpu_parity import _values
    n, block = 4, 128
    x = torch.stack([_values(kind, n * block * 7, 50 + r) for r in range(n)])
    compare(gu, x, block, flavour)


@pytest.mark.parametrize("flavour", (6 | eq.FLAVOUR_E4M3, 6 | eq.FLAVOUR_E5M2))
def test_fp8_stress_blocks(gu, flavour):
    compare(gu, wl.make_inputs(wl.C5, count=64 * 256 * 4), 256, flavour)


def test_fp8_flavour_bits_are_validated(gu):
    assert eq.allreduce_sim_flavour_workspace_bytes(4, 4 * 64, 64, eq.FLAVOUR_E4M3) == 0            # nothing quantized
    assert eq.allreduce_sim_flavour_workspace_bytes(4, 4 * 64, 64, 6 | eq.FLAVOUR_E4M3 | eq.FLAVOUR_E5M2) == 0
    assert eq.allreduce_sim_flavour_workspace_bytes(4, 4 * 64, 64, 6 | eq.FLAVOUR_E5M2) == binding.PIPELINE_MIN_WORKSPACE_BYTES
    assert eq.allreduce_sim_flavour_workspace_bytes(4, 4 * 64, 64, 32) == 0


@pytest.mark.parametrize("flavour", (0, 5, 7, 6 | eq.FLAVOUR_E4M3))
def test_flavours_in_place(gu, flavour):
    """out[r] == in[r]: a tile's inputs are all read before any of its outputs is written."""
    n, block = 8, 128
    count = n * block * 21
    x = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=90 + flavour))
    semi, qr, qa = decode(flavour)
    exp = oracle.allreduce_variant(wl.as_u16(x), block, semi, qr, qa, payload=payload_of(flavour))["out"]
    bufs = [gu.Guarded(2 * count) for _ in range(n)]
    for r in range(n):
        bufs[r].view(torch.bfloat16).copy_(x[r])
    wb = eq.allreduce_sim_flavour_workspace_bytes(n, count, block, flavour, False)
    ws = gu.Guarded(wb)
    eq.allreduce_sim_flavour(bufs, bufs, n, count, block, flavour, ws, wb, False, gu.stream_handle())
    torch.cuda.synchronize()
    ws.check()
    for b in bufs:
        b.check()
    gu.assert_same_words(torch.stack([b.view(torch.bfloat16) for b in bufs]), exp, f"flavour {flavour} in place")


def test_host_entry_with_sixty_four_ranks(gu):
    n, block = 64, 64
    count = n * block * 3
    x = wl.make_inputs(wl.Workload("t", n, count, block, "uniform", seed=17))
    exp = oracle.allreduce(wl.as_u16(x), block)["out"]
    h = x.clone().pin_memory()
    sb = eq.allreduce_sim_host_staging_bytes(n, count)
    stage = gu.Guarded(sb)
    eq.allreduce_sim_host([h[r] for r in range(n)], [h[r] for r in range(n)], n, count, block, stage, sb,
                          gu.stream_handle())
    torch.cuda.synchronize()
    stage.check()
    gu.assert_same_words(h, exp, "host entry, 64 ranks, in place")
