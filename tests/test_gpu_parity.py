"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs.  Bar: bit-exact int8 codes, bit-exact fp32
scales, and 0-ulp bf16 outputs (there is no op-order freedom in the path: the
max is order independent and every rounding step is an explicit IEEE op)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

BLOCKS = (64, 128, 256, 512)


def _values(kind, count, seed, nranks=4):
    g = torch.Generator().manual_seed(seed)
    if kind == "normal":
        v = torch.randn(count, generator=g)
    elif kind == "wide":        # 40 binades per tensor: exercises scale range and tiny/huge ratios
        v = torch.randn(count, generator=g) * torch.exp2(torch.randint(-20, 20, (count,), generator=g).float())
    elif kind == "halves":      # exact .5 products against a block max of 127: ties
        v = torch.randint(-254, 255, (count,), generator=g).float() / 2.0
        v[::64] = 127.0
    elif kind == "tiny":        # around the flush threshold and among bf16 subnormals
        v = (torch.randint(-127, 128, (count,), generator=g).double()
             * torch.exp2(torch.randint(-133, -112, (count,), generator=g).double()))
    elif kind == "huge":        # as large as the fp32 partial sums of nranks tensors allow (finite sums are the contract)
        v = torch.randn(count, generator=g).clamp(-6, 6).double() * 2.0 ** 125 / (2 * max(nranks, 3))
    elif kind == "zeros":
        v = torch.zeros(count)
        v[1::7] = -0.0
    else:
        raise ValueError(kind)
    return v.to(torch.bfloat16)


KINDS = ("normal", "wide", "halves", "tiny", "huge", "zeros")


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


@pytest.mark.parametrize("block", BLOCKS)
@pytest.mark.parametrize("kind", KINDS)
def test_step_kernels_match_oracle(gu, block, kind):
    """quantize -> hop -> hop -> all-gather dequantize on one buffer; several 4096-element
    tiles plus a ragged tail of 5 blocks."""
    count = 3 * 4096 + 5 * block
    x = [_values(kind, count, 100 + i) for i in range(3)]
    xw = [wl.as_u16(t) for t in x]
    xd = [t.cuda() for t in x]
    nb = count // block
    codes = [gu.Guarded(count) for _ in range(3)]
    scales = [gu.Guarded(4 * nb) for _ in range(3)]
    out = gu.Guarded(2 * count)
    s = gu.stream_handle()
    eq.quantize_blocks(xd[0], count, block, codes[0], scales[0], s)
    eq.rs_step_dequant_add_requant(codes[0], scales[0], xd[1], count, block, codes[1], scales[1], s)
    eq.rs_step_dequant_add_requant(codes[1], scales[1], xd[2], count, block, codes[2], scales[2], s)
    eq.ag_dequant(codes[2], scales[2], count, block, out, s)
    torch.cuda.synchronize()
    for b in codes + scales + [out]:
        b.check()
    c0, s0 = oracle.quantize_blocks(xw[0], block)
    c1, s1 = oracle.rs_step(c0, s0, xw[1], block)
    c2, s2 = oracle.rs_step(c1, s1, xw[2], block)
    o = oracle.ag_dequant(c2, s2, block)
    for i, (c, sc) in enumerate(((c0, s0), (c1, s1), (c2, s2))):
        assert np.array_equal(codes[i].view(torch.int8).cpu().numpy(), c), f"codes of event {i}"
        assert np.array_equal(scales[i].view(torch.float32).cpu().numpy().view(np.uint32), sc.view(np.uint32)), \
            f"scales of event {i}"
    gu.assert_same_words(out.view(torch.bfloat16), o, "all-gather output")


@pytest.mark.parametrize("block", BLOCKS)
def test_single_block_and_one_tile_edges(gu, block):
    for count in (block, 4096, 4096 + block):
        if count % block:
            continue
        x = _values("normal", count, count)
        c = gu.Guarded(count)
        sc = gu.Guarded(4 * (count // block))
        eq.quantize_blocks(x.cuda(), count, block, c, sc, gu.stream_handle())
        torch.cuda.synchronize()
        c.check(); sc.check()
        ec, es = oracle.quantize_blocks(wl.as_u16(x), block)
        assert np.array_equal(c.view(torch.int8).cpu().numpy(), ec)
        assert np.array_equal(sc.view(torch.float32).cpu().numpy().view(np.uint32), es.view(np.uint32))


VARIANTS = ("steps", "pipelined")


def _compare_full(gu, x, block, in_place=False):
    """Both schedules (one launch per ring step; one deep-pipelined launch) against the oracle:
    the whole trace of messages and the outputs, bit for bit."""
    n_ranks, count = x.shape
    xd = x.cuda()
    res = oracle.allreduce(wl.as_u16(x), block, trace=True)
    last = {}
    for variant in VARIANTS:
        out, ws = gu.run_sim(xd, block, keep_trace=True, in_place=in_place, variant=variant)
        sc, co = eq.trace_views(ws.u8, n_ranks, count, block, keep_trace=True)
        assert np.array_equal(co.cpu().numpy().reshape(res["codes"].shape), res["codes"]), f"{variant}: trace codes"
        assert np.array_equal(sc.cpu().numpy().view(np.uint32).reshape(res["scales"].shape),
                              res["scales"].view(np.uint32)), f"{variant}: trace scales"
        gu.assert_same_words(out, res["out"], f"{variant}: outputs")
        # without a trace (what the bench runs): same outputs; the step schedule leaves the last two
        # events of every shard in its ping-pong workspace
        out2, ws2 = gu.run_sim(xd, block, keep_trace=False, in_place=in_place, variant=variant)
        assert torch.equal(out2.view(torch.int16), out.view(torch.int16)), variant
        if variant == "steps":
            sc2, co2 = eq.trace_views(ws2.u8, n_ranks, count, block, keep_trace=False)
            for k in range(n_ranks):
                for j in range(max(0, n_ranks - 2), n_ranks):
                    assert np.array_equal(co2[2 * k + (j & 1)].cpu().numpy(), res["codes"][k, j]), (k, j)
                    assert np.array_equal(sc2[2 * k + (j & 1)].cpu().numpy().view(np.uint32),
                                          res["scales"][k, j].view(np.uint32)), (k, j)


def test_config1_small_normal_full(gu):
    x = wl.make_inputs(wl.C1)
    _compare_full(gu, x, wl.C1.block)


@pytest.mark.parametrize("nranks", (1, 2, 3, 5, 8, 16, 64))
@pytest.mark.parametrize("block", BLOCKS)
def test_rank_counts_and_blocks(gu, nranks, block):
    # 5 blocks per shard for the large blocks (ragged vs the 4096-element tile), more for small ones
    bps = 5 if block >= 256 else 37
    w = wl.Workload("t", nranks, nranks * bps * block, block, "normal", seed=nranks)
    _compare_full(gu, wl.make_inputs(w), block)


@pytest.mark.parametrize("w,rows", [(wl.C2, 32), (wl.C3, 32)])
def test_activation_shaped_configs_reduced(gu, w, rows):
    """Configs 2 and 3 with fewer token rows (same hidden size, outlier channels, distribution)."""
    count = rows * w.hidden
    assert count % (w.nranks * w.block) == 0
    _compare_full(gu, wl.make_inputs(w, count=count), w.block)


def test_stress_config_reduced(gu):
    w = wl.C5
    _compare_full(gu, wl.make_inputs(w, count=64 * 256 * 16), 256)


def test_in_place(gu):
    w = wl.Workload("t", 8, 8 * 256 * 33, 256, "normal", seed=5)
    _compare_full(gu, wl.make_inputs(w), 256, in_place=True)


@pytest.fixture(scope="module")
def full_size_expected():
    """Oracle outputs of the full-size configs, computed once per test session (the oracle
    evaluates all of config 2 in well under a second and all of config 3 in a few seconds)."""
    cache = {}

    def get(w):
        if w.name not in cache:
            x = wl.make_inputs(w, device="cuda")
            cache.clear()                                   # one config's host copy at a time
            cache[w.name] = (x, oracle.allreduce(wl.as_u16(x), w.block)["out"][0].copy())
        return cache[w.name]
    return get


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("w", [wl.C2, wl.C3], ids=lambda w: w.name)
def test_full_size_every_word(gu, w, variant, full_size_expected):
    """Configs 2 and 3 at full size, in the launch configuration the bench times (no trace):
    EVERY output word of every rank against the oracle's evaluation of the whole tensor."""
    x, exp = full_size_expected(w)
    out, ws = gu.run_sim(x, w.block, keep_trace=False, variant=variant)
    exp_dev = torch.from_numpy(exp.view(np.int16)).cuda()
    for r in range(w.nranks):
        same = torch.equal(out[r].view(torch.int16), exp_dev)
        if not same:
            gu.assert_same_words(out[r], exp, f"{variant} {w.name} rank {r}")
    if variant == "steps":
        _check_last_messages(ws, w)


def _check_last_messages(ws, w):
    # the last two messages of every shard are still in the workspace: codes within +-127
    # and, per block, scale 0 or at least one |code| == 127
    sc, co = eq.trace_views(ws.u8, w.nranks, w.count, w.block, keep_trace=False)
    assert int(co.min()) >= -127
    amax = co.view(2 * w.nranks, -1, w.block).abs().amax(dim=2)
    assert bool(((amax == 127) | (sc == 0)).all())
    assert bool(((sc != 0) | (amax == 0)).all())


@pytest.mark.parametrize("variant", VARIANTS)
def test_stress_config_full_size_sampled(gu, variant):
    """Config 5 at full size (64 ranks x 16 Mi elements: the oracle needs minutes for all of it):
    300 sampled blocks of every shard bit for bit, plus properties that hold at any size."""
    w = wl.C5
    x = wl.make_inputs(w, device="cuda")
    out, ws = gu.run_sim(x, w.block, keep_trace=False, variant=variant)
    for r in range(1, w.nranks):
        assert torch.equal(out[0].view(torch.int16), out[r].view(torch.int16)), "outputs differ across ranks"
    bps = w.count // w.nranks // w.block
    picks = gu.sample_blocks(w.nranks, bps, 300, seed=1)
    exp = gu.oracle_out_on_samples(x, picks, w.block)
    got = gu.gather_blocks(out, picks, w.block)
    gu.assert_same_words(got, exp, "sampled outputs")
    if variant == "steps":
        _check_last_messages(ws, w)


@pytest.mark.parametrize("nranks,count", [(1, 4096), (2, 2 * 4096 + 32), (4, 65536), (7, 7 * 16 * 301), (64, 64 * 4096)])
def test_bf16_comparator_matches_oracle(gu, nranks, count):
    w = wl.Workload("t", nranks, count, 256, "normal", seed=3)
    x = wl.make_inputs(w)
    xd = x.cuda()
    wb = eq.allreduce_sim_bf16_workspace_bytes(nranks, count)
    ws = gu.Guarded(wb)
    outs = [gu.Guarded(2 * count) for _ in range(nranks)]
    eq.allreduce_sim_bf16([xd[r] for r in range(nranks)], outs, nranks, count, ws, wb, gu.stream_handle())
    torch.cuda.synchronize()
    ws.check()
    exp = oracle.allreduce_bf16(wl.as_u16(x))
    for r in range(nranks):
        outs[r].check()
        gu.assert_same_words(outs[r].view(torch.bfloat16), exp[r], f"bf16 ring output of rank {r}")


def test_error_within_bound_on_gpu_outputs(gu):
    """End-to-end error of the GPU result against the exact fp64 sum stays under the bound
    accumulated over the hops (bound evaluated by the oracle from the GPU's own trace)."""
    w = wl.C5
    count = 64 * 256 * 8
    x = wl.make_inputs(w, count=count)
    out, ws = gu.run_sim(x.cuda(), 256, keep_trace=True)
    sc, _ = eq.trace_views(ws.u8, 64, count, 256, keep_trace=True)
    bound = oracle.error_bound(sc.cpu().numpy().reshape(64, 64, -1), wl.as_u16(out[0]), 64, 256)
    exact = x.double().sum(dim=0).numpy()
    err = np.abs(out[0].double().cpu().numpy() - exact)
    assert np.all(err <= bound)


def test_error_within_bound_on_config5_at_full_size(gu):
    """Config 5 as specified (64 ranks x 16 Mi elements of zero, spike, subnormal and cancelling blocks):
    the GPU's outputs against the exact fp64 sum, under the bound the oracle derives from the GPU's own
    trace (1.1 GB of messages); int8 range respected in every event; zero blocks stay exactly zero."""
    w = wl.C5
    x = wl.make_inputs(w, device="cuda")
    out, ws = gu.run_sim(x, w.block, keep_trace=True, variant="pipelined")
    sc, co = eq.trace_views(ws.u8, w.nranks, w.count, w.block, keep_trace=True)
    assert int(co.min()) >= -127
    exact = torch.zeros(w.count, dtype=torch.float64, device="cuda")
    for r in range(w.nranks):
        exact += x[r].double()
    bound = oracle.error_bound(sc.cpu().numpy().reshape(w.nranks, w.nranks, -1), wl.as_u16(out[0]), w.nranks, w.block)
    err = (out[0].double() - exact).abs().cpu().numpy()
    assert np.all(err <= bound)
    # the bound is not vacuous: on spike blocks it is far below the spike, on zero blocks it is ~0
    zero_blocks = (x.view(w.nranks, -1, w.block) == 0).all(dim=2).all(dim=0)
    assert bool(zero_blocks.any())
    assert bool((out[0].view(-1, w.block)[zero_blocks] == 0).all())
    assert float(bound.reshape(-1, w.block)[zero_blocks.cpu().numpy()].max()) < 1e-30
    del out, ws, sc, co
    torch.cuda.empty_cache()


def test_launch_ranges_compose_to_the_whole_schedule(gu):
    w = wl.Workload("t", 5, 5 * 256 * 9, 256, "normal", seed=9)
    x = wl.make_inputs(w).cuda()
    ref, _ = gu.run_sim(x, 256)
    wb = eq.allreduce_sim_workspace_bytes(5, w.count, 256, False)
    ws = gu.Guarded(wb)
    outs = [gu.Guarded(2 * w.count) for _ in range(5)]
    ins = [x[r] for r in range(5)]
    for first, last in ((0, 0), (1, 2), (3, 3), (4, 5)):
        eq.allreduce_sim_range(ins, outs, 5, w.count, 256, ws, wb, False, first, last, gu.stream_handle())
    torch.cuda.synchronize()
    for r in range(5):
        outs[r].check()
        assert torch.equal(outs[r].view(torch.int16), ref[r].view(torch.int16))
    with pytest.raises(eq.EquarxError):
        eq.allreduce_sim_range(ins, outs, 5, w.count, 256, ws, wb, False, 2, 6, gu.stream_handle())


SWEEP_SMALL = [(n, b, d, s) for n in (4, 8, 16) for b in (128, 256, 512) for d in ("uniform", "normal")
               for s in (1 << 14, 1 << 17, 1 << 20)]


@pytest.mark.parametrize("nranks,block,dist,nbytes", SWEEP_SMALL)
def test_sweep_points_small_full_compare(gu, nranks, block, dist, nbytes):
    """Message-size sweep, 16 KB .. 1 MB per rank: every output word of both schedules."""
    w = wl.sweep_point(nranks, nbytes, block, dist)
    x = wl.make_inputs(w)
    exp = oracle.allreduce(wl.as_u16(x), block)["out"]
    xd = x.cuda()
    for variant in VARIANTS:
        out, _ = gu.run_sim(xd, block, variant=variant)
        gu.assert_same_words(out, exp, f"{variant} {w.name}")


SWEEP_LARGE = [(n, b, "uniform" if (n + b) % 3 else "normal", s) for n in (4, 8, 16) for b in (128, 256, 512)
               for s in (1 << 24, 1 << 26, 1 << 28)]


@pytest.mark.parametrize("nranks,block,dist,nbytes", SWEEP_LARGE)
def test_sweep_points_large_sampled(gu, nranks, block, dist, nbytes):
    """16 MB, 64 MB and 256 MB per rank, one distribution per (N, block): sampled blocks bit for bit,
    all ranks' outputs identical."""
    w = wl.sweep_point(nranks, nbytes, block, dist)
    x = wl.make_inputs(w, device="cuda")
    picks = gu.sample_blocks(nranks, w.count // nranks // block, 12, seed=nbytes % 1000 + nranks)
    exp = gu.oracle_out_on_samples(x, picks, block)
    for variant in VARIANTS:
        out, _ = gu.run_sim(x, block, variant=variant)
        for r in range(1, nranks):
            assert torch.equal(out[0].view(torch.int16), out[r].view(torch.int16))
        gu.assert_same_words(gu.gather_blocks(out, picks, block), exp, f"{variant} {w.name}")
        del out
    torch.cuda.empty_cache()


def _random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for _ in range(n):
        nranks = int(rng.choice([1, 2, 3, 4, 6, 7, 8, 12, 16, 24, 32, 48, 64]))
        block = int(rng.choice(BLOCKS))
        bps = int(rng.integers(1, 40))
        kind = str(rng.choice(KINDS))
        cases.append((nranks, block, bps, kind, int(rng.integers(0, 1 << 30))))
    return cases


@pytest.mark.parametrize("nranks,block,bps,kind,seed", _random_cases(40, 2024))
def test_randomized_shapes_and_value_ranges(gu, nranks, block, bps, kind, seed):
    """Seeded random draws over rank counts, block sizes, shard lengths (ragged against the
    512-element tile and the 4096-element CTA) and value ranges: both schedules, full trace."""
    count = nranks * bps * block
    x = torch.stack([_values(kind, count, seed + r, nranks) for r in range(nranks)])
    _compare_full(gu, x, block)


def test_chain_fused_form_leaves_its_workspace_alone(gu):
    """Without a trace the single-launch schedule keeps every hop message in registers: the
    (token) workspace must come back untouched."""
    n, block = 4, 128
    count = n * 8 * block
    x = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=77)).cuda()
    wb = eq.allreduce_sim_pipelined_workspace_bytes(n, count, block, False)
    assert wb == binding.PIPELINE_MIN_WORKSPACE_BYTES
    ws = torch.full((4096,), 0x5A, dtype=torch.uint8, device="cuda")
    out = torch.empty_like(x)
    eq.allreduce_sim_pipelined([x[r] for r in range(n)], [out[r] for r in range(n)], n, count, block, ws, wb, False,
                               gu.stream_handle())
    torch.cuda.synchronize()
    assert bool((ws == 0x5A).all())
    gu.assert_same_words(out, oracle.allreduce(wl.as_u16(x), block)["out"], "chain-fused outputs")


@pytest.mark.parametrize("pinned", (True, False))
@pytest.mark.parametrize("in_place", (False, True))
def test_host_buffer_entry_matches_oracle(gu, pinned, in_place):
    """equarx_allreduce_sim_host: host tensors in, host tensors out, copies issued by the library
    on the caller's stream; two calls back to back on two streams with two staging buffers."""
    n, block = 8, 256
    count = n * block * 37
    xs = [wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=s)) for s in (3, 4)]
    exp = [oracle.allreduce(wl.as_u16(x), block)["out"] for x in xs]
    h_in = [x.clone().pin_memory() if pinned else x.clone() for x in xs]
    h_out = h_in if in_place else [torch.zeros_like(x).pin_memory() if pinned else torch.zeros_like(x) for x in xs]
    sb = eq.allreduce_sim_host_staging_bytes(n, count)
    stage = [gu.Guarded(sb) for _ in xs]
    streams = [torch.cuda.Stream() for _ in xs]
    warm = torch.zeros((n, count), dtype=torch.bfloat16).pin_memory()
    eq.allreduce_sim_host([warm[r] for r in range(n)], [warm[r] for r in range(n)], n, count, block, stage[0], sb,
                          streams[0].cuda_stream)        # first use loads the kernel's code onto the device
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for i in range(2):
        eq.allreduce_sim_host([h_in[i][r] for r in range(n)], [h_out[i][r] for r in range(n)], n, count, block,
                              stage[i], sb, streams[i].cuda_stream)
    for st in streams:
        st.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0, "the call changed the amount of free device memory"
    for i in range(2):
        stage[i].check()
        gu.assert_same_words(h_out[i], exp[i], f"host entry, call {i}")
        gu.assert_same_words(stage[i].view(torch.bfloat16).view(n, count), exp[i], "staging holds the reduced tensors")


def test_step_schedule_reuses_its_message_slots_without_stale_reads(gu):
    """The launch-per-step schedule without a trace reuses its ping-pong message slots every two
    steps and every call, under programmatic dependent launch.  Sixty calls back to back on one
    stream, each on different data, must each give the bits of a traced run of the same data."""
    n, block = 8, 256
    count = n * block * 96
    xs = [wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=200 + i)).cuda() for i in range(6)]
    refs = [gu.run_sim(x, block, keep_trace=True)[0] for x in xs]
    wb = eq.allreduce_sim_workspace_bytes(n, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    outs = [torch.empty_like(xs[0]) for _ in range(60)]
    s = gu.stream_handle()
    for i in range(60):
        x = xs[i % 6]
        eq.allreduce_sim([x[r] for r in range(n)], [outs[i][r] for r in range(n)], n, count, block, ws, wb, False, s)
    torch.cuda.synchronize()
    for i in range(60):
        assert torch.equal(outs[i].view(torch.int16), refs[i % 6].view(torch.int16)), f"call {i}"


@pytest.mark.parametrize("nranks", (4, 8, 16))
@pytest.mark.parametrize("block", (128, 256, 512))
@pytest.mark.parametrize("dist", ("uniform", "normal"))
def test_every_sweep_point_sampled(gu, nranks, block, dist):
    """All 15 message sizes (16 KB .. 256 MB per rank) of one (N, block, distribution) line of the
    sweep, in the configuration the sweep times (no trace): sampled blocks of the pipelined schedule
    against the oracle, and the launch-per-step schedule against the pipelined one, word for word."""
    for p in range(14, 29):
        w = wl.sweep_point(nranks, 1 << p, block, dist)
        bps = w.count // nranks // block
        x = wl.make_inputs(w, device="cuda")
        out, _ = gu.run_sim(x, block, variant="pipelined")
        picks = gu.sample_blocks(nranks, bps, 6, seed=p)
        exp = gu.oracle_out_on_samples(x, picks, block)
        gu.assert_same_words(gu.gather_blocks(out, picks, block), exp, w.name)
        out2, _ = gu.run_sim(x, block, variant="steps")
        assert torch.equal(out.view(torch.int16), out2.view(torch.int16)), w.name
        del out, out2, x
        torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", VARIANTS)
def test_offsets_beyond_four_gigabytes(gu, variant):
    """Two ranks of 2^31 + 1024 elements each (4.3 GB per tensor): element and byte offsets pass 2^32.
    Sampled blocks, including the last blocks of both shards, against the oracle."""
    n, block = 2, 512
    count = (1 << 31) + 2 * 512
    g = torch.Generator(device="cuda").manual_seed(99)
    x = torch.empty((n, count), dtype=torch.bfloat16, device="cuda")
    for r in range(n):
        x[r].normal_(generator=g)
    out, _ = gu.run_sim(x, block, variant=variant)
    bps = count // n // block
    picks = gu.sample_blocks(n, bps, 16, seed=3)
    exp = gu.oracle_out_on_samples(x, picks, block)
    gu.assert_same_words(gu.gather_blocks(out, picks, block), exp, variant)
    assert torch.equal(out[0].view(torch.int16), out[1].view(torch.int16))
    del out, x
    torch.cuda.empty_cache()


def test_runs_on_the_stream_it_is_given(gu):
    """The work is enqueued on the caller's stream: issued on a side stream behind a long-running
    fill of the input, it must see the filled input, and the default stream must stay idle."""
    n, block = 4, 256
    count = n * block * 64
    side = torch.cuda.Stream()
    x = torch.zeros((n, count), dtype=torch.bfloat16, device="cuda")
    src = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=31)).cuda()
    out = torch.empty_like(x)
    wb = eq.allreduce_sim_pipelined_workspace_bytes(n, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        big = torch.empty(1 << 28, dtype=torch.float32, device="cuda")
        for _ in range(8):
            big.fill_(1.0)                 # keeps the side stream busy for a while
        x.copy_(src)                       # the inputs only become valid behind that work
        eq.allreduce_sim_pipelined([x[r] for r in range(n)], [out[r] for r in range(n)], n, count, block, ws, wb,
                                   False, side.cuda_stream)
    side.synchronize()
    exp = oracle.allreduce(wl.as_u16(src), block)["out"]
    gu.assert_same_words(out, exp, "side stream")


def test_unordered_single_launch_back_to_back_on_independent_tensors(gu):
    """equarx_allreduce_sim_pipelined_unordered: thirty calls back to back on six independent tensor sets
    (each launch may start while its predecessors are still finishing) give the oracle's bits, and work
    enqueued afterwards still finds ALL earlier work complete: a large ordered AllReduce, a small unordered
    one that finishes its own work first, then a copy of the large one's output."""
    n, block = 8, 256
    count = n * block * 64
    xs = [wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=300 + i)) for i in range(6)]
    exp = [oracle.allreduce(wl.as_u16(x), block)["out"] for x in xs]
    xd = [x.cuda() for x in xs]
    outs = [torch.zeros_like(x) for x in xd]
    s = gu.stream_handle()
    for i in range(30):
        j = i % 6
        eq.allreduce_sim_pipelined_unordered([xd[j][r] for r in range(n)], [outs[j][r] for r in range(n)], n, count,
                                             block, s)
    torch.cuda.synchronize()
    for j in range(6):
        gu.assert_same_words(outs[j], exp[j], f"unordered, set {j}")

    big = wl.make_inputs(wl.C2, device="cuda")                 # 8 x 15.7 MB: tens of microseconds
    big_out = torch.zeros_like(big)
    wb = eq.allreduce_sim_pipelined_workspace_bytes(8, wl.C2.count, 256, False)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    small_out = torch.zeros_like(xd[0])
    torch.cuda.synchronize()
    eq.allreduce_sim_pipelined([big[r] for r in range(8)], [big_out[r] for r in range(8)], 8, wl.C2.count, 256, ws, wb,
                               False, s)
    eq.allreduce_sim_pipelined_unordered([xd[0][r] for r in range(n)], [small_out[r] for r in range(n)], n, count, block, s)
    snapshot = big_out.clone()                                 # ordinary stream work after the unordered call
    torch.cuda.synchronize()
    assert torch.equal(snapshot.view(torch.int16), big_out.view(torch.int16))
    gu.assert_same_words(snapshot, oracle.allreduce(wl.as_u16(big), 256)["out"], "work after an unordered call")
    gu.assert_same_words(small_out, exp[0], "the unordered call itself")


def test_schedules_can_be_recorded_in_a_cuda_graph(gu):
    """The simulation calls only enqueue launches on the given stream (no synchronisation, no allocation),
    so stream capture records them; replaying the graph on new data gives the oracle's bits.  Small
    messages are bound by launch and host-call overhead, which a graph replay removes."""
    n, block = 4, 256
    count = n * block * 24
    x = torch.zeros((n, count), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(x)
    ins, outs = [x[r] for r in range(n)], [out[r] for r in range(n)]
    wb = eq.allreduce_sim_workspace_bytes(n, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    wbf = eq.allreduce_sim_flavour_workspace_bytes(n, count, block, 7, False)
    calls = {"launch per step": lambda s: eq.allreduce_sim(ins, outs, n, count, block, ws, wb, False, s),
             "single launch": lambda s: eq.allreduce_sim_pipelined(ins, outs, n, count, block, ws, wb, False, s),
             "semi-loop flavour": lambda s: eq.allreduce_sim_flavour(ins, outs, n, count, block, 7, ws, wbf, False, s)}
    for name, call in calls.items():
        call(gu.stream_handle())                       # first use outside capture: loads the kernels
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            call(torch.cuda.current_stream().cuda_stream)
        for seed in (61, 62):
            src = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=seed))
            x.copy_(src)
            out.zero_()
            graph.replay()
            torch.cuda.synchronize()
            if name == "semi-loop flavour":
                exp = oracle.allreduce_variant(wl.as_u16(src), block, True, True, True)["out"]
            else:
                exp = oracle.allreduce(wl.as_u16(src), block)["out"]
            gu.assert_same_words(out, exp, f"{name}, graph replay, seed {seed}")


def test_launch_errors_are_reported_not_raised_on_the_gpu(gu, monkeypatch):
    """A failing launch (injected on the host: no kernel runs, the GPU is not touched) comes back
    as EQUARX_ERR_CUDA with the CUDA error code available, from every kind of entry point, and
    the library works again afterwards."""
    n, block = 4, 256
    count = n * block * 4
    x = wl.make_inputs(wl.Workload("t", n, count, block, "normal", seed=1)).cuda()
    out = torch.empty_like(x)
    ins, outs = [x[r] for r in range(n)], [out[r] for r in range(n)]
    wb = max(eq.allreduce_sim_workspace_bytes(n, count, block), eq.allreduce_sim_pipelined_workspace_bytes(n, count, block),
             eq.allreduce_sim_flavour_workspace_bytes(n, count, block, 7))
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    codes = torch.empty(count, dtype=torch.int8, device="cuda")
    scales = torch.empty(count // block, device="cuda")
    s = gu.stream_handle()
    monkeypatch.setenv("EQUARX_INJECT_LAUNCH_ERROR", "719")          # cudaErrorLaunchFailure
    calls = [lambda: eq.allreduce_sim(ins, outs, n, count, block, ws, wb, False, s),
             lambda: eq.allreduce_sim_pipelined(ins, outs, n, count, block, ws, wb, False, s),
             lambda: eq.allreduce_sim_flavour(ins, outs, n, count, block, 7, ws, wb, False, s),
             lambda: eq.quantize_blocks(x[0], count, block, codes, scales, s),
             lambda: eq.allreduce_sim_static(ins, outs, n, count, block, s)]
    for call in calls:
        with pytest.raises(eq.EquarxError) as err:
            call()
        assert err.value.status == binding.ERR_CUDA and eq.last_cuda_error() == 719
    monkeypatch.delenv("EQUARX_INJECT_LAUNCH_ERROR")
    eq.allreduce_sim_pipelined(ins, outs, n, count, block, ws, wb, False, s)
    torch.cuda.synchronize()
    gu.assert_same_words(out, oracle.allreduce(wl.as_u16(x.cpu()), block)["out"], "after the injected failures")
