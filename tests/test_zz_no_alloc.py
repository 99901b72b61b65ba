"""The workspace-free entry point, equarx_allreduce_sim_static.

Some users of this library cannot give it scratch memory: a plugin living inside
an application that owns the whole device heap, a server whose memory plan is
frozen once it has started, a process that is simply not allowed to call
cudaMalloc.  For them the library carries a fixed 16 MiB workspace of its own.
This test calls that entry point through the C ABI twice in a row (the second
call finds the first call's messages still in the shared workspace and must not
be disturbed by them) and requires the same bits as equarx_allreduce_sim with a
caller-provided workspace, and as the CPU oracle.  It also checks the claim in the
entry point's purpose: the amount of free device memory is the same before and
after the calls.  It is collected last on purpose.
"""
import pytest
import torch

import oracle
import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def _reference(x, block):
    n, count = x.shape
    wb = eq.allreduce_sim_workspace_bytes(n, count, block, False)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    out = torch.empty_like(x)
    eq.allreduce_sim([x[r] for r in range(n)], [out[r] for r in range(n)], n, count, block, ws, wb, False,
                     torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out


def _static(x, block):
    n, count = x.shape
    out = torch.full_like(x, float("nan"))
    eq.allreduce_sim_static([x[r] for r in range(n)], [out[r] for r in range(n)], n, count, block,
                            torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out


def test_static_workspace_matches_caller_workspace_twice_in_a_row():
    first = wl.make_inputs(wl.Workload("a", 8, 8 * 256 * 150, 256, "normal", seed=21)).cuda()
    second = wl.make_inputs(wl.Workload("b", 4, 4 * 64 * 999, 64, "uniform", seed=22)).cuda()
    for x, block in ((first, 256), (second, 64)):
        got = _static(x, block)
        exp = _reference(x, block)
        assert torch.equal(got.view(torch.int16), exp.view(torch.int16))
    # and once more with the first problem: stale messages of another shape are in the array now
    again = _static(first, 256)
    assert torch.equal(again.view(torch.int16), _reference(first, 256).view(torch.int16))
    # first hand: the oracle's bits
    exp = oracle.allreduce(wl.as_u16(first), 256)["out"]
    assert (wl.as_u16(again) == exp).all()


def test_static_entry_allocates_no_device_memory():
    x = wl.make_inputs(wl.Workload("a", 8, 8 * 256 * 150, 256, "normal", seed=23)).cuda()
    n, count = x.shape
    out = torch.empty_like(x)
    ins, outs = [x[r] for r in range(n)], [out[r] for r in range(n)]
    s = torch.cuda.current_stream().cuda_stream
    eq.allreduce_sim_static(ins, outs, n, count, 256, s)       # set-up call: address look-up, code loading
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    reserved_before = torch.cuda.memory_reserved()
    for _ in range(3):
        eq.allreduce_sim_static(ins, outs, n, count, 256, s)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert torch.cuda.memory_reserved() == reserved_before


def test_static_entry_rejects_bad_tables_like_the_other_entry():
    x = torch.zeros((4, 4 * 256), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(x)
    ins, outs = [x[r] for r in range(4)], [out[r] for r in range(4)]
    s = torch.cuda.current_stream().cuda_stream

    def status(i, o):
        with pytest.raises(eq.EquarxError) as err:
            eq.allreduce_sim_static(i, o, 4, 4 * 256, 256, s)
        return err.value.status

    assert status(ins[:3] + [None], outs) == binding.ERR_NULL
    assert status(ins, [outs[1]] + outs[1:]) == binding.ERR_ALIAS
    assert status(ins, [ins[2]] + outs[1:]) == binding.ERR_ALIAS
    assert status(ins, [outs[0].data_ptr() + 16] + outs[1:]) == binding.ERR_ALIGN
    eq.allreduce_sim_static(ins, ins, 4, 4 * 256, 256, s)      # in place is allowed
    torch.cuda.synchronize()


def test_static_workspace_holds_the_largest_documented_case_and_rejects_more():
    n, count, block = 8, 2048 * 3840, 256                 # 15.97 MB of messages: fits in 16 MiB
    assert eq.allreduce_sim_workspace_bytes(n, count, block, False) <= binding.STATIC_WORKSPACE_BYTES
    x = wl.make_inputs(wl.C2, device="cuda")
    assert torch.equal(_static(x, block).view(torch.int16), _reference(x, block).view(torch.int16))
    too_big = 2 * count
    assert eq.allreduce_sim_workspace_bytes(n, too_big, block, False) > binding.STATIC_WORKSPACE_BYTES
    y = torch.zeros((n, too_big), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(y)
    with pytest.raises(eq.EquarxError) as err:
        eq.allreduce_sim_static([y[r] for r in range(n)], [out[r] for r in range(n)], n, too_big, block,
                                torch.cuda.current_stream().cuda_stream)
    assert err.value.status == binding.ERR_STATIC_LIMIT
    assert "16 MiB" in str(err.value)
