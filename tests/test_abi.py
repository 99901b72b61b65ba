"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function include/equarx.h declares, and rejects bad arguments before
touching CUDA (fake, never dereferenced device addresses are enough)."""
import ctypes
import os
import re

import paper_2506_17615_b200 as eq
from paper_2506_17615_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
A = 0x7000_0000_0000          # a made-up, well aligned "device address"
MB = 1 << 20


def declared_functions():
    text = open(os.path.join(ROOT, "include", "equarx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(equarx_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    names = declared_functions()
    assert len(names) >= 9
    raw = ctypes.CDLL(eq.LIB_PATH)
    for name in names:
        assert hasattr(raw, name), name
    assert sorted(binding.EXPORTS) == names


def test_binding_has_the_same_names():
    for name in declared_functions():
        assert hasattr(eq, name[len("equarx_"):]), name


def test_status_strings():
    for st in range(9):
        s = eq.status_string(st)
        assert s.startswith("EQUARX_")
    assert "unknown" in eq.status_string(99)


def test_workspace_bytes():
    # N=4, n=65536: shard 16384 = 32 tiles of 512 elements, 544 bytes per record
    assert eq.allreduce_sim_workspace_bytes(4, 65536, 256, False) == 8 * 32 * 544
    assert eq.allreduce_sim_workspace_bytes(4, 65536, 256, True) == 16 * 32 * 544
    # a shard smaller than a tile still takes one record per slot
    assert eq.allreduce_sim_workspace_bytes(1, 64, 64, False) == 2 * 544
    assert eq.allreduce_sim_workspace_bytes(3, 3 * 5 * 128, 128, True) == 9 * 2 * 544     # 640 elements: 2 tiles
    assert eq.allreduce_sim_workspace_bytes(3, 65536, 256, False) == 0      # not divisible
    assert eq.allreduce_sim_workspace_bytes(4, 65536, 100, False) == 0
    assert eq.allreduce_sim_workspace_bytes(65, 65 * 256, 256, False) == 0
    assert eq.allreduce_sim_pipelined_workspace_bytes(4, 65536, 256, False) == binding.PIPELINE_MIN_WORKSPACE_BYTES
    assert eq.allreduce_sim_pipelined_workspace_bytes(4, 65536, 256, True) == 16 * 32 * 544
    assert eq.allreduce_sim_pipelined_workspace_bytes(4, 65536, 99, True) == 0
    assert eq.allreduce_sim_bf16_workspace_bytes(4, 65536) == 4 * 65536
    assert eq.allreduce_sim_bf16_workspace_bytes(4, 65530) == 0


def test_trace_views_unpack_records():
    import numpy as np
    n, count, block = 2, 2 * 640, 128          # shard 640 = 5 blocks = 2 tiles (the second one ragged)
    ws = np.zeros(eq.allreduce_sim_workspace_bytes(n, count, block, True), np.uint8)
    rec = ws.reshape(4, 2, 544)
    for slot in range(4):
        for t in range(2):
            hdr = np.zeros(8, np.float32)
            hdr[:4] = [slot * 100 + t * 4 + i for i in range(4)]
            rec[slot, t, :32] = hdr.view(np.uint8)
            rec[slot, t, 32:] = (np.arange(512) % 100 + slot).astype(np.int8).view(np.uint8)
    sc, co = eq.trace_views(ws, n, count, block, True)
    assert sc.shape == (4, 5) and co.shape == (4, 640)
    assert list(sc[3]) == [300, 301, 302, 303, 304]
    assert co[2, 0] == 2 and co[2, 511] == 11 % 100 + 2 and co[2, 512] == 2 and co[2, 639] == 127 % 100 + 2


def status_of(fn, *args, **kw):
    try:
        fn(*args, **kw)
    except eq.EquarxError as e:
        return e.status
    return 0


def test_per_step_calls_reject_bad_arguments():
    q = eq.quantize_blocks
    assert status_of(q, 0, 256, 256, A + MB, A + 2 * MB) == binding.ERR_NULL
    assert status_of(q, A, 256, 96, A + MB, A + 2 * MB) == binding.ERR_BLOCK
    assert status_of(q, A, 0, 256, A + MB, A + 2 * MB) == binding.ERR_COUNT
    assert status_of(q, A, 300, 256, A + MB, A + 2 * MB) == binding.ERR_COUNT
    assert status_of(q, A + 16, 256, 256, A + MB, A + 2 * MB) == binding.ERR_ALIGN   # bf16 needs 32 bytes
    assert status_of(q, A, 256, 256, A + MB + 8, A + 2 * MB) == binding.ERR_ALIGN
    assert status_of(q, A, 256, 256, A + MB, A + 2 * MB + 2) == binding.ERR_ALIGN
    assert status_of(q, A, 256, 256, A + 256, A + 2 * MB) == binding.ERR_ALIAS       # codes inside x

    s = eq.rs_step_dequant_add_requant
    ok = dict(codes_in=A, scales_in=A + MB, local_bf16=A + 2 * MB, count=512, block=128,
              codes_out=A + 3 * MB, scales_out=A + 4 * MB)
    for key in ("codes_in", "scales_in", "local_bf16", "codes_out", "scales_out"):
        assert status_of(s, **{**ok, key: 0}) == binding.ERR_NULL
    assert status_of(s, **{**ok, "block": 32}) == binding.ERR_BLOCK
    assert status_of(s, **{**ok, "count": 520}) == binding.ERR_COUNT
    assert status_of(s, **{**ok, "codes_out": A}) == binding.ERR_ALIAS               # in place is not allowed
    assert status_of(s, **{**ok, "scales_out": A + MB}) == binding.ERR_ALIAS
    assert status_of(s, **{**ok, "local_bf16": A + 2 * MB + 16}) == binding.ERR_ALIGN

    d = eq.ag_dequant
    assert status_of(d, A, A + MB, 512, 512, 0) == binding.ERR_NULL
    assert status_of(d, A, A + MB, 512, 1024, A + 2 * MB) == binding.ERR_BLOCK
    assert status_of(d, A, A + MB, 512, 512, A + 2 * MB + 8) == binding.ERR_ALIGN
    assert status_of(d, A, A + MB, 512, 512, A) == binding.ERR_ALIAS


def sim_args(nranks=4, count=65536, block=256, in_place=False):
    ins = [A + r * 16 * MB for r in range(nranks)]
    outs = ins if in_place else [A + (64 + r) * 16 * MB for r in range(nranks)]
    ws = A + 200 * 16 * MB
    wb = eq.allreduce_sim_workspace_bytes(nranks, count, block)
    return dict(in_bf16=ins, out_bf16=list(outs), nranks=nranks, count=count, block=block,
                workspace=ws, workspace_bytes=wb)


def test_sim_rejects_bad_arguments():
    f = eq.allreduce_sim
    a = sim_args()
    assert status_of(f, **{**a, "nranks": 0}) == binding.ERR_NRANKS
    assert status_of(f, **{**a, "nranks": 65}) == binding.ERR_NRANKS
    assert status_of(f, **{**a, "block": 100}) == binding.ERR_BLOCK
    assert status_of(f, **{**a, "count": 65536 + 256}) == binding.ERR_COUNT   # not a multiple of N*B
    assert status_of(f, **{**a, "workspace": 0}) == binding.ERR_NULL
    assert status_of(f, **{**a, "workspace_bytes": a["workspace_bytes"] - 1}) == binding.ERR_WORKSPACE
    assert status_of(f, **{**a, "workspace": a["workspace"] + 8}) == binding.ERR_ALIGN
    bad = dict(a); bad["in_bf16"] = a["in_bf16"][:3] + [0]
    assert status_of(f, **bad) == binding.ERR_NULL
    bad = dict(a); bad["out_bf16"] = [a["out_bf16"][0] + 16] + a["out_bf16"][1:]
    assert status_of(f, **bad) == binding.ERR_ALIGN
    bad = dict(a); bad["out_bf16"] = [a["in_bf16"][1]] + a["out_bf16"][1:]     # out[0] on another rank's input
    assert status_of(f, **bad) == binding.ERR_ALIAS
    bad = dict(a); bad["out_bf16"] = [a["in_bf16"][0] + 64] + a["out_bf16"][1:]  # partial overlap with own input
    assert status_of(f, **bad) == binding.ERR_ALIAS
    bad = dict(a); bad["out_bf16"] = [a["out_bf16"][1]] + a["out_bf16"][1:]     # two outputs share a buffer
    assert status_of(f, **bad) == binding.ERR_ALIAS
    bad = dict(a); bad["workspace"] = a["in_bf16"][2]
    assert status_of(f, **bad) == binding.ERR_ALIAS
    assert status_of(f, None, a["out_bf16"], 4, 65536, 256, a["workspace"], a["workspace_bytes"]) == binding.ERR_NULL


def test_bf16_sim_rejects_bad_arguments():
    f = eq.allreduce_sim_bf16
    ins = [A + r * 16 * MB for r in range(4)]
    outs = [A + (64 + r) * 16 * MB for r in range(4)]
    ws = A + 200 * 16 * MB
    assert status_of(f, ins, outs, 0, 65536, ws, 4 * 65536) == binding.ERR_NRANKS
    assert status_of(f, ins, outs, 4, 65536 + 8, ws, 4 * 65536 + 32) == binding.ERR_COUNT
    assert status_of(f, ins, outs, 4, 65536, 0, 4 * 65536) == binding.ERR_NULL
    assert status_of(f, ins, outs, 4, 65536, ws, 4 * 65536 - 1) == binding.ERR_WORKSPACE
    assert status_of(f, ins, [ins[1]] + outs[1:], 4, 65536, ws, 4 * 65536) == binding.ERR_ALIAS


def test_host_entry_rejects_bad_arguments():
    """equarx_allreduce_sim_host validates before any copy is enqueued."""
    f = eq.allreduce_sim_host
    H = 0x5000_0000_0000           # made-up host addresses
    hin = [H + r * MB for r in range(4)]
    hout = [H + (16 + r) * MB for r in range(4)]
    stage = A
    sb = eq.allreduce_sim_host_staging_bytes(4, 65536)
    assert sb == 2 * 65536 * 4
    assert eq.allreduce_sim_host_staging_bytes(0, 65536) == 0
    assert status_of(f, hin, hout, 0, 65536, 256, stage, sb) == binding.ERR_NRANKS
    assert status_of(f, hin, hout, 4, 65536, 96, stage, sb) == binding.ERR_BLOCK
    assert status_of(f, hin, hout, 4, 65536 + 256, 256, stage, sb + 4096) == binding.ERR_COUNT
    assert status_of(f, hin, hout, 4, 65536, 256, 0, sb) == binding.ERR_NULL
    assert status_of(f, hin[:3] + [0], hout, 4, 65536, 256, stage, sb) == binding.ERR_NULL
    assert status_of(f, None, hout, 4, 65536, 256, stage, sb) == binding.ERR_NULL
    assert status_of(f, hin, hout, 4, 65536, 256, stage, sb - 1) == binding.ERR_WORKSPACE
    assert status_of(f, hin, hout, 4, 65536, 256, stage + 16, sb) == binding.ERR_ALIGN
    assert status_of(f, [hin[0] + 1] + hin[1:], hout, 4, 65536, 256, stage, sb) == binding.ERR_ALIGN
    assert status_of(f, hin, [hin[1]] + hout[1:], 4, 65536, 256, stage, sb) == binding.ERR_ALIAS
    assert status_of(f, hin, [hout[1]] + hout[1:], 4, 65536, 256, stage, sb) == binding.ERR_ALIAS


def test_static_entry_validates_before_any_cuda_call():
    """NULL, misaligned and aliased tables, and problems beyond the built-in workspace, are
    rejected on the host: these calls run on a machine without a GPU."""
    f = eq.allreduce_sim_static
    a = sim_args()
    ins, outs = a["in_bf16"], a["out_bf16"]
    assert status_of(f, ins[:3] + [0], outs, 4, 65536, 256) == binding.ERR_NULL
    assert status_of(f, None, outs, 4, 65536, 256) == binding.ERR_NULL
    assert status_of(f, ins, [outs[0] + 16] + outs[1:], 4, 65536, 256) == binding.ERR_ALIGN
    assert status_of(f, ins, [ins[1]] + outs[1:], 4, 65536, 256) == binding.ERR_ALIAS
    assert status_of(f, ins, outs, 4, 65536, 100) == binding.ERR_BLOCK
    big = 8 * 256 * 4096 * 4            # needs more than 16 MiB of message slots
    assert eq.allreduce_sim_workspace_bytes(8, big, 256) > binding.STATIC_WORKSPACE_BYTES
    assert status_of(f, [A] * 8, [A] * 8, 8, big, 256) == binding.ERR_STATIC_LIMIT
    assert eq.last_cuda_error() == 0


def test_no_cuda_error_recorded_by_validation():
    assert eq.last_cuda_error() == 0


def test_rounded_code_never_leaves_the_int8_range_without_a_clamp():
    """The kernels omit the oracle's clamp to [-127, 127].  That is safe iff
    rne(fl(amax * fl(127 / amax))) == 127 for every block maximum: the largest |v| of a block
    gives the largest product, and multiplication by a positive constant is monotone.  Checked
    for every fp32 mantissa in several binades (scaling amax by a power of two scales
    fl(127 / amax) by the inverse power exactly, as long as nothing leaves the normal range),
    including the smallest block that is still quantized (2^-118) and the bf16 maximum."""
    import numpy as np
    mant = np.arange(1 << 23, dtype=np.uint32)
    for exp_field in (9, 64, 127, 128, 200, 254):          # 2^-118, ..., 1, 2, ..., up to 2^127
        amax = ((np.uint32(exp_field) << np.uint32(23)) | mant).view(np.float32)
        inv = np.float32(127.0) / amax
        assert np.all(np.isfinite(inv)) and np.all(inv > 0)
        top = amax * inv                                   # fp32 multiply, round to nearest even
        assert top.dtype == np.float32
        assert float(top.max()) < 127.5 and float(top.min()) > 126.5
        # and the scale that travels is a normal number
        scale = amax / np.float32(127.0)
        assert float(scale.min()) >= 2.0 ** -126
