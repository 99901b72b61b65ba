"""Python binding of the C ABI in include/equarx.h (ctypes, argument marshalling only).

Every function has the name of its C entry point without the ``equarx_``
prefix, takes device pointers as integers or as objects with ``data_ptr()``
(torch tensors), and raises :class:`EquarxError` on a non-zero status.
There is no CPU fallback: if the library cannot be loaded the import fails.
"""
import ctypes

from . import _build

MAX_RANKS = 64
(OK, ERR_NULL, ERR_NRANKS, ERR_BLOCK, ERR_COUNT, ERR_ALIGN, ERR_WORKSPACE, ERR_ALIAS, ERR_CUDA, ERR_STATIC_LIMIT,
 ERR_FLAVOUR) = range(11)
FLAVOUR_SEMI_LOOP, FLAVOUR_QUANT_RS, FLAVOUR_QUANT_AG, FLAVOUR_E4M3, FLAVOUR_E5M2 = 1, 2, 4, 8, 16
FLAVOUR_FIFO_BYTES = 16 * 1024 * 1024
STATIC_WORKSPACE_BYTES = 16 * 1024 * 1024

EXPORTS = (
    "equarx_quantize_blocks",
    "equarx_rs_step_dequant_add_requant",
    "equarx_ag_dequant",
    "equarx_allreduce_sim_workspace_bytes",
    "equarx_allreduce_sim",
    "equarx_allreduce_sim_flavour",
    "equarx_allreduce_sim_flavour_workspace_bytes",
    "equarx_allreduce_sim_pipelined",
    "equarx_allreduce_sim_pipelined_workspace_bytes",
    "equarx_allreduce_sim_host",
    "equarx_allreduce_sim_pipelined_unordered",
    "equarx_ring_allreduce",
    "equarx_ring_mailbox_bytes",
    "equarx_allreduce_sim_host_staging_bytes",
    "equarx_allreduce_sim_range",
    "equarx_allreduce_sim_static",
    "equarx_allreduce_sim_bf16_workspace_bytes",
    "equarx_allreduce_sim_bf16",
    "equarx_status_string",
    "equarx_last_cuda_error",
)


class EquarxError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)}")


def _load():
    path = _build.build()
    lib = ctypes.CDLL(path)
    vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.equarx_quantize_blocks.argtypes = [vp, sz, ci, vp, vp, vp]
    lib.equarx_rs_step_dequant_add_requant.argtypes = [vp, vp, vp, sz, ci, vp, vp, vp]
    lib.equarx_ag_dequant.argtypes = [vp, vp, sz, ci, vp, vp]
    lib.equarx_allreduce_sim_workspace_bytes.argtypes = [ci, sz, ci, ci]
    lib.equarx_allreduce_sim_workspace_bytes.restype = sz
    lib.equarx_allreduce_sim.argtypes = [vp, vp, ci, sz, ci, vp, sz, ci, vp]
    lib.equarx_allreduce_sim_range.argtypes = [vp, vp, ci, sz, ci, vp, sz, ci, ci, ci, vp]
    lib.equarx_allreduce_sim_pipelined.argtypes = [vp, vp, ci, sz, ci, vp, sz, ci, vp]
    lib.equarx_allreduce_sim_pipelined_workspace_bytes.argtypes = [ci, sz, ci, ci]
    lib.equarx_allreduce_sim_pipelined_workspace_bytes.restype = sz
    lib.equarx_allreduce_sim_pipelined_unordered.argtypes = [vp, vp, ci, sz, ci, vp]
    lib.equarx_allreduce_sim_host.argtypes = [vp, vp, ci, sz, ci, vp, sz, vp]
    lib.equarx_allreduce_sim_host_staging_bytes.argtypes = [ci, sz]
    lib.equarx_allreduce_sim_host_staging_bytes.restype = sz
    lib.equarx_ring_mailbox_bytes.argtypes = [ci, sz, ci]
    lib.equarx_ring_mailbox_bytes.restype = sz
    lib.equarx_ring_allreduce.argtypes = [vp, vp, ci, ci, ci, sz, ci, vp, ctypes.c_uint32, ctypes.c_uint64, vp, vp]
    lib.equarx_allreduce_sim_flavour.argtypes = [vp, vp, ci, sz, ci, ci, vp, sz, ci, vp]
    lib.equarx_allreduce_sim_flavour_workspace_bytes.argtypes = [ci, sz, ci, ci, ci]
    lib.equarx_allreduce_sim_flavour_workspace_bytes.restype = sz
    lib.equarx_allreduce_sim_static.argtypes = [vp, vp, ci, sz, ci, vp]
    lib.equarx_allreduce_sim_bf16_workspace_bytes.argtypes = [ci, sz]
    lib.equarx_allreduce_sim_bf16_workspace_bytes.restype = sz
    lib.equarx_allreduce_sim_bf16.argtypes = [vp, vp, ci, sz, vp, sz, vp]
    lib.equarx_status_string.argtypes = [ci]
    lib.equarx_status_string.restype = ctypes.c_char_p
    lib.equarx_last_cuda_error.argtypes = []
    for name in EXPORTS:
        if getattr(lib, name).restype is None:
            getattr(lib, name).restype = ci
    return lib


lib = _load()
LIB_PATH = lib._name


def _ptr(x):
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return int(x)


def _table(ptrs):
    if ptrs is None:
        return None
    return (ctypes.c_void_p * len(ptrs))(*[_ptr(p) for p in ptrs])


def _check(status, where):
    if status != OK:
        raise EquarxError(status, where)


def status_string(status):
    return lib.equarx_status_string(int(status)).decode()


def last_cuda_error():
    return lib.equarx_last_cuda_error()


def quantize_blocks(x_bf16, count, block, codes, scales, stream=0):
    _check(lib.equarx_quantize_blocks(_ptr(x_bf16), count, block, _ptr(codes), _ptr(scales), _ptr(stream)),
           "equarx_quantize_blocks")


def rs_step_dequant_add_requant(codes_in, scales_in, local_bf16, count, block, codes_out, scales_out, stream=0):
    _check(lib.equarx_rs_step_dequant_add_requant(_ptr(codes_in), _ptr(scales_in), _ptr(local_bf16), count, block,
                                                  _ptr(codes_out), _ptr(scales_out), _ptr(stream)),
           "equarx_rs_step_dequant_add_requant")


def ag_dequant(codes, scales, count, block, out_bf16, stream=0):
    _check(lib.equarx_ag_dequant(_ptr(codes), _ptr(scales), count, block, _ptr(out_bf16), _ptr(stream)),
           "equarx_ag_dequant")


def allreduce_sim_workspace_bytes(nranks, count, block, keep_trace=False):
    return lib.equarx_allreduce_sim_workspace_bytes(nranks, count, block, int(bool(keep_trace)))


def allreduce_sim(in_bf16, out_bf16, nranks, count, block, workspace, workspace_bytes, keep_trace=False, stream=0):
    _check(lib.equarx_allreduce_sim(_table(in_bf16), _table(out_bf16), nranks, count, block, _ptr(workspace),
                                    workspace_bytes, int(bool(keep_trace)), _ptr(stream)),
           "equarx_allreduce_sim")


def allreduce_sim_pipelined_workspace_bytes(nranks, count, block, keep_trace=False):
    return lib.equarx_allreduce_sim_pipelined_workspace_bytes(nranks, count, block, int(bool(keep_trace)))


def allreduce_sim_pipelined(in_bf16, out_bf16, nranks, count, block, workspace, workspace_bytes, keep_trace=False,
                            stream=0):
    _check(lib.equarx_allreduce_sim_pipelined(_table(in_bf16), _table(out_bf16), nranks, count, block,
                                              _ptr(workspace), workspace_bytes, int(bool(keep_trace)), _ptr(stream)),
           "equarx_allreduce_sim_pipelined")


def allreduce_sim_pipelined_unordered(in_bf16, out_bf16, nranks, count, block, stream=0):
    """The chain-fused single launch for a call that is independent of the stream's unfinished earlier
    work (the caller's promise): starts while that work is finishing, completes after it."""
    _check(lib.equarx_allreduce_sim_pipelined_unordered(_table(in_bf16), _table(out_bf16), nranks, count, block,
                                                        _ptr(stream)),
           "equarx_allreduce_sim_pipelined_unordered")


def allreduce_sim_host_staging_bytes(nranks, count):
    return lib.equarx_allreduce_sim_host_staging_bytes(nranks, count)


def allreduce_sim_host(host_in, host_out, nranks, count, block, staging, staging_bytes, stream=0):
    """equarx_allreduce_sim_host: host_in / host_out are HOST pointers (integers, or pinned CPU
    tensors with data_ptr()), staging is device memory; copies and kernel go to `stream`."""
    _check(lib.equarx_allreduce_sim_host(_table(host_in), _table(host_out), nranks, count, block, _ptr(staging),
                                         staging_bytes, _ptr(stream)),
           "equarx_allreduce_sim_host")


def ring_mailbox_bytes(nranks, count, block):
    return lib.equarx_ring_mailbox_bytes(nranks, count, block)


def ring_allreduce(in_bf16, out_bf16, rank_first, ranks_here, nranks, count, block, mailboxes, epoch, timeout_ns,
                   status, stream=0):
    """equarx_ring_allreduce: the ranks rank_first .. rank_first+ranks_here-1 of the ring on the current
    device; `mailboxes` lists every rank's mailbox, `status` is 4 uint32 words on the device, zeroed once; status[0] == epoch after a call means it timed out."""
    _check(lib.equarx_ring_allreduce(_table(in_bf16), _table(out_bf16), rank_first, ranks_here, nranks, count, block,
                                     _table(mailboxes), epoch, timeout_ns, _ptr(status), _ptr(stream)),
           "equarx_ring_allreduce")


def allreduce_sim_flavour_workspace_bytes(nranks, count, block, flavour, keep_trace=False):
    return lib.equarx_allreduce_sim_flavour_workspace_bytes(nranks, count, block, flavour, int(bool(keep_trace)))


def allreduce_sim_flavour(in_bf16, out_bf16, nranks, count, block, flavour, workspace, workspace_bytes,
                          keep_trace=False, stream=0):
    _check(lib.equarx_allreduce_sim_flavour(_table(in_bf16), _table(out_bf16), nranks, count, block, flavour,
                                            _ptr(workspace), workspace_bytes, int(bool(keep_trace)), _ptr(stream)),
           "equarx_allreduce_sim_flavour")


def allreduce_sim_range(in_bf16, out_bf16, nranks, count, block, workspace, workspace_bytes, keep_trace,
                        first_launch, last_launch, stream=0):
    _check(lib.equarx_allreduce_sim_range(_table(in_bf16), _table(out_bf16), nranks, count, block, _ptr(workspace),
                                          workspace_bytes, int(bool(keep_trace)), first_launch, last_launch,
                                          _ptr(stream)),
           "equarx_allreduce_sim_range")


def allreduce_sim_static(in_bf16, out_bf16, nranks, count, block, stream=0):
    """equarx_allreduce_sim with the library's built-in 16 MiB workspace: for callers that
    have no scratch memory to give and may not allocate any.  All calls on a device share
    that workspace, so calls that could overlap on the GPU must be ordered by the caller;
    make the first call on a device outside stream capture."""
    _check(lib.equarx_allreduce_sim_static(_table(in_bf16), _table(out_bf16), nranks, count, block, _ptr(stream)),
           "equarx_allreduce_sim_static")


def allreduce_sim_bf16_workspace_bytes(nranks, count):
    return lib.equarx_allreduce_sim_bf16_workspace_bytes(nranks, count)


def allreduce_sim_bf16(in_bf16, out_bf16, nranks, count, workspace, workspace_bytes, stream=0):
    _check(lib.equarx_allreduce_sim_bf16(_table(in_bf16), _table(out_bf16), nranks, count, _ptr(workspace),
                                         workspace_bytes, _ptr(stream)),
           "equarx_allreduce_sim_bf16")


RECORD_BYTES, RECORD_HEADER, TILE_ELEMS = 544, 32, 512
PIPELINE_MIN_WORKSPACE_BYTES = 32


def trace_views(workspace_u8, nranks, count, block, keep_trace=True):
    """Unpack a message workspace (1-D uint8 torch tensor or numpy array) into
    (scales float32 [slots, blocks per shard], codes int8 [slots, shard]) copies.

    slots = N*N for a trace (slot k*N + j = event j of shard k) or 2*N for the ping-pong
    layout (slot 2*k + (j&1)).  The workspace stores 544-byte records: 8 floats of metadata,
    then 512 codes, one record per 512-element tile of a message.
    """
    shard = count // nranks
    bps = shard // block
    tiles = (shard + TILE_ELEMS - 1) // TILE_ELEMS
    slots = nranks * nranks if keep_trace else 2 * nranks
    per_tile = TILE_ELEMS // block
    rec = workspace_u8[:slots * tiles * RECORD_BYTES].reshape(slots, tiles, RECORD_BYTES)
    if hasattr(workspace_u8, "numpy"):      # torch tensor
        import torch
        hdr = rec[:, :, :RECORD_HEADER].contiguous().view(torch.float32)
        sc = hdr[:, :, :per_tile].reshape(slots, tiles * per_tile)[:, :bps].contiguous()
        co = rec[:, :, RECORD_HEADER:].contiguous().view(torch.int8).reshape(slots, tiles * TILE_ELEMS)[:, :shard]
        return sc, co.contiguous()
    import numpy as np
    hdr = np.ascontiguousarray(rec[:, :, :RECORD_HEADER]).view(np.float32)
    sc = np.ascontiguousarray(hdr[:, :, :per_tile].reshape(slots, tiles * per_tile)[:, :bps])
    co = np.ascontiguousarray(rec[:, :, RECORD_HEADER:]).view(np.int8).reshape(slots, tiles * TILE_ELEMS)[:, :shard]
    return sc, np.ascontiguousarray(co)
