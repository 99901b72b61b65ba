"""ctypes front end of the C oracle: compiles it with gcc on first use.

Argument marshalling only; every number comes from ``equarx_oracle.c``.
"""
import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "equarx_oracle.c")
_SO = os.path.join(_HERE, "libequarx_oracle.so")
_lock = threading.Lock()
_lib = None


class OracleError(RuntimeError):
    def __init__(self, status, where):
        super().__init__(f"{where}: oracle status {status}")
        self.status = status


def lib_path():
    return _SO


def build(force=False):
    """Compile the oracle (gcc, -O2, no contraction, no fast-math)."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = f"{_SO}.{os.getpid()}.tmp"
            cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
                   "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        lib.equarx_oracle_quantize_blocks.argtypes = [vp, sz, ci, vp, vp]
        lib.equarx_oracle_rs_step.argtypes = [vp, vp, vp, sz, ci, vp, vp]
        lib.equarx_oracle_ag_dequant.argtypes = [vp, vp, sz, ci, vp]
        lib.equarx_oracle_allreduce.argtypes = [vp, vp, ci, sz, ci, vp, vp, vp]
        lib.equarx_oracle_allreduce_bf16.argtypes = [vp, vp, ci, sz]
        lib.equarx_oracle_allreduce_variant.argtypes = [vp, vp, ci, sz, ci, ci, ci, ci, ci, vp, vp]
        lib.equarx_oracle_error_bound.argtypes = [vp, vp, ci, sz, ci, vp]
        for name in ("quantize_blocks", "rs_step", "ag_dequant", "allreduce",
                     "allreduce_bf16", "error_bound", "allreduce_variant"):
            getattr(lib, "equarx_oracle_" + name).restype = ci
        _lib = lib
    return _lib


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a):
    return ctypes.c_void_p(a.ctypes.data)


def _check(status, where):
    if status != 0:
        raise OracleError(status, where)


def quantize_blocks(x_bf16, block):
    """x_bf16: uint16[count] -> (codes int8[count], scales float32[count/block])."""
    x = _arr(x_bf16, np.uint16).ravel()
    if block < 1 or x.size % block:
        raise OracleError(4 if block >= 1 else 3, "quantize_blocks")
    codes = np.empty(x.size, np.int8)
    scales = np.empty(x.size // block, np.float32)
    _check(_load().equarx_oracle_quantize_blocks(_p(x), x.size, block, _p(codes), _p(scales)),
           "quantize_blocks")
    return codes, scales


def rs_step(codes_in, scales_in, local_bf16, block):
    ci = _arr(codes_in, np.int8).ravel()
    si = _arr(scales_in, np.float32).ravel()
    lo = _arr(local_bf16, np.uint16).ravel()
    if block < 1 or ci.size % block or lo.size != ci.size or si.size != ci.size // block:
        raise OracleError(4, "rs_step")
    co = np.empty(ci.size, np.int8)
    so = np.empty(si.size, np.float32)
    _check(_load().equarx_oracle_rs_step(_p(ci), _p(si), _p(lo), ci.size, block, _p(co), _p(so)),
           "rs_step")
    return co, so


def ag_dequant(codes, scales, block):
    c = _arr(codes, np.int8).ravel()
    s = _arr(scales, np.float32).ravel()
    if block < 1 or c.size % block or s.size != c.size // block:
        raise OracleError(4, "ag_dequant")
    out = np.empty(c.size, np.uint16)
    _check(_load().equarx_oracle_ag_dequant(_p(c), _p(s), c.size, block, _p(out)), "ag_dequant")
    return out


def _ptr_array(rows):
    return (ctypes.c_void_p * len(rows))(*[r.ctypes.data for r in rows])


def allreduce(inputs_bf16, block, trace=False, exact=False):
    """inputs_bf16: uint16[nranks, count].

    Returns a dict: ``out`` uint16[nranks, count]; with ``trace`` also
    ``scales`` float32[N shards, N events, blocks/shard] and ``codes``
    int8[N, N, count/N]; with ``exact`` also ``exact_sum`` float64[count].
    """
    x = _arr(inputs_bf16, np.uint16)
    if x.ndim != 2:
        raise ValueError("inputs must be [nranks, count]")
    n_ranks, count = x.shape
    if block < 1:
        raise OracleError(3, "allreduce")
    if count == 0 or count % (n_ranks * block):
        raise OracleError(4, "allreduce")
    out = np.empty_like(x)
    rows_in = [x[r] for r in range(n_ranks)]
    rows_out = [out[r] for r in range(n_ranks)]
    res = {"out": out}
    ts = tc = ex = None
    if trace:
        bps = count // n_ranks // block
        ts = np.empty((n_ranks, n_ranks, bps), np.float32)
        tc = np.empty((n_ranks, n_ranks, count // n_ranks), np.int8)
        res["scales"], res["codes"] = ts, tc
    if exact:
        ex = np.empty(count, np.float64)
        res["exact_sum"] = ex
    _check(_load().equarx_oracle_allreduce(
        _ptr_array(rows_in), _ptr_array(rows_out), n_ranks, count, block,
        _p(ts) if trace else None, _p(tc) if trace else None, _p(ex) if exact else None),
        "allreduce")
    return res


PAYLOADS = {"int8": 0, "e4m3": 1, "e5m2": 2}


def allreduce_variant(inputs_bf16, block, semi_loop=False, quant_rs=True, quant_ag=True, trace=False,
                      payload="int8"):
    """The flavours of Sections 3.3 / 3.4: full-loop or semi-loop ring, with the reduce-scatter
    hops and/or the all-gather quantized, int8 or FP8 payload.  Returns a dict like allreduce();
    trace codes are the raw payload bytes."""
    x = _arr(inputs_bf16, np.uint16)
    n_ranks, count = x.shape
    if block < 1:
        raise OracleError(3, "allreduce_variant")
    if count == 0 or count % (n_ranks * block):
        raise OracleError(4, "allreduce_variant")
    out = np.empty_like(x)
    res = {"out": out}
    ts = tc = None
    if trace:
        ts = np.empty((n_ranks, n_ranks, count // n_ranks // block), np.float32)
        tc = np.empty((n_ranks, n_ranks, count // n_ranks), np.int8)
        res["scales"], res["codes"] = ts, tc
    _check(_load().equarx_oracle_allreduce_variant(
        _ptr_array([x[r] for r in range(n_ranks)]), _ptr_array([out[r] for r in range(n_ranks)]),
        n_ranks, count, block, int(semi_loop), int(quant_rs), int(quant_ag), PAYLOADS[payload],
        _p(ts) if trace else None, _p(tc) if trace else None), "allreduce_variant")
    return res


def allreduce_bf16(inputs_bf16):
    x = _arr(inputs_bf16, np.uint16)
    n_ranks, count = x.shape
    if count == 0 or count % n_ranks:
        raise OracleError(4, "allreduce_bf16")
    out = np.empty_like(x)
    _check(_load().equarx_oracle_allreduce_bf16(
        _ptr_array([x[r] for r in range(n_ranks)]), _ptr_array([out[r] for r in range(n_ranks)]),
        n_ranks, count), "allreduce_bf16")
    return out


def error_bound(trace_scales, out_row_bf16, n_ranks, block):
    ts = _arr(trace_scales, np.float32)
    o = _arr(out_row_bf16, np.uint16).ravel()
    bound = np.empty(o.size, np.float64)
    _check(_load().equarx_oracle_error_bound(_p(ts), _p(o), n_ranks, o.size, block, _p(bound)),
           "error_bound")
    return bound
