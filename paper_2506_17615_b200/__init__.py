"""B200-native hot path of EQuARX (arXiv 2506.17615): block-wise int8 quantize,
per-hop dequantize / fp32 add / requantize and all-gather dequantize of a ring
AllReduce, simulated on one GPU over N ranks.  The work is done by
hand-written sm_100a kernels behind a C ABI (include/equarx.h); this package
is the thin binding.  ``workloads`` holds the seeded synthetic inputs.

The CUDA library is loaded (and, if stale, built) on the first access to one of
the binding's names, not on ``import``: ``workloads`` draws random tensors only and
can be used without the library.  There is no CPU path: the first access to a
binding name raises if the library cannot be built or loaded.
"""
import importlib

_BINDING_NAMES = (
    "FLAVOUR_E4M3",
    "FLAVOUR_E5M2",
    "FLAVOUR_QUANT_AG",
    "FLAVOUR_QUANT_RS",
    "FLAVOUR_SEMI_LOOP",
    "EquarxError",
    "LIB_PATH",
    "MAX_RANKS",
    "ag_dequant",
    "allreduce_sim",
    "allreduce_sim_bf16",
    "allreduce_sim_bf16_workspace_bytes",
    "allreduce_sim_flavour",
    "allreduce_sim_flavour_workspace_bytes",
    "allreduce_sim_host",
    "allreduce_sim_host_staging_bytes",
    "allreduce_sim_pipelined",
    "allreduce_sim_pipelined_unordered",
    "allreduce_sim_pipelined_workspace_bytes",
    "allreduce_sim_range",
    "allreduce_sim_static",
    "allreduce_sim_workspace_bytes",
    "last_cuda_error",
    "lib",
    "quantize_blocks",
    "ring_allreduce",
    "ring_mailbox_bytes",
    "rs_step_dequant_add_requant",
    "status_string",
    "trace_views",
)

__all__ = list(_BINDING_NAMES) + ["binding", "workloads"]


def __getattr__(name):
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(".binding", __name__), name)
    if name in ("binding", "workloads", "ring"):
        return importlib.import_module("." + name, __name__)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
