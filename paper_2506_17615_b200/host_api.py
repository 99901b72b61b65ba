"""Host-buffer front end: the quantized AllReduce simulation for tensors that live in pinned
host memory.  Copies and kernels are torch/CUDA-runtime plumbing; the arithmetic is the C ABI's.

``HostPipeline`` keeps two sets of device buffers and three streams, so that the upload of call
i+1, the kernels of call i and the download of call i-1 overlap (PCIe is full duplex).  Each
``submit`` is one complete AllReduce: N host tensors in, N host tensors out.
"""
import torch

from . import binding as _b


class HostPipeline:
    def __init__(self, nranks, count, block, device=None, depth=2):
        self.n, self.count, self.block = nranks, count, block
        self.dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.depth = depth
        self.h2d, self.comp, self.d2h = (torch.cuda.Stream(self.dev) for _ in range(3))
        self.d_in = [torch.empty((nranks, count), dtype=torch.bfloat16, device=self.dev) for _ in range(depth)]
        self.d_out = [torch.empty((nranks, count), dtype=torch.bfloat16, device=self.dev) for _ in range(depth)]
        self.wb = _b.allreduce_sim_pipelined_workspace_bytes(nranks, count, block, False)
        self.ws = torch.empty(self.wb, dtype=torch.uint8, device=self.dev)
        self.uploaded = [torch.cuda.Event() for _ in range(depth)]
        self.computed = [torch.cuda.Event() for _ in range(depth)]
        self.downloaded = [torch.cuda.Event() for _ in range(depth)]
        self.calls = 0

    def submit(self, host_in, host_out):
        """host_in, host_out: pinned bf16 tensors [nranks, count].  Asynchronous; call wait()."""
        s = self.calls % self.depth
        if self.calls >= self.depth:
            self.h2d.wait_event(self.computed[s])        # the kernels that read d_in[s] are done
            self.comp.wait_event(self.downloaded[s])     # the copy that read d_out[s] is done
        with torch.cuda.stream(self.h2d):
            self.d_in[s].copy_(host_in, non_blocking=True)
            self.uploaded[s].record(self.h2d)
        self.comp.wait_event(self.uploaded[s])
        ins = [self.d_in[s][r] for r in range(self.n)]
        outs = [self.d_out[s][r] for r in range(self.n)]
        _b.allreduce_sim_pipelined(ins, outs, self.n, self.count, self.block, self.ws, self.wb, False,
                                   self.comp.cuda_stream)
        self.computed[s].record(self.comp)
        self.d2h.wait_event(self.computed[s])
        with torch.cuda.stream(self.d2h):
            host_out.copy_(self.d_out[s], non_blocking=True)
            self.downloaded[s].record(self.d2h)
        self.calls += 1

    def wait(self):
        self.d2h.synchronize()
        self.comp.synchronize()
        self.h2d.synchronize()
