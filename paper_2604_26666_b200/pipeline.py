"""Host-buffer front end: stream GEMM problems that live in pinned host memory through the GPU.

`Handle.gemm` takes device tensors.  A caller whose operands sit in host memory pays for the PCIe copies;
`fact_gemm_host` (the library's host-buffer entry point) overlaps them with the kernels -- the copy-in of
problem i+1, the product of problem i and the copy-out of problem i-1 run on the handle's three streams --
as long as consecutive calls are given different device scratch buffers.  `HostGemmPipeline` only owns those
scratch buffers (`depth` per distinct problem shape) and hands them out in turn; every copy and every
product is enqueued by the library call.
"""
from __future__ import annotations

from typing import Sequence, Tuple

import torch

from .binding import Handle


class HostGemmPipeline:
    """C_i = A_i @ B_i for a sequence of problems given as pinned host tensors.

    h       : a libfact Handle
    shapes  : the distinct (M, N, K) shapes that will be submitted (device scratch is preallocated)
    layout  : "KN" (B is [K, N]) or "NK" (B is [N, K])
    """

    def __init__(self, h: Handle, shapes: Sequence[Tuple[int, int, int]], layout: str = "KN", depth: int = 2,
                 out_dtype=torch.bfloat16):
        self.h = h
        self.layout = layout
        self.dev = torch.device(f"cuda:{h.device}")
        self.depth = depth
        self.out_dtype = out_dtype
        self.scratch = {}
        for (M, N, K) in set(shapes):
            nbytes = h.gemm_host_scratch_bytes(M, N, K, out_dtype, layout)
            self.scratch[(M, N, K)] = [torch.empty(nbytes, dtype=torch.uint8, device=self.dev) for _ in range(depth)]
        self.turn = {k: 0 for k in self.scratch}
        self.h2d_bytes = 0
        self.d2h_bytes = 0

    def submit(self, A_host: torch.Tensor, B_host: torch.Tensor, C_host: torch.Tensor, stream=None):
        """Enqueue one problem; returns immediately.  `C_host` is valid after `finish()`."""
        M, K = A_host.shape
        N = C_host.shape[1]
        key = (M, N, K)
        bufs = self.scratch[key]
        scratch = bufs[self.turn[key] % self.depth]
        self.turn[key] += 1
        self.h.gemm_host(A_host, B_host, C_host, scratch, layout=self.layout, stream=stream)
        self.h2d_bytes += (A_host.numel() + B_host.numel()) * A_host.element_size()
        self.d2h_bytes += C_host.numel() * C_host.element_size()

    def finish(self, stream=None):
        """Block until every submitted problem's result is in host memory."""
        s = stream if stream is not None else torch.cuda.current_stream(self.dev)
        self.h.gemm_host_wait(s)
        s.synchronize()
