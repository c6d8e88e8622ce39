"""Host-buffer front end: stream GEMM problems that live in pinned host memory through the GPU.

`Handle.gemm` takes device tensors.  A caller whose operands sit in host memory pays for the
PCIe copies; `HostGemmPipeline` overlaps them with the kernels: the host-to-device copies of problem
i+1, the GEMM of problem i and the device-to-host copy of problem i-1 run on three streams, with two
device buffer sets per distinct problem shape so that a copy never overwrites operands a kernel is
still reading.  All arithmetic still runs in libfact's kernels; this module only moves bytes and
orders streams.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from .binding import Handle


class HostGemmPipeline:
    """C_i = A_i @ B_i for a sequence of problems given as pinned host tensors.

    h       : a libfact Handle
    shapes  : the distinct (M, N, K) shapes that will be submitted (device buffers are preallocated)
    layout  : "KN" (B is [K, N]) or "NK" (B is [N, K])
    """

    def __init__(self, h: Handle, shapes: Sequence[Tuple[int, int, int]], layout: str = "KN", depth: int = 2):
        self.h = h
        self.layout = layout
        self.dev = torch.device(f"cuda:{h.device}")
        self.depth = depth
        self.s_in = torch.cuda.Stream(self.dev)
        self.s_mm = torch.cuda.Stream(self.dev)
        self.s_out = torch.cuda.Stream(self.dev)
        self.bufs = {}
        for (M, N, K) in set(shapes):
            bshape = (K, N) if layout == "KN" else (N, K)
            self.bufs[(M, N, K)] = [
                {"A": torch.empty((M, K), dtype=torch.bfloat16, device=self.dev),
                 "B": torch.empty(bshape, dtype=torch.bfloat16, device=self.dev),
                 "C": torch.empty((M, N), dtype=torch.bfloat16, device=self.dev),
                 "free": None}  # event: the D2H copy that last used this set has finished
                for _ in range(depth)]
        self.turn = {k: 0 for k in self.bufs}
        self.h2d_bytes = 0
        self.d2h_bytes = 0

    def submit(self, A_host: torch.Tensor, B_host: torch.Tensor, C_host: torch.Tensor):
        """Enqueue one problem; returns immediately.  `C_host` is valid after `finish()`."""
        M, K = A_host.shape
        N = C_host.shape[1]
        key = (M, N, K)
        sets = self.bufs[key]
        slot = sets[self.turn[key] % self.depth]
        self.turn[key] += 1
        with torch.cuda.stream(self.s_in):
            if slot["free"] is not None:
                self.s_in.wait_event(slot["free"])  # the previous result has left this buffer set
            slot["A"].copy_(A_host, non_blocking=True)
            slot["B"].copy_(B_host, non_blocking=True)
            loaded = torch.cuda.Event()
            loaded.record(self.s_in)
        with torch.cuda.stream(self.s_mm):
            self.s_mm.wait_event(loaded)
            self.h.gemm(slot["A"], slot["B"], layout=self.layout, out=slot["C"], stream=self.s_mm)
            done = torch.cuda.Event()
            done.record(self.s_mm)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(done)
            C_host.copy_(slot["C"], non_blocking=True)
            freed = torch.cuda.Event()
            freed.record(self.s_out)
        slot["free"] = freed
        self.h2d_bytes += (A_host.numel() + B_host.numel()) * 2
        self.d2h_bytes += C_host.numel() * 2

    def finish(self):
        """Block until every submitted problem's result is in host memory."""
        self.s_out.synchronize()
        self.s_mm.synchronize()
        self.s_in.synchronize()
