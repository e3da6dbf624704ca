"""Host-to-host calls: the tensor starts and ends in (pinned) host memory.

A shard that receives its activations over the network holds them in host buffers.  These
helpers stream such a buffer through the GPU in chunks on three CUDA streams, so that the
upload of chunk i+1, the kernel on chunk i and the download of chunk i-1 overlap (PCIe is
full duplex and the copy engines run beside the SMs).  Every step of the method still runs
in the library's kernels; this module only moves bytes and orders streams.
"""
from __future__ import annotations

import torch

from .binding import Codebook, bq_dequantize, bq_quantize, bq_roundtrip


class HostBoundary:
    """Chunked, triple-buffered quantize / dequantize / roundtrip between pinned host tensors.

    ``chunk`` is the number of elements per piece (a multiple of every block size used with
    this object); ``slots`` pieces are in flight at once.  Device staging buffers are
    allocated once, here.
    """

    def __init__(self, cb: Codebook, dtype: torch.dtype, chunk: int = 1 << 25, slots: int = 3, max_blocks_per_chunk: int | None = None):
        self.cb, self.dtype, self.chunk, self.slots = cb, dtype, int(chunk), int(slots)
        dev = cb.device
        self.dev = dev
        nb = max_blocks_per_chunk or (self.chunk // 16)
        self.x = [torch.empty(self.chunk, dtype=dtype, device=dev) for _ in range(slots)]
        self.y = [torch.empty(self.chunk, dtype=dtype, device=dev) for _ in range(slots)]
        self.c = [torch.empty(self.chunk, dtype=torch.uint8, device=dev) for _ in range(slots)]
        self.a = [torch.empty(nb, dtype=torch.float32, device=dev) for _ in range(slots)]
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
        self.free = [torch.cuda.Event() for _ in range(slots)]

    def _pieces(self, n: int, block: int):
        if self.chunk % block:
            raise ValueError("chunk must be a multiple of the block size")
        for i, lo in enumerate(range(0, n, self.chunk)):
            yield i % self.slots, lo, min(n, lo + self.chunk)

    def _run(self, n, block, upload, kernel, download):
        """Common ordering: upload on s_in, kernel on s_run, download on s_out, per piece."""
        start = torch.cuda.Event()
        start.record(torch.cuda.current_stream(self.dev))
        for s in (self.s_in, self.s_run, self.s_out):
            s.wait_event(start)
        used = [False] * self.slots
        for slot, lo, hi in self._pieces(n, block):
            if used[slot]:
                self.s_in.wait_event(self.free[slot])           # the slot's previous download has finished
            used[slot] = True
            with torch.cuda.stream(self.s_in):
                upload(slot, lo, hi)
                ev_in = torch.cuda.Event()
                ev_in.record(self.s_in)
            self.s_run.wait_event(ev_in)
            with torch.cuda.stream(self.s_run):
                kernel(slot, lo, hi)
                ev_k = torch.cuda.Event()
                ev_k.record(self.s_run)
            self.s_out.wait_event(ev_k)
            with torch.cuda.stream(self.s_out):
                download(slot, lo, hi)
                self.free[slot].record(self.s_out)
        done = torch.cuda.Event()
        done.record(self.s_out)
        torch.cuda.current_stream(self.dev).wait_event(done)

    def roundtrip(self, x_host: torch.Tensor, block: int, y_host: torch.Tensor) -> None:
        n = x_host.numel()
        xf, yf = x_host.view(-1), y_host.view(-1)
        self._run(n, block,
                  lambda s, lo, hi: self.x[s][: hi - lo].copy_(xf[lo:hi], non_blocking=True),
                  lambda s, lo, hi: bq_roundtrip(self.x[s][: hi - lo], block, self.cb, y_out=self.y[s][: hi - lo]),
                  lambda s, lo, hi: yf[lo:hi].copy_(self.y[s][: hi - lo], non_blocking=True))

    def quantize(self, x_host: torch.Tensor, block: int, codes_host: torch.Tensor, absmax_host: torch.Tensor) -> None:
        n = x_host.numel()
        xf = x_host.view(-1)

        def down(s, lo, hi):
            b0, b1 = lo // block, (hi + block - 1) // block
            codes_host[lo:hi].copy_(self.c[s][: hi - lo], non_blocking=True)
            absmax_host[b0:b1].copy_(self.a[s][: b1 - b0], non_blocking=True)

        self._run(n, block,
                  lambda s, lo, hi: self.x[s][: hi - lo].copy_(xf[lo:hi], non_blocking=True),
                  lambda s, lo, hi: bq_quantize(self.x[s][: hi - lo], block, self.cb, self.c[s][: hi - lo],
                                                self.a[s][: (hi - lo + block - 1) // block]),
                  down)

    def dequantize(self, codes_host: torch.Tensor, absmax_host: torch.Tensor, block: int, y_host: torch.Tensor) -> None:
        n = codes_host.numel()
        yf = y_host.view(-1)

        def up(s, lo, hi):
            b0, b1 = lo // block, (hi + block - 1) // block
            self.c[s][: hi - lo].copy_(codes_host[lo:hi], non_blocking=True)
            self.a[s][: b1 - b0].copy_(absmax_host[b0:b1], non_blocking=True)

        self._run(n, block, up,
                  lambda s, lo, hi: bq_dequantize(self.c[s][: hi - lo], self.a[s][: (hi - lo + block - 1) // block], block, self.cb,
                                                  self.dtype, self.y[s][: hi - lo]),
                  lambda s, lo, hi: yf[lo:hi].copy_(self.y[s][: hi - lo], non_blocking=True))
