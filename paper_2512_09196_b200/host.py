"""Host-buffer entry: runs one op on tensors that live in pinned host memory.

Plumbing only (copies, streams, events): the rows are cut into blocks, and block k's host-to-device copy, the
kernel call through the C ABI on block k-1 and the device-to-host copy of block k-2 run on three streams, so
the two PCIe directions overlap each other and the kernels.  Rows are independent, so a row block is a
complete problem for the library.  Consecutive calls may overlap as well (``join=False``): block i of the next call
is copied in as soon as the kernel of the previous call has consumed block i, and computed as soon as block i of the
previous result has left the device.
"""
from __future__ import annotations

import torch

from . import tf_layernorm_fwd, tf_rmsnorm_fwd, tf_softmax_fwd


class HostPipeline:
    """Reusable device staging buffers and streams for a fixed [rows, cols] problem."""

    def __init__(self, op: str, rows: int, cols: int, dtype: torch.dtype, device, blocks: int = 8):
        self.op, self.rows, self.cols, self.device = op, rows, cols, torch.device(device)
        self.blocks = max(1, min(blocks, rows))
        self.dx = torch.empty((rows, cols), dtype=dtype, device=self.device)
        self.dy = torch.empty_like(self.dx)
        self.dmean = torch.empty(rows, dtype=torch.float32, device=self.device)
        self.drstd = torch.empty(rows, dtype=torch.float32, device=self.device)
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream(self.device) for _ in range(3))
        self.bounds = [(rows * b // self.blocks, rows * (b + 1) // self.blocks) for b in range(self.blocks)]
        self.ev_in = [torch.cuda.Event() for _ in self.bounds]
        self.ev_run = [torch.cuda.Event() for _ in self.bounds]
        self.ev_out = [torch.cuda.Event() for _ in self.bounds]

    def run(self, hx, hy, params: dict, dparams: dict, eps: float = 0.0, hmean=None, hrstd=None, join: bool = True):
        """hx, hy (and hmean/hrstd, params' values) are pinned host tensors; dparams are preallocated device
        tensors of the parameters' shapes.  Returns after enqueueing; the caller synchronises.  With ``join=False``
        the current stream is not made to wait for this call, so the next call can overlap it; call ``finish()``
        before relying on the current stream (or synchronise the device).  The waits below on events of the previous
        call order the reuse of the staging buffers; an event that was never recorded does not block."""
        cur = torch.cuda.current_stream(self.device)
        for s in (self.s_in, self.s_run, self.s_out):
            s.wait_stream(cur)
        with torch.cuda.stream(self.s_in):
            self.s_in.wait_event(self.ev_run[-1])             # the previous call's last kernel has read the parameters
            for k, v in params.items():
                dparams[k].copy_(v, non_blocking=True)
            for i, (r0, r1) in enumerate(self.bounds):
                self.s_in.wait_event(self.ev_run[i])          # the previous call's kernel has consumed this block of dx
                self.dx[r0:r1].copy_(hx[r0:r1], non_blocking=True)
                self.ev_in[i].record(self.s_in)
        for i, (r0, r1) in enumerate(self.bounds):
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(self.ev_in[i])
                self.s_run.wait_event(self.ev_out[i])         # the previous call's block of dy has left the device
                x, y = self.dx[r0:r1], self.dy[r0:r1]
                if self.op == "softmax":
                    tf_softmax_fwd(x, y)
                elif self.op == "layernorm":
                    tf_layernorm_fwd(x, dparams["gamma"], dparams["beta"], eps, y, self.dmean[r0:r1], self.drstd[r0:r1])
                else:
                    tf_rmsnorm_fwd(x, dparams["w"], eps, y)
                self.ev_run[i].record(self.s_run)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(self.ev_run[i])
                hy[r0:r1].copy_(self.dy[r0:r1], non_blocking=True)
                if self.op == "layernorm" and hmean is not None:
                    hmean[r0:r1].copy_(self.dmean[r0:r1], non_blocking=True)
                    hrstd[r0:r1].copy_(self.drstd[r0:r1], non_blocking=True)
                self.ev_out[i].record(self.s_out)
        if join:
            self.finish()

    def finish(self):
        """Makes the current stream wait for everything enqueued by ``run`` so far."""
        cur = torch.cuda.current_stream(self.device)
        for s in (self.s_in, self.s_run, self.s_out):
            cur.wait_stream(s)
