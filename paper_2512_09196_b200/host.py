"""Host-buffer entry: runs one op on tensors that live in pinned host memory.

Plumbing only (copies, streams, events): the rows are cut into blocks, and block k's host-to-device copy, the
kernel call through the C ABI on block k-1 and the device-to-host copy of block k-2 run on three streams, so
the two PCIe directions overlap each other and the kernels.  Rows are independent, so a row block is a
complete problem for the library.
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

    def run(self, hx, hy, params: dict, dparams: dict, eps: float = 0.0, hmean=None, hrstd=None):
        """hx, hy (and hmean/hrstd, params' values) are pinned host tensors; dparams are preallocated device
        tensors of the parameters' shapes.  Returns after enqueueing; the caller synchronises."""
        cur = torch.cuda.current_stream(self.device)
        for s in (self.s_in, self.s_run, self.s_out):
            s.wait_stream(cur)
        with torch.cuda.stream(self.s_in):
            for k, v in params.items():
                dparams[k].copy_(v, non_blocking=True)
            for i, (r0, r1) in enumerate(self.bounds):
                self.dx[r0:r1].copy_(hx[r0:r1], non_blocking=True)
                self.ev_in[i].record(self.s_in)
        for i, (r0, r1) in enumerate(self.bounds):
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(self.ev_in[i])
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
        cur.wait_stream(self.s_out)
