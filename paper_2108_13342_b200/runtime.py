"""Builds a dnnf graph from a plain graph description and runs it on torch-owned
device memory.  torch is used for allocation, host<->device copies and streams
only; all computation happens in libdnnf.so."""
from __future__ import annotations

import numpy as np

from . import binding as B

_DT = {"f32": B.F32, "bf16": B.BF16}


def build_graph(desc):
    """desc: workloads.GraphDesc.  Returns (Graph, name -> tensor id)."""
    g = B.Graph()
    ids = {}
    for name, t in desc.tensors.items():
        ids[name] = g.add_tensor(name, _DT[t.dtype], t.shape, B.WEIGHT if t.kind == "weight" else B.INPUT)
    for op in desc.ops:
        outs = g.add_op(op.op, [ids[n] for n in op.inputs], **op.attrs)
        assert len(outs) == len(op.outputs), (op.op, outs, op.outputs)
        for n, i in zip(op.outputs, outs):
            ids[n] = i
    for n in desc.outputs:
        g.mark_output(ids[n])
    return g, ids


class Session:
    """A planned graph bound to torch tensors on one device."""

    def __init__(self, workload, plan_flags=B.PLAN_FUSED, rewrite_flags=B.REWRITE_DEFAULT, device="cuda:0",
                 upload=True):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.desc = workload.graph
        self.g, self.ids = build_graph(self.desc)
        self.rewrite_stats = self.g.rewrite(rewrite_flags)
        self.plan_stats = self.g.plan(plan_flags)
        self.buffers = {}
        self.host_inputs = workload.inputs
        if upload:
            for name, t in self.desc.tensors.items():
                self.set_input(name, workload.inputs[name])
        for name in self.desc.outputs:
            dt, dims = self.g.tensor_info(self.ids[name])
            buf = torch.empty(dims, dtype=torch.float32 if dt == B.F32 else torch.bfloat16, device=self.device)
            self.buffers[name] = buf
            self.g.bind(self.ids[name], buf.data_ptr())
        ws = self.g.workspace_size()
        self.workspace = torch.zeros(max(ws, 256), dtype=torch.uint8, device=self.device)
        self.g.bind_workspace(self.workspace.data_ptr(), self.workspace.numel())

    def set_input(self, name, array):
        torch = self.torch
        t = self.desc.tensors[name]
        host = torch.from_numpy(np.ascontiguousarray(array, dtype=np.float32))
        dev = host.to(self.device)
        if t.dtype == "bf16":
            dev = dev.to(torch.bfloat16)        # values are bf16-representable: exact
        dev = dev.contiguous()
        self.buffers[name] = dev
        self.g.bind(self.ids[name], dev.data_ptr())

    def run(self, stream=None):
        s = self.torch.cuda.current_stream(self.device) if stream is None else stream
        self.g.run(s.cuda_stream)

    def run_block(self, b, stream=None):
        s = self.torch.cuda.current_stream(self.device) if stream is None else stream
        self.g.run_block(b, s.cuda_stream)

    def output(self, name=None):
        name = name or self.desc.outputs[0]
        self.torch.cuda.synchronize(self.device)
        return self.buffers[name].float().cpu().numpy().astype(np.float64)
