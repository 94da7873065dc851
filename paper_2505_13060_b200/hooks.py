"""Calibration of a PyTorch model through module hooks (Algorithm 1 step 2:
"wrap the model", then one high-precision forward and backward per sample).

``Calibrator`` registers every ``torch.nn.Linear`` of a model as a linear layer
of a scoring context and every ``BatchedMatmul`` (a module that only wraps
``torch.matmul``, so that the attention products Q K^T and P V are visible to
hooks) as a batched GEMM with operands X0, X1 (Sec. 2.2).  While a sample runs, a forward hook keeps the layer input X
and a backward hook receives dL/dX and dL/dY; the sample's weight gradient
dL/dW = dL/dY^T X is formed by a torch matmul (the GEMM that produces a gradient
is not part of the scoring path) and both operands of the layer are streamed to
``ampq_stream_sample``, so the R per-sample weight gradients never exist at the
same time: a sample's tensors are released as soon as the library's work on
them is ordered before any reuse of their memory -- at once when the context
runs on torch's current stream (the caching allocator hands a freed block only
to later work of the same stream), else when a CUDA event recorded on the
context's stream after the sample has completed, with at most two samples
pending.  Everything the method computes happens in the CUDA library; this
module only moves pointers.

``quantised(...)`` runs the model with chosen layers' inputs and weights replaced
by their FP8-rounded values (``ampq_fake_quant``), which is how the predicted
loss MSE is checked against a measured one (Sec. 3.2).
"""
from __future__ import annotations

import contextlib

import torch

from . import binding as ampq


class BatchedMatmul(torch.nn.Module):
    """``torch.matmul(a, b)`` as a module: a batched GEMM layer Y = X0 (x) X1 whose
    two operands and their gradients the calibrator can see."""

    def forward(self, a, b):
        return torch.matmul(a, b)


class Calibrator:
    def __init__(self, ctx: "ampq.Context", model: torch.nn.Module, R: int):
        self.ctx, self.model, self.R = ctx, model, R
        self.modules, self.layer_ids = [], []
        for name, m in model.named_modules():
            if isinstance(m, torch.nn.Linear):
                self.modules.append((name, m))
                self.layer_ids.append(ctx.register_layer(ampq.LINEAR, name, R))
            elif isinstance(m, BatchedMatmul):
                self.modules.append((name, m))
                self.layer_ids.append(ctx.register_layer(ampq.BGEMM, name, R))
        self._r = None
        self._x = {}
        self._keep = []      # tensors the library borrowed during the current sample
        self._pending = []   # (event on the context's stream, tensors) of earlier samples
        self._handles = []

    # -- lifetime of borrowed tensors -------------------------------------------
    def _same_stream(self) -> bool:
        return torch.cuda.current_stream().cuda_stream == self.ctx.stream

    def _release_sample(self):
        """Called when a sample's block ends: nothing more will be launched on its tensors."""
        if not self._keep:
            return
        if self._same_stream():
            self._keep = []   # stream order protects the memory
            return
        ev = torch.cuda.Event()
        ev.record(torch.cuda.ExternalStream(self.ctx.stream))
        self._pending.append((ev, self._keep))
        self._keep = []
        self._pending = [(e, t) for e, t in self._pending if not e.query()]
        while len(self._pending) > 2:
            self._pending.pop(0)[0].synchronize()

    # -- hooks ----------------------------------------------------------------
    def _fwd(self, idx):
        def hook(module, inputs, output):
            if self._r is not None:
                self._x[idx] = tuple(t.detach() for t in inputs) if isinstance(module, BatchedMatmul) else inputs[0].detach()
        return hook

    def _bwd(self, idx):
        def hook(module, grad_input, grad_output):
            if self._r is None:
                return
            if not self._same_stream():   # the library's stream reads what torch's stream has just produced
                torch.cuda.ExternalStream(self.ctx.stream).wait_stream(torch.cuda.current_stream())
            if isinstance(module, BatchedMatmul):   # both operands belong to the sample
                lid = self.layer_ids[idx]
                for k, (x, gx) in enumerate(zip(self._x.pop(idx), grad_input)):
                    x = x.contiguous()
                    gx = (torch.zeros_like(x) if gx is None else gx.detach().reshape(x.shape)).contiguous()
                    self.ctx.stream_sample(lid, k, self._r, ampq.torch_dtype_code(x), x.data_ptr(), gx.data_ptr(), x.numel())
                    self._keep += [x, gx]
                return
            x = self._x.pop(idx).contiguous()
            gy = grad_output[0].detach()
            gx = grad_input[0]
            w = module.weight.detach().contiguous()
            if gx is None:   # the model input needs no gradient: form dL/dX here
                gx = gy.reshape(-1, gy.shape[-1]) @ w
            gx = gx.detach().reshape(x.shape).contiguous()
            gw = (gy.reshape(-1, gy.shape[-1]).t() @ x.reshape(-1, x.shape[-1])).contiguous()
            code = ampq.torch_dtype_code(x)
            lid = self.layer_ids[idx]
            self.ctx.stream_sample(lid, 0, self._r, code, x.data_ptr(), gx.data_ptr(), x.numel())
            self.ctx.stream_sample(lid, 1, self._r, code, w.data_ptr(), gw.data_ptr(), w.numel())
            self._keep += [x, gx, w, gw]
        return hook

    def begin(self):
        self._handles = []
        for idx, (_, m) in enumerate(self.modules):
            self._handles.append(m.register_forward_hook(self._fwd(idx)))
            self._handles.append(m.register_full_backward_hook(self._bwd(idx)))
        self.ctx.stream_begin()

    @contextlib.contextmanager
    def sample(self, r: int):
        """Run one sample's forward and backward inside this block."""
        self._r = r
        try:
            yield
        finally:
            self._r = None
            self._x.clear()
            self._release_sample()

    def end(self):
        self.ctx.stream_end()
        res = [self.ctx.get_layer(lid) for lid in self.layer_ids]   # synchronises: the borrowed tensors are free
        self._keep = []
        self._pending = []
        for h in self._handles:
            h.remove()
        self._handles = []
        return res

    # -- running the model in a low-precision configuration --------------------
    @contextlib.contextmanager
    def quantised(self, fmt_of_layer, amax_x=None):
        """Inside this block layer i (index into ``modules``) runs with its input and
        weight rounded to format ``fmt_of_layer[i]`` (0 leaves it alone).
        ``amax_x[i]`` is the static amax of the layer's input (measured per call if
        absent); the weight's amax is always measured."""
        saved, handles = [], []
        for idx, (_, m) in enumerate(self.modules):
            fmt = fmt_of_layer[idx]
            if not fmt:
                continue
            if isinstance(m, BatchedMatmul):   # both inputs rounded, each with its own measured amax

                def pre2(module, inputs, fmt=fmt):
                    outs = []
                    for x in inputs:
                        x = x.contiguous()
                        out = torch.empty_like(x)
                        self.ctx.fake_quant(ampq.torch_dtype_code(x), fmt, x.data_ptr(), x.numel(), -1.0, out.data_ptr())
                        self._keep.append(x)
                        outs.append(out)
                    return tuple(outs)

                handles.append(m.register_forward_pre_hook(pre2))
                continue
            w = m.weight.data
            saved.append((m, w.clone()))
            self.ctx.fake_quant(ampq.torch_dtype_code(w), fmt, w.data_ptr(), w.numel(), -1.0, w.data_ptr())

            def pre(module, inputs, fmt=fmt, a=(-1.0 if amax_x is None else float(amax_x[idx]))):
                x = inputs[0].contiguous()
                out = torch.empty_like(x)
                self.ctx.fake_quant(ampq.torch_dtype_code(x), fmt, x.data_ptr(), x.numel(), a, out.data_ptr())
                self._keep.append(x)
                return (out,) + tuple(inputs[1:])

            handles.append(m.register_forward_pre_hook(pre))
        try:
            yield
        finally:
            torch.cuda.current_stream().synchronize()
            for h in handles:
                h.remove()
            for m, w in saved:
                m.weight.data.copy_(w)
            if not self._same_stream():
                torch.cuda.ExternalStream(self.ctx.stream).synchronize()
            self._keep = []
