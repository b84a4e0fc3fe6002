"""Hooks that run Algorithm 1 (saliency and Hessian steps) on a PyTorch model: plumbing around the library calls.

The method needs, per linear layer, the end-loss gradients of the layer's outputs (only their group-wise
mean squares s_k are kept: O(n g) per layer, Section 3.2) and the layer's inputs.  As in the paper this takes
two passes over the same calibration batches in the same order:

    cap = GuidedHessianCapture({"mlp.up": model.mlp.up, ...}, g=4)
    with cap.saliency_pass():            # pass 1: backward hooks, gq_saliency on every output gradient
        for batch in batches: loss_fn(model(batch)).backward()
    with cap.hessian_pass():             # pass 2: forward hooks, gq_hessian_accumulate with the stored s
        for batch in batches: model(batch)
    H = cap.finalize()                   # {name: [g, d_in, d_in] fp32}, complete symmetric matrices

No arithmetic of the method happens here.  The backward hook hands the gradient over as autograd produced it
(``[batch, seq, d_out]`` in bf16, fp16 or fp32, any batch / sequence strides) to gq_saliency_strided, so no cast
and no contiguous copy of it is ever made; other layouts are flattened and cast to bf16 for gq_saliency.  The
forward hook flattens the layer input to bf16 tokens (the Hessian kernel's input type) and calls
gq_hessian_accumulate; finalize() calls gq_hessian_finalize.  All on the tensors' own device and stream."""
from __future__ import annotations

import contextlib
from typing import Dict

import torch

from . import api


class GuidedHessianCapture:
    def __init__(self, layers: Dict[str, torch.nn.Module], g: int, grad_scale: float = 1e3):
        self.layers = dict(layers)
        self.g = int(g)
        self.grad_scale = float(grad_scale)
        self.s: Dict[str, list] = {k: [] for k in self.layers}       # per layer: one [g, n_batch] tensor per batch
        self.H: Dict[str, torch.Tensor] = {}
        self._next: Dict[str, int] = {}
        self._ws: Dict[str, torch.Tensor] = {}

    @staticmethod
    def _tokens(t: torch.Tensor) -> torch.Tensor:
        return t.reshape(-1, t.shape[-1]).to(torch.bfloat16).contiguous()

    @contextlib.contextmanager
    def saliency_pass(self):
        """Registers backward hooks; every backward call appends one saliency block per layer."""
        handles = []
        for name, mod in self.layers.items():
            def hook(_mod, _grad_in, grad_out, name=name):
                grad = grad_out[0].detach()
                if (grad.dim() == 3 and grad.dtype in (torch.bfloat16, torch.float16, torch.float32)
                        and (grad.shape[2] == 1 or grad.stride(2) == 1)):
                    self.s[name].append(api.gq_saliency_strided(grad, self.g, self.grad_scale))
                else:
                    self.s[name].append(api.gq_saliency(self._tokens(grad), self.g, self.grad_scale))
            handles.append(mod.register_full_backward_hook(hook))
        try:
            yield self
        finally:
            for h in handles:
                h.remove()

    @contextlib.contextmanager
    def hessian_pass(self):
        """Registers forward hooks; the i-th forward call of a layer is paired with its i-th saliency block."""
        handles = []
        self._next = {k: 0 for k in self.layers}
        for name, mod in self.layers.items():
            def hook(_mod, inputs, name=name):
                x = self._tokens(inputs[0].detach())
                i = self._next[name]
                if i >= len(self.s[name]):
                    raise RuntimeError("layer %s: more forward calls than saliency blocks" % name)
                s = self.s[name][i]
                if s.shape[1] != x.shape[0]:
                    raise RuntimeError("layer %s, call %d: %d tokens but saliency of %d" % (name, i, x.shape[0], s.shape[1]))
                self._next[name] = i + 1
                d_in = x.shape[1]
                if name not in self.H:
                    self.H[name] = torch.zeros((self.g, d_in, d_in), dtype=torch.float32, device=x.device)
                need = api.gq_hessian_workspace_bytes(x.shape[0], d_in, self.g)
                if name not in self._ws or self._ws[name].numel() < need:
                    self._ws[name] = api.alloc_workspace(need, x.device)
                api.gq_hessian_accumulate(x, s, self.H[name], self._ws[name])
            handles.append(mod.register_forward_pre_hook(hook))
        try:
            yield self
        finally:
            for h in handles:
                h.remove()

    def finalize(self) -> Dict[str, torch.Tensor]:
        for name, H in self.H.items():
            if self._next.get(name, 0) != len(self.s[name]):
                raise RuntimeError("layer %s: %d saliency blocks but %d forward calls"
                                   % (name, len(self.s[name]), self._next.get(name, 0)))
            api.gq_hessian_finalize(H)
        api.gq_check()
        return self.H
