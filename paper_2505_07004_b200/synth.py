"""Seeded synthetic layer inputs (activations, output gradients, weights).

This module only *draws inputs*: it contains none of the method's arithmetic
(no saliency, no Gram matrix, no objective).  Both the CUDA path and the CPU
oracle are fed the arrays produced here, so neither side ever generates an
input for the other.

The five layer shapes are stand-ins for the calibration tensors the paper uses
(Llama-2 linear-layer inputs and end-loss output gradients on 1024 x 4096
RedPajama tokens, Section 5 "Experiments"); dataset and checkpoints are not
available, so values are drawn from seeded distributions that keep the
activation-outlier structure:

* ``lognormal`` activations: ``xi[i,a] * f[a]`` with ``xi ~ N(0,1)``,
  ``f = exp(N(0,1))`` per input feature and a fraction of the features
  multiplied by an outlier factor;
* ``silu`` activations: ``u * sigmoid(v)`` with independent standard normals
  (post-SiLU-like, skewed), again with outlier features;
* gradients: ``1e-3 * zeta[i,j] * exp(t[i])`` (per-token log-normal factor);
* weights ``W ~ N(0, std 0.02)`` stored ``[d_out, d_in]`` (one output channel
  per row) and ``W_hat`` = ``W`` rounded to a 16-level uniform grid spanning
  each channel's [min, max].

Values are computed in fp32 and rounded to bf16 once.  Every tensor/chunk has
its own seed ``seed*1000003 + tensor_id*8191 + chunk_index`` so chunks can be
regenerated independently and in any order.
"""
from __future__ import annotations

import dataclasses
from typing import Tuple

import torch

_T_FEAT, _T_OUTLIER, _T_X, _T_GRAD, _T_W = 1, 2, 3, 4, 5


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    n: int            # calibration tokens
    chunk: int        # tokens per streamed chunk
    d_in: int
    d_out: int
    groups: Tuple[int, ...]   # values of g this config is run with
    x_kind: str       # "lognormal" | "silu"
    outlier_frac: float
    outlier_mult: float

    @property
    def g(self) -> int:
        return self.groups[0]

    @property
    def n_chunks(self) -> int:
        return (self.n + self.chunk - 1) // self.chunk


CONFIGS = {
    "c0_tiny": LayerConfig("c0_tiny", 2048, 2048, 256, 512, (4,), "lognormal", 0.01, 20.0),
    "c1_7b_attn": LayerConfig("c1_7b_attn", 131072, 8192, 4096, 4096, (4,), "lognormal", 0.01, 20.0),
    "c2_7b_down": LayerConfig("c2_7b_down", 131072, 8192, 11008, 4096, (4,), "silu", 0.005, 50.0),
    "c3_70b_mlp": LayerConfig("c3_70b_mlp", 65536, 4096, 28672, 8192, (2,), "silu", 0.005, 50.0),
    "c4_sweep": LayerConfig("c4_sweep", 1048576, 16384, 4096, 11008, (1, 2, 4, 8, 16), "lognormal", 0.01, 20.0),
}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


class LayerSynth:
    """Draws the tensors of one synthetic layer on ``device`` (cpu or cuda)."""

    def __init__(self, cfg: LayerConfig, device="cpu", seed: int = 0):
        self.cfg = cfg
        self.device = torch.device(device)
        self.seed = int(seed)
        d_in = cfg.d_in
        if cfg.x_kind == "lognormal":
            z = torch.randn(d_in, generator=self._g(_T_FEAT, 0), device=self.device, dtype=torch.float32)
            scale = torch.exp(z)
        elif cfg.x_kind == "silu":
            scale = torch.ones(d_in, device=self.device, dtype=torch.float32)
        else:
            raise ValueError(cfg.x_kind)
        n_out = max(1, int(round(cfg.outlier_frac * d_in)))
        perm = torch.randperm(d_in, generator=self._g(_T_OUTLIER, 0), device=self.device)
        scale[perm[:n_out]] *= cfg.outlier_mult
        self.feature_scale = scale
        self.outlier_features = perm[:n_out]

    def _g(self, tensor_id: int, chunk_idx: int) -> torch.Generator:
        return _gen(self.device, self.seed * 1000003 + tensor_id * 8191 + chunk_idx)

    def chunk_tokens(self, c_idx: int) -> int:
        cfg = self.cfg
        return min(cfg.chunk, cfg.n - c_idx * cfg.chunk)

    def x_chunk(self, c_idx: int, n_tokens: int | None = None) -> torch.Tensor:
        """bf16 ``[n_tokens, d_in]`` activations of chunk ``c_idx`` (row = token)."""
        cfg = self.cfg
        n_tok = self.chunk_tokens(c_idx) if n_tokens is None else int(n_tokens)
        gen = self._g(_T_X, c_idx)
        u = torch.randn(n_tok, cfg.d_in, generator=gen, device=self.device, dtype=torch.float32)
        if cfg.x_kind == "silu":
            v = torch.randn(n_tok, cfg.d_in, generator=gen, device=self.device, dtype=torch.float32)
            u = u * torch.sigmoid(v)
        u *= self.feature_scale
        return u.to(torch.bfloat16)

    def grad_chunk(self, c_idx: int, n_tokens: int | None = None) -> torch.Tensor:
        """bf16 ``[n_tokens, d_out]`` end-loss gradients w.r.t. the layer output."""
        cfg = self.cfg
        n_tok = self.chunk_tokens(c_idx) if n_tokens is None else int(n_tokens)
        gen = self._g(_T_GRAD, c_idx)
        t = torch.randn(n_tok, 1, generator=gen, device=self.device, dtype=torch.float32)
        z = torch.randn(n_tok, cfg.d_out, generator=gen, device=self.device, dtype=torch.float32)
        z *= 1e-3 * torch.exp(t)
        return z.to(torch.bfloat16)

    def weights(self) -> Tuple[torch.Tensor, torch.Tensor]:
        """fp32 ``W`` and ``W_hat``, both ``[d_out, d_in]`` (row j = output channel j)."""
        cfg = self.cfg
        w = 0.02 * torch.randn(cfg.d_out, cfg.d_in, generator=self._g(_T_W, 0),
                               device=self.device, dtype=torch.float32)
        return w, uniform_grid_round(w, 16)


def uniform_grid_round(w: torch.Tensor, levels: int) -> torch.Tensor:
    """Round every row of ``w`` to ``levels`` equally spaced values on [row min, row max]."""
    lo = w.amin(dim=1, keepdim=True)
    hi = w.amax(dim=1, keepdim=True)
    step = (hi - lo) / float(levels - 1)
    safe = torch.where(step > 0, step, torch.ones_like(step))
    q = torch.round((w - lo) / safe)          # half-to-even
    w_hat = lo + q * safe
    return torch.where(step > 0, w_hat, w).contiguous()


def bf16_bits(t: torch.Tensor):
    """numpy uint16 view (host copy) of a bf16 tensor's bit patterns."""
    import numpy as np
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
