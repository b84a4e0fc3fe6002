"""gq_objective_noalloc: the objective for callers that may not allocate device memory.

Some callers of libgq cannot call cudaMalloc (a region being captured into a CUDA graph, an allocator-free
callback, a process whose memory was all given to another pool), so this entry point keeps its scratch in a
fixed 4 MiB + 256 KiB array inside the library.  The test drives it through the C-ABI and compares it with
gq_objective (caller workspace) AND with the CPU fp64 oracle's objective on two consecutive calls with different
inputs: the second call runs over whatever the first one left in the shared scratch and must not be affected by
it.  (The oracle comparison matters: the kernel behind this entry point is not the one behind gq_objective.)
This file is named so that pytest collects it after every other test file.
"""
import numpy as np
import pytest
import torch

from oracle import gq_oracle as orc
from paper_2505_07004_b200 import api as libgq
from paper_2505_07004_b200 import synth

pytestmark = pytest.mark.gpu

L_RTOL = 1e-3        # the objective tolerance used by the parity tests


def _layer(dev, d_in, d_out, g, seed):
    gen = torch.Generator(device=dev).manual_seed(seed)
    X = (torch.randn(300, d_in, generator=gen, device=dev) * torch.exp(torch.randn(d_in, generator=gen, device=dev)))
    X = X.to(torch.bfloat16)
    s = torch.rand(g, 300, generator=gen, device=dev)
    H = torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev)
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(300, d_in, g), dev)
    libgq.gq_hessian_accumulate(X, s, H, ws)
    libgq.gq_hessian_finalize(H)
    W = 0.02 * torch.randn(d_out, d_in, generator=gen, device=dev)
    return H, W, synth.uniform_grid_round(W, 16)


def test_noalloc_objective_matches_workspace_objective_twice():
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    cases = [(512, 256, 2, 1), (384, 640, 5, 2)]      # second call: other shape, other data, same scratch
    for d_in, d_out, g, seed in cases:
        H, W, What = _layer(dev, d_in, d_out, g, seed)
        ws = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(d_in, d_out, g), dev)
        ref = libgq.gq_objective(W, What, H, ws)
        loss = torch.full((g + 1,), float("nan"), dtype=torch.float64, device=dev)
        libgq.gq_objective_noalloc(W, What, H, loss)
        libgq.gq_check()
        ref_h, got_h = ref.cpu().numpy(), loss.cpu().numpy()
        assert np.all(np.isfinite(got_h)) and np.all(ref_h > 0)
        assert np.all(np.abs(got_h - ref_h) <= L_RTOL * np.abs(ref_h)), (got_h, ref_h)
        oracle = orc.objective(W.cpu().numpy(), What.cpu().numpy(), H.cpu().numpy().astype(np.float64))
        assert np.all(np.abs(got_h - oracle) <= L_RTOL * np.abs(oracle)), (got_h, oracle)
    # the same inputs again straight after: identical values (nothing stale is read)
    loss2 = torch.empty_like(loss)
    libgq.gq_objective_noalloc(W, What, H, loss2)
    libgq.gq_check()
    assert torch.equal(loss, loss2)


def test_noalloc_objective_rejects_layers_beyond_its_scratch():
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    d_in, d_out, g = 2048, 1024, 2                     # 2^21 weights > 2^20
    W = torch.zeros((d_out, d_in), device=dev)
    H = torch.zeros((g, d_in, d_in), device=dev)
    loss = torch.zeros(g + 1, dtype=torch.float64, device=dev)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_objective_noalloc(W, W, H, loss)
    assert "GQ_ERR_UNSUPPORTED_SHAPE" in str(e.value)
    assert torch.count_nonzero(loss).item() == 0
