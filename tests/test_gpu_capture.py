"""The two-pass capture (backward hooks -> saliency, forward hooks -> guided Hessians) on a small random
PyTorch model against the oracle, which gets the fp32 gradients and the bf16 bit patterns of the inputs that
the hooks see (recorded by independent hooks of the test).  The gradients reach the library in autograd's own
dtype and layout (gq_saliency_strided), so the oracle reads the same fp32 values."""
import numpy as np
import pytest
import torch

from oracle import gq_oracle as orc
from paper_2505_07004_b200 import synth
from paper_2505_07004_b200.capture import GuidedHessianCapture

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["fp32", "bf16"])
def test_capture_matches_oracle(dtype):
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    torch.manual_seed(0)
    model = torch.nn.Sequential(torch.nn.Linear(64, 128), torch.nn.GELU(), torch.nn.Linear(128, 64)).to(dev).to(dtype)
    layers = {"fc1": model[0], "fc2": model[2]}
    g, scale = 4, 1e3
    batches = [torch.randn(3, 50, 64, device=dev).to(dtype), torch.randn(2, 37, 64, device=dev).to(dtype)]
    target = [torch.randint(0, 64, (3, 50), device=dev), torch.randint(0, 64, (2, 37), device=dev)]

    seen_x = {k: [] for k in layers}
    seen_g = {k: [] for k in layers}
    spies = []
    for name, mod in layers.items():
        spies.append(mod.register_forward_pre_hook(
            lambda m, inp, name=name: seen_x[name].append(inp[0].detach().reshape(-1, inp[0].shape[-1]).to(torch.bfloat16))))
        spies.append(mod.register_full_backward_hook(
            lambda m, gi, go, name=name: seen_g[name].append(go[0].detach().clone())))

    cap = GuidedHessianCapture(layers, g, grad_scale=scale)
    with cap.saliency_pass():
        for x, t in zip(batches, target):
            out = model(x)
            torch.nn.functional.cross_entropy(out.reshape(-1, 64).float(), t.reshape(-1), reduction="sum").backward()
    for k in seen_x:
        seen_x[k].clear()
    with cap.hessian_pass():
        with torch.no_grad():
            for x in batches:
                model(x)
    H = cap.finalize()
    for h in spies:
        h.remove()

    for name in layers:
        xb = np.concatenate([synth.bf16_bits(t.cpu()) for t in seen_x[name]])
        assert all(t.dim() == 3 and t.dtype == dtype for t in seen_g[name])
        if dtype == torch.float32:
            s_o = np.concatenate([orc.saliency_strided(t.cpu().numpy(), "fp32", g, scale) for t in seen_g[name]], axis=1)
        else:
            s_o = np.concatenate([orc.saliency_strided(synth.bf16_bits(t.cpu()).reshape(tuple(t.shape)), "bf16", g, scale)
                                  for t in seen_g[name]], axis=1)
        s_g = torch.cat(cap.s[name], dim=1).cpu().numpy().astype(np.float64)
        assert np.all(np.abs(s_g - s_o) <= 1e-4 * np.abs(s_o) + 1e-30)
        H_o = orc.hessian(xb, s_o)
        H_g = H[name].cpu().numpy().astype(np.float64)
        for k in range(g):
            assert np.linalg.norm(H_g[k] - H_o[k]) <= 5e-3 * np.linalg.norm(H_o[k])
            assert np.abs(H_g[k] - H_o[k]).max() <= 1e-2 * np.abs(H_o[k]).max()
        assert np.array_equal(H_g, H_g.transpose(0, 2, 1))
