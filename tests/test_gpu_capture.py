"""The two-pass capture (backward hooks -> saliency, forward hooks -> guided Hessians) on a small random
PyTorch model against the oracle, which gets the same bf16 bit patterns of the gradients and inputs that the
hooks see (recorded by independent hooks of the test)."""
import numpy as np
import pytest
import torch

from oracle import gq_oracle as orc
from paper_2505_07004_b200 import synth
from paper_2505_07004_b200.capture import GuidedHessianCapture

pytestmark = pytest.mark.gpu


def test_capture_matches_oracle():
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    torch.manual_seed(0)
    model = torch.nn.Sequential(torch.nn.Linear(64, 128), torch.nn.GELU(), torch.nn.Linear(128, 64)).to(dev)
    layers = {"fc1": model[0], "fc2": model[2]}
    g, scale = 4, 1e3
    batches = [torch.randn(3, 50, 64, device=dev), torch.randn(2, 37, 64, device=dev)]
    target = [torch.randint(0, 64, (3, 50), device=dev), torch.randint(0, 64, (2, 37), device=dev)]

    seen_x = {k: [] for k in layers}
    seen_g = {k: [] for k in layers}
    spies = []
    for name, mod in layers.items():
        spies.append(mod.register_forward_pre_hook(
            lambda m, inp, name=name: seen_x[name].append(inp[0].detach().reshape(-1, inp[0].shape[-1]).to(torch.bfloat16))))
        spies.append(mod.register_full_backward_hook(
            lambda m, gi, go, name=name: seen_g[name].append(go[0].detach().reshape(-1, go[0].shape[-1]).to(torch.bfloat16))))

    cap = GuidedHessianCapture(layers, g, grad_scale=scale)
    with cap.saliency_pass():
        for x, t in zip(batches, target):
            out = model(x)
            torch.nn.functional.cross_entropy(out.reshape(-1, 64), t.reshape(-1), reduction="sum").backward()
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
        gb = np.concatenate([synth.bf16_bits(t.cpu()) for t in seen_g[name]])
        xb = np.concatenate([synth.bf16_bits(t.cpu()) for t in seen_x[name]])
        s_o = orc.saliency(gb, g, scale)
        s_g = torch.cat(cap.s[name], dim=1).cpu().numpy().astype(np.float64)
        assert np.all(np.abs(s_g - s_o) <= 1e-4 * np.abs(s_o) + 1e-30)
        H_o = orc.hessian(xb, s_o)
        H_g = H[name].cpu().numpy().astype(np.float64)
        for k in range(g):
            assert np.linalg.norm(H_g[k] - H_o[k]) <= 5e-3 * np.linalg.norm(H_o[k])
            assert np.abs(H_g[k] - H_o[k]).max() <= 1e-2 * np.abs(H_o[k]).max()
        assert np.array_equal(H_g, H_g.transpose(0, 2, 1))
