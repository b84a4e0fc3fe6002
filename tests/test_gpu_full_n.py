"""Full-size parity: every token of the large configurations, launched exactly as bench.py launches them.

The oracle's d_in x d_in matrices need O(n d_in^2 g) fp64 operations and cannot be formed for these sizes.  Two
consequences of the definition H_k = X^T Diag(s_k) X can: the diagonal, diag(H_k)[a] = sum_i s_k[i] X[i][a]^2,
and the action on probe vectors, H_k v = X^T (s_k * (X v)); both cost O(n d_in g) and are accumulated by the
oracle chunk by chunk over ALL tokens, from the oracle's own saliency on every chunk.  The library's saliency is
compared with the oracle's on every chunk, its finalized H with the two forms.

Tolerances.  The only rounding in the Hessian kernel that is not of fp32 size is the one bf16 rounding (8
significant bits) of each product s_k[i] X[i][a]: relative error e_ia, |e_ia| <= 2^-8, independent from product to
product, so every error below is a sum of independent terms and is compared with 8 of its standard deviations
(e uniform within half a unit: rms 2^-8 / sqrt(3)), plus 2e-5 of the diagonal entry for fp32 accumulation:
  diagonal  error of H[a][a] = sum_i e_ia s_i X[i][a]^2: variance (2^-8)^2 / 3 * sum_i s_i^2 X[i][a]^4.
  probes    error of (H v)[a] = sum of e * s_i X[i][a] X[i][b] v[b]; with probe entries of random sign its variance
            is at most (2^-8)^2 / 3 * sum_i s_i^2 X[i][a]^2 q_i, q_i = sum_b v[b]^2 X[i][b]^2.
Both variance sums are diagonal forms again (other weights, squared activations), which the oracle evaluates.  For
these inputs (independent features) the probe tolerance is about one per cent of what the entries off the diagonal
contribute to (H v)[a], so a tile or a piece of a tile that is dropped, doubled or added to the wrong group shows.
"""
import numpy as np
import pytest
import torch

from oracle import gq_oracle as orc
from paper_2505_07004_b200 import api as libgq
from paper_2505_07004_b200 import synth

pytestmark = pytest.mark.gpu

S_RTOL = 1e-4
EPS_RMS = 2.0 ** -8 / np.sqrt(3.0)
SIGMAS = 8.0
ACC_SLACK = 2e-5
N_PROBES = 4


@pytest.mark.parametrize("name,groups", [
    ("c1_7b_attn", (4,)),
    ("c2_7b_down", (4,)),
    ("c3_70b_mlp", (2,)),                 # 16 chunks of 4096 tokens into a resident 6.6 GB H
    ("c4_sweep", (1, 2, 4, 8, 16)),       # 64 chunks of 16384 tokens, every group count of the sweep
])
def test_full_n_diagonal_and_probes(name, groups):
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    cfg = synth.CONFIGS[name]
    syn = synth.LayerSynth(cfg, dev, seed=0)
    d_in = cfg.d_in
    rng = np.random.default_rng(5)
    V = rng.choice([-1.0, 1.0], size=(N_PROBES, d_in))                 # random signs
    V2 = V * V
    Hs = {g: torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev) for g in groups}
    wss = {g: [libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, d_in, g), dev) for _ in range(2)]
           for g in groups}
    diag = {g: np.zeros((g, d_in)) for g in groups}
    hv = {g: np.zeros((g, N_PROBES, d_in)) for g in groups}
    var = {g: np.zeros((g * N_PROBES, d_in)) for g in groups}
    dvar = {g: np.zeros((g, d_in)) for g in groups}
    worst_s = 0.0
    # bench.py's chunk loop: the first chunk's saliency as a launch of its own, then one call per chunk that adds the
    # chunk to H and computes the next chunk's saliency (two scratch blocks in turn)
    PREP = libgq.GQ_HESSIAN_S_PREPARED
    grad_next = syn.grad_chunk(0)
    s_gpu = {g: libgq.gq_saliency_prepared(grad_next, g, wss[g][0], 1.0) for g in groups}
    for c in range(cfg.n_chunks):
        X, grad = syn.x_chunk(c), grad_next
        grad_next = syn.grad_chunk(c + 1) if c + 1 < cfg.n_chunks else None
        s_after = {}
        for g in groups:
            if grad_next is not None:
                s_after[g] = libgq.gq_hessian_accumulate_ahead(X, s_gpu[g], Hs[g], wss[g][c & 1], grad_next,
                                                               wss[g][(c + 1) & 1], 1.0, flags=PREP)
            else:
                libgq.gq_hessian_accumulate(X, s_gpu[g], Hs[g], wss[g][c & 1], flags=PREP)
        xb, gb = synth.bf16_bits(X), synth.bf16_bits(grad)
        del X, grad
        x = orc.bf16_bits_to_f64(xb)                                   # widened once per chunk, exactly
        x2 = x * x
        q = x2 @ V2.T                                                  # [n, probes]: sum_b v_b^2 x_ib^2
        for g in groups:
            s_ref = orc.saliency(gb, g)
            got = s_gpu[g].cpu().numpy().astype(np.float64)
            floor = 1e-10 * np.abs(s_ref).max()
            err = np.abs(got - s_ref) / (np.abs(s_ref) + floor)
            worst_s = max(worst_s, float(err.max()))
            assert err.max() <= S_RTOL * (1 + 1e-6), "chunk %d, g %d: saliency rel err %.3e" % (c, g, err.max())
            orc.hessian_diag(x, s_ref, diag[g], impl="numpy")
            orc.hessian_apply(x, s_ref, V, hv[g], impl="numpy")
            w = (s_ref[:, None, :] ** 2 * q.T[None, :, :]).reshape(g * N_PROBES, -1)     # s_k[i]^2 q_i per (k, probe)
            orc.hessian_diag(x, w, var[g], impl="numpy")
            orc.hessian_diag(x2, s_ref ** 2, dvar[g], impl="numpy")                      # sum_i s_i^2 x_ia^4
        s_gpu = s_after
    libgq.gq_check()
    Vd = torch.from_numpy(V).to(dev)
    for g in groups:
        H = Hs[g]
        libgq.gq_hessian_finalize(H)
        libgq.gq_check()
        for k in range(g):
            d_gpu = torch.diagonal(H[k]).double().cpu().numpy()
            d_err = np.abs(d_gpu - diag[g][k])
            d_tol = SIGMAS * EPS_RMS * np.sqrt(dvar[g][k]) + ACC_SLACK * diag[g][k] + 1e-300
            assert np.all(d_err <= d_tol), "g %d group %d: diagonal off by %.2f of its tolerance (%.3e relative)" % (
                g, k, (d_err / d_tol).max(), (d_err / np.maximum(diag[g][k], 1e-300)).max())
            # probes through the finalized (full, mirrored) matrix; the product is formed in fp64 row block by row block
            got = np.empty((N_PROBES, d_in))
            for r0 in range(0, d_in, 4096):
                got[:, r0:r0 + 4096] = (H[k, r0:r0 + 4096].double() @ Vd.T).T.cpu().numpy()
            tol = SIGMAS * EPS_RMS * np.sqrt(var[g][k * N_PROBES:(k + 1) * N_PROBES]) + ACC_SLACK * diag[g][k][None, :]
            p_err = np.abs(got - hv[g][k])
            assert np.all(p_err <= tol), "g %d group %d: probe off by %.2f of its tolerance at %s" % (
                g, k, (p_err / tol).max(), np.unravel_index(np.argmax(p_err / tol), p_err.shape))
        del H
    Hs.clear()
    torch.cuda.empty_cache()
