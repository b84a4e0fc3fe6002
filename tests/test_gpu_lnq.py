"""GPU parity of gq_codebook_update (Eq. 8) and of the LNQ loop built from it and gq_cd_cycles (Algorithm 2)
against the CPU fp64 oracle.

The codebook step is a least-squares solve; its solution is unique, so the codebooks are compared value by
value (tolerance relative to the channel's largest level), and, because a level that hardly any coordinate
uses is poorly determined, also through what the levels are for: each channel's objective at the GPU's
codebook must be within 1e-3 of the optimum the oracle finds, and never above the objective before the step.
"""
import numpy as np
import pytest
import torch

from oracle import cd_oracle as cdo
from paper_2505_07004_b200 import api as libgq

pytestmark = pytest.mark.gpu

C_RTOL = 2e-4            # |c - c_oracle| <= C_RTOL * max_q |c_oracle[j, q]|
F_RTOL = 1e-3            # objective at the GPU's codebook vs the oracle's optimum


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    return torch.device("cuda:0")


def make_problem(seed, d_in, d_out, g, m, n=None):
    rng = np.random.default_rng(seed)
    n = n or 2 * d_in
    X = rng.standard_normal((n, d_in)) * np.exp(0.7 * rng.standard_normal(d_in))
    H = np.stack([(X * (rng.random((n, 1)) * np.exp(rng.standard_normal((n, 1))))).T @ X for _ in range(g)])
    H = ((H + H.transpose(0, 2, 1)) / 2).astype(np.float32)
    W = (0.02 * rng.standard_normal((d_out, d_in))).astype(np.float32)
    lo, hi = W.min(1, keepdims=True), W.max(1, keepdims=True)
    cb = (lo + (hi - lo) * (np.arange(m)[None, :] + 0.5) / m).astype(np.float32)
    W0, Q0 = cdo.round_to_codebook(W, cb)
    return W, W0.astype(np.float32), Q0, cb, H


def per_channel_objective(W, What, H):
    mk = W.shape[0] // H.shape[0]
    return np.array([cdo.channel_objective(What[j].astype(np.float64) - W[j], H[j // mk].astype(np.float64))
                     for j in range(W.shape[0])])


def gpu_codebook(dev, W, Q, m, H, lam=1e-7):
    d_out, d_in = W.shape
    Wd, Qd, Hd = torch.from_numpy(W).to(dev), torch.from_numpy(Q.astype(np.uint8)).to(dev), torch.from_numpy(H).to(dev)
    ws = libgq.alloc_workspace(libgq.gq_codebook_workspace_bytes(d_in, d_out, H.shape[0], m), dev)
    What = torch.empty_like(Wd)
    cb, What = libgq.gq_codebook_update(Wd, Qd, m, Hd, ws, lam=lam, W_hat=What)
    libgq.gq_check()
    return cb.cpu().numpy(), What.cpu().numpy()


@pytest.mark.parametrize("seed,d_in,d_out,g,m", [
    (0, 128, 64, 2, 4),
    (1, 328, 96, 3, 8),         # ragged row block, three groups
    (2, 520, 48, 2, 16),        # 24 channels per group
    (3, 1032, 256, 1, 2),
    (4, 768, 2304, 2, 16),      # 1152 channels per group: two slabs of one-hot columns (1024 + 128)
    (5, 520, 192, 2, 8),        # 768 one-hot columns per group: three column tiles, the wide product's odd last tile
    (6, 264, 208, 2, 8),        # 832 columns: four column tiles, the last one ragged
])
def test_codebook_update_matches_oracle(dev, seed, d_in, d_out, g, m):
    W, W0, Q0, cb0, H = make_problem(seed, d_in, d_out, g, m)
    cb_g, What_g = gpu_codebook(dev, W, Q0, m, H)
    cb_o = cdo.codebook_update(W, Q0, H, m)
    assert np.array_equal(What_g, np.take_along_axis(cb_g, Q0, axis=1))
    scale = np.abs(cb_o).max(axis=1, keepdims=True)
    err = np.abs(cb_g - cb_o) / scale
    f_before = per_channel_objective(W, W0, H)
    f_g = per_channel_objective(W, What_g, H)
    f_o = per_channel_objective(W, np.take_along_axis(cb_o, Q0, axis=1), H)
    print("codebook max rel err %.2e; objective excess max %.2e" % (err.max(), ((f_g - f_o) / f_o).max()))
    assert err.max() <= C_RTOL
    assert np.all(f_g <= f_o * (1 + F_RTOL))
    assert np.all(f_g <= f_before * (1 + 1e-6))


def test_codebook_update_unused_level_and_errors(dev):
    W, W0, Q0, cb0, H = make_problem(5, 256, 32, 2, 4)
    Q1 = Q0.copy()
    Q1[Q1 == 3] = 2                                       # nobody uses level 3
    cb_g, _ = gpu_codebook(dev, W, Q1, 4, H)
    cb_o = cdo.codebook_update(W, Q1, H, 4)
    assert np.all(cb_g[:, 3] == 0.0)
    assert np.abs(cb_g - cb_o).max() <= C_RTOL * np.abs(cb_o).max()
    Wd, Qd, Hd = torch.from_numpy(W).to(dev), torch.from_numpy(Q1.astype(np.uint8)).to(dev), torch.from_numpy(H).to(dev)
    ws = libgq.alloc_workspace(libgq.gq_codebook_workspace_bytes(256, 32, 2, 4), dev)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_codebook_update(Wd, Qd, 17, Hd, ws)
    assert "GQ_ERR_UNSUPPORTED_SHAPE" in str(e.value)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_codebook_update(Wd, Qd, 4, Hd, ws[:4096])
    assert "GQ_ERR_WORKSPACE" in str(e.value)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_codebook_update(Wd, Qd, 4, Hd, ws, lam=-1.0)
    assert "GQ_ERR_INVALID_ARG" in str(e.value)
    assert libgq.gq_codebook_workspace_bytes(256, 32, 2, 0) == 0


def test_lnq_loop_descends_like_the_oracle(dev):
    """Algorithm 2 with T = 2, K = 2 from the calls of the library: every step is a descent step for every
    channel, and the final objective is within 2 % of the oracle's run (the two follow slightly different
    paths wherever a rounding decision was a near-tie, see test_gpu_cd.py)."""
    d_in, d_out, g, m = 640, 256, 2, 8
    W, W0, Q0, cb0, H = make_problem(21, d_in, d_out, g, m)
    Wd, Hd = torch.from_numpy(W).to(dev), torch.from_numpy(H).to(dev)
    Q = torch.from_numpy(Q0.astype(np.uint8)).to(dev)
    What = torch.from_numpy(W0.copy()).to(dev)
    cbw = libgq.alloc_workspace(libgq.gq_codebook_workspace_bytes(d_in, d_out, g, m), dev)
    cdw = libgq.alloc_workspace(libgq.gq_cd_workspace_bytes(d_in, d_out, g), dev)
    f = [per_channel_objective(W, W0, H)]
    for _ in range(2):
        cb, What = libgq.gq_codebook_update(Wd, Q, m, Hd, cbw, W_hat=What)
        f.append(per_channel_objective(W, What.cpu().numpy(), H))
        What, Q = libgq.gq_cd_cycles(Wd, What, cb, Hd, 2, cdw, Q=Q)
        f.append(per_channel_objective(W, What.cpu().numpy(), H))
    cb, What = libgq.gq_codebook_update(Wd, Q, m, Hd, cbw, W_hat=What)
    libgq.gq_check()
    f.append(per_channel_objective(W, What.cpu().numpy(), H))
    for a, b in zip(f[:-1], f[1:]):
        assert np.all(b <= a * (1 + 1e-5)), "a step of the LNQ loop increased a channel's objective"
    What_o, Q_o, cb_o = cdo.lnq(W, Q0, H, m, T=2, K=2)
    f_o = per_channel_objective(W, What_o, H)
    mk = d_out // g
    tg, to = f[-1].reshape(g, mk).sum(1), f_o.reshape(g, mk).sum(1)
    print("LNQ objective per group: start %s, GPU %s, oracle %s" % (f[0].reshape(g, mk).sum(1), tg, to))
    assert np.all(np.abs(tg - to) <= 2e-2 * to)
    assert np.all(tg < 0.9 * f[0].reshape(g, mk).sum(1))


def test_full_size_layer_sampled_channels(dev):
    """The layer size the timing script uses (d_in = d_out = 4096, 4 groups, 16 levels), whole layer on the GPU,
    oracle on sampled channels (channels are independent given H_k and the codes): codebook step, then one CD
    cycle, then the codebook step on the new codes.  Inputs are drawn on the device with torch and the same
    bits are handed to the oracle."""
    d_in = d_out = 4096
    g, m, n = 4, 16, 8192
    mk = d_out // g
    gen = torch.Generator(device=dev).manual_seed(31)
    X = torch.randn(n, d_in, device=dev, generator=gen) * torch.exp(0.7 * torch.randn(d_in, device=dev, generator=gen))
    sal = torch.rand(g, n, device=dev, generator=gen) * torch.exp(torch.randn(g, n, device=dev, generator=gen))
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    Hd = torch.stack([(X * sal[k][:, None]).T @ X for k in range(g)])
    torch.backends.cuda.matmul.allow_tf32 = old
    Hd = ((Hd + Hd.transpose(1, 2)) / 2).contiguous()
    del X, sal
    Wd = 0.02 * torch.randn(d_out, d_in, device=dev, generator=gen)
    lo, hi = Wd.min(1, keepdim=True).values, Wd.max(1, keepdim=True).values
    cb0 = lo + (hi - lo) * (torch.arange(m, device=dev)[None, :] + 0.5) / m
    Q0 = ((Wd - lo) / (hi - lo) * m).floor().clamp_(0, m - 1).to(torch.uint8)          # a valid starting assignment
    sel = np.concatenate([k * mk + np.array([0, 1, 517, mk - 1]) for k in range(g)])
    W, H = Wd.cpu().numpy(), Hd.cpu().numpy()

    cbw = libgq.alloc_workspace(libgq.gq_codebook_workspace_bytes(d_in, d_out, g, m), dev)
    cdw = libgq.alloc_workspace(libgq.gq_cd_workspace_bytes(d_in, d_out, g), dev)
    What = torch.empty_like(Wd)
    cb1, What = libgq.gq_codebook_update(Wd, Q0, m, Hd, cbw, W_hat=What)
    cb1_h, What1_h = cb1.cpu().numpy(), What.cpu().numpy()
    What2, Q2 = libgq.gq_cd_cycles(Wd, What, cb1, Hd, 1, cdw, Q=Q0.clone())
    cb3, What3 = libgq.gq_codebook_update(Wd, Q2, m, Hd, cbw, W_hat=torch.empty_like(Wd))
    libgq.gq_check()
    Q0_h, Q2_h, What2_h = Q0.cpu().numpy().astype(np.int32), Q2.cpu().numpy().astype(np.int32), What2.cpu().numpy()
    cb3_h = cb3.cpu().numpy()

    n_tie = 0
    for j in sel:
        Hk = H[j // mk][None].astype(np.float64)
        # codebook step on the starting codes
        c_o = cdo.codebook_update(W[j:j + 1], Q0_h[j:j + 1], Hk, m)[0]
        assert np.abs(cb1_h[j] - c_o).max() <= C_RTOL * np.abs(c_o).max()
        assert np.array_equal(What1_h[j], cb1_h[j][Q0_h[j]])
        # one CD cycle from the GPU's own codebook and starting point
        Wo, Qo = cdo.cd(W[j:j + 1], What1_h[j:j + 1], cb1_h[j:j + 1], Hk, 1, 128)
        assert np.array_equal(What2_h[j], cb1_h[j][Q2_h[j]])
        f0 = cdo.channel_objective(What1_h[j].astype(np.float64) - W[j], Hk[0])
        fg = cdo.channel_objective(What2_h[j].astype(np.float64) - W[j], Hk[0])
        fo = cdo.channel_objective(Wo[0].astype(np.float64) - W[j], Hk[0])
        assert fg <= f0 * (1 + 1e-6)
        if not np.array_equal(Q2_h[j], Qo[0]):
            i = int(np.nonzero(Q2_h[j] != Qo[0])[0][0])
            state = What1_h[j].astype(np.float64).copy()
            state[:i] = Wo[0, :i]
            t, mag = cdo.coordinate_target(W[j], state, Hk[0], i)
            da, db = abs(t - float(cb1_h[j, Q2_h[j, i]])), abs(t - float(cb1_h[j, Qo[0, i]]))
            assert abs(da - db) <= 2e-4 * mag, "channel %d coordinate %d is no near-tie" % (j, i)
            assert abs(fg - fo) <= 2e-2 * fo
            n_tie += 1
        # codebook step on the GPU's new codes
        c_o = cdo.codebook_update(W[j:j + 1], Q2_h[j:j + 1], Hk, m)[0]
        assert np.abs(cb3_h[j] - c_o).max() <= C_RTOL * np.abs(c_o).max()
    print("sampled channels on a near-tie path: %d of %d" % (n_tie, len(sel)))
    assert n_tie <= len(sel) // 2


def test_gq_lnq_is_the_sequence_of_its_steps(dev):
    """gq_lnq (Algorithm 2 as one call) must give bit for bit what the separate calls give, and land where the
    oracle's LNQ lands (objective per group within 2 %, see test_lnq_loop_descends_like_the_oracle)."""
    d_in, d_out, g, m, T, K = 640, 256, 2, 8, 2, 2
    W, W0, Q0, cb0, H = make_problem(21, d_in, d_out, g, m)
    Wd, Hd = torch.from_numpy(W).to(dev), torch.from_numpy(H).to(dev)
    ws = libgq.alloc_workspace(libgq.gq_lnq_workspace_bytes(d_in, d_out, g, m), dev)
    assert ws.numel() == max(libgq.gq_codebook_workspace_bytes(d_in, d_out, g, m), libgq.gq_cd_workspace_bytes(d_in, d_out, g))
    What1, Q1, cb1 = libgq.gq_lnq(Wd, torch.from_numpy(Q0.astype(np.uint8)).to(dev), m, Hd, T, K, ws)
    libgq.gq_check()
    Q = torch.from_numpy(Q0.astype(np.uint8)).to(dev)
    What = torch.empty_like(Wd)
    for _ in range(T):
        cb, What = libgq.gq_codebook_update(Wd, Q, m, Hd, ws, W_hat=What)
        What, Q = libgq.gq_cd_cycles(Wd, What, cb, Hd, K, ws, Q=Q)
    cb, What = libgq.gq_codebook_update(Wd, Q, m, Hd, ws, W_hat=What)
    libgq.gq_check()
    assert torch.equal(Q1, Q) and torch.equal(cb1, cb) and torch.equal(What1, What)
    What_o, Q_o, cb_o = cdo.lnq(W, Q0, H, m, T=T, K=K)
    mk = d_out // g
    tg = per_channel_objective(W, What1.cpu().numpy(), H).reshape(g, mk).sum(1)
    to = per_channel_objective(W, What_o, H).reshape(g, mk).sum(1)
    assert np.all(np.abs(tg - to) <= 2e-2 * to)
    # K = 0: only codebook steps, the assignment is untouched
    What0, Qk, cbk = libgq.gq_lnq(Wd, torch.from_numpy(Q0.astype(np.uint8)).to(dev), m, Hd, 3, 0, ws)
    assert np.array_equal(Qk.cpu().numpy(), Q0.astype(np.uint8))
    cb_first, _ = libgq.gq_codebook_update(Wd, Qk, m, Hd, ws)
    assert torch.equal(cbk, cb_first)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_lnq(Wd, Qk, m, Hd, 1, 1, ws[:4096])
    assert "GQ_ERR_WORKSPACE" in str(e.value)
    with pytest.raises(libgq.GQError):
        libgq.gq_lnq(Wd, Qk, 17, Hd, 1, 1, ws)
    with pytest.raises(libgq.GQError):
        libgq.gq_lnq(Wd, Qk, m, Hd, -1, 1, ws)


def test_whole_pipeline_guided_hessian_to_quantised_layer(dev):
    """Everything through the library: saliency -> guided Hessians -> finalize -> LNQ -> objective.  The
    objective the library reports for the quantised layer must match the oracle's evaluation (Eq. 7) on the
    oracle's own Hessians, and LNQ must have lowered it below nearest-level rounding to a uniform grid."""
    from oracle import gq_oracle as orc
    from paper_2505_07004_b200 import synth
    cfg = synth.LayerConfig("p", 3000, 1024, 512, 256, (2,), "lognormal", 0.02, 20.0)
    syn = synth.LayerSynth(cfg, dev, seed=9)
    g, m = 2, 8
    H = torch.zeros(g, cfg.d_in, cfg.d_in, device=dev)
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev)
    xb, gb = [], []
    for c in range(cfg.n_chunks):
        x, gr = syn.x_chunk(c), syn.grad_chunk(c)
        xb.append(synth.bf16_bits(x))
        gb.append(synth.bf16_bits(gr))
        libgq.gq_hessian_accumulate(x, libgq.gq_saliency(gr, g, 1e3), H, ws)
    libgq.gq_hessian_finalize(H)
    W, _ = syn.weights()
    lo, hi = W.min(1, keepdim=True).values, W.max(1, keepdim=True).values
    Q0 = ((W - lo) / (hi - lo) * m).floor().clamp_(0, m - 1).to(torch.uint8)
    W_grid = lo + (hi - lo) * (Q0.float() + 0.5) / m
    ows = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(cfg.d_in, cfg.d_out, g), dev)
    f_grid = libgq.gq_objective(W, W_grid.contiguous(), H, ows).cpu().numpy()
    lws = libgq.alloc_workspace(libgq.gq_lnq_workspace_bytes(cfg.d_in, cfg.d_out, g, m), dev)
    What, Q, cb = libgq.gq_lnq(W, Q0.clone(), m, H, 2, 2, lws)
    f_lnq = libgq.gq_objective(W, What, H, ows).cpu().numpy()
    libgq.gq_check()
    assert torch.equal(What, torch.gather(cb, 1, Q.long()))
    assert np.all(f_lnq[:g] < 0.5 * f_grid[:g])
    # oracle: its own saliency and Hessians from the same bits, its own objective of the GPU's W_hat
    s_o = orc.saliency(np.concatenate(gb), g, 1e3)
    H_o = orc.hessian(np.concatenate(xb), s_o)
    f_o = orc.objective(W.cpu().numpy(), What.cpu().numpy(), H_o)
    assert np.all(np.abs(f_lnq - f_o) <= 1e-3 * np.abs(f_o)), (f_lnq, f_o)
