"""GPU parity: libgq (through the C-ABI binding) against the CPU fp64 oracle, same seeded inputs.

Tolerances of this path:
  saliency   |s - s_o| <= 1e-4 * |s_o| per element (plus a floor of 1e-4 * max|s_o| * 1e-6 for zeros)
  Hessian    ||H_k - H_k_o||_F <= 5e-3 ||H_k_o||_F   and   max|H_k - H_k_o| <= 1e-2 max|H_k_o|
             and, entry by entry, |H_k - H_k_o|[a][b] <= 4.5e-3 sqrt(H_k_o[a][a] H_k_o[b][b])
  objective  |loss - loss_o| <= 1e-3 |loss_o|
The entry-wise bound does not depend on the scale of a feature (the first two are set by the few outlier
features): the only rounding of the Hessian kernel that is not of fp32 size is the one bf16 rounding of each
product s_k[i] X[i][a] (8 significant bits), a relative error of at most 2^-8, so
|error of H[a][b]| <= 2^-8 sum_i s_i |X[i][a]| |X[i][b]| <= 2^-8 sqrt(H[a][a] H[b][b]) (Cauchy-Schwarz) = 3.9e-3 of
that geometric mean, reached only by a single token whose product rounds by half a unit; 4.5e-3 leaves room for
the two-term saliency (2^-17) and fp32 accumulation.
"""
import numpy as np
import pytest
import torch

from oracle import gq_oracle as orc
from paper_2505_07004_b200 import api as libgq
from paper_2505_07004_b200 import synth

pytestmark = pytest.mark.gpu

S_RTOL, H_FRO, H_MAX, H_ENTRY, L_RTOL = 1e-4, 5e-3, 1e-2, 4.5e-3, 1e-3


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    return torch.device("cuda:0")


def check_s(s_gpu, s_ref):
    s_gpu = s_gpu.detach().cpu().numpy().astype(np.float64)
    floor = 1e-10 * np.abs(s_ref).max()
    assert np.all(np.abs(s_gpu - s_ref) <= S_RTOL * np.abs(s_ref) + floor), \
        "saliency max rel err %.3e" % (np.abs(s_gpu - s_ref) / (np.abs(s_ref) + floor)).max()


def check_H(H_gpu, H_ref, upper_only=False):
    H_gpu = H_gpu.detach().cpu().numpy().astype(np.float64)
    for k in range(H_ref.shape[0]):
        a, b = H_gpu[k], H_ref[k]
        if upper_only:
            a, b = np.triu(a), np.triu(b)
        fro = np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)
        mx = np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)
        assert fro <= H_FRO and mx <= H_MAX, "group %d: rel Frobenius %.3e, max-elem %.3e" % (k, fro, mx)
        # scale-free companion: every entry against the geometric mean of its two diagonal entries
        dg = np.sqrt(np.maximum(np.diag(H_ref[k]), 0.0))
        scale = np.outer(dg, dg)
        excess = np.abs(a - b) - H_ENTRY * scale
        assert np.all(excess <= 1e-30), "group %d: entry %s off by %.3e of sqrt(H_aa H_bb)" % (
            k, np.unravel_index(np.argmax(excess), excess.shape), (np.abs(a - b) / np.maximum(scale, 1e-300)).max())


def check_loss(loss_gpu, loss_ref):
    loss_gpu = loss_gpu.detach().cpu().numpy()
    assert np.all(np.isfinite(loss_gpu))
    scale = np.maximum(np.abs(loss_ref), 1e-300)
    assert np.all(np.abs(loss_gpu - loss_ref) <= L_RTOL * scale), \
        "objective rel err %s" % (np.abs(loss_gpu - loss_ref) / scale)


def gpu_hessian(X_chunks, s_chunks, d_in, g, dev, finalize=True, flags=0):
    H = torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev)
    n_max = max([x.shape[0] for x in X_chunks] + [1])
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(n_max, d_in, g, flags), dev)
    for x, s in zip(X_chunks, s_chunks):
        libgq.gq_hessian_accumulate(x, s, H, ws, flags=flags)
    if finalize:
        libgq.gq_hessian_finalize(H)
    libgq.gq_check()
    return H


# ------------------------------------------------------------------------------------------ saliency
@pytest.mark.parametrize("n,d_out,g,pad,scale", [
    (2048, 512, 4, 0, 1.0),       # tiny config
    (1, 8, 1, 0, 1.0),            # one token, one vector
    (333, 4096, 4, 0, 1.0),       # m = 1024: one full unrolled pass
    (257, 11008, 16, 0, 1.0),     # m = 688: tail path only
    (100, 2560, 2, 64, 1e3),      # m = 1280: unrolled pass + tail; padded rows; paper's scale
    (65, 24, 3, 8, 1.0),          # m = 8
])
def test_saliency_parity(dev, n, d_out, g, pad, scale):
    gen = torch.Generator(device=dev).manual_seed(n * 7 + d_out)
    full = (torch.randn(n, d_out + pad, generator=gen, device=dev) * 1e-3).to(torch.bfloat16)
    grad = full[:, :d_out]
    s = libgq.gq_saliency(grad, g, scale)
    libgq.gq_check()
    s_ref = orc.saliency(synth.bf16_bits(grad.contiguous()), g, scale)
    check_s(s, s_ref)


def test_saliency_empty_and_errors(dev):
    grad = torch.zeros((0, 64), dtype=torch.bfloat16, device=dev)
    s = libgq.gq_saliency(grad, 2)
    assert tuple(s.shape) == (2, 0)
    grad = torch.zeros((4, 24), dtype=torch.bfloat16, device=dev)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_saliency(grad, 5)                      # 24 % 5 != 0
    assert "GQ_ERR_INVALID_ARG" in str(e.value)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_saliency(grad, 6)                      # m = 4 is not a multiple of 8
    assert "GQ_ERR_UNSUPPORTED_SHAPE" in str(e.value)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_saliency(grad, 1, float("nan"))
    assert "GQ_ERR_INVALID_ARG" in str(e.value)


@pytest.mark.parametrize("dtype,np_dtype,name", [(torch.bfloat16, np.uint16, "bf16"), (torch.float16, np.float16, "fp16"),
                                                 (torch.float32, np.float32, "fp32")])
@pytest.mark.parametrize("batch,seq,d_out,g,pad,bstep", [(3, 37, 512, 4, 0, 1), (2, 65, 688, 2, 40, 2), (1, 1, 8, 1, 0, 1),
                                                          (4, 19, 11008, 16, 0, 1), (2, 8, 2560, 2, 8, 3)])
def test_saliency_strided_parity(dev, dtype, np_dtype, name, batch, seq, d_out, g, pad, bstep):
    """gq_saliency_strided on [batch, seq, d_out] views (padded rows, every bstep-th slab of a larger buffer) in the
    three gradient dtypes, written into a slice of a wider s buffer, against the oracle on the same bits."""
    gen = torch.Generator(device=dev).manual_seed(batch * 1000 + seq + d_out)
    base = (torch.randn(batch * bstep, seq, d_out + pad, generator=gen, device=dev) * 3e-3)
    base = (base * torch.exp(torch.randn(batch * bstep, seq, 1, generator=gen, device=dev))).to(dtype)
    view = base[::bstep, :, :d_out]
    n, off = batch * seq, 24
    s_all = torch.full((g, n + 48), -1.0, device=dev)
    libgq.gq_saliency_strided(view, g, 2.0, s=s_all[:, off:off + n])
    libgq.gq_check()
    host = base.cpu()
    host_np = host.view(torch.int16).numpy().view(np.uint16) if dtype == torch.bfloat16 else host.numpy()
    s_ref = orc.saliency_strided(host_np[::bstep, :, :d_out], name, g, 2.0)
    check_s(s_all[:, off:off + n], s_ref)
    assert torch.all(s_all[:, :off] == -1.0) and torch.all(s_all[:, off + n:] == -1.0)      # nothing else is touched
    if dtype == torch.bfloat16 and pad == 0 and bstep == 1:
        s_plain = libgq.gq_saliency(view.reshape(n, d_out), g, 2.0)
        assert torch.equal(s_plain, s_all[:, off:off + n])                                  # same arithmetic, same bits


def test_saliency_strided_errors(dev):
    grad = torch.zeros((2, 4, 68), dtype=torch.float16, device=dev)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_saliency_strided(grad[:, :, :64], 2)            # row stride 68 is not a multiple of 16 bytes
    assert "GQ_ERR_ALIGNMENT" in str(e.value)
    with pytest.raises(ValueError):
        libgq.gq_saliency_strided(torch.zeros((2, 4, 64), dtype=torch.float64, device=dev), 2)
    s = libgq.gq_saliency_strided(torch.zeros((0, 4, 64), dtype=torch.float32, device=dev), 2)
    assert tuple(s.shape) == (2, 0)


# ------------------------------------------------------------------------------------------ Hessian
@pytest.mark.parametrize("flags", [0, libgq.GQ_HESSIAN_DETERMINISTIC])
@pytest.mark.parametrize("n,d_in,g,chunks", [
    (2048, 256, 4, [2048]),                 # tiny config: one 256 x 256 tile per group, cut along tokens
    (677, 384, 2, [677]),                   # ragged K tail, d_in = 1.5 column blocks
    (1, 8, 1, [1]),                         # smallest legal problem
    (130, 520, 3, [64, 1, 65]),             # several chunks incl. a 1-token chunk; ragged tiles
    (300, 1032, 2, [300]),                  # 5 column blocks, tail of 8 features
    (96, 640, 5, [0, 96]),                  # an empty chunk is a no-op
    (1500, 3080, 2, [1000, 500]),           # 182 units on 74 SM pairs: two whole rounds plus a cut tail
    (200, 1288, 1, [200]),                  # one group: units of two column tiles (6 column blocks)
    (150, 1800, 3, [90, 60]),               # odd g: pair units for groups 0-1, column-pair units for group 2
    (70, 1096, 1, [70]),                    # one group, odd number of column blocks (5): a lone last column
])
def test_hessian_parity_small(dev, n, d_in, g, chunks, flags):
    gen = torch.Generator(device=dev).manual_seed(n + d_in)
    feat = torch.exp(torch.randn(d_in, generator=gen, device=dev))
    X = (torch.randn(n, d_in, generator=gen, device=dev) * feat).to(torch.bfloat16)
    s = (torch.rand(g, n, generator=gen, device=dev) * torch.exp(torch.randn(1, n, generator=gen, device=dev)))
    s = s.contiguous()
    xs, ss, lo = [], [], 0
    for c in chunks:
        xs.append(X[lo:lo + c])
        ss.append(s[:, lo:lo + c])
        lo += c
    assert lo == n
    H = gpu_hessian(xs, ss, d_in, g, dev, finalize=False, flags=flags)
    H_ref = orc.hessian(synth.bf16_bits(X), s.cpu().numpy().astype(np.float64))
    check_H(H, H_ref, upper_only=True)
    libgq.gq_hessian_finalize(H)
    libgq.gq_check()
    check_H(H, H_ref)
    Hc = H.cpu()
    assert torch.equal(Hc, Hc.transpose(1, 2)), "finalized H must be exactly symmetric"


def test_hessian_unit_saliency_is_gram_and_deterministic(dev):
    n, d_in = 2000, 512
    gen = torch.Generator(device=dev).manual_seed(3)
    X = torch.randn(n, d_in, generator=gen, device=dev).to(torch.bfloat16)
    s = torch.ones(1, n, device=dev)
    H1 = gpu_hessian([X, X], [s, s], d_in, 1, dev, flags=libgq.GQ_HESSIAN_DETERMINISTIC)
    H2 = gpu_hessian([X, X], [s, s], d_in, 1, dev, flags=libgq.GQ_HESSIAN_DETERMINISTIC)
    assert torch.equal(H1, H2)          # single writer per element: bit-reproducible
    H3 = gpu_hessian([X, X], [s, s], d_in, 1, dev)          # balanced: tiles cut along tokens, atomics
    assert torch.allclose(H1, H3, rtol=1e-5, atol=1e-3)
    H1 = gpu_hessian([X], [s], d_in, 1, dev, flags=libgq.GQ_HESSIAN_DETERMINISTIC)
    ref = X.double().T @ X.double()
    rel = (H1[0].double() - ref).norm() / ref.norm()
    assert rel.item() < 1e-5            # unit weights are exact in bf16: only fp32 accumulation error remains


@pytest.mark.parametrize("n,d_in,d_out,g", [(700, 520, 512, 4), (333, 264, 120, 3), (64, 256, 8, 1)])
def test_prepared_saliency_gives_the_same_hessian(dev, n, d_in, d_out, g):
    """gq_saliency_prepared + GQ_HESSIAN_S_PREPARED (two launches) against gq_saliency + gq_hessian_accumulate
    (three): same fp32 s, and with the single-writer schedule the same H bit for bit."""
    gen = torch.Generator(device=dev).manual_seed(n + d_in + g)
    X = torch.randn(n, d_in, generator=gen, device=dev).to(torch.bfloat16)
    grad = (torch.randn(n, d_out, generator=gen, device=dev) * torch.exp(torch.randn(n, 1, generator=gen, device=dev)))
    grad = grad.to(torch.bfloat16)
    flags = libgq.GQ_HESSIAN_DETERMINISTIC
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(n, d_in, g, flags), dev)
    s1 = libgq.gq_saliency(grad, g)
    H1 = torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev)
    libgq.gq_hessian_accumulate(X, s1, H1, ws, flags=flags)
    ws.fill_(0xFF)                                       # nothing of the first run may be left in the workspace
    s2 = libgq.gq_saliency_prepared(grad, g, ws)
    H2 = torch.zeros_like(H1)
    libgq.gq_hessian_accumulate(X, s2, H2, ws, flags=flags | libgq.GQ_HESSIAN_S_PREPARED)
    libgq.gq_check()
    assert torch.equal(s1, s2)
    assert torch.equal(H1, H2)
    check_s(s2, orc.saliency(synth.bf16_bits(grad), g))
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_saliency_prepared(grad, g, ws[:8])
    assert "GQ_ERR_WORKSPACE" in str(e.value)


@pytest.mark.parametrize("chunks,d_in,d_out,g", [
    ([300, 257, 64, 1], 520, 512, 4),      # ragged chunks, short segments (two per round of the look-ahead warps)
    ([200, 333], 264, 120, 3),             # odd g: the last group's second word is written as 0
    ([96, 160, 31], 2048, 4096, 1),        # segments of 512 vectors: two rounds of the long-segment loop
    ([130, 70], 1024, 2080, 2),            # 130 vectors per segment: just over the short-segment limit
])
def test_accumulate_ahead_matches_oracle_and_two_launch_path(dev, chunks, d_in, d_out, g):
    """The chunk loop with the saliency of chunk c + 1 computed inside the Hessian launch of chunk c
    (gq_hessian_accumulate_ahead): s of every chunk against the oracle and bit-equal to gq_saliency_prepared, H
    against the oracle and (single-writer schedule) bit-equal to the two-launch loop."""
    gen = torch.Generator(device=dev).manual_seed(sum(chunks) + d_in + g)
    X = [torch.randn(n, d_in, generator=gen, device=dev).to(torch.bfloat16) for n in chunks]
    G = [(torch.randn(n, d_out, generator=gen, device=dev) * torch.exp(torch.randn(n, 1, generator=gen, device=dev))
          ).to(torch.bfloat16) for n in chunks]
    flags = libgq.GQ_HESSIAN_DETERMINISTIC | libgq.GQ_HESSIAN_S_PREPARED
    nb = libgq.gq_hessian_workspace_bytes(max(chunks), d_in, g, flags)
    ws = [libgq.alloc_workspace(nb, dev) for _ in range(2)]
    for w in ws:
        w.fill_(0xFF)
    n_all = sum(chunks)
    s_all = torch.full((g, n_all + 3), -1.0, dtype=torch.float32, device=dev)      # one buffer for all chunks, padded
    offs = np.concatenate([[0], np.cumsum(chunks)])
    view = lambda c: s_all[:, offs[c]:offs[c + 1]]
    H = torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev)
    launches = libgq.gq_launch_count()
    libgq.gq_saliency_prepared(G[0], g, ws[0], 1.0, view(0))
    for c in range(len(chunks)):
        if c + 1 < len(chunks):
            libgq.gq_hessian_accumulate_ahead(X[c], view(c), H, ws[c & 1], G[c + 1], ws[(c + 1) & 1], 1.0, view(c + 1), flags)
        else:
            libgq.gq_hessian_accumulate(X[c], view(c), H, ws[c & 1], flags)
    # every case has enough CTAs for its gradient blocks to be hidden: one launch per chunk
    assert libgq.gq_launch_count() - launches == len(chunks) + 1
    libgq.gq_check()
    assert torch.all(s_all[:, n_all:] == -1.0)
    # two launches per chunk, same flags
    H2 = torch.zeros_like(H)
    ws2 = libgq.alloc_workspace(nb, dev)
    for c in range(len(chunks)):
        s2 = libgq.gq_saliency_prepared(G[c], g, ws2)
        assert torch.equal(s2, view(c))
        used = (g + 1) // 2 * chunks[c] * 8
        assert torch.equal(ws2[:used], ws[c & 1][:used]) or c + 2 < len(chunks)      # a later chunk reused the block
        libgq.gq_hessian_accumulate(X[c], s2, H2, ws2, flags)
    libgq.gq_check()
    assert torch.equal(H, H2)
    s_o = np.concatenate([orc.saliency(synth.bf16_bits(gr), g) for gr in G], axis=1)
    check_s(s_all[:, :n_all], s_o)
    H_o = orc.hessian(np.concatenate([synth.bf16_bits(x) for x in X]), s_o)
    check_H(H, H_o, upper_only=True)


@pytest.mark.parametrize("d_in,d_out,n", [(64, 32768, 512),       # two CTAs
                                         (1024, 8192, 4096)])    # fourteen CTAs, 67 MB of gradients
def test_accumulate_ahead_runs_saliency_separately_when_it_cannot_hide(dev, d_in, d_out, n):
    """One group and many output channels: the next chunk's gradients would take longer to stream than this chunk's
    Hessian work, so the call launches the saliency kernel on its own.  Same results."""
    g = 1
    gen = torch.Generator(device=dev).manual_seed(5)
    X = torch.randn(n, d_in, generator=gen, device=dev).to(torch.bfloat16)
    G = torch.randn(n, d_out, generator=gen, device=dev).to(torch.bfloat16)
    nb = libgq.gq_hessian_workspace_bytes(n, d_in, g)
    ws, ws_next = libgq.alloc_workspace(nb, dev), libgq.alloc_workspace(nb, dev)
    ws_next.fill_(0xFF)
    s = libgq.gq_saliency_prepared(G, g, ws)
    H = torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev)
    launches = libgq.gq_launch_count()
    s_next = libgq.gq_hessian_accumulate_ahead(X, s, H, ws, G, ws_next,
                                               flags=libgq.GQ_HESSIAN_S_PREPARED | libgq.GQ_HESSIAN_DETERMINISTIC)
    assert libgq.gq_launch_count() - launches == 2
    libgq.gq_check()
    assert torch.equal(s_next, s) and torch.equal(ws_next[:n * 8], ws[:n * 8])
    check_s(s_next, orc.saliency(synth.bf16_bits(G), g))
    check_H(H, orc.hessian(synth.bf16_bits(X), s_next.cpu().numpy().astype(np.float64)), upper_only=True)


def test_accumulate_ahead_degenerate_and_errors(dev):
    g, d_in, d_out, n = 2, 64, 32, 48
    X = torch.randn(n, d_in, device=dev).to(torch.bfloat16)
    G = torch.randn(n, d_out, device=dev).to(torch.bfloat16)
    nb = libgq.gq_hessian_workspace_bytes(n, d_in, g)
    ws, ws_next = libgq.alloc_workspace(nb, dev), libgq.alloc_workspace(nb, dev)
    s = libgq.gq_saliency_prepared(G, g, ws)
    H = torch.zeros((g, d_in, d_in), dtype=torch.float32, device=dev)
    # no next chunk: plain accumulate
    libgq.gq_hessian_accumulate_ahead(X, s, H, ws, G[:0], ws_next, flags=libgq.GQ_HESSIAN_S_PREPARED)
    H1 = torch.zeros_like(H)
    libgq.gq_hessian_accumulate(X, s, H1, ws, libgq.GQ_HESSIAN_S_PREPARED)
    assert torch.equal(torch.triu(H), torch.triu(H1))
    # without GQ_HESSIAN_S_PREPARED the call prepares s itself (three kernels' work in two launches)
    H2 = torch.zeros_like(H)
    ws.fill_(0xFF)
    ws_next.fill_(0xFF)
    s_again = libgq.gq_hessian_accumulate_ahead(X, s, H2, ws, G, ws_next)
    assert torch.equal(s_again, s) and torch.equal(torch.triu(H2), torch.triu(H1))
    libgq.gq_saliency_prepared(G, g, ws)                 # restore the packed form of s for the checks below
    # no current chunk: the saliency step alone, H untouched
    s_next = libgq.gq_hessian_accumulate_ahead(X[:0], s[:, :0], H, ws, G, ws_next)
    assert torch.equal(s_next, s) and torch.equal(torch.triu(H), torch.triu(H1))
    used = g // 2 * n * 8
    assert torch.equal(ws_next[:used], ws[:used])
    # the second scratch block must be a different one; next_s must not be the s being read
    for bad in (lambda: libgq.gq_hessian_accumulate_ahead(X, s, H, ws, G, ws, flags=libgq.GQ_HESSIAN_S_PREPARED),
                lambda: libgq.gq_hessian_accumulate_ahead(X, s, H, ws, G, ws_next, next_s=s),
                lambda: libgq.gq_hessian_accumulate_ahead(X, s, H, ws, G, ws_next, next_s=H.view(-1)[:g * n].view(g, n))):
        with pytest.raises(libgq.GQError) as e:
            bad()
        assert "GQ_ERR_INVALID_ARG" in str(e.value)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_hessian_accumulate_ahead(X, s, H, ws, G, ws_next[:8])
    assert "GQ_ERR_WORKSPACE" in str(e.value)
    libgq.gq_check()
    assert torch.equal(torch.triu(H), torch.triu(H1))    # nothing was written by the rejected calls


def test_hessian_errors(dev):
    X = torch.zeros((16, 64), dtype=torch.bfloat16, device=dev)
    s = torch.zeros((2, 16), dtype=torch.float32, device=dev)
    H = torch.zeros((2, 64, 64), dtype=torch.float32, device=dev)
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(16, 64, 2), dev)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_hessian_accumulate(X, s, H, ws[:16])
    assert "GQ_ERR_WORKSPACE" in str(e.value)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_hessian_accumulate(X, s, H, ws, flags=4)
    assert "GQ_ERR_INVALID_ARG" in str(e.value)
    Xbad = torch.zeros((16, 68), dtype=torch.bfloat16, device=dev)
    Hbad = torch.zeros((2, 68, 68), dtype=torch.float32, device=dev)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_hessian_accumulate(Xbad, s, Hbad, ws)
    assert "GQ_ERR_UNSUPPORTED_SHAPE" in str(e.value)
    assert libgq.gq_hessian_workspace_bytes(16, 68, 2) == 0
    assert torch.count_nonzero(H).item() == 0            # nothing was written by the rejected calls


# ------------------------------------------------------------------------------------------ objective
@pytest.mark.parametrize("d_in,d_out,g", [(256, 512, 4), (384, 256, 2), (8, 8, 1), (520, 120, 3), (1032, 64, 1)])
def test_objective_on_oracle_hessian(dev, d_in, d_out, g):
    """Isolates Eq. 7: H comes from the oracle (rounded to fp32), only the objective runs on the GPU."""
    rng = np.random.default_rng(d_in + d_out)
    n = 200
    xb = orc.f64_to_bf16_bits(rng.standard_normal((n, d_in)) * np.exp(rng.standard_normal(d_in)))
    s = rng.random((g, n)) * np.exp(rng.standard_normal(n))
    H32 = orc.hessian(xb, s).astype(np.float32)
    W = (0.02 * rng.standard_normal((d_out, d_in))).astype(np.float32)
    What = synth.uniform_grid_round(torch.from_numpy(W), 16).numpy()
    loss_ref = orc.objective(W, What, H32.astype(np.float64))
    Hd = torch.from_numpy(H32).to(dev)
    ws = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(d_in, d_out, g), dev)
    loss = libgq.gq_objective(torch.from_numpy(W).to(dev), torch.from_numpy(What).to(dev), Hd, ws)
    libgq.gq_check()
    check_loss(loss, loss_ref)
    # only the upper triangle may be read: garbage below the diagonal must not change the result
    Hd2 = Hd.clone()
    tril = torch.tril(torch.ones(d_in, d_in, device=dev, dtype=torch.bool), diagonal=-1)
    Hd2[:, tril] = 1e30
    loss2 = libgq.gq_objective(torch.from_numpy(W).to(dev), torch.from_numpy(What).to(dev), Hd2, ws)
    libgq.gq_check()
    assert torch.equal(loss, loss2)


def test_objective_zero_and_single_entry(dev):
    d_in, d_out, g = 128, 16, 2
    gen = torch.Generator(device=dev).manual_seed(5)
    X = torch.randn(64, d_in, generator=gen, device=dev).to(torch.bfloat16)
    s = torch.rand(g, 64, generator=gen, device=dev)
    H = gpu_hessian([X], [s], d_in, g, dev)
    W = torch.randn(d_out, d_in, generator=gen, device=dev)
    ws = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(d_in, d_out, g), dev)
    loss = libgq.gq_objective(W, W.clone(), H, ws)
    libgq.gq_check()
    assert torch.count_nonzero(loss).item() == 0
    # a single perturbed weight with a value that neither fp16 nor bf16 holds exactly: the result must still be
    # inside the objective's tolerance (11 significant bits per factor: 2^-11 at worst)
    What = W.clone()
    What[11, 77] += 0.123456789
    loss = libgq.gq_objective(W, What, H, ws)
    libgq.gq_check()
    delta = float(W[11, 77].double() - What[11, 77].double())
    expect = delta * delta * float(H[1, 77, 77])
    got = loss.cpu().numpy()
    assert got[0] == 0.0
    assert abs(got[1] - expect) <= L_RTOL * expect and abs(got[2] - expect) <= L_RTOL * expect


# ------------------------------------------------------------------------------------------ whole path
def run_layer(cfg, dev, n_tokens=None, grad_scale=1.0, seed=0):
    syn = synth.LayerSynth(cfg, dev, seed=seed)
    g = cfg.g
    n = cfg.n if n_tokens is None else n_tokens
    H = torch.zeros((g, cfg.d_in, cfg.d_in), dtype=torch.float32, device=dev)
    ws = [libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev) for _ in range(2)]
    xs, gs, ss = [], [], []
    done, c = 0, 0
    while done < n:
        nt = min(cfg.chunk, n - done)
        xs.append(syn.x_chunk(c, nt)), gs.append(syn.grad_chunk(c, nt))
        done += nt
        c += 1
    # the chunk loop bench.py times: saliency of the first chunk, then one launch per chunk that adds the chunk to H
    # and computes the next chunk's saliency (two scratch blocks in turn)
    ss.append(libgq.gq_saliency_prepared(gs[0], g, ws[0], grad_scale))
    for c in range(len(xs)):
        if c + 1 < len(xs):
            ss.append(libgq.gq_hessian_accumulate_ahead(xs[c], ss[c], H, ws[c & 1], gs[c + 1], ws[(c + 1) & 1], grad_scale,
                                                        flags=libgq.GQ_HESSIAN_S_PREPARED))
        else:
            libgq.gq_hessian_accumulate(xs[c], ss[c], H, ws[c & 1], flags=libgq.GQ_HESSIAN_S_PREPARED)
    libgq.gq_hessian_finalize(H)
    W, What = syn.weights()
    ows = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(cfg.d_in, cfg.d_out, g), dev)
    loss = libgq.gq_objective(W, What, H, ows)
    libgq.gq_check()
    return xs, gs, ss, H, W, What, loss


@pytest.mark.parametrize("grad_scale", [1.0, 1e3])
def test_tiny_config_end_to_end(dev, grad_scale):
    cfg = synth.CONFIGS["c0_tiny"]
    xs, gs, ss, H, W, What, loss = run_layer(cfg, dev, grad_scale=grad_scale)
    xb = np.concatenate([synth.bf16_bits(x) for x in xs])
    gb = np.concatenate([synth.bf16_bits(x) for x in gs])
    s_ref = orc.saliency(gb, cfg.g, grad_scale)
    check_s(torch.cat(ss, dim=1), s_ref)
    H_ref = orc.hessian(xb, s_ref)
    check_H(H, H_ref)
    check_loss(loss, orc.objective(W.cpu().numpy(), What.cpu().numpy(), H_ref))
    # PSD up to rounding: the smallest eigenvalue is not below -1e-3 of the largest
    for k in range(cfg.g):
        ev = np.linalg.eigvalsh(H[k].cpu().numpy().astype(np.float64))
        assert ev.min() >= -1e-3 * ev.max()


@pytest.mark.parametrize("name,prefix", [("c1_7b_attn", 512), ("c2_7b_down", 128), ("c4_sweep", 160)])
def test_large_shapes_token_prefix(dev, name, prefix):
    """Full d_in / d_out of the large layers on a token prefix the oracle finishes in seconds."""
    cfg = synth.CONFIGS[name]
    for g in (cfg.groups if name == "c4_sweep" else cfg.groups[:1]):
        c = synth.LayerConfig(cfg.name, prefix, min(cfg.chunk, 200), cfg.d_in, cfg.d_out, (g,), cfg.x_kind,
                              cfg.outlier_frac, cfg.outlier_mult)
        xs, gs, ss, H, W, What, loss = run_layer(c, dev)
        xb = np.concatenate([synth.bf16_bits(x) for x in xs])
        gb = np.concatenate([synth.bf16_bits(x) for x in gs])
        s_ref = orc.saliency(gb, g)
        check_s(torch.cat(ss, dim=1), s_ref)
        H_ref = orc.hessian(xb, s_ref)
        check_H(H, H_ref)
        # objective through the token form (never forms the fp64 H product with all channels)
        delta = (W.double() - What.double()).cpu().numpy()
        z = orc.bf16_bits_to_f64(xb) @ delta.T                            # [n, d_out]
        m = cfg.d_out // g
        loss_ref = np.array([(s_ref[k][:, None] * z[:, k * m:(k + 1) * m] ** 2).sum() for k in range(g)])
        check_loss(loss[:g], loss_ref)
        check_loss(loss[g:], np.array([loss_ref.sum()]))
        del H, xs, gs, ss
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name,g,n_tokens,_unused", [
    ("c1_7b_attn", 4, None, None),      # the workload bench.py times, in full: 131072 tokens, 16 chunks
    ("c2_7b_down", 4, None, None),      # in full: 131072 tokens, d_in 11008 (H 1.9 GB)
    ("c3_70b_mlp", 2, 8192, None),      # full d_in 28672 (H 6.6 GB resident), two 4096-token chunks
    ("c4_sweep", 16, 32768, None),      # sixteen groups, two 16384-token chunks
    ("c4_sweep", 1, 32768, None),       # one group (units of two column tiles)
])
def test_full_shapes_sampled(dev, name, g, n_tokens, _unused):
    """The large configurations at full layer size, launched exactly as bench.py launches them.

    The oracle cannot form g x d_in^2 x n products in seconds, so it is run exactly on a sampled
    sub-problem: for ~48 sampled input features F it computes H_k[F][:, F] from the columns X[:, F] alone,
    which are the same entries of the full H_k; s is checked against the oracle on every chunk; the objective
    is checked with the weight error restricted to the sampled features (W_hat = W elsewhere), which needs
    only those entries of H."""
    base = synth.CONFIGS[name]
    cfg = synth.LayerConfig(base.name, base.n if n_tokens is None else n_tokens, base.chunk, base.d_in, base.d_out,
                            (g,), base.x_kind, base.outlier_frac, base.outlier_mult)
    xs, gs, ss, H, W, What, loss = run_layer(cfg, dev)
    rng = np.random.default_rng(0)
    syn = synth.LayerSynth(cfg, dev, seed=0)
    F = np.unique(np.concatenate([rng.choice(cfg.d_in, 40, replace=False), syn.outlier_features[:8].cpu().numpy()]))
    Ft = torch.from_numpy(F).to(dev)
    xb = np.concatenate([synth.bf16_bits(x[:, Ft].contiguous()) for x in xs])          # [n, |F|]
    # saliency: the oracle on every chunk of the gradient; the oracle's Hessian is built from the oracle's own
    # saliency throughout
    s_all = np.concatenate([orc.saliency(synth.bf16_bits(gc), g) for gc in gs], axis=1)
    check_s(torch.cat(ss, dim=1), s_all)
    H_ref = orc.hessian(xb, s_all)                                                     # [g, |F|, |F|]
    H_sub = H[:, Ft][:, :, Ft]
    check_H(H_sub, H_ref)
    Hc = H[g - 1, :2048, :2048].cpu()
    assert torch.equal(Hc, Hc.T)
    # objective: restrict to the sampled features by zeroing delta elsewhere (W_hat = W off F)
    mask = torch.zeros(cfg.d_in, dtype=torch.bool, device=dev)
    mask[Ft] = True
    What_f = torch.where(mask[None, :], What, W)
    ows = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(cfg.d_in, cfg.d_out, g), dev)
    loss_f = libgq.gq_objective(W, What_f, H, ows)
    libgq.gq_check()
    loss_ref = orc.objective(W[:, Ft].contiguous().cpu().numpy(), What[:, Ft].contiguous().cpu().numpy(), H_ref)
    check_loss(loss_f, loss_ref)
    assert np.all(loss.cpu().numpy() > 0)
    del xs, gs, ss, H, W, What, What_f, ows
    torch.cuda.empty_cache()


# ------------------------------------------------------------------------------------------ extreme sizes
def test_largest_feature_count(dev):
    """d_in = 65536, the largest the interface accepts (H is 17 GB, 32896 tiles): index arithmetic beyond 2^31
    elements.  The oracle is run on sampled features (which are the same entries of the full H), on the diagonal of
    all features, and the objective on a weight error confined to the sampled features."""
    d_in, n, g, d_out = 65536, 96, 1, 16
    gen = torch.Generator(device=dev).manual_seed(65536)
    X = (torch.randn(n, d_in, generator=gen, device=dev) * torch.exp(0.5 * torch.randn(d_in, generator=gen, device=dev)))
    X = X.to(torch.bfloat16)
    s = torch.rand(g, n, generator=gen, device=dev) + 0.1
    H = gpu_hessian([X], [s], d_in, g, dev)
    rng = np.random.default_rng(1)
    F = np.unique(np.concatenate([rng.choice(d_in, 60, replace=False), [0, 255, 256, 32767, 32768, 65280, 65535]]))
    Ft = torch.from_numpy(F).to(dev)
    s64 = s.cpu().numpy().astype(np.float64)
    H_ref = orc.hessian(synth.bf16_bits(X[:, Ft].contiguous()), s64)
    check_H(H[:, Ft][:, :, Ft], H_ref)
    diag = orc.hessian_diag(synth.bf16_bits(X), s64)
    d_gpu = torch.diagonal(H[0]).double().cpu().numpy()
    assert np.all(np.abs(d_gpu - diag[0]) <= H_ENTRY * diag[0] + 1e-30)
    corner = H[0, 65000:, 65000:].cpu()
    assert torch.equal(corner, corner.T)
    W = 0.02 * torch.randn(d_out, d_in, generator=gen, device=dev)
    What = W.clone()
    What[:, Ft] += 0.01 * torch.randn(d_out, len(F), generator=gen, device=dev)
    ows = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(d_in, d_out, g), dev)
    loss = libgq.gq_objective(W, What, H, ows)
    libgq.gq_check()
    loss_ref = orc.objective(W[:, Ft].contiguous().cpu().numpy(), What[:, Ft].contiguous().cpu().numpy(),
                             H[:, Ft][:, :, Ft].double().cpu().numpy())
    check_loss(loss, loss_ref)
    del H, X, W, What, ows
    torch.cuda.empty_cache()


def test_largest_group_count(dev):
    """g = 1024 groups of 8 channels, the most the interface accepts: 512 pairs of groups per tile."""
    n, d_in, g = 300, 264, 1024
    cfg = synth.LayerConfig("g1024", n, 128, d_in, 8 * g, (g,), "lognormal", 0.01, 20.0)
    xs, gs, ss, H, W, What, loss = run_layer(cfg, dev)
    xb = np.concatenate([synth.bf16_bits(x) for x in xs])
    gb = np.concatenate([synth.bf16_bits(x) for x in gs])
    s_ref = orc.saliency(gb, g)
    check_s(torch.cat(ss, dim=1), s_ref)
    H_ref = orc.hessian(xb, s_ref)
    check_H(H, H_ref)
    check_loss(loss, orc.objective(W.cpu().numpy(), What.cpu().numpy(), H_ref))


# ------------------------------------------------------------------------------------------ failure detection
def test_device_wait_timeout_is_reported_and_context_survives(dev):
    """A pipeline wait that runs out of its time budget makes the kernel return (no trap, no hang), the status
    word reports it once, and the library keeps working afterwards."""
    libgq.gq_check()
    libgq.gq_selftest_wait_timeout(20)
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_check()
    assert "GQ_ERR_TIMEOUT" in str(e.value)
    assert e.value.detail[1] == 99                        # the site id of the self-test wait
    libgq.gq_check()                                      # reported once, then clear
    grad = torch.ones((8, 16), dtype=torch.bfloat16, device=dev)
    s = libgq.gq_saliency(grad, 2)
    libgq.gq_check()
    assert torch.allclose(s, torch.ones_like(s))


def test_hessian_padded_rows_and_saliency_stride(dev):
    """ld_x > d_in and ld_s > n: views into wider buffers."""
    n, d_in, g = 200, 264, 3
    gen = torch.Generator(device=dev).manual_seed(9)
    Xw = torch.randn(n, d_in + 40, generator=gen, device=dev).to(torch.bfloat16)
    sw = torch.rand(g, n + 24, generator=gen, device=dev)
    X, s = Xw[:, :d_in], sw[:, :n]
    H = gpu_hessian([X], [s], d_in, g, dev)
    H_ref = orc.hessian(synth.bf16_bits(X.contiguous()), s.contiguous().cpu().numpy().astype(np.float64))
    check_H(H, H_ref)


# ------------------------------------------------------------------------------------------ host path
@pytest.mark.parametrize("d_out,g", [(256, 2), (1024, 128)])       # 129 fp64 results need more than 1 KiB
def test_host_pipeline_matches_device_calls(dev, d_out, g):
    cfg = synth.LayerConfig("host", 700, 256, 384, d_out, (g,), "lognormal", 0.01, 20.0)
    xs, gs, ss, H, W, What, loss = run_layer(cfg, dev)
    X_host = torch.cat(xs).cpu().pin_memory()
    grad_host = torch.cat(gs).cpu().pin_memory()
    arena = libgq.alloc_workspace(libgq.gq_layer_host_arena_bytes(cfg.chunk, cfg.d_in, cfg.d_out, cfg.g), dev)
    H_host = torch.empty((cfg.g, cfg.d_in, cfg.d_in), dtype=torch.float32).pin_memory()
    loss_host = libgq.gq_layer_objective_host(X_host, grad_host, cfg.chunk, cfg.g, 1.0, W.cpu(), What.cpu(), arena,
                                              H_host=H_host)
    # same kernels, same order; tiles that are cut along tokens are summed with atomics (last-bit freedom)
    assert torch.allclose(H_host, H.cpu(), rtol=1e-5, atol=1e-6 * H.abs().max().item())
    assert torch.allclose(loss_host, loss.cpu(), rtol=1e-6, atol=0.0)
