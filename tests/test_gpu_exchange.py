"""Token-sharded accumulation: gq_hessian_reduce_share / gq_hessian_gather_shares.

The exchange kernels read every rank's matrix through plain pointers, so all "ranks" can live in one address
space: the tests hold R matrices on one GPU and call the two steps for every rank in turn (no kernel waits
for another one), exactly the sequence R GPUs would run between their host barriers."""
import numpy as np
import pytest
import torch

from oracle import gq_oracle as orc
from paper_2505_07004_b200 import api as libgq
from paper_2505_07004_b200 import shard, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    return torch.device("cuda:0")


def run_exchange(Hs, d_in, g):
    for r in range(len(Hs)):
        libgq.gq_hessian_reduce_share(Hs, r, d_in, g)
    torch.cuda.synchronize()
    for r in range(len(Hs)):
        libgq.gq_hessian_gather_shares(Hs, r, d_in, g)
    torch.cuda.synchronize()
    libgq.gq_check()


@pytest.mark.parametrize("ranks,d_in,g", [(2, 264, 1), (3, 264, 3), (4, 1024, 2), (8, 520, 1), (16, 136, 2), (5, 8, 1)])
def test_exchange_is_the_rank_ordered_sum_of_the_upper_triangle(dev, ranks, d_in, g):
    gen = torch.Generator(device=dev).manual_seed(ranks * 1000 + d_in)
    orig = [torch.randn(g, d_in, d_in, device=dev, generator=gen) for _ in range(ranks)]
    Hs = [h.clone() for h in orig]
    run_exchange(Hs, d_in, g)
    want = orig[0].clone()
    for h in orig[1:]:
        want += h                                      # fp32, rank order: bit-exact expectation
    upper = torch.triu(torch.ones(d_in, d_in, dtype=torch.bool, device=dev))
    blk = torch.arange(d_in, device=dev) // 128
    below_blocks = blk[:, None] > blk[None, :]          # blocks strictly below the diagonal are never touched
    for r in range(ranks):
        assert torch.equal(Hs[r][:, upper], want[:, upper]), "rank %d: upper triangle is not the sum" % r
        assert torch.equal(Hs[r][:, below_blocks], orig[r][:, below_blocks])
        assert torch.equal(Hs[r][:, ~below_blocks], Hs[0][:, ~below_blocks])    # all ranks agree bit for bit


def test_token_sharded_accumulate_matches_unsharded_and_oracle(dev):
    cfg = synth.LayerConfig("x", 2048 + 512 + 37, 512, 264, 48, (3,), "lognormal", 0.02, 20.0)
    syn = synth.LayerSynth(cfg, dev, seed=5)
    g, d_in = 3, cfg.d_in
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, d_in, g), dev)
    s_buf = torch.empty((g, cfg.chunk), dtype=torch.float32, device=dev)

    def accumulate(H, chunks):
        for c in chunks:
            x, gr = syn.x_chunk(c), syn.grad_chunk(c)
            nt = x.shape[0]
            libgq.gq_saliency(gr, g, 1.0, s=s_buf[:, :nt])
            libgq.gq_hessian_accumulate(x, s_buf[:, :nt], H, ws, flags=libgq.GQ_HESSIAN_DETERMINISTIC)

    H_one = torch.zeros(g, d_in, d_in, device=dev)
    accumulate(H_one, range(cfg.n_chunks))
    libgq.gq_hessian_finalize(H_one)
    for world in (2, 3):
        Hs = [torch.zeros(g, d_in, d_in, device=dev) for _ in range(world)]
        seen = []
        for r in range(world):
            mine = shard.chunks_for_rank(cfg.n_chunks, r, world)
            seen += mine
            accumulate(Hs[r], mine)
        assert sorted(seen) == list(range(cfg.n_chunks))
        torch.cuda.synchronize()
        for r in range(world):                           # what every rank runs between its barriers
            libgq.gq_hessian_reduce_share(Hs, r, d_in, g)
        for r in range(world):
            libgq.gq_hessian_gather_shares(Hs, r, d_in, g)
        for r in range(world):
            libgq.gq_hessian_finalize(Hs[r])
        libgq.gq_check()
        for r in range(world):
            assert torch.equal(Hs[r], Hs[0])
            assert torch.allclose(Hs[r], H_one, rtol=1e-5, atol=1e-6 * float(H_one.abs().max()))
    # against the oracle (same tolerances as the unsharded path)
    xb = np.concatenate([synth.bf16_bits(syn.x_chunk(c).cpu()) for c in range(cfg.n_chunks)])
    gb = np.concatenate([synth.bf16_bits(syn.grad_chunk(c).cpu()) for c in range(cfg.n_chunks)])
    H_o = orc.hessian(xb, orc.saliency(gb, g, 1.0))
    H_g = Hs[1].cpu().numpy().astype(np.float64)
    for k in range(g):
        assert np.linalg.norm(H_g[k] - H_o[k]) <= 5e-3 * np.linalg.norm(H_o[k])
        assert np.abs(H_g[k] - H_o[k]).max() <= 1e-2 * np.abs(H_o[k]).max()


def test_exchange_single_rank_and_errors(dev):
    H = torch.randn(1, 64, 64, device=dev)
    before = H.clone()
    libgq.gq_hessian_reduce_share([H], 0, 64, 1)
    libgq.gq_hessian_gather_shares([H], 0, 64, 1)
    libgq.gq_check()
    assert torch.equal(H, before)
    # exchange_hessian with one rank only finalizes
    shard.exchange_hessian(H, [H], 0)
    assert torch.equal(H, torch.triu(before) + torch.triu(before, 1).transpose(1, 2))
    with pytest.raises(libgq.GQError) as e:
        libgq.gq_hessian_reduce_share([H] * 17, 0, 64, 1)
    assert "GQ_ERR_INVALID_ARG" in str(e.value)
    with pytest.raises(libgq.GQError):
        libgq.gq_hessian_gather_shares([H, H], 2, 64, 1)
    with pytest.raises(libgq.GQError):
        libgq.gq_hessian_reduce_share([H, 0], 0, 64, 1)
