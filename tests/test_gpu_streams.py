"""The library enqueues on the caller's stream and allocates nothing: the whole path runs on a side stream and
inside a captured CUDA graph, with the same bits as on the default stream."""
import pytest
import torch

from paper_2505_07004_b200 import api as libgq
from paper_2505_07004_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    return torch.device("cuda:0")


def make(dev):
    cfg = synth.LayerConfig("s", 1024 + 200, 512, 520, 64, (2,), "lognormal", 0.02, 20.0)
    syn = synth.LayerSynth(cfg, dev, seed=11)
    xs = [syn.x_chunk(c) for c in range(cfg.n_chunks)]
    gs = [syn.grad_chunk(c) for c in range(cfg.n_chunks)]
    W, What = syn.weights()
    return cfg, xs, gs, W, What


def run_path(cfg, xs, gs, W, What, bufs):
    H, s_buf, ws, ows, loss = bufs
    g = cfg.g
    H.zero_()
    for x, gr in zip(xs, gs):
        nt = x.shape[0]
        libgq.gq_saliency_prepared(gr, g, ws, 1.0, s=s_buf[:, :nt])
        libgq.gq_hessian_accumulate(x, s_buf[:, :nt], H, ws,
                                    flags=libgq.GQ_HESSIAN_DETERMINISTIC | libgq.GQ_HESSIAN_S_PREPARED)
    libgq.gq_hessian_finalize(H)
    libgq.gq_objective(W, What, H, ows, loss=loss)


def buffers(cfg, dev):
    g = cfg.g
    return (torch.empty(g, cfg.d_in, cfg.d_in, device=dev), torch.empty(g, cfg.chunk, device=dev),
            libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev),
            libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(cfg.d_in, cfg.d_out, g), dev),
            torch.empty(g + 1, dtype=torch.float64, device=dev))


def test_side_stream_and_graph_replay_match_the_default_stream(dev):
    cfg, xs, gs, W, What = make(dev)
    ref = buffers(cfg, dev)
    run_path(cfg, xs, gs, W, What, ref)
    torch.cuda.synchronize()
    libgq.gq_check()

    side = torch.cuda.Stream()
    b1 = buffers(cfg, dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run_path(cfg, xs, gs, W, What, b1)
    side.synchronize()
    libgq.gq_check()
    assert torch.equal(b1[0], ref[0]) and torch.equal(b1[4], ref[4])

    b2 = buffers(cfg, dev)
    graph = torch.cuda.CUDAGraph()
    launches0 = libgq.gq_launch_count()
    with torch.cuda.graph(graph):
        run_path(cfg, xs, gs, W, What, b2)
    per_step = libgq.gq_launch_count() - launches0
    assert per_step == 2 * cfg.n_chunks + 5          # saliency, Hessian per chunk; mirror, maximum, fp16, dot, reduce
    for _ in range(2):
        b2[0].fill_(7.0)
        b2[4].zero_()
        graph.replay()
    torch.cuda.synchronize()
    libgq.gq_check()
    assert torch.equal(b2[0], ref[0]) and torch.equal(b2[4], ref[4])


def run_path_ahead(cfg, xs, gs, W, What, bufs, extra):
    """The same path with one launch per chunk: the saliency of chunk c + 1 is computed inside the Hessian launch
    of chunk c (two saliency buffers and scratch blocks in turn)."""
    H, s_buf, ws, ows, loss = bufs
    sb, wb = (s_buf, extra[0]), (ws, extra[1])
    g = cfg.g
    flags = libgq.GQ_HESSIAN_DETERMINISTIC | libgq.GQ_HESSIAN_S_PREPARED
    H.zero_()
    libgq.gq_saliency_prepared(gs[0], g, wb[0], 1.0, s=sb[0][:, :gs[0].shape[0]])
    for c, x in enumerate(xs):
        nt = x.shape[0]
        if c + 1 < len(xs):
            libgq.gq_hessian_accumulate_ahead(x, sb[c & 1][:, :nt], H, wb[c & 1], gs[c + 1], wb[(c + 1) & 1], 1.0,
                                              sb[(c + 1) & 1][:, :gs[c + 1].shape[0]], flags=flags)
        else:
            libgq.gq_hessian_accumulate(x, sb[c & 1][:, :nt], H, wb[c & 1], flags=flags)
    libgq.gq_hessian_finalize(H)
    libgq.gq_objective(W, What, H, ows, loss=loss)


def test_one_launch_per_chunk_in_a_graph_gives_the_same_bits(dev):
    cfg, xs, gs, W, What = make(dev)
    assert cfg.n_chunks >= 3
    ref = buffers(cfg, dev)
    run_path(cfg, xs, gs, W, What, ref)
    torch.cuda.synchronize()
    b = buffers(cfg, dev)
    extra = (torch.empty_like(b[1]), libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, cfg.g), dev))
    graph = torch.cuda.CUDAGraph()
    launches0 = libgq.gq_launch_count()
    with torch.cuda.graph(graph):
        run_path_ahead(cfg, xs, gs, W, What, b, extra)
    assert libgq.gq_launch_count() - launches0 == cfg.n_chunks + 1 + 5
    for _ in range(2):
        b[0].fill_(7.0)
        b[4].zero_()
        graph.replay()
    torch.cuda.synchronize()
    libgq.gq_check()
    assert torch.equal(b[0], ref[0]) and torch.equal(b[4], ref[4])
