"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, one synthetic layer each, max-over-ranks timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_07004_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = synth.LayerConfig("t", 64, 64, 32, 16, (2,), "lognormal", 0.05, 20.0)
        syn = synth.LayerSynth(cfg, "cpu", seed=shard.layer_seed_for_rank(0, rank))
        checksum = float(syn.x_chunk(0).float().abs().sum())
        times = shard.max_over_ranks([10.0 + rank, 5.0 - rank])
        sums = shard.gather_scalars(checksum)
        value = shard.whole_job_throughput(cfg.n, 3, times[0], world)
        torch.save({"times": times, "sums": sums, "value": value}, os.path.join(out_dir, "r%d.pt" % rank))
    finally:
        dist.destroy_process_group()


def test_two_rank_timing_reduction_and_distinct_layers(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(os.path.join(tmp_path, "r%d.pt" % i)) for i in range(world)]
    for i in range(world):
        assert r[i]["times"] == [11.0, 5.0]                  # element-wise max over ranks
        assert r[i]["value"] == 64 * 2 * 3 / 11.0            # whole-job units / slowest rank
        assert r[i]["sums"] == r[0]["sums"]
    assert r[0]["sums"][0] != r[0]["sums"][1]                # each rank drew its own layer


def test_single_process_fallbacks():
    assert shard.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert shard.gather_scalars(3.0) == [3.0]


def _token_worker(rank, world, port, out_dir):
    """Token sharding of one layer: every rank sums the oracle's partial Hessians of its chunks; adding the
    partial matrices over the ranks (here: gloo all-reduce, on the GPUs: the library's exchange kernels) must
    give the Hessian of all tokens."""
    import numpy as np
    from oracle import gq_oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = synth.LayerConfig("t", 5 * 32 + 7, 32, 24, 16, (2,), "lognormal", 0.05, 20.0)
        syn = synth.LayerSynth(cfg, "cpu", seed=3)                      # the same layer on every rank
        H = np.zeros((2, cfg.d_in, cfg.d_in))
        mine = shard.chunks_for_rank(cfg.n_chunks, rank, world)
        for c in mine:
            xb, gb = synth.bf16_bits(syn.x_chunk(c)), synth.bf16_bits(syn.grad_chunk(c))
            orc.hessian(xb, orc.saliency(gb, 2, 1.0), H)
        t = torch.from_numpy(H)
        dist.all_reduce(t)
        torch.save({"H": t, "mine": mine}, os.path.join(out_dir, "t%d.pt" % rank))
    finally:
        dist.destroy_process_group()


def test_two_rank_token_sharding_adds_up(tmp_path):
    import numpy as np
    from oracle import gq_oracle as orc
    world, port = 2, _free_port()
    mp.spawn(_token_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(os.path.join(tmp_path, "t%d.pt" % i)) for i in range(world)]
    assert sorted(r[0]["mine"] + r[1]["mine"]) == list(range(6))
    cfg = synth.LayerConfig("t", 5 * 32 + 7, 32, 24, 16, (2,), "lognormal", 0.05, 20.0)
    syn = synth.LayerSynth(cfg, "cpu", seed=3)
    xb = np.concatenate([synth.bf16_bits(syn.x_chunk(c)) for c in range(cfg.n_chunks)])
    gb = np.concatenate([synth.bf16_bits(syn.grad_chunk(c)) for c in range(cfg.n_chunks)])
    H_all = orc.hessian(xb, orc.saliency(gb, 2, 1.0))
    for i in range(world):
        assert np.allclose(r[i]["H"].numpy(), H_all, rtol=1e-12, atol=1e-14 * np.abs(H_all).max())


def test_chunks_for_rank_partitions():
    for n_chunks in (0, 1, 5, 16):
        for world in (1, 2, 3, 8):
            got = sorted(c for r in range(world) for c in shard.chunks_for_rank(n_chunks, r, world))
            assert got == list(range(n_chunks))


class _CpuExchangeOps:
    """CPU stand-ins for the three library calls exchange_hessian makes.  The ranks are separate processes without
    shared memory, so "reading a peer's matrix" is an all-gather here; shares are row ranges.  What is under test
    is exchange_hessian's own sequence: reduce only after every partial matrix is complete, gather only after
    every share is reduced, finalize last."""

    def __init__(self, H, world):
        self.H, self.world, self.log = H, world, []

    def _all(self):
        mats = [torch.empty_like(self.H) for _ in range(self.world)]
        dist.all_gather(mats, self.H)
        return mats

    def _rows(self, r):
        d = self.H.shape[1]
        return slice(d * r // self.world, d * (r + 1) // self.world)

    def gq_hessian_reduce_share(self, ptrs, rank, d_in, g):
        self.log.append("reduce")
        mats = self._all()
        acc = torch.zeros_like(self.H[:, self._rows(rank)])
        for m in mats:                                   # rank order: the same bits on whichever rank adds them
            acc += m[:, self._rows(rank)]
        self.H[:, self._rows(rank)] = acc

    def gq_hessian_gather_shares(self, ptrs, rank, d_in, g):
        self.log.append("gather")
        mats = self._all()
        for r in range(self.world):
            if r != rank:
                self.H[:, self._rows(r)] = mats[r][:, self._rows(r)]

    def gq_hessian_finalize(self, H):
        self.log.append("finalize")
        up = torch.triu(H)
        H.copy_(up + torch.triu(H, 1).transpose(1, 2))


def _exchange_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        gen = torch.Generator().manual_seed(100 + rank)
        H = torch.triu(torch.randn(2, 12, 12, generator=gen, dtype=torch.float64))      # this rank's partial sums
        partial = H.clone()
        ops = _CpuExchangeOps(H, world)
        shard.exchange_hessian(H, [None] * world, rank, ops=ops)
        torch.save({"H": H, "partial": partial, "log": ops.log}, os.path.join(out_dir, "x%d.pt" % rank))
    finally:
        dist.destroy_process_group()


def test_exchange_hessian_sequence_with_cpu_stand_ins(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_exchange_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(os.path.join(tmp_path, "x%d.pt" % i)) for i in range(world)]
    total = r[0]["partial"] + r[1]["partial"]
    expect = total + torch.triu(total, 1).transpose(1, 2)
    for i in range(world):
        assert r[i]["log"] == ["reduce", "gather", "finalize"]
        assert torch.equal(r[i]["H"], expect)                       # every rank ends with the same full matrix
    # one rank: no exchange, only finalize
    H = torch.triu(torch.randn(1, 6, 6, dtype=torch.float64))
    ops = _CpuExchangeOps(H, 1)
    shard.exchange_hessian(H, [None], 0, ops=ops)
    assert ops.log == ["finalize"] and torch.equal(H, H.transpose(1, 2))
    assert shard.exchange_bytes_per_rank(4096, 4, 8) == 2 * (4 * 32 * 33 // 2 * 7 // 8) * 128 * 128 * 4
