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
