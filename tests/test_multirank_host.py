"""The multi-GPU arm of the benchmark shards tokens across ranks with replicated weights and no
data-path collective; the only exchange is the max-over-ranks of the measured times.  These tests
run that host logic as two gloo ranks on CPU."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
import synth_inputs as si


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # each rank times its own steps; the job's time is the slowest rank's
        local = [10.0 + 5.0 * rank, 7.0 - rank]
        reduced = bench.reduce_max(local, torch.device("cpu"), world)
        # each rank draws its own activations, all ranks the same weights
        wl = si.single_layer_small()
        x = si.make_activations(bench.rank_seed(si.DEFAULT_SEED, rank), "layer_in", 8, 16)
        w = si.make_weight(si.DEFAULT_SEED, si.LinearSpec("w", 16, 16, False, 2.0, 4))
        gathered_x = [torch.zeros(8 * 16, dtype=torch.int32) for _ in range(world)]
        gathered_w = [torch.zeros(16 * 16, dtype=torch.int32) for _ in range(world)]
        dist.all_gather(gathered_x, torch.from_numpy(x.astype(np.int32).ravel()))
        dist.all_gather(gathered_w, torch.from_numpy(w.astype(np.int32).ravel()))
        out.put((rank, reduced, bool(torch.equal(gathered_x[0], gathered_x[1])), bool(torch.equal(gathered_w[0], gathered_w[1])), wl.tokens))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_times_and_shard_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, reduced, same_x, same_w, tokens in results:
        assert reduced == [15.0, 7.0]          # element-wise max over the two ranks
        assert not same_x and same_w           # different token batches, replicated weights
        assert tokens == 128


def test_job_throughput_is_aggregate_over_ranks():
    one = bench.job_throughput(1, 19_327_352_832, 10, 1.0)
    assert bench.job_throughput(8, 19_327_352_832, 10, 1.0) == 8 * one
    assert abs(one - 193.27352832) < 1e-9      # 19.33 GFLOP x 10 steps in 1 ms
    assert bench.reduce_max([3.0, 4.0], None, 1) == [3.0, 4.0]
