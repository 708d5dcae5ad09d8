"""The N > 1 path of the benchmark on CPU: two gloo ranks shard the id space, time a step each,
and agree on the slowest time and the whole-job rate.  (The codec itself never communicates.)"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from fixtures import replicas, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        base = synth.Boundary("shard", 8, 2, 4, 64, "fp16", 4, 64, 2, "normal", 0.02, seed=11)
        cfg = replicas.shard_for_rank(base, rank, world)
        act = synth.activation(cfg, [0, 1], 1)
        dist.barrier()
        my_ms = 10.0 * (rank + 1)                     # rank 1 is the slow one
        slowest = replicas.max_over_ranks(my_ms, dist)
        rate = replicas.whole_job_rate(1000.0, world, slowest)
        gathered = [None] * world
        dist.all_gather_object(gathered, (cfg.stream, slowest, rate,
                                          act.view(torch.int16).numpy().tobytes(),
                                          replicas.global_sample_id(cfg, rank, 3)))
        if rank == 0:
            np.save(os.path.join(out_dir, "ok.npy"), np.array([1]))
            streams = [g[0] for g in gathered]
            assert streams == [base.stream + r for r in range(world)]
            assert all(g[1] == 10.0 * world for g in gathered)          # everyone sees the slowest rank
            assert all(abs(g[2] - world * 1000.0 / (10.0 * world * 1e-3)) < 1e-6 for g in gathered)
            assert gathered[0][3] != gathered[1][3]                       # shards hold different activations
            assert [g[4] for g in gathered] == [3, 8 + 3]                 # disjoint global ids
            np.save(os.path.join(out_dir, "checked.npy"), np.array([1]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_ids_and_agree_on_the_slowest_time(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "checked.npy").exists()


def test_single_process_is_the_identity():
    base = synth.GPT2_XL
    assert replicas.shard_for_rank(base, 0, 1) == base
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(10.0, 1, 1000.0) == 10.0
