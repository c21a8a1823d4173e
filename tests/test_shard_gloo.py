"""The N > 1 path on CPU: two gloo ranks shard independent units, compress them with the
oracle (standing in for a GPU each), and the bookkeeping reduces to the slowest rank."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_04704_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import lagkv_oracle
        lagkv_oracle.set_threads(1)
        B, H, D, S, sink, L, k = 3, 2, 16, 4 + 5 * 8 + 3, 4, 8, 2
        K, V = synth.make_kv(B, H, S, D, seed=5)                 # the same full cache on every rank
        Kb, Vb = synth.to_bits(K).reshape(B * H, 1, S, D), synth.to_bits(V).reshape(B * H, 1, S, D)
        mine = shard.shard_units(B * H, rank, world)
        res = lagkv_oracle.compress(Kb[mine.start:mine.stop], Vb[mine.start:mine.stop], sink, L, k)
        np.save(os.path.join(out_dir, f"idx{rank}.npy"), res["idx"])
        slow = shard.max_over_ranks(10.0 * (rank + 1))
        assert slow == 10.0 * world
        assert shard.job_throughput(100, world, slow) == pytest.approx(world * 100 / (slow * 1e-3))
        assert shard.rank_seed(7, rank) != shard.rank_seed(7, (rank + 1) % world)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_units_without_data_collective(tmp_path, oracle):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    B, H, D, S, sink, L, k = 3, 2, 16, 4 + 5 * 8 + 3, 4, 8, 2
    K, V = synth.make_kv(B, H, S, D, seed=5)
    whole = oracle.compress(synth.to_bits(K).reshape(B * H, 1, S, D), synth.to_bits(V).reshape(B * H, 1, S, D), sink, L, k)
    parts = np.concatenate([np.load(tmp_path / f"idx{r}.npy") for r in range(world)], axis=0)
    np.testing.assert_array_equal(parts, whole["idx"])           # shards reassemble to the one-rank result


def test_shard_units_cover_everything_once():
    for total in (1, 7, 256, 1792):
        for world in (1, 2, 3, 8):
            got = [u for r in range(world) for u in shard.shard_units(total, r, world)]
            assert got == list(range(total))
            sizes = [len(shard.shard_units(total, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_max_over_ranks_without_process_group():
    assert shard.max_over_ranks(3.5) == 3.5
