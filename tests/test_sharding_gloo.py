"""The N > 1 host logic on CPU: two gloo ranks take disjoint batches of the seeded position stream,
together covering what one rank would generate, and timings reduce to the maximum over ranks."""
import hashlib
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import importlib.util
    spec = importlib.util.spec_from_file_location(
        "az_sharding", os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                                    "paper_2609_37447_b200", "sharding.py"))
    sharding = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(sharding)
    from inputs import configs, positions

    cfg = configs.CONFIGS["c3"]
    B = 48
    rec = positions.for_config(cfg, B, first_index=sharding.rank_first_index(rank, B))
    digest = hashlib.sha256(rec.tobytes()).digest()
    gathered = [None] * world
    dist.all_gather_object(gathered, digest)
    whole = positions.for_config(cfg, B * world)
    expect = [hashlib.sha256(whole[r * B:(r + 1) * B].tobytes()).digest() for r in range(world)]
    assert gathered == expect                                  # disjoint, ordered, and covering
    # the search workloads shard their games the same way: every rank's roots (records with the last eight moves)
    # are its own stretch of the one seeded stream
    from inputs import pnet_weights
    pcfg = pnet_weights.PNET_CONFIGS["p14"]
    games = 24
    roots = positions.generate_moves(pcfg.position_seed, games, pcfg.plies, first_index=sharding.rank_first_index(rank, games))[0]
    gathered = [None] * world
    dist.all_gather_object(gathered, hashlib.sha256(roots.tobytes()).digest())
    all_roots = positions.generate_moves(pcfg.position_seed, games * world, pcfg.plies)[0]
    assert gathered == [hashlib.sha256(all_roots[r * games:(r + 1) * games].tobytes()).digest() for r in range(world)]
    # strong-scaling split: contiguous, disjoint, covering, sizes differ by at most one
    ranges = [sharding.split_batch(101, r, world) for r in range(world)]
    assert ranges[0][0] == 0 and ranges[-1][1] == 101
    assert all(ranges[i][1] == ranges[i + 1][0] for i in range(world - 1))
    assert max(e - b for b, e in ranges) - min(e - b for b, e in ranges) <= 1
    # timing reduction: every rank sees the slowest rank's figure
    sharding.barrier()
    got = sharding.max_over_ranks([1.0 + rank, 10.0 - rank])
    assert got == [float(world), 10.0]
    np.save(os.path.join(out_dir, f"ok{rank}.npy"), np.array(got))
    dist.destroy_process_group()


def test_two_ranks_shard_the_stream_and_reduce_timings(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert np.load(tmp_path / f"ok{r}.npy").tolist() == [2.0, 10.0]
