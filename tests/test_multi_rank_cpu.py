"""The N>1 path on CPU: two gloo ranks shard a batch, each convolves its own images with the
oracle standing in for the device kernel, and only the timing is reduced over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_1909_05073_b200 import shard, synth


def test_shard_range_partitions_exactly():
    for n in (0, 1, 7, 64, 257):
        for world in (1, 2, 3, 8):
            spans = [shard.shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = synth.LayerSpec("t", 6, 8, 9, 9, 1, 0.5)
    w, b, _ = synth.gen_weights(spec, 3)
    x = synth.gen_input(spec, 5, 3)                       # the whole batch, same on every rank
    lo, hi = shard.shard_range(x.shape[0], rank, world)
    y = oracle.conv3x3(x[lo:hi], w, b, 1, True)           # no exchange with the other rank
    np.save(os.path.join(out_dir, "y%d.npy" % rank), y)
    t = shard.max_over_ranks([1.0 + rank, 5.0 - rank])    # max over ranks of two "timings"
    assert t == [float(world), 5.0]
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_the_batch(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    spec = synth.LayerSpec("t", 6, 8, 9, 9, 1, 0.5)
    w, b, _ = synth.gen_weights(spec, 3)
    x = synth.gen_input(spec, 5, 3)
    whole = oracle.conv3x3(x, w, b, 1, True)
    parts = np.concatenate([np.load(tmp_path / ("y%d.npy" % r)) for r in range(2)])
    assert np.array_equal(parts, whole)
