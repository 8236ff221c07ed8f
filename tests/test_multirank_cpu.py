"""Data-parallel form of the path on CPU ranks (gloo, world size 2): the batch is split over
tokens, every rank runs the whole path on its shard against replicated factors and weights, and
the gathered outputs equal the single-process result bit for bit.  No collective sits on the data
path; the only communication is the gather the test itself uses to compare."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import singlequant_oracle as ora
from paper_2511_22316_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.TINY
    X, W = wl.make_layer(w)
    # the factors come from one calibration pass over the whole batch and are replicated
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    start, count = wl.shard_rows(w.M, world, rank)
    Y = ora.linear(X[start:start + count], W, R1, R2)
    sizes = [wl.shard_rows(w.M, world, r)[1] for r in range(world)]
    parts = [torch.empty((c, w.N), dtype=torch.float16) for c in sizes]
    dist.all_gather(parts, torch.from_numpy(Y.astype(np.float16)))
    # timing is reduced the way the benchmark does it: maximum over ranks
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        np.save(os.path.join(out_dir, "gathered.npy"), torch.cat(parts).numpy())
        np.save(os.path.join(out_dir, "tmax.npy"), t.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_shard_rows_partitions_the_batch():
    for M in (0, 1, 7, 64, 2048):
        for world in (1, 2, 3, 8):
            spans = [wl.shard_rows(M, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == M
            for (s0, c0), (s1, _) in zip(spans, spans[1:]):
                assert s0 + c0 == s1
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def test_token_sharded_ranks_reproduce_the_single_process_result(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = wl.TINY
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    full = ora.linear(X, W, R1, R2).astype(np.float16)
    got = np.load(tmp_path / "gathered.npy")
    assert np.array_equal(got.view(np.uint16), full.view(np.uint16))
    assert np.load(tmp_path / "tmax.npy")[0] == 2.0
