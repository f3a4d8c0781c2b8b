"""Multi-GPU layout of the path, exercised with two CPU ranks (gloo).

Rows are independent, so N GPUs take N row blocks, the partition tables are replicated and the data
path needs no collective; the only communication of the bench is the max-over-ranks of the timed
region. Here each rank runs the CPU oracle (standing in for its GPU) on its row block and rank 0
checks that the gathered results equal the single-process result, and that the reduction the bench
uses returns the slowest rank's time.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import synth
from paper_2605_29986_b200 import rows


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.make_workload(4, B=22, V=6000, K=300)      # mixed partitions, B not divisible by world
        cm, z = w.class_masks(0), w.logits(0)
        lo, hi = rows.shard_rows(w.B, rank, world)
        out = oracle.decode_step(w.partitions, w.row_part[lo:hi], cm[lo:hi], z[lo:hi].copy())
        mine = torch.from_numpy(np.stack([out["argmax"], out["rep"]], axis=1).astype(np.int64))
        sizes = [rows.shard_rows(w.B, r, world) for r in range(world)]
        gathered = [torch.empty((b - a, 2), dtype=torch.int64) for a, b in sizes]
        dist.all_gather(gathered, mine)
        slowest = rows.max_over_ranks(0.5 + rank, dist)
        if rank == 0:
            full = oracle.decode_step(w.partitions, w.row_part, cm, z.copy())
            got = torch.cat(gathered).numpy()
            assert np.array_equal(got[:, 0], full["argmax"]) and np.array_equal(got[:, 1], full["rep"])
            assert slowest == 0.5 + (world - 1)
            open(os.path.join(out_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_row_sharding_needs_no_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "ok").exists()


def test_shard_rows_partitions_the_batch():
    for B in (0, 1, 7, 32, 1000):
        for world in (1, 2, 3, 8):
            spans = [rows.shard_rows(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
