"""World-size-2 checks on CPU (gloo) of the multi-GPU path's host logic: row-slab sharding
needs no collective on the data path, and the timing reduction takes the max over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2202_03293_b200 import inputs, sharding


def test_row_slabs_partition_exactly():
    for extent in (0, 1, 7, 128, 1001):
        for world in (1, 2, 3, 8):
            slabs = [sharding.row_slab(extent, r, world) for r in range(world)]
            assert slabs[0][0] == 0 and slabs[-1][1] == extent
            assert all(a[1] == b[0] for a, b in zip(slabs, slabs[1:]))
            sizes = [e - b for b, e in slabs]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import ref
        seed = inputs.BASE_SEED
        a = inputs.uniform((37, 19), seed, 1)
        b = inputs.uniform((19, 11), seed, 2)
        m0, m1 = sharding.row_slab(37, rank, world)
        part, _ = ref.matmul(a[m0:m1], b, threads=1)       # each rank: its slab of A, all of B
        np.save(os.path.join(out_dir, f"part{rank}.npy"), part)
        # conv: shard the batch iterator
        i = inputs.uniform((5, 9, 3), seed, 3)
        k = inputs.uniform((2, 3, 4), seed, 4)
        n0, n1 = sharding.row_slab(5, rank, world)
        cpart, _ = ref.conv1d_nwc_wcf(i[n0:n1], k, threads=1)
        np.save(os.path.join(out_dir, f"cpart{rank}.npy"), cpart)
        t = sharding.max_over_ranks(1.0 + rank)
        assert t == float(world)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_stitch_to_the_whole(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    from oracle import ref
    seed = inputs.BASE_SEED
    a = inputs.uniform((37, 19), seed, 1)
    b = inputs.uniform((19, 11), seed, 2)
    whole, _ = ref.matmul(a, b)
    parts = np.concatenate([np.load(tmp_path / f"part{r}.npy") for r in range(2)])
    assert np.array_equal(parts, whole)
    i = inputs.uniform((5, 9, 3), seed, 3)
    k = inputs.uniform((2, 3, 4), seed, 4)
    cwhole, _ = ref.conv1d_nwc_wcf(i, k)
    cparts = np.concatenate([np.load(tmp_path / f"cpart{r}.npy") for r in range(2)])
    assert np.array_equal(cparts, cwhole)
