"""The N > 1 path on CPU: two gloo ranks shard a batch of independent images, each reduces its
share (here with the CPU oracle standing in for the device), and the job's throughput is
all units over the slowest rank's time.  No data-path collective exists to test: the shards are
disjoint and their union is the batch."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_08966_b200 import sharding, workloads


def test_shard_units_partitions_exactly():
    for n in (0, 1, 4, 16, 17, 31):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in sharding.shard_units(n, r, world)]
            assert got == list(range(n))
            sizes = [len(sharding.shard_units(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_units(4, 2, 2)
    assert sharding.rank_seed(1, 0) == 1 and sharding.rank_seed(1, 3) == 301


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from tests.helpers import oracle_image
        wl = workloads.batched(B=3, N=120, T=4, d=64, n_h=2, d_h=16)
        mine = sharding.shard_units(len(wl.images), rank, world)
        labels = {i: oracle_image(wl, wl.images[i])["label"] for i in mine}
        units = sum(wl.images[i].N for i in mine)
        secs = 0.5 if rank == 0 else 2.0                       # rank 1 is the slow one
        thr = sharding.job_throughput(units, secs)
        slow = sharding.max_over_ranks(secs)
        gathered = [None] * world
        dist.all_gather_object(gathered, {i: v.tolist() for i, v in labels.items()})
        if rank == 0:
            merged = {}
            for g in gathered:
                assert not (set(g) & set(merged))                  # disjoint shards
                merged.update(g)
            out.put((thr, slow, sorted(merged), {i: merged[i] for i in merged}))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_a_batch_without_collectives_on_the_data_path():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    thr, slow, ids, merged = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ids == [0, 1, 2] and slow == 2.0
    assert thr == pytest.approx(3 * 120 / 2.0)
    # the sharded result equals the unsharded one
    from tests.helpers import oracle_image
    wl = workloads.batched(B=3, N=120, T=4, d=64, n_h=2, d_h=16)
    for i, img in enumerate(wl.images):
        assert np.array_equal(np.array(merged[i]), oracle_image(wl, img)["label"])
