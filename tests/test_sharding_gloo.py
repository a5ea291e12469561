"""The multi-rank form of the path on CPU: two gloo ranks split the boxes with
box_shard, bound their slices, and gather.  The float64 oracle stands in for
the per-rank bounding call (test infrastructure), so what is checked here is
the host logic: the partition, the gather, and that slices are independent."""
import os
import socket

import numpy as np
import pytest

from paper_2507_20055_b200 import sharding
from paper_2507_20055_b200 import workloads as wl


def test_box_shard_partitions_every_batch():
    for batch in range(0, 40):
        for world in range(1, 9):
            spans = [sharding.box_shard(batch, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == batch
            for (a0, b0), (a1, b1) in zip(spans, spans[1:]):
                assert b0 == a1
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
            assert sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        sharding.box_shard(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, batch, out_dir):
    import torch
    import torch.distributed as dist
    from oracle import deeppoly_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.small_fc([12, 20, 16, 5], batch=batch, eps=0.05, seed=91)
        mine = sharding.shard_centers(w.centers, rank, world)
        n_total = sum(l.n_out for l in w.layers)
        if mine.shape[0] > 0:
            r = orc.deeppoly(w.layers, mine, w.eps, w.clip_lo, w.clip_hi, n_threads=1)
            lb, ub = torch.from_numpy(r["lb"]), torch.from_numpy(r["ub"])
        else:
            lb = torch.zeros((0, n_total), dtype=torch.float64)
            ub = torch.zeros((0, n_total), dtype=torch.float64)
        full_lb, full_ub = sharding.gather_bounds(lb, ub, batch)
        np.save(os.path.join(out_dir, f"lb_{rank}.npy"), full_lb.numpy())
        np.save(os.path.join(out_dir, f"ub_{rank}.npy"), full_ub.numpy())
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("batch", [5, 4, 1])
def test_two_ranks_match_the_unsharded_result(batch, tmp_path):
    import torch.multiprocessing as mp
    from oracle import deeppoly_oracle as orc
    orc.build()
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), batch, str(tmp_path)), nprocs=world, join=True)
    w = wl.small_fc([12, 20, 16, 5], batch=batch, eps=0.05, seed=91)
    ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, n_threads=1)
    for rank in range(world):
        lb = np.load(tmp_path / f"lb_{rank}.npy")
        ub = np.load(tmp_path / f"ub_{rank}.npy")
        assert lb.shape == ref["lb"].shape
        np.testing.assert_array_equal(lb, ref["lb"])
        np.testing.assert_array_equal(ub, ref["ub"])
