"""The N > 1 path on CPU: two gloo ranks split a frame list, each produces the rows of its own
shard (a function of the frame index stands in for the per-rank GPU forward), and the plumbing
(contiguous shards, max over ranks of the timings, gathering the rows in frame order) is checked
against the unsharded result."""
import os
import socket

import numpy as np
import pytest

from paper_2507_14959_b200 import shard


def test_shard_range_partitions():
    for n in (0, 1, 7, 16, 256, 257):
        for world in (1, 2, 3, 8):
            cuts = [shard.shard_range(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            for (b0, e0), (b1, e1) in zip(cuts, cuts[1:]):
                assert e0 == b1
            sizes = [e - b for b, e in cuts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.shard_range(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, n_total, out_dir):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b, e = shard.shard_range(n_total, rank, world)
        # stand-in for this rank's forward: row f of the result depends only on the frame index
        local = torch.tensor([[f, 10.0 * f + 1.0, -f] for f in range(b, e)], dtype=torch.float32).reshape(e - b, 3)
        rows = shard.gather_rows(local, n_total)
        ms, ms_e2e = shard.max_over_ranks([10.0 + rank, 5.0 - rank])
        np.save(os.path.join(out_dir, f"rows{rank}.npy"), rows.numpy())
        np.save(os.path.join(out_dir, f"t{rank}.npy"), np.asarray([ms, ms_e2e]))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n_total", [5, 8])
def test_two_gloo_ranks_shard_and_gather(tmp_path, n_total):
    import torch.multiprocessing as mp
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), n_total, str(tmp_path)), nprocs=world, join=True)
    want = np.asarray([[f, 10.0 * f + 1.0, -f] for f in range(n_total)], dtype=np.float32)
    for r in range(world):
        np.testing.assert_array_equal(np.load(tmp_path / f"rows{r}.npy"), want)
        np.testing.assert_array_equal(np.load(tmp_path / f"t{r}.npy"), [11.0, 5.0])


def test_single_process_is_identity():
    import torch
    x = torch.arange(6.0).reshape(3, 2)
    assert shard.gather_rows(x, 3) is x
    assert shard.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
