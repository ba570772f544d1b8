"""The multi-GPU plumbing on CPU: two gloo ranks shard a batch by rows, each compacts its own
mask (the CPU compaction standing in for the device call), and the bookkeeping that crosses ranks
(slowest time, totals, count offsets) is checked against the unsharded result."""
import os
import socket

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_17307_b200 import sharding


def test_rank_rows_partition():
    for n in (0, 1, 2, 7, 64, 65, 1000):
        for world in (1, 2, 3, 8):
            spans = [sharding.rank_rows(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        sharding.rank_rows(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, mask, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        b, e = sharding.rank_rows(mask.size, rank, world)
        idx, cnt = oracle.compact(mask[b:e])
        counts = sharding.gather_counts(cnt, dist)
        offset = sum(counts[:rank])
        glob = sharding.global_index(idx, b)
        ms, units, launches = sharding.reduce_step_stats(10.0 + rank, float(e - b), 3 + rank, dist)
        np.savez(os.path.join(out_dir, "r%d.npz" % rank), glob=glob, offset=offset, counts=np.array(counts),
                 ms=ms, units=units, launches=launches)
    finally:
        dist.destroy_process_group()


def test_two_ranks_row_sharding(tmp_path, oracle):
    import rstitch_inputs as gen
    world = 2
    mask = gen.random_mask(65, 0.4, seed=11)
    mp.spawn(_worker, args=(world, _free_port(), mask, str(tmp_path)), nprocs=world, join=True)
    ref_idx, ref_cnt = oracle.compact(mask)
    parts = [np.load(os.path.join(tmp_path, "r%d.npz" % r)) for r in range(world)]
    merged = np.full(ref_cnt, -1, dtype=np.int64)
    for p in parts:
        merged[int(p["offset"]):int(p["offset"]) + p["glob"].size] = p["glob"]
        assert p["counts"].sum() == ref_cnt
        assert float(p["ms"]) == 11.0 and float(p["units"]) == 65.0 and int(p["launches"]) == 7
    assert np.array_equal(merged, ref_idx)


def test_single_process_passthrough():
    assert sharding.reduce_step_stats(1.5, 4, 2) == (1.5, 4.0, 2)
    assert sharding.gather_counts(5) == [5]
