"""The vocabulary-parallel head's plumbing on CPU: shard bounds, the all-gather of the per-row statistics
between two gloo ranks (the fp64 oracle standing in for the head kernels, the merge written out here in
fp64), and the result against the oracle on the whole vocabulary."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_17307_b200 import sharding


def test_vocab_shard_partition():
    for V in (2, 17, 1000, 151936, 152064):
        for world in (1, 2, 3, 8):
            sh = [sharding.vocab_shard(V, r, world) for r in range(world)]
            assert sh[0][0] == 0 and sh[-1][1] == V
            for a, b in zip(sh, sh[1:]):
                assert a[1] == b[0] and (a[0] % 16 == 0 or a[0] == V)
            sizes = [e - b for b, e in sh]
            assert all(s >= 0 for s in sizes) and max(sizes) - min(sizes) < 32
    with pytest.raises(ValueError):
        sharding.vocab_shard(100, 3, 3)


def _stats_words(z, v_base):
    """(m, s, u, best, index) of one shard's logits as the five 32-bit words a shard emits."""
    m = z.max()
    e = np.exp(z - m)
    f = np.array([m, e.sum(), (e * (z - m)).sum(), m], dtype=np.float32)
    return np.concatenate([f.view(np.int32), np.array([int(np.argmax(z)) + v_base], dtype=np.int32)])


def _merge(words):
    """fp64 merge of [n_shards, 5] words in shard order -> (H nats, token)."""
    M, s, u, bv, bi = -np.inf, 0.0, 0.0, -np.inf, 2 ** 31 - 1
    for w in words:
        f = w[:4].view(np.float32).astype(np.float64)
        if f[0] == -np.inf:
            continue
        Mn = max(M, f[0])
        a = 0.0 if M == -np.inf else np.exp(M - Mn)
        b = np.exp(f[0] - Mn)
        u = a * (u + (M - Mn) * s if M != -np.inf else 0.0) + b * (f[2] + (f[0] - Mn) * f[1])
        s = a * s + b * f[1]
        M = Mn
        if f[3] > bv or (f[3] == bv and int(w[4]) < bi):
            bv, bi = f[3], int(w[4])
    return np.log(s) - u / s, bi


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, hid, w_bits, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        R, V = hid.shape[0], w_bits.shape[0]
        b, e = sharding.vocab_shard(V, rank, world)
        if e - b >= 2:
            mine = np.stack([_stats_words(oracle.logits_row(hid[r], w_bits[b:e]), b) for r in range(R)])
            mine = torch.from_numpy(mine)
        else:
            mine = sharding.empty_shard_stats(R)
        allg = sharding.gather_shard_stats(mine, dist)
        assert tuple(allg.shape) == (world, R, 5)
        np.save(os.path.join(out_dir, "g%d.npy" % rank), allg.numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,V", [(2, 1000), (3, 40)])
def test_ranks_vocab_sharding(tmp_path, oracle, world, V):
    import rstitch_inputs as gen
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], B=5, d=64, V=V, seed=4242 + V)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    mp.spawn(_worker, args=(world, _free_port(), hid, w_bits, str(tmp_path)), nprocs=world, join=True)
    ref = oracle.route(hid, w_bits, w.tau_nats)
    g0 = np.load(os.path.join(tmp_path, "g0.npy"))
    for r in range(1, world):
        assert np.array_equal(g0, np.load(os.path.join(tmp_path, "g%d.npy" % r)))   # every rank holds the same
    for r in range(w.B):
        H, tok = _merge(g0[:, r, :])
        assert abs(H - ref["ent"][r]) < 1e-4
        assert tok == ref["tok"][r] or ref["gap"][r] < 1e-3


def test_single_process_gather_and_empty_shard():
    st = torch.arange(10, dtype=torch.int32).reshape(2, 5)
    assert torch.equal(sharding.gather_shard_stats(st), st.unsqueeze(0))
    e = sharding.empty_shard_stats(3).numpy()
    assert e.shape == (3, 5) and e[:, :4].view(np.float32)[0, 0] == -np.inf and e[0, 4] == 2 ** 31 - 1
    w = _stats_words(np.array([0.5, 2.0, -1.0]), 7)
    H1, t1 = _merge(np.stack([w]))
    H2, t2 = _merge(np.stack([e[0], w, e[0]]))
    assert H1 == H2 and t1 == t2 == 8
