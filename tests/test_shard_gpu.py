"""GPU parity of the vocabulary-parallel head: the shards of one call run one after another on one GPU
(independent launches, nothing waits on anything), their statistics are stacked as an all-gather would
stack them, and rstitch_shard_route's decision is compared with the fp64 oracle on the WHOLE vocabulary
under the usual tolerance rules."""
import math

import numpy as np
import pytest

import rstitch_inputs as gen
from parity_util import compare, to_dev_bf16, to_dev_i32
from paper_2507_17307_b200 import sharding

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rs():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2507_17307_b200 import build
    build.build_library()
    import paper_2507_17307_b200 as rs
    return rs


@pytest.fixture(scope="module")
def handle(rs):
    h = rs.Handle(1024, 8192, 160000)
    yield h
    h.destroy()


def run_sharded(rs, handle, hid_dev, w_dev, V, world, tau, *, flags=0, sample=None, row_idx=None, n_rows_dev=None,
                R=None, B=None, row_seq=None, seq_len=None, kv_len=None):
    import torch
    parts = []
    for rank in range(world):
        b, e = sharding.vocab_shard(V, rank, world)
        if e - b < 2:
            n = R if R is not None else (row_idx.shape[0] if row_idx is not None else hid_dev.shape[0])
            parts.append(sharding.empty_shard_stats(n, "cuda"))
            continue
        parts.append(rs.shard_stats(handle, hid_dev, w_dev[b:e], b, R=R, row_idx=row_idx, n_rows_dev=n_rows_dev,
                                    flags=flags, sample=sample))
    gathered = torch.stack(parts).contiguous()
    out = rs.shard_route(handle, gathered, V, tau, R=R, B=B, row_seq=row_seq, n_rows_dev=n_rows_dev,
                         seq_len=seq_len, kv_len=kv_len)
    torch.cuda.synchronize()
    res = {k: getattr(out, k).cpu().numpy() for k in ("tok", "ent", "mask", "llm_idx", "llm_count")}
    if out.llm_span is not None:
        res["llm_span"] = out.llm_span.cpu().numpy()
        res["llm_row_off"] = out.llm_row_off.cpu().numpy()
    return res, gathered


@pytest.mark.parametrize("B,d,V,world,path", [
    (1, 256, 4096, 2, "gemv"), (1, 1536, 9001, 3, "gemv"), (4, 64, 1000, 8, "gemv"),
    (5, 128, 4097, 2, "umma"), (16, 512, 40009, 4, "umma"), (70, 256, 6007, 3, "umma"),
    (129, 64, 2500, 2, "umma"), (300, 256, 4099, 5, "umma"), (300, 136, 777, 8, "auto"),
])
def test_sharded_head_matches_oracle(rs, handle, oracle, B, d, V, world, path):
    flags = {"gemv": rs.PATH_GEMV, "umma": rs.PATH_UMMA, "auto": 0}[path]
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=9300 + B + d + V, sigma_w=0.5 / math.sqrt(d))
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    for step in (0, 1):
        hid, _ = gen.make_hidden(w, w_bits, step)
        seq_len, kv_len = gen.make_kv_state(w, step)
        ref = oracle.route(hid, w_bits, w.tau_nats, seq_len=seq_len, kv_len=kv_len)
        gpu, _ = run_sharded(rs, handle, to_dev_bf16(hid), w_dev, V, world, w.tau_nats, flags=flags,
                             seq_len=to_dev_i32(seq_len), kv_len=to_dev_i32(kv_len))
        compare(gpu, ref, w.tau_nats, B, B, oracle=oracle, seq_len=seq_len, kv_len=kv_len)
    st = rs.last_status(handle)
    assert st["status"] == 0 and st["nan_rows"] == 0 and st["timeouts"] == 0


def test_one_shard_is_the_whole_call(rs, handle, oracle):
    # world = 1: the statistics of the whole vocabulary, then the tail; bit-identical to rstitch_route_ex
    import torch
    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=6007, d=512, B=16)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid = to_dev_bf16(gen.make_hidden(w, w_bits, 0)[0])
    gpu, gathered = run_sharded(rs, handle, hid, w_dev, w.V, 1, w.tau_nats)
    direct = rs.route_ex(handle, hid, w_dev, w.tau_nats)
    torch.cuda.synchronize()
    assert np.array_equal(gpu["tok"], direct.tok.cpu().numpy())
    assert np.array_equal(gpu["ent"], direct.ent.cpu().numpy())
    assert np.array_equal(gpu["mask"], direct.mask.cpu().numpy())
    assert np.array_equal(gpu["llm_idx"], direct.llm_idx.cpu().numpy())
    # the statistics words: s >= 1, u <= 0, the best score equals the largest logit, the index is in range
    g = gathered.cpu().numpy()[0]
    f = g[:, :4].view(np.float32)
    assert (f[:, 1] >= 1.0).all() and (f[:, 2] <= 0.0).all() and np.array_equal(f[:, 0], f[:, 3])
    assert (g[:, 4] >= 0).all() and (g[:, 4] < w.V).all()


def test_sharded_gather_live_count_and_spans(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c4_llm_b64"], V=3000, d=512, B=64)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    row_idx = np.array([3, 9, 10, 31, 40, 63, 0, 0], dtype=np.int32)
    live = 6
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=row_idx[:live])
    for flags in (rs.PATH_GEMV, rs.PATH_UMMA):
        gpu, _ = run_sharded(rs, handle, to_dev_bf16(hid), w_dev, w.V, 3, w.tau_nats, flags=flags,
                             row_idx=to_dev_i32(row_idx), n_rows_dev=to_dev_i32([live]), R=8)
        compare(gpu, ref, w.tau_nats, live, live)
        assert (gpu["tok"][live:8] == -1).all() and (gpu["mask"][live:8] == 255).all()
    # multi-row spans: the last row of each sequence decides
    w = gen.scaled(gen.WORKLOADS["c5_catchup"], V=2500, d=320, B=40)
    w_bits = gen.make_w_head(w)
    k = gen.make_spans(w, 0)
    R = int(k.sum())
    row_seq = np.repeat(np.arange(w.B, dtype=np.int32), k)
    hid, _ = gen.make_hidden(gen.scaled(w, B=R), w_bits, 0)
    ref = oracle.route(hid, w_bits, w.tau_nats, row_seq=row_seq, B=w.B)
    gpu, _ = run_sharded(rs, handle, to_dev_bf16(hid), to_dev_bf16(w_bits), w.V, 4, w.tau_nats, R=R, B=w.B,
                         row_seq=to_dev_i32(row_seq))
    compare(gpu, ref, w.tau_nats, R, w.B, row_seq=row_seq)


@pytest.mark.parametrize("B,d,V,world,path", [(16, 256, 4097, 3, "gemv"), (40, 128, 6007, 4, "umma")])
def test_sharded_sampled_token_does_not_depend_on_the_split(rs, handle, oracle, B, d, V, world, path):
    flags = rs.PATH_GEMV if path == "gemv" else rs.PATH_UMMA
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=9400 + B + d + V, sigma_w=0.5 / math.sqrt(d))
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    hid_dev, w_dev = to_dev_bf16(hid), to_dev_bf16(w_bits)
    for T_s, seed, draw in [(1.0, 7, 0), (0.6, 2 ** 40 + 5, 2 ** 33 + 9)]:
        tok, gap = oracle.sample_rows(hid, w_bits, T_s, seed, draw)
        gpu, _ = run_sharded(rs, handle, hid_dev, w_dev, V, world, w.tau_nats, flags=flags, sample=(T_s, seed, draw))
        ok = (gpu["tok"][:B] == tok) | (gap < 1e-3)
        assert ok.all(), (T_s, seed, draw, np.flatnonzero(~ok)[:8])


def test_shard_argument_errors(rs, handle):
    import torch
    hid = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    assert rs.shard_stats(handle, hid, W, -1, check=False) == -1                  # negative base index
    assert rs.shard_stats(handle, hid, W[:1], 0, check=False) == -3               # a one-row shard
    g = torch.zeros((2, 4, 5), dtype=torch.int32, device="cuda")
    assert rs.shard_route(handle, g, 1, 0.3, check=False) == -1                   # vocabulary of one entry
    assert rs.shard_route(handle, g, 128, float("nan"), check=False) == -1
    assert rs.shard_route(handle, g, 128, 0.3, B=3, check=False) == -1            # B != R without row_seq
