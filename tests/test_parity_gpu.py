"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded bf16 inputs (element by element at sizes the oracle finishes in seconds)."""
import math

import numpy as np
import pytest

import rstitch_inputs as gen
from parity_util import compare, run_gpu, to_dev_bf16, to_dev_i32

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


def check_case(rs, handle, oracle, w, steps, tau=None, flags=0, w_bits=None, w_dev=None):
    tau = w.tau_nats if tau is None else tau
    if w_bits is None:
        w_bits = gen.make_w_head(w)
    if w_dev is None:
        w_dev = to_dev_bf16(w_bits)
    stats = []
    for step in steps:
        hid, _ = gen.make_hidden(w, w_bits, step)
        seq_len, kv_len = gen.make_kv_state(w, step)
        ref = oracle.route(hid, w_bits, tau, seq_len=seq_len, kv_len=kv_len)
        gpu = run_gpu(handle, hid, w_dev, tau, seq_len=seq_len, kv_len=kv_len, flags=flags)
        stats.append(compare(gpu, ref, tau, w.B, w.B, oracle=oracle, seq_len=seq_len, kv_len=kv_len))
    st = rs.last_status(handle)
    assert st["status"] == 0 and st["nan_rows"] == 0 and st["bad_span"] == 0 and st["timeouts"] == 0
    return stats


def test_c1_tiny_all_steps(rs, handle, oracle):
    w = gen.WORKLOADS["c1_tiny"]
    stats = check_case(rs, handle, oracle, w, range(w.steps))
    assert max(s["max_ent_err"] for s in stats) < 1e-3


@pytest.mark.parametrize("B", [1, 2, 3, 4, 5, 7, 16, 17])
@pytest.mark.parametrize("d,V", [(8, 2), (8, 3), (64, 1000), (256, 4097), (1536, 2053), (24, 777)])
def test_shapes_and_ragged_tails(rs, handle, oracle, B, d, V):
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=7000 + B + d + V,
                   sigma_w=0.5 / math.sqrt(d))
    check_case(rs, handle, oracle, w, [0, 1])


@pytest.mark.parametrize("name,V,B", [("c2_slm_b1", 9001, 1), ("c3_llm_b1", 6007, 1), ("c3_llm_b4", 6007, 4),
                                       ("c3_llm_b16", 6007, 16), ("c4_slm_b64", 5003, 64),
                                       ("c4_llm_b64", 3001, 23)])
def test_reduced_vocab_workloads(rs, handle, oracle, name, V, B):
    # the paper-shaped heads with the vocabulary cut down so that the oracle covers every row
    w = gen.scaled(gen.WORKLOADS[name], V=V, B=B)
    stats = check_case(rs, handle, oracle, w, [0, 1, 2])
    if name.startswith(("c3", "c4")):
        rates = [s["route_rate"] for s in stats]
        assert 0.0 <= min(rates) and max(rates) <= 1.0


# ---- the tensor-core kernel, forced, on shapes that span several tiles and ragged tails ----------
@pytest.mark.parametrize("B,d,V", [
    (1, 64, 256), (5, 64, 1000), (16, 128, 4097), (17, 72, 2053), (64, 256, 6007), (128, 192, 3001),
    (3, 1536, 9001), (33, 512, 40009),
    (129, 64, 777), (200, 136, 2500), (300, 256, 4099), (544, 320, 1031),
])
def test_tensor_core_path_shapes(rs, handle, oracle, B, d, V):
    assert rs.path_name(B, d, V, rs.PATH_UMMA) == "umma"
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=9000 + B + d + V,
                   sigma_w=0.5 / math.sqrt(d))
    check_case(rs, handle, oracle, w, [0, 1], flags=rs.PATH_UMMA)


def test_tensor_core_path_gather_live_count_and_spans(rs, handle, oracle):
    # row gather + device-side live row count, then multi-row spans over several M tiles
    w = gen.scaled(gen.WORKLOADS["c4_llm_b64"], V=3000, d=512, B=64)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    row_idx = np.array([3, 9, 10, 31, 40, 63, 0, 0], dtype=np.int32)
    live = 6
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=row_idx[:live])
    gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=row_idx, n_rows_dev=live, R=8, flags=rs.PATH_UMMA)
    compare(gpu, ref, w.tau_nats, live, live)
    assert (gpu["tok"][live:8] == -1).all() and (gpu["ent"][live:8] == -1.0).all()
    # a live count of zero: nothing is evaluated, nothing is routed, every output row stays untouched
    for flags in (rs.PATH_UMMA, rs.PATH_GEMV):
        gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=row_idx, n_rows_dev=0, R=8, flags=flags)
        assert int(gpu["llm_count"][0]) == 0 and (gpu["tok"][:8] == -1).all() and (gpu["mask"][:8] == 255).all()
    bad = np.array([1, 64, -5, 2], dtype=np.int32)
    gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=bad, flags=rs.PATH_UMMA)
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=np.array([1, 0, 0, 2], dtype=np.int32))
    compare(gpu, ref, w.tau_nats, 4, 4)
    assert rs.last_status(handle)["bad_row_idx"] == 2

    w = gen.scaled(gen.WORKLOADS["c5_catchup"], V=2500, d=320, B=40)
    w_bits = gen.make_w_head(w)
    k = gen.make_spans(w, 0)
    R = int(k.sum())
    assert R > 128
    row_seq = np.repeat(np.arange(w.B, dtype=np.int32), k)
    hid, _ = gen.make_hidden(w, w_bits, 0, rows=R)
    seq_len, kv_len = gen.make_kv_state(w, 0, span=k)
    ref = oracle.route(hid, w_bits, w.tau_nats, row_seq=row_seq, B=w.B, seq_len=seq_len, kv_len=kv_len)
    gpu = run_gpu(handle, hid, to_dev_bf16(w_bits), w.tau_nats, row_seq=row_seq, B=w.B,
                  seq_len=seq_len, kv_len=kv_len, flags=rs.PATH_UMMA)
    compare(gpu, ref, w.tau_nats, R, w.B, row_seq=row_seq, oracle=oracle, seq_len=seq_len, kv_len=kv_len)


def test_tensor_core_path_nan_row_and_determinism(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], V=1024, d=64, B=9)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    hid[4, 5] = 0x7FC0
    ref = oracle.route(hid, w_bits, 100.0)
    a = run_gpu(handle, hid, to_dev_bf16(w_bits), 100.0, flags=rs.PATH_UMMA)
    compare(a, ref, 100.0, 9, 9)
    assert a["mask"][:9].tolist() == [0, 0, 0, 0, 1, 0, 0, 0, 0] and a["tok"][4] == 0
    assert rs.last_status(handle)["nan_rows"] == 1
    b = run_gpu(handle, hid, to_dev_bf16(w_bits), 100.0, flags=rs.PATH_UMMA)
    for k in a:
        assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8)), k


def test_path_choice(rs):
    assert rs.path_name(1, 1536, 151936) == "gemv" and rs.path_name(4, 3584, 152064) == "umma"
    assert rs.path_name(2, 3584, 152064) == "umma" and rs.path_name(3, 3584, 152064) == "umma"
    assert rs.path_name(16, 3584, 152064) == "umma" and rs.path_name(544, 5120, 152064) == "umma"
    assert rs.path_name(64, 32, 4096) == "gemv"          # too small for the tensor-core tiles
    assert rs.path_name(64, 1536, 151936, rs.PATH_GEMV) == "gemv"


def test_all_routed_none_routed_and_threshold_ends(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], V=2048, d=128, B=64, sigma_w=0.05)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    for tau, expect in [(-1.0, 64), (100.0, 0)]:
        ref = oracle.route(hid, w_bits, tau)
        gpu = run_gpu(handle, hid, w_dev, tau)
        compare(gpu, ref, tau, 64, 64)
        assert int(gpu["llm_count"][0]) == expect
    # exactly one routed sequence, at either end: threshold between the largest entropies
    ref = oracle.route(hid, w_bits, 0.0)
    order = np.argsort(ref["ent"])
    tau = 0.5 * (ref["ent"][order[-1]] + ref["ent"][order[-2]])
    if ref["ent"][order[-1]] - ref["ent"][order[-2]] > 0.01:
        gpu = run_gpu(handle, hid, w_dev, tau)
        assert int(gpu["llm_count"][0]) == 1 and gpu["llm_idx"][0] == order[-1]


def test_normalized_tau_flag(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=4096, d=256)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 5)
    for tau_paper in (0.0005, 0.001, 0.005, 0.01, 0.02, 0.03, 0.05):
        tau_nats = tau_paper * math.log(w.V)
        ref = oracle.route(hid, w_bits, tau_nats)
        gpu = run_gpu(handle, hid, to_dev_bf16(w_bits), tau_paper, flags=rs.TAU_NORMALIZED)
        compare(gpu, ref, tau_nats, w.B, w.B)


def test_row_gather_and_live_row_count(rs, handle, oracle):
    # the LLM head on the compacted subset of an earlier call: row_idx = llm_idx, rows = llm_count
    w = gen.scaled(gen.WORKLOADS["c4_llm_b64"], V=3000, d=512, B=64)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    row_idx = np.array([3, 9, 10, 31, 40, 63, 0, 0], dtype=np.int32)
    live = 6
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=row_idx[:live])
    gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=row_idx, n_rows_dev=live, R=8)
    compare(gpu, ref, w.tau_nats, live, live)
    assert (gpu["tok"][live:8] == -1).all() and (gpu["ent"][live:8] == -1.0).all()
    assert (gpu["mask"][live:8] == 255).all()
    # an out-of-range gather entry is counted, not dereferenced
    bad = np.array([1, 64, -5, 2], dtype=np.int32)
    gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=bad)
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=np.array([1, 0, 0, 2], dtype=np.int32))
    compare(gpu, ref, w.tau_nats, 4, 4)
    assert rs.last_status(handle)["bad_row_idx"] == 2


def test_multi_row_spans_decide_on_last_row(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c5_catchup"], V=2500, d=320, B=12)
    w_bits = gen.make_w_head(w)
    k = gen.make_spans(w, 0)
    R = int(k.sum())
    row_seq = np.repeat(np.arange(w.B, dtype=np.int32), k)
    hid, _ = gen.make_hidden(w, w_bits, 0, rows=R)
    seq_len, kv_len = gen.make_kv_state(w, 0, span=k)
    ref = oracle.route(hid, w_bits, w.tau_nats, row_seq=row_seq, B=w.B, seq_len=seq_len, kv_len=kv_len)
    gpu = run_gpu(handle, hid, to_dev_bf16(w_bits), w.tau_nats, row_seq=row_seq, B=w.B,
                  seq_len=seq_len, kv_len=kv_len)
    compare(gpu, ref, w.tau_nats, R, w.B, row_seq=row_seq, oracle=oracle, seq_len=seq_len, kv_len=kv_len)
    cnt = int(gpu["llm_count"][0])
    assert gpu["llm_row_off"][cnt] == k[gpu["llm_idx"][:cnt]].sum()


def test_bad_span_is_counted(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], V=512, d=64, B=4)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    seq_len = np.array([10, 10, 10, 10], dtype=np.int32)
    kv_len = np.array([9, 10, 12, 5], dtype=np.int32)
    gpu = run_gpu(handle, hid, to_dev_bf16(w_bits), -1.0, seq_len=seq_len, kv_len=kv_len)
    assert gpu["llm_span"][:4].tolist() == [1, 0, -2, 5]
    assert rs.last_status(handle)["bad_span"] == 2


def test_nan_row_is_routed_and_counted(rs, handle, oracle):
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], V=1024, d=64, B=3)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    hid[1, 5] = 0x7FC0
    ref = oracle.route(hid, w_bits, 100.0)
    gpu = run_gpu(handle, hid, to_dev_bf16(w_bits), 100.0)
    compare(gpu, ref, 100.0, 3, 3)
    assert gpu["mask"][:3].tolist() == [0, 1, 0] and gpu["tok"][1] == 0
    assert rs.last_status(handle)["nan_rows"] == 1


def test_determinism_bitwise(rs, handle):
    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=20011, d=512)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    a = run_gpu(handle, hid, w_dev, w.tau_nats)
    for _ in range(3):
        b = run_gpu(handle, hid, w_dev, w.tau_nats)
        for k in a:
            assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8)), k


def test_basic_entry_point_and_empty_batch(rs, oracle):
    import torch
    w = gen.WORKLOADS["c1_tiny"]
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 1)
    out = rs.route(to_dev_bf16(hid), to_dev_bf16(w_bits), w.tau_nats)
    torch.cuda.synchronize()
    ref = oracle.route(hid, w_bits, w.tau_nats)
    gpu = {k: getattr(out, k).cpu().numpy() for k in ("tok", "ent", "mask", "llm_idx", "llm_count")}
    compare(gpu, ref, w.tau_nats, w.B, w.B)
    # B = 0: valid, count = 0, nothing else touched
    empty = torch.empty((0, w.d), dtype=torch.bfloat16, device="cuda")
    out = rs.route(empty, to_dev_bf16(w_bits), w.tau_nats)
    torch.cuda.synchronize()
    assert int(out.llm_count.item()) == 0 and int(out.tok[0].item()) == -1


def test_host_buffer_entry_point(rs, handle, oracle):
    import torch
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], V=4099, d=256, B=64)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 2)
    hh = torch.from_numpy(hid.view(np.int16)).view(torch.bfloat16).pin_memory()
    host = {"tok": torch.full((64,), -1, dtype=torch.int32).pin_memory(),
            "ent": torch.zeros(64, dtype=torch.float32).pin_memory(),
            "mask": torch.zeros(64, dtype=torch.uint8).pin_memory(),
            "llm_idx": torch.full((64,), -1, dtype=torch.int32).pin_memory(),
            "llm_count": torch.zeros(1, dtype=torch.int32).pin_memory()}
    rs.route_host(handle, hh, to_dev_bf16(w_bits), w.tau_nats, host)
    ref = oracle.route(hid, w_bits, w.tau_nats)
    gpu = {k: v.numpy() for k, v in host.items()}
    cnt = int(gpu["llm_count"][0])
    gpu["llm_idx"][cnt:] = -1          # the copy brings back the whole staging array
    compare(gpu, ref, w.tau_nats, 64, 64)


def test_host_buffer_extended_entry_point(rs, handle, oracle):
    # multi-row spans with everything per-step in host memory, then a row gather driven from the host
    import torch
    w = gen.scaled(gen.WORKLOADS["c5_catchup"], V=2500, d=320, B=12)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    k = gen.make_spans(w, 1)
    R = int(k.sum())
    row_seq = np.repeat(np.arange(w.B, dtype=np.int32), k)
    hid, _ = gen.make_hidden(w, w_bits, 1, rows=R)
    seq_len, kv_len = gen.make_kv_state(w, 1, span=k)

    def host_out(R, B):
        return {"tok": torch.full((R,), -1, dtype=torch.int32).pin_memory(),
                "ent": torch.zeros(R, dtype=torch.float32).pin_memory(),
                "mask": torch.zeros(B, dtype=torch.uint8).pin_memory(),
                "llm_idx": torch.full((B,), -1, dtype=torch.int32).pin_memory(),
                "llm_count": torch.zeros(1, dtype=torch.int32).pin_memory(),
                "llm_span": torch.full((B,), -1, dtype=torch.int32).pin_memory(),
                "llm_row_off": torch.full((B + 1,), -1, dtype=torch.int32).pin_memory()}

    hh = torch.from_numpy(hid.view(np.int16)).view(torch.bfloat16).pin_memory()
    out = rs.route_ex_host(handle, hh, w_dev, w.tau_nats, host_out(R, w.B), R=R, B=w.B,
                           row_seq=torch.from_numpy(row_seq), seq_len=torch.from_numpy(seq_len),
                           kv_len=torch.from_numpy(kv_len))
    ref = oracle.route(hid, w_bits, w.tau_nats, row_seq=row_seq, B=w.B, seq_len=seq_len, kv_len=kv_len)
    gpu = {k_: v.numpy() for k_, v in out.items()}
    cnt = int(gpu["llm_count"][0])
    gpu["llm_idx"][cnt:] = -1
    compare(gpu, ref, w.tau_nats, R, w.B, row_seq=row_seq, oracle=oracle, seq_len=seq_len, kv_len=kv_len)

    row_idx = np.array([5, 0, R - 1, 7, 7], dtype=np.int32)
    out = rs.route_ex_host(handle, hh, w_dev, w.tau_nats, host_out(5, 5), row_idx=torch.from_numpy(row_idx))
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=row_idx)
    gpu = {k_: v.numpy() for k_, v in out.items()}
    gpu["llm_idx"][int(gpu["llm_count"][0]):] = -1
    compare(gpu, ref, w.tau_nats, 5, 5)


def test_caller_workspace(rs, handle, oracle):
    import torch
    w = gen.scaled(gen.WORKLOADS["c3_llm_b4"], V=3001, d=128)
    w_bits = gen.make_w_head(w)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    n = rs.workspace_bytes(w.B, w.d, w.V)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda").fill_(0xAB)
    out = rs.route_ex(handle, to_dev_bf16(hid), to_dev_bf16(w_bits), w.tau_nats, workspace=ws)
    torch.cuda.synchronize()
    ref = oracle.route(hid, w_bits, w.tau_nats)
    gpu = {k: getattr(out, k).cpu().numpy() for k in ("tok", "ent", "mask", "llm_idx", "llm_count")}
    compare(gpu, ref, w.tau_nats, w.B, w.B)
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    assert rs.route_ex(handle, to_dev_bf16(hid), to_dev_bf16(w_bits), 0.3, workspace=small, check=False) == -5


def test_device_side_argument_errors(rs, handle):
    import torch
    w_dev = torch.zeros((64, 32), dtype=torch.bfloat16, device="cuda")
    hid = torch.zeros((5, 32), dtype=torch.bfloat16, device="cuda")
    assert rs.route_ex(handle, hid, w_dev, float("nan"), check=False) == -1
    assert rs.route_ex(handle, hid, w_dev, 0.3, B=3, check=False) == -1          # B != R without row_seq
    assert rs.route_ex(handle, hid, w_dev, 0.3, flags=0x30, check=False) == -1
    assert rs.route_ex(handle, hid, w_dev, 0.3, flags=0x4000, check=False) == -1         # unknown flag
    flat = torch.zeros(5 * 32 + 8, dtype=torch.bfloat16, device="cuda")
    mis = flat[1:1 + 5 * 32].view(5, 32)                                           # 2-byte offset
    assert rs.route_ex(handle, mis, w_dev, 0.3, check=False) == -2
    big = torch.zeros((2, 16384 + 8), dtype=torch.bfloat16, device="cuda")
    wbig = torch.zeros((4, 16384 + 8), dtype=torch.bfloat16, device="cuda")
    assert rs.route_ex(handle, big, wbig, 0.3, check=False) == -3


@pytest.mark.parametrize("B", [0, 1, 31, 32, 33, 255, 256, 257, 1000, 65536, 65537, 300001])
def test_standalone_compaction(rs, oracle, B):
    import torch
    for p in (0.1, 0.5, 0.9):
        m = gen.random_mask(B, p, seed=B)
        md = torch.from_numpy(m).cuda() if B else torch.zeros(0, dtype=torch.uint8, device="cuda")
        idx, cnt = rs.compact(md)
        torch.cuda.synchronize()
        ref_idx, ref_cnt = oracle.compact(m)
        assert int(cnt.item()) == ref_cnt
        assert np.array_equal(idx.cpu().numpy()[:ref_cnt], ref_idx)
        if B:
            assert (idx.cpu().numpy()[ref_cnt:] == -1).all()
    for fill in (0, 1):
        if B:
            md = torch.full((B,), fill, dtype=torch.uint8, device="cuda")
            idx, cnt = rs.compact(md)
            assert int(cnt.item()) == fill * B


# ---- sampled token ---------------------------------------------------------------------------------
@pytest.mark.parametrize("B,d,V,flags", [
    (1, 64, 300, "gemv"), (3, 256, 4097, "gemv"), (4, 1536, 9001, "gemv"),
    (5, 64, 1000, "umma"), (16, 128, 4097, "umma"), (64, 256, 6007, "umma"), (200, 136, 2500, "umma"),
    (300, 256, 4099, "umma"),
])
def test_sampled_token(rs, handle, oracle, B, d, V, flags):
    flag = rs.PATH_GEMV if flags == "gemv" else rs.PATH_UMMA
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=9900 + B + d + V, sigma_w=0.5 / math.sqrt(d))
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    ref = oracle.route(hid, w_bits, w.tau_nats)
    exempt = 0
    seen = []
    for T_s, seed, draw in [(1.0, 7, 0), (1.0, 7, 1), (0.6, 2 ** 40 + 5, 2 ** 33 + 9), (2.5, 1, 123456)]:
        tok, gap = oracle.sample_rows(hid, w_bits, T_s, seed, draw)
        gpu = run_gpu(handle, hid, w_dev, w.tau_nats, flags=flag, sample=(T_s, seed, draw))
        ok = (gpu["tok"][:B] == tok) | (gap < 1e-3)
        assert ok.all(), (T_s, seed, draw, np.flatnonzero(~ok)[:8])
        exempt += int((gap < 1e-3).sum())
        # entropy, mask and compaction do not depend on the draw
        assert np.abs(gpu["ent"][:B] - ref["ent"]).max() <= 2e-3
        clear = np.abs(ref["ent"] - w.tau_nats) > 2e-3
        assert np.array_equal(gpu["mask"][:B][clear], ref["mask"][clear])
        seen.append(gpu["tok"][:B].copy())
    assert exempt <= max(1, B // 20)
    if B >= 16:
        assert not np.array_equal(seen[0], seen[1])          # a new draw number gives new tokens
        assert not np.array_equal(seen[0], ref["tok"])       # and they are not simply the greedy ones
    # temperature -> 0 reproduces the greedy token wherever the top-2 logit gap is clear
    gpu = run_gpu(handle, hid, w_dev, w.tau_nats, flags=flag, sample=(1e-3, 7, 0))
    clear = ref["gap"] > 0.05
    assert np.array_equal(gpu["tok"][:B][clear], ref["tok"][clear])
    assert rs.route_ex(handle, to_dev_bf16(hid), w_dev, 0.3, sample=(0.0, 1, 1), check=False) == -1
    assert rs.route_ex(handle, to_dev_bf16(hid), w_dev, 0.3, sample=(float("nan"), 1, 1), check=False) == -1


def test_step_loop_replays_from_a_cuda_graph(rs, handle, oracle):
    # a chain of calls with no host synchronisation (SLM head, then the LLM head on the routed subset with
    # the count on the device) records into a CUDA graph; replays give what the direct calls gave
    import torch
    ws = gen.scaled(gen.WORKLOADS["c4_slm_b64"], V=3000, d=512, B=64)
    wl = gen.scaled(gen.WORKLOADS["c4_llm_b64"], V=2600, d=640, B=64)
    s_bits, l_bits = gen.make_w_head(ws), gen.make_w_head(wl)
    s_dev, l_dev = to_dev_bf16(s_bits), to_dev_bf16(l_bits)
    hs = to_dev_bf16(gen.make_hidden(ws, s_bits, 0)[0])
    hl = to_dev_bf16(gen.make_hidden(wl, l_bits, 0)[0])
    h2 = rs.Handle(64, 640, 2600)
    side = torch.cuda.Stream()
    out_s = rs.RouteOutputs.allocate(64, 64, hs.device)
    out_l = rs.RouteOutputs.allocate(64, 64, hs.device)
    c1 = rs.PreparedCall(handle, hs, s_dev, ws.tau_nats, out_s, stream=side)
    c2 = rs.PreparedCall(h2, hl, l_dev, wl.tau_nats, out_l, R=64, B=64, row_idx=out_s.llm_idx,
                         n_rows_dev=out_s.llm_count, stream=side)
    with torch.cuda.stream(side):
        assert c1.launch() == 0 and c2.launch() == 0            # first calls outside the capture
    side.synchronize()
    want = [t.clone() for t in (out_s.tok, out_s.ent, out_s.mask, out_s.llm_count, out_l.tok, out_l.ent, out_l.llm_count)]
    cnt = int(out_s.llm_count.item())
    assert 0 < cnt < 64
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        assert c1.launch() == 0 and c2.launch() == 0
    for t in (out_s.tok, out_s.ent, out_l.tok, out_l.ent):
        t.fill_(-1)
    g.replay()
    torch.cuda.synchronize()
    got = [out_s.tok, out_s.ent, out_s.mask, out_s.llm_count, out_l.tok, out_l.ent, out_l.llm_count]
    for i, (a, b) in enumerate(zip(want, got)):
        n = cnt if i in (4, 5) else a.shape[0]          # the LLM head wrote only the routed rows
        assert torch.equal(a[:n], b[:n]), i
    h2.destroy()


@pytest.mark.parametrize("B,d,V,path", [(16384, 64, 512, "umma"), (16384, 64, 300, "gemv"), (3, 16384, 300, "gemv"),
                                         (5, 16384, 512, "umma"), (200, 16384, 256, "umma")])
def test_maximum_sizes(rs, oracle, B, d, V, path):
    # the largest row count and the largest hidden size the library accepts, each beside a small other side
    flag = rs.PATH_GEMV if path == "gemv" else rs.PATH_UMMA
    h = rs.Handle(B, d, V)
    try:
        w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=9700 + B + d + V, sigma_w=0.5 / math.sqrt(d))
        check_case(rs, h, oracle, w, [0], flags=flag)
        assert rs.route_ex(h, to_dev_bf16(np.zeros((B, d), dtype=np.uint16)), to_dev_bf16(gen.make_w_head(w)),
                           0.3, R=B + 1, check=False) != 0        # one row more than the handle was made for
    finally:
        h.destroy()
    assert rs.workspace_bytes(16385, 64, 512) == 0 and rs.workspace_bytes(4, 16392, 512) == 0


def test_bounded_wait_runs_out_and_the_handle_stays_usable(rs, handle, oracle):
    # every device-side wait in the kernels has a cycle limit; this makes one run out (a barrier nothing
    # arrives at, limited to ~1 ms) and checks the report, then that the same handle still decides correctly
    import time
    import torch
    rs.last_status(handle)
    t0 = time.perf_counter()
    assert rs.selftest_wait(handle) == 0
    st = rs.last_status(handle)
    assert time.perf_counter() - t0 < 1.0
    assert st["status"] == -6 and st["timeouts"] == 1 and st["timeout_site"] == rs.SELFTEST_SITE
    assert rs.status_string(-6) == "device-side wait timed out"
    w = gen.scaled(gen.WORKLOADS["c3_llm_b4"], V=6007, d=512)
    for flags in (rs.PATH_GEMV, rs.PATH_UMMA):
        check_case(rs, handle, oracle, w, [0], flags=flags)          # asserts a clean status word again
    assert torch.cuda.is_available()


def test_random_shapes_sweep(rs, handle, oracle):
    # seeded draw of shapes across both kernel families: odd hidden sizes (k-steps that do not fill a group,
    # half-empty last k-step), vocabularies that end inside a 16-row unit, row counts around the M-tile and
    # M = 64 boundaries, last rounds that split into pieces
    rng = np.random.default_rng(20260)
    edges = [1, 2, 3, 8, 9, 16, 17, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 320, 385, 512, 640]
    done = 0
    while done < 48:
        B = int(rng.choice(edges)) if rng.random() < 0.7 else int(rng.integers(1, 700))
        d = 8 * int(rng.integers(1, 129))
        V = int(rng.integers(2, 6000))
        if B * d * V > 2.5e8:
            continue
        path = rng.choice(["auto", "gemv", "umma"])
        if path == "gemv" and B > 40:
            path = "auto"
        flags = {"auto": 0, "gemv": rs.PATH_GEMV, "umma": rs.PATH_UMMA}[str(path)]
        w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=31000 + done, sigma_w=0.5 / math.sqrt(d))
        try:
            check_case(rs, handle, oracle, w, [0], flags=flags)
        except AssertionError as e:
            raise AssertionError("case %d: B=%d d=%d V=%d path=%s: %s" % (done, B, d, V, path, e))
        done += 1


def test_back_to_back_calls_share_one_scratch(rs, handle, oracle):
    # A call's head kernel is allowed to start while the call before it on the stream is still merging
    # its partial statistics (programmatic dependent launch); the two share the handle's scratch.  A long
    # train of calls of mixed shapes, row counts and kernel families is enqueued without any host
    # synchronisation, every call into its own output buffers, the inputs of call i + 1 written by a
    # copy kernel enqueued right behind call i; afterwards every call's decision is compared with the
    # oracle's.  A head kernel that read its hidden rows, or wrote the scratch, before the kernels ahead
    # of it had finished would show up here.
    import torch
    shapes = [(1, 512, 9001), (16, 256, 4099), (1, 64, 300), (64, 320, 5003), (3, 128, 2000), (130, 256, 2304),
              (2, 1024, 30011), (40, 64, 777)]
    cases = []
    for k, (B, d, V) in enumerate(shapes):
        w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=d, V=V, seed=9700 + k, sigma_w=0.5 / math.sqrt(d))
        w_bits = gen.make_w_head(w)
        hids = [gen.make_hidden(w, w_bits, s)[0] for s in range(3)]
        cases.append({"w": w, "w_bits": w_bits, "w_dev": to_dev_bf16(w_bits), "hid_bits": hids,
                      "staged": [to_dev_bf16(h) for h in hids],                 # where the inputs wait
                      "live": torch.zeros((B, d), dtype=torch.bfloat16, device="cuda")})   # what the calls read
    order = [(k, s) for s in range(3) for k in range(len(cases))]
    outs = [rs.RouteOutputs.allocate(cases[k]["w"].B, cases[k]["w"].B, "cuda") for k, _ in order]   # (fills: kernels)
    torch.cuda.synchronize()
    for (k, s), out in zip(order, outs):
        c = cases[k]
        if s == 1:
            hid = c["staged"][s]                         # nothing between this call and the one before it
        else:
            hid = c["live"]
            hid.copy_(c["staged"][s])                    # a kernel right in front of the call writes its input
        rs.route_ex(handle, hid, c["w_dev"], c["w"].tau_nats, out=out)
    torch.cuda.synchronize()
    for (k, s), out in zip(order, outs):
        c = cases[k]
        w = c["w"]
        gpu = {n: getattr(out, n).cpu().numpy() for n in ("tok", "ent", "mask", "llm_idx", "llm_count")}
        compare(gpu, oracle.route(c["hid_bits"][s], c["w_bits"], w.tau_nats), w.tau_nats, w.B, w.B)
    st = rs.last_status(handle)
    assert st["timeouts"] == 0 and st["nan_rows"] == 0


@pytest.mark.parametrize("path", ["gemv", "umma"])
@pytest.mark.parametrize("gather", [False, True])
def test_live_row_count_of_zero_on_the_device(rs, handle, oracle, path, gather):
    # a device-side row count of zero (the LLM's batch in a round in which no sequence sits on the LLM): the
    # head kernel has already asked for its first ring of W_head when it learns that; nothing may be written
    # but llm_count = 0, no wait may run out, and the very next call on the handle must be a normal one
    flags = rs.PATH_GEMV if path == "gemv" else rs.PATH_UMMA
    w = gen.scaled(gen.WORKLOADS["c4_llm_b64"], V=5003, d=512, B=40)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    hid, _ = gen.make_hidden(w, w_bits, 0)
    row_idx = np.arange(w.B, dtype=np.int32)[::-1].copy() if gather else None
    for _ in range(3):
        gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=row_idx, n_rows_dev=0, R=w.B, flags=flags)
        assert int(gpu["llm_count"][0]) == 0
        assert (gpu["tok"] == -1).all() and (gpu["ent"] == -1.0).all()
        assert (gpu["mask"] == 255).all() and (gpu["llm_idx"] == -1).all()
    st = rs.last_status(handle)
    assert st["timeouts"] == 0 and st["nan_rows"] == 0 and st["bad_row_idx"] == 0
    ref = oracle.route(hid, w_bits, w.tau_nats, row_idx=row_idx)
    gpu = run_gpu(handle, hid, w_dev, w.tau_nats, row_idx=row_idx, flags=flags)
    compare(gpu, ref, w.tau_nats, w.B, w.B)
    assert rs.last_status(handle)["timeouts"] == 0
