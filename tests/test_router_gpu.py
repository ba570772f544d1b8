"""GPU parity of the R-Stitch+ router forward against the oracle, alone and chained after the routing
decision (entropy rule -> router on the routed rows -> refined mask -> compaction)."""
import numpy as np
import pytest

import rstitch_inputs as gen
from parity_util import to_dev_bf16, to_dev_i32

pytestmark = pytest.mark.gpu
LOGIT_TOL = 2e-3


@pytest.fixture(scope="module")
def rs():
    import torch
    assert torch.cuda.is_available()
    from paper_2507_17307_b200 import build
    build.build_library()
    import paper_2507_17307_b200 as rs
    return rs


def dev_weights(w):
    import torch
    return {k: torch.from_numpy(v).cuda() for k, v in w.items()}


@pytest.mark.parametrize("R,d,h,ff,L", [(1, 64, 8, 16, 1), (7, 256, 32, 64, 6), (64, 1536, 32, 64, 6),
                                         (33, 3584, 40, 80, 6), (5, 512, 256, 1024, 2), (3, 128, 16, 32, 0)])
def test_router_logits_and_switch(rs, oracle, R, d, h, ff, L):
    import torch
    w = gen.make_router_weights(d, h, ff, max(L, 1), seed=R + d)
    if L == 0:
        w = {k: (v[:0] if k in ("W1", "b1", "W2", "b2") else v) for k, v in w.items()}
        w["W1"] = np.zeros((0, ff, h), np.float32); w["W2"] = np.zeros((0, h, ff), np.float32)
        w["b1"] = np.zeros((0, ff), np.float32); w["b2"] = np.zeros((0, h), np.float32)
    rng = np.random.default_rng(R * 31 + d)
    hid = gen.f32_to_bf16_bits((rng.standard_normal((R + 3, d)) * 2.0).astype(np.float32))
    idx = rng.integers(0, R + 3, size=R).astype(np.int32)
    router = rs.Router(dev_weights(w))
    for row_idx in (None, idx):
        ref_logits, ref_sw = oracle.router_rows(hid, w, row_idx=row_idx) if row_idx is not None else \
            oracle.router_rows(hid[:R], w)
        logits, sw = router.forward(to_dev_bf16(hid), R, row_idx=None if row_idx is None else to_dev_i32(row_idx))
        torch.cuda.synchronize()
        got = logits.cpu().numpy()[:R]
        assert np.abs(got - ref_logits).max() <= LOGIT_TOL
        clear = np.abs(ref_logits[:, 1] - ref_logits[:, 0]) > 2 * LOGIT_TOL
        assert np.array_equal(sw.cpu().numpy()[:R][clear], ref_sw[clear])


def test_router_after_the_entropy_rule(rs, oracle):
    import torch
    ws = gen.scaled(gen.WORKLOADS["c4_slm_b64"], V=3000, d=512, B=64)
    w_bits = gen.make_w_head(ws)
    hid, _ = gen.make_hidden(ws, w_bits, 1)
    rw = gen.make_router_weights(512, 32, 64, 6, seed=5)
    handle = rs.Handle(64, 512, 3000)
    hid_dev = to_dev_bf16(hid)
    out = rs.route_ex(handle, hid_dev, to_dev_bf16(w_bits), ws.tau_nats)
    router = rs.Router(dev_weights(rw))
    mask = out.mask.clone()
    logits, sw = router.forward(hid_dev, 64, row_idx=out.llm_idx, n_rows_dev=out.llm_count, refine_mask=mask)
    idx2, cnt2 = rs.compact(mask)
    torch.cuda.synchronize()
    ref = oracle.route(hid, w_bits, ws.tau_nats)
    assert (np.abs(ref["ent"] - ws.tau_nats) > 2e-3).all(), "pick another step: a row sits in the tolerance band"
    cnt = int(out.llm_count.item())
    assert cnt == ref["llm_count"] and 0 < cnt < 64
    r_logits, r_sw = oracle.router_rows(hid, rw, row_idx=ref["llm_idx"])
    assert np.abs(logits.cpu().numpy()[:cnt] - r_logits).max() <= LOGIT_TOL
    assert (np.abs(r_logits[:, 1] - r_logits[:, 0]) > 2 * LOGIT_TOL).all()
    want_mask = np.zeros(64, np.uint8)
    want_mask[ref["llm_idx"]] = r_sw                      # routed only where the router says LLM
    assert np.array_equal(mask.cpu().numpy(), want_mask)
    assert (sw.cpu().numpy()[cnt:] == 255).all()          # entries past the live count are untouched
    want_idx = np.flatnonzero(want_mask)
    assert int(cnt2.item()) == want_idx.size and np.array_equal(idx2.cpu().numpy()[:want_idx.size], want_idx)
    assert 0 < want_idx.size < cnt                        # the router kept some steps on the SLM
    # the one-launch form: same refined mask, same compaction, three times in a row (the ticket rewinds)
    for _ in range(3):
        mask3 = out.mask.clone()
        idx3 = torch.full((64,), -1, dtype=torch.int32, device="cuda")
        cnt3 = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        logits3, sw3 = router.route(hid_dev, 64, out.llm_idx, mask3, idx3, cnt3, n_rows_dev=out.llm_count)
        torch.cuda.synchronize()
        assert torch.equal(mask3, mask) and torch.equal(logits3[:cnt], logits[:cnt]) and torch.equal(sw3, sw)
        assert int(cnt3.item()) == want_idx.size and np.array_equal(idx3.cpu().numpy()[:want_idx.size], want_idx)
        assert (idx3.cpu().numpy()[want_idx.size:] == -1).all()
    # nothing routed by the entropy rule: the router has no rows, the compaction still runs
    zero = torch.zeros(1, dtype=torch.int32, device="cuda")
    mask0 = torch.zeros(64, dtype=torch.uint8, device="cuda")
    router.route(hid_dev, 64, out.llm_idx, mask0, idx3, cnt3, n_rows_dev=zero)
    torch.cuda.synchronize()
    assert int(cnt3.item()) == 0 and int(mask0.sum().item()) == 0
    assert router.route(hid_dev, 64, None, mask0, idx3, cnt3, check=False) == -1       # row_idx is required
    handle.destroy()


def test_router_argument_errors(rs):
    import torch
    w = dev_weights(gen.make_router_weights(64, 8, 16, 1, seed=1))
    r = rs.Router(w)
    hid = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    mask = torch.zeros(4, dtype=torch.uint8, device="cuda")
    assert r.forward(hid, 4, refine_mask=mask, check=False) == -1            # refine needs row_idx
    big = rs.Router(dev_weights(gen.make_router_weights(64, 300, 16, 1, seed=1)))
    assert big.forward(hid, 4, check=False) == -3
    assert r.forward(hid, 0)[0] is not None                                  # empty batch is fine


def test_router_bad_index_decides_nothing(rs, oracle):
    # an entry of row_idx outside [0, n_src) reads row 0, gets switch 0 and leaves the mask alone
    # (it used to refine sequence 0's decision); rows to read with no row present is an argument error
    import torch
    d, n_src = 128, 6
    w = gen.make_router_weights(d, 16, 32, 2, seed=3)
    router = rs.Router(dev_weights(w))
    hid_bits = gen.f32_to_bf16_bits((np.random.default_rng(1).standard_normal((n_src, d)) * 2.0).astype(np.float32))
    hid = to_dev_bf16(hid_bits)
    idx = np.array([4, -1, 2, 99, 0], dtype=np.int32)
    mask = torch.full((n_src,), 7, dtype=torch.uint8, device="cuda")
    logits, sw = router.forward(hid, idx.size, row_idx=to_dev_i32(idx), refine_mask=mask)
    torch.cuda.synchronize()
    ref_logits, ref_sw = oracle.router_rows(hid_bits, w, row_idx=np.array([4, 0, 2, 0, 0], dtype=np.int32))
    got_sw, got_mask = sw.cpu().numpy()[:idx.size], mask.cpu().numpy()
    assert np.abs(logits.cpu().numpy()[:idx.size] - ref_logits).max() <= LOGIT_TOL
    good = np.array([0, 2, 4])
    assert np.array_equal(got_sw[good], ref_sw[good]) and (got_sw[[1, 3]] == 0).all()
    assert got_mask[4] == ref_sw[0] and got_mask[2] == ref_sw[2] and got_mask[0] == ref_sw[4]
    assert (got_mask[[1, 3, 5]] == 7).all()                      # untouched
    empty = torch.zeros((0, d), dtype=torch.bfloat16, device="cuda")
    assert router.forward(empty, 2, row_idx=to_dev_i32([0, 0]), check=False) == -1
    torch.cuda.synchronize()


def test_read_stream_probe(rs):
    # the measurement aid: whole 16 KiB chunks are read, nothing is written, no bounded wait runs out
    import torch
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    for n in (0, 100, 16 * 1024, 5 * 16 * 1024 + 7, 64 << 20):
        buf = torch.full((n,), 3, dtype=torch.uint8, device="cuda")
        assert rs.probe_read_stream(buf, gave_up) == 0
        torch.cuda.synchronize()
        assert int(gave_up.item()) == 0
        assert n == 0 or (int(buf[0].item()) == 3 and int(buf[-1].item()) == 3)
