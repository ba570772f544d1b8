"""The allocation-free entry point against the regular one and against the oracle.

rstitch_route_static serves callers that may not call cudaMalloc (a serving engine that owns the
device's memory, a decode loop that cannot take an allocation's synchronisation).  It must give
the same decision as rstitch_route_ex on the same inputs, call after call, although every call
reuses one fixed scratch array that still holds the previous call's data, and it must leave the
device's free memory exactly as it found it.  This file is collected last so that a run that
stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

import rstitch_inputs as gen
from parity_util import ENT_TOL, compare, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rs():
    import torch
    assert torch.cuda.is_available()
    from paper_2507_17307_b200 import build
    build.build_library()
    import paper_2507_17307_b200 as rs
    return rs


def static_outputs(rs, hid_dev, w_dev, tau, B):
    import torch
    out = rs.RouteOutputs.allocate(B, B, hid_dev.device)          # caller-owned outputs
    rs.route_static(hid_dev, w_dev, tau, out)
    torch.cuda.synchronize()
    return {k: getattr(out, k).cpu().numpy() for k in ("tok", "ent", "mask", "llm_idx", "llm_count")}


def test_static_scratch_matches_handle_path_twice_in_a_row(rs, oracle):
    import torch
    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=30011, d=1024, B=rs.STATIC_MAX_ROWS)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    handle = rs.Handle(64, w.d, w.V)
    # calls in a row on different batches (the second with fewer rows, so stale partials of the first
    # call sit in the scratch; the third with one row, which takes the streaming kernel), then the
    # first batch again
    plan = [(0, w.B), (1, 5), (2, 1), (0, w.B)]
    for step, B in plan:
        hid, _ = gen.make_hidden(w, w_bits, step, rows=B)
        hid_dev = to_dev_bf16(hid)
        ref = rs.route_ex(handle, hid_dev, w_dev, w.tau_nats)
        out = static_outputs(rs, hid_dev, w_dev, w.tau_nats, B)
        ent_a, ent_b = out["ent"][:B], ref.ent.cpu().numpy()[:B]
        assert np.abs(ent_a.astype(np.float64) - ent_b).max() <= ENT_TOL
        assert np.array_equal(out["tok"][:B], ref.tok.cpu().numpy()[:B])
        clear = np.abs(ent_b - w.tau_nats) > ENT_TOL
        assert np.array_equal(out["mask"][:B][clear], ref.mask.cpu().numpy()[:B][clear])
        cnt = int(out["llm_count"][0])
        own = np.flatnonzero(out["mask"][:B]).astype(np.int32)
        assert cnt == own.size and np.array_equal(out["llm_idx"][:cnt], own)
        if clear.all():
            assert cnt == int(ref.llm_count.item())
            assert np.array_equal(out["llm_idx"][:cnt], ref.llm_idx.cpu().numpy()[:cnt])
        # and against the oracle, under the same rules as every other entry point
        compare(out, oracle.route(hid, w_bits, w.tau_nats), w.tau_nats, B, B)
    # sizes beyond the fixed scratch are refused, and nothing is launched
    big = torch.zeros((rs.STATIC_MAX_ROWS + 1, w.d), dtype=torch.bfloat16, device="cuda")
    out = rs.RouteOutputs.allocate(rs.STATIC_MAX_ROWS + 1, rs.STATIC_MAX_ROWS + 1, big.device)
    assert rs.route_static(big, w_dev, 0.3, out, check=False) == -3
    assert int(out.llm_count.item()) == -1
    # an empty batch is valid
    empty = torch.zeros((0, w.d), dtype=torch.bfloat16, device="cuda")
    out = rs.RouteOutputs.allocate(0, 0, empty.device)
    rs.route_static(empty, w_dev, 0.3, out)
    torch.cuda.synchronize()
    assert int(out.llm_count.item()) == 0
    handle.destroy()


def test_static_entry_on_shapes_the_tensor_core_kernel_does_not_take(rs, oracle):
    # several rows of a shape too small for the tensor-core kernel (d < 64 or V < 256) stay on the
    # streaming kernel; one row always does
    for B, d, V in [(4, 8, 3), (3, 32, 200), (1, 8, 2), (16, 48, 1000), (1, 1024, 30011)]:
        w = gen.scaled(gen.WORKLOADS["c1_tiny"], B=B, d=d, V=V, sigma_w=0.3)
        w_bits = gen.make_w_head(w)
        w_dev = to_dev_bf16(w_bits)
        for step in range(2):
            hid, _ = gen.make_hidden(w, w_bits, step)
            out = static_outputs(rs, to_dev_bf16(hid), w_dev, w.tau_nats, B)
            compare(out, oracle.route(hid, w_bits, w.tau_nats), w.tau_nats, B, B)


def test_static_entry_allocates_nothing(rs):
    # free device memory is the same before and after a few hundred calls of every kind (one row,
    # several rows, a tiny shape), once the first call on the device has resolved the array's address
    import torch
    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=30011, d=1024, B=rs.STATIC_MAX_ROWS)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    tiny = gen.scaled(gen.WORKLOADS["c1_tiny"], B=4, d=8, V=3)
    tiny_w = to_dev_bf16(gen.make_w_head(tiny))
    cases = []
    for B in (rs.STATIC_MAX_ROWS, 1, 5):
        hid, _ = gen.make_hidden(w, w_bits, 0, rows=B)
        hid_dev = to_dev_bf16(hid)
        cases.append((hid_dev, w_dev, rs.RouteOutputs.allocate(B, B, hid_dev.device)))
    hid, _ = gen.make_hidden(tiny, gen.make_w_head(tiny), 0)
    hid_dev = to_dev_bf16(hid)
    cases.append((hid_dev, tiny_w, rs.RouteOutputs.allocate(4, 4, hid_dev.device)))
    for c in cases:                                     # warm-up: every kernel loaded and configured
        rs.route_static(c[0], c[1], 0.3, c[2])
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for i in range(200):
        c = cases[i % len(cases)]
        rs.route_static(c[0], c[1], 0.3, c[2])
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
