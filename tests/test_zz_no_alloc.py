"""The allocation-free entry point against the regular one.

rstitch_route_static serves callers that may not call cudaMalloc (a serving engine that owns the
device's memory, a decode loop that cannot take an allocation's synchronisation).  It must give
the same decision as rstitch_route_ex on the same inputs, call after call, although every call
reuses one fixed scratch array that still holds the previous call's data.  This file is collected
last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

import rstitch_inputs as gen
from parity_util import ENT_TOL, to_dev_bf16

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_handle_path_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    from paper_2507_17307_b200 import build
    build.build_library()
    import paper_2507_17307_b200 as rs

    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=30011, d=1024, B=rs.STATIC_MAX_ROWS)
    w_bits = gen.make_w_head(w)
    w_dev = to_dev_bf16(w_bits)
    handle = rs.Handle(64, w.d, w.V)
    # two calls in a row on different batches (the second also with fewer rows, so stale partials
    # of the first call sit in the scratch), then the first batch again
    plan = [(0, w.B), (1, 5), (0, w.B)]
    for step, B in plan:
        hid, _ = gen.make_hidden(w, w_bits, step, rows=B)
        hid_dev = to_dev_bf16(hid)
        ref = rs.route_ex(handle, hid_dev, w_dev, w.tau_nats)
        out = rs.RouteOutputs.allocate(B, B, hid_dev.device)      # caller-owned outputs
        rs.route_static(hid_dev, w_dev, w.tau_nats, out)
        torch.cuda.synchronize()
        ent_a, ent_b = out.ent.cpu().numpy()[:B], ref.ent.cpu().numpy()[:B]
        assert np.abs(ent_a.astype(np.float64) - ent_b).max() <= ENT_TOL
        assert np.array_equal(out.tok.cpu().numpy()[:B], ref.tok.cpu().numpy()[:B])
        clear = np.abs(ent_b - w.tau_nats) > ENT_TOL
        assert np.array_equal(out.mask.cpu().numpy()[:B][clear], ref.mask.cpu().numpy()[:B][clear])
        cnt = int(out.llm_count.item())
        own = np.flatnonzero(out.mask.cpu().numpy()[:B]).astype(np.int32)
        assert cnt == own.size and np.array_equal(out.llm_idx.cpu().numpy()[:cnt], own)
        if clear.all():
            assert cnt == int(ref.llm_count.item())
            assert np.array_equal(out.llm_idx.cpu().numpy()[:cnt], ref.llm_idx.cpu().numpy()[:cnt])
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
