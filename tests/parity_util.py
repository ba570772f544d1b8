"""Shared helpers of the GPU parity tests: run one case through the C ABI and compare it with the
fp64 oracle under the tolerance rules.

Rules (floating point decides integers here, so the exemptions are explicit and counted):
  * entropy: |H_gpu - H_oracle| <= 2e-3 nats for every row;
  * token: bit-exact unless the row's top-2 logit gap (oracle, fp64) is below 1e-3;
  * mask: exact unless |H_oracle - tau| < 2e-3 for the deciding row;
  * llm_idx / llm_count / spans: bit-exact against the oracle when no mask entry is exempt,
    and always bit-exact against the oracle's compaction of the GPU's own mask.
"""
from __future__ import annotations

import numpy as np

ENT_TOL = 2e-3
GAP_TOL = 1e-3


def to_dev_bf16(bits: np.ndarray, device="cuda"):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device)
    return t.view(torch.bfloat16)


def to_dev_i32(a, device="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)


def run_gpu(handle, hid_bits, w_dev, tau, *, row_idx=None, row_seq=None, B=None, seq_len=None,
            kv_len=None, n_rows_dev=None, flags=0, hid_dev=None, R=None, sample=None):
    """One rstitch_route_ex call; returns numpy outputs (full buffers, canaries included)."""
    import torch
    import paper_2507_17307_b200 as rs
    if hid_dev is None:
        hid_dev = to_dev_bf16(hid_bits)
    kw = {}
    if row_idx is not None:
        kw["row_idx"] = to_dev_i32(row_idx)
    if row_seq is not None:
        kw["row_seq"] = to_dev_i32(row_seq)
    if seq_len is not None:
        kw["seq_len"], kw["kv_len"] = to_dev_i32(seq_len), to_dev_i32(kv_len)
    if n_rows_dev is not None:
        kw["n_rows_dev"] = to_dev_i32([n_rows_dev])
    out = rs.route_ex(handle, hid_dev, w_dev, tau, B=B, R=R, flags=flags, sample=sample, **kw)
    torch.cuda.synchronize()
    res = {k: getattr(out, k).cpu().numpy() for k in ("tok", "ent", "mask", "llm_idx", "llm_count")}
    if out.llm_span is not None:
        res["llm_span"] = out.llm_span.cpu().numpy()
        res["llm_row_off"] = out.llm_row_off.cpu().numpy()
    return res


def compare(gpu: dict, ref: dict, tau: float, R: int, B: int, row_seq=None, oracle=None,
            seq_len=None, kv_len=None):
    """Assert parity under the rules above; returns the counts of exempt rows."""
    ent_g, ent_o = gpu["ent"][:R].astype(np.float64), ref["ent"][:R]
    finite = np.isfinite(ent_o)
    err = np.abs(ent_g[finite] - ent_o[finite])
    assert err.size == 0 or err.max() <= ENT_TOL, "entropy off by %g" % err.max()
    assert np.array_equal(np.isnan(ent_g), np.isnan(ent_o))
    tok_exempt = (ref["gap"][:R] < GAP_TOL) | ~finite
    bad_tok = (gpu["tok"][:R] != ref["tok"][:R]) & ~tok_exempt
    assert not bad_tok.any(), "token mismatch at rows %s" % np.flatnonzero(bad_tok)[:8]
    # an exempt row must still hold a near-maximal token: checked by the caller when it matters
    if row_seq is None:
        dec_H = ent_o[:B]
    else:
        dec_H = np.full(B, np.inf)
        for r in range(R):
            if r == R - 1 or row_seq[r + 1] != row_seq[r]:
                dec_H[row_seq[r]] = ent_o[r]
    mask_exempt = np.abs(dec_H - tau) < ENT_TOL
    bad_mask = (gpu["mask"][:B] != ref["mask"][:B]) & ~mask_exempt
    assert not bad_mask.any(), "mask mismatch at %s" % np.flatnonzero(bad_mask)[:8]
    cnt = int(gpu["llm_count"][0])
    if not (gpu["mask"][:B] != ref["mask"][:B]).any():
        assert cnt == ref["llm_count"]
        assert np.array_equal(gpu["llm_idx"][:cnt], ref["llm_idx"])
    own_idx = np.flatnonzero(gpu["mask"][:B]).astype(np.int32)
    assert cnt == own_idx.size and np.array_equal(gpu["llm_idx"][:cnt], own_idx)
    assert (gpu["llm_idx"][cnt:B] == -1).all(), "llm_idx written past llm_count"
    if seq_len is not None:
        span, off = oracle.spans(own_idx, seq_len, kv_len)
        assert np.array_equal(gpu["llm_span"][:cnt], span)
        assert np.array_equal(gpu["llm_row_off"][:cnt + 1], off)
    return {"tok_exempt": int(tok_exempt.sum()), "mask_exempt": int(mask_exempt.sum()),
            "max_ent_err": float(err.max()) if err.size else 0.0,
            "route_rate": float(gpu["mask"][:B].mean()) if B else 0.0}
