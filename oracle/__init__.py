"""ctypes front end of the fp64 CPU oracle.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its binding never do.  The arithmetic lives
in ``rstitch_oracle.c`` (plain C, fp64); this file only builds it with gcc,
marshals numpy arrays and returns numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rstitch_oracle.c")
_LIB = os.path.join(_HERE, "librstitch_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-fno-fast-math", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        u16p, i32p, f64p, u8p = (c.POINTER(c.c_uint16), c.POINTER(c.c_int32),
                                 c.POINTER(c.c_double), c.POINTER(c.c_uint8))
        lib.oracle_num_threads.restype = c.c_int
        lib.oracle_logits_row.argtypes = [u16p, u16p, c.c_int, c.c_int, f64p]
        lib.oracle_logits_row.restype = None
        lib.oracle_greedy.argtypes = [f64p, c.c_int, i32p, f64p]
        lib.oracle_greedy.restype = None
        lib.oracle_entropy_nats.argtypes = [f64p, c.c_int]
        lib.oracle_entropy_nats.restype = c.c_double
        lib.oracle_entropy_normalized.argtypes = [f64p, c.c_int]
        lib.oracle_entropy_normalized.restype = c.c_double
        lib.oracle_rule.argtypes = [c.c_double, c.c_double]
        lib.oracle_rule.restype = c.c_uint8
        lib.oracle_head_rows.argtypes = [u16p, i32p, u16p, c.c_int, c.c_int, c.c_int,
                                         i32p, f64p, f64p, f64p]
        lib.oracle_head_rows.restype = None
        lib.oracle_mask.argtypes = [f64p, i32p, c.c_int, c.c_int, c.c_double, u8p]
        lib.oracle_mask.restype = None
        lib.oracle_compact.argtypes = [u8p, c.c_int, i32p, i32p]
        lib.oracle_compact.restype = None
        lib.oracle_spans.argtypes = [i32p, c.c_int32, i32p, i32p, i32p, i32p]
        lib.oracle_spans.restype = None
        u32p = c.POINTER(c.c_uint32)
        lib.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        lib.oracle_philox4x32_10.restype = None
        lib.oracle_sample_uniform.argtypes = [c.c_uint64, c.c_uint64, c.c_uint32, c.c_uint32]
        lib.oracle_sample_uniform.restype = c.c_double
        lib.oracle_sample_token.argtypes = [f64p, c.c_int, c.c_double, c.c_uint64, c.c_uint64, c.c_uint32, i32p, f64p]
        lib.oracle_sample_token.restype = None
        lib.oracle_sample_rows.argtypes = [u16p, i32p, u16p, c.c_int, c.c_int, c.c_int, c.c_double, c.c_uint64,
                                           c.c_uint64, i32p, f64p]
        lib.oracle_sample_rows.restype = None
        f32p = c.POINTER(c.c_float)
        lib.oracle_router_rows.argtypes = [u16p, i32p, c.c_int, c.c_int, c.c_int, c.c_int, c.c_int] + [f32p] * 10 + \
                                          [f64p, u8p]
        lib.oracle_router_rows.restype = None
        lib.oracle_latency_ms.argtypes = [f64p, c.c_int32, c.c_int32]
        lib.oracle_latency_ms.restype = c.c_double
        lib.oracle_alg1_sequence.argtypes = [c.c_int32, c.c_int32, c.c_double, c.c_int32, i32p, f64p, i32p, f64p,
                                             f64p, f64p, u8p, i32p, i32p, i32p, i32p, i32p, f64p, i32p, i32p, i32p,
                                             i32p]
        lib.oracle_alg1_sequence.restype = None
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 inputs are passed as uint16 bit patterns"
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def logits_row(hidden_row: np.ndarray, w_head: np.ndarray) -> np.ndarray:
    """z[v] = sum_k hidden[k] * W_head[v, k] in fp64 (Section 3.1)."""
    h, w = _u16(hidden_row), _u16(w_head)
    V, d = w.shape
    assert h.shape == (d,)
    z = np.empty(V, dtype=np.float64)
    _load().oracle_logits_row(_p(h, ctypes.c_uint16), _p(w, ctypes.c_uint16), d, V,
                              _p(z, ctypes.c_double))
    return z


def greedy(z: np.ndarray):
    """(token, top-2 gap): lowest index of the maximum logit."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    tok, gap = ctypes.c_int32(0), ctypes.c_double(0.0)
    _load().oracle_greedy(_p(z, ctypes.c_double), z.size, ctypes.byref(tok), ctypes.byref(gap))
    return int(tok.value), float(gap.value)


def entropy_nats(z: np.ndarray) -> float:
    """Softmax entropy of a logit vector, nats (numerator of Eq. 1)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    return float(_load().oracle_entropy_nats(_p(z, ctypes.c_double), z.size))


def entropy_normalized(z: np.ndarray) -> float:
    """Eq. 1: entropy / log V."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    return float(_load().oracle_entropy_normalized(_p(z, ctypes.c_double), z.size))


def rule(H: float, tau: float) -> int:
    """Eq. 2 / Algorithm 1: 1 iff H > tau (NaN routes to the LLM)."""
    return int(_load().oracle_rule(float(H), float(tau)))


def head_rows(hidden: np.ndarray, w_head: np.ndarray, row_idx: Optional[np.ndarray] = None):
    """Per-row (tok int32, H nats, H / log V, top-2 gap) for R rows."""
    h, w = _u16(hidden), _u16(w_head)
    V, d = w.shape
    assert h.ndim == 2 and h.shape[1] == d
    if row_idx is not None:
        row_idx = np.ascontiguousarray(row_idx, dtype=np.int32)
        R = row_idx.size
        assert R == 0 or (row_idx.min() >= 0 and row_idx.max() < h.shape[0])
    else:
        R = h.shape[0]
    tok = np.zeros(R, dtype=np.int32)
    H = np.zeros(R, dtype=np.float64)
    Hn = np.zeros(R, dtype=np.float64)
    gap = np.zeros(R, dtype=np.float64)
    if R:
        _load().oracle_head_rows(_p(h, ctypes.c_uint16), _p(row_idx, ctypes.c_int32),
                                 _p(w, ctypes.c_uint16), R, d, V, _p(tok, ctypes.c_int32),
                                 _p(H, ctypes.c_double), _p(Hn, ctypes.c_double),
                                 _p(gap, ctypes.c_double))
    return tok, H, Hn, gap


def mask(H_nats: np.ndarray, tau: float, B: Optional[int] = None,
         row_seq: Optional[np.ndarray] = None) -> np.ndarray:
    """Per-sequence route mask (uint8 [B]); decision row = last row of each span."""
    H = np.ascontiguousarray(H_nats, dtype=np.float64)
    R = H.size
    if B is None:
        B = R
    if row_seq is not None:
        row_seq = np.ascontiguousarray(row_seq, dtype=np.int32)
        assert row_seq.size == R
    out = np.zeros(B, dtype=np.uint8)
    _load().oracle_mask(_p(H, ctypes.c_double), _p(row_seq, ctypes.c_int32), R, B, float(tau),
                        _p(out, ctypes.c_uint8))
    return out


def compact(mask_u8: np.ndarray):
    """(llm_idx int32 [count], count): ascending indices of the routed sequences."""
    m = np.ascontiguousarray(mask_u8, dtype=np.uint8)
    idx = np.zeros(max(m.size, 1), dtype=np.int32)
    cnt = ctypes.c_int32(0)
    _load().oracle_compact(_p(m, ctypes.c_uint8), m.size, _p(idx, ctypes.c_int32), ctypes.byref(cnt))
    return idx[:cnt.value].copy(), int(cnt.value)


def spans(llm_idx: np.ndarray, seq_len: np.ndarray, kv_len: np.ndarray):
    """(llm_span [count], llm_row_off [count + 1]) of the routed sequences."""
    idx = np.ascontiguousarray(llm_idx, dtype=np.int32)
    sl = np.ascontiguousarray(seq_len, dtype=np.int32)
    kl = np.ascontiguousarray(kv_len, dtype=np.int32)
    n = idx.size
    span = np.zeros(max(n, 1), dtype=np.int32)
    off = np.zeros(n + 1, dtype=np.int32)
    _load().oracle_spans(_p(idx, ctypes.c_int32), n, _p(sl, ctypes.c_int32), _p(kl, ctypes.c_int32),
                         _p(span, ctypes.c_int32), _p(off, ctypes.c_int32))
    return span[:n].copy(), off


def route(hidden, w_head, tau_nats, row_idx=None, row_seq=None, B=None, seq_len=None, kv_len=None):
    """The whole decision of one step, as a dict of numpy arrays."""
    tok, H, Hn, gap = head_rows(hidden, w_head, row_idx)
    m = mask(H, tau_nats, B=B, row_seq=row_seq)
    idx, cnt = compact(m)
    out = {"tok": tok, "ent": H, "ent_norm": Hn, "gap": gap, "mask": m,
           "llm_idx": idx, "llm_count": cnt}
    if seq_len is not None:
        out["llm_span"], out["llm_row_off"] = spans(idx, seq_len, kv_len)
    return out


def latency_ms(coef, n_inf: int, n_kv: int) -> float:
    """Eq. 5: a * n_inf * n_kv + b * n_inf^2 + c * n_inf + d, milliseconds; coef = (a, b, c, d)."""
    cf = np.ascontiguousarray(coef, dtype=np.float64)
    assert cf.shape == (4,)
    return float(_load().oracle_latency_ms(_p(cf, ctypes.c_double), int(n_inf), int(n_kv)))


def alg1_sequence(prompt_len: int, t_max: int, tau: float, eos_id: int, tok_slm, ent_slm, tok_llm, ent_llm,
                  coef_slm, coef_llm, switch_slm=None) -> dict:
    """Algorithm 1 for one sequence over recorded (token, entropy) streams of the two models.
    switch_slm (optional uint8 [t_max]): the router's decision per loop index (R-Stitch+), consulted
    only when the SLM's entropy exceeds tau; None is R-Stitch (always switch)."""
    ts = np.ascontiguousarray(tok_slm, dtype=np.int32)
    tl = np.ascontiguousarray(tok_llm, dtype=np.int32)
    es = np.ascontiguousarray(ent_slm, dtype=np.float64)
    el = np.ascontiguousarray(ent_llm, dtype=np.float64)
    assert min(ts.size, tl.size, es.size, el.size) >= t_max
    cs = np.ascontiguousarray(coef_slm, dtype=np.float64)
    cl = np.ascontiguousarray(coef_llm, dtype=np.float64)
    sw = None
    if switch_slm is not None:
        sw = np.ascontiguousarray(switch_slm, dtype=np.uint8)
        assert sw.size >= t_max
    y = np.full(max(t_max, 1), -1, dtype=np.int32)
    i32 = lambda n=1: np.zeros(n, dtype=np.int32)
    n_out, active, L, ln, kept, steps, done, iters = i32(), i32(), i32(2), i32(), i32(2), i32(2), i32(), i32()
    lat = np.zeros(1, dtype=np.float64)
    P = lambda a: _p(a, ctypes.c_int32)
    D = lambda a: _p(a, ctypes.c_double)
    _load().oracle_alg1_sequence(int(prompt_len), int(t_max), float(tau), int(eos_id), P(ts), D(es), P(tl), D(el),
                                 D(cs), D(cl), _p(sw, ctypes.c_uint8), P(y), P(n_out), P(active), P(L), P(ln), D(lat), P(kept), P(steps),
                                 P(done), P(iters))
    n = int(n_out[0])
    return {"y": y[:n].copy(), "n_out": n, "active": int(active[0]), "L_slm": int(L[0]), "L_llm": int(L[1]),
            "len": int(ln[0]), "lat_ms": float(lat[0]), "kept_slm": int(kept[0]), "kept_llm": int(kept[1]),
            "steps_slm": int(steps[0]), "steps_llm": int(steps[1]), "done": int(done[0]), "iters": int(iters[0])}


def philox4x32_10(ctr, key):
    """Philox-4x32-10 (Salmon et al., SC'11): four 32-bit outputs for a 128-bit counter and 64-bit key."""
    c4 = np.ascontiguousarray(ctr, dtype=np.uint32)
    k2 = np.ascontiguousarray(key, dtype=np.uint32)
    assert c4.shape == (4,) and k2.shape == (2,)
    out = np.zeros(4, dtype=np.uint32)
    P = lambda a: a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32))
    _load().oracle_philox4x32_10(P(c4), P(k2), P(out))
    return out


def sample_uniform(seed: int, draw: int, row: int, v: int) -> float:
    """The uniform in (0, 1) attached to vocabulary entry v of row `row` at draw number `draw`."""
    return float(_load().oracle_sample_uniform(int(seed), int(draw), int(row), int(v)))


def sample_token(z: np.ndarray, temperature: float, seed: int, draw: int, row: int):
    """(token, score gap to the runner-up) of the Gumbel-max draw from softmax(z / temperature)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    tok, gap = ctypes.c_int32(0), ctypes.c_double(0.0)
    _load().oracle_sample_token(_p(z, ctypes.c_double), z.size, float(temperature), int(seed), int(draw), int(row),
                                ctypes.byref(tok), ctypes.byref(gap))
    return int(tok.value), float(gap.value)


def sample_rows(hidden, w_head, temperature: float, seed: int, draw: int, row_idx=None):
    """Sampled token and score gap per row (row r draws with row id r)."""
    h, w = _u16(hidden), _u16(w_head)
    V, d = w.shape
    if row_idx is not None:
        row_idx = np.ascontiguousarray(row_idx, dtype=np.int32)
        R = row_idx.size
    else:
        R = h.shape[0]
    tok = np.zeros(R, dtype=np.int32)
    gap = np.zeros(R, dtype=np.float64)
    if R:
        _load().oracle_sample_rows(_p(h, ctypes.c_uint16), _p(row_idx, ctypes.c_int32), _p(w, ctypes.c_uint16), R, d,
                                   V, float(temperature), int(seed), int(draw), _p(tok, ctypes.c_int32),
                                   _p(gap, ctypes.c_double))
    return tok, gap


ROUTER_KEYS = ("W_in", "b_in", "W1", "b1", "W2", "b2", "ln_g", "ln_b", "W_out", "b_out")


def router_rows(hidden, weights: dict, row_idx=None):
    """R-Stitch+ router forward: (logits float64 [R, 2], switch uint8 [R]).  weights holds float32 arrays
    W_in [h, d], b_in [h], W1 [L, ff, h], b1 [L, ff], W2 [L, h, ff], b2 [L, h], ln_g [h], ln_b [h],
    W_out [2, h], b_out [2]."""
    hb = _u16(hidden)
    w = {k: np.ascontiguousarray(weights[k], dtype=np.float32) for k in ROUTER_KEYS}
    h, d = w["W_in"].shape
    L, ff, _ = w["W1"].shape
    assert hb.shape[1] == d and w["W2"].shape == (L, h, ff) and w["W_out"].shape == (2, h)
    if row_idx is not None:
        row_idx = np.ascontiguousarray(row_idx, dtype=np.int32)
        R = row_idx.size
    else:
        R = hb.shape[0]
    logits = np.zeros((max(R, 1), 2), dtype=np.float64)
    sw = np.zeros(max(R, 1), dtype=np.uint8)
    if R:
        _load().oracle_router_rows(_p(hb, ctypes.c_uint16), _p(row_idx, ctypes.c_int32), R, d, h, ff, L,
                                   *[_p(w[k], ctypes.c_float) for k in ROUTER_KEYS],
                                   _p(logits, ctypes.c_double), _p(sw, ctypes.c_uint8))
    return logits[:R], sw[:R]
