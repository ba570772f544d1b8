"""Seeded synthetic inputs for the R-Stitch routing-decision path.

This module only draws random numbers and packs them as bf16 bit patterns
(numpy uint16).  It holds none of the method's arithmetic: no logits, no
softmax, no entropy, no threshold, no compaction.  Both the CPU oracle and
the CUDA library consume exactly the bits produced here, so neither side
ever sees a value the other side computed.

The five workloads take the LM-head shapes of the Qwen-family models the
paper pairs (Section 4, implementation details) and a heavy-tailed
per-row scale in place of real hidden states; they stand in for the paper's
benchmark prompts, none of which is reproduced here.

Row recipe
----------
A *diffuse* row is ``hidden = s * g`` with ``g ~ N(0, 1)`` and
``s ~ LogUniform(s_lo, s_hi)``: its logits are close to i.i.d. Gaussian and
its entropy is high.  A *peaked* row adds a planted direction,
``hidden = s * g + beta * W[j] / |W[j]|^2``, which lifts the logit of one
vocabulary entry ``j`` by ``beta``; ``beta`` is drawn as
``ln V + (s * sigma_W * sqrt(d))^2 / 2 + delta`` with
``delta ~ Uniform(delta_lo, delta_hi)`` so that some peaked rows fall close to
the routing threshold and most fall far below it.  The share of diffuse rows
is the knob that sets the route rate; the rate actually obtained is measured
by the caller (tests, bench) and reported, never assumed.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "bf16_bits_to_f64", "make_w_head", "make_hidden", "make_spans",
    "make_kv_state", "random_mask", "make_router_weights",
]


# --------------------------------------------------------------------------
# bf16 packing (format conversion only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even), return uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float64 exactly."""
    return bf16_bits_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------
# workload descriptions
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    B: int                  # sequences decided per step
    d: int                  # hidden size
    V: int                  # vocabulary rows of W_head
    sigma_w: float          # std of W_head entries
    s_lo: float             # per-row scale range (log-uniform)
    s_hi: float
    tau_nats: float         # default threshold, nats
    seed: int
    steps: int              # decode steps the workload names
    diffuse_frac: Tuple[float, float] = (1.0, 1.0)  # per-step share of diffuse rows ~ U(lo, hi)
    delta_lo: float = 2.0   # planted-peak margin range (peaked rows only)
    delta_hi: float = 25.0
    span_max: int = 1       # >1: each sequence contributes k ~ U{1..span_max} rows
    note: str = ""
    tau_sweep: Tuple[float, ...] = field(default_factory=tuple)


WORKLOADS: Dict[str, Workload] = {
    # tiny correctness case
    "c1_tiny": Workload("c1_tiny", B=4, d=256, V=4096, sigma_w=0.02, s_lo=0.1, s_hi=10.0,
                        tau_nats=0.5, seed=1001, steps=64,
                        note="tiny: pure scaled Gaussian rows"),
    # SLM head, Qwen2.5-1.5B shape, batch 1: the headline GEMV case
    "c2_slm_b1": Workload("c2_slm_b1", B=1, d=1536, V=151936, sigma_w=0.02, s_lo=0.1, s_hi=10.0,
                          tau_nats=0.3, seed=1002, steps=1024, tau_sweep=(0.1, 0.3, 0.5, 1.0),
                          note="SLM head B=1: pure scaled Gaussian rows"),
    # LLM head, Qwen2.5-7B shape, B in {1, 4, 16}; ~30 % of rows above tau = 0.3
    "c3_llm_b1": Workload("c3_llm_b1", B=1, d=3584, V=152064, sigma_w=0.015, s_lo=0.1, s_hi=10.0,
                          tau_nats=0.3, seed=1003, steps=256, diffuse_frac=(0.2, 0.2), delta_lo=2.0),
    "c3_llm_b4": Workload("c3_llm_b4", B=4, d=3584, V=152064, sigma_w=0.015, s_lo=0.1, s_hi=10.0,
                          tau_nats=0.3, seed=1003, steps=256, diffuse_frac=(0.2, 0.2), delta_lo=2.0),
    "c3_llm_b16": Workload("c3_llm_b16", B=16, d=3584, V=152064, sigma_w=0.015, s_lo=0.1, s_hi=10.0,
                           tau_nats=0.3, seed=1003, steps=256, diffuse_frac=(0.2, 0.2), delta_lo=2.0),
    # batched serving step: SLM head on 64 sequences, then LLM head on the routed subset
    "c4_slm_b64": Workload("c4_slm_b64", B=64, d=1536, V=151936, sigma_w=0.02, s_lo=0.05, s_hi=20.0,
                           tau_nats=0.3, seed=1004, steps=256, diffuse_frac=(0.1, 0.5), delta_lo=2.0),
    "c4_llm_b64": Workload("c4_llm_b64", B=64, d=3584, V=152064, sigma_w=0.015, s_lo=0.05, s_hi=20.0,
                           tau_nats=0.3, seed=1014, steps=256, diffuse_frac=(0.1, 0.5), delta_lo=2.0),
    # 32B-class catch-up: 64 routed sequences x stitched span k ~ U{1..16} rows
    "c5_catchup": Workload("c5_catchup", B=64, d=5120, V=152064, sigma_w=0.012, s_lo=0.1, s_hi=10.0,
                           tau_nats=0.3, seed=1005, steps=64, diffuse_frac=(0.3, 0.3), delta_lo=2.0,
                           span_max=16),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (reduced sizes for the oracle)."""
    return replace(w, **kw)


# --------------------------------------------------------------------------
# generators
# --------------------------------------------------------------------------
def _rng(*key: int) -> np.random.Generator:
    return np.random.default_rng([int(k) & 0xFFFFFFFF for k in key])


def make_w_head(w: Workload, chunk_rows: int = 8192) -> np.ndarray:
    """W_head as bf16 bits, shape [V, d], entries ~ N(0, sigma_w); drawn once per workload."""
    out = np.empty((w.V, w.d), dtype=np.uint16)
    rng = _rng(w.seed, 0x57)
    for v0 in range(0, w.V, chunk_rows):
        v1 = min(w.V, v0 + chunk_rows)
        blk = rng.standard_normal((v1 - v0, w.d), dtype=np.float32)
        blk *= np.float32(w.sigma_w)
        out[v0:v1] = f32_to_bf16_bits(blk)
    return out


def make_hidden(w: Workload, w_head_bits: np.ndarray, step: int,
                rows: Optional[int] = None) -> Tuple[np.ndarray, dict]:
    """Hidden states of one decode step as bf16 bits, shape [rows, d].

    Returns the bits and a dict of what was drawn per row (scale, class,
    planted vocabulary entry), for reporting only.
    """
    R = w.B if rows is None else int(rows)
    rng = _rng(w.seed, 0x48, step)
    frac = rng.uniform(w.diffuse_frac[0], w.diffuse_frac[1])
    hid = np.empty((R, w.d), dtype=np.float32)
    scale = np.empty(R, dtype=np.float64)
    diffuse = np.empty(R, dtype=bool)
    planted = np.full(R, -1, dtype=np.int64)
    for r in range(R):
        rr = _rng(w.seed, 0x48, step, r)
        s = math.exp(rr.uniform(math.log(w.s_lo), math.log(w.s_hi)))
        g = rr.standard_normal(w.d, dtype=np.float32)
        is_diffuse = bool(rr.uniform() < frac)
        row = np.float32(s) * g
        if not is_diffuse:
            j = int(rr.integers(0, w.V))
            wj = bf16_bits_to_f32(w_head_bits[j]).astype(np.float64)
            n2 = float(wj @ wj)
            if n2 > 0.0:
                sig = s * w.sigma_w * math.sqrt(w.d)
                beta = math.log(w.V) + 0.5 * sig * sig + rr.uniform(w.delta_lo, w.delta_hi)
                row = row + (beta / n2 * wj).astype(np.float32)
                planted[r] = j
        hid[r] = row
        scale[r] = s
        diffuse[r] = is_diffuse
    info = {"scale": scale, "diffuse": diffuse, "planted": planted, "diffuse_frac": frac}
    return f32_to_bf16_bits(hid), info


def make_spans(w: Workload, step: int) -> np.ndarray:
    """Stitched-span length per sequence, k_b ~ Uniform{1..span_max}; int32 [B]."""
    rng = _rng(w.seed, 0x53, step)
    return rng.integers(1, w.span_max + 1, size=w.B).astype(np.int32)


def make_kv_state(w: Workload, step: int, span: Optional[np.ndarray] = None,
                  max_len: int = 8192) -> Tuple[np.ndarray, np.ndarray]:
    """(seq_len, kv_len) int32 [B] with seq_len - kv_len = span (default spans of make_spans)."""
    if span is None:
        span = make_spans(replace(w, span_max=max(w.span_max, 16)), step)
    rng = _rng(w.seed, 0x4B, step)
    kv_len = rng.integers(16, max_len - 32, size=w.B).astype(np.int32)
    seq_len = (kv_len + span).astype(np.int32)
    return seq_len, kv_len


def random_mask(B: int, p: float, seed: int) -> np.ndarray:
    """Random routing: each sequence is routed with a fixed probability p; uint8 [B]."""
    rng = _rng(seed, 0x4D, int(round(p * 1000)), B)
    return (rng.uniform(size=B) < p).astype(np.uint8)


def make_router_weights(d: int, h: int = 32, ff: int = 64, n_blocks: int = 6, seed: int = 1) -> dict:
    """Random float32 weights for a router network of the shape the paper sketches (an input projection
    d -> h, n_blocks feed-forward blocks h -> ff -> h, a normalisation and a two-way head); the scales
    keep activations O(1).  Only random draws: no arithmetic of the network lives here."""
    rng = _rng(seed, 0x52)
    n = lambda *shape, s=1.0: (rng.standard_normal(shape) * s).astype(np.float32)
    return {"W_in": n(h, d, s=1.0 / math.sqrt(d)), "b_in": n(h, s=0.1),
            "W1": n(n_blocks, ff, h, s=1.0 / math.sqrt(h)), "b1": n(n_blocks, ff, s=0.1),
            "W2": n(n_blocks, h, ff, s=0.5 / math.sqrt(ff)), "b2": n(n_blocks, h, s=0.1),
            "ln_g": (1.0 + 0.1 * rng.standard_normal(h)).astype(np.float32), "ln_b": n(h, s=0.1),
            "W_out": n(2, h, s=1.0 / math.sqrt(h)), "b_out": n(2, s=0.1)}
