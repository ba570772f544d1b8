"""Pins for the fp64 oracle: closed forms, textbook special cases, an
extended-precision brute force and a library log-softmax.  None of these
re-types the oracle's own formula; each would fail on a dropped term, a wrong
sign, a transposed operand or an off-by-one index in the oracle."""
import itertools
import math

import mpmath as mp
import numpy as np
import pytest
import scipy.special
import scipy.stats

import rstitch_inputs as gen

LN5 = {4096: 8.31777, 151936: 11.93121, 152064: 11.93206}     # ln V to five decimals


def bits(x):
    b = gen.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))
    # the pins below rely on inputs that bf16 holds exactly
    assert np.array_equal(gen.bf16_bits_to_f32(b), np.asarray(x, dtype=np.float32))
    return b


def test_bf16_roundtrip_and_rounding():
    # 1 + 2^-8 is a tie between bf16 neighbours 1.0 and 1 + 2^-7: ties go to even (1.0)
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0], dtype=np.float32)
    b = gen.f32_to_bf16_bits(x)
    back = gen.bf16_bits_to_f32(b)
    assert back.tolist() == [1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, -2.5, 0.0]
    assert b[0] == 0x3F80 and b[4] == 0xC020


@pytest.mark.parametrize("V", [2, 3, 4096, 151936, 152064])
def test_uniform_logits_give_ln_v(oracle, V):
    # hidden = 0 => every logit is 0 => H = ln V, H / ln V = 1, greedy token = lowest index
    d = 8
    rng = np.random.default_rng(V)
    w = gen.f32_to_bf16_bits(rng.standard_normal((V, d), dtype=np.float32))
    h = bits(np.zeros((1, d)))
    tok, H, Hn, gap = oracle.head_rows(h, w)
    assert tok[0] == 0 and gap[0] == 0.0
    assert abs(H[0] - math.log(V)) < 1e-9      # plain summation over V terms
    if V in LN5:
        assert abs(H[0] - LN5[V]) < 6e-6
        mp.mp.dps = 40
        assert abs(H[0] - float(mp.log(V))) < 1e-9
    assert abs(Hn[0] - 1.0) < 1e-10
    assert oracle.mask(H, math.log(V) - 1e-6)[0] == 1      # routed for any tau < ln V
    assert oracle.mask(H, math.log(V) + 1e-6)[0] == 0


def test_one_hot_limit(oracle):
    # W[j] = e_1, hidden = a e_1: p_j -> 1 as a grows, H -> 0, tok = j, never routed
    V, d, j = 1000, 16, 613
    w = np.zeros((V, d), dtype=np.float32)
    w[j, 1] = 1.0
    prev = None
    for a in [1.0, 4.0, 16.0, 64.0, 256.0]:
        h = np.zeros((1, d), dtype=np.float32)
        h[0, 1] = a
        tok, H, Hn, gap = oracle.head_rows(bits(h), bits(w))
        assert tok[0] == j and gap[0] == a
        assert H[0] >= 0.0
        if prev is not None:
            assert H[0] < prev
        prev = H[0]
    assert prev < 1e-100
    assert oracle.mask(np.array([prev]), 0.006)[0] == 0


@pytest.mark.parametrize("V,k,a", [(17, 1, 2.0), (4096, 3, 5.0), (4096, 100, 0.5), (151936, 7, 12.0),
                                    (64, 64, 3.0), (1000, 2, -4.0)])
def test_two_level_closed_form(oracle, V, k, a):
    # k rows of W equal e_1, the rest are 0, hidden = a e_1:
    #   p_hi = e^a / (k e^a + V - k),  p_lo = 1 / (k e^a + V - k)
    #   H = -k p_hi ln p_hi - (V - k) p_lo ln p_lo
    d = 8
    rng = np.random.default_rng(V + k)
    rows = np.sort(rng.choice(V, size=k, replace=False))
    w = np.zeros((V, d), dtype=np.float32)
    w[rows, 1] = 1.0
    h = np.zeros((1, d), dtype=np.float32)
    h[0, 1] = a
    tok, H, Hn, gap = oracle.head_rows(bits(h), bits(w))
    mp.mp.dps = 50
    ea = mp.e ** mp.mpf(a)
    Z = k * ea + (V - k)
    p_hi, p_lo = ea / Z, 1 / Z
    H_ref = -k * p_hi * mp.log(p_hi) - (V - k) * p_lo * mp.log(p_lo)
    assert abs(H[0] - float(H_ref)) < 1e-11
    assert abs(Hn[0] - float(H_ref / mp.log(V))) < 1e-12
    if a > 0:
        assert tok[0] == rows[0]                 # ties among the k rows: lowest index
        assert gap[0] == (0.0 if k > 1 else a)
    elif k < V:
        zero_rows = np.setdiff1d(np.arange(V), rows)
        assert tok[0] == zero_rows[0]


@pytest.mark.parametrize("z0,z1", [(0.0, 1.0), (2.5, -3.0), (0.0, 0.0), (-7.0, 9.0)])
def test_v2_is_binary_entropy_of_sigmoid(oracle, z0, z1):
    d = 8
    w = np.zeros((2, d), dtype=np.float32)
    w[0, 0], w[1, 3] = z0, z1
    h = np.zeros((1, d), dtype=np.float32)
    h[0, 0] = h[0, 3] = 1.0
    tok, H, Hn, gap = oracle.head_rows(bits(h), bits(w))
    mp.mp.dps = 50
    q = 1 / (1 + mp.e ** (-(mp.mpf(z1) - mp.mpf(z0))))
    Hb = -(q * mp.log(q) + (1 - q) * mp.log(1 - q))
    assert abs(H[0] - float(Hb)) < 1e-13
    assert tok[0] == (1 if z1 > z0 else 0)
    assert abs(gap[0] - abs(z1 - z0)) == 0.0


def test_contraction_orientation_and_library_log_softmax(oracle):
    # random bf16 inputs; logits against numpy's fp64 matmul over the exactly widened values
    # (a transposed or mis-strided W would fail), entropy against scipy's log_softmax / entropy
    rng = np.random.default_rng(7)
    for V, d, R in [(5, 8, 3), (257, 24, 4), (4096, 256, 2)]:
        w = gen.f32_to_bf16_bits(rng.standard_normal((V, d), dtype=np.float32) * np.float32(0.3))
        h = gen.f32_to_bf16_bits(rng.standard_normal((R, d), dtype=np.float32) * np.float32(2.0))
        zref = gen.bf16_bits_to_f64(h) @ gen.bf16_bits_to_f64(w).T
        tok, H, Hn, gap = oracle.head_rows(h, w)
        for r in range(R):
            z = oracle.logits_row(h[r], w)
            assert np.allclose(z, zref[r], rtol=0, atol=1e-12)
            lp = scipy.special.log_softmax(zref[r])
            H_lib = -np.sum(np.exp(lp) * lp)
            assert abs(H[r] - H_lib) < 1e-11
            assert abs(H[r] - scipy.stats.entropy(scipy.special.softmax(zref[r]))) < 1e-11
            assert tok[r] == int(np.argmax(zref[r]))
            srt = np.sort(zref[r])
            assert abs(gap[r] - (srt[-1] - srt[-2])) < 1e-12
            assert abs(Hn[r] - H_lib / math.log(V)) < 1e-12


@pytest.mark.parametrize("V", [2, 3, 5, 17])
def test_brute_force_extended_precision(oracle, V):
    # direct p = e^z / sum e^z with no max subtraction, 60 digits
    rng = np.random.default_rng(100 + V)
    for d in (8, 16):
        w = gen.f32_to_bf16_bits(rng.standard_normal((V, d), dtype=np.float32))
        h = gen.f32_to_bf16_bits(rng.standard_normal((2, d), dtype=np.float32) * np.float32(3.0))
        tok, H, Hn, gap = oracle.head_rows(h, w)
        mp.mp.dps = 60
        hw, ww = gen.bf16_bits_to_f64(h), gen.bf16_bits_to_f64(w)
        for r in range(2):
            z = [mp.fsum(mp.mpf(float(hw[r, k])) * mp.mpf(float(ww[v, k])) for k in range(d)) for v in range(V)]
            e = [mp.e ** zi for zi in z]
            S = mp.fsum(e)
            Hbf = -mp.fsum((ei / S) * mp.log(ei / S) for ei in e)
            assert abs(H[r] - float(Hbf)) < 1e-12
            assert tok[r] == max(range(V), key=lambda v: (z[v], -v))


def test_invariants_bounds_shift_scale(oracle):
    rng = np.random.default_rng(11)
    V, d = 2048, 32
    w = rng.standard_normal((V, d), dtype=np.float32) * np.float32(0.25)
    w[:, d - 1] = 1.0                       # last column of ones: hidden[d-1] = c shifts every logit by c
    g = rng.standard_normal(d, dtype=np.float32)
    g[d - 1] = 0.0
    wb = gen.f32_to_bf16_bits(w)
    base = None
    for c in [0.0, 4.0, -32.0, 128.0]:
        h = g.copy()
        h[d - 1] = c
        tok, H, Hn, gap = oracle.head_rows(gen.f32_to_bf16_bits(h[None]), wb)
        assert 0.0 <= H[0] <= math.log(V) and 0.0 <= Hn[0] <= 1.0
        if base is None:
            base = (tok[0], H[0], gap[0])
        assert tok[0] == base[0]
        assert abs(H[0] - base[1]) < 1e-10 and abs(gap[0] - base[2]) < 1e-10
    # H is non-increasing in the row scale (dH/ds = -s Var_p(z) <= 0); powers of two keep bf16 exact
    g[d - 1] = 0.0
    gb = gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(g))
    prev = math.inf
    for s in [0.125, 0.5, 1.0, 2.0, 8.0, 32.0]:
        tok, H, Hn, gap = oracle.head_rows(gen.f32_to_bf16_bits((gb * np.float32(s))[None]), wb)
        assert H[0] <= prev + 1e-12
        prev = H[0]


def test_gaussian_logits_small_sigma(oracle):
    # i.i.d. Gaussian logits with std sigma << sqrt(2 ln V): H ~= ln V - sigma^2 / 2
    w = gen.WORKLOADS["c2_slm_b1"]
    small = gen.scaled(w, V=32768, d=256)
    wb = gen.make_w_head(small)
    rng = np.random.default_rng(5)
    for s in (0.5, 1.5):
        g = rng.standard_normal((4, small.d), dtype=np.float32) * np.float32(s)
        hb = gen.f32_to_bf16_bits(g)
        tok, H, Hn, gap = oracle.head_rows(hb, wb)
        hw = gen.bf16_bits_to_f64(hb)
        for r in range(4):
            sigma2 = (small.sigma_w ** 2) * float(hw[r] @ hw[r])   # variance of that row's logits
            assert abs(H[r] - (math.log(small.V) - sigma2 / 2)) < 0.02


def test_rule_is_strict(oracle):
    # Eq. 2 / Algorithm 1: switch iff H > tau; H == tau is not routed
    for H in [0.0, 0.3, 11.93121, 1e-9]:
        assert oracle.rule(H, H) == 0
        assert oracle.rule(H, np.nextafter(H, -np.inf)) == 1
        assert oracle.rule(H, np.nextafter(H, np.inf)) == 0
    assert oracle.rule(float("nan"), 0.3) == 1
    # normalised and un-normalised forms give the same decision on the paper's tau grid
    with open(__file__.rsplit("/", 1)[0] + "/golden/tau_grid.txt") as f:
        grid = [float(t) for line in f if not line.startswith("#") for t in line.split()]
    assert grid == [0.0005, 0.001, 0.005, 0.01, 0.02, 0.03, 0.05]
    rng = np.random.default_rng(3)
    V = 151936
    for H in rng.uniform(0.0, 1.0, size=200):
        for t in grid:
            assert oracle.rule(H, t * math.log(V)) == int(H / math.log(V) > t)


def test_mask_last_row_of_each_span(oracle):
    H = np.array([5.0, 0.1, 0.2, 9.0, 0.05, 7.0, 0.0])
    row_seq = np.array([0, 0, 1, 2, 2, 4, 4], dtype=np.int32)   # sequence 3 has no rows
    m = oracle.mask(H, 0.15, B=5, row_seq=row_seq)
    assert m.tolist() == [0, 1, 0, 0, 0]
    m = oracle.mask(H, 0.15)
    assert m.tolist() == [1, 0, 1, 1, 0, 1, 0]


def test_compaction_all_masks_up_to_12(oracle):
    for B in range(0, 13):
        for bitsv in itertools.product((0, 1), repeat=B) if B <= 10 else \
                [tuple(int(c) for c in np.binary_repr(i, B)) for i in range(0, 1 << B, 7)]:
            m = np.array(bitsv, dtype=np.uint8)
            idx, cnt = oracle.compact(m)
            assert cnt == int(m.sum()) and len(idx) == cnt
            assert all(idx[i] < idx[i + 1] for i in range(cnt - 1))
            assert all(m[i] == 1 for i in idx)
            rest = np.setdiff1d(np.arange(B), idx)
            assert all(m[i] == 0 for i in rest)


@pytest.mark.parametrize("p", [0.1, 0.3, 0.5, 0.7, 0.9])
def test_compaction_random_routing(oracle, p):
    for B in (1, 31, 32, 33, 64, 1000, 4097):
        m = gen.random_mask(B, p, seed=17)
        idx, cnt = oracle.compact(m)
        assert np.array_equal(idx, np.flatnonzero(m).astype(np.int32))
        assert cnt == np.count_nonzero(m)
    assert oracle.compact(np.zeros(9, np.uint8))[1] == 0
    assert oracle.compact(np.ones(9, np.uint8))[0].tolist() == list(range(9))


def test_spans_follow_algorithm_1(oracle):
    # a model whose cache holds L tokens prefills (x + y)[L:], i.e. |x + y| - L rows
    seq_len = np.array([100, 50, 75, 12, 900], dtype=np.int32)
    kv_len = np.array([90, 49, 75, 2, 884], dtype=np.int32)
    idx = np.array([0, 1, 3, 4], dtype=np.int32)
    span, off = oracle.spans(idx, seq_len, kv_len)
    assert span.tolist() == [10, 1, 10, 16]
    assert off.tolist() == [0, 10, 11, 21, 37]
    assert off[-1] == span.sum()
    span, off = oracle.spans(np.zeros(0, np.int32), seq_len, kv_len)
    assert span.size == 0 and off.tolist() == [0]


def test_nan_row_policy(oracle):
    V, d = 64, 8
    rng = np.random.default_rng(2)
    w = gen.f32_to_bf16_bits(rng.standard_normal((V, d), dtype=np.float32))
    h = gen.f32_to_bf16_bits(rng.standard_normal((2, d), dtype=np.float32))
    h[1, 3] = 0x7FC0                                     # quiet NaN
    tok, H, Hn, gap = oracle.head_rows(h, w)
    assert np.isfinite(H[0]) and np.isnan(H[1]) and tok[1] == 0
    assert oracle.mask(H, 100.0).tolist() == [0, 1]


def test_workload_generators_are_deterministic_and_shaped():
    w = gen.scaled(gen.WORKLOADS["c3_llm_b16"], V=512, d=64)
    wb = gen.make_w_head(w)
    assert wb.shape == (512, 64) and wb.dtype == np.uint16
    assert np.array_equal(wb, gen.make_w_head(w))
    assert abs(gen.bf16_bits_to_f64(wb).std() - w.sigma_w) < 0.1 * w.sigma_w
    h0, info = gen.make_hidden(w, wb, step=3)
    h1, _ = gen.make_hidden(w, wb, step=3)
    h2, _ = gen.make_hidden(w, wb, step=4)
    assert h0.shape == (16, 64) and np.array_equal(h0, h1) and not np.array_equal(h0, h2)
    assert (info["scale"] >= w.s_lo).all() and (info["scale"] <= w.s_hi).all()
    k = gen.make_spans(gen.WORKLOADS["c5_catchup"], 0)
    assert k.shape == (64,) and k.min() >= 1 and k.max() <= 16
    sl, kl = gen.make_kv_state(gen.WORKLOADS["c5_catchup"], 0, span=k)
    assert np.array_equal(sl - kl, k)
