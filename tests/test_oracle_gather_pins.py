"""Pins for the two oracle entry points that address rows through an index list: `head_rows(...,
row_idx=...)` (the LLM head evaluated on the compacted subset) and `sample_rows` (which row id enters
the generator's counter when rows are gathered).  The expected values come from closed forms and from
the single-row functions pinned elsewhere, never from the gathered call itself."""
import math

import mpmath as mp
import numpy as np

import rstitch_inputs as gen


def bits(x):
    b = gen.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))
    assert np.array_equal(gen.bf16_bits_to_f32(b), np.asarray(x, dtype=np.float32))
    return b


def two_level_entropy(a, k, V):
    """k logits equal to a, V - k equal to 0: H in 40-digit arithmetic."""
    mp.mp.dps = 40
    a = mp.mpf(a)
    Z = k * mp.e ** a + (V - k)
    p_hi, p_lo = mp.e ** a / Z, 1 / Z
    return float(-(k * p_hi * mp.log(p_hi) + (V - k) * p_lo * mp.log(p_lo)))


def two_level_case():
    # source row i is a_i e_{c_i}; k_c rows of W equal e_c for three columns c with different k_c and
    # different lowest row, so every source row has its own closed-form entropy and its own token
    V, d = 300, 16
    w = np.zeros((V, d), dtype=np.float32)
    groups = {1: [7, 40, 41], 5: [3, 250], 9: [120, 121, 122, 123, 299]}
    for c, rows in groups.items():
        w[rows, c] = 1.0
    amps = [0.5, 1.0, 2.0, 3.0, 4.0, 6.0, 8.0]
    cols = [1, 5, 9, 1, 5, 9, 1]
    hid = np.zeros((len(amps), d), dtype=np.float32)
    for i, (a, c) in enumerate(zip(amps, cols)):
        hid[i, c] = a
    H = [two_level_entropy(a, len(groups[c]), V) for a, c in zip(amps, cols)]
    tok = [min(groups[c]) for c in cols]
    return bits(hid), bits(w), np.array(H), np.array(tok, dtype=np.int32), V


def test_head_rows_gather_reads_the_indexed_row(oracle):
    hid, w, H, tok, V = two_level_case()
    assert len(set(np.round(H, 6))) == len(H)                    # every source row is told apart
    for idx in ([6, 5, 4, 3, 2, 1, 0],                           # a permutation
                [3, 3, 0, 6, 3],                                 # repeats
                [5, 1, 4, 0],                                    # out of order, a subset
                [2],
                []):
        idx = np.array(idx, dtype=np.int32)
        t, Hn, Hnorm, gap = oracle.head_rows(hid, w, row_idx=idx)
        assert t.shape == (idx.size,) and Hn.shape == (idx.size,)
        assert np.array_equal(t, tok[idx])
        assert np.allclose(Hn, H[idx], rtol=0, atol=1e-12)
        assert np.allclose(Hnorm, H[idx] / math.log(V), rtol=0, atol=1e-12)
        assert (gap == 0.0).all()                                # every maximum is attained k >= 2 times
    # the ungathered call is the identity list
    t0, H0, _, _ = oracle.head_rows(hid, w)
    t1, H1, _, _ = oracle.head_rows(hid, w, row_idx=np.arange(hid.shape[0], dtype=np.int32))
    assert np.array_equal(t0, t1) and np.array_equal(H0, H1)
    assert np.array_equal(t0, tok) and np.allclose(H0, H, rtol=0, atol=1e-12)


def test_head_rows_gather_on_random_rows(oracle):
    # random rows: the gathered call equals the single-row functions applied to the indexed source row
    rng = np.random.default_rng(31)
    V, d, n_src = 257, 24, 9
    w = gen.f32_to_bf16_bits((0.3 * rng.standard_normal((V, d))).astype(np.float32))
    hid = gen.f32_to_bf16_bits((2.0 * rng.standard_normal((n_src, d))).astype(np.float32))
    idx = np.array([8, 0, 8, 3, 5, 5, 1], dtype=np.int32)
    t, H, Hn, gap = oracle.head_rows(hid, w, row_idx=idx)
    wf = gen.bf16_bits_to_f32(w).astype(np.float64)
    hf = gen.bf16_bits_to_f32(hid).astype(np.float64)
    for r, src in enumerate(idx):
        z = wf @ hf[src]                                         # numpy's product on the widened bits
        p = np.exp(z - z.max())
        p /= p.sum()
        assert t[r] == int(np.argmax(z))
        assert abs(H[r] - float(-(p * np.log(p)).sum())) < 1e-10
        top = np.sort(z)
        assert abs(gap[r] - (top[-1] - top[-2])) < 1e-10
    # route() with the list: the mask follows the gathered entropies, in list order
    tau = float(np.median(H))
    out = oracle.route(hid, w, tau, row_idx=idx)
    assert np.array_equal(out["mask"], (H > tau).astype(np.uint8))
    assert np.array_equal(out["llm_idx"], np.flatnonzero(H > tau))


def test_sample_rows_counts_output_rows(oracle):
    # the generator's row id is the OUTPUT row r, with and without a gather: each token equals the
    # single-row draw on the indexed source row's logits with row = r
    rng = np.random.default_rng(5)
    V, d, n_src = 64, 16, 6
    w = gen.f32_to_bf16_bits((0.5 * rng.standard_normal((V, d))).astype(np.float32))
    hid = gen.f32_to_bf16_bits(rng.standard_normal((n_src, d)).astype(np.float32))
    T, seed = 0.8, 0x1234567890
    differs_from_source_id = 0
    for draw in range(12):
        for idx in (None, np.array([4, 4, 0, 5, 2, 4, 1, 3], dtype=np.int32)):
            tok, gap = oracle.sample_rows(hid, w, T, seed, draw, row_idx=idx)
            rows = range(n_src) if idx is None else idx
            assert tok.shape == (len(rows),)
            for r, src in enumerate(rows):
                z = oracle.logits_row(hid[src], w)
                t_r, g_r = oracle.sample_token(z, T, seed, draw, r)
                assert tok[r] == t_r and gap[r] == g_r
                # and from the published pieces: scores z / T - ln(-ln U(seed, draw, r, v))
                s = [z[v] / T - math.log(-math.log(oracle.sample_uniform(seed, draw, r, v))) for v in range(V)]
                assert tok[r] == int(np.argmax(s))
                if idx is not None and src != r:
                    differs_from_source_id += int(oracle.sample_token(z, T, seed, draw, int(src))[0] != tok[r])
    # the pin tells the two conventions apart: with the source row as id many draws would differ
    assert differs_from_source_id > 10
    # equal source rows at different output rows draw different noise
    tok, _ = oracle.sample_rows(hid, w, 50.0, seed, 3, row_idx=np.zeros(32, dtype=np.int32))
    assert len(set(tok.tolist())) > 8
