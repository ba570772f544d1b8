"""GPU parity of the batched Algorithm 1 steps (plan / commit kernels and the Eq. 5 latency sum)
against the oracle's per-sequence loop: first on recorded (token, entropy) streams, then end to end
with the routing decision itself producing the tokens and masks on two small LM heads."""
import os

import numpy as np
import pytest

import rstitch_inputs as gen
from parity_util import ENT_TOL, GAP_TOL, to_dev_bf16, to_dev_i32

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "latency_coeffs.txt")


def coeffs():
    out = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            name, a, b, c, d = line.split()
            out[name] = (float(a), float(b), float(c), float(d))
    return out


@pytest.fixture(scope="module")
def rs():
    import torch
    assert torch.cuda.is_available()
    from paper_2507_17307_b200 import build
    build.build_library()
    import paper_2507_17307_b200 as rs
    return rs


def state_to_host(st):
    f = lambda t: t.cpu().numpy()
    B = st.B
    return {"active": f(st.active)[:B], "kv_slm": f(st.kv_slm)[:B], "kv_llm": f(st.kv_llm)[:B],
            "seq_len": f(st.seq_len)[:B], "n_out": f(st.n_out)[:B], "done": f(st.done)[:B], "iters": f(st.iters)[:B],
            "kept": f(st.kept).reshape(2, -1)[:, :B], "steps": f(st.steps).reshape(2, -1)[:, :B],
            "lat_ms": f(st.lat_ms)[:B], "y": f(st.y)[:B]}


def check_against_oracle(oracle, got, b, ref):
    assert got["y"][b][:ref["n_out"]].tolist() == ref["y"].tolist(), b
    assert got["n_out"][b] == ref["n_out"] and got["active"][b] == ref["active"]
    assert (got["kv_slm"][b], got["kv_llm"][b], got["seq_len"][b]) == (ref["L_slm"], ref["L_llm"], ref["len"])
    assert (got["kept"][0][b], got["kept"][1][b]) == (ref["kept_slm"], ref["kept_llm"])
    assert (got["steps"][0][b], got["steps"][1][b]) == (ref["steps_slm"], ref["steps_llm"])
    assert got["iters"][b] == ref["iters"] and got["done"][b] == ref["done"]
    assert got["lat_ms"][b] == pytest.approx(ref["lat_ms"], rel=1e-12, abs=1e-9)


@pytest.mark.parametrize("B,T,seed", [(1, 12, 1), (37, 40, 2), (300, 25, 3), (1000, 9, 4)])
def test_recorded_streams(rs, oracle, B, T, seed):
    import torch
    rng = np.random.default_rng(seed)
    c = coeffs()
    lat = [rs.LatencyModel(*c["SLM-1.5B"]), rs.LatencyModel(*c["LLM-7B"])]
    tau, eos = 0.3, 5
    prompt = rng.integers(1, 2000, size=B).astype(np.int32)
    tok = rng.integers(0, 40, size=(2, B, T)).astype(np.int32)              # 5 = EOS turns up now and then
    ent = rng.choice([0.0, 0.05, tau, np.nextafter(tau, 1.0), 0.9, 6.0], size=(2, B, T))
    st = rs.Alg1State(B, y_cap=T)
    st.init(to_dev_i32(prompt))
    for t in range(T):
        for m in (0, 1):                       # both plans first: a round is one loop iteration per sequence
            st.plan(m, T, lat[m])
        for m in (0, 1):
            n = int(st.run_count[m].item())
            idx = st.run_idx[m].cpu().numpy()[:n]
            n_inf = st.n_inf[m].cpu().numpy()[:n]
            off = st.row_off[m].cpu().numpy()[:n + 1]
            assert (np.diff(idx) > 0).all() and (n_inf >= 1).all()
            assert off[0] == 0 and np.array_equal(np.diff(off), n_inf)
            rows = np.full(max(int(off[n]), 1), -7, dtype=np.int32)        # only span ends carry tokens
            if n:
                rows[off[1:] - 1] = tok[m, idx, t]
            mask = (ent[m, idx, t] > tau).astype(np.uint8) if n else np.zeros(1, np.uint8)
            st.commit(m, to_dev_i32(rows), torch.from_numpy(mask).cuda(), eos)
        if t == 0:
            assert int(st.run_count[0].item()) == B and int(st.run_count[1].item()) == 0     # decoding starts on the SLM
    torch.cuda.synchronize()
    got = state_to_host(st)
    for b in range(B):
        ref = oracle.alg1_sequence(int(prompt[b]), T, tau, eos, tok[0, b], ent[0, b], tok[1, b], ent[1, b],
                                   c["SLM-1.5B"], c["LLM-7B"])
        check_against_oracle(oracle, got, b, ref)
    # one more round: T_max iterations are used up, nothing runs and nothing changes
    for m in (0, 1):
        st.plan(m, T, lat[m])
        assert int(st.run_count[m].item()) == 0 and int(st.row_off[m][0].item()) == 0
    again = state_to_host(st)
    for k in got:
        assert np.array_equal(got[k], again[k]), k


@pytest.mark.parametrize("fused", [False, True])
def test_end_to_end_with_the_routing_decision(rs, oracle, fused):
    # two small heads; the tokens and masks come from rstitch_route_ex on the model's batch of rows.
    # fused: no commit launches and only the first round's plans -- the routing calls carry the decision
    # block in their own tail (alg1_tail), the LLM's call also the next round's planning
    import torch
    B, T, tau, eos = 16, 10, 0.3, -1
    c = coeffs()
    lat = [rs.LatencyModel(*c["SLM-1.5B"]), rs.LatencyModel(*c["LLM-14B"])]
    handle = rs.Handle(512, 64, 512)
    for seed in range(20):
        ws = [gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B * T, d=64, V=512, sigma_w=0.06, seed=8100 + seed,
                         diffuse_frac=(0.4, 0.4)),
              gen.scaled(gen.WORKLOADS["c4_llm_b64"], B=B * T, d=64, V=512, sigma_w=0.06, seed=8200 + seed,
                         diffuse_frac=(0.6, 0.6))]
        w_bits = [gen.make_w_head(w) for w in ws]
        hid = [gen.make_hidden(ws[m], w_bits[m], 0)[0].reshape(B, T, 64) for m in (0, 1)]
        ref_rows = [oracle.route(hid[m].reshape(B * T, 64), w_bits[m], tau) for m in (0, 1)]
        clear = all((np.abs(r["ent"] - tau) > 4 * ENT_TOL).all() for r in ref_rows)
        if clear:
            break
    assert clear, "no seed kept every stream entropy outside the tolerance band"
    tok = [r["tok"].reshape(B, T).copy() for r in ref_rows]
    tie = [(r["gap"] < GAP_TOL).reshape(B, T) for r in ref_rows]      # near-ties: either token is right
    ent = [r["ent"].reshape(B, T) for r in ref_rows]
    w_dev = [to_dev_bf16(w) for w in w_bits]
    rng = np.random.default_rng(77)
    prompt = rng.integers(1, 9, size=B).astype(np.int32)        # short prompts keep the spans small
    st = rs.Alg1State(B, y_cap=T)
    st.init(to_dev_i32(prompt))
    tails = [st.tail(0, eos), st.tail(1, eos, plan_next=True, t_max=T, latency=lat)]
    empty_calls = 0
    for t in range(T):
        if not fused or t == 0:
            for m in (0, 1):
                st.plan(m, T, lat[m])
        counts = [int(st.run_count[m].item()) for m in (0, 1)]      # both read before the LLM call replans
        for m in (0, 1):
            n = counts[m]
            if n == 0:
                if fused:      # no rows, but the loop goes on: the call runs the block on its own
                    rs.route_ex(handle, torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda"), w_dev[m], tau,
                                R=0, B=0, alg1_tail=tails[m])
                    empty_calls += 1
                continue
            idx = st.run_idx[m].cpu().numpy()[:n]
            off = st.row_off[m].cpu().numpy()[:n + 1]
            R = int(off[n])
            rows = gen.f32_to_bf16_bits(rng.standard_normal((R, 64)).astype(np.float32))   # span filler rows
            rows[off[1:] - 1] = hid[m][idx, t]                                            # span ends: the real step
            row_seq = np.repeat(np.arange(n, dtype=np.int32), np.diff(off))
            out = rs.route_ex(handle, to_dev_bf16(rows), w_dev[m], tau, R=R, B=n, row_seq=to_dev_i32(row_seq),
                              alg1_tail=tails[m] if fused else None)
            if not fused:
                st.commit(m, out.tok, out.mask, eos)
            seen = out.tok.cpu().numpy()[off[1:] - 1]
            exact = ~tie[m][idx, t]
            assert np.array_equal(seen[exact], tok[m][idx, t][exact])
            tok[m][idx, t] = seen              # on a near-tie the stream takes the token the GPU chose
    torch.cuda.synchronize()
    got = state_to_host(st)
    routed_any = False
    for b in range(B):
        ref = oracle.alg1_sequence(int(prompt[b]), T, tau, eos, tok[0][b], ent[0][b], tok[1][b], ent[1][b],
                                   c["SLM-1.5B"], c["LLM-14B"])
        check_against_oracle(oracle, got, b, ref)
        routed_any |= ref["steps_llm"] > 0
    assert routed_any, "the workload never handed a step to the LLM"
    assert rs.last_status(handle)["timeouts"] == 0
    assert not fused or empty_calls > 0, "the stand-alone form of the block never ran"
    handle.destroy()


def test_fused_tail_on_both_kernel_families_and_bad_structures(rs, oracle):
    # one round on a single-row-per-entry batch through each head kernel, against plan + call + commit
    import torch
    B, tau, eos = 40, 0.3, 3
    c = coeffs()
    lat = [rs.LatencyModel(*c["SLM-1.5B"]), rs.LatencyModel(*c["LLM-7B"])]
    w = gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=256, V=2053, seed=8300)
    w_bits = gen.make_w_head(w)
    w_dev, hid = to_dev_bf16(w_bits), to_dev_bf16(gen.make_hidden(w, w_bits, 0)[0])
    prompt = to_dev_i32(np.arange(5, 5 + B))
    handle = rs.Handle(512, 256, 4096)
    for flags in (rs.PATH_GEMV, rs.PATH_UMMA):
        ref_st, st = rs.Alg1State(B, y_cap=4), rs.Alg1State(B, y_cap=4)
        for s_ in (ref_st, st):
            s_.init(prompt)
            s_.plan(0, 9, lat[0])
            s_.plan(1, 9, lat[1])
        out = rs.route_ex(handle, hid, w_dev, tau, n_rows_dev=ref_st.run_count[0], flags=flags)
        ref_st.commit(0, out.tok, out.mask, eos, spans=False)
        ref_st.plan(0, 9, lat[0])
        ref_st.plan(1, 9, lat[1])
        tail = st.tail(0, eos, spans=False, plan_next=True, t_max=9, latency=lat)
        rs.route_ex(handle, hid, w_dev, tau, n_rows_dev=st.run_count[0], flags=flags, alg1_tail=tail)
        torch.cuda.synchronize()
        a, b = state_to_host(ref_st), state_to_host(st)
        for k in a:
            assert np.array_equal(a[k], b[k]), (flags, k)
        for m in (0, 1):
            n = int(ref_st.run_count[m].item())
            assert n == int(st.run_count[m].item()) and (m == 0 or n > 0)
            assert torch.equal(ref_st.run_idx[m][:n], st.run_idx[m][:n])
            assert torch.equal(ref_st.row_off[m][:n + 1], st.row_off[m][:n + 1])
            assert torch.equal(ref_st.n_inf[m][:n], st.n_inf[m][:n]) and torch.equal(ref_st.n_kv[m][:n], st.n_kv[m][:n])
    bad = st.tail(0, eos)
    bad.model = 2
    assert rs.route_ex(handle, hid, w_dev, tau, alg1_tail=bad, check=False) == -1
    bad = st.tail(1, eos, plan_next=True, t_max=9, latency=lat)
    bad.next_row_off[1] = None
    assert rs.route_ex(handle, hid, w_dev, tau, alg1_tail=bad, check=False) == -1
    bad = st.tail(0, eos)
    bad.run_count = None
    assert rs.route_ex(handle, hid, w_dev, tau, alg1_tail=bad, check=False) == -1
    handle.destroy()


def test_argument_errors(rs):
    import torch
    st = rs.Alg1State(4, y_cap=4)
    lat = rs.LatencyModel(0, 0, 0, 1)
    L = rs.lib()
    import ctypes as C
    assert L.rstitch_alg1_plan(C.byref(st._c), 4, 2, 4, C.byref(lat), None, None, None, None, None, None) == -1
    p = [st.run_idx[0].data_ptr(), st.run_count[0].data_ptr(), st.n_inf[0].data_ptr(), st.n_kv[0].data_ptr(),
         st.row_off[0].data_ptr()]
    assert L.rstitch_alg1_plan(C.byref(st._c), 4, 0, 4, None, *p, None) == -1
    bad = rs.LatencyModel(float("nan"), 0, 0, 1)
    assert L.rstitch_alg1_plan(C.byref(st._c), 4, 0, 4, C.byref(bad), *p, None) == -1
    assert L.rstitch_alg1_init(None, 4, None, None) == -1
    assert L.rstitch_alg1_commit(C.byref(st._c), 4, 0, None, None, None, None, None, 0, None) == -1
    torch.cuda.synchronize()


def test_fused_loop_replays_from_one_cuda_graph(rs, oracle):
    # several rounds of the hybrid loop -- two routing calls per round, Algorithm 1's decision block and the
    # planning inside them, nothing on the host -- recorded into ONE CUDA graph; replaying it gives the state
    # the same calls give when issued directly, and that state matches the oracle's per-sequence loop
    import torch
    # T_max = the number of rounds: the planning the last LLM call carries then selects nothing, so the state
    # is the one Algorithm 1 leaves after T_max iterations
    B, rounds, tau, eos = 48, 6, 0.3, -1
    c = coeffs()
    lat = [rs.LatencyModel(*c["SLM-1.5B"]), rs.LatencyModel(*c["LLM-7B"])]
    for seed in range(20):
        ws = [gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=256, V=2053, seed=8400 + seed, diffuse_frac=(0.4, 0.4)),
              gen.scaled(gen.WORKLOADS["c4_llm_b64"], B=B, d=320, V=3001, seed=8500 + seed, diffuse_frac=(0.6, 0.6))]
        w_bits = [gen.make_w_head(w) for w in ws]
        # run entry j of a model's batch reads row j of that model's pool in every round
        pools_bits = [gen.make_hidden(ws[m], w_bits[m], 0)[0] for m in (0, 1)]
        refs = [oracle.route(pools_bits[m], w_bits[m], tau) for m in (0, 1)]
        if all((np.abs(r["ent"] - tau) > 4 * ENT_TOL).all() and (r["gap"] > GAP_TOL).all() for r in refs):
            break
    else:
        raise AssertionError("no seed kept every row clear of the tolerance bands")
    w_dev = [to_dev_bf16(b) for b in w_bits]
    pools = [to_dev_bf16(p) for p in pools_bits]
    prompt = to_dev_i32(np.arange(3, 3 + B))
    handles = [rs.Handle(64, 256, 4096), rs.Handle(64, 320, 4096)]
    side = torch.cuda.Stream()

    def make(state):
        tails = [state.tail(0, eos, spans=False), state.tail(1, eos, spans=False, plan_next=True, t_max=rounds, latency=lat)]
        outs = [rs.RouteOutputs.allocate(B, B, "cuda") for _ in (0, 1)]
        calls = [rs.PreparedCall(handles[m], pools[m], w_dev[m], tau, outs[m], n_rows_dev=state.run_count[m],
                                 stream=side, alg1_tail=tails[m]) for m in (0, 1)]
        return calls, tails, outs

    def start(state):
        with torch.cuda.stream(side):
            state.init(prompt, stream=side)
            state.plan(0, rounds, lat[0], stream=side)
            state.plan(1, rounds, lat[1], stream=side)

    direct, graphed = rs.Alg1State(B, y_cap=rounds), rs.Alg1State(B, y_cap=rounds)
    calls_d, keep_d, _ = make(direct)
    start(direct)
    with torch.cuda.stream(side):
        for _ in range(rounds):
            assert calls_d[0].launch() == 0 and calls_d[1].launch() == 0
    side.synchronize()

    calls_g, keep_g, _ = make(graphed)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for _ in range(rounds):
            assert calls_g[0].launch() == 0 and calls_g[1].launch() == 0
    start(graphed)            # the capture ran nothing: the state starts here
    side.synchronize()
    g.replay()
    torch.cuda.synchronize()
    a, b = state_to_host(direct), state_to_host(graphed)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    assert a["kept"][1].sum() > 0 and a["kept"][0].sum() > 0        # both models produced tokens
    # against the oracle: sequence b saw (token, entropy) of pool row j whenever it was run entry j; with
    # every sequence alive in every round the run lists are the ascending ids of each model's sequences,
    # which the oracle's own loop reproduces when fed the per-round streams recorded below
    active = np.zeros(B, dtype=np.int64)
    tok_s = np.zeros((2, B, rounds), dtype=np.int32)
    ent_s = np.zeros((2, B, rounds))
    for t in range(rounds):
        nxt = active.copy()
        for m in (0, 1):
            ids = np.flatnonzero(active == m)
            for j, sid in enumerate(ids):
                tok_s[m, sid, t], ent_s[m, sid, t] = refs[m]["tok"][j], refs[m]["ent"][j]
                routed = refs[m]["ent"][j] > tau
                nxt[sid] = 1 if (m == 0 and routed) or (m == 1 and routed) else 0
        active = nxt
    for sid in range(B):
        ref = oracle.alg1_sequence(3 + sid, rounds, tau, eos, tok_s[0, sid], ent_s[0, sid], tok_s[1, sid], ent_s[1, sid],
                                   c["SLM-1.5B"], c["LLM-7B"])
        check_against_oracle(oracle, a, sid, ref)
    for h in handles:
        assert rs.last_status(h)["timeouts"] == 0
        h.destroy()


def test_rstitch_plus_rounds_with_the_router_in_the_loop(rs, oracle):
    # Algorithm 1 with its R-Stitch+ lines, batched and on the device: a round is the SLM head's call
    # (no decision block of its own), the router on the rows whose entropy exceeded tau -- its last block
    # refines the mask to (H > tau and switch), compacts it and runs the SLM's decision block on it --
    # and the LLM head's call with its decision block and the next planning.  Three launches, no host
    # work; the rounds are issued directly and replayed from one CUDA graph, and the final state is the
    # oracle's per-sequence loop fed the oracle router's switches.
    import torch
    B, rounds, tau, eos = 48, 7, 0.3, -1
    c = coeffs()
    lat = [rs.LatencyModel(*c["SLM-1.5B"]), rs.LatencyModel(*c["LLM-7B"])]
    for seed in range(40):
        ws = [gen.scaled(gen.WORKLOADS["c4_slm_b64"], B=B, d=256, V=2053, seed=8600 + seed, diffuse_frac=(0.6, 0.6)),
              gen.scaled(gen.WORKLOADS["c4_llm_b64"], B=B, d=320, V=3001, seed=8700 + seed, diffuse_frac=(0.6, 0.6))]
        w_bits = [gen.make_w_head(w) for w in ws]
        pools_bits = [gen.make_hidden(ws[m], w_bits[m], 0)[0] for m in (0, 1)]
        refs = [oracle.route(pools_bits[m], w_bits[m], tau) for m in (0, 1)]
        rw = gen.make_router_weights(256, 32, 64, 6, seed=900 + seed)
        r_logits, r_sw = oracle.router_rows(pools_bits[0], rw)
        clear = all((np.abs(r["ent"] - tau) > 4 * ENT_TOL).all() and (r["gap"] > GAP_TOL).all() for r in refs)
        unsure = refs[0]["ent"] > tau
        if clear and (np.abs(r_logits[:, 1] - r_logits[:, 0]) > 1e-3).all() and \
                0 < r_sw[unsure].sum() < unsure.sum():          # the router keeps some rows and hands some over
            break
    else:
        raise AssertionError("no seed kept every row clear of the tolerance bands")
    w_dev = [to_dev_bf16(b) for b in w_bits]
    pools = [to_dev_bf16(p) for p in pools_bits]
    router = rs.Router({k: torch.from_numpy(v).cuda() for k, v in rw.items()})
    prompt = to_dev_i32(np.arange(3, 3 + B))
    handles = [rs.Handle(64, 256, 4096), rs.Handle(64, 320, 4096)]
    side = torch.cuda.Stream()

    def make(state):
        tails = [state.tail(0, eos, spans=False), state.tail(1, eos, spans=False, plan_next=True, t_max=rounds, latency=lat)]
        outs = [rs.RouteOutputs.allocate(B, B, "cuda") for _ in (0, 1)]
        slm = rs.PreparedCall(handles[0], pools[0], w_dev[0], tau, outs[0], n_rows_dev=state.run_count[0], stream=side)
        llm = rs.PreparedCall(handles[1], pools[1], w_dev[1], tau, outs[1], n_rows_dev=state.run_count[1], stream=side,
                              alg1_tail=tails[1])
        bufs = {"logits": torch.zeros((B, 2), dtype=torch.float32, device="cuda"),
                "switch": torch.zeros(B, dtype=torch.uint8, device="cuda"),
                "idx": torch.full((B,), -1, dtype=torch.int32, device="cuda"),
                "cnt": torch.full((1,), -1, dtype=torch.int32, device="cuda")}

        def one_round():
            assert slm.launch() == 0
            router.route(pools[0], B, outs[0].llm_idx, outs[0].mask, bufs["idx"], bufs["cnt"],
                         n_rows_dev=outs[0].llm_count, logits=bufs["logits"], switch=bufs["switch"], stream=side,
                         alg1_tail=tails[0], tok=outs[0].tok, n_seq_dev=state.run_count[0])
            assert llm.launch() == 0
        return one_round, (tails, outs, slm, llm, bufs)

    def start(state):
        with torch.cuda.stream(side):
            state.init(prompt, stream=side)
            state.plan(0, rounds, lat[0], stream=side)
            state.plan(1, rounds, lat[1], stream=side)

    direct, graphed = rs.Alg1State(B, y_cap=rounds), rs.Alg1State(B, y_cap=rounds)
    round_d, keep_d = make(direct)
    start(direct)
    with torch.cuda.stream(side):
        for _ in range(rounds):
            round_d()
    side.synchronize()
    round_g, keep_g = make(graphed)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for _ in range(rounds):
            round_g()
    start(graphed)
    side.synchronize()
    g.replay()
    torch.cuda.synchronize()
    a, b = state_to_host(direct), state_to_host(graphed)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    # the oracle's loop per sequence, fed what each sequence saw: as run entry j of a model's batch it
    # read row j of that model's pool, and on the SLM the router's switch for that row
    active = np.zeros(B, dtype=np.int64)
    tok_s = np.zeros((2, B, rounds), dtype=np.int32)
    ent_s = np.zeros((2, B, rounds))
    sw_s = np.zeros((B, rounds), dtype=np.uint8)
    kept_on_slm_despite_entropy = 0
    for t in range(rounds):
        nxt = active.copy()
        for m in (0, 1):
            for j, sid in enumerate(np.flatnonzero(active == m)):
                tok_s[m, sid, t], ent_s[m, sid, t] = refs[m]["tok"][j], refs[m]["ent"][j]
                unsure_j = refs[m]["ent"][j] > tau
                if m == 0:
                    sw_s[sid, t] = r_sw[j]
                    nxt[sid] = 1 if (unsure_j and r_sw[j]) else 0
                    kept_on_slm_despite_entropy += int(unsure_j and not r_sw[j])
                else:
                    nxt[sid] = 1 if unsure_j else 0
        active = nxt
    assert kept_on_slm_despite_entropy > 0, "the router never overruled the entropy rule"
    differs = 0
    for sid in range(B):
        ref = oracle.alg1_sequence(3 + sid, rounds, tau, eos, tok_s[0, sid], ent_s[0, sid], tok_s[1, sid], ent_s[1, sid],
                                   c["SLM-1.5B"], c["LLM-7B"], switch_slm=sw_s[sid])
        check_against_oracle(oracle, a, sid, ref)
        plain = oracle.alg1_sequence(3 + sid, rounds, tau, eos, tok_s[0, sid], ent_s[0, sid], tok_s[1, sid],
                                     ent_s[1, sid], c["SLM-1.5B"], c["LLM-7B"])
        differs += int(plain["y"].tolist() != ref["y"].tolist() or plain["active"] != ref["active"])
    assert differs > 0, "R-Stitch+ and R-Stitch gave the same trajectories: the test would not tell them apart"
    assert a["kept"][1].sum() > 0 and a["kept"][0].sum() > 0
    for h in handles:
        assert rs.last_status(h)["timeouts"] == 0
        h.destroy()


def test_router_route_alg1_argument_errors(rs):
    import torch
    rw = gen.make_router_weights(64, 16, 32, 2, seed=5)
    router = rs.Router({k: torch.from_numpy(v).cuda() for k, v in rw.items()})
    st = rs.Alg1State(8, y_cap=4)
    hid = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(8, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    mask = torch.zeros(8, dtype=torch.uint8, device="cuda")
    tok = torch.zeros(8, dtype=torch.int32, device="cuda")
    tail = st.tail(1, -1, spans=False)                       # the LLM's block has no business here
    assert router.route(hid, 8, idx, mask, idx.clone(), cnt, alg1_tail=tail, tok=tok, check=False) == -1
    tail = st.tail(0, -1, spans=False)
    assert router.route(hid, 8, idx, mask, idx.clone(), cnt, alg1_tail=tail, tok=None, check=False) == -1
    torch.cuda.synchronize()
