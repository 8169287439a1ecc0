"""The drafting loop of Algorithm 1 run on the device: the position-indexed draft step
(svip_draft_step_at) and the loop recorded inside a CUDA graph (svip_graph_loop_begin / _end), against the
same loop run with the oracle on the host."""
import numpy as np
import pytest

import svip_testlib as tl
from oracle import svip_policy as P
from paper_2411_18462_b200 import workloads as W
from test_gpu_policy import host_round, pools

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 12)
    yield c
    c.destroy()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("T", [1.0, 0.0])
def test_draft_step_at_reads_and_writes_the_slot_of_each_sequence(ctx, oracle, dtype, T):
    import torch
    rng = np.random.default_rng(5)
    B, K, V, h = 7, 5, 5003, 0.3
    x = (rng.standard_normal((K, B, V)) * rng.uniform(0.3, 6.0, size=(K, B, 1))).astype(np.float32)
    logits = W.to_bf16_bits(x) if dtype == "bf16" else x
    pos = rng.integers(0, K, size=B).astype(np.int32)
    active = np.array([1, 1, 0, 1, 1, 1, 0], dtype=np.uint8)
    u = rng.random((K, B)).astype(np.float32)
    d_x = tl.to_device(logits.reshape(K * B, V))
    d_tok = torch.full((K * B,), -7, dtype=torch.int32, device="cuda")
    d_ent = torch.full((K * B,), -1.0, device="cuda")
    d_stats = torch.full((K * B, 2), -2.0, device="cuda")
    d_stop = torch.full((B,), 9, dtype=torch.uint8, device="cuda")
    ctx.draft_step_at(d_x, tl.dtype_code(logits), B, V, V, B * V, tl.to_device(pos), B, T, h,
                      tl.to_device(u.reshape(-1)), tl.to_device(active), d_tok, d_ent, d_stop, d_stats)
    torch.cuda.synchronize()
    tok = d_tok.cpu().numpy().reshape(K, B); ent = d_ent.cpu().numpy().reshape(K, B)
    stats = d_stats.cpu().numpy().reshape(K, B, 2); stop = d_stop.cpu().numpy()
    rows = [b for b in range(B) if active[b]]
    sel = np.ascontiguousarray(np.stack([logits[pos[b], b] for b in rows]))
    got = (np.array([tok[pos[b], b] for b in rows]), np.array([ent[pos[b], b] for b in rows]),
           np.array([stop[b] for b in rows]), None)
    tl.check_draft_against_oracle(oracle, sel, T, h, np.array([u[pos[b], b] for b in rows]), got, "draft_step_at")
    # nothing else was written: other slots, and the sequences that are not drafting
    touched = np.zeros((K, B), dtype=bool)
    for b in rows:
        touched[pos[b], b] = True
    assert np.all(tok[~touched] == -7) and np.all(ent[~touched] == -1.0) and np.all(stats[~touched] == -2.0)
    assert np.all(stop[active == 0] == 9)
    # the normalisers land in the same slot: (largest logit, Z) of that row
    for b in rows:
        row = W.bf16_bits_to_f32(sel[rows.index(b)]) if dtype == "bf16" else sel[rows.index(b)]
        m = float(row.max())
        Z = float(np.exp((row.astype(np.float64) - m) / (T if T > 0 else 1.0)).sum())
        assert stats[pos[b], b, 0] == np.float32(m)
        assert abs(stats[pos[b], b, 1] - Z) <= 1e-5 * Z


def record_loop(ctx, st, policy, bufs, dt, B, V, T, h, K_cap, max_iters, fused=True):
    """Records: loop { draft step at each sequence's own position; policy advance } then packing."""
    ctx.graph_begin(st)
    watch = bufs["nact"] if fused else bufs["watch"]
    body = ctx.graph_loop_begin(st, watch, max_iters)
    ctx.draft_step_at(bufs["q"], dt, B, V, V, B * V, bufs["len"], B, T, h, bufs["ud"], bufs["act"], bufs["tok"],
                      bufs["ent"], bufs["stop"], bufs["stats"], stream=body)
    ctx.policy_advance(policy, bufs["stop"], bufs["gamma"], bufs["len"], bufs["act"], B, K_cap, bufs["nact"],
                       stream=body)
    ctx.graph_loop_end()
    ctx.pack_ragged(bufs["len"], B, K_cap, bufs["cu"], stream=st)
    return ctx.graph_end(st)


def make_bufs(torch, q_pm, B, K_cap, gamma_h):
    bufs = {
        "q": tl.to_device(q_pm.reshape(K_cap * B, -1)),
        "gamma": torch.tensor(gamma_h, dtype=torch.int32, device="cuda"),
        "len": torch.zeros(B, dtype=torch.int32, device="cuda"),
        "act": torch.ones(B, dtype=torch.uint8, device="cuda"),
        "nact": torch.zeros(1, dtype=torch.int32, device="cuda"),
        "watch": torch.ones(1, dtype=torch.int32, device="cuda"),
        "tok": torch.full((K_cap * B,), -1, dtype=torch.int32, device="cuda"),
        "ent": torch.zeros(K_cap * B, device="cuda"),
        "stop": torch.zeros(B, dtype=torch.uint8, device="cuda"),
        "stats": torch.zeros(K_cap * B, 2, device="cuda"),
        "ud": torch.zeros(K_cap * B, device="cuda"),
        "cu": torch.zeros(B + 1, dtype=torch.int32, device="cuda"),
    }
    torch.cuda.synchronize()    # filled on the default stream, used on the test's own stream
    return bufs


@pytest.mark.parametrize("policy", [P.ENTROPY, P.CONSTANT, P.HEURISTIC])
def test_graph_loop_drafts_whole_rounds_like_the_host_loop(ctx, oracle, policy):
    """One replay = one whole drafting phase (Algorithm 1's inner loop for B sequences, each stopping at
    its own length) plus the packing; verification follows outside the graph.  Three rounds."""
    import torch
    if policy == P.ENTROPY:
        w = W.make_workload("ragged", B=6, V=4096, K_max=10)
    else:
        w = W.make_workload("chat", B=6, V=4096, K_max=8)
    K_cap, B, V, T, h = w.K_max, w.B, w.V, w.T, w.h
    q_pm, t_seq = pools(w)
    dt = tl.dtype_code(w.q_logits)
    gamma_h = [5, 2, 8, 3, 1, 6]
    bufs = make_bufs(torch, q_pm, B, K_cap, gamma_h)
    d_nacc = torch.zeros(B, dtype=torch.int32, device="cuda"); d_next = torch.zeros(B, dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()
    launches_before = ctx.launch_count()
    graph = record_loop(ctx, st, policy, bufs, dt, B, V, T, h, K_cap, max_iters=K_cap)
    assert ctx.launch_count() - launches_before == 3    # the advance kernel decides the loop itself
    rng = np.random.default_rng(99 + policy)
    with torch.cuda.stream(st):
        for rnd in range(3):
            ud = rng.random((K_cap, B)).astype(np.float32)
            uv_pool = [rng.random(K_cap + 1).astype(np.float32) for _ in range(B)]
            lens, tok, n_acc, nxt, uv, cu, t_packed = host_round(oracle, policy, q_pm, t_seq, T, h, ud, uv_pool,
                                                               gamma_h, K_cap)
            bufs["ud"].copy_(torch.from_numpy(ud.reshape(-1)))
            bufs["tok"].fill_(-1)
            graph.launch(st)
            st.synchronize()
            assert bufs["nact"].item() == 0 and int(bufs["act"].sum()) == 0
            assert np.array_equal(bufs["len"].cpu().numpy(), lens), (policy, rnd, bufs["len"].cpu().numpy(), lens)
            assert np.array_equal(bufs["tok"].cpu().numpy().reshape(K_cap, B), tok)
            assert np.array_equal(bufs["cu"].cpu().numpy(), cu)
            d_t = tl.to_device(t_packed); d_uv = tl.to_device(uv)
            ctx.verify(bufs["tok"], bufs["q"], V, bufs["stats"], 1, B, d_t, V, dt, bufs["cu"], B, K_cap, int(cu[-1]),
                       V, T, d_uv, d_nacc, d_next, stream=st)
            ctx.policy_update(policy, d_nacc, bufs["len"], bufs["gamma"], bufs["act"], B, K_cap, stream=st)
            st.synchronize()
            assert np.array_equal(d_nacc.cpu().numpy(), n_acc) and np.array_equal(d_next.cpu().numpy(), nxt)
            P.update(policy, n_acc.tolist(), lens.tolist(), gamma_h, [0] * B, K_cap)
            assert bufs["gamma"].cpu().tolist() == gamma_h
    graph.destroy()
    assert ctx.read_status() == 0


def test_loop_never_runs_more_than_max_iters(ctx):
    """The iteration limit holds whatever the data say, and counts from zero at every replay."""
    import torch
    w = W.make_workload("chat", B=4, V=2048, K_max=8)
    K_cap, B, V = w.K_max, w.B, w.V
    q_pm, _ = pools(w)
    bufs = make_bufs(torch, q_pm, B, K_cap, [8, 8, 2, 8])
    st = torch.cuda.Stream()
    graph = record_loop(ctx, st, P.CONSTANT, bufs, tl.dtype_code(w.q_logits), B, V, w.T, w.h, K_cap, max_iters=3)
    with torch.cuda.stream(st):
        for _ in range(2):
            bufs["len"].zero_(); bufs["act"].fill_(1)
            graph.launch(st)
            st.synchronize()
            assert bufs["len"].cpu().tolist() == [3, 3, 2, 3]
            assert bufs["nact"].item() == 3
    graph.destroy()


@pytest.mark.parametrize("watch_value,expect", [(0, 1), (1, 5)])
def test_loop_decided_by_its_own_kernel(ctx, watch_value, expect):
    """A body without a policy step on the loop's counter: svip_graph_loop_end adds the deciding
    kernel.  The counter is a constant here, so the body runs once (0) or max_iters times (1)."""
    import torch
    w = W.make_workload("chat", B=4, V=2048, K_max=8)
    K_cap, B, V = w.K_max, w.B, w.V
    q_pm, _ = pools(w)
    bufs = make_bufs(torch, q_pm, B, K_cap, [8, 8, 8, 8])
    bufs["watch"].fill_(watch_value)
    st = torch.cuda.Stream()
    before = ctx.launch_count()
    graph = record_loop(ctx, st, P.CONSTANT, bufs, tl.dtype_code(w.q_logits), B, V, w.T, w.h, K_cap, max_iters=5,
                        fused=False)
    assert ctx.launch_count() - before == 4
    with torch.cuda.stream(st):
        graph.launch(st)
        st.synchronize()
    assert bufs["len"].cpu().tolist() == [expect] * B
    graph.destroy()


def test_loop_state_errors(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()
    with pytest.raises(SvipError):
        ctx.graph_loop_begin(st, n, 4)          # not recording
    with pytest.raises(SvipError):
        ctx.graph_loop_end()
    ctx.graph_begin(st)
    with pytest.raises(SvipError):
        ctx.graph_loop_begin(st, n, 0)          # needs a positive limit
    ctx.graph_loop_begin(st, n, 4)
    with pytest.raises(SvipError):
        ctx.graph_loop_begin(st, n, 4)          # no nesting
    with pytest.raises(SvipError):
        ctx.graph_end(st)                       # body left open: no graph is handed out
    # the context records and replays normally afterwards
    gamma = torch.full((4,), 3, dtype=torch.int32, device="cuda")
    lens = torch.zeros(4, dtype=torch.int32, device="cuda"); b = torch.ones(4, dtype=torch.uint8, device="cuda")
    ctx.graph_begin(st)
    ctx.policy_advance(P.CONSTANT, None, gamma, lens, b, 4, 8, n, stream=st)
    g = ctx.graph_end(st)
    with torch.cuda.stream(st):
        g.launch(st)
        st.synchronize()
    g.destroy()
    assert lens.cpu().tolist() == [1] * 4 and n.item() == 4
