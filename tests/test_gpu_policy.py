"""Device-side drafting loop (masked draft step + policy kernels + packing + verify) against the same
loop run with the oracle on the host, for the paper's rule and its two baselines (Algorithm 1; Section 3)."""
import numpy as np
import pytest

import svip_testlib as tl
from oracle import svip_policy as P
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 12)
    yield c
    c.destroy()


def pools(w):
    """Per-sequence pools of logits: draft [K_max, B, V] (position-major) and target [B][K_max+1, V]."""
    K = w.K_max
    q_pm = np.zeros((K, w.B, w.V), dtype=w.q_logits.dtype)
    t_seq = []
    for i in range(w.B):
        Ki = int(w.draft_len[i]); r0 = int(w.cu_rows[i]) - i
        q_pm[:Ki, i] = w.q_logits[r0:r0 + Ki]
        t = np.zeros((K + 1, w.V), dtype=w.target_logits.dtype)
        t[:Ki + 1] = w.target_logits[w.cu_rows[i]:w.cu_rows[i] + Ki + 1]
        t_seq.append(t)
    return q_pm, t_seq


def host_round(oracle, policy, q_pm, t_seq, T, h, ud, uv_pool, gamma, K_cap):
    """One round with the oracle: returns draft_len, tokens [K,B], n_accepted, next_token, guarded uniforms."""
    K, B, V = q_pm.shape
    draft_len, active = [0] * B, [1] * B
    tok = np.full((K, B), -1, dtype=np.int64)
    for j in range(K_cap):
        rows = [i for i in range(B) if active[i]]
        if not rows:
            break
        t_, _, s_ = oracle.draft_step(np.ascontiguousarray(q_pm[j, rows]), T, h, ud[j, rows])
        stop = [0] * B
        for k, i in enumerate(rows):
            tok[j, i] = t_[k]; stop[i] = int(s_[k])
        P.advance(policy, stop, gamma, draft_len, active, K_cap)
    lens = np.array(draft_len, dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum(lens + 1)]).astype(np.int64)
    q_packed = np.concatenate([q_pm[:lens[i], i] for i in range(B)])
    t_packed = np.concatenate([t_seq[i][:lens[i] + 1] for i in range(B)])
    tok_packed = np.concatenate([tok[:lens[i], i] for i in range(B)]).astype(np.int32)
    uv = np.concatenate([uv_pool[i][:lens[i] + 1] for i in range(B)]).astype(np.float32)
    uv, _ = tl.guard_accept_uniforms(oracle, tok_packed, q_packed, t_packed, cu, T, uv, threads=4)
    n_acc, nxt, _ = oracle.verify(tok_packed, q_packed, t_packed, cu, T, uv.astype(np.float64), threads=4)
    return lens, tok, n_acc, nxt, uv, cu, t_packed


@pytest.mark.parametrize("policy", [P.ENTROPY, P.CONSTANT, P.HEURISTIC])
def test_three_rounds_match_the_host_loop(ctx, oracle, policy):
    import torch
    if policy == P.ENTROPY:
        w = W.make_workload("ragged", B=6, V=4096, K_max=10)
    else:
        w = W.make_workload("chat", B=6, V=4096, K_max=8)
    K_cap, B, V, T, h = w.K_max, w.B, w.V, w.T, w.h
    q_pm, t_seq = pools(w)
    dt = tl.dtype_code(w.q_logits)
    d_q = tl.to_device(q_pm.reshape(K_cap * B, V))
    gamma_h = [5, 2, 8, 3, 1, 6]
    d_gamma = torch.tensor(gamma_h, dtype=torch.int32, device="cuda")
    d_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    d_act = torch.ones(B, dtype=torch.uint8, device="cuda")
    d_nact = torch.zeros(1, dtype=torch.int32, device="cuda")
    d_tok = torch.full((K_cap * B,), -1, dtype=torch.int32, device="cuda")
    d_ent = torch.zeros(K_cap * B, device="cuda"); d_stop = torch.zeros(K_cap * B, dtype=torch.uint8, device="cuda")
    d_stats = torch.zeros(K_cap * B, 2, device="cuda")
    d_cu = torch.zeros(B + 1, dtype=torch.int32, device="cuda")
    d_nacc = torch.zeros(B, dtype=torch.int32, device="cuda"); d_next = torch.zeros(B, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(99 + policy)
    esz = w.q_logits.itemsize
    for rnd in range(3):
        ud = rng.random((K_cap, B)).astype(np.float32)
        uv_pool = [rng.random(K_cap + 1).astype(np.float32) for _ in range(B)]
        lens, tok, n_acc, nxt, uv, cu, t_packed = host_round(oracle, policy, q_pm, t_seq, T, h, ud, uv_pool, gamma_h,
                                                           K_cap)
        # device: the whole drafting loop without looking at anything on the host
        d_ud = tl.to_device(ud.reshape(-1))
        d_tok.fill_(-1)
        for j in range(K_cap):
            o = j * B
            ctx.draft_step_masked(d_q.data_ptr() + o * V * esz, dt, B, V, V, T, h, d_ud.data_ptr() + 4 * o, d_act,
                                  d_tok.data_ptr() + 4 * o, d_ent.data_ptr() + 4 * o, d_stop.data_ptr() + o,
                                  d_stats.data_ptr() + 8 * o)
            ctx.policy_advance(policy, d_stop.data_ptr() + o, d_gamma, d_len, d_act, B, K_cap, d_nact)
        ctx.pack_ragged(d_len, B, K_cap, d_cu)
        torch.cuda.synchronize()
        assert d_nact.item() == 0 and int(d_act.sum()) == 0
        assert np.array_equal(d_len.cpu().numpy(), lens), (policy, rnd, d_len.cpu().numpy(), lens)
        got_tok = d_tok.cpu().numpy().reshape(K_cap, B)
        assert np.array_equal(got_tok, tok), "tokens of skipped rows must stay untouched, drafted ones must match"
        assert np.array_equal(d_cu.cpu().numpy(), cu)
        # the target forward is the host's job: it packs the rows for the lengths the device chose
        d_t = tl.to_device(t_packed); d_uv = tl.to_device(uv)
        ctx.verify(d_tok, d_q, V, d_stats, 1, B, d_t, V, dt, d_cu, B, K_cap, int(cu[-1]), V, T, d_uv, d_nacc, d_next)
        ctx.policy_update(policy, d_nacc, d_len, d_gamma, d_act, B, K_cap)
        torch.cuda.synchronize()
        assert np.array_equal(d_nacc.cpu().numpy(), n_acc) and np.array_equal(d_next.cpu().numpy(), nxt)
        P.update(policy, n_acc.tolist(), lens.tolist(), gamma_h, [0] * B, K_cap)
        assert d_gamma.cpu().tolist() == gamma_h
        assert d_len.cpu().tolist() == [0] * B and d_act.cpu().tolist() == [1] * B
    assert ctx.read_status() == 0


def test_policy_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    i = torch.zeros(4, dtype=torch.int32, device="cuda"); b = torch.zeros(4, dtype=torch.uint8, device="cuda")
    with pytest.raises(SvipError):
        ctx.policy_advance(7, b, i, i, b, 4, 8)
    with pytest.raises(SvipError):
        ctx.policy_advance(P.ENTROPY, None, i, i, b, 4, 8)       # the entropy rule needs the stop flags
    with pytest.raises(SvipError):
        ctx.policy_advance(P.CONSTANT, b, None, i, b, 4, 8)      # the baselines need gamma
    with pytest.raises(SvipError):
        ctx.policy_update(P.HEURISTIC, None, i, i, b, 4, 8)
    ctx.policy_advance(P.ENTROPY, b, None, i, b, 0, 8)           # empty batch
