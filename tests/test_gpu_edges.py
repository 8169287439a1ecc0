"""Edge cases of the GPU path: very long rows, very many short rows, padded row strides, long drafts,
normalisers recomputed inside svip_verify, masked rows left untouched."""
import numpy as np
import pytest

import svip_testlib as tl
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 17)
    yield c
    c.destroy()


@pytest.mark.parametrize("V,bf16", [(1000003, False), (2000001, True)])
def test_very_long_rows(ctx, oracle, V, bf16):
    rng = np.random.default_rng(V)
    x = (rng.standard_normal((3, V)) * np.array([[0.5], [3.0], [8.0]])).astype(np.float32)
    x = W.to_bf16_bits(x) if bf16 else x
    u = np.array([0.123, 0.5, 0.987], dtype=np.float32)
    for S in (0, 1, 8):
        ctx.set_cluster_size(S)
        for T in (1.0, 0.0):
            got = tl.gpu_draft_step(ctx, x, T, 0.3, u)
            tl.check_draft_against_oracle(oracle, x, T, 0.3, u, got, "V=%d S=%d T=%g" % (V, S, T), threads=3)
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def test_many_short_rows(ctx, oracle):
    """More rows than a grid dimension of 65535: the grid is one-dimensional in blocks, not limited by it."""
    rng = np.random.default_rng(1)
    B, V = 70001, 24
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    u = rng.random(B).astype(np.float32)
    got = tl.gpu_draft_step(ctx, x, 1.0, 0.3, u)
    tl.check_draft_against_oracle(oracle, x, 1.0, 0.3, u, got, "many rows", threads=16)
    got = tl.gpu_draft_step(ctx, W.to_bf16_bits(x), 0.0, 0.3, None)
    tl.check_draft_against_oracle(oracle, W.to_bf16_bits(x), 0.0, 0.3, None, got, "many rows greedy", threads=16)


def test_padded_strides_and_recomputed_normalisers(ctx, oracle):
    """Target and draft rows with padding between them (NaN-poisoned), q_stats not supplied."""
    import torch
    rng = np.random.default_rng(5)
    B, V, K = 7, 3001, 5
    lens = rng.integers(1, K + 1, size=B).astype(np.int32)
    cu = np.concatenate([[0], np.cumsum(lens + 1)]).astype(np.int64)
    Rp, Rq = int(cu[-1]), int(cu[-1]) - B
    base = (rng.standard_normal((Rp, V)) * 2).astype(np.float32)
    tgt = (base + rng.standard_normal((Rp, V)).astype(np.float32) * 0.4).astype(np.float32)
    q = np.concatenate([base[cu[i]:cu[i] + lens[i]] for i in range(B)])
    tok, _, _ = oracle.draft_step(q, 1.0, 0.3, rng.random(Rq))
    tok = tok.astype(np.int32)
    uv, _ = tl.guard_accept_uniforms(oracle, tok, q, tgt, cu, 1.0, rng.random(Rp).astype(np.float32))
    ts, qs = V + 13, V + 5
    tbuf = np.full((Rp, ts), np.nan, dtype=np.float32); tbuf[:, :V] = tgt
    qbuf = np.full((Rq, qs), np.nan, dtype=np.float32); qbuf[:, :V] = q
    d_t, d_q = tl.to_device(tbuf), tl.to_device(qbuf)
    n_acc = torch.zeros(B, dtype=torch.int32, device="cuda"); nxt = torch.zeros(B, dtype=torch.int32, device="cuda")
    for S in (0, 2, 5):
        ctx.set_cluster_size(S)
        ctx.verify(tl.to_device(tok), d_q, qs, None, -1, 0, d_t, ts, 0, tl.to_device(cu.astype(np.int32)), B, K, Rp, V,
                   1.0, tl.to_device(uv), n_acc, nxt)
        torch.cuda.synchronize()
        tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, 1.0, uv, (n_acc.cpu().numpy(), nxt.cpu().numpy()),
                                       "padded strides S=%d" % S)
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def test_long_draft_of_200_tokens(ctx, oracle):
    rng = np.random.default_rng(8)
    K, V = 200, 257
    base = (rng.standard_normal((K + 1, V)) * 2).astype(np.float32)
    tgt = (base + rng.standard_normal((K + 1, V)).astype(np.float32) * 0.05).astype(np.float32)   # nearly always accepted
    q = base[:K].copy()
    tgt[:150] = q[:150]                  # identical rows: accepted for any draw
    cu = np.array([0, K + 1])
    tok, _, _ = oracle.draft_step(q, 1.0, 0.3, rng.random(K))
    tok = tok.astype(np.int32)
    uv, _ = tl.guard_accept_uniforms(oracle, tok, q, tgt, cu, 1.0, rng.random(K + 1).astype(np.float32))
    got, early = tl.gpu_verify(ctx, tok, q, tgt, cu, K, 1.0, uv, fixed_K=True, early_exit=True)
    c = tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, 1.0, uv, got, "K=200")
    assert c["mean_accepted"] >= 150     # the first rejection lies beyond four ballots of 32
    tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, 1.0, uv, early, "K=200 (early exit)")


def test_masked_draft_step_leaves_skipped_rows_alone(ctx, oracle):
    import torch
    rng = np.random.default_rng(4)
    B, V = 9, 5000
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    u = rng.random(B).astype(np.float32)
    active = np.array([1, 0, 1, 1, 0, 0, 1, 0, 1], dtype=np.uint8)
    x[1, :] = np.nan                        # a skipped row is never read: its NaNs must not raise the status
    d = tl.to_device(x)
    tok = torch.full((B,), -3, dtype=torch.int32, device="cuda"); ent = torch.full((B,), -3.0, device="cuda")
    stop = torch.full((B,), 7, dtype=torch.uint8, device="cuda"); stats = torch.full((B, 2), -3.0, device="cuda")
    ctx.draft_step_masked(d, 0, B, V, V, 1.0, 0.3, tl.to_device(u), tl.to_device(active), tok, ent, stop, stats)
    torch.cuda.synchronize()
    on = active.astype(bool)
    t_o, H_o, s_o = oracle.draft_step(x[on], 1.0, 0.3, u[on])
    assert np.array_equal(tok.cpu().numpy()[on], t_o) and np.array_equal(stop.cpu().numpy()[on], s_o)
    assert np.all(tok.cpu().numpy()[~on] == -3) and np.all(ent.cpu().numpy()[~on] == -3.0)
    assert np.all(stop.cpu().numpy()[~on] == 7) and np.all(stats.cpu().numpy()[~on] == -3.0)
    assert ctx.read_status() == 0


def test_a_wait_that_nothing_ends_times_out_with_a_status_bit(ctx, oracle):
    """The blocks of a cluster wait for one another's partial results on an mbarrier, for a bounded time.
    The self-test waits with the same routine on an mbarrier that nothing completes: the wait must run out,
    report SVIP_STATUS_WAIT_TIMEOUT, and leave the context usable (the next draft step is correct)."""
    import time
    import torch
    from paper_2411_18462_b200 import SvipError, binding
    assert ctx.read_status() == 0
    t0 = time.perf_counter()
    ctx.selftest_wait_timeout(2_000_000)          # two milliseconds
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert ctx.read_status() == binding.SVIP_STATUS_WAIT_TIMEOUT
    assert 0.0015 < waited < 1.0, waited
    assert ctx.read_status() == 0                 # reading clears the word
    for bad in (0, -5, 10**9):
        with pytest.raises(SvipError):
            ctx.selftest_wait_timeout(bad)
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((6, 40000)) * 2).astype(np.float32)
    u = rng.random(6).astype(np.float32)
    got = tl.gpu_draft_step(ctx, x, 1.0, 0.3, u)   # clusters of several blocks: the real exchange
    tl.check_draft_against_oracle(oracle, x, 1.0, 0.3, u, got, "after the time-out")
    assert ctx.read_status() == 0
