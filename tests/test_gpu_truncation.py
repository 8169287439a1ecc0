"""svip_row_threshold (top-k / nucleus cut of every row) against the oracle's sorted-row definition."""
import numpy as np
import pytest

import svip_testlib as tl
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu

NUCLEUS_TOL = 1e-5      # in units of the top-k mass, like the CDF tolerance of sampled tokens


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 12)
    yield c
    c.destroy()


def values_of(rows):
    return W.bf16_bits_to_f32(rows).astype(np.float64) if rows.dtype == np.uint16 else rows.astype(np.float64)


def gpu_threshold(ctx, rows, T, k, p, pad_elems=0, row_stride=None):
    import torch
    n, V = rows.shape
    stride = V if row_stride is None else row_stride
    buf = np.zeros(pad_elems + n * stride + 16, dtype=rows.dtype)
    buf[:] = np.nan if rows.dtype == np.float32 else 0x7FC0      # poison between the rows
    for r in range(n):
        buf[pad_elems + r * stride: pad_elems + r * stride + V] = rows[r]
    d = tl.to_device(buf)
    thr = torch.full((n,), 123.0, device="cuda")
    ctx.row_threshold(d.data_ptr() + pad_elems * rows.itemsize, tl.dtype_code(rows), n, V, stride, T, k, p, thr)
    torch.cuda.synchronize()
    return thr.cpu().numpy()


def check(oracle, rows, T, k, p, got, label=""):
    """tau_k is exact.  The nucleus cut is exact unless the running mass comes within NUCLEUS_TOL of top_p at
    the oracle's cut; then the GPU's cut must still satisfy the definition within that tolerance."""
    tau, Zk, _, _ = oracle.threshold(rows, T, k, p, threads=8)
    vals = values_of(rows)
    n_soft = 0
    for r in range(rows.shape[0]):
        v = vals[r]
        want = tau[r] if np.isfinite(tau[r]) else -np.inf
        if (v >= want).all():
            assert (v >= got[r]).all(), "%s row %d: nothing is dropped, got thr %r" % (label, r, got[r])
            continue
        if got[r] == np.float32(want):
            continue
        assert p < 1.0, "%s row %d: top-k cut must be exact: %r vs %r" % (label, r, got[r], want)
        finite = v[np.isfinite(v)]
        w = np.where(np.isfinite(v), np.exp((v - finite.max()) / T), 0.0)
        g = float(got[r])
        assert (v == g).any(), "%s row %d: thr %r is not a logit of the row" % (label, r, g)
        tau_k = np.sort(v)[::-1][k - 1] if 1 <= k < v.size else v.min()
        assert g >= tau_k
        assert w[v >= g].sum() >= (p - NUCLEUS_TOL) * Zk[r], (label, r)
        assert w[v > g].sum() < (p + NUCLEUS_TOL) * Zk[r], (label, r)
        n_soft += 1
    return n_soft


CASES = [(0, 0.9), (50, 1.0), (50, 0.8), (1, 1.0), (0, 0.5), (1000, 0.95), (0, 0.999)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [777, 32000, 152064])
def test_threshold_matches_the_oracle(ctx, oracle, dtype, V):
    rng = np.random.default_rng(V + (dtype == "bf16"))
    n = 12
    x = (rng.standard_normal((n, V)) * rng.uniform(0.3, 6.0, size=(n, 1))).astype(np.float32)
    x[3, rng.integers(0, V)] += 25.0            # a peaked row
    x[4] = 0.0                                  # all equal: one group of ties
    x[5, ::3] = -np.inf                         # dropped tokens in the input
    rows = W.to_bf16_bits(x) if dtype == "bf16" else x
    soft = 0
    for k, p in CASES:
        kk = min(k, V - 1) if k else 0
        got = gpu_threshold(ctx, rows, 1.0, kk, p)
        soft += check(oracle, rows, 1.0, kk, p, got, "V=%d %s k=%d p=%g" % (V, dtype, kk, p))
    assert soft <= 2, "cuts decided inside the tolerance band should be rare: %d" % soft


@pytest.mark.parametrize("S", [1, 2, 3, 5, 8])
def test_every_cluster_size_and_unaligned_rows(ctx, oracle, S):
    rng = np.random.default_rng(40 + S)
    V = 40013
    for dtype in ("f32", "bf16"):
        x = (rng.standard_normal((5, V)) * 2.5).astype(np.float32)
        rows = W.to_bf16_bits(x) if dtype == "bf16" else x
        ctx.set_cluster_size(S)
        try:
            for pad, stride in ((0, V), (3, V + 5), (1, V + 1)):
                got = gpu_threshold(ctx, rows, 0.7, 300, 0.9, pad_elems=pad, row_stride=stride)
                check(oracle, rows, 0.7, 300, 0.9, got, "S=%d %s pad=%d" % (S, dtype, pad))
        finally:
            ctx.set_cluster_size(0)


def test_small_and_degenerate_rows(ctx, oracle):
    rng = np.random.default_rng(9)
    for V in (1, 2, 5, 17, 33, 300):
        x = (rng.standard_normal((4, V)) * 2).astype(np.float32)
        x[1] = x[1, 0]                                  # all tied
        for k, p in ((0, 0.7), (1, 1.0), (2, 0.6), (V - 1, 1.0), (V, 0.9), (V + 5, 1.0)):
            got = gpu_threshold(ctx, x, 1.0, k, p)
            check(oracle, x, 1.0, k, p, got, "V=%d k=%d p=%g" % (V, k, p))
    # signed zeros are one value; NaN counts as a dropped token
    x = np.array([[0.0, -0.0, 1.0, -1.0, np.nan, 0.0, -2.0, 0.5]], dtype=np.float32)
    got = gpu_threshold(ctx, x, 1.0, 3, 1.0)
    assert got[0] == 0.0                                # third largest is a zero; every zero is kept
    y = np.where(np.isnan(x), -np.inf, x).astype(np.float32)
    for k, p in ((2, 1.0), (0, 0.8), (5, 0.9)):
        assert np.array_equal(gpu_threshold(ctx, x, 1.0, k, p), gpu_threshold(ctx, y, 1.0, k, p))
        check(oracle, y, 1.0, k, p, gpu_threshold(ctx, y, 1.0, k, p), "nan row")
    # a row of dropped tokens only: nothing to cut
    z = np.full((1, 64), -np.inf, dtype=np.float32)
    assert gpu_threshold(ctx, z, 1.0, 4, 0.9)[0] == -np.inf


def test_both_off_drops_nothing(ctx):
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((3, 5000)) * 2).astype(np.float32)
    got = gpu_threshold(ctx, x, 1.0, 0, 1.0)
    assert np.all(got == -np.inf)
    # the statistics are then those of the whole row
    import torch
    st = torch.zeros(3, 2, device="cuda"); thr = torch.zeros(3, device="cuda")
    ctx.row_threshold(tl.to_device(x), 0, 3, 5000, 5000, 1.0, 0, 1.0, thr, st)
    torch.cuda.synchronize()
    Z = np.exp(x.astype(np.float64) - x.max(axis=1, keepdims=True)).sum(axis=1)
    assert np.array_equal(st.cpu().numpy()[:, 0], x.max(axis=1)) and np.allclose(st.cpu().numpy()[:, 1], Z, rtol=1e-5)


def test_published_shapes(ctx, oracle):
    """Rows of the ragged (bf16, heavy-tailed scales, planted tokens) and stress (fp32 Zipf) recipes."""
    w = W.make_workload("ragged", B=8)
    rows = np.ascontiguousarray(w.q_logits[:40])
    for k, p in ((0, 0.9), (64, 0.95)):
        check(oracle, rows, w.T, k, p, gpu_threshold(ctx, rows, w.T, k, p), "ragged")
    w = W.make_workload("stress", B=4)
    rows = np.ascontiguousarray(w.q_logits[:16])
    for k, p in ((0, 0.9), (100, 1.0), (4000, 0.99)):
        check(oracle, rows, w.T, k, p, gpu_threshold(ctx, rows, w.T, k, p), "stress")


def test_threshold_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    x = torch.zeros(4, 64, device="cuda"); t = torch.zeros(4, device="cuda")
    for bad in (dict(T=0.0), dict(top_p=0.0), dict(top_k=-1), dict(V=0)):
        a = dict(T=1.0, top_k=3, top_p=0.9, V=64)
        a.update(bad)
        with pytest.raises(SvipError):
            ctx.row_threshold(x, 0, 4, a["V"], 64, a["T"], a["top_k"], a["top_p"], t)
    ctx.row_threshold(x, 0, 0, 64, 64, 1.0, 3, 0.9, t)      # no rows


# ------------------------------------------------------------------ truncated draft step and verify

def gpu_thresholds(ctx, rows, T, k, p, stats=None):
    import torch
    d = tl.to_device(rows)
    thr = torch.empty(rows.shape[0], device="cuda")
    ctx.row_threshold(d, tl.dtype_code(rows), rows.shape[0], rows.shape[1], rows.shape[1], T, k, p, thr, stats)
    torch.cuda.synchronize()
    return d, thr


@pytest.mark.parametrize("dtype,V", [("bf16", 32000), ("f32", 50021), ("bf16", 152064)])
@pytest.mark.parametrize("k,p", [(50, 1.0), (0, 0.9), (200, 0.8)])
def test_filtered_draft_step_matches_the_oracle_on_the_kept_set(ctx, oracle, dtype, V, k, p):
    import torch
    rng = np.random.default_rng(V + k)
    B, T, h = 24, 0.8, 0.3
    x = (rng.standard_normal((B, V)) * rng.uniform(0.3, 5.0, size=(B, 1))).astype(np.float32)
    x[2, rng.integers(0, V)] += 20.0
    rows = W.to_bf16_bits(x) if dtype == "bf16" else x
    u = rng.random(B).astype(np.float32)
    d_rows, thr = gpu_thresholds(ctx, rows, T, k, p)
    check(oracle, rows, T, k, p, thr.cpu().numpy(), "draft rows")
    masked = oracle.mask_below(rows, thr.cpu().numpy().astype(np.float64))     # the kept set the GPU was given
    for S in (0, 1, 3, 8):
        ctx.set_cluster_size(S)
        try:
            tok = torch.full((B,), -7, dtype=torch.int32, device="cuda"); ent = torch.zeros(B, device="cuda")
            stop = torch.zeros(B, dtype=torch.uint8, device="cuda"); stats = torch.zeros(B, 2, device="cuda")
            ctx.draft_step_filtered(d_rows, tl.dtype_code(rows), B, V, V, T, h, tl.to_device(u), None, thr, tok, ent,
                                    stop, stats)
            torch.cuda.synchronize()
        finally:
            ctx.set_cluster_size(0)
        got = (tok.cpu().numpy(), ent.cpu().numpy(), stop.cpu().numpy(), None)
        tl.check_draft_against_oracle(oracle, masked, T, h, u, got, "filtered draft S=%d" % S)
        vals = values_of(rows)
        assert np.all(vals[np.arange(B), got[0]] >= thr.cpu().numpy()), "a sampled token lies outside the kept set"
        # (m, Z) of the truncated distribution
        st = stats.cpu().numpy()
        for b in range(0, B, 5):
            keep = vals[b] >= float(thr[b])
            Z = np.exp((vals[b][keep] - vals[b].max()) / T).sum()
            assert st[b, 0] == np.float32(vals[b].max()) and abs(st[b, 1] - Z) <= 1e-5 * Z
    assert ctx.read_status() == 0


@pytest.mark.parametrize("name,give_stats", [("chat", True), ("chat", False), ("tiny", True)])
@pytest.mark.parametrize("k,p", [(40, 1.0), (0, 0.85), (300, 0.9), (2000, 0.95)])
def test_filtered_verify_matches_the_oracle(ctx, oracle, name, give_stats, k, p):
    import torch
    w = W.make_workload(name, B=8 if name == "chat" else None, K_max=6 if name == "chat" else None)
    B, V, K, T = w.B, w.V, w.K_max, w.T
    dt = tl.dtype_code(w.q_logits)
    d_q, q_thr = gpu_thresholds(ctx, w.q_logits, T, k, p)
    # with give_stats the normalisers of the target rows come from the threshold kernel as well
    p_stats = torch.full((w.n_target_rows, 2), -5.0, device="cuda") if give_stats else None
    d_t, p_thr = gpu_thresholds(ctx, w.target_logits, T, k, p, p_stats)
    if give_stats:
        tv_all = values_of(w.target_logits)
        ps = p_stats.cpu().numpy()
        for r in range(0, w.n_target_rows, 7):
            keep = tv_all[r] >= float(p_thr[r])
            Z = np.exp((tv_all[r][keep] - tv_all[r].max()) / T).sum()
            assert ps[r, 0] == np.float32(tv_all[r].max()) and abs(ps[r, 1] - Z) <= 1e-5 * Z, (r, ps[r], Z)
    qm = oracle.mask_below(w.q_logits, q_thr.cpu().numpy().astype(np.float64))
    tm = oracle.mask_below(w.target_logits, p_thr.cpu().numpy().astype(np.float64))
    # draft tokens from the truncated draft distributions (GPU), with their normalisers
    Rq = w.q_logits.shape[0]
    tok = torch.zeros(Rq, dtype=torch.int32, device="cuda"); ent = torch.zeros(Rq, device="cuda")
    stop = torch.zeros(Rq, dtype=torch.uint8, device="cuda"); stats = torch.zeros(Rq, 2, device="cuda")
    ctx.draft_step_filtered(d_q, dt, Rq, V, V, T, w.h, tl.to_device(w.draft_uniforms.astype(np.float32)), None, q_thr,
                            tok, ent, stop, stats)
    torch.cuda.synchronize()
    tokens = tok.cpu().numpy()
    uv, moved = tl.guard_accept_uniforms(oracle, tokens, qm, tm, w.cu_rows, T, w.verify_uniforms, threads=8)
    n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda"); nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    launches = ctx.launch_count()
    ctx.verify_filtered(tok, d_q, V, stats if give_stats else None, q_thr, -1, 0, d_t, V, p_thr, dt,
                        tl.to_device(w.cu_rows.astype(np.int32)), B, K, w.n_target_rows, V, T, tl.to_device(uv), n_acc, nxt,
                        p_stats=p_stats)
    assert ctx.launch_count() - launches == (1 if give_stats else 3)     # no pass over rows whose (m, Z) is given
    torch.cuda.synchronize()
    got = (n_acc.cpu().numpy(), nxt.cpu().numpy())
    c = tl.check_verify_against_oracle(oracle, tokens, qm, tm, w.cu_rows, T, uv, got, "filtered verify %s" % name)
    # the emitted token is never one that the target's truncation dropped
    tv = values_of(w.target_logits)
    for i in range(B):
        r = int(w.cu_rows[i]) + int(got[0][i])
        assert tv[r, got[1][i]] >= float(p_thr[r])
    assert 0 <= c["mean_accepted"] <= K
    assert ctx.read_status() == 0


def test_filtered_entry_points_reject_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    x = torch.zeros(4, 64, device="cuda"); f = torch.zeros(8, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda"); b = torch.zeros(8, dtype=torch.uint8, device="cuda")
    with pytest.raises(SvipError):
        ctx.draft_step_filtered(x, 0, 4, 64, 64, 1.0, 0.3, f, None, None, i, f, b)       # no thresholds
    with pytest.raises(SvipError):
        ctx.draft_step_filtered(x, 0, 4, 64, 64, 0.0, 0.3, f, None, f, i, f, b)          # greedy has nothing to truncate
    with pytest.raises(SvipError):
        ctx.verify_filtered(i, x, 64, None, None, -1, 0, x, 64, f, 0, None, 1, 1, 2, 64, 1.0, f, i, i)
    with pytest.raises(SvipError):
        ctx.row_threshold(x, 0, 4, 64, 64, 1.0, 3, 0.9, f, f.data_ptr() + 4)                 # stats must be 8-byte aligned


@pytest.mark.parametrize("dtype,V", [("bf16", 32000), ("f32", 50021), ("bf16", 152064), ("f32", 777)])
@pytest.mark.parametrize("k,p", [(50, 1.0), (50, 0.9), (1, 1.0), (0, 0.9), (3000, 0.9)])
def test_truncated_draft_step_in_one_call(ctx, oracle, dtype, V, k, p):
    """svip_draft_step_truncated: thresholds and the truncated draft step together.  With a small k the
    first kernel finishes rows from its candidates; the other cases (nucleus alone, large k, a row of ties)
    fall through to the streaming kernel.  Either way the outputs must match the oracle on the kept set
    that the returned thresholds define, and the thresholds must match the oracle's."""
    import torch
    rng = np.random.default_rng(V * 7 + k)
    B, T, h = 20, 0.8, 0.3
    x = (rng.standard_normal((B, V)) * rng.uniform(0.3, 5.0, size=(B, 1))).astype(np.float32)
    x[2, rng.integers(0, V)] += 20.0
    x[4] = 1.5                                   # one group of ties: the candidates cannot hold it
    rows = W.to_bf16_bits(x) if dtype == "bf16" else x
    u = rng.random(B).astype(np.float32)
    active = np.ones(B, dtype=np.uint8); active[[3, 11]] = 0
    kk = min(k, V - 1) if k else 0
    d_rows = tl.to_device(rows)
    for S in (0, 1, 4, 8):
        ctx.set_cluster_size(S)
        try:
            thr = torch.full((B,), 77.0, device="cuda")
            tok = torch.full((B,), -7, dtype=torch.int32, device="cuda"); ent = torch.full((B,), -1.0, device="cuda")
            stop = torch.full((B,), 9, dtype=torch.uint8, device="cuda"); stats = torch.full((B, 2), -2.0, device="cuda")
            ctx.draft_step_truncated(d_rows, tl.dtype_code(rows), B, V, V, T, h, kk, p, tl.to_device(u),
                                     tl.to_device(active), thr, tok, ent, stop, stats)
            torch.cuda.synchronize()
        finally:
            ctx.set_cluster_size(0)
        on = np.nonzero(active)[0]; off = np.nonzero(active == 0)[0]
        thr_h = thr.cpu().numpy()
        check(oracle, rows[on], T, kk, p, thr_h[on], "truncated step S=%d" % S)
        masked = oracle.mask_below(rows[on], thr_h[on].astype(np.float64))
        got = (tok.cpu().numpy()[on], ent.cpu().numpy()[on], stop.cpu().numpy()[on], None)
        tl.check_draft_against_oracle(oracle, masked, T, h, u[on], got, "truncated step S=%d k=%d p=%g" % (S, kk, p))
        vals = values_of(rows)
        assert np.all(vals[on, got[0]] >= thr_h[on])
        st = stats.cpu().numpy()
        for b in on[::4]:
            keep = vals[b] >= float(thr_h[b])
            Z = np.exp((vals[b][keep] - vals[b].max()) / T).sum()
            assert st[b, 0] == np.float32(vals[b].max()) and abs(st[b, 1] - Z) <= 1e-5 * Z
        # sequences that are not drafting are left alone
        assert np.all(tok.cpu().numpy()[off] == -7) and np.all(ent.cpu().numpy()[off] == -1.0)
        assert np.all(stop.cpu().numpy()[off] == 9)
    assert ctx.read_status() == 0


def test_truncated_draft_step_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    x = torch.zeros(4, 64, device="cuda"); f = torch.zeros(8, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda"); b = torch.zeros(8, dtype=torch.uint8, device="cuda")
    with pytest.raises(SvipError):
        ctx.draft_step_truncated(x, 0, 4, 64, 64, 0.0, 0.3, 5, 0.9, f, None, f, i, f, b)     # greedy
    with pytest.raises(SvipError):
        ctx.draft_step_truncated(x, 0, 4, 64, 64, 1.0, 0.3, 5, 0.9, None, None, f, i, f, b)  # no uniforms
    ctx.draft_step_truncated(x, 0, 0, 64, 64, 1.0, 0.3, 5, 0.9, f, None, f, i, f, b)         # empty batch
