"""GPU parity of svip_pair_stats (Eq. 1-6, appendix B) against the fp64 oracle."""
import numpy as np
import pytest

import svip_testlib as tl
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu

# beta and the bounds are O(1); entropies and KL reach ~12 nats: 1e-4 absolute like the entropy of the
# draft step, relative above 1 (gamma can be large when H_q is small)
ATOL = 1e-4
C_BOUND = 0.18


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 13)
    yield c
    c.destroy()


def gpu_pair_stats(ctx, t, q, T, c_bound):
    import torch
    n, V = t.shape
    dt, dq = tl.to_device(t), tl.to_device(q)
    out = torch.full((n, 8), -7.0, dtype=torch.float32, device="cuda")
    ctx.pair_stats(dq, V, dt, V, tl.dtype_code(t), n, V, T, c_bound, out)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


def gpu_pair_stats_given(ctx, t, q, T, c_bound):
    """The same with the rows' normalisers handed over (taken from svip_draft_step's row_stats)."""
    import torch
    n, V = t.shape
    zeros = np.zeros(n, np.float32)
    ps = tl.gpu_draft_step(ctx, t, T, 0.3, zeros)[3]
    qs = tl.gpu_draft_step(ctx, q, T, 0.3, zeros)[3]
    ctx.read_status()                       # rows without mass set the status word there; not under test here
    dt, dq = tl.to_device(t), tl.to_device(q)
    out = torch.full((n, 8), -7.0, dtype=torch.float32, device="cuda")
    ctx.pair_stats_given(dq, V, tl.to_device(qs), dt, V, tl.to_device(ps), tl.dtype_code(t), n, V, T, c_bound, out)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


def check(got, want, label):
    err = np.abs(got - want)
    tol = ATOL * np.maximum(1.0, np.abs(want))
    # gamma = H_qp / H_q inherits the absolute error of both entropies divided by H_q: it is
    # ill-conditioned for near one-hot drafts, and is checked to that condition number
    Hq = np.maximum(want[:, 1], 1e-30)
    tol[:, 4] = ATOL * (1.0 + np.abs(want[:, 4])) / np.minimum(1.0, Hq)
    # the bounds are 1 - sqrt(.) of KL or H_q: near zero the root magnifies the 1e-4 of its argument,
    # so allow what a shift of the argument by ATOL does to the bound (plus ATOL)
    KL = np.where(np.isfinite(want[:, 3]), want[:, 3], 0.0)
    for col, f, x in ((5, lambda k: 1 - np.sqrt(k / 2), KL),
                      (6, lambda k: 1 - np.sqrt(1 - np.exp(-k)), KL),
                      (7, lambda h: 1 - np.sqrt(C_BOUND * h), want[:, 1])):
        lo, hi = np.maximum(x - ATOL, 0.0), x + ATOL
        tol[:, col] = ATOL + np.maximum(np.abs(f(lo) - f(x)), np.abs(f(hi) - f(x)))
    assert not np.isnan(got).any(), label + ": NaN written"
    finite = np.isfinite(want)
    assert np.all(err[finite] <= tol[finite]), "%s: worst %g at %s" % (
        label, (err[finite] / tol[finite]).max(), np.argwhere(~(err <= tol) & finite)[:4].tolist())
    assert np.array_equal(np.isinf(got), np.isinf(want)), label + ": infinities differ"


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("V", [2, 33, 1000, 4099, 32000])
def test_small_shapes(ctx, oracle, V, bf16):
    rng = np.random.default_rng(700 + V + int(bf16))
    n = 6
    d = (rng.standard_normal((n, V)) * rng.uniform(0.3, 5.0, size=(n, 1))).astype(np.float32)
    t = d + (rng.standard_normal((n, V)) * rng.uniform(0.02, 1.5, size=(n, 1))).astype(np.float32)
    t[1] = d[1]                              # identical rows: beta = 1, KL = 0
    if V >= 33:
        d[2, rng.integers(0, V, size=5)] = -np.inf    # draft masks tokens: fine, zero mass
        t[3, 7] = -np.inf                               # target masks a token the draft likes: KL = inf
    if bf16:
        d, t = W.to_bf16_bits(d), W.to_bf16_bits(t)
    for T in (1.0, 0.6):
        for S in (1, 3, 8, 0):
            ctx.set_cluster_size(S)
            got = gpu_pair_stats(ctx, t, d, T, 0.18)
            want = oracle.pair_stats(t, d, T, 0.18, threads=4)
            check(got, want, "V=%d S=%d T=%g" % (V, S, T))
            check(gpu_pair_stats_given(ctx, t, d, T, 0.18), want, "given V=%d S=%d T=%g" % (V, S, T))
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


@pytest.mark.parametrize("name", ["tiny", "chat", "reasoning"])
def test_published_configs(ctx, oracle, name):
    """Every draft position of a configuration against the target row of the same position."""
    w = W.make_workload(name)
    rows_t = np.concatenate([np.arange(w.cu_rows[i], w.cu_rows[i] + w.draft_len[i]) for i in range(w.B)])
    t = np.ascontiguousarray(w.target_logits[rows_t])
    got = gpu_pair_stats(ctx, t, w.q_logits, w.T, 0.18)
    want = oracle.pair_stats(t, w.q_logits, w.T, 0.18, threads=16)
    check(got, want, name)
    check(gpu_pair_stats_given(ctx, t, w.q_logits, w.T, 0.18), want, name + " (normalisers given)")
    # the bounds are bounds (Eq. 3, appendix B), on the GPU's own numbers
    assert np.all(got[:, 0] >= got[:, 5] - 2e-4) and np.all(got[:, 0] >= got[:, 6] - 2e-4)
    print("pair stats", name, "rows", len(want), "mean beta %.3f mean KL %.3f" % (want[:, 0].mean(), want[:, 3].mean()))


def test_one_hot_rows_and_unaligned_pairs(ctx, oracle):
    """A one-hot draft row has H_q = 0: gamma is 1 when the target agrees and +inf otherwise, never NaN.
    Rows that start off a 16-byte boundary (each side with its own phase) take the masking path."""
    import torch
    V = 5003
    rng = np.random.default_rng(8)
    d = (rng.standard_normal((4, V)) * 2).astype(np.float32)
    t = (d + rng.standard_normal((4, V)).astype(np.float32) * 0.5).astype(np.float32)
    d[0] = -np.inf; d[0, 77] = 2.0; t[0] = d[0]                 # both one-hot on the same token
    d[1] = -np.inf; d[1, 9] = 0.0                               # draft one-hot, target spread
    got = gpu_pair_stats(ctx, t, d, 1.0, 0.18)
    want = oracle.pair_stats(t, d, 1.0, 0.18)
    check(got, want, "one-hot")
    assert got[0, 4] == 1.0 and got[1, 4] == np.inf and got[0, 0] == 1.0
    # unaligned: target rows shifted by 1 element, draft rows by 3
    bt = np.full(4 * (V + 5) + 16, np.nan, np.float32); bq = np.full(4 * (V + 7) + 16, np.nan, np.float32)
    for r in range(4):
        bt[1 + r * (V + 5): 1 + r * (V + 5) + V] = t[r]
        bq[3 + r * (V + 7): 3 + r * (V + 7) + V] = d[r]
    dbt, dbq = tl.to_device(bt), tl.to_device(bq)
    out = torch.full((4, 8), -7.0, device="cuda")
    for S in (0, 1, 4):
        ctx.set_cluster_size(S)
        ctx.pair_stats(dbq.data_ptr() + 12, V + 7, dbt.data_ptr() + 4, V + 5, 0, 4, V, 1.0, 0.18, out)
        torch.cuda.synchronize()
        check(out.cpu().numpy().astype(np.float64), want, "unaligned S=%d" % S)
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def test_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    x = torch.zeros(64, device="cuda")
    with pytest.raises(SvipError):
        ctx.pair_stats(x, 8, x, 8, 0, 2, 8, 0.0, 0.18, x)       # T must be positive
    with pytest.raises(SvipError):
        ctx.pair_stats(x, 8, x, 8, 0, -1, 8, 1.0, 0.18, x)
    ctx.pair_stats(x, 8, x, 8, 0, 0, 8, 1.0, 0.18, x)           # nothing to do
