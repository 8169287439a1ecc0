"""GPU parity of svip_verify and svip_pack_ragged (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest

import svip_testlib as tl
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 14)
    yield c
    c.destroy()


def small_case(rng, B, V, K_max, bf16, noise=0.5, ragged=True):
    lens = rng.integers(1, K_max + 1, size=B).astype(np.int32) if ragged else np.full(B, K_max, np.int32)
    cu = np.concatenate([[0], np.cumsum(lens + 1)]).astype(np.int64)
    Rp = int(cu[-1]); Rq = Rp - B
    scale = np.exp(rng.uniform(np.log(0.3), np.log(6.0), size=(Rp, 1)))
    base = (rng.standard_normal((Rp, V)) * scale).astype(np.float32)
    tgt = base + (rng.standard_normal((Rp, V)) * noise).astype(np.float32)
    q = np.empty((Rq, V), np.float32)
    for i in range(B):
        q[cu[i] - i: cu[i] - i + lens[i]] = base[cu[i]: cu[i] + lens[i]]
    if bf16:
        q = W.to_bf16_bits(q); tgt = W.to_bf16_bits(tgt)
    return lens, cu, q, tgt, rng.random(Rq).astype(np.float32), rng.random(Rp).astype(np.float32)


def run_case(ctx, oracle, lens, cu, q, tgt, ud, uv, T, K_max, label, with_stats=True, fixed=False):
    tok, _, _ = oracle.draft_step(q, T, 0.3, ud, threads=8)
    tok = tok.astype(np.int32)
    uv, moved = tl.guard_accept_uniforms(oracle, tok, q, tgt, cu, T, uv)
    stats = None
    if with_stats and T > 0:
        stats = tl.gpu_draft_step(ctx, q, T, 0.3, ud)[3]
    got, early = tl.gpu_verify(ctx, tok, q, tgt, cu, K_max, T, uv if T > 0 else None, q_stats=stats, fixed_K=fixed,
                               early_exit=True)
    tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, T, uv, early, label + " (early exit)")
    return tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, T, uv, got, label)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("V", [2, 8, 33, 1000, 4099, 32000])
def test_small_ragged_all_cluster_sizes(ctx, oracle, V, bf16):
    rng = np.random.default_rng(4000 + V + int(bf16))
    lens, cu, q, tgt, ud, uv = small_case(rng, 6, V, 5, bf16)
    for T in (1.0, 0.7, 0.0):
        for S in (1, 2, 3, 4, 5, 6, 7, 8, 0):
            ctx.set_cluster_size(S)
            run_case(ctx, oracle, lens, cu, q, tgt, ud, uv, T, 5, "V=%d S=%d T=%g" % (V, S, T),
                     with_stats=(S % 2 == 0))
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def test_fixed_k_and_long_drafts(ctx, oracle):
    rng = np.random.default_rng(9)
    for K in (1, 3, 40, 64, 70):
        lens, cu, q, tgt, ud, uv = small_case(rng, 3, 300, K, False, noise=0.15, ragged=False)
        for T in (1.0, 0.0):
            c = run_case(ctx, oracle, lens, cu, q, tgt, ud, uv, T, K, "K=%d T=%g" % (K, T), fixed=True)
    assert ctx.read_status() == 0


def test_all_accept_gives_bonus_and_reject_at_zero(ctx, oracle):
    rng = np.random.default_rng(10)
    lens, cu, q, tgt, ud, uv = small_case(rng, 4, 2000, 6, True)
    # target == draft on every draft position: every token accepted for any uniform
    for i in range(4):
        tgt[cu[i]: cu[i] + lens[i]] = q[cu[i] - i: cu[i] - i + lens[i]]
    tok, _, _ = oracle.draft_step(q, 1.0, 0.3, ud)
    uv2 = uv.copy(); uv2[:] = 1.0 - 2.0 ** -24
    got = tl.gpu_verify(ctx, tok.astype(np.int32), q, tgt, cu, 6, 1.0, uv2)
    assert np.array_equal(got[0], lens)
    tl.check_verify_against_oracle(oracle, tok.astype(np.int32), q, tgt, cu, 1.0, uv2, got, "all-accept")
    # p(x) = 0 at the first draft token: rejected at position 0 whatever the uniform
    tgt2 = W.bf16_bits_to_f32(tgt).copy()
    for i in range(4):
        tgt2[cu[i], tok[cu[i] - i]] = -np.inf
    tgt2 = W.to_bf16_bits(tgt2)
    uv3 = uv.copy(); uv3[cu[:-1]] = 0.0
    got = tl.gpu_verify(ctx, tok.astype(np.int32), q, tgt2, cu, 6, 1.0, uv3)
    assert np.all(got[0] == 0)
    tl.check_verify_against_oracle(oracle, tok.astype(np.int32), q, tgt2, cu, 1.0, uv3, got, "reject-at-0")


def test_position_major_draft_layout(ctx, oracle):
    """Draft-side arrays laid out [K_max, B] (one logits buffer per draft step) via the two strides."""
    rng = np.random.default_rng(12)
    B, V, K = 5, 777, 4
    lens, cu, q, tgt, ud, uv = small_case(rng, B, V, K, True)
    tok, _, _ = oracle.draft_step(q, 1.0, 0.3, ud)
    q_pm = np.zeros((K * B, V), np.uint16); tok_pm = np.zeros(K * B, np.int32)
    for i in range(B):
        for j in range(lens[i]):
            q_pm[j * B + i] = q[cu[i] - i + j]; tok_pm[j * B + i] = tok[cu[i] - i + j]
    uv, _ = tl.guard_accept_uniforms(oracle, tok.astype(np.int32), q, tgt, cu, 1.0, uv)
    got, early = tl.gpu_verify(ctx, tok_pm, q_pm, tgt, cu, K, 1.0, uv, layout="strided", q_seq_stride=1, q_pos_stride=B,
                               early_exit=True)
    tl.check_verify_against_oracle(oracle, tok.astype(np.int32), q, tgt, cu, 1.0, uv, got, "position-major")
    tl.check_verify_against_oracle(oracle, tok.astype(np.int32), q, tgt, cu, 1.0, uv, early, "position-major (early exit)")


def test_pack_ragged(ctx, oracle):
    import torch
    rng = np.random.default_rng(3)
    for B, K_max in ((1, 1), (7, 64), (128, 64), (1500, 9), (65536, 2)):
        lens = rng.integers(1, K_max + 1, size=B).astype(np.int32)
        cu_o, seq_o, pos_o = oracle.pack_ragged(lens)
        d = torch.from_numpy(lens).cuda()
        cu = torch.zeros(B + 1, dtype=torch.int32, device="cuda")
        seq = torch.full((B * (K_max + 1),), -1, dtype=torch.int32, device="cuda")
        pos = torch.full((B * (K_max + 1),), -1, dtype=torch.int32, device="cuda")
        ctx.pack_ragged(d, B, K_max, cu, seq, pos)
        torch.cuda.synchronize()
        R = int(cu_o[-1])
        assert np.array_equal(cu.cpu().numpy(), cu_o)
        assert np.array_equal(seq.cpu().numpy()[:R], seq_o) and np.array_equal(pos.cpu().numpy()[:R], pos_o)
        assert np.all(seq.cpu().numpy()[R:] == -1)
    assert ctx.read_status() == 0
    bad = torch.tensor([3, 0, 99, 2], dtype=torch.int32, device="cuda")
    cu = torch.zeros(5, dtype=torch.int32, device="cuda")
    ctx.pack_ragged(bad, 4, 8, cu)
    assert ctx.read_status() == 2
    assert cu.cpu().tolist() == [0, 4, 6, 15, 18]


def test_workspace_limit_and_bad_arguments():
    import torch
    from paper_2411_18462_b200 import Context, SvipError
    c = Context(0, 8)
    t = torch.zeros(64, device="cuda"); i = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(SvipError) as e:
        c.verify(i, t, 4, None, -1, 0, t, 4, 0, None, 3, 2, 9, 4, 1.0, t, i, i)
    assert e.value.code == -3
    with pytest.raises(SvipError):   # fixed K needs exactly B*(K+1) rows
        c.verify(i, t, 4, None, -1, 0, t, 4, 0, None, 2, 2, 5, 4, 1.0, t, i, i)
    with pytest.raises(SvipError):   # sampling needs uniforms
        c.verify(i, t, 4, None, -1, 0, t, 4, 0, None, 2, 2, 6, 4, 1.0, None, i, i)
    c.destroy()


@pytest.mark.parametrize("early_exit", [False, True])
def test_graph_replay_matches_direct_calls(ctx, oracle, early_exit):
    """B = 1: eight draft steps, packing and the verify round recorded once, replayed on new inputs."""
    import torch
    verify = ctx.verify_early_exit if early_exit else ctx.verify
    w = W.make_workload("tiny")
    K, V = w.K_max, w.V
    dq = tl.to_device(w.q_logits); dt = tl.to_device(w.target_logits)
    ud = tl.to_device(w.draft_uniforms); uv = tl.to_device(w.verify_uniforms)
    tok = torch.zeros(K, dtype=torch.int32, device="cuda"); ent = torch.zeros(K, device="cuda")
    stop = torch.zeros(K, dtype=torch.uint8, device="cuda"); stats = torch.zeros(K, 2, device="cuda")
    lens = torch.tensor([K], dtype=torch.int32, device="cuda"); cu = torch.zeros(2, dtype=torch.int32, device="cuda")
    nacc = torch.zeros(1, dtype=torch.int32, device="cuda"); nxt = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()

    def enqueue():
        for j in range(K):
            ctx.draft_step(dq.data_ptr() + j * V * 4, 0, 1, V, V, 1.0, w.h, ud.data_ptr() + 4 * j,
                           tok.data_ptr() + 4 * j, ent.data_ptr() + 4 * j, stop.data_ptr() + j,
                           stats.data_ptr() + 8 * j, st)
        ctx.pack_ragged(lens, 1, K, cu, None, None, st)
        verify(tok, dq, V, stats, -1, 0, dt, V, 0, cu, 1, K, K + 1, V, 1.0, uv, nacc, nxt, st)

    enqueue(); st.synchronize()
    direct = (tok.cpu().numpy().copy(), nacc.item(), nxt.item())
    ctx.graph_begin(st); enqueue(); g = ctx.graph_end(st)
    # new inputs in place: target := draft (all accepted), replay must see them
    dt[:K].copy_(dq)
    g.launch(st); st.synchronize()
    assert nacc.item() == K
    dt.copy_(tl.to_device(w.target_logits))
    tok.zero_(); nacc.zero_(); nxt.zero_()
    g.launch(st); st.synchronize()
    assert np.array_equal(tok.cpu().numpy(), direct[0]) and (nacc.item(), nxt.item()) == direct[1:]
    g.destroy()
    tok_o, _, _ = oracle.draft_step(w.q_logits, 1.0, w.h, w.draft_uniforms)
    assert np.array_equal(direct[0], tok_o)


@pytest.mark.parametrize("name", ["tiny", "chat", "reasoning", "ragged", "stress"])
def test_published_configs(ctx, oracle, name):
    """Each published configuration at full size, automatic launch shape, q_stats from the draft step."""
    w = W.make_workload(name)
    temps = {"tiny": (1.0, 0.0), "chat": (1.0, 0.0), "reasoning": (0.7,), "ragged": (1.0,), "stress": (1.0, 0.0)}[name]
    fixed = name != "ragged"
    for T in temps:
        tok, _, _ = oracle.draft_step(w.q_logits, T, w.h, w.draft_uniforms, threads=16)
        tok = tok.astype(np.int32)
        uv, moved = tl.guard_accept_uniforms(oracle, tok, w.q_logits, w.target_logits, w.cu_rows, T,
                                             w.verify_uniforms, threads=16)
        stats = tl.gpu_draft_step(ctx, w.q_logits, T, w.h, w.draft_uniforms)[3] if T > 0 else None
        got, early = tl.gpu_verify(ctx, tok, w.q_logits, w.target_logits, w.cu_rows, w.K_max, T,
                                   uv if T > 0 else None, q_stats=stats, fixed_K=fixed, early_exit=True)
        c = tl.check_verify_against_oracle(oracle, tok, w.q_logits, w.target_logits, w.cu_rows, T, uv, got,
                                           "%s T=%g" % (name, T), threads=16)
        ce = tl.check_verify_against_oracle(oracle, tok, w.q_logits, w.target_logits, w.cu_rows, T, uv, early,
                                            "%s T=%g (early exit)" % (name, T), threads=16)
        # the two entry points cut the rows over different numbers of blocks, so the fp32 normalisers differ in
        # their last bits: the accepted counts must agree (the accept draws are off the boundary), the next
        # token may fall on the other side of a CDF boundary within the tolerance
        assert np.array_equal(got[0], early[0])
        print("verify parity", name, "T=%g" % T, c, "early exit:", ce, "same next token in",
              int((got[1] == early[1]).sum()), "of", len(got[1]), "uniforms moved off the accept boundary:", moved)
    if name == "tiny":   # target := draft everywhere: all K accepted, bonus token from row K
        t2 = w.target_logits.copy(); t2[:w.K_max] = w.q_logits
        tok, _, _ = oracle.draft_step(w.q_logits, 1.0, w.h, w.draft_uniforms)
        got = tl.gpu_verify(ctx, tok.astype(np.int32), w.q_logits, t2, w.cu_rows, w.K_max, 1.0, w.verify_uniforms,
                            fixed_K=True)
        assert got[0][0] == w.K_max
        tl.check_verify_against_oracle(oracle, tok.astype(np.int32), w.q_logits, t2, w.cu_rows, 1.0,
                                       w.verify_uniforms, got, "tiny all-accept")
    assert ctx.read_status() == 0


@pytest.mark.parametrize("bf16", [False, True])
def test_accept_ratio_of_very_unlikely_tokens(ctx, oracle, bf16):
    """Draft tokens that both models find almost impossible (probabilities far below the smallest fp32
    number) still have a well-defined ratio p(x)/q(x); the accept count must follow it (Algorithm 2), not
    the ratio of two underflowed exponentials.  Only the accept counts are compared: at such positions
    p and q may agree so closely that the residual of Algorithm 4 is below fp32 resolution."""
    rng = np.random.default_rng(31)
    B, V, K, T = 48, 20011, 1, 0.5
    base = (rng.standard_normal((B, V)) * 8.0).astype(np.float32)          # margins of ~60 logits, /T -> 120
    tgt_first = base + (rng.standard_normal((B, V)) * 1.5).astype(np.float32)
    tgt = np.empty((2 * B, V), np.float32)
    tgt[0::2] = tgt_first
    tgt[1::2] = base                                                       # the bonus row, unused here
    q = base.copy()
    if bf16:
        q = W.to_bf16_bits(q); tgt = W.to_bf16_bits(tgt)
    qv = W.bf16_bits_to_f32(q) if bf16 else q
    tok = qv.argmin(axis=1).astype(np.int32)                               # the least likely token of each row
    margin = (qv.max(axis=1) - qv[np.arange(B), tok]) / T * 1.4427
    assert margin.min() > 127                                              # below 2^-127 under the draft model
    cu = (np.arange(B + 1) * 2).astype(np.int64)
    uv = rng.random(2 * B).astype(np.float32)
    uv, _ = tl.guard_accept_uniforms(oracle, tok, q, tgt, cu, T, uv, threads=8)
    n_g, _ = tl.gpu_verify(ctx, tok, q, tgt, cu, K, T, uv)
    n_o, _, ap = oracle.verify(tok, q, tgt, cu, T, uv.astype(np.float64), want_accept_prob=True, threads=8)
    assert np.array_equal(n_g.astype(np.int64), n_o)
    probs = np.array([a[0] for a in ap])
    assert (probs < 0.9).sum() > 5 and (probs >= 1.0).sum() > 5            # both outcomes are exercised
    assert 0 < n_o.sum() < B


@pytest.mark.parametrize("bf16", [False, True])
def test_draft_token_outside_the_draft_support(ctx, oracle, bf16):
    """A draft token whose own draft logit is -inf while the target's is finite: q(x) = 0 < p(x), the
    ratio of Algorithm 2 is +inf and every draw accepts, also the largest one.  With the target logit
    at -inf too there is nothing to accept: rejected whatever the draw."""
    rng = np.random.default_rng(515 + int(bf16))
    B, V, K, T = 6, 3001, 3, 0.9
    lens, cu, q, tgt, ud, uv = small_case(rng, B, V, K, False, ragged=False)
    tok, _, _ = oracle.draft_step(q, T, 0.3, ud)
    tok = tok.astype(np.int32)
    # position 1 of every sequence: the draft model excludes its own token
    for i in range(B):
        r = int(cu[i]) - i + 1
        x = int(rng.integers(0, V))
        tok[r] = x
        q[r, x] = -np.inf
        tgt[cu[i] + 1, x] = rng.standard_normal() if i % 2 == 0 else -np.inf
    if bf16:
        q = W.to_bf16_bits(q); tgt = W.to_bf16_bits(tgt)
    uv = uv.copy()
    uv, _ = tl.guard_accept_uniforms(oracle, tok, q, tgt, cu, T, uv)
    uv[cu[:-1]] = 0.0                            # position 0 accepted (p(x) > 0 for a token drawn from q)
    uv[cu[:-1] + 1] = 1.0 - 2.0 ** -24           # the hardest draw at the position under test
    for S in (0, 1, 4):
        ctx.set_cluster_size(S)
        try:
            for with_stats in (False, True):
                stats = tl.gpu_draft_step(ctx, q, T, 0.3, ud)[3] if with_stats else None
                got = tl.gpu_verify(ctx, tok, q, tgt, cu, K, T, uv, q_stats=stats, fixed_K=True)
                tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, T, uv, got, "q(x)=0 S=%d" % S)
                assert np.all(got[0][0::2] >= 2), got[0]      # q(x) = 0 < p(x): accepted
                assert np.all(got[0][1::2] == 1), got[0]      # q(x) = 0 = p(x): rejected
        finally:
            ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def _nearly_equal_pair(rng, V, q_of_x):
    """A draft row and a target row that differ in ONE logit, the target's one unit in the last place
    lower, at a token of draft probability about q_of_x: p(x)/q(x) = 1 - 2e-6, so the largest draw
    rejects, and max(0, p - q) is carried by the normalisers' difference alone (about 2e-6 * q(x))."""
    d = (rng.standard_normal(V) * 1.5).astype(np.float32)
    x = int(rng.integers(0, V))
    Z = np.exp(d.astype(np.float64) - d.max()).sum()
    d[x] = np.float32(d.max() + np.log(q_of_x * Z))
    if not 16.0 <= abs(d[x]) < 32.0:                        # one unit in the last place = 1.9e-6 there
        shift = np.float32((-24.0 if d[x] < 0 else 24.0) - d[x])
        d = (d + shift).astype(np.float32)
    t = d.copy()
    t[x] = np.nextafter(d[x], np.float32(-np.inf))
    return d, t, x


def test_rejection_with_a_residual_below_fp32_resolution(ctx, oracle):
    """Algorithm 4 when p and q agree to the last place.  After a rejection max(0, p - q) has mass in exact
    arithmetic, but it can vanish in the arithmetic that computes it; the correction token is then drawn
    from p (p and q are indistinguishable there).  Two families:
      (a) the differing token is so unlikely (1e-11) that even the fp64 normalisers coincide: oracle and
          GPU both see a zero residual and both sample from p: full parity;
      (b) the differing token has probability 1e-3 .. 1e-5: the fp64 residual has mass ~1e-9..1e-11, the
          fp32 one is zero or rounding noise: only what is unique is compared (the rejection itself, a
          token the target gives weight, a clear status word)."""
    rng = np.random.default_rng(99)
    V, T = 8192, 1.0
    top = np.float32(1.0 - 2.0 ** -24)
    n_a = n_b_zero64 = 0
    for case, q_of_x in enumerate((1e-11, 1e-11, 1e-11, 1e-3, 1e-4, 1e-5, 1e-3, 1e-4)):
        d, t, x = _nearly_equal_pair(rng, V, q_of_x)
        q_rows = d[None, :]
        t_rows = np.stack([t, (rng.standard_normal(V)).astype(np.float32)])
        cu = np.array([0, 2], dtype=np.int64)
        tok = np.array([x], dtype=np.int32)
        p64 = oracle.softmax(t_rows[0], T); q64 = oracle.softmax(q_rows[0], T)
        _, S64 = oracle.residual(p64, q64)
        for u in (0.0, 0.37, 0.93):
            uv = np.array([top, u], dtype=np.float32)
            n_o, nx_o, ap = oracle.verify(tok, q_rows, t_rows, cu, T, uv.astype(np.float64), want_accept_prob=True)
            assert n_o[0] == 0 and ap[0][0] < float(top)             # the oracle rejects
            for S in (0, 1, 2):
                ctx.set_cluster_size(S)
                try:
                    got = tl.gpu_verify(ctx, tok, q_rows, t_rows, cu, 1, T, uv, fixed_K=True)
                finally:
                    ctx.set_cluster_size(0)
                assert got[0][0] == 0, "the GPU must reject as well (case %d)" % case
                assert 0 <= got[1][0] < V and p64[got[1][0]] > 0.0
                if S64 == 0.0:        # family (a): both sides fall back to p
                    tl.check_verify_against_oracle(oracle, tok, q_rows, t_rows, cu, T, uv, got, "zero residual")
                    n_a += 1
        n_b_zero64 += int(S64 == 0.0)
    assert n_a >= 9 and n_b_zero64 <= 5      # both families occurred
    assert ctx.read_status() == 0


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("T", [1.0, 0.0])
def test_early_exit_never_reads_rows_after_the_first_rejection(ctx, oracle, bf16, T):
    """The target rows after a sequence's first rejection are overwritten with NaN: svip_verify_early_exit
    must still give the oracle's result on the clean rows and raise no status bit (a NaN row that is read
    raises the non-finite bit, as the plain entry point shows on the same buffers)."""
    import torch
    rng = np.random.default_rng(77 + int(bf16) + int(T * 10))
    lens, cu, q, tgt, ud, uv = small_case(rng, 24, 3000, 7, bf16, noise=0.8)
    tok, _, _ = oracle.draft_step(q, T if T > 0 else 1.0, 0.3, ud, threads=8)
    tok = tok.astype(np.int32)
    uv, _ = tl.guard_accept_uniforms(oracle, tok, q, tgt, cu, T, uv)
    n_ref, nx_ref, _ = oracle.verify(tok, q, tgt, cu, T, uv)
    assert (n_ref < lens).sum() >= 8, "the case needs early rejections"
    dirty = tgt.copy()
    nan = np.uint16(0x7FC0) if bf16 else np.float32(np.nan)
    poisoned = 0
    for i in range(len(lens)):
        lo, hi = cu[i] + n_ref[i] + 1, cu[i + 1]
        dirty[lo:hi] = nan
        poisoned += hi - lo
    assert poisoned > 20
    B, K = len(lens), 7
    Rp, V = tgt.shape
    dt = tl.dtype_code(tgt)
    d_tok, d_q, d_t = tl.to_device(tok), tl.to_device(q), tl.to_device(dirty)
    d_cu, d_u = tl.to_device(cu.astype(np.int32)), tl.to_device(uv.astype(np.float32))
    n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda"); nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    for S in (0, 1, 2, 3, 8):
        ctx.set_cluster_size(S)
        assert ctx.read_status() == 0
        n_acc.fill_(-7); nxt.fill_(-7)
        ctx.verify_early_exit(d_tok, d_q, V, None, -1, 0, d_t, V, dt, d_cu, B, K, Rp, V, T, d_u if T > 0 else None, n_acc, nxt)
        torch.cuda.synchronize()
        assert ctx.read_status() == 0, "a row after the first rejection was read (S=%d)" % S
        tl.check_verify_against_oracle(oracle, tok, q, tgt, cu, T, uv, (n_acc.cpu().numpy(), nxt.cpu().numpy()),
                                       "early exit, poisoned tail, S=%d" % S)
    ctx.set_cluster_size(0)
    ctx.verify(d_tok, d_q, V, None, -1, 0, d_t, V, dt, d_cu, B, K, Rp, V, T, d_u if T > 0 else None, n_acc, nxt)
    torch.cuda.synchronize()
    assert ctx.read_status() & 1, "the plain entry point reads every row, the NaN ones too"
