"""GPU parity of svip_verify_tree (through the C ABI) against the oracle's tree verification."""
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


def random_forest(rng, oracle, B, N, V, bf16, T, branching=3, noise=0.7, from_draft=0.8):
    """B random trees of N candidate nodes: the parent of node i is a random earlier node (or the root) that
    still has fewer than `branching` children; tokens are drawn from the parent's draft row (mostly)."""
    parent = np.zeros((B, N), np.int32)
    for b in range(B):
        kids = {-1: 0}
        for i in range(N):
            open_nodes = [n for n, c in kids.items() if c < branching]
            par = int(rng.choice(open_nodes))
            parent[b, i] = par
            kids[par] += 1
            kids[i] = 0
    rows = B * (N + 1)
    scale = np.exp(rng.uniform(np.log(0.5), np.log(4.0), size=(rows, 1)))
    q = (rng.standard_normal((rows, V)) * scale).astype(np.float32)
    t = (q + rng.standard_normal((rows, V)).astype(np.float32) * noise).astype(np.float32)
    if bf16:
        q = W.to_bf16_bits(q); t = W.to_bf16_bits(t)
    tokens = rng.integers(0, V, size=(B, N)).astype(np.int32)
    Ts = T if T > 0 else 1.0
    for b in range(B):
        prow = b * (N + 1) + parent[b] + 1
        drawn = oracle.draft_step(q[prow], Ts, 0.3, rng.random(N))[0].astype(np.int32)
        use = rng.random(N) < from_draft
        tokens[b] = np.where(use, drawn, tokens[b])
    u = rng.random((B, N + 1)).astype(np.float32)
    return parent, tokens, q, t, u


def guard_tree_uniforms(oracle, parent, tokens, q, t, T, u, threads=8):
    """Moves accept draws that lie within ACCEPT_GUARD of the oracle's acceptance probability of a candidate
    the walk tries; repeated because a moved draw can change the walk."""
    u = u.copy()
    moved = 0
    if not T > 0:
        return u, 0
    for _ in range(6):
        _, _, _, ap = oracle.verify_tree(parent, tokens, q, t, T, u.astype(np.float64), want_accept_prob=True,
                                         threads=threads)
        N = parent.shape[1]
        tried = (ap >= 0) & (ap < 1.0)
        close = tried & (np.abs(u[:, :N].astype(np.float64) - ap) < tl.ACCEPT_GUARD)
        if not close.any():
            return u, moved
        for b, i in zip(*np.nonzero(close)):
            a = ap[b, i]
            new = a + 2 * tl.ACCEPT_GUARD if u[b, i] >= a else a - 2 * tl.ACCEPT_GUARD
            if new >= 1.0:
                new = a - 2 * tl.ACCEPT_GUARD
            if new < 0.0:
                new = a + 2 * tl.ACCEPT_GUARD
            u[b, i] = np.float32(new)
            moved += 1
    raise AssertionError("accept draws keep landing on a boundary")


def gpu_tree(ctx, parent, tokens, q, t, T, u, q_stats=None):
    import torch
    B, N = parent.shape
    V = t.shape[1]
    n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    path = torch.full((B, N), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ctx.verify_tree(tl.to_device(tokens), tl.to_device(parent), tl.to_device(q), V,
                    tl.to_device(q_stats) if q_stats is not None else None, tl.to_device(t), V, tl.dtype_code(t),
                    B, N, V, T, tl.to_device(u) if T > 0 else None, n_acc, path, nxt)
    torch.cuda.synchronize()
    return n_acc.cpu().numpy(), path.cpu().numpy(), nxt.cpu().numpy()


def check_tree(oracle, parent, tokens, q, t, T, u, got, label):
    B, N = parent.shape
    V = t.shape[1]
    fw = np.zeros((B, V)) if T > 0 else None
    n_o, path_o, nx_o, _ = oracle.verify_tree(parent, tokens, q, t, T, u.astype(np.float64), threads=8, final_weights=fw)
    n_g, path_g, nx_g = got
    assert np.array_equal(n_g.astype(np.int64), n_o), "%s: n_accepted %s vs %s" % (label, n_g[:12], n_o[:12])
    assert np.array_equal(path_g, path_o), label + ": accepted paths differ"
    boundary = 0
    for b in np.nonzero(nx_g.astype(np.int64) != nx_o)[0]:
        assert T > 0, label + ": greedy next tokens differ"
        assert tl.within_cdf_tolerance(fw[b], u[b, N], int(nx_g[b])), \
            "%s seq %d: next %d vs oracle %d, beyond the CDF tolerance" % (label, b, nx_g[b], nx_o[b])
        boundary += 1
    return {"sequences": B, "mean_accepted": float(n_o.mean()), "next_boundary": boundary}


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("V", [5, 33, 1000, 32000])
def test_random_trees_all_cluster_sizes(ctx, oracle, V, bf16):
    rng = np.random.default_rng(700 + V + int(bf16))
    B, N = 6, 12
    for T in (1.0, 0.7, 0.0):
        parent, tokens, q, t, u = random_forest(rng, oracle, B, N, V, bf16, T)
        u, moved = guard_tree_uniforms(oracle, parent, tokens, q, t, T, u)
        for S in (0, 1, 2, 3, 5, 8):
            ctx.set_cluster_size(S)
            try:
                got = gpu_tree(ctx, parent, tokens, q, t, T, u)
            finally:
                ctx.set_cluster_size(0)
            c = check_tree(oracle, parent, tokens, q, t, T, u, got, "V=%d S=%d T=%g" % (V, S, T))
        assert 0 <= c["mean_accepted"] <= N
    assert ctx.read_status() == 0


def test_one_candidate_per_node_matches_the_linear_round(ctx, oracle):
    """A chain is the linear round: svip_verify_tree must give what svip_verify gives (and the oracle)."""
    rng = np.random.default_rng(41)
    B, K, V, T = 8, 5, 3000, 0.9
    parent = np.tile(np.arange(-1, K - 1, dtype=np.int32), (B, 1))
    _, tokens, q, t, u = random_forest(rng, oracle, B, K, V, True, T, branching=1, noise=0.4)
    # random_forest drew the tokens from parents of ITS tree; redo for the chain
    for b in range(B):
        tokens[b] = oracle.draft_step(q[b * (K + 1): b * (K + 1) + K], T, 0.3, rng.random(K))[0]
    u, _ = guard_tree_uniforms(oracle, parent, tokens, q, t, T, u)
    got = gpu_tree(ctx, parent, tokens, q, t, T, u)
    check_tree(oracle, parent, tokens, q, t, T, u, got, "chain")
    # the linear call on the same data: draft rows packed without the unused row of the last node
    cu = (np.arange(B + 1) * (K + 1)).astype(np.int64)
    q_lin = np.concatenate([q[b * (K + 1): b * (K + 1) + K] for b in range(B)])
    lin = tl.gpu_verify(ctx, tokens.reshape(-1), q_lin, t, cu, K, T, u.reshape(-1), fixed_K=True)
    assert np.array_equal(lin[0], got[0])
    same = lin[1] == got[2]
    assert same.mean() >= 0.75          # identical arithmetic up to the order of the segment sums
    assert ctx.read_status() == 0


def test_many_candidates_and_normalisers_from_the_draft_step(ctx, oracle):
    """Wide nodes (up to 8 candidates, unlikely ones: long rejection chains) with q_stats handed over."""
    rng = np.random.default_rng(43)
    B, N, V, T = 5, 16, 8000, 1.0
    parent, tokens, q, t, u = random_forest(rng, oracle, B, N, V, False, T, branching=8, noise=1.5, from_draft=0.5)
    u, _ = guard_tree_uniforms(oracle, parent, tokens, q, t, T, u)
    stats = tl.gpu_draft_step(ctx, q, T, 0.3, np.zeros(q.shape[0], np.float32))[3]
    got = gpu_tree(ctx, parent, tokens, q, t, T, u, q_stats=stats)
    c = check_tree(oracle, parent, tokens, q, t, T, u, got, "wide")
    got2 = gpu_tree(ctx, parent, tokens, q, t, T, u)
    assert np.array_equal(got[0], got2[0]) and np.array_equal(got[1], got2[1])
    assert ctx.read_status() == 0


def test_published_shape(ctx, oracle):
    """Trees over rows of the reasoning recipe (V = 152064 bf16, T = 0.7): 8 sequences, 10 nodes each."""
    w = W.make_workload("reasoning", B=8, K_max=10)
    B, N, V, T = 8, 10, w.V, w.T
    rng = np.random.default_rng(5)
    q = np.zeros((B * (N + 1), V), np.uint16); t = np.zeros_like(q)
    for b in range(B):
        q[b * (N + 1): b * (N + 1) + N] = w.q_logits[b * N: b * N + N]
        q[b * (N + 1) + N] = w.q_logits[b * N]
        t[b * (N + 1): (b + 1) * (N + 1)] = w.target_logits[b * (N + 1): (b + 1) * (N + 1)]
    parent = np.tile(np.array([-1, -1, 0, 0, 1, 2, 2, 4, 5, 5], np.int32), (B, 1))
    tokens = np.zeros((B, N), np.int32)
    for b in range(B):
        prow = b * (N + 1) + parent[b] + 1
        tokens[b] = oracle.draft_step(q[prow], T, 0.3, rng.random(N))[0]
    u = rng.random((B, N + 1)).astype(np.float32)
    u, moved = guard_tree_uniforms(oracle, parent, tokens, q, t, T, u)
    got = gpu_tree(ctx, parent, tokens, q, t, T, u)
    c = check_tree(oracle, parent, tokens, q, t, T, u, got, "reasoning rows")
    print("tree parity", c, "accept draws moved:", moved)
    assert ctx.read_status() == 0


def test_malformed_trees_and_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError, binding
    B, N, V = 2, 20, 64
    rng = np.random.default_rng(2)
    q = (rng.standard_normal((B * (N + 1), V))).astype(np.float32)
    t = (rng.standard_normal((B * (N + 1), V))).astype(np.float32)
    parent = np.full((B, N), -1, np.int32)              # 20 candidates at the root: more than can be rejected
    tokens = np.tile(np.argmin(t[0]).astype(np.int32), (B, N))
    t[:, tokens[0, 0]] = -np.inf                        # p = 0 there: every candidate is rejected
    u = np.full((B, N + 1), 0.5, np.float32)
    n_acc, path, nxt = gpu_tree(ctx, parent, tokens, q, t, 1.0, u)
    assert np.all(n_acc == 0) and np.all(path == -1) and np.all((nxt >= 0) & (nxt < V))
    assert ctx.read_status() & binding.SVIP_STATUS_BAD_TREE
    parent2 = np.full((B, N), -1, np.int32); parent2[:, 3] = 7      # a parent above its node
    gpu_tree(ctx, parent2[:, :5], tokens[:, :5], q[:B * 6], t[:B * 6], 1.0, u[:, :6])
    assert ctx.read_status() & binding.SVIP_STATUS_BAD_TREE
    i = torch.zeros(64, dtype=torch.int32, device="cuda"); f = torch.zeros(4096, device="cuda")
    for bad in (dict(N=0), dict(V=0), dict(T=-1.0), dict(uniforms=None), dict(B=1 << 14)):
        a = dict(B=2, N=3, V=16, T=1.0, uniforms=f)
        a.update(bad)
        with pytest.raises(SvipError):
            ctx.verify_tree(i, i, f, 16, None, f, 16, 0, a["B"], a["N"], a["V"], a["T"], a["uniforms"], i, i, i)
    ctx.verify_tree(i, i, f, 16, None, f, 16, 0, 0, 3, 16, 1.0, f, i, i, i)      # empty batch
