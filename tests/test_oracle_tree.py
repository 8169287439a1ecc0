"""Pins of the oracle's tree (multi-candidate) verification, svip_oracle_verify_tree.

The paper applies its length policy on top of EAGLE-2's candidate trees (Section 3.3) without stating an
accept rule for several candidates per position; the oracle uses the published recursive rejection rule.
What fixes it here, independently of the oracle's own code:
  * with one candidate per node it must be the linear verification round (Algorithms 1, 2, 4), which is
    pinned on its own;
  * a worked example small enough to do by hand;
  * the property the paper relies on: every emitted token follows the target distribution of its
    position when the candidates are drawn independently from the draft distribution (chi-square, tiny V),
    and the first candidate is accepted with probability beta = sum min(p, q) (Eq. 1).
"""
import math

import numpy as np
from scipy import stats


def logits_of(p):
    return np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)


def tree_arrays(parent, tokens, q_rows, t_rows, u):
    N = len(parent)
    return (np.asarray(parent, np.int32).reshape(1, N), np.asarray(tokens, np.int32).reshape(1, N),
            np.asarray(q_rows, np.float32), np.asarray(t_rows, np.float32), np.asarray(u, np.float64).reshape(1, N + 1))


def test_one_candidate_per_node_is_the_linear_round(oracle):
    rng = np.random.default_rng(5)
    V = 40
    top = 1.0 - 2.0 ** -24
    for trial in range(300):
        K = int(rng.integers(1, 6))
        d = (rng.standard_normal((K + 1, V)) * 1.5).astype(np.float32)        # row K of the draft is never read
        t = (d + rng.standard_normal((K + 1, V)).astype(np.float32) * rng.uniform(0.1, 1.5)).astype(np.float32)
        T = float(rng.choice([1.0, 0.6, 0.0]))
        tok = rng.integers(0, V, size=K).astype(np.int32)
        if trial % 3 == 0:      # plausible drafts: drawn from the draft rows
            tok = oracle.draft_step(d[:K], T if T > 0 else 1.0, 0.3, rng.random(K))[0].astype(np.int32)
        u = rng.random(K + 1)
        if trial % 7 == 0:
            u[:K] = top
        n_l, nx_l, _ = oracle.verify(tok, d[:K], t, np.array([0, K + 1]), T, u)
        parent = np.arange(-1, K - 1)
        n_t, path, nx_t, _ = oracle.verify_tree(parent[None, :], tok[None, :], d, t, T, u[None, :])
        assert n_t[0] == n_l[0] and nx_t[0] == nx_l[0], (trial, n_t, n_l, nx_t, nx_l)
        assert path[0, :n_t[0]].tolist() == list(range(n_t[0])) and np.all(path[0, n_t[0]:] == -1)


def test_worked_example_two_candidates(oracle):
    """p = (0.5, 0.3, 0.2), q = (0.2, 0.5, 0.3) at the root, two candidates.
    Candidate 1 = token 1: accepted with probability 0.3 / 0.5 = 0.6.  If rejected, p_2 = max(0, p - q)
    = (0.3, 0, 0) / 0.3 = (1, 0, 0).  Candidate 2 = token 2 then has p_2 = 0: always rejected, and p_3 =
    max(0, p_2 - q) = (0.8, 0, 0) / 0.8 = (1, 0, 0): the next token is 0 whatever the last draw.
    Candidate 2 = token 0 has p_2 / q = 1 / 0.2 > 1: always accepted."""
    p = [0.5, 0.3, 0.2]; q = [0.2, 0.5, 0.3]
    rows_t = np.stack([logits_of(p)] * 3); rows_q = np.stack([logits_of(q)] * 3)
    for u_last in (0.0, 0.5, 0.999):
        a = tree_arrays([-1, -1], [1, 2], rows_q, rows_t, [0.61, 0.0, u_last])
        n, path, nx, ap = oracle.verify_tree(*a[:4], 1.0, a[4], want_accept_prob=True)
        assert n[0] == 0 and nx[0] == 0
        assert abs(ap[0, 0] - 0.6) < 1e-6 and ap[0, 1] == 0.0
    a = tree_arrays([-1, -1], [1, 2], rows_q, rows_t, [0.59, 0.9, 0.3])
    n, path, nx, ap = oracle.verify_tree(*a[:4], 1.0, a[4], want_accept_prob=True)
    assert n[0] == 1 and path[0, 0] == 0 and ap[0, 1] == -1.0          # accepted: the second one is not tried
    assert nx[0] == oracle.invcdf(np.array(p), 0.3)                    # leaf: the next token comes from its own p
    a = tree_arrays([-1, -1], [1, 0], rows_q, rows_t, [0.61, 1.0 - 2.0 ** -24, 0.3])
    n, path, nx, ap = oracle.verify_tree(*a[:4], 1.0, a[4], want_accept_prob=True)
    assert n[0] == 1 and path[0, 0] == 1 and ap[0, 1] == 1.0


def test_children_are_tried_in_index_order_and_the_walk_descends(oracle):
    """Root with children 0 and 2; node 0 has child 1; node 2 has child 3.  Identical draft and target rows:
    every tried candidate is accepted, so the walk takes node 0, then node 1, and samples at that leaf."""
    rng = np.random.default_rng(1)
    V = 9
    rows = (rng.standard_normal((5, V))).astype(np.float32)
    parent = [-1, 0, -1, 2]; tokens = [3, 4, 5, 6]
    a = tree_arrays(parent, tokens, rows, rows, [0.99, 0.99, 0.99, 0.99, 0.42])
    n, path, nx, ap = oracle.verify_tree(*a[:4], 1.0, a[4], want_accept_prob=True)
    assert n[0] == 2 and path[0, :2].tolist() == [0, 1]
    assert ap[0].tolist() == [1.0, 1.0, -1.0, -1.0]
    assert nx[0] == oracle.invcdf(oracle.softmax(rows[2], 1.0), 0.42)   # row of node 1 is row 2
    # greedy: the child whose token is the argmax of the node's target row
    t = rows.copy(); t[0, 5] = 50.0; t[3, 6] = 50.0; t[4, 1] = 50.0
    n, path, nx, _ = oracle.verify_tree(a[0], a[1], rows, t, 0.0, a[4])
    assert n[0] == 2 and path[0, :2].tolist() == [2, 3] and nx[0] == 1
    t[0, 8] = 60.0                                                      # no child holds the argmax
    n, path, nx, _ = oracle.verify_tree(a[0], a[1], rows, t, 0.0, a[4])
    assert n[0] == 0 and nx[0] == 8


def _chi_square_ok(counts, probs, alpha=1e-3):
    counts = np.asarray(counts, dtype=np.float64); probs = np.asarray(probs, dtype=np.float64)
    keep = probs > 0
    assert counts[~keep].sum() == 0
    exp = probs[keep] * counts.sum()
    chi2 = ((counts[keep] - exp) ** 2 / exp).sum()
    return chi2 < stats.chi2.ppf(1 - alpha, keep.sum() - 1), chi2


def test_emitted_tokens_follow_the_target_distribution(oracle):
    """Two levels, three candidates per node, V = 4.  Candidates are drawn from the node's draft row with the
    oracle's own sampler.  The first emitted token must follow the root's target distribution; given that a
    child c was accepted, the second emitted token must follow the target distribution of node c; and the
    first candidate is accepted with probability beta (Eq. 1)."""
    rng = np.random.default_rng(2024)
    V, k, Bn = 4, 3, 60000
    N = k + k * k
    parent = np.array([-1] * k + [c for c in range(k) for _ in range(k)], np.int32)
    q_node = (rng.standard_normal((N + 1, V)) * 1.2).astype(np.float32)
    t_node = (rng.standard_normal((N + 1, V)) * 1.2).astype(np.float32)
    q_all = np.tile(q_node, (Bn, 1)); t_all = np.tile(t_node, (Bn, 1))
    tokens = np.zeros((Bn, N), np.int32)
    for node_row, kids in [(0, range(0, k))] + [(1 + c, range(k + c * k, k + c * k + k)) for c in range(k)]:
        for j in kids:
            tok, _, _ = oracle.draft_step(np.tile(q_node[node_row], (Bn, 1)), 1.0, 0.3, rng.random(Bn))
            tokens[:, j] = tok
    u = rng.random((Bn, N + 1))
    n_acc, path, nxt, _ = oracle.verify_tree(np.tile(parent, (Bn, 1)), tokens, q_all, t_all, 1.0, u, threads=8)
    first = np.where(n_acc > 0, tokens[np.arange(Bn), np.maximum(path[:, 0], 0)], nxt)
    p_root = oracle.softmax(t_node[0], 1.0)
    ok, chi2 = _chi_square_ok(np.bincount(first, minlength=V), p_root)
    assert ok, chi2
    beta = oracle.beta(p_root, oracle.softmax(q_node[0], 1.0))
    f = np.mean((n_acc > 0) & (path[:, 0] == 0))
    assert abs(f - beta) < 5 * math.sqrt(beta * (1 - beta) / Bn)
    for c in range(k):
        sel = (n_acc > 0) & (path[:, 0] == c)
        assert sel.sum() > 500
        second = np.where(n_acc[sel] > 1, tokens[sel, np.maximum(path[sel, 1], 0)], nxt[sel])
        ok, chi2 = _chi_square_ok(np.bincount(second, minlength=V), oracle.softmax(t_node[1 + c], 1.0))
        assert ok, (c, chi2)


def test_a_rule_without_renormalisation_would_fail(oracle):
    """The residual must be renormalised before the next candidate is tested: with p_2 = max(0, p - q) left
    unnormalised the second candidate is accepted too rarely and the emitted token no longer follows p.
    (Guards the pin above: it is sharp enough to see that mistake.)"""
    rng = np.random.default_rng(7)
    V, Bn = 4, 40000
    # p_2 = (1/3, 2/3, 0, 0): token 0 has p_2 / q = 1.11 (always accepted), unnormalised 0.33
    p = np.array([0.4, 0.3, 0.2, 0.1]); q = np.array([0.3, 0.1, 0.3, 0.3])
    x = rng.choice(V, size=(Bn, 2), p=q)
    u = rng.random((Bn, 3))
    out = np.zeros(Bn, np.int64)
    for b in range(Bn):
        w = p.copy()
        done = False
        for i in range(2):
            a = min(1.0, w[x[b, i]] / q[x[b, i]])
            if u[b, i] < a:
                out[b] = x[b, i]; done = True
                break
            w = np.maximum(w - q, 0.0)            # the planted mistake: no division by its sum
        if not done:
            c = np.cumsum(w)
            out[b] = int(np.searchsorted(c, u[b, 2] * c[-1], side="right"))
    ok, _ = _chi_square_ok(np.bincount(np.minimum(out, V - 1), minlength=V), p)
    assert not ok
