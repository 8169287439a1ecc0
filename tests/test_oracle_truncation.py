"""Pins of the oracle's top-k / nucleus truncation (the paper does not define it; the oracle follows the
published definitions with a threshold reading of ties).  Hand-made rows, an independent brute-force
construction of the kept set, the defining inequalities, the special cases that reduce to the plain
path, and the law of the emitted token on a tiny vocabulary."""
import math

import numpy as np
import pytest
from scipy import stats


def bf16_bits(x):
    b = np.asarray(x, dtype=np.float32).view(np.uint32)
    return ((b + 0x7FFF + ((b >> 16) & 1)) >> 16).astype(np.uint16)


def bf16_values(b):
    return (b.astype(np.uint32) << 16).view(np.float32)


def test_top_k_by_hand(oracle):
    l = np.array([[3, 1, 2, 2, 0]], dtype=np.float32)
    tau, Zk, Zt, n = oracle.threshold(l, 1.0, 2, 1.0)
    # second largest is 2; both 2s tie with it and stay: {3, 2, 2}
    assert tau[0] == 2.0 and n[0] == 3
    assert abs(Zt[0] - (1 + 2 * math.exp(-1))) < 1e-15 and Zk[0] == Zt[0]
    tau, _, Zt, n = oracle.threshold(l, 1.0, 1, 1.0)
    assert tau[0] == 3.0 and n[0] == 1 and Zt[0] == 1.0
    for k in (0, 5, 9):          # off, or not below V: nothing is dropped
        tau, _, _, n = oracle.threshold(l, 1.0, k, 1.0)
        assert tau[0] == 0.0 and n[0] == 5
    assert np.array_equal(oracle.mask_below(l, [2.0]), np.array([[3, -np.inf, 2, 2, -np.inf]], dtype=np.float32))


def test_nucleus_by_hand(oracle):
    probs = np.array([0.5, 0.2, 0.2, 0.1])
    l = np.log(probs)[None, :].astype(np.float32)
    # 0.5 >= 0.45: the most likely token alone
    tau, _, Zt, n = oracle.threshold(l, 1.0, 0, 0.45)
    assert n[0] == 1 and tau[0] == l[0, 0]
    # 0.5 < 0.6: the next group is the two tied tokens, both kept (0.9 of the mass)
    tau, Zk, Zt, n = oracle.threshold(l, 1.0, 0, 0.6)
    assert n[0] == 3 and tau[0] == l[0, 1] and abs(Zt[0] / Zk[0] - 0.9) < 1e-6
    tau, _, _, n = oracle.threshold(l, 1.0, 0, 0.95)
    assert n[0] == 4
    # top-k first, the nucleus inside it: k = 3 keeps {0.5, 0.2, 0.2} (mass 0.9); 0.5/0.9 < 0.6
    tau, Zk, Zt, n = oracle.threshold(l, 1.0, 3, 0.6)
    assert n[0] == 3 and abs(Zk[0] / 2.0 - 0.9) < 1e-6
    tau, Zk, Zt, n = oracle.threshold(l, 1.0, 3, 0.55)
    assert n[0] == 1             # 0.5/0.9 = 0.556 >= 0.55
    # temperature sharpens the distribution before the nucleus is taken
    tau, _, _, n = oracle.threshold(l, 0.5, 0, 0.6)   # probs^2 normalised: 0.735, ...
    assert n[0] == 1


def brute_kept_set(values, T, k, p):
    """Independent construction: for every candidate cut value, count and weigh the tokens at or above it."""
    v = values.astype(np.float64)
    V = v.size
    w = np.exp(v / T - v.max() / T)
    cands = np.unique(v)[::-1]                       # distinct values, descending
    if 1 <= k < V:
        tau_k = [c for c in cands if (v > c).sum() < k <= (v >= c).sum()][0]
    else:
        tau_k = cands[-1]
    Zk = w[v >= tau_k].sum()
    tau = tau_k
    if p < 1.0:
        ok = [c for c in cands if c >= tau_k and w[v >= c].sum() >= p * Zk]
        tau = max(ok)
    return tau, v >= tau


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_threshold_against_brute_force(oracle, dtype):
    rng = np.random.default_rng(11)
    n_checked = 0
    for trial in range(60):
        V = int(rng.integers(5, 400))
        x = (rng.standard_normal(V) * rng.uniform(0.2, 5.0)).astype(np.float32)
        if dtype == "bf16":
            row = bf16_bits(x); vals = bf16_values(row)          # plenty of exact ties
        else:
            row = x.copy(); row[rng.integers(0, V, size=V // 4)] = row[0]   # planted ties
            vals = row
        T = float(rng.choice([0.5, 1.0, 1.7]))
        k = int(rng.choice([0, 1, 2, V // 3 + 1, V - 1, V]))
        p = float(rng.choice([1.0, 0.97, 0.8, 0.31]))
        tau_b, kept_b = brute_kept_set(vals, T, k, p)
        # the comparison of sums against p * Z_k is the only place where summation order could matter:
        # skip draws whose margin is at rounding level
        w = np.exp(vals.astype(np.float64) / T - float(vals.max()) / T)
        Zk = w[vals >= (np.sort(vals)[::-1][k - 1] if 1 <= k < V else vals.min())].sum()
        margins = [abs(w[vals >= c].sum() - p * Zk) for c in np.unique(vals)]
        if p < 1.0 and min(margins) < 1e-9 * Zk:
            continue
        tau, _, Zt, n = oracle.threshold(row[None, :], T, k, p)
        assert tau[0] == tau_b, (trial, V, T, k, p)
        assert n[0] == kept_b.sum()
        assert abs(Zt[0] - w[kept_b].sum()) <= 1e-12 * Zt[0]
        masked = oracle.mask_below(row[None, :], tau)[0]
        mv = bf16_values(masked) if dtype == "bf16" else masked
        assert np.array_equal(np.isfinite(mv) | (vals == -np.inf), kept_b | (vals == -np.inf))
        n_checked += 1
    assert n_checked > 40


def test_defining_inequalities(oracle):
    """Fewer than k tokens lie strictly above tau_k; the kept mass reaches top_p of the top-k mass and would
    not without the lowest kept group."""
    rng = np.random.default_rng(3)
    V = 3000
    rows = bf16_bits(rng.standard_normal((8, V)) * 3.0)
    vals = bf16_values(rows).astype(np.float64)
    for k, p in ((50, 1.0), (0, 0.9), (200, 0.7)):
        tau, Zk, Zt, n = oracle.threshold(rows, 1.0, k, p)
        for r in range(8):
            v = vals[r]; w = np.exp(v - v.max())
            if k:
                tk = np.sort(v)[::-1][k - 1]
                assert (v > tk).sum() < k <= (v >= tk).sum()
                assert abs(Zk[r] - w[v >= tk].sum()) < 1e-10 * Zk[r]
                assert tau[r] >= tk
            if p < 1.0:
                assert Zt[r] >= p * Zk[r] * (1 - 1e-12)
                assert w[v > tau[r]].sum() < p * Zk[r] * (1 + 1e-12)
            assert n[r] == (v >= tau[r]).sum()


def test_no_truncation_is_the_plain_path(oracle):
    rng = np.random.default_rng(5)
    l = (rng.standard_normal((6, 777)) * 2).astype(np.float32)
    u = rng.random(6)
    a = oracle.draft_step(l, 0.8, 0.3, u)
    b = oracle.draft_step_filtered(l, 0.8, 0.3, u, 0, 1.0)
    c = oracle.draft_step_filtered(l, 0.8, 0.3, u, 777, 1.0)
    for x, y, z in zip(a, b, c):
        assert np.array_equal(x, y) and np.array_equal(x, z)


def test_top_1_is_the_argmax_with_zero_entropy(oracle):
    rng = np.random.default_rng(6)
    l = (rng.standard_normal((5, 300)) * 2).astype(np.float32)      # no ties in continuous draws
    tok, H, stop = oracle.draft_step_filtered(l, 1.0, 0.3, rng.random(5), 1, 1.0)
    assert np.array_equal(tok, l.argmax(axis=1)) and np.all(H == 0.0) and not stop.any()
    # tied maxima all stay: the draw picks among them in index order, H = ln(ties) and its root exceeds 0.3
    l[0, 7] = l[0].max(); l[0, 200] = l[0].max()
    ties = np.nonzero(l[0] == l[0].max())[0]
    tok, H, stop = oracle.draft_step_filtered(l[:1], 1.0, 0.3, [0.75], 1, 1.0)
    assert tok[0] == ties[int(0.75 * len(ties))] and abs(H[0] - math.log(len(ties))) < 1e-12 and stop[0] == 1


def test_truncated_entropy_and_tokens(oracle):
    """H is the entropy of the renormalised kept set; tokens never leave it; H never exceeds ln(n_kept)."""
    rng = np.random.default_rng(7)
    V = 2000
    l = (rng.standard_normal((4, V)) * 2.5).astype(np.float32)
    tau, _, Zt, n = oracle.threshold(l, 1.0, 40, 0.9)
    for r in range(4):
        us = rng.random(300)
        tok, H, _ = oracle.draft_step_filtered(np.repeat(l[r:r + 1], 300, 0), 1.0, 0.3, us, 40, 0.9)
        assert np.all(l[r, tok] >= tau[r])
        keep = l[r] >= tau[r]
        q = np.exp(l[r, keep].astype(np.float64) - l[r].max()); q /= q.sum()
        assert abs(H[0] - -(q * np.log(q)).sum()) < 1e-12
        assert H[0] <= math.log(n[r]) + 1e-12


def test_chi_square_truncated_round_follows_the_truncated_target(oracle):
    """Draft from the truncated q, verify against the truncated p: the token emitted at position 0 follows
    the truncated target exactly (so never a token the target's truncation dropped)."""
    rng = np.random.default_rng(78)
    V, K, N = 7, 2, 60000
    d = (rng.standard_normal((K, V)) * 0.8).astype(np.float32)
    t = (d[[0, 1, 1]] + 0.5 * rng.standard_normal((K + 1, V))).astype(np.float32)
    k, p = 5, 0.85
    tau_t, _, _, n_t = oracle.threshold(t, 1.0, k, p)
    assert 1 < n_t[0] < V
    p0 = oracle.softmax(oracle.mask_below(t[:1], tau_t[:1])[0], 1.0)
    us = rng.random((N, 2 * K + 1))
    x, _, _ = oracle.draft_step_filtered(np.tile(d, (N, 1)), 1.0, 0.3, us[:, :K].reshape(-1), k, p, threads=4)
    x = x.reshape(N, K)
    cu = np.arange(N + 1) * (K + 1)
    n_acc, nxt, _ = oracle.verify_filtered(x.reshape(-1).astype(np.int32), np.tile(d, (N, 1)), np.tile(t, (N, 1)), cu,
                                           1.0, us[:, K:].reshape(-1), k, p, threads=4)
    first = np.where(n_acc >= 1, x[:, 0], nxt)
    hist = np.bincount(first, minlength=V).astype(np.float64)
    assert np.all(hist[p0 == 0] == 0)
    live = p0 > 0
    chi = ((hist[live] - N * p0[live]) ** 2 / (N * p0[live])).sum()
    assert chi < stats.chi2.ppf(1 - 1e-3, live.sum() - 1), (chi, hist / N, p0)
