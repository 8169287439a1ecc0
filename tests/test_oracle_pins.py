"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible slip in the oracle (wrong sign of the residual, entropy in bits,
a non-strict comparison, an off-by-one in the inverse CDF, a transposed p/q)
fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy import special, stats

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def bf16_bits(x):
    """float32 -> bfloat16 bit patterns (round to nearest even)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    return r


def read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append(line.split())
    return rows


# ---------------------------------------------------------------- entropy / softmax

def test_entropy_closed_forms(oracle):
    """Uniform rows give ln V; one logit L above V-1 zeros gives the two-level closed form."""
    for kind, V, L, value in read_table("closed_forms.txt"):
        V = int(V); L = float(L); value = float(value)
        row = np.zeros(V, dtype=np.float32)
        if kind == "spike":
            row[V // 3] = L
        for arr in (row, bf16_bits(row)):
            H = oracle.entropy(oracle.softmax(arr, 1.0))
            assert abs(H - value) < 1e-10 * max(1.0, value), (kind, V, L, H, value)


def test_entropy_uniform_stops_and_onehot_does_not(oracle):
    h = 0.3
    for V in (32000, 152064, 256000):
        row = np.full(V, 1.25, dtype=np.float32)
        tok, H, stop = oracle.draft_step(row, 1.0, h, [0.5 + 0.25 / V])
        assert abs(H[0] - math.log(V)) < 1e-10 and stop[0] == 1
        # uniform row: first i with (i+1)/V > 1/2 + 1/(4V) (off the boundary) is V/2
        assert tok[0] == V // 2
        one = np.full(V, -np.inf, dtype=np.float32)
        one[V - 7] = 3.0
        tok, H, stop = oracle.draft_step(one, 1.0, h, [0.999])
        assert H[0] == 0.0 and stop[0] == 0 and tok[0] == V - 7
        margin = np.zeros(V, dtype=np.float32)
        margin[11] = 60.0
        tok, H, stop = oracle.draft_step(margin, 1.0, h, [0.3])
        assert H[0] < 1e-18 and stop[0] == 0 and tok[0] == 11


def test_two_point_row_is_binary_entropy(oracle):
    for d in (0.0, 0.3, 2.0, 7.5):
        d = float(np.float32(d))
        row = np.array([-np.inf, d, -np.inf, 0.0, -np.inf], dtype=np.float32)
        a = 1.0 / (1.0 + math.exp(-d))
        Hb = -(a * math.log(a) + (1 - a) * math.log(1 - a))
        assert abs(oracle.entropy(oracle.softmax(row, 1.0)) - Hb) < 1e-14


def test_entropy_is_in_nats_not_bits(oracle):
    row = np.zeros(2, dtype=np.float32)
    assert abs(oracle.entropy(oracle.softmax(row, 1.0)) - math.log(2.0)) < 1e-15


def test_softmax_matches_library_and_sums_to_one(oracle):
    rng = np.random.default_rng(11)
    for V, T in ((7, 1.0), (1000, 0.7), (32000, 2.5)):
        row = (rng.standard_normal(V) * 3).astype(np.float32)
        p = oracle.softmax(row, T)
        assert abs(p.sum() - 1.0) < 1e-12
        ref = special.softmax(row.astype(np.float64) / T)
        assert np.max(np.abs(p - ref)) < 1e-13
        lse = special.logsumexp(row.astype(np.float64) / T)
        assert np.max(np.abs(np.log(p) - (row.astype(np.float64) / T - lse))) < 1e-10
        # bf16 bit patterns decode to the same values as their float32 expansion
        b = bf16_bits(row)
        as_f32 = (b.astype(np.uint32) << 16).view(np.float32)
        assert np.array_equal(oracle.softmax(b, T), oracle.softmax(as_f32, T))


def test_entropy_shift_invariance_and_temperature_monotone(oracle):
    rng = np.random.default_rng(5)
    row = (rng.standard_normal(512) * 2).astype(np.float32)
    H0 = oracle.entropy(oracle.softmax(row, 1.0))
    H1 = oracle.entropy(oracle.softmax((row.astype(np.float64) + 8.0).astype(np.float32), 1.0))
    assert abs(H0 - H1) < 1e-5  # float32 rounding of the shifted row only
    Hs = [oracle.entropy(oracle.softmax(row, T)) for T in (0.25, 0.5, 1.0, 2.0, 4.0, 50.0)]
    assert all(a < b for a, b in zip(Hs, Hs[1:]))
    assert Hs[-1] < math.log(512)


def test_greedy_entropy_is_temperature_one(oracle):
    rng = np.random.default_rng(6)
    row = (rng.standard_normal(300) * 2).astype(np.float32)
    _, Hg, _ = oracle.draft_step(row, 0.0, 0.3, [0.1])
    assert abs(Hg[0] - oracle.entropy(oracle.softmax(row, 1.0))) < 1e-15


# ---------------------------------------------------------------- stop rule (Eq. 7)

def test_stop_rule_flips_exactly_at_threshold(oracle):
    """Two-point rows have closed-form H; the flag must flip where sqrt(H) crosses h, strictly."""
    for d in (1.0, 3.0, 4.5, 6.0):
        row = np.array([d, 0.0], dtype=np.float32)
        a = 1.0 / (1.0 + math.exp(-d))
        H = -(a * math.log(a) + (1 - a) * math.log(1 - a))
        s = math.sqrt(H)
        for h, want in ((s * (1 - 1e-9), 1), (s * (1 + 1e-9), 0)):
            _, Ho, stop = oracle.draft_step(row, 1.0, h, [0.0])
            assert stop[0] == want, (d, h, s, Ho)
        # strictness: h equal to the oracle's own sqrt(H) must not stop
        _, Ho, _ = oracle.draft_step(row, 1.0, 0.0, [0.0])
        _, _, stop = oracle.draft_step(row, 1.0, math.sqrt(Ho[0]), [0.0])
        assert stop[0] == 0


def test_threshold_reparametrisation(oracle):
    """1 - sqrt(c H) < h_hat  <=>  sqrt(H) > h with h = (1 - h_hat)/sqrt(c) (text before Eq. 7)."""
    consts = {k: float(v) for k, v in read_table("paper_constants.txt")}
    c, h = consts["c"], consts["h"]
    h_hat = 1.0 - h * math.sqrt(c)
    for d in np.linspace(0.0, 9.0, 37):
        row = np.array([d, 0.0, 0.0], dtype=np.float32)
        _, H, stop = oracle.draft_step(row, 1.0, h, [0.0])
        lhs = 1.0 - math.sqrt(c * H[0]) < h_hat
        if abs(math.sqrt(H[0]) - h) > 1e-9:
            assert bool(stop[0]) == lhs


# ---------------------------------------------------------------- inverse CDF

def test_invcdf_step_function(oracle):
    w = np.array([0.0, 2.0, 0.0, 1.0, 1.0, 0.0])
    # cumulative/total: 0, .5, .5, .75, 1, 1 ; first index whose cumulative EXCEEDS u
    cases = [(0.0, 1), (0.49, 1), (0.5, 3), (0.74, 3), (0.75, 4), (0.999999, 4)]
    for u, want in cases:
        assert oracle.invcdf(w, u) == want
    # rounding fallback: nothing exceeds -> last index with positive weight
    assert oracle.invcdf(w, 1.0) == 4


def test_invcdf_interval_measure(oracle):
    rng = np.random.default_rng(3)
    w = rng.random(9)
    w[[2, 5]] = 0.0
    N = 1 << 14
    toks = np.array([oracle.invcdf(w, (k + 0.5) / N) for k in range(N)])
    freq = np.bincount(toks, minlength=9) / N
    assert np.max(np.abs(freq - w / w.sum())) <= 1.0 / N + 1e-12
    assert np.all(np.diff(toks) >= 0)


# ---------------------------------------------------------------- accept test (Algorithm 2, Eq. 1)

def _verify_one(oracle, x, q_rows, t_rows, T, r):
    K = len(x)
    cu = np.array([0, K + 1])
    n, nx, a = oracle.verify(np.asarray(x, np.int32), q_rows, t_rows, cu, T, np.asarray(r, np.float64),
                             want_accept_prob=True)
    return int(n[0]), int(nx[0]), a[0]


def test_identical_distributions_always_accept(oracle):
    rng = np.random.default_rng(21)
    V, K = 50, 4
    q_rows = (rng.standard_normal((K, V)) * 2).astype(np.float32)
    t_rows = np.concatenate([q_rows, (rng.standard_normal((1, V))).astype(np.float32)])
    top = 1.0 - 2.0 ** -24
    for r_val in (0.0, 0.5, top):
        for x in ([0, 1, 2, 3], [49, 7, 7, 30]):
            n, nx, a = _verify_one(oracle, x, q_rows, t_rows, 1.0, [r_val] * K + [0.25])
            assert n == K and np.all(a == 1.0)
            assert nx == oracle.invcdf(oracle.softmax(t_rows[K], 1.0), 0.25)


def test_zero_target_probability_always_rejects(oracle):
    V = 6
    q_rows = np.zeros((1, V), dtype=np.float32)
    t_rows = np.zeros((2, V), dtype=np.float32)
    t_rows[0, 2] = -np.inf
    for r_val in (0.0, 1e-300, 0.9):
        n, nx, a = _verify_one(oracle, [2], q_rows, t_rows, 1.0, [r_val, 0.5])
        assert n == 0 and a[0] == 0.0 and nx != 2


def test_token_outside_draft_support_is_accepted_iff_target_has_it(oracle):
    """q(x) = 0 < p(x): the ratio of Algorithm 2 is +inf, so min(1, p/q) = 1 and every r in [0,1)
    accepts (the limit of p/q as q -> 0+ shows it: the acceptance probability rises to 1 and stays).
    q(x) = 0 = p(x): nothing to accept, rejected for every r."""
    V = 6
    top = 1.0 - 2.0 ** -24
    t_rows = np.zeros((2, V), dtype=np.float32)
    t_rows[0] = [0.3, -1.0, 0.5, 0.0, 2.0, -0.7]
    for x in range(V):
        q_rows = np.array([[0.1, 0.2, -0.4, 1.0, 0.0, 0.6]], dtype=np.float32)
        q_rows[0, x] = -np.inf
        for r_val in (0.0, 0.5, top):
            n, nx, a = _verify_one(oracle, [x], q_rows, t_rows, 1.0, [r_val, 0.5])
            assert a[0] == 1.0 and n == 1
            assert nx == oracle.invcdf(oracle.softmax(t_rows[1], 1.0), 0.5)
        # the limit: the draft logit of x sinks, the acceptance probability rises to 1 and stays there
        last = 0.0
        for lx in (0.0, -5.0, -20.0, -80.0, -700.0, -1e30):
            q_rows[0, x] = lx
            _, _, a = _verify_one(oracle, [x], q_rows, t_rows, 1.0, [0.0, 0.5])
            assert a[0] >= last
            last = a[0]
        assert last == 1.0
        # both models exclude x: rejected whatever the draw, and the correction avoids x
        q_rows[0, x] = -np.inf
        t2 = t_rows.copy(); t2[0, x] = -np.inf
        for r_val in (0.0, top):
            n, nx, a = _verify_one(oracle, [x], q_rows, t2, 1.0, [r_val, 0.5])
            assert a[0] == 0.0 and n == 0 and nx != x


def test_accept_probability_is_min_one_ratio(oracle):
    rng = np.random.default_rng(8)
    V = 12
    q_row = (rng.standard_normal((1, V)) * 1.5).astype(np.float32)
    t_rows = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    for T in (1.0, 0.7):
        p = special.softmax(t_rows[0].astype(np.float64) / T)
        q = special.softmax(q_row[0].astype(np.float64) / T)
        for x in range(V):
            _, _, a = _verify_one(oracle, [x], q_row, t_rows, T, [0.0, 0.0])
            assert abs(a[0] - min(1.0, p[x] / q[x])) < 1e-13
            # strict comparison r < a: just below accepts, at-or-above rejects
            if a[0] < 1.0:
                n_lo, _, _ = _verify_one(oracle, [x], q_row, t_rows, T, [a[0] * (1 - 1e-12), 0.0])
                n_eq, _, _ = _verify_one(oracle, [x], q_row, t_rows, T, [a[0], 0.0])
                assert n_lo == 1 and n_eq == 0


def test_beta_identities_and_pinsker(oracle):
    """Eq. 1-4: beta = sum min = 1 - TVD >= 1 - sqrt(KL(q||p)/2); residual mass = 1 - beta."""
    rng = np.random.default_rng(4)
    for V in (5, 300, 32000):
        for scale in (0.3, 1.0, 4.0):
            d = (rng.standard_normal(V) * scale).astype(np.float32)
            t = (d + rng.standard_normal(V).astype(np.float32) * 0.5).astype(np.float32)
            p = oracle.softmax(t, 1.0); q = oracle.softmax(d, 1.0)
            b = oracle.beta(p, q)
            assert abs(b - (1.0 - oracle.tvd(p, q))) < 1e-12
            kl = oracle.cross_entropy(q, p) - oracle.entropy(q)
            assert kl >= -1e-12
            assert b >= 1.0 - math.sqrt(max(kl, 0.0) / 2.0) - 1e-12
            assert b >= 1.0 - math.sqrt(1.0 - math.exp(-max(kl, 0.0))) - 1e-12  # Bretagnolle-Huber, appendix B
            w, S = oracle.residual(p, q)
            assert abs(S - (1.0 - b)) < 1e-12
            assert np.all(w[q >= p] == 0.0) and np.all(w[p > q] > 0.0)


def test_empirical_acceptance_equals_beta(oracle):
    """Draft tokens drawn from q by the oracle's own sampler are accepted with frequency beta (Eq. 1)."""
    rng = np.random.default_rng(77)
    V, N = 7, 120000
    d = (rng.standard_normal((1, V)) * 1.2).astype(np.float32)
    t = (rng.standard_normal((2, V)) * 1.2).astype(np.float32)
    p = oracle.softmax(t[0], 1.0); q = oracle.softmax(d[0], 1.0)
    b = oracle.beta(p, q)
    us = rng.random((N, 3))
    acc = 0
    for k in range(N):
        x, _, _ = oracle.draft_step(d, 1.0, 0.3, [us[k, 0]])
        n, _, _ = _verify_one(oracle, [int(x[0])], d, t, 1.0, [us[k, 1], us[k, 2]])
        acc += n
    sigma = math.sqrt(b * (1 - b) / N)
    assert abs(acc / N - b) < 5 * sigma


# ---------------------------------------------------------------- correction token (Algorithm 4)

def test_correction_never_lands_where_draft_dominates(oracle):
    rng = np.random.default_rng(9)
    V = 10
    d = (rng.standard_normal((1, V)) * 2).astype(np.float32)
    t = (rng.standard_normal((2, V)) * 2).astype(np.float32)
    p = oracle.softmax(t[0], 1.0); q = oracle.softmax(d[0], 1.0)
    x = int(np.argmax(q / p))          # a token with p/q < 1
    assert p[x] / q[x] < 0.99
    seen = set()
    for u in np.linspace(0.0, 0.99999, 4001):
        n, nx, _ = _verify_one(oracle, [x], d, t, 1.0, [0.999, u])
        assert n == 0
        seen.add(nx)
    assert seen == set(np.nonzero(p > q)[0].tolist())


def test_disjoint_supports_correction_follows_target(oracle):
    V = 8
    d = np.full((1, V), -np.inf, dtype=np.float32); d[0, :4] = [0.0, 1.0, 0.5, -0.3]
    t = np.full((2, V), -np.inf, dtype=np.float32); t[0, 4:] = [0.2, 1.5, -1.0, 0.0]; t[1, :] = 0.0
    p = oracle.softmax(t[0], 1.0)
    N = 1 << 13
    toks = [_verify_one(oracle, [1], d, t, 1.0, [0.0, (k + 0.5) / N])[1] for k in range(N)]
    freq = np.bincount(toks, minlength=V) / N
    assert np.max(np.abs(freq - p)) <= 1.0 / N + 1e-12


# ---------------------------------------------------------------- greedy (Algorithms 3 and 5)

def test_greedy_verify_by_hand(oracle):
    V = 6
    t = np.array([[0, 5, 1, 5, 0, 0],      # tie between 1 and 3 -> lowest index 1
                  [9, 0, 0, 0, 0, 0],
                  [0, 0, 0, 0, 2, 2],      # tie 4/5 -> 4
                  [1, 2, 3, 4, 5, 6]], dtype=np.float32)
    d = np.zeros((3, V), dtype=np.float32)
    assert _verify_one(oracle, [1, 0, 4], d, t, 0.0, [0, 0, 0, 0])[:2] == (3, 5)
    assert _verify_one(oracle, [3, 0, 4], d, t, 0.0, [0, 0, 0, 0])[:2] == (0, 1)
    assert _verify_one(oracle, [1, 0, 5], d, t, 0.0, [0, 0, 0, 0])[:2] == (2, 4)
    assert _verify_one(oracle, [1, 2, 4], d, t, 0.0, [0, 0, 0, 0])[:2] == (1, 0)
    tb = bf16_bits(t)
    assert _verify_one(oracle, [1, 0, 4], bf16_bits(d), tb, 0.0, [0, 0, 0, 0])[:2] == (3, 5)
    tok, _, _ = oracle.draft_step(t, 0.0, 0.3, [0.9, 0.9, 0.9, 0.9])
    assert tok.tolist() == [1, 0, 4, 5]


# ---------------------------------------------------------------- the whole round

def _round_law_by_enumeration(oracle, d, t, T, K, V, N):
    """Law of (n_accepted, token emitted at position n_accepted) by enumerating all V^K draft
    tuples.  Accept probabilities come from the oracle; the law of the corrected / bonus token comes
    from running the oracle's sampler over a dense grid of the last uniform."""
    q = [oracle.softmax(d[j], T) for j in range(K)]
    law = np.zeros((K + 1, V))
    reach_check = np.zeros(K + 1)
    grid = (np.arange(N) + 0.5) / N
    for x in itertools.product(range(V), repeat=K):
        wq = math.prod(q[j][x[j]] for j in range(K))
        _, _, a = _verify_one(oracle, list(x), d, t, T, [0.0] * (K + 1))
        reach = 1.0
        for j in range(K + 1):
            # outcome "first rejection at j" (or "all accepted" for j == K)
            pr = reach * ((1.0 - a[j]) if j < K else 1.0)
            if pr > 0.0:
                r = [0.0] * (K + 1)
                if j < K:
                    r[j] = 0.9999999999
                    if not (r[j] >= a[j]):
                        pr = 0.0
                if pr > 0.0:
                    hist = np.zeros(V)
                    for u in grid:
                        r[K] = u
                        n, nx, _ = _verify_one(oracle, list(x), d, t, T, r)
                        assert n == j
                        hist[nx] += 1.0 / N
                    law[j] += wq * pr * hist
                    reach_check[j] += wq * pr
            if j < K:
                reach *= a[j]
    return law, reach_check


def test_brute_force_round_law(oracle):
    """V=4, K=2, every draft tuple: the token emitted at each position follows the target row, and
    P(n_accepted >= j) = prod_{i<j} beta_i.  Fails for the residual sign as printed in Algorithm 4."""
    rng = np.random.default_rng(31)
    V, K, N = 4, 2, 512
    d = (rng.standard_normal((K, V)) * 1.3).astype(np.float32)
    t = (rng.standard_normal((K + 1, V)) * 1.3).astype(np.float32)
    for T in (1.0, 0.6):
        law, reach = _round_law_by_enumeration(oracle, d, t, T, K, V, N)
        p = [oracle.softmax(t[j], T) for j in range(K + 1)]
        q = [oracle.softmax(d[j], T) for j in range(K)]
        betas = [oracle.beta(p[j], q[j]) for j in range(K)]
        surv = 1.0
        for j in range(K + 1):
            # P(first rejection at j) = prod_{i<j} beta_i * (1 - beta_j); all accepted for j == K
            want = surv * ((1.0 - betas[j]) if j < K else 1.0)
            assert abs(reach[j] - want) < 1e-12
            if j < K:
                # token finally placed at position j given position j was reached:
                # accepted draft (min(p,q)) + correction ((1-beta) * residual) == p_j
                placed = np.minimum(p[j], q[j]) * surv + law[j]
                assert np.max(np.abs(placed - surv * p[j])) < 2.0 * V / N
                surv *= betas[j]
            else:
                assert np.max(np.abs(law[j] - surv * p[K])) < 2.0 * V / N


def test_chi_square_draft_then_verify_follows_target(oracle):
    """Draft K tokens from q with the oracle's sampler, verify, and histogram the token that ends
    up at position 0 and the bonus token: both must follow the target rows (chi-square, alpha=1e-3)."""
    rng = np.random.default_rng(1234)
    V, K, N = 6, 3, 100000
    d = (rng.standard_normal((K, V)) * 1.1).astype(np.float32)
    t = (d[:1].repeat(K + 1, 0) * 0 + rng.standard_normal((K + 1, V)) * 1.1).astype(np.float32)
    t[1] = d[1] + 0.2 * rng.standard_normal(V).astype(np.float32)   # close rows so the bonus is reached
    t[2] = d[2] + 0.2 * rng.standard_normal(V).astype(np.float32)
    t[0] = d[0] + 0.4 * rng.standard_normal(V).astype(np.float32)
    p = [oracle.softmax(t[j], 1.0) for j in range(K + 1)]
    q = [oracle.softmax(d[j], 1.0) for j in range(K)]
    us = rng.random((N, 2 * K + 1))
    first = np.zeros(V); bonus = np.zeros(V); nacc_hist = np.zeros(K + 1)
    for k in range(N):
        x, _, _ = oracle.draft_step(d, 1.0, 0.3, us[k, :K])
        n, nx, _ = _verify_one(oracle, x.tolist(), d, t, 1.0, us[k, K:])
        nacc_hist[n] += 1
        first[x[0] if n >= 1 else nx] += 1
        if n == K:
            bonus[nx] += 1
    chi_first = ((first - N * p[0]) ** 2 / (N * p[0])).sum()
    assert chi_first < stats.chi2.ppf(1 - 1e-3, V - 1), (chi_first, first / N, p[0])
    nb = bonus.sum()
    assert nb > 2000
    chi_bonus = ((bonus - nb * p[K]) ** 2 / (nb * p[K])).sum()
    assert chi_bonus < stats.chi2.ppf(1 - 1e-3, V - 1)
    betas = [oracle.beta(p[j], q[j]) for j in range(K)]
    surv = np.cumprod([1.0] + betas)            # P(n_acc >= j)
    want = np.array([surv[j] * (1 - betas[j]) for j in range(K)] + [surv[K]])
    chi_n = ((nacc_hist - N * want) ** 2 / (N * want)).sum()
    assert chi_n < stats.chi2.ppf(1 - 1e-3, K)


def test_residual_sign_as_printed_would_fail(oracle):
    """The printed sign max(q-p,0) makes the emitted law collapse towards q; the law with the
    oracle's sign equals p.  Guards the reading of Algorithm 4 against a silent flip."""
    rng = np.random.default_rng(2)
    V = 5
    d = (rng.standard_normal(V) * 1.5).astype(np.float32)
    t = (rng.standard_normal(V) * 1.5).astype(np.float32)
    p = oracle.softmax(t, 1.0); q = oracle.softmax(d, 1.0)
    w, S = oracle.residual(p, q)
    law_good = np.minimum(p, q) + (1 - oracle.beta(p, q)) * w / S
    w_bad = np.maximum(q - p, 0.0)
    law_bad = np.minimum(p, q) + (1 - oracle.beta(p, q)) * w_bad / w_bad.sum()
    assert np.max(np.abs(law_good - p)) < 1e-14
    assert np.max(np.abs(law_bad - q)) < 1e-14 and np.max(np.abs(law_bad - p)) > 1e-2


# ---------------------------------------------------------------- analysis quantities (Eq. 1-6, appendix B)

def test_pair_stats_closed_forms(oracle):
    """Two-token rows: everything has a closed form.  p = (a, 1-a), q = (b, 1-b)."""
    consts = {k: float(v) for k, v in read_table("paper_constants.txt")}
    for dp, dq in ((0.0, 0.0), (1.0, -0.5), (2.5, 0.25), (-1.0, 3.0)):
        t = np.array([[dp, 0.0]], dtype=np.float32); d = np.array([[dq, 0.0]], dtype=np.float32)
        for T in (1.0, 0.5):
            a = 1.0 / (1.0 + math.exp(-dp / T)); b = 1.0 / (1.0 + math.exp(-dq / T))
            out = oracle.pair_stats(t, d, T, consts["c"])[0]
            beta = min(a, b) + min(1 - a, 1 - b)
            Hq = -(b * math.log(b) + (1 - b) * math.log(1 - b))
            Hqp = -(b * math.log(a) + (1 - b) * math.log(1 - a))
            KL = b * math.log(b / a) + (1 - b) * math.log((1 - b) / (1 - a))
            want = [beta, Hq, Hqp, KL, Hqp / Hq, 1 - math.sqrt(KL / 2), 1 - math.sqrt(1 - math.exp(-KL)),
                    1 - math.sqrt(consts["c"] * Hq)]
            assert np.allclose(out, want, rtol=1e-11, atol=1e-12), (dp, dq, T, out, want)
            assert abs(out[3] - (out[2] - out[1])) < 1e-15


def test_pair_stats_inequalities_and_gamma_condition(oracle):
    """beta >= both lower bounds; the approximation bound is conservative exactly when
    gamma <= 2c + 1 (the condition stated for the constant c); p == q gives beta = 1, KL = 0, gamma = 1."""
    rng = np.random.default_rng(17)
    V = 2000
    d = (rng.standard_normal((40, V)) * rng.uniform(0.3, 4.0, size=(40, 1))).astype(np.float32)
    t = (d + rng.standard_normal((40, V)).astype(np.float32) * rng.uniform(0.05, 1.5, size=(40, 1))).astype(np.float32)
    for c in (0.18, 0.5, 2.0):
        out = oracle.pair_stats(t, d, 1.0, c)
        beta, Hq, Hqp, KL, gamma, pin, bh, approx = out.T
        assert np.all(beta >= pin - 1e-12) and np.all(beta >= bh - 1e-12) and np.all(bh >= 0)
        assert np.all(KL >= -1e-12) and np.all(gamma >= 1 - 1e-12)
        conservative = approx <= pin + 1e-12
        assert np.array_equal(conservative, gamma <= 2 * c + 1 + 1e-12)
        assert np.allclose(pin, 1 - np.sqrt(0.5 * (gamma - 1) * Hq), atol=1e-12)     # Eq. 5
    same = oracle.pair_stats(d[:3], d[:3], 0.7, 0.18)
    assert np.allclose(same[:, 0], 1.0, atol=1e-12) and np.allclose(same[:, 3], 0.0, atol=1e-12)
    assert np.allclose(same[:, 4], 1.0, atol=1e-12)


def test_gamma_of_a_one_hot_draft_row(oracle):
    """gamma = H_qp / H_q = 1 + KL / H_q (Section 2.2 with Eq. 4).  For a one-hot draft row H_q = 0: with KL = 0
    (the target puts all its mass on the same token) gamma - 1 = KL / H_q is 0 along every path to that point,
    so gamma = 1; with KL > 0 the ratio diverges: +inf.  Never NaN."""
    V = 7
    q = np.full((1, V), -np.inf, dtype=np.float32); q[0, 3] = 1.5
    same = q.copy()
    spread = np.zeros((1, V), dtype=np.float32)
    out = oracle.pair_stats(np.concatenate([same, spread]), np.concatenate([q, q]), 1.0, 0.18)
    assert out[0, 1] == 0.0 and out[0, 3] == 0.0 and out[0, 4] == 1.0 and out[0, 0] == 1.0
    assert out[1, 1] == 0.0 and abs(out[1, 3] - math.log(V)) < 1e-12 and out[1, 4] == np.inf
    assert not np.isnan(out).any()
    # approaching the one-hot row: gamma stays finite and tends to 1 when p follows q
    for L in (5.0, 20.0, 40.0):
        d = np.zeros((1, V), dtype=np.float32); d[0, 3] = L
        o = oracle.pair_stats(d, d, 1.0, 0.18)
        assert abs(o[0, 4] - 1.0) < 1e-9


# ---------------------------------------------------------------- ragged packing

def test_pack_ragged_is_exclusive_scan(oracle):
    lens = [3, 1, 64, 2]
    cu, seq, pos = oracle.pack_ragged(lens)
    assert cu.tolist() == [0, 4, 6, 71, 74]
    assert np.array_equal(cu[1:], np.cumsum(np.array(lens) + 1))
    for r in range(cu[-1]):
        assert cu[seq[r]] + pos[r] == r and 0 <= pos[r] <= lens[seq[r]]
