"""Pins of the draft-length policy loops (Algorithm 1 inner loop; Section 3 baselines), by inspection."""
from oracle import svip_policy as P


def run_round(policy, stops_per_step, gamma, K_cap):
    B = len(gamma)
    draft_len, active = [0] * B, [1] * B
    steps = 0
    while any(active):
        stop = stops_per_step[steps] if steps < len(stops_per_step) else [0] * B
        P.advance(policy, stop, gamma, draft_len, active, K_cap)
        steps += 1
    return draft_len, steps


def test_entropy_policy_stops_at_first_flag_or_cap():
    stops = [[0, 1, 0], [0, 0, 0], [1, 1, 0], [0, 0, 0]]
    lens, steps = run_round(P.ENTROPY, stops, [5, 5, 5], 6)
    assert lens == [3, 1, 6] and steps == 6      # the third sequence never sees a flag: the cap ends it


def test_constant_policy_drafts_exactly_gamma():
    lens, steps = run_round(P.CONSTANT, [[1, 1, 1]] * 10, [5, 2, 50], 40)
    assert lens == [5, 2, 40] and steps == 40     # stop flags are ignored; gamma above the cap is clipped


def test_heuristic_policy_plus_two_minus_one():
    gamma, K_cap = [5, 5, 1, 39], 40
    draft_len, active = [5, 5, 1, 39], [0, 0, 0, 0]
    P.update(P.HEURISTIC, [5, 3, 0, 39], draft_len, gamma, active, K_cap)
    assert gamma == [7, 4, 1, 40]                 # all accepted: +2 (capped); otherwise -1 (floored at 1)
    assert draft_len == [0, 0, 0, 0] and active == [1, 1, 1, 1]
    seq = []
    g, d, a = [5], [0], [1]
    for accepted_all in (True, True, False, False, False, True):
        d[0] = g[0]
        P.update(P.HEURISTIC, [g[0] if accepted_all else 0], d, g, a, K_cap)
        seq.append(g[0])
    assert seq == [7, 9, 8, 7, 6, 8]
    g2 = [5]
    P.update(P.CONSTANT, [5], [5], g2, [0], K_cap)
    assert g2 == [5]
