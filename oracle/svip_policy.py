"""Draft-length policies as plain integer loops -- TEST INFRASTRUCTURE ONLY (see svip_oracle.c).

The three policies of the paper, per sequence:
  entropy    Algorithm 1: keep drafting until the stop test of Eq. 7 fires (or the cap is reached)
  constant   Section 3, baseline 1: draft exactly gamma tokens
  heuristic  Section 3, baseline 2: like constant, but after each verification gamma grows by 2 if
             every draft token was accepted and shrinks by 1 otherwise
gamma is kept within [1, K_cap]; the paper caps the draft length at 40 for both the heuristic and SVIP.
"""
ENTROPY, CONSTANT, HEURISTIC = 0, 1, 2


def advance(policy, stop, gamma, draft_len, active, K_cap):
    """After one draft step.  Lists are updated in place; returns the number still drafting."""
    n = 0
    for i in range(len(active)):
        if not active[i]:
            continue
        draft_len[i] += 1
        if policy == ENTROPY:
            done = bool(stop[i]) or draft_len[i] >= K_cap
        else:
            done = draft_len[i] >= min(gamma[i], K_cap)
        if done:
            active[i] = 0
        else:
            n += 1
    return n


def update(policy, n_accepted, draft_len, gamma, active, K_cap):
    """After one verification round: adapt gamma (heuristic only) and re-arm every sequence."""
    for i in range(len(active)):
        if policy == HEURISTIC:
            if n_accepted[i] == draft_len[i]:
                gamma[i] = min(gamma[i] + 2, K_cap)
            else:
                gamma[i] = max(gamma[i] - 1, 1)
        draft_len[i] = 0
        active[i] = 1
