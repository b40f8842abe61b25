"""Pins of the oracle's adaptive tier rule (tiers by rank of the spatial score among the tokens of a frame that are not
reused, in fixed shares).  Pinned by the exact quotas, by the fixed-threshold rule it must reduce to when Eq. 8's
thresholds are put between the right order statistics, by a quadratic rank count in numpy, by tie handling and by the
invariance under a shift of all scores (the point of adapting the thresholds)."""
import numpy as np
import pytest

import oracle

P = oracle.Params(tau_t=0.5, theta_R=0.9, patch_reuse=1)
SHARES = (317, 71, 214)       # per mille of the stored-or-pruned tokens


def _quotas(n_live, shares):
    left, out = n_live, []
    for pm in shares:
        q = min((n_live * pm + 500) // 1000, left)
        out.append(q)
        left -= q
    return out


@pytest.mark.parametrize("has_prev", [False, True])
def test_quotas_are_exact_and_the_rule_reduces_to_fixed_thresholds(has_prev):
    rng = np.random.default_rng(1 + has_prev)
    n = 576
    s = rng.permutation(np.linspace(0.05, 0.95, n)).astype(np.float32)       # distinct scores
    dP = rng.uniform(0.0, 1.0, n).astype(np.float32)
    dec, idx, counts, red = oracle.select_ranked(dP, s, has_prev, SHARES, P)
    live = np.ones(n, bool) if not has_prev else dP >= np.float32(P.tau_t)
    q16, q8, q4 = _quotas(int(live.sum()), SHARES)
    assert counts.tolist() == [n - int(live.sum()), int(live.sum()) - q16 - q8 - q4, q4, q8, q16] and red == 0
    # the same decisions from Eq. 8 with thresholds between the order statistics of the live scores
    order = np.sort(s[live])[::-1].astype(np.float64)
    mid = lambda k: float((order[k - 1] + order[k]) / 2)
    import dataclasses
    p_fixed = dataclasses.replace(P, tau_high=mid(q16), tau_med=mid(q16 + q8), tau_low=mid(q16 + q8 + q4))
    d2, i2, c2, r2, _ = oracle.select(dP, s, has_prev, p_fixed)
    assert np.array_equal(dec, d2) and np.array_equal(idx, i2) and np.array_equal(counts, c2)
    # the lists are ascending token ids, padded with -1
    for row, code in zip(idx, (oracle.FP16, oracle.INT8, oracle.INT4)):
        want = np.flatnonzero(dec == code)
        assert np.array_equal(row[:len(want)], want) and (row[len(want):] == -1).all()


def test_rank_count_in_numpy_with_ties_and_a_redundant_frame():
    rng = np.random.default_rng(3)
    n = 200
    s = rng.integers(0, 12, n).astype(np.float32) / 16        # many ties
    dP = rng.uniform(0.0, 1.0, n).astype(np.float32)
    for patch_reuse in (0, 1):
        import dataclasses
        p = dataclasses.replace(P, patch_reuse=patch_reuse)
        dec, idx, counts, red = oracle.select_ranked(dP, s, True, (250, 250, 250), p)
        live = dP >= np.float32(p.tau_t) if patch_reuse else np.ones(n, bool)
        ids = np.flatnonzero(live)
        rank = np.array([np.sum((s[ids] > s[i]) | ((s[ids] == s[i]) & (ids < i))) for i in ids])
        q16, q8, q4 = _quotas(len(ids), (250, 250, 250))
        want = np.zeros(n, np.uint8)
        want[ids] = np.where(rank < q16, 4, np.where(rank < q16 + q8, 3, np.where(rank < q16 + q8 + q4, 2, 1)))
        assert np.array_equal(dec, want) and red == 0
    # more than theta_R of the patches static: every token reused, nothing ranked
    dec, idx, counts, red = oracle.select_ranked(np.zeros(n, np.float32), s, True, (250, 250, 250), P)
    assert red == 1 and (dec == oracle.REUSE).all() and (idx == -1).all() and counts.tolist() == [n, 0, 0, 0, 0]


def test_decisions_follow_the_ranks_not_the_level_of_the_scores():
    """A frame that is dim everywhere (all scores low) keeps the same shares as a frame with high scores: adding a
    constant to every score, or compressing their range, changes nothing; the fixed thresholds prune it wholly."""
    rng = np.random.default_rng(5)
    n = 576
    s = rng.uniform(0.0, 0.2, n).astype(np.float32)
    base = oracle.select_ranked(None, s, False, SHARES, P)
    for t in (s + np.float32(0.5), s * np.float32(0.25), np.sqrt(s)):     # strictly increasing maps keep the ranks
        if len(np.unique(t)) < len(np.unique(s)):
            continue
        other = oracle.select_ranked(None, t.astype(np.float32), False, SHARES, P)
        assert all(np.array_equal(a, b) for a, b in zip(base[:3], other[:3]))
    fixed, *_ = oracle.select(None, s, False, P)
    assert (fixed == oracle.PRUNE).all() and (base[0] != oracle.PRUNE).mean() > 0.55


def test_shares_are_clipped_to_the_tokens_there_are():
    s = np.linspace(0, 1, 10).astype(np.float32)
    dec, idx, counts, red = oracle.select_ranked(None, s, False, (700, 700, 700), P)
    assert counts.tolist() == [0, 0, 0, 3, 7]                  # 7 FP16, then only 3 left for INT8
    dec, idx, counts, red = oracle.select_ranked(None, s, False, (0, 0, 0), P)
    assert (dec == oracle.PRUNE).all()
    dec, idx, counts, red = oracle.select_ranked(None, s, False, (50, 0, 1000), P)
    assert counts.tolist() == [0, 0, 9, 0, 1] and dec[9] == oracle.FP16      # (10 * 50 + 500) / 1000 = 1
