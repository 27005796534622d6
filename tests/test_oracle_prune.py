"""Pins for the oracle's advantages, candidate sets, masks and rescaling factors.

Each test checks the oracle against something the paper or the mathematics fixes
(closed forms, brute force, exact enumeration, a published known-answer vector),
never against the oracle's own formula.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.stats

import oracle
from oracle import philox

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- generator
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert oracle.philox4x32_10(v[0:4], v[4:6]) == tuple(v[6:10])


def test_uniform53_range_and_layout():
    out = oracle.philox4x32_10((7, philox.DOMAIN_COMPLETION, 5, 0), (0x1234, 0))
    x = out[0] | (out[1] << 32)
    u = oracle.uniform53(0x1234, 5, philox.DOMAIN_COMPLETION, 7)
    assert u == (x >> 11) / 2.0 ** 53 and 0.0 <= u < 1.0
    # different domains / steps / seeds give different draws
    base = oracle.uniform53(1, 0, 1, 0)
    assert len({base, oracle.uniform53(1, 0, 2, 0), oracle.uniform53(1, 1, 1, 0),
                oracle.uniform53(2, 0, 1, 0), oracle.uniform53(1 << 32, 0, 1, 0),
                oracle.uniform53(1, 1 << 32, 1, 0)}) == 6


def test_uniform53_frequency():
    n = 60000
    us = np.array([oracle.uniform53(99, 3, 2, i) for i in range(n)])
    for r in (0.25, 0.5, 0.9):
        p_hat = (us < r).mean()
        assert abs(p_hat - r) < 4 * math.sqrt(r * (1 - r) / n)
    assert abs(us.mean() - 0.5) < 4 / math.sqrt(12 * n)


# ---------------------------------------------------------------- advantages (Eq. 2, Eq. 14)
def test_advantages_zero_mean_unit_std():
    rng = np.random.default_rng(0)
    r = rng.normal(size=(16, 8)).astype(np.float32)
    adv, mabs = oracle.group_advantages(r, ddof=0, std_eps=0.0)
    assert np.abs(adv.astype(np.float64).sum(axis=1)).max() < 1e-6
    assert np.allclose((adv.astype(np.float64) ** 2).mean(axis=1), 1.0, atol=1e-6)
    assert np.allclose(mabs, np.abs(adv.astype(np.float64)).mean(axis=1), atol=1e-6)


def test_advantages_match_library_zscore():
    rng = np.random.default_rng(1)
    r = rng.random((10, 5)).astype(np.float32)
    for ddof in (0, 1):
        adv, _ = oracle.group_advantages(r, ddof=ddof, std_eps=0.0)
        ref = scipy.stats.zscore(r.astype(np.float64), axis=1, ddof=ddof)
        assert np.allclose(adv, ref, rtol=0, atol=1e-6)


def test_advantages_all_equal_rewards_are_zero():
    r = np.array([[1, 1, 1, 1], [0, 0, 0, 0], [0.3, 0.3, 0.3, 0.3]], dtype=np.float32)
    adv, mabs = oracle.group_advantages(r)
    assert (adv == 0).all() and (mabs == 0).all()


@pytest.mark.parametrize("G", [2, 4, 5, 8, 16])
def test_advantages_binary_closed_form(G):
    # k successes of G, p = k/G, population std:  A_succ = sqrt((1-p)/p), A_fail = -sqrt(p/(1-p)),
    # mean|A| = 2 sqrt(p(1-p))
    for k in range(1, G):
        r = np.zeros((1, G), dtype=np.float32)
        r[0, :k] = 1
        adv, mabs = oracle.group_advantages(r, ddof=0, std_eps=0.0)
        p = k / G
        assert np.allclose(adv[0, :k], math.sqrt((1 - p) / p), rtol=1e-6)
        assert np.allclose(adv[0, k:], -math.sqrt(p / (1 - p)), rtol=1e-6)
        assert math.isclose(float(mabs[0]), 2 * math.sqrt(p * (1 - p)), rel_tol=1e-6)
        # the default guard 1e-6 only rescales by sigma/(sigma+1e-6)
        adv2, _ = oracle.group_advantages(r)
        sigma = math.sqrt(p * (1 - p))
        assert np.allclose(adv2, adv * (sigma / (sigma + 1e-6)), rtol=1e-6)


# ---------------------------------------------------------------- candidates (Eq. 15, Eq. 17)
@pytest.mark.parametrize("G", [2, 3, 4, 5, 8])
def test_completion_candidates_are_majority_class(G):
    # binary rewards: |A| <= mean|A| holds exactly for the majority outcome (everyone on a tie or
    # when all rewards are equal)
    for bits in itertools.product([0, 1], repeat=G):
        r = np.array([bits], dtype=np.float32)
        adv, _ = oracle.group_advantages(r)
        cand = oracle.completion_candidates(adv)[0]
        k = sum(bits)
        for i, b in enumerate(bits):
            if k == 0 or k == G or 2 * k == G:
                want = 1
            else:
                want = int((b == 1) == (2 * k > G))
            assert cand[i] == want, (bits, i)
        rev = oracle.completion_candidates(adv, reverse=True)[0]
        assert (rev == 1 - cand).all()


def test_completion_candidates_continuous_rewards():
    rng = np.random.default_rng(3)
    r = rng.normal(size=(50, 6)).astype(np.float32)
    adv, mabs = oracle.group_advantages(r)
    cand = oracle.completion_candidates(adv)
    a = np.abs(adv.astype(np.float64))
    gap = np.abs(a - a.mean(axis=1, keepdims=True))
    clear = gap > 1e-6
    assert ((a <= a.mean(axis=1, keepdims=True)) == cand.astype(bool))[clear].all()
    # at least one candidate and (unless all equal) at least one non-candidate per group
    assert (cand.sum(axis=1) >= 1).all() and (cand.sum(axis=1) < 6).all()


def test_prompt_candidates_rank_count():
    rng = np.random.default_rng(4)
    for P in (1, 2, 5, 8, 33):
        H = np.round(rng.random(P), 1).astype(np.float32)    # many ties
        cand = oracle.prompt_candidates(H, P)
        assert cand.sum() == P // 2
        for k in range(P):     # rank = #(strictly lower) + #(equal with lower index)
            rank = sum(1 for j in range(P) if H[j] < H[k] or (H[j] == H[k] and j < k))
            assert cand[k] == int(rank < P // 2)
        rev = oracle.prompt_candidates(H, P, reverse=True)
        for k in range(P):
            rank = sum(1 for j in range(P) if H[j] > H[k] or (H[j] == H[k] and j < k))
            assert rev[k] == int(rank < P // 2)
    assert oracle.prompt_candidates(None, 7).sum() == 0


# ---------------------------------------------------------------- masks (Eq. 15, Eq. 17)
def _fixed_case(P=3, G=4, seed=5):
    rng = np.random.default_rng(seed)
    r = (rng.random((P, G)) < 0.5).astype(np.float32)
    r[0] = [1, 0, 0, 0][:G] if G >= 4 else r[0]
    adv, mabs = oracle.group_advantages(r)
    H = rng.random(P).astype(np.float32)
    return adv, mabs, H


def test_no_pruning_recovers_grpo():
    adv, mabs, H = _fixed_case()
    out = oracle.prune_and_rescale(adv, mabs, H, 0.0, 0.0, seed=1, step=2)
    assert out["keep_q"].all() and out["keep_o"].all()
    assert (out["gamma_q"] == 1).all() and (out["gamma_o"] == 1).all()
    assert np.allclose(out["w_seq"], 1.0 / adv.size)


def test_masks_follow_explicit_uniforms():
    adv, mabs, H = _fixed_case(P=4, G=4, seed=8)
    P, G = adv.shape
    cand_o = oracle.completion_candidates(adv)
    cand_q = oracle.prompt_candidates(H, P)
    u_q = np.full(P, 0.1); u_o = np.full((P, G), 0.1)        # every candidate is pruned at r = 0.5
    out = oracle.prune_and_rescale(adv, mabs, H, 0.5, 0.5, u_q=u_q, u_o=u_o)
    assert (out["keep_q"] == 1 - cand_q).all()
    for k in range(P):
        want = (1 - cand_o[k]) * out["keep_q"][k]
        assert (out["keep_o"][k] == want).all()
        assert out["n_keep_o"][k] == want.sum()
    assert out["n_keep_q"] == P - P // 2
    u_q[:] = 0.5; u_o[:] = 0.5                               # u == r is NOT pruned (u < r prunes)
    out = oracle.prune_and_rescale(adv, mabs, H, 0.5, 0.5, u_q=u_q, u_o=u_o)
    assert out["keep_q"].all() and out["keep_o"].all()
    # non-candidates survive any draw
    u_q[:] = 0.0; u_o[:] = 0.0
    out = oracle.prune_and_rescale(adv, mabs, H, 0.99, 0.99, u_q=u_q, u_o=u_o)
    assert (out["keep_q"][cand_q == 0] == 1).all()
    kept_rows = out["keep_q"] == 1
    assert (out["keep_o"][kept_rows][cand_o[kept_rows] == 0] == 1).all()
    # first epoch: no history, no prompt pruning
    out = oracle.prune_and_rescale(adv, mabs, None, 0.99, 0.0, u_q=u_q, u_o=u_o)
    assert out["keep_q"].all() and out["cand_q"].sum() == 0


def test_rescaling_factors_and_counts():
    # Eq. 18 with the counts as counted
    adv, mabs, H = _fixed_case(P=4, G=4, seed=11)
    P, G = adv.shape
    r_q, r_o = 0.3, 0.6
    out = oracle.prune_and_rescale(adv, mabs, H, r_q, r_o, seed=3, step=9)
    nq = int(out["keep_q"].sum())
    assert out["n_keep_q"] == nq
    for k in range(P):
        no = int(out["keep_o"][k].sum())
        assert out["n_keep_o"][k] == no
        if out["keep_q"][k]:
            Pq = r_q if out["cand_q"][k] else 0.0
            assert math.isclose(out["gamma_q"][k], (nq / P) / (1 - Pq), rel_tol=1e-6)
        else:
            assert out["gamma_q"][k] == 0 and no == 0
        for i in range(G):
            if out["keep_o"][k, i]:
                Po = r_o if out["cand_o"][k, i] else 0.0
                assert math.isclose(out["gamma_o"][k, i], (no / G) / (1 - Po), rel_tol=1e-6)
                # the sequence weight is gamma_q gamma_o / (|S^q| |S^o|)
                assert math.isclose(out["w_seq"][k, i],
                                    out["gamma_q"][k] * out["gamma_o"][k, i] / (nq * no), rel_tol=1e-6)
            else:
                assert out["gamma_o"][k, i] == 0 and out["w_seq"][k, i] == 0


def test_history_carry_forward():
    adv, mabs, H = _fixed_case(P=4, G=4, seed=12)
    u_q = np.zeros(4); u_o = np.ones((4, 4)) * 0.99
    out = oracle.prune_and_rescale(adv, mabs, H, 0.5, 0.5, u_q=u_q, u_o=u_o)
    for k in range(4):
        assert out["H_next"][k] == (mabs[k] if out["keep_q"][k] else H[k])
    assert (out["keep_q"] == 0).sum() == 2
    out = oracle.prune_and_rescale(adv, mabs, None, 0.5, 0.5, u_q=u_q, u_o=u_o)
    assert (out["H_next"] == mabs).all()


# ---------------------------------------------------------------- unbiasedness (Eq. 9, 12, 13)
def _enumerate_expectation(adv, mabs, H, r_q, r_o, ell, weight_fn):
    """sum over all keep/drop patterns of Pr[pattern] * estimator(pattern)."""
    P, G = adv.shape
    cand_o = oracle.completion_candidates(adv)
    cand_q = oracle.prompt_candidates(H, P)
    cq = [k for k in range(P) if cand_q[k]]
    co = [(k, i) for k in range(P) for i in range(G) if cand_o[k, i]]
    total, prob_total = 0.0, 0.0
    for pat_q in itertools.product([0, 1], repeat=len(cq)):
        for pat_o in itertools.product([0, 1], repeat=len(co)):
            u_q = np.full(P, 0.999); u_o = np.full((P, G), 0.999)
            pr = 1.0
            for k, drop in zip(cq, pat_q):
                u_q[k] = 0.0 if drop else 0.999
                pr *= r_q if drop else (1 - r_q)
            for (k, i), drop in zip(co, pat_o):
                u_o[k, i] = 0.0 if drop else 0.999
                pr *= r_o if drop else (1 - r_o)
            out = oracle.prune_and_rescale(adv, mabs, H, r_q, r_o, u_q=u_q, u_o=u_o)
            total += pr * weight_fn(out, ell)
            prob_total += pr
    assert math.isclose(prob_total, 1.0, rel_tol=1e-12)
    return total


@pytest.mark.parametrize("P,G,r_q,r_o", [(2, 3, 0.5, 0.5), (2, 4, 0.3, 0.7), (3, 3, 0.9, 0.25),
                                         (2, 4, 0.0, 0.5), (3, 2, 0.5, 0.0)])
def test_rescaled_estimator_is_unbiased_by_enumeration(P, G, r_q, r_o):
    rng = np.random.default_rng(100 + P * 10 + G)
    r = (rng.random((P, G)) < 0.4).astype(np.float32)
    r[0, 0] = 1.0; r[0, 1:] = 0.0                # a group with a clear minority
    adv, mabs = oracle.group_advantages(r)
    H = rng.random(P).astype(np.float32)
    ell = rng.normal(size=(P, G))                # arbitrary per-completion terms (loss or gradient entry)
    full = ell.mean()                            # (1/P) sum_k (1/G) sum_i ell

    est = _enumerate_expectation(adv, mabs, H, r_q, r_o, ell,
                                 lambda out, ell: float((out["w_seq"].astype(np.float64) * ell).sum()))
    assert math.isclose(est, full, rel_tol=0, abs_tol=2e-7)

    # the same through Eq. 18's factors: mean over retained prompts of gamma_q * mean over retained
    # completions of gamma_o * ell
    def via_gammas(out, ell):
        nq = out["n_keep_q"]
        acc = 0.0
        for k in range(P):
            if out["keep_q"][k] and out["n_keep_o"][k] > 0:
                inner = sum(float(out["gamma_o"][k, i]) * ell[k, i]
                            for i in range(G) if out["keep_o"][k, i]) / out["n_keep_o"][k]
                acc += float(out["gamma_q"][k]) * inner
        return acc / nq if nq else 0.0
    est2 = _enumerate_expectation(adv, mabs, H, r_q, r_o, ell, via_gammas)
    assert math.isclose(est2, full, rel_tol=0, abs_tol=2e-7)


def test_other_normalisation_would_be_biased():
    # dividing the retained sum by the ORIGINAL group size while also applying Eq. 18's |S|/|O|
    # factor double-counts the shrinkage: the enumeration exposes it
    P, G, r_q, r_o = 2, 4, 0.0, 0.5
    r = np.array([[1, 0, 0, 0], [1, 1, 0, 1]], dtype=np.float32)
    adv, mabs = oracle.group_advantages(r)
    H = np.array([0.2, 0.9], dtype=np.float32)
    ell = np.array([[1.0, 2.0, 3.0, 4.0], [0.5, 0.25, 2.0, 1.0]])

    def biased(out, ell):
        return sum(float(out["gamma_q"][k]) * float(out["gamma_o"][k, i]) * ell[k, i]
                   for k in range(P) for i in range(G) if out["keep_o"][k, i]) / (P * G)
    est = _enumerate_expectation(adv, mabs, H, r_q, r_o, ell, biased)
    assert abs(est - ell.mean()) > 0.05


def test_rescaled_estimator_is_unbiased_by_monte_carlo():
    P, G, r_q, r_o = 2, 4, 0.5, 0.5
    r = np.array([[1, 0, 0, 0], [1, 1, 0, 1]], dtype=np.float32)
    adv, mabs = oracle.group_advantages(r)
    H = np.array([0.2, 0.9], dtype=np.float32)
    ell = np.array([[1.0, -2.0, 3.0, 0.5], [0.5, 0.25, -2.0, 1.0]])
    n = 6000
    vals = np.empty(n)
    for s in range(n):
        out = oracle.prune_and_rescale(adv, mabs, H, r_q, r_o, seed=s, step=7)
        vals[s] = (out["w_seq"].astype(np.float64) * ell).sum()
    se = vals.std(ddof=1) / math.sqrt(n)
    assert se > 0 and abs(vals.mean() - ell.mean()) < 4 * se
    # retention frequency of a candidate completion through the real generator
    cand = oracle.completion_candidates(adv)
    keeps = np.array([oracle.prune_and_rescale(adv, mabs, None, 0.0, 0.25, seed=s, step=1)["keep_o"]
                      for s in range(3000)])
    freq = keeps.mean(axis=0)
    assert (freq[cand == 0] == 1).all()
    assert np.abs(freq[cand == 1] - 0.75).max() < 4 * math.sqrt(0.75 * 0.25 / 3000)


def test_variance_factor_matches_printed_values():
    # Theorem D.1: E_{q~P~}[gamma(q)^2] = (1-b r)(1-(1-b) r)/(1-r); realised with a mask whose retained
    # count equals its expectation so that C_q = 1 - b r exactly
    rows = [l.split() for l in open(os.path.join(GOLDEN, "variance_factor.txt"))
            if l.strip() and not l.startswith("#")]
    for b, r, printed, rel in rows:
        b, r, printed = float(b), float(r), float(printed)
        P = 20
        n_cand = int(b * P)
        n_keep_c = round(n_cand * (1 - r))
        H = np.arange(P, dtype=np.float32)           # prompts 0..n_cand-1 are the candidates
        u_q = np.full(P, 0.999); u_q[n_keep_c:n_cand] = 0.0
        adv = np.zeros((P, 2), dtype=np.float32); mabs = np.zeros(P, dtype=np.float32)
        out = oracle.prune_and_rescale(adv, mabs, H, r, 0.0, u_q=u_q, u_o=np.ones((P, 2)))
        assert out["cand_q"][:n_cand].all() and out["n_keep_q"] == P - n_cand + n_keep_c
        kept = out["gamma_q"][out["keep_q"] == 1].astype(np.float64)
        factor = (kept ** 2).mean()                  # q ~ P~ is uniform over the retained prompts
        closed = (1 - b * r) * (1 - (1 - b) * r) / (1 - r)
        assert math.isclose(factor, closed, rel_tol=1e-6)
        if rel == "le":
            assert factor <= printed and printed - factor < 0.02
        else:
            assert math.isclose(factor, printed, rel_tol=1e-3)


# ---------------------------------------------------------------- fixed-fraction mode (Appendix A, Algorithm 1)
def test_fixed_fraction_counts_and_choice():
    adv, mabs, H = _fixed_case(P=6, G=4, seed=21)
    P, G = adv.shape
    rng = np.random.default_rng(1)
    u_q = rng.random(P); u_o = rng.random((P, G))
    for r_q, r_o in [(0.5, 0.5), (0.4, 0.7), (0.0, 0.99), (0.99, 0.0)]:
        out = oracle.prune_and_rescale(adv, mabs, H, r_q, r_o, u_q=u_q, u_o=u_o, mode=1)
        B = [k for k in range(P) if out["cand_q"][k]]
        m_q = math.floor(r_q * len(B))
        pruned_q = [k for k in B if not out["keep_q"][k]]
        assert len(pruned_q) == m_q                                  # floor(r_q |B|) prompts go
        assert sorted(pruned_q) == sorted(sorted(B, key=lambda k: (u_q[k], k))[:m_q])   # the smallest draws
        assert all(out["keep_q"][k] for k in range(P) if k not in B)
        for k in range(P):
            C = [i for i in range(G) if out["cand_o"][k, i]]
            m_o = math.floor(r_o * len(C))
            if out["keep_q"][k]:
                pruned_o = [i for i in C if not out["keep_o"][k, i]]
                assert len(pruned_o) == m_o
                assert sorted(pruned_o) == sorted(sorted(C, key=lambda i: (u_o[k, i], i))[:m_o])
                # weights use the realised fraction as the pruning probability
                for i in range(G):
                    if out["keep_o"][k, i]:
                        Pq = (m_q / len(B)) if k in B else 0.0
                        Po = (m_o / len(C)) if i in C else 0.0
                        assert math.isclose(out["w_seq"][k, i], 1 / (P * G * (1 - Pq) * (1 - Po)), rel_tol=1e-6)
            else:
                assert out["keep_o"][k].sum() == 0


def test_fixed_fraction_is_unbiased_with_realised_fraction_only():
    # enumerate every equally likely choice of the pruned subsets
    P, G, r_q, r_o = 4, 4, 0.5, 0.5
    r = np.array([[1, 0, 0, 0], [1, 1, 0, 1], [0, 1, 0, 0], [1, 0, 1, 0]], dtype=np.float32)   # |C| = 3, 3, 3, 4
    adv, mabs = oracle.group_advantages(r)
    H = np.array([0.1, 0.9, 0.2, 0.8], dtype=np.float32)
    ell = np.random.default_rng(3).normal(size=(P, G))
    cand_o = oracle.completion_candidates(adv); cand_q = oracle.prompt_candidates(H, P)
    B = [k for k in range(P) if cand_q[k]]
    Cs = [[i for i in range(G) if cand_o[k, i]] for k in range(P)]
    m_q = math.floor(r_q * len(B)); m_os = [math.floor(r_o * len(C)) for C in Cs]
    assert any(r_o * len(C) != m for C, m in zip(Cs, m_os))          # a case where floor() bites
    choices = [list(itertools.combinations(B, m_q))] + [list(itertools.combinations(C, m)) for C, m in zip(Cs, m_os)]
    total, total_eq18, n = 0.0, 0.0, 0
    for pick in itertools.product(*choices):
        u_q = np.full(P, 0.9); u_o = np.full((P, G), 0.9)
        for k in pick[0]:
            u_q[k] = 0.1
        for k in range(P):
            for i in pick[1 + k]:
                u_o[k, i] = 0.1
        out = oracle.prune_and_rescale(adv, mabs, H, r_q, r_o, u_q=u_q, u_o=u_o, mode=1)
        total += float((out["w_seq"].astype(np.float64) * ell).sum())
        # Eq. 18 taken literally (P = r) on the same masks
        lit = 0.0
        for k in range(P):
            for i in range(G):
                if out["keep_o"][k, i]:
                    lit += ell[k, i] / (P * G * (1 - (r_q if cand_q[k] else 0)) * (1 - (r_o if cand_o[k, i] else 0)))
        total_eq18 += lit
        n += 1
    assert math.isclose(total / n, ell.mean(), abs_tol=2e-7)
    assert abs(total_eq18 / n - ell.mean()) > 1e-3                   # the printed factors are biased here


# ---------------------------------------------------------------- history table across epochs (Eq. 16, Algorithm 1)
def test_history_epochs_carry_forward_and_first_epoch():
    N, G, P = 12, 4, 4
    rng = np.random.default_rng(0)
    rate = rng.random(N)
    rewards = [(rng.random((N, G)) < rate[:, None]).astype(np.float32) for _ in range(4)]
    batches = [[list(range(i, i + P)) for i in range(0, N, P)] for _ in range(4)]
    batches[2] = [[0, 5, 10, 3], [1, 6, 11, 4], [2, 7, 8, 9]]            # another batching in the third epoch
    table, log = oracle.history_epochs(rewards, batches, N, G, 0.6, 0.5, seed=9)
    assert all(out["keep_q"].all() for out in log[:3])                     # first epoch: no prompt pruning
    assert any((out["keep_q"] == 0).any() for out in log[3:])              # later epochs prune some prompts
    # replay by hand: a prompt's score changes exactly when it was retained, to that epoch's mean |A|
    H = np.zeros(N, dtype=np.float32)
    i = 0
    for t in range(4):
        for ids in batches[t]:
            out = log[i]; i += 1
            mabs = oracle.group_advantages(rewards[t][ids])[1]
            if t > 0:                                                      # candidates = lowest half of the scores read
                order = sorted(range(P), key=lambda k: (H[ids[k]], k))
                assert sorted(np.nonzero(out["cand_q"])[0]) == sorted(order[:P // 2])
            for k, q in enumerate(ids):
                if out["keep_q"][k]:
                    H[q] = mabs[k]
    assert np.array_equal(H, table)
