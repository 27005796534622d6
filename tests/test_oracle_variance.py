"""Pins of the variance diagnostics in oracle/variance.py (Appendix D): each function is checked against something
other than itself — brute force over every keep pattern, numpy's population variance, the law of total variance,
the two values Appendix D.3 prints, and a Monte-Carlo run through the oracle's own pruning draws."""
import os

import numpy as np
import pytest

import oracle
from oracle import variance as V

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _case(P, G, seed, r_q, r_o, frac_q=0.5):
    rng = np.random.default_rng(seed)
    psi = rng.normal(size=(P, G))
    cand_q = np.zeros(P, dtype=np.uint8); cand_q[:int(P * frac_q)] = 1
    cand_o = (rng.random((P, G)) < 0.6).astype(np.uint8)
    Pq, Po = V.pruning_probabilities(cand_q, cand_o, r_q, r_o)
    return psi, cand_q, cand_o, Pq, Po


def test_estimator_variance_closed_form_equals_brute_force():
    # every keep pattern of 2 prompts x 2 completions (64 patterns) and of 3 x 2 (512), weighted by its probability
    for P, G, seed in ((2, 2, 0), (3, 2, 1), (2, 3, 2)):
        psi, _, _, Pq, Po = _case(P, G, seed, 0.4, 0.7)
        Pq[0] = 0.4; Po[0, 0] = 0.7                              # at least one candidate of each kind
        mean, var = V.estimator_moments_by_enumeration(psi, Pq, Po)
        assert abs(mean - psi.mean()) <= 1e-12                   # unbiased: the full-batch mean
        assert abs(var - V.estimator_variance(psi, Pq, Po)) <= 1e-12 * max(var, 1.0)
    # nothing pruned: no variance at all
    psi = np.arange(6.0).reshape(2, 3)
    assert V.estimator_variance(psi, np.zeros(2), np.zeros((2, 3))) == 0.0


def test_estimator_variance_matches_the_oracles_own_draws():
    # Monte Carlo through draw_uniforms -> prune_masks -> rescale (the path the masks take), 4000 steps
    P, G, r_q, r_o = 4, 4, 0.5, 0.5
    rng = np.random.default_rng(3)
    rewards = (rng.random((P, G)) < np.array([0.2, 0.5, 0.7, 0.4])[:, None]).astype(np.float32)
    adv, mabs = oracle.group_advantages(rewards)
    H_prev = np.array([0.9, 0.1, 0.5, 0.3], dtype=np.float32)
    psi = rng.normal(size=(P, G))
    cand_o = oracle.completion_candidates(adv); cand_q = oracle.prompt_candidates(H_prev, P)
    Pq, Po = V.pruning_probabilities(cand_q, cand_o, r_q, r_o)
    vals = []
    for step in range(4000):
        out = oracle.prune_and_rescale(adv, mabs, H_prev, r_q, r_o, seed=11, step=step)
        vals.append(float(np.sum(out["w_seq"].astype(np.float64) * psi)))
    mc = V.monte_carlo_summary(vals)
    exact = V.estimator_variance(psi, Pq, Po)
    assert abs(mc["mean"] - psi.mean()) <= 5 * mc["se_mean"]
    assert abs(mc["var"] - exact) <= 5 * mc["se_var"], (mc, exact)


def test_single_sample_variance_against_definitions():
    psi, _, _, Pq, Po = _case(6, 5, 4, 0.5, 0.7)
    out = V.single_sample_variance(psi, Pq, Po)
    assert abs(out["mean"] - psi.mean()) <= 1e-12                            # Eq. 13: unbiased under both prunings
    assert abs(out["total"] - (out["term_I"] + out["term_II"])) <= 1e-12     # law of total variance
    for k in range(6):                                                       # the printed completion-level formula
        assert abs(out["comp_var"][k] - V.completion_variance_formula(psi[k], Po[k])) <= 1e-12
    # no pruning: the plain population variances
    none = V.single_sample_variance(psi, np.zeros(6), np.zeros((6, 5)))
    assert abs(none["total"] - np.var(psi)) <= 1e-12
    assert abs(none["term_I"] - np.var(psi.mean(axis=1))) <= 1e-12
    assert abs(none["var_Q"] - np.var(psi.mean(axis=1))) <= 1e-12
    assert abs(none["mean_var_O"] - np.mean(np.var(psi, axis=1))) <= 1e-12
    assert abs(none["gamma_q_second_moment"] - 1.0) <= 1e-15
    # a sampled check of the definition: draw (q, o) from the pruned distributions and average
    rng = np.random.default_rng(0)
    P, G = psi.shape
    p_q = (1 - Pq) / (1 - Pq).sum(); C_q = (1 - Pq).mean()
    n = 200000
    qs = rng.choice(P, size=n, p=p_q)
    vals = np.empty(n)
    for k in range(P):
        idx = np.nonzero(qs == k)[0]
        p_o = (1 - Po[k]) / (1 - Po[k]).sum(); C_o = (1 - Po[k]).mean()
        os_ = rng.choice(G, size=len(idx), p=p_o)
        vals[idx] = (C_q / (1 - Pq[k])) * (C_o / (1 - Po[k, os_])) * psi[k, os_]
    assert abs(vals.mean() - out["mean"]) <= 5 * vals.std() / np.sqrt(n)
    assert abs(vals.var() - out["total"]) <= 0.03 * out["total"]


def test_gamma_q_second_moment_is_the_printed_factor():
    # Appendix D.3: a fraction b of the prompts pruned with probability r; and the two values the paper prints
    for b, r in ((0.5, 0.5), (0.5, 0.7), (0.5, 0.9), (0.25, 0.6)):
        P = 40
        Pq = np.zeros(P); Pq[:int(b * P)] = r
        out = V.single_sample_variance(np.ones((P, 2)), Pq, np.zeros((P, 2)))
        assert abs(out["gamma_q_second_moment"] - V.gamma_q_factor(b, r)) <= 1e-12
    printed = {}
    for line in open(os.path.join(GOLDEN, "variance_factor.txt")):
        if line.strip() and not line.startswith("#"):
            _, r, val = line.split()[:3]                                         # columns: b r printed relation
            printed[float(r)] = float(val)
    assert abs(V.gamma_q_factor(0.5, 0.7) - printed[0.7]) <= 0.012 and V.gamma_q_factor(0.5, 0.7) <= 1.42
    assert abs(V.gamma_q_factor(0.5, 0.9) - printed[0.9]) <= 1e-9


def test_theorem_bound_holds_when_low_score_items_have_small_terms():
    # the theorem's conditions: candidates (the pruned-with-probability-r items) carry the smaller terms
    rng = np.random.default_rng(8)
    P, G, r = 8, 6, 0.5
    psi = rng.normal(size=(P, G))
    cand_o = np.zeros((P, G), dtype=np.uint8); cand_q = np.zeros(P, dtype=np.uint8)
    for k in range(P):
        small = np.argsort(np.abs(psi[k]))[:G // 2]
        cand_o[k, small] = 1
        psi[k, small] *= 0.3
    order = np.argsort(np.abs(psi.mean(axis=1)))
    cand_q[order[:P // 2]] = 1
    psi[order[:P // 2]] *= 0.3
    Pq, Po = V.pruning_probabilities(cand_q, cand_o, r, r)
    out = V.single_sample_variance(psi, Pq, Po)
    assert out["total"] <= out["bound"] * (1 + 1e-12)
    assert all(out["comp_var"][k] <= np.var(psi[k]) * (1 + 1e-12) for k in range(P))   # completion level: no increase
    assert out["term_I"] <= out["var_Q"] * (1 + 1e-12)                                   # prompt level: no increase
    # and the reverse rule (large terms are the candidates) breaks the completion-level statement
    Pq_r, Po_r = V.pruning_probabilities(1 - cand_q, 1 - cand_o, r, r)
    rev = V.single_sample_variance(psi, Pq_r, Po_r)
    assert any(rev["comp_var"][k] > np.var(psi[k]) for k in range(P))
