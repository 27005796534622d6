"""Variance of the rescaled estimator (Appendix D), written out from the definitions.

TEST INFRASTRUCTURE ONLY — see the package docstring.

Two different quantities carry the name "variance" here and both are computed exactly:

1. Appendix D's: the variance of G_hat = gamma(q) gamma(o,q) Psi(q,o) for ONE draw q ~ P~, o ~ pi~(.|q) from the
   pruned distributions of Eq. 10 and Eq. 6, with the batch as the population (every prompt, and every completion
   of a prompt, equally likely before pruning).  `single_sample_variance` evaluates the expectations as plain sums
   over all (q, o), together with the law-of-total-variance split (Term I, Term II), the second moment of gamma(q)
   (whose closed form under "a fraction b of the prompts pruned with probability r" Appendix D.3 prints), the
   completion-level formula and Theorem D.1's bound.
2. What a training step sees: the variance, over the pruning draws, of the batch estimator sum_{k,i} w_seq[k,i]
   psi[k,i] of `rescale` (independent Bernoulli pruning).  `estimator_variance` is its closed form, derived below
   from the independence of the keep decisions.

psi[k, i] is any fixed scalar per completion (a loss term, one gradient coordinate).
"""
import itertools
import math

import numpy as np


def pruning_probabilities(cand_q, cand_o, r_q, r_o):
    """P^q(q_k) = r_q on prompt candidates, 0 elsewhere; P^o likewise (Eq. 17, Eq. 15)."""
    Pq = np.where(np.asarray(cand_q) != 0, float(r_q), 0.0)
    Po = np.where(np.asarray(cand_o) != 0, float(r_o), 0.0)
    return Pq, Po


def single_sample_variance(psi, Pq, Po):
    """Appendix D with the batch as population.

    pi~(o_i | q_k) = (1 - Po[k,i]) / (G C_o(q_k)),  C_o(q_k) = (1/G) sum_i (1 - Po[k,i])         (Eq. 6)
    P~(q_k)        = (1 - Pq[k]) / (P C_q),          C_q     = (1/P) sum_k (1 - Pq[k])            (Eq. 10)
    gamma(o,q) = C_o(q)/(1 - Po),  gamma(q) = C_q/(1 - Pq)                                        (Eq. 8, Eq. 11)

    Returns a dict: mean (= the plain batch mean of psi: Eq. 13), total = Var[G_hat], term_I = Var_{q~P~}[gamma(q)
    G(q)], term_II = E_{q~P~}[gamma(q)^2 Var_{o~pi~}[gamma(o,q) psi]], gamma_q_second_moment = E_{q~P~}[gamma(q)^2],
    comp_var[k] = Var_{o~pi~}[gamma(o,q_k) psi], var_Q = Var_Q[G(q)], mean_var_O = E_q[Var_O[psi]] (population
    variances before pruning) and bound = var_Q + gamma_q_second_moment * mean_var_O (Theorem D.1).
    """
    psi = np.asarray(psi, dtype=np.float64)
    Pq = np.asarray(Pq, dtype=np.float64); Po = np.asarray(Po, dtype=np.float64)
    P, G = psi.shape
    C_q = float(np.mean(1.0 - Pq))
    C_o = np.mean(1.0 - Po, axis=1)
    p_q = (1.0 - Pq) / (P * C_q)                         # P~(q_k)
    p_o = (1.0 - Po) / (G * C_o[:, None])                # pi~(o_i | q_k)
    g_q = C_q / (1.0 - Pq)
    g_o = C_o[:, None] / (1.0 - Po)
    # expectations as sums over all (q, o)
    joint = p_q[:, None] * p_o
    ghat = g_q[:, None] * g_o * psi
    mean = float(np.sum(joint * ghat))
    total = float(np.sum(joint * ghat * ghat)) - mean * mean
    inner_mean = np.sum(p_o * g_o * psi, axis=1)         # E_{o~pi~}[gamma(o,q) psi] = G(q_k)
    comp_var = np.sum(p_o * (g_o * psi) ** 2, axis=1) - inner_mean ** 2
    term_I = float(np.sum(p_q * (g_q * inner_mean) ** 2)) - mean * mean
    term_II = float(np.sum(p_q * g_q ** 2 * comp_var))
    second = float(np.sum(p_q * g_q ** 2))
    Gq = psi.mean(axis=1)
    var_Q = float(np.mean(Gq ** 2) - np.mean(Gq) ** 2)
    mean_var_O = float(np.mean(np.mean(psi ** 2, axis=1) - Gq ** 2))
    return dict(mean=mean, total=total, term_I=term_I, term_II=term_II, gamma_q_second_moment=second,
                comp_var=comp_var, var_Q=var_Q, mean_var_O=mean_var_O, bound=var_Q + second * mean_var_O)


def completion_variance_formula(psi_k, Po_k):
    """The printed completion-level variance for one prompt: (C_o/G) sum_o psi_o^2/(1 - P_o) - G(q)^2, with
    C_o = (1/G) sum (1 - P_o)."""
    psi_k = np.asarray(psi_k, dtype=np.float64); Po_k = np.asarray(Po_k, dtype=np.float64)
    G = len(psi_k)
    C_o = float(np.mean(1.0 - Po_k))
    return C_o / G * float(np.sum(psi_k ** 2 / (1.0 - Po_k))) - float(np.mean(psi_k)) ** 2


def gamma_q_factor(b, r):
    """Appendix D.3: E_{q~P~}[gamma(q)^2] when a fraction b of the prompts is pruned with probability r."""
    return (1.0 - b * r) * (1.0 - (1.0 - b) * r) / (1.0 - r)


def estimator_variance(psi, Pq, Po):
    """Variance over the pruning draws of X = sum_{k,i} I_k J_ki psi_ki / (P G (1 - Pq_k)(1 - Po_ki)), the batch
    estimator with the weights of `rescale`, for independent keep decisions I_k ~ Bernoulli(1 - Pq_k),
    J_ki ~ Bernoulli(1 - Po_ki).

    Per prompt, Y_k = sum_i J_ki psi_ki/(1 - Po_ki) has mean s_k = sum_i psi_ki and variance
    v_k = sum_i psi_ki^2 Po_ki/(1 - Po_ki); I_k Y_k/(1 - Pq_k) has mean s_k and variance
    v_k/(1 - Pq_k) + s_k^2 Pq_k/(1 - Pq_k); prompts are independent.  E[X] = mean(psi).
    """
    psi = np.asarray(psi, dtype=np.float64)
    Pq = np.asarray(Pq, dtype=np.float64); Po = np.asarray(Po, dtype=np.float64)
    P, G = psi.shape
    s = psi.sum(axis=1)
    v = np.sum(psi ** 2 * Po / (1.0 - Po), axis=1)
    per_prompt = v / (1.0 - Pq) + s ** 2 * Pq / (1.0 - Pq)
    return float(per_prompt.sum()) / float(P * G) ** 2


def estimator_moments_by_enumeration(psi, Pq, Po):
    """Mean and variance of the same estimator by brute force over every keep pattern (tiny P, G only)."""
    psi = np.asarray(psi, dtype=np.float64)
    P, G = psi.shape
    Pq = [float(x) for x in np.asarray(Pq).reshape(-1)]
    Po = [float(x) for x in np.asarray(Po).reshape(-1)]
    flat = [float(x) for x in psi.reshape(-1)]
    m1 = m2 = 0.0
    for kq in itertools.product((0, 1), repeat=P):
        prob_q = 1.0
        for k in range(P):
            prob_q *= (1.0 - Pq[k]) if kq[k] else Pq[k]
        if prob_q == 0.0:
            continue
        for ko in itertools.product((0, 1), repeat=P * G):
            prob = prob_q
            x = 0.0
            for j in range(P * G):
                prob *= (1.0 - Po[j]) if ko[j] else Po[j]
                if ko[j] and kq[j // G]:
                    x += flat[j] / (P * G * (1.0 - Pq[j // G]) * (1.0 - Po[j]))
            m1 += prob * x
            m2 += prob * x * x
    return m1, m2 - m1 * m1


def monte_carlo_summary(values):
    """Sample mean, unbiased sample variance and the standard error of that variance (from the fourth central
    moment) of a list of estimator values."""
    x = np.asarray(values, dtype=np.float64)
    n = len(x)
    mean = float(x.mean())
    d = x - mean
    var = float(np.sum(d * d) / (n - 1))
    m4 = float(np.mean(d ** 4))
    se_var = math.sqrt(max(m4 - var * var * (n - 3) / (n - 1), 0.0) / n)
    return dict(n=n, mean=mean, var=var, se_mean=math.sqrt(var / n), se_var=se_var)
