"""Empirical variance of the rescaled estimator through the library's pruning, beside Appendix D's expressions.

Ten thousand pruning steps of one fixed batch go through dppo_prune_and_rescale; the masks and weights of every
step must equal the oracle's bit for bit, and the sample mean / variance of the batch estimator sum w_seq * psi
(psi: fixed per-completion terms) must agree with the full-batch mean (unbiasedness, Eq. 13) and with the exact
variance of that estimator (oracle/variance.py, itself pinned by brute force).  A second case checks the second
moment of gamma(q), the factor of Theorem D.1, at r = 0.5 / 0.7 / 0.9."""
import numpy as np
import pytest
import torch

import oracle
from oracle import variance as V

pytestmark = pytest.mark.gpu


def _run_steps(B, adv, mabs, H_prev, P, G, r_q, r_o, seed, n_steps):
    """n_steps calls of the library on one batch; returns keep_q [n,P], keep_o [n,P*G], w_seq [n,P*G], gamma_q [n,P]."""
    n = P * G
    f32 = dict(dtype=torch.float32, device="cuda"); i32 = dict(dtype=torch.int32, device="cuda"); u8 = dict(dtype=torch.uint8, device="cuda")
    d_adv = torch.from_numpy(adv.reshape(-1)).cuda(); d_mabs = torch.from_numpy(mabs).cuda()
    d_H = torch.from_numpy(H_prev).cuda()
    cand_q = torch.zeros(P, **u8); cand_o = torch.zeros(n, **u8)
    keep_q = torch.zeros((n_steps, P), **u8); keep_o = torch.zeros((n_steps, n), **u8)
    nq = torch.zeros(1, **i32); no = torch.zeros(P, **i32)
    gq = torch.zeros((n_steps, P), **f32); go = torch.zeros(n, **f32); ws = torch.zeros((n_steps, n), **f32)
    H_next = torch.zeros(P, **f32); status = torch.zeros(1, **i32)
    for step in range(n_steps):
        prm = B.PruneParams(P, G, r_q, r_o, 0, 0, seed, step)
        B.prune_and_rescale(prm, d_adv, d_mabs, d_H, None, None, cand_q, cand_o, keep_q[step], keep_o[step], nq, no,
                            gq[step], go, ws[step], H_next, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return (keep_q.cpu().numpy(), keep_o.cpu().numpy(), ws.cpu().numpy(), gq.cpu().numpy(),
            cand_q.cpu().numpy(), cand_o.cpu().numpy().reshape(P, G))


def test_estimator_variance_over_ten_thousand_steps():
    from paper_2603_04135_b200 import binding as B
    P, G, r_q, r_o, seed, n_steps = 8, 4, 0.5, 0.5, 21, 10000
    rng = np.random.default_rng(6)
    rate = np.array([0.1, 0.3, 0.5, 0.5, 0.6, 0.8, 0.9, 0.4])
    rewards = (rng.random((P, G)) < rate[:, None]).astype(np.float32)
    rewards[3] = [1, 0, 0, 1]; rewards[6] = [1, 1, 1, 0]            # a tie group and a one-off group
    adv, mabs = oracle.group_advantages(rewards)
    H_prev = oracle.group_advantages((rng.random((P, G)) < rate[:, None]).astype(np.float32))[1]
    psi = rng.normal(size=(P, G)) * (0.3 + np.abs(adv))             # larger terms where |A| is larger
    keep_q, keep_o, w_seq, _, cand_q, cand_o = _run_steps(B, adv, mabs, H_prev, P, G, r_q, r_o, seed, n_steps)

    # every step: the oracle's masks and weights, bit for bit
    for step in range(n_steps):
        ref = oracle.prune_and_rescale(adv, mabs, H_prev, r_q, r_o, seed=seed, step=step)
        assert np.array_equal(keep_q[step], ref["keep_q"]) and np.array_equal(keep_o[step], ref["keep_o"].reshape(-1)), step
        assert np.array_equal(w_seq[step].view(np.uint32), ref["w_seq"].reshape(-1).view(np.uint32)), step
    assert np.array_equal(cand_q, oracle.prompt_candidates(H_prev, P)) and np.array_equal(cand_o, oracle.completion_candidates(adv))

    # the estimator over the steps: unbiased, and with the variance the keep probabilities imply
    vals = (w_seq.astype(np.float64) * psi.reshape(-1)[None, :]).sum(axis=1)
    mc = V.monte_carlo_summary(vals)
    Pq, Po = V.pruning_probabilities(cand_q, cand_o, r_q, r_o)
    exact = V.estimator_variance(psi, Pq, Po)
    assert exact > 0
    assert abs(mc["mean"] - psi.mean()) <= 5 * mc["se_mean"], (mc, psi.mean())
    assert abs(mc["var"] - exact) <= 5 * mc["se_var"], (mc, exact)
    # retention frequencies: 1 - r on candidates, 1 elsewhere (prompt level; completion level given the prompt)
    fq = keep_q.mean(axis=0)
    assert np.all(np.abs(fq - (1 - Pq)) <= 5 * np.sqrt(0.25 / n_steps) + 1e-12)
    kept_prompt = keep_q.astype(bool)
    for k in range(P):
        fo = keep_o.reshape(n_steps, P, G)[kept_prompt[:, k], k].mean(axis=0)
        assert np.all(np.abs(fo - (1 - Po[k])) <= 5 * np.sqrt(0.25 / kept_prompt[:, k].sum()) + 1e-12)


@pytest.mark.parametrize("r", [0.5, 0.7, 0.9])
def test_gamma_q_second_moment_over_many_steps(r):
    """Theorem D.1's factor E_{q ~ pruned}[gamma(q)^2] = (1 - b r)(1 - (1 - b) r)/(1 - r), b = 1/2: the average over
    4000 steps of the mean of gamma_q^2 over the retained prompts (64 prompts, so |S^q|/P stays near 1 - b r)."""
    from paper_2603_04135_b200 import binding as B
    P, G, n_steps = 64, 2, 4000
    adv = np.zeros((P, G), dtype=np.float32); mabs = np.zeros(P, dtype=np.float32)
    H_prev = np.arange(P, dtype=np.float32)
    keep_q, _, _, gq, cand_q, _ = _run_steps(B, adv, mabs, H_prev, P, G, r, 0.0, 5, n_steps)
    assert cand_q.sum() == P // 2
    for step in (0, 1, 2, 17, n_steps - 1):                          # the masks are the oracle's
        ref = oracle.prune_and_rescale(adv, mabs, H_prev, r, 0.0, seed=5, step=step)
        assert np.array_equal(keep_q[step], ref["keep_q"]) and np.array_equal(gq[step].view(np.uint32), ref["gamma_q"].view(np.uint32))
    kept = keep_q.astype(bool)
    per_step = np.array([(gq[s][kept[s]].astype(np.float64) ** 2).mean() for s in range(n_steps)])
    closed = V.gamma_q_factor(0.5, r)
    # a ratio of random sums: unbiased only to first order in 1/P (about +3 % at r = 0.9), so 5 % plus the sampling error
    assert abs(per_step.mean() - closed) <= 0.05 * closed + 5 * per_step.std() / np.sqrt(n_steps), (per_step.mean(), closed)
