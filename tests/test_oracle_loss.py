"""Pins for the oracle's per-token log-prob, GRPO terms (Eq. 1), dlogits and the LM-head variant."""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _case(T=37, V=53, S=5, seed=0, sigma=0.3):
    rng = np.random.default_rng(seed)
    z = rng.normal(size=(T, V)) * 1.5
    y = rng.integers(0, V, size=T)
    cuts = np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False))
    cu = np.concatenate([[0], cuts, [T]])
    logp = scipy.special.log_softmax(z, axis=1)[np.arange(T), y]
    logp_old = logp + sigma * rng.normal(size=T)
    logp_ref = logp + sigma * rng.normal(size=T)
    adv = rng.normal(size=S); adv[0] = 0.0
    w = rng.random(S) + 0.1
    return z, y, logp_old, logp_ref, cu, adv, w


def test_logprob_matches_library_log_softmax():
    rng = np.random.default_rng(1)
    z = rng.normal(size=(20, 1000)) * 3 + 50.0       # large offsets: needs the max subtraction
    y = rng.integers(0, 1000, size=20)
    logp, lse = oracle.token_logprob(z, y)
    assert np.allclose(logp, scipy.special.log_softmax(z, axis=1)[np.arange(20), y], rtol=0, atol=1e-12)
    assert np.allclose(lse, torch.logsumexp(torch.from_numpy(z), dim=1).numpy(), rtol=0, atol=1e-12)
    logp2, _ = oracle.token_logprob(z, y, tau=2.0)
    assert np.allclose(logp2, scipy.special.log_softmax(z / 2.0, axis=1)[np.arange(20), y], atol=1e-12)
    # a two-logit row in closed form: log sigmoid
    lp, _ = oracle.token_logprob(np.array([[1.5, -0.5]]), [0])
    assert math.isclose(lp[0], -math.log1p(math.exp(-2.0)), rel_tol=1e-14)


def test_clip_branches_golden():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "clip_branches.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 9
    for A, rho, surr, clipped in rows:
        A, rho, surr, clipped = float(A), float(rho), float(surr), int(clipped)
        tt = oracle.token_terms(np.array([math.log(rho)]), np.array([0.0]), np.array([math.log(rho)]),
                                np.array([A]), 0.2, 0.2, 0.04)
        assert math.isclose(tt["surr"][0], surr, rel_tol=1e-12, abs_tol=1e-15)
        assert bool(tt["clipped"][0]) == bool(clipped)
        assert abs(tt["kl"][0]) < 1e-15                        # rho_hat = 1
        want_dj = 0.0 if clipped else A * rho                  # clipped branch is constant in theta
        assert math.isclose(tt["dj"][0], want_dj, rel_tol=1e-12, abs_tol=1e-15)
    # the boundary itself still passes gradient
    tt = oracle.token_terms(np.array([math.log(1.2)]), np.array([0.0]), np.array([0.0]), np.array([1.0]),
                            0.2, 0.2, 0.0)
    assert not tt["clipped"][0]
    # decoupled bounds: eps_lo = 0.2, eps_hi = 0.5
    tt = oracle.token_terms(np.log([1.4, 0.7]), np.zeros(2), np.zeros(2), np.array([1.0, -1.0]), 0.2, 0.5, 0.0)
    assert list(tt["clipped"]) == [False, True] and math.isclose(tt["surr"][1], -0.8)


def test_kl_estimator_nonnegative_and_zero_at_one():
    d = np.linspace(-3, 3, 601)
    tt = oracle.token_terms(np.zeros_like(d), np.zeros_like(d), d, np.zeros_like(d), 0.2, 0.2, 1.0)
    assert (tt["kl"] >= 0).all()
    assert tt["kl"][300] == 0 and (tt["kl"][np.arange(601) != 300] > 0).all()
    # rho_hat - log rho_hat - 1 at rho_hat = e: e - 2
    tt = oracle.token_terms(np.array([0.0]), np.array([0.0]), np.array([1.0]), np.array([0.0]), 0.2, 0.2, 1.0)
    assert math.isclose(tt["kl"][0], math.e - 2.0, rel_tol=1e-14)


def test_dlogits_rows_sum_to_zero_and_match_finite_differences():
    z, y, lo, lr, cu, adv, w = _case()
    out = oracle.grpo_loss(z, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04)
    assert np.abs(out["dlogits"].sum(axis=1)).max() < 1e-14
    assert math.isclose(out["loss"], out["pg"] + 0.04 * out["kl"], rel_tol=1e-12)
    assert out["clipped"].any() and not out["clipped"].all()
    rng = np.random.default_rng(5)
    h = 1e-6
    checked = 0
    for _ in range(40):
        t = int(rng.integers(0, z.shape[0])); v = int(rng.integers(0, z.shape[1]))
        if rng.random() < 0.3:
            v = int(y[t])
        if min(abs(out["rho"][t] - 0.8), abs(out["rho"][t] - 1.2)) < 1e-3:
            continue                                            # kink of the clip
        zp = z.copy(); zp[t, v] += h
        zm = z.copy(); zm[t, v] -= h
        fp = oracle.grpo_loss(zp, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, want_dlogits=False)["loss"]
        fm = oracle.grpo_loss(zm, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, want_dlogits=False)["loss"]
        fd = (fp - fm) / (2 * h)
        assert math.isclose(fd, out["dlogits"][t, v], rel_tol=1e-5, abs_tol=1e-9), (t, v)
        checked += 1
    assert checked > 25
    # temperature: gradient w.r.t. the raw logits
    out_t = oracle.grpo_loss(z, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, tau=1.7)
    t, v = 3, int(y[3])
    zp = z.copy(); zp[t, v] += h
    zm = z.copy(); zm[t, v] -= h
    fd = (oracle.grpo_loss(zp, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, tau=1.7, want_dlogits=False)["loss"]
          - oracle.grpo_loss(zm, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, tau=1.7, want_dlogits=False)["loss"]) / (2 * h)
    assert math.isclose(fd, out_t["dlogits"][t, v], rel_tol=1e-5, abs_tol=1e-9)


def test_on_policy_special_case():
    # rho == 1 and beta == 0: per sequence the surrogate is A, so loss = -sum_s w_s A_s and the
    # logp-gradients of a sequence add up to -w_s A_s
    z, y, _, _, cu, adv, w = _case(T=60, seed=3)
    logp = scipy.special.log_softmax(z, axis=1)[np.arange(len(y)), y]
    out = oracle.grpo_loss(z, y, logp, logp, cu, adv, w, 0.2, 0.2, 0.0)
    assert math.isclose(out["loss"], -float((w * adv).sum()), rel_tol=1e-12)
    for s in range(len(adv)):
        assert math.isclose(out["g"][cu[s]:cu[s + 1]].sum(), -w[s] * adv[s], rel_tol=1e-12, abs_tol=1e-15)
    assert out["clip_frac"] == 0 and abs(out["kl"]) < 1e-15
    # un-pruned GRPO on policy: w = 1/(P G) and group advantages sum to zero -> zero loss
    r = np.array([[1, 0, 0, 1, 0], [0, 0, 1, 0, 0]], dtype=np.float32)
    A, mabs = oracle.group_advantages(r)
    pr = oracle.prune_and_rescale(A, mabs, None, 0.0, 0.0)
    T = 50
    cu2 = np.arange(0, T + 1, 5)
    out = oracle.grpo_loss(z[:T], y[:T], logp[:T], logp[:T], cu2, A.reshape(-1), pr["w_seq"].reshape(-1),
                           0.2, 0.2, 0.0)
    assert abs(out["loss"]) < 1e-7


def test_rows_subset_and_chunking_agree():
    z, y, lo, lr, cu, adv, w = _case(T=41, seed=7)
    full = oracle.grpo_loss(z, y, lo, lr, cu, adv, w)
    rows = [0, 5, 17, 40]
    sub = oracle.grpo_loss(z[rows], y, lo, lr, cu, adv, w, rows=rows, chunk=3)
    assert np.array_equal(sub["dlogits"], full["dlogits"][rows])
    assert np.array_equal(sub["logp"], full["logp"][rows])
    small = oracle.grpo_loss(z, y, lo, lr, cu, adv, w, chunk=7)
    assert np.array_equal(small["dlogits"], full["dlogits"]) and small["loss"] == full["loss"]
    # token weights: W_t = w_s / |o_s|
    for s in range(len(adv)):
        assert np.allclose(full["W"][cu[s]:cu[s + 1]], w[s] / (cu[s + 1] - cu[s]))


def test_pruned_loss_is_unbiased_for_the_full_loss():
    # exact enumeration over keep/drop patterns of value and gradient of the real loss
    import itertools
    P, G, V = 2, 3, 11
    rng = np.random.default_rng(9)
    r = np.array([[1, 0, 0], [1, 1, 0]], dtype=np.float32)
    adv, mabs = oracle.group_advantages(r)
    H = np.array([0.1, 0.7], dtype=np.float32)
    lens = rng.integers(2, 5, size=P * G)
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    z = rng.normal(size=(T, V)); y = rng.integers(0, V, size=T)
    lo = scipy.special.log_softmax(z, axis=1)[np.arange(T), y] + 0.2 * rng.normal(size=T)
    lr = lo + 0.1 * rng.normal(size=T)
    r_q, r_o = 0.5, 0.4
    full_pr = oracle.prune_and_rescale(adv, mabs, H, 0.0, 0.0)
    full = oracle.grpo_loss(z, y, lo, lr, cu, adv.reshape(-1), full_pr["w_seq"].reshape(-1))
    cand_o = oracle.completion_candidates(adv); cand_q = oracle.prompt_candidates(H, P)
    cq = [k for k in range(P) if cand_q[k]]
    co = [(k, i) for k in range(P) for i in range(G) if cand_o[k, i]]
    e_loss, e_grad = 0.0, np.zeros_like(z)
    for pat in itertools.product([0, 1], repeat=len(cq) + len(co)):
        u_q = np.full(P, 0.999); u_o = np.full((P, G), 0.999); pr = 1.0
        for k, drop in zip(cq, pat[:len(cq)]):
            u_q[k] = 0.0 if drop else 0.999; pr *= r_q if drop else 1 - r_q
        for (k, i), drop in zip(co, pat[len(cq):]):
            u_o[k, i] = 0.0 if drop else 0.999; pr *= r_o if drop else 1 - r_o
        o = oracle.prune_and_rescale(adv, mabs, H, r_q, r_o, u_q=u_q, u_o=u_o)
        # pruned sequences carry weight 0: the same token layout serves every pattern
        res = oracle.grpo_loss(z, y, lo, lr, cu, adv.reshape(-1), o["w_seq"].reshape(-1))
        e_loss += pr * res["loss"]; e_grad += pr * res["dlogits"]
    assert math.isclose(e_loss, full["loss"], rel_tol=0, abs_tol=1e-7 * full["abs_sum"] + 1e-9)
    assert np.abs(e_grad - full["dlogits"]).max() < 1e-7 * np.abs(full["dlogits"]).max() + 1e-10


def test_lmhead_variant():
    rng = np.random.default_rng(11)
    T, Hd, V, S = 12, 8, 17, 3
    h = rng.normal(size=(T, Hd)); Wm = rng.normal(size=(V, Hd)) / math.sqrt(Hd)
    y = rng.integers(0, V, size=T); cu = np.array([0, 4, 9, 12])
    adv = np.array([1.0, -0.5, 0.3]); w = np.array([0.2, 0.3, 0.1])
    z = np.einsum("th,vh->tv", h, Wm)
    lo = scipy.special.log_softmax(z, axis=1)[np.arange(T), y] + 0.1 * rng.normal(size=T)
    lr = lo + 0.1 * rng.normal(size=T)
    out = oracle.lmhead_grpo_loss(h, Wm, y, lo, lr, cu, adv, w)
    direct = oracle.grpo_loss(z, y, lo, lr, cu, adv, w)
    assert math.isclose(out["loss"], direct["loss"], rel_tol=1e-12)
    eps = 1e-6
    for (t, c) in [(0, 0), (5, 3), (11, 7)]:
        hp = h.copy(); hp[t, c] += eps; hm = h.copy(); hm[t, c] -= eps
        fd = (oracle.lmhead_grpo_loss(hp, Wm, y, lo, lr, cu, adv, w)["loss"]
              - oracle.lmhead_grpo_loss(hm, Wm, y, lo, lr, cu, adv, w)["loss"]) / (2 * eps)
        assert math.isclose(fd, out["dhidden"][t, c], rel_tol=1e-5, abs_tol=1e-10)
    for (v, c) in [(0, 0), (int(y[2]), 1), (16, 7)]:
        Wp = Wm.copy(); Wp[v, c] += eps; Wn = Wm.copy(); Wn[v, c] -= eps
        fd = (oracle.lmhead_grpo_loss(h, Wp, y, lo, lr, cu, adv, w)["loss"]
              - oracle.lmhead_grpo_loss(h, Wn, y, lo, lr, cu, adv, w)["loss"]) / (2 * eps)
        assert math.isclose(fd, out["dW"][v, c], rel_tol=1e-5, abs_tol=1e-10)


def test_bf16_conversions_match_torch():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.normal(size=5000) * 10.0, [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3e38, 1e-30]])
    bits = oracle.f64_to_bf16_bits(x)
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    back = oracle.bf16_bits_to_f64(bits)
    assert np.array_equal(back, torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).double().numpy())


def test_variant_without_length_normalisation():
    z, y, lo, lr, cu, adv, w = _case(T=60, seed=4)
    logp = scipy.special.log_softmax(z, axis=1)[np.arange(len(y)), y]
    # on policy, beta = 0: every token's surrogate is A, so the loss is -sum_s w_s A_s |o_s|
    out = oracle.grpo_loss(z, y, logp, logp, cu, adv, w, 0.2, 0.2, 0.0, length_norm=False)
    lens = np.diff(cu)
    assert math.isclose(out["loss"], -float((w * adv * lens).sum()), rel_tol=1e-12)
    # it is the normalised loss with weights w_s |o_s|
    a = oracle.grpo_loss(z, y, lo, lr, cu, adv, w, length_norm=False)
    b = oracle.grpo_loss(z, y, lo, lr, cu, adv, w * lens)
    assert math.isclose(a["loss"], b["loss"], rel_tol=1e-12) and np.allclose(a["dlogits"], b["dlogits"], rtol=1e-12, atol=0)


def test_sequence_level_ratio_variant():
    z, y, lo, lr, cu, adv, w = _case(T=45, V=31, S=4, seed=6, sigma=0.25)
    T = len(y)

    def loss_of(zz):
        logp = scipy.special.log_softmax(zz, axis=1)[np.arange(T), y]
        slr = oracle.sequence_log_ratio(logp, lo, cu)
        return oracle.grpo_loss(zz, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, seq_log_ratio=slr, want_dlogits=False)["loss"], slr

    base, slr = loss_of(z)
    # the mean token log-ratio per sequence, against a direct numpy mean
    logp = scipy.special.log_softmax(z, axis=1)[np.arange(T), y]
    for s in range(len(adv)):
        assert math.isclose(slr[s], float((logp - lo)[cu[s]:cu[s + 1]].mean()), rel_tol=1e-12, abs_tol=1e-15)
    out = oracle.grpo_loss(z, y, lo, lr, cu, adv, w, 0.2, 0.2, 0.04, seq_log_ratio=slr)
    assert math.isclose(out["loss"], base, rel_tol=1e-14)
    # every token of a sequence shares the ratio
    for s in range(len(adv)):
        assert np.allclose(out["rho"][cu[s]:cu[s + 1]], math.exp(slr[s]), rtol=1e-13)
    # the analytic gradient is the gradient of the whole two-stage map logits -> logp -> sequence ratio -> loss
    rng = np.random.default_rng(2)
    h, checked = 1e-6, 0
    for _ in range(30):
        t = int(rng.integers(0, T)); v = int(rng.integers(0, z.shape[1])) if rng.random() > 0.3 else int(y[t])
        s = int(np.searchsorted(cu, t, side="right") - 1)
        if min(abs(math.exp(slr[s]) - 0.8), abs(math.exp(slr[s]) - 1.2)) < 1e-3:
            continue
        zp = z.copy(); zp[t, v] += h; zm = z.copy(); zm[t, v] -= h
        fd = (loss_of(zp)[0] - loss_of(zm)[0]) / (2 * h)
        assert math.isclose(fd, out["dlogits"][t, v], rel_tol=1e-5, abs_tol=1e-9), (t, v)
        checked += 1
    assert checked > 15
    # when every token of every sequence has the same log-ratio the two objectives coincide
    lo2 = logp - 0.07
    a = oracle.grpo_loss(z, y, lo2, lr, cu, adv, w)
    b = oracle.grpo_loss(z, y, lo2, lr, cu, adv, w, seq_log_ratio=oracle.sequence_log_ratio(logp, lo2, cu))
    assert math.isclose(a["loss"], b["loss"], rel_tol=1e-12) and np.allclose(a["dlogits"], b["dlogits"], rtol=1e-10, atol=1e-18)
