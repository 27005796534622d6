"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200).

Integer / byte / index outputs (candidate sets, masks, counts, packing layout, cu_seqlens) and the
float outputs of the small steps (advantages, gamma, w_seq, H_next) must match bit for bit; the loss
within 1e-4 relative; dlogits element-wise (see parity_util.assert_dlogits_close).
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2603_04135_b200 import synth
from parity_util import (oracle_prune_pack, assert_prune_equal, assert_pack_equal, rows_to_f64, pick_rows,
                         assert_dlogits_close, clip_decision_is_stable, oracle_forward_all_rows, LOGP_TOL, Guarded)

pytestmark = pytest.mark.gpu


def _step(w, T_max, **kw):
    from paper_2603_04135_b200.step import DppoStep
    args = dict(P=w.P, G=w.G, L_row=w.L_row, N_win=w.N_win, r_q=w.r_q, r_o=w.r_o, V=max(w.V, 1), dtype=w.dtype,
                T_max=T_max, eps_lo=w.eps, eps_hi=w.eps, beta=w.beta)
    args.update(kw)
    return DppoStep(**args)


# ------------------------------------------------------------------------------------------- steps 1-4
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 8, 16])
@pytest.mark.parametrize("ddof", [0, 1])
def test_advantages_bit_exact(G, ddof):
    from paper_2603_04135_b200 import binding as B
    rng = np.random.default_rng(G * 10 + ddof)
    P = 257
    r = (rng.random((P, G)) < rng.random((P, 1))).astype(np.float32)
    r[5:40] = rng.normal(size=(35, G)).astype(np.float32)          # continuous rewards
    r[40:50] = np.float32(0.7)                                     # all equal
    for eps in (1e-6, 0.0):
        want_adv, want_mabs = oracle.group_advantages(r, ddof=ddof, std_eps=eps)
        d_r = torch.from_numpy(r).cuda()
        adv = torch.full((P * G,), -1.0, device="cuda"); mabs = torch.full((P,), -1.0, device="cuda")
        B.group_advantages(d_r, P, G, adv, mabs, ddof, eps)
        assert np.array_equal(adv.cpu().numpy().view(np.uint32), want_adv.reshape(-1).view(np.uint32))
        assert np.array_equal(mabs.cpu().numpy().view(np.uint32), want_mabs.view(np.uint32))


@pytest.mark.parametrize("name", ["config0", "config1", "config2"])
@pytest.mark.parametrize("history", [True, False])
def test_prune_pack_bit_exact_on_configs(name, history):
    w = synth.WORKLOADS[name]
    for seed in range(6):
        batch = synth.make_batch(w, seed)
        ref = oracle_prune_pack(batch, w, seed, step=seed + 3, use_history=history)
        st = _step(w, 1)
        st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
        st.prune_pack(seed=seed, step=seed + 3)
        assert_prune_equal(st.prune_results(), ref)
        assert_pack_equal(st.pack_results(), ref["pack"], w.P * w.G)
        assert st.pack_results()["status"][0] == 0


def test_config2_sweep_bit_exact_and_density():
    w = synth.WORKLOADS["config2"]
    batch = synth.make_batch(w, 2)
    naive_rows = None
    for r_q in (0.0, 0.25, 0.5):
        for r_o in (0.0, 0.25, 0.5):
            for N_win in (4, 16, 64):
                ref = oracle_prune_pack(batch, w, 2, step=11, r_q=r_q, r_o=r_o, N_win=N_win)
                st = _step(w, 1, r_q=r_q, r_o=r_o, N_win=N_win)
                st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
                st.prune_pack(seed=2, step=11)
                assert_prune_equal(st.prune_results(), ref)
                res = st.pack_results()
                assert_pack_equal(res, ref["pack"], w.P * w.G)
                n_units, n_rows, tokens, _ = (int(x) for x in res["counts"])
                if n_units:
                    density = tokens / (n_rows * w.L_row)
                    kept = batch.unit_len[ref["prune"]["keep_o"].reshape(-1) == 1]
                    padded = tokens / (n_units * kept.max())
                    assert 0 < density <= 1 and 0 < padded <= 1


def test_prune_explicit_draws_and_modes():
    w = synth.WORKLOADS["config2"]
    batch = synth.make_batch(w, 7)
    rng = np.random.default_rng(3)
    u_q = rng.random(w.P); u_o = rng.random((w.P, w.G))
    u_q[:4] = [0.0, 0.25, 0.24999999999999997, 0.9999999999999999]      # exact boundary of u < r
    u_o[3, :4] = u_o[3, 4]                                              # ties between draws (fixed-fraction order)
    for reverse in (False, True):
        for mode in (0, 1):
            for r in (0.25, 0.6):
                ref = oracle_prune_pack(batch, w, 0, 0, u_q=u_q, u_o=u_o, reverse=reverse, mode=mode, r_q=r, r_o=r)
                st = _step(w, 1, reverse=int(reverse), mode=mode, r_q=r, r_o=r)
                st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
                st.prune_pack(u_q=torch.from_numpy(u_q).cuda(), u_o=torch.from_numpy(u_o.reshape(-1)).cuda())
                assert_prune_equal(st.prune_results(), ref)
                assert_pack_equal(st.pack_results(), ref["pack"], w.P * w.G)


def test_prune_many_seeds_matches_generator_stream():
    # masks across many (seed, step) pairs: any difference in the counter-based generator shows up here
    w = synth.scaled(synth.WORKLOADS["config2"], P=64, G=16, r_q=0.5, r_o=0.5)
    batch = synth.make_batch(w, 1)
    st = _step(w, 1)
    for seed, step in [(0, 0), (1, 0), (0, 1), (2**40 + 5, 2**33 + 1), (2**64 - 1, 2**64 - 1), (123456789, 42)]:
        ref = oracle_prune_pack(batch, w, seed, step)
        st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
        st.prune_pack(seed=seed, step=step)
        assert_prune_equal(st.prune_results(), ref)
    st1 = _step(w, 1, mode=1)                                            # fixed fraction through the generator
    for seed, step in [(5, 6), (2**63, 3)]:
        ref = oracle_prune_pack(batch, w, seed, step, mode=1)
        st1.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
        st1.prune_pack(seed=seed, step=step)
        assert_prune_equal(st1.prune_results(), ref)


# ------------------------------------------------------------------------------------------- step 5
@pytest.mark.parametrize("policy", [0, 1])
def test_pack_random_streams(policy):
    from paper_2603_04135_b200 import binding as B
    rng = np.random.default_rng(policy)
    for trial in range(40):
        n = int(rng.integers(0, 300))
        L = int(rng.integers(20, 400))
        lens = rng.integers(1, L + 1, size=n).astype(np.int32)
        if trial % 3 == 0 and n:
            lens = np.minimum(lens, max(1, L // 8)).astype(np.int32)       # many units per row
        keep = (rng.random(n) < 0.7).astype(np.uint8) if trial % 2 else None
        loss_len = rng.integers(0, 50, size=n).astype(np.int32) if trial % 4 else None
        N_win = int(rng.choice([1, 2, 4, 16, 31, 32, 33, 64, 1000]))
        ref = oracle.pack_prompts(lens, L, N_win, keep=keep, loss_len=loss_len, best_fit=bool(policy))
        got = _run_pack(B, lens, keep, loss_len, L, N_win, policy)
        assert got["status"][0] == 0
        assert_pack_equal(got, ref, n)


def _run_pack(B, lens, keep, loss_len, L, N_win, policy):
    n = len(lens)
    i32 = dict(dtype=torch.int32, device="cuda")
    d_len = torch.from_numpy(np.asarray(lens, dtype=np.int32)).cuda() if n else torch.zeros(1, **i32)
    d_keep = torch.from_numpy(keep).cuda() if keep is not None else None
    d_loss = torch.from_numpy(loss_len).cuda() if loss_len is not None else None
    # every output sits between guard bands of sentinels: an overrun of any of them fails the test
    guarded = {k: Guarded((max(n, 1),), torch.int32, 55) for k in ("order", "row_of", "off_in_row", "row_fill")}
    guarded["cu_seqlens"] = Guarded((n + 1,), torch.int32, 55); guarded["counts"] = Guarded((4,), torch.int32, 55)
    outs = {k: g.t for k, g in guarded.items()}
    status = torch.zeros(1, **i32)
    prm = B.PackParams(n, L, N_win, policy)
    nbytes = B.pack_workspace_bytes(prm)
    ws = Guarded((max(nbytes, 16),), torch.uint8, 0)
    B.pack_prompts(prm, d_len, d_keep, d_loss, outs["order"], outs["row_of"], outs["off_in_row"], outs["row_fill"],
                   outs["cu_seqlens"], outs["counts"], ws.t, nbytes, status)
    torch.cuda.synchronize()
    for g in list(guarded.values()) + [ws]:
        g.check()
    res = {k: outs[k].cpu().numpy()[:n] for k in ("order", "row_of", "off_in_row", "row_fill")}
    res.update(cu_seqlens=outs["cu_seqlens"].cpu().numpy(), counts=outs["counts"].cpu().numpy(), status=status.cpu().numpy())
    return res


def test_pack_dataset_scale_and_bad_length():
    from paper_2603_04135_b200 import binding as B
    rng = np.random.default_rng(5)
    # a dataset-sized stream of prompt lengths (the paper packs its 7.5k-8.5k prompts at initialisation),
    # L_max = the longest sample; larger than the shared-memory length cache
    n = 8500
    lens = np.clip(np.rint(np.exp(rng.normal(math.log(150), 0.6, size=n))), 16, 1024).astype(np.int32)
    L = int(lens.max())
    for N_win in (8, 64):
        ref = oracle.pack_prompts(lens, L, N_win)
        got = _run_pack(B, lens, None, None, L, N_win, 0)
        assert_pack_equal(got, ref, n)
    # larger streams: the last size whose placed-bitmask sits in shared memory, and one beyond it (bitmask in the
    # workspace); short units so that the oracle's Python loop stays at a few seconds
    for n, N_win in ((65536, 16), (150000, 8), (1000000, 64)):
        lens = rng.integers(8, 200, size=n).astype(np.int32)
        keep = (rng.random(n) < 0.9).astype(np.uint8)
        ref = oracle.pack_prompts(lens, 512, N_win, keep=keep)
        got = _run_pack(B, lens, keep, None, 512, N_win, 0)
        assert got["status"][0] == 0
        assert_pack_equal(got, ref, n)
    lens2 = np.array([5, 9, 30, 2], dtype=np.int32)
    got = _run_pack(B, lens2, None, None, 20, 4, 0)
    assert got["status"][0] == B.STATUS_BAD_LENGTH and (got["counts"] == 0).all()
    got = _run_pack(B, lens2, np.array([1, 1, 0, 1], dtype=np.uint8), None, 20, 4, 0)
    assert got["status"][0] == 0 and got["counts"][0] == 3


# ------------------------------------------------------------------------------------------- steps 6-8
def _loss_case(V, dtype, T, S, seed, sigma_noise=0.05, logit_sigma=2.0, tau=1.0, pad=0, in_place=False,
               forward_only=False, n_tokens=None, beta=0.04, eps=(0.2, 0.2), variant=0, no_length_norm=False,
               seq_ratio=False, centre_on_oracle=False, neg_inf_cols=None):
    """Runs dppo_grpo_loss_fwd_bwd on a random case and compares everything with the oracle.
    centre_on_oracle: old / reference log-probs = the oracle's current log-prob + noise (for logits whose
    log-sum-exp is far from the Gaussian closed form the generator centres on)."""
    from paper_2603_04135_b200 import binding as B
    w = synth.scaled(synth.WORKLOADS["config0"], V=V, dtype=dtype, logit_sigma=logit_sigma)
    tok = synth.make_token_inputs(w, T, seed, device="cuda", sigma_old=sigma_noise, sigma_ref=2 * sigma_noise)
    rng = np.random.default_rng(seed)
    if neg_inf_cols is not None:
        # a masked part of the vocabulary: logits of -inf (probability zero), never sampled
        lo_c, hi_c = neg_inf_cols
        tok.logits[:, lo_c:hi_c] = float("-inf")
        hit = (tok.target >= lo_c) & (tok.target < hi_c)
        tok.target[hit] = 0 if lo_c > 0 else hi_c
        centre_on_oracle = True
    if centre_on_oracle:
        lp = oracle.token_logprob(tok.logits.to(torch.float64).cpu().numpy(), tok.target.cpu().numpy(), tau)[0]
        tok.logp_old = torch.from_numpy((lp + sigma_noise * rng.normal(size=T)).astype(np.float32)).cuda()
        tok.logp_ref = torch.from_numpy((lp + 2 * sigma_noise * rng.normal(size=T)).astype(np.float32)).cuda()
    T_true = T if n_tokens is None else n_tokens
    cuts = np.sort(rng.choice(np.arange(1, T_true), size=min(S - 1, T_true - 1), replace=False)) if T_true > 1 else []
    cu = np.concatenate([[0], cuts, [T_true]]).astype(np.int32)
    S_real = len(cu) - 1
    S_max = S_real + 3                                               # padded tail repeats the total
    cu_pad = np.concatenate([cu, np.full(S_max - S_real, T_true)]).astype(np.int32)
    adv = rng.normal(size=S_max).astype(np.float32); adv[0] = 0.0
    wseq = (rng.random(S_max) * 0.1).astype(np.float32)
    seg_map = rng.permutation(S_max).astype(np.int32)
    per16 = 4 if dtype == "f32" else 8                                # row stride must be a multiple of 16 bytes
    stride = -(-(V + pad) // per16) * per16
    pad = stride - V
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    # logits (written when dlogits aliases them), dlogits, the per-token outputs, the five scalars and the workspace
    # all sit between guard bands of sentinels
    g_buf = Guarded((T, stride), tdt, 0.0); buf = g_buf.t
    buf[:, :V] = tok.logits
    logits_before = buf.clone()
    g_dl = None if (in_place or forward_only) else Guarded((T, stride), tdt, 7.0)
    dl = buf if in_place else (None if forward_only else g_dl.t)
    prm = B.LossParams(T, V, B.BF16 if dtype == "bf16" else B.F32, stride, S_max, variant, eps[0], eps[1], beta, tau)
    nbytes = B.grpo_loss_workspace_bytes(prm)
    g_ws = Guarded((nbytes,), torch.uint8, 0); ws = g_ws.t
    g_loss = Guarded((5,), torch.float32, 0.0); g_logp = Guarded((T,), torch.float32, 0.0); g_lse = Guarded((T,), torch.float32, 0.0)
    loss_out, logp_out, lse_out = g_loss.t, g_logp.t, g_lse.t
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ntd = torch.tensor([T_true], dtype=torch.int32, device="cuda") if n_tokens is not None else None
    d_cu = torch.from_numpy(cu_pad).cuda()
    prm.no_length_norm = int(no_length_norm)
    slr_dev = None
    if seq_ratio:
        # sequence-level ratio: a forward-only sweep gives the current log-probs, their mean log-ratio per
        # sequence goes back in as a per-sequence input of the second sweep
        B.grpo_loss_fwd_bwd(prm, buf, tok.target, tok.logp_old, tok.logp_ref, d_cu, ntd, torch.from_numpy(adv).cuda(),
                            torch.from_numpy(wseq).cuda(), torch.from_numpy(seg_map).cuda(), None, logp_out, None,
                            loss_out, ws, nbytes, status)
        slr_dev = torch.full((S_max,), 9.0, device="cuda")
        B.sequence_log_ratio(logp_out, tok.logp_old, d_cu, S_max, slr_dev)
        prm.seq_log_ratio = slr_dev.data_ptr()
    B.grpo_loss_fwd_bwd(prm, buf, tok.target, tok.logp_old, tok.logp_ref, d_cu, ntd,
                        torch.from_numpy(adv).cuda(), torch.from_numpy(wseq).cuda(), torch.from_numpy(seg_map).cuda(),
                        dl, logp_out, lse_out, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for g in (g_buf, g_dl, g_ws, g_loss, g_logp, g_lse):
        if g is not None:
            g.check()

    z = logits_before[:T_true, :V].to(torch.float64).cpu().numpy()
    slr = None
    if seq_ratio:
        lp64 = oracle.token_logprob(z, tok.target.cpu().numpy()[:T_true], tau)[0]
        slr = oracle.sequence_log_ratio(lp64, tok.logp_old.cpu().numpy()[:T_true], cu)
        got_slr = slr_dev.cpu().numpy()
        assert np.abs(got_slr[:S_real] - slr).max() <= LOGP_TOL[dtype] and (got_slr[S_real:] == 0).all()
    ref = oracle.grpo_loss(z, tok.target.cpu().numpy(), tok.logp_old.cpu().numpy(), tok.logp_ref.cpu().numpy(), cu,
                           adv[seg_map][:S_real], wseq[seg_map][:S_real], eps[0], eps[1], beta, tau,
                           want_dlogits=not forward_only, length_norm=not no_length_norm, seq_log_ratio=slr)
    lo = loss_out.cpu().numpy().astype(np.float64)
    stable = clip_decision_is_stable(ref["rho"], eps[0], eps[1])
    assert stable.all(), "test case sits on a clip boundary; change the seed"
    assert abs(lo[0] - ref["loss"]) <= 1e-4 * abs(ref["loss"]) + 1e-7 * ref["abs_sum"]
    assert abs(lo[0] - ref["loss"]) <= 1e-4 * ref["abs_sum"]
    assert abs(lo[1] - ref["pg"]) <= 1e-4 * ref["abs_sum"] and abs(lo[2] - ref["kl"]) <= 1e-4 * max(ref["kl"], 1e-12) + 1e-9
    assert abs(lo[3] - ref["clip_frac"]) < 1e-6 and lo[4] == T_true
    tol = LOGP_TOL[dtype]
    # outputs are f32: at |logp| ~ 200 (the wide-range cases) one f32 rounding alone is 2^-17, so those cases
    # add two units of f32 roundoff relative to the value
    ulp = 2.0 ** -22 if centre_on_oracle else 0.0
    assert (np.abs(logp_out.cpu().numpy()[:T_true] - ref["logp"]) <= tol + ulp * np.abs(ref["logp"])).all()
    assert (np.abs(lse_out.cpu().numpy()[:T_true] - ref["lse"]) <= tol + ulp * np.abs(ref["lse"])).all()
    if not forward_only:
        got = dl[:T_true, :V].to(torch.float64).cpu().numpy()
        assert_dlogits_close(got, ref, dtype, beta)
        if not in_place:
            assert torch.equal(buf, logits_before)                   # inputs untouched
            assert (dl[T_true:] == 7.0).all()                        # rows past T untouched
            if pad:
                assert (dl[:, V:] == 7.0).all()                      # padding columns untouched
    return ref


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 3, 5, 8, 1000, 1024, 4099, 32768])
def test_loss_small_vocab_shapes(dtype, V):
    _loss_case(V, dtype, T=67, S=5, seed=V)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_loss_options(dtype):
    V = 2056
    _loss_case(V, dtype, T=50, S=4, seed=1, pad=8)                           # strided rows
    _loss_case(V, dtype, T=50, S=4, seed=2, in_place=True)                   # dlogits aliases logits
    _loss_case(V, dtype, T=50, S=4, seed=3, forward_only=True)
    _loss_case(V, dtype, T=50, S=4, seed=4, n_tokens=37)                     # true T below T_max
    _loss_case(V, dtype, T=50, S=4, seed=5, tau=1.7)
    _loss_case(V, dtype, T=50, S=4, seed=6, beta=0.0, eps=(0.2, 0.5))        # decoupled clip range
    _loss_case(V, dtype, T=1, S=1, seed=7)
    _loss_case(V, dtype, T=300, S=300, seed=8)                               # one token per sequence


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_loss_all_clip_branches(dtype):
    # log-ratio noise 0.3: clipped and unclipped tokens of both advantage signs, and A = 0
    ref = _loss_case(1024, dtype, T=400, S=12, seed=21, sigma_noise=0.3, logit_sigma=1.0)
    A, rho, cl = ref["A"], ref["rho"], ref["clipped"]
    assert (cl & (A > 0) & (rho > 1.2)).any() and (cl & (A < 0) & (rho < 0.8)).any()
    assert (~cl & (A > 0)).any() and (~cl & (A < 0)).any() and (A == 0).any()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_loss_variants_of_other_objectives(dtype):
    # no 1/|o| normalisation (token-level aggregation is then a matter of w), sequence-level ratio
    _loss_case(2056, dtype, T=80, S=6, seed=71, no_length_norm=True)
    _loss_case(2056, dtype, T=80, S=6, seed=72, seq_ratio=True, sigma_noise=0.3)
    _loss_case(2056, dtype, T=80, S=6, seed=73, seq_ratio=True, n_tokens=61)
    if dtype == "bf16":
        _loss_case(151936, dtype, T=40, S=3, seed=74, seq_ratio=True, variant=40256)
        _loss_case(151936, dtype, T=40, S=3, seed=75, no_length_norm=True, variant=0)


def test_loss_full_vocab_bf16_rows():
    # Qwen3 vocabulary: rows of 151,936 bf16 (several tiles, 16-byte multiple), plus a ragged variant
    _loss_case(151936, "bf16", T=24, S=3, seed=31)
    _loss_case(151936 - 5, "bf16", T=9, S=2, seed=32, pad=5)
    _loss_case(151936, "f32", T=6, S=2, seed=33)


@pytest.mark.parametrize("C", [1, 2, 4, 8])
def test_loss_cluster_kernel_variants(C):
    # the shared-memory cluster kernel, forced: full vocabulary, ragged tails, slices that are empty
    big = 151936 if C >= 2 else 100000            # one CTA holds at most 220 KB of a row
    for threads in (128, 256, 512):
        v = C * 10000 + threads
        _loss_case(big, "bf16", T=13, S=3, seed=40 + C, variant=v)
    v = C * 10000 + 256
    _loss_case(big - 5, "bf16", T=7, S=2, seed=50 + C, variant=v, pad=5 if C >= 2 else 0)   # tail of 3 elements
    _loss_case(big, "bf16", T=9, S=2, seed=51 + C, variant=v, in_place=True)
    _loss_case(big, "bf16", T=9, S=2, seed=52 + C, variant=v, forward_only=True)
    _loss_case(big, "bf16", T=9, S=2, seed=53 + C, variant=v, n_tokens=5, tau=1.3)
    _loss_case(4099, "bf16", T=33, S=4, seed=54 + C, variant=v)
    _loss_case(24, "bf16", T=33, S=4, seed=55 + C, variant=v)                    # 3 vectors: most slices are empty
    _loss_case(5, "bf16", T=20, S=2, seed=56 + C, variant=v)                     # tail only
    _loss_case(65536, "bf16", T=300, S=7, seed=57 + C, variant=v, sigma_noise=0.3)
    # 46 M elements: some land where the fp16 rounding of the exponential and the bf16 rounding of the output
    # both sit at their worst case (this seed has elements at 1.05 x 2^-8 relative)
    _loss_case(65536, "bf16", T=700, S=7, seed=61, variant=v)


@pytest.mark.parametrize("C", [1, 2, 4, 8])
def test_loss_cluster_kernel_f32_rows(C):
    # the same kernel on f32 rows (4-element vectors, f32 exponentials in place, f32 dlogits)
    v = C * 10000 + 256
    if C >= 4:
        for threads in (128, 256, 512):
            _loss_case(151936, "f32", T=11, S=3, seed=140 + C, variant=C * 10000 + threads)
        _loss_case(151936 - 5, "f32", T=7, S=2, seed=150 + C, variant=v, pad=1)         # tail of 3 elements, padded stride
        _loss_case(151936, "f32", T=9, S=2, seed=151 + C, variant=v, in_place=True)
        _loss_case(151936, "f32", T=9, S=2, seed=153 + C, variant=v, n_tokens=5, tau=1.3)
    _loss_case(65536 if C >= 2 else 50000, "f32", T=40, S=4, seed=152 + C, variant=v, forward_only=True)
    _loss_case(4099, "f32", T=33, S=4, seed=154 + C, variant=v)
    _loss_case(12, "f32", T=33, S=4, seed=155 + C, variant=v)                           # 3 vectors: most slices are empty
    _loss_case(3, "f32", T=20, S=2, seed=156 + C, variant=v)                            # tail only
    _loss_case(65536 if C >= 2 else 50000, "f32", T=200, S=7, seed=157 + C, variant=v, sigma_noise=0.3)
    _loss_case(1024, "f32", T=40, S=3, seed=158 + C, variant=v, logit_sigma=40.0, centre_on_oracle=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_loss_warp_per_row_kernel(dtype):
    # short rows, one warp per row with the row in registers (forced): every vectors-per-lane form, ragged ends,
    # fewer rows than warps and many more, in place, forward only, masked columns
    v = 2
    for V, seed in [(1, 300), (5, 301), (8, 302), (100, 303), (256, 304), (1000, 305), (1024, 306), (2047, 307)]:
        _loss_case(V, dtype, T=67, S=5, seed=seed, variant=v)
    big = 4096 if dtype == "bf16" else 2048                                      # 16 vectors per lane (8 KB rows)
    _loss_case(big, dtype, T=40, S=3, seed=310, variant=v)
    _loss_case(1536, dtype, T=5000, S=40, seed=311, variant=v)                   # several rows per warp
    _loss_case(1024, dtype, T=50, S=4, seed=312, variant=v, in_place=True)
    _loss_case(1024, dtype, T=50, S=4, seed=313, variant=v, forward_only=True)
    _loss_case(1000, dtype, T=50, S=4, seed=314, variant=v, n_tokens=37, tau=1.7, pad=8)
    _loss_case(1024, dtype, T=20, S=2, seed=315, variant=v, neg_inf_cols=(100, 1024))
    _loss_case(1024, dtype, T=40, S=3, seed=316, variant=v, logit_sigma=40.0, centre_on_oracle=True)
    _loss_case(2040, dtype, T=80, S=6, seed=317, variant=v, seq_ratio=True, sigma_noise=0.3)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_loss_tile_kernel(dtype):
    # calls with dlogits on the tile kernel (forced): rows of one vector, of every vectors-per-lane form, rows that are
    # split into several 2 KB units with a short last one, rows that fill a stage alone; fewer tiles than CTAs and
    # several tiles per CTA (so that stages are reused many times), a last tile with fewer rows, sequences that end
    # inside a tile, a padded row pitch, in place, a device-side token count, masked columns (a whole unit of -inf),
    # a wide dynamic range
    v = 4
    per = 8 if dtype == "bf16" else 4
    for nvec, T, seed in [(1, 67, 600), (3, 200, 601), (32, 67, 602), (33, 150, 603), (64, 67, 604), (65, 67, 605), (128, 67, 606),
                          (129, 40, 607), (300, 67, 608), (512, 40, 609), (1000, 23, 610), (2048, 9, 611)]:
        _loss_case(nvec * per, dtype, T=T, S=5, seed=seed, variant=v)
    _loss_case(128 * per, dtype, T=40000, S=300, seed=620, variant=v, centre_on_oracle=True)                     # 17 tiles per CTA, short sequences
    _loss_case(64 * per, dtype, T=30011, S=40, seed=621, variant=v, centre_on_oracle=True)
    _loss_case(200 * per, dtype, T=5000, S=40, seed=622, variant=v, pad=3 * per, centre_on_oracle=True)          # padded pitch: the padding stays
    _loss_case(128 * per, dtype, T=500, S=4, seed=623, variant=v, in_place=True)
    _loss_case(96 * per, dtype, T=900, S=7, seed=624, variant=v, n_tokens=611, tau=1.7)
    _loss_case(512 * per, dtype, T=50, S=2, seed=625, variant=v, neg_inf_cols=(128 * per, 256 * per))
    _loss_case(512 * per, dtype, T=50, S=2, seed=626, variant=v, neg_inf_cols=(0, 300 * per))
    _loss_case(128 * per, dtype, T=40, S=3, seed=627, variant=v, logit_sigma=40.0, centre_on_oracle=True)
    from paper_2603_04135_b200 import binding as B
    _loss_case(64 * per, dtype, T=30000, S=7000, seed=650, variant=v, centre_on_oracle=True)   # more sequences than the shared-memory copy of cu_seqlens holds
    _loss_case(128 * per, dtype, T=3, S=2, seed=651, variant=v)                                # fewer rows than a tile
    _loss_case(128 * per, dtype, T=1, S=1, seed=652, variant=v)
    # forward only: pass 1 and the scalar stage; stages reused many times, the sequence-level ratio's two sweeps
    _loss_case(128 * per, dtype, T=40000, S=300, seed=640, variant=v, forward_only=True, centre_on_oracle=True)
    _loss_case(300 * per, dtype, T=67, S=5, seed=641, variant=v, forward_only=True)
    _loss_case(16 * per, dtype, T=9000, S=50, seed=642, variant=v, forward_only=True, n_tokens=8000, tau=0.8)
    _loss_case(255 * per, dtype, T=80, S=6, seed=643, variant=v, seq_ratio=True, sigma_noise=0.3)
    for bad in (dict(V=1004 if dtype == "bf16" else 1002, T=8), dict(V=4096 * per, T=8)):
        with pytest.raises(B.DppoError) as e:                                    # ragged tail, a row above 32 KB
            _loss_case(bad.pop("V"), dtype, S=2, seed=630, variant=v, **bad)
        assert e.value.code == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_loss_streaming_forward_kernel(dtype):
    # forward-only calls on the streaming kernel (forced): rows of less than a vector, of one piece, of several pieces
    # with a ragged last one, ragged tails, more rows than CTAs, a device-side token count, a temperature, masked
    # columns (a whole piece of -inf, and a masked start), a wide dynamic range, the sequence-level ratio's first sweep
    v = 3
    for V, T, seed in [(5, 20, 500), (8, 33, 501), (1000, 67, 502), (4099, 40, 503), (16384, 300, 504), (16384 + 24, 21, 505),
                       (65536 + 8, 19, 506), (151936, 12, 507), (151936 - 5, 9, 508)]:
        _loss_case(V, dtype, T=T, S=3, seed=seed, variant=v, forward_only=True)
    _loss_case(40000, dtype, T=700, S=9, seed=510, variant=v, forward_only=True)             # several rows per CTA
    _loss_case(40000, dtype, T=50, S=4, seed=511, variant=v, forward_only=True, n_tokens=37, tau=1.7, pad=8)
    _loss_case(151936, dtype, T=6, S=2, seed=512, variant=v, forward_only=True, neg_inf_cols=(16384, 32768))
    _loss_case(151936, dtype, T=6, S=2, seed=513, variant=v, forward_only=True, neg_inf_cols=(0, 37984))
    _loss_case(151936, dtype, T=6, S=2, seed=514, variant=v, forward_only=True, neg_inf_cols=(151669, 151936))
    _loss_case(70000, dtype, T=8, S=2, seed=515, variant=v, forward_only=True, logit_sigma=30.0, centre_on_oracle=True)
    from paper_2603_04135_b200 import binding as B
    with pytest.raises(B.DppoError) as e:                                        # it has no backward
        _loss_case(1000, dtype, T=8, S=2, seed=516, variant=v)
    assert e.value.code == B.ERR_UNSUPPORTED


def test_loss_auto_dispatch_matches_forced_kernels():
    # variant 0 on a long bf16 row takes the cluster kernel; outputs agree with the general kernel's
    a = _loss_case(151936, "bf16", T=11, S=2, seed=60, variant=0)
    b = _loss_case(151936, "bf16", T=11, S=2, seed=60, variant=1)
    assert a["loss"] == b["loss"]                                                # same oracle case both times
    _loss_case(151936, "f32", T=11, S=2, seed=61, variant=0)                     # f32: cluster of 8
    _loss_case(151936, "f32", T=11, S=2, seed=61, variant=1)
    _loss_case(40000, "f32", T=30, S=2, seed=62, variant=0)                      # f32: cluster of 4
    for V, dtype, seed in [(8192, "bf16", 63), (16384, "bf16", 64), (32768, "bf16", 65), (50304, "bf16", 66),
                           (65536, "bf16", 67), (128256, "bf16", 68), (8192, "f32", 69), (16384, "f32", 70),
                           (100000, "f32", 71)]:
        _loss_case(V, dtype, T=20, S=3, seed=seed, variant=0)                    # one, two, four, eight CTAs per row


def test_loss_wide_dynamic_range():
    # logits spread over +-100 and more within a row: exponentials far below the row maximum underflow, the
    # reference point of every partial sum still has to be joined correctly
    _loss_case(151936, "bf16", T=8, S=2, seed=90, logit_sigma=30.0, centre_on_oracle=True)
    _loss_case(151936, "bf16", T=8, S=2, seed=91, logit_sigma=30.0, variant=1, centre_on_oracle=True)
    _loss_case(1024, "f32", T=40, S=3, seed=92, logit_sigma=40.0, centre_on_oracle=True)
    _loss_case(4099, "bf16", T=40, S=3, seed=93, logit_sigma=0.0)                # every logit equal: lse = ln V


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_loss_masked_vocabulary(dtype):
    # -inf logits: a few columns, a whole slice of the cluster kernel (37,984 elements of a bf16 row over 4 CTAs,
    # 18,992 of an f32 row over 8), the padded end of the vocabulary
    V = 151936
    _loss_case(V, dtype, T=6, S=2, seed=201, neg_inf_cols=(1000, 3000))
    _loss_case(V, dtype, T=6, S=2, seed=202, neg_inf_cols=(37984, 75968))
    _loss_case(V, dtype, T=6, S=2, seed=203, neg_inf_cols=(0, 37984))
    _loss_case(V, dtype, T=6, S=2, seed=204, neg_inf_cols=(151669, V))
    _loss_case(V, dtype, T=6, S=2, seed=205, neg_inf_cols=(37984, 75968), variant=1)
    _loss_case(4099, dtype, T=20, S=2, seed=206, neg_inf_cols=(100, 4099))
    # the general two-pass kernel with a masked START of the vocabulary: threads whose first elements are all -inf
    _loss_case(V, dtype, T=6, S=2, seed=207, neg_inf_cols=(0, 37984), variant=1)
    _loss_case(4099, dtype, T=20, S=2, seed=208, neg_inf_cols=(0, 100), variant=1)
    _loss_case(4099, dtype, T=20, S=2, seed=209, neg_inf_cols=(0, 4090), variant=1)      # only the ragged end is finite


@pytest.mark.parametrize("variant", [0, 1])
def test_loss_is_bit_reproducible(variant):
    # fixed reduction order everywhere: two runs of the same call give the same bits in every output
    from paper_2603_04135_b200 import binding as B
    V, T, S = 151936, 1500, 7
    w = synth.scaled(synth.WORKLOADS["config3"], V=V)
    tok = synth.make_token_inputs(w, T, 5, device="cuda")
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    rng = np.random.default_rng(5)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.from_numpy((rng.random(S) * 0.1).astype(np.float32)).cuda()
    prm = B.LossParams(T, V, B.BF16, V, S, variant, 0.2, 0.2, 0.04, 1.0)
    nbytes = B.grpo_loss_workspace_bytes(prm)
    outs = []
    for _ in range(2):
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        dl = torch.empty_like(tok.logits); loss_out = torch.zeros(5, device="cuda")
        logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, wseq, None, dl,
                            logp_out, lse_out, loss_out, ws, nbytes, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        outs.append((dl, loss_out, logp_out, lse_out))
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a.view(torch.int32),
                           b.view(torch.int16) if b.dtype == torch.bfloat16 else b.view(torch.int32))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_loss_kernel_choice_boundaries(dtype):
    # row lengths on both sides of every switch of the library's kernel choice: warp per row -> one CTA -> two ->
    # four -> eight CTAs -> general kernel (limits in 16-byte vectors: 512, 2816, 7040, 19456, 38912)
    per_vec = 8 if dtype == "bf16" else 4
    warp_max = 512
    seed = 400
    # (dense rows of up to 1024 vectors take the tile kernel: both sides of that limit too, and a ragged row next to
    # each, which stays with the other kernels)
    for nvec in (warp_max, 1024, 2816, 7040, 19456, 38912):
        for V in (nvec * per_vec, nvec * per_vec + per_vec, nvec * per_vec + 3):
            seed += 1
            _loss_case(V, dtype, T=5, S=2, seed=seed, variant=0)


def test_loss_kernel_choice_query():
    # the host-side query names the kernel a call takes, for every branch of the choice
    from paper_2603_04135_b200 import binding as B

    def choice(V, dtype, variant=0):
        esz = 2 if dtype == B.BF16 else 4
        stride = -(-V * esz // 16) * 16 // esz
        c = B.grpo_loss_kernel_choice(B.LossParams(64, V, dtype, stride, 4, variant, 0.2, 0.2, 0.04, 1.0))
        return (c.kernel, c.ctas_per_row, c.threads, c.fell_back)

    assert choice(1024, B.BF16) == (B.KERNEL_TILE, 1, 512, 0)            # dense rows of up to 16 KB
    assert choice(2048, B.F32) == (B.KERNEL_TILE, 1, 512, 0)
    assert choice(8192, B.BF16) == (B.KERNEL_TILE, 1, 512, 0)
    assert choice(16384, B.BF16) == (B.KERNEL_SHARED, 1, 256, 0)
    assert choice(1020, B.BF16) == (B.KERNEL_WARP, 1, 32, 0)             # a ragged tail of 4 elements
    assert choice(4092, B.BF16) == (B.KERNEL_WARP, 1, 32, 0)
    assert choice(8200, B.BF16) == (B.KERNEL_SHARED, 1, 128, 0)          # 16,400 B: one row would leave half a stage empty
    assert choice(12288, B.BF16) == (B.KERNEL_SHARED, 1, 128, 0)
    assert choice(16392, B.BF16) == (B.KERNEL_SHARED, 1, 256, 0)
    assert choice(32768, B.BF16) == (B.KERNEL_SHARED, 2, 256, 0)
    fwd_short = B.grpo_loss_kernel_choice(B.LossParams(64, 1024, B.BF16, 1024, 4, 0, 0.2, 0.2, 0.04, 1.0), forward_only=True)
    assert fwd_short.kernel == B.KERNEL_TILE                             # forward only as well
    assert choice(151936, B.BF16) == (B.KERNEL_SHARED, 4, 256, 0)        # the benchmark's rows
    assert choice(151936, B.F32) == (B.KERNEL_SHARED, 8, 256, 0)
    assert choice(400000, B.BF16) == (B.KERNEL_GENERAL, 1, 512, 0)       # too long for eight slices: not a fall-back
    prm = B.LossParams(64, 151936, B.BF16, 151936, 4, 0, 0.2, 0.2, 0.04, 1.0)
    fwd = B.grpo_loss_kernel_choice(prm, forward_only=True)                # long rows, no dlogits: streamed
    assert (fwd.kernel, fwd.fell_back) == (B.KERNEL_STREAM, 0)
    prm = B.LossParams(64, 32768, B.BF16, 32768, 4, 0, 0.2, 0.2, 0.04, 1.0)
    assert B.grpo_loss_kernel_choice(prm, forward_only=True).kernel == B.KERNEL_SHARED   # 64 KB rows stay
    assert choice(151936, B.BF16, variant=1)[0] == B.KERNEL_GENERAL
    assert choice(151936, B.BF16, variant=80128) == (B.KERNEL_SHARED, 8, 128, 0)
    with pytest.raises(B.DppoError) as e:
        choice(151936, B.F32, variant=10256)                              # one CTA cannot hold 594 KB
    assert e.value.code == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype,V,variant,forward_only", [
    ("bf16", 1024, 1, False), ("bf16", 1016, 2, False), ("bf16", 1024, 4, False), ("f32", 4096, 4, False), ("bf16", 1024, 4, True),
    ("bf16", 16384, 10256, False), ("bf16", 65536, 0, False), ("bf16", 151936, 3, True)])
def test_loss_rows_that_no_sequence_covers(dtype, V, variant, forward_only):
    """cu_seqlens that ends before the token count (a caller's mistake): the rows past its last entry belong to no
    sequence.  Every kernel reports DPPO_STATUS_BAD_SEGMENTS, leaves those rows as rows that add nothing (dlogits and
    logp_out of zero) and gives the covered rows exactly what a call on the covered rows alone gives."""
    from paper_2603_04135_b200 import binding as B
    T, covered, S = 45, 29, 3
    per16 = 8 if dtype == "bf16" else 4
    stride = -(-V // per16) * per16
    w = synth.scaled(synth.WORKLOADS["config0"], V=stride, dtype=dtype)
    tok = synth.make_token_inputs(w, T, 700, device="cuda")
    tok.target.clamp_(max=V - 1)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    rng = np.random.default_rng(700)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.from_numpy((rng.random(S) * 0.1).astype(np.float32)).cuda()
    cu = torch.tensor([0, 10, 17, covered], dtype=torch.int32, device="cuda")

    def call(T_call):
        prm = B.LossParams(T_call, V, B.BF16 if dtype == "bf16" else B.F32, stride, S, variant, 0.2, 0.2, 0.04, 1.0)
        nbytes = B.grpo_loss_workspace_bytes(prm)
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        dl = None if forward_only else torch.full((T, stride), 7.0, dtype=tdt, device="cuda")
        loss_out = torch.full((5,), 7.0, device="cuda")
        logp_out = torch.full((T,), 7.0, device="cuda"); lse_out = torch.full((T,), 7.0, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, wseq, None, dl,
                            logp_out, lse_out, loss_out, ws, nbytes, status)
        torch.cuda.synchronize()
        return dl, logp_out, lse_out, loss_out, int(status.item())

    dl, logp_out, lse_out, loss_out, status = call(T)
    ref_dl, ref_logp, ref_lse, ref_loss, ref_status = call(covered)
    assert ref_status == 0 and status == B.STATUS_BAD_SEGMENTS
    assert bool((logp_out[covered:] == 0).all()) and bool(torch.isfinite(lse_out).all())
    assert torch.equal(logp_out[:covered], ref_logp[:covered]) and torch.equal(lse_out[:covered], ref_lse[:covered])
    assert torch.equal(loss_out[:4], ref_loss[:4]) and float(loss_out[4]) == T and float(ref_loss[4]) == covered
    if not forward_only:
        assert bool((dl[covered:, :V] == 0).all())
        assert torch.equal(dl[:covered].view(torch.int16 if dtype == "bf16" else torch.int32),
                           ref_dl[:covered].view(torch.int16 if dtype == "bf16" else torch.int32))


def test_loss_bad_target_and_empty():
    from paper_2603_04135_b200 import binding as B
    V, T = 512, 8
    w = synth.scaled(synth.WORKLOADS["config0"], V=V)
    tok = synth.make_token_inputs(w, T, 0, device="cuda")
    tok.target[3] = V                                                 # outside the vocabulary
    cu = torch.tensor([0, T], dtype=torch.int32, device="cuda")
    adv = torch.ones(1, device="cuda"); ws_ = torch.ones(1, device="cuda")
    prm = B.LossParams(T, V, B.F32, V, 1, 0, 0.2, 0.2, 0.04, 1.0)
    nbytes = B.grpo_loss_workspace_bytes(prm)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    dl = torch.full((T, V), 7.0, device="cuda"); loss_out = torch.zeros(5, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, ws_, None, dl, None,
                        None, loss_out, ws, nbytes, status)
    assert status.item() == B.STATUS_BAD_TARGET
    assert (dl[3] == 0).all() and (dl[2] != 7.0).all() and torch.isfinite(loss_out).all()
    # T_max = 0: only the reduction runs
    prm0 = B.LossParams(0, V, B.F32, V, 0, 0, 0.2, 0.2, 0.04, 1.0)
    B.grpo_loss_fwd_bwd(prm0, None, None, None, None, None, None, None, None, None, None, None, None, loss_out, ws,
                        nbytes, None)
    assert (loss_out.cpu().numpy() == 0).all()
    # host-side validation
    for bad, code in [(B.LossParams(T, V, 7, V, 1, 0, 0.2, 0.2, 0.04, 1.0), B.ERR_UNSUPPORTED),
                      (B.LossParams(T, V, B.F32, V - 1, 1, 0, 0.2, 0.2, 0.04, 1.0), B.ERR_BAD_SHAPE),
                      (B.LossParams(T, V, B.F32, V + 1, 1, 0, 0.2, 0.2, 0.04, 1.0), B.ERR_MISALIGNED),
                      (B.LossParams(T, V, B.F32, V, 1, 0, 0.2, 0.2, 0.04, 0.0), B.ERR_INVALID_ARG)]:
        with pytest.raises(B.DppoError) as e:
            B.grpo_loss_fwd_bwd(bad, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, ws_, None, dl,
                                None, None, loss_out, ws, nbytes, status)
        assert e.value.code == code
    with pytest.raises(B.DppoError) as e:
        B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, ws_, None, dl, None,
                            None, loss_out, ws, 16, status)
    assert e.value.code == B.ERR_WORKSPACE_TOO_SMALL


# ------------------------------------------------------------------------------------------- whole path
def _run_config(w, seed, n_sample_rows, all_rows, use_history=True, in_place=False):
    batch = synth.make_batch(w, seed)
    ref = oracle_prune_pack(batch, w, seed, step=1, use_history=use_history)
    pk = ref["pack"]
    T = pk["counts"][3]
    st = _step(w, T)
    st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
    st.prune_pack(seed=seed, step=1)
    assert_prune_equal(st.prune_results(), ref)
    assert_pack_equal(st.pack_results(), pk, w.P * w.G)
    assert st.n_tokens() == T
    tok = synth.make_token_inputs(w, T, seed, device="cuda")
    dl = tok.logits.clone() if in_place else torch.empty_like(tok.logits)
    st.loss(dl if in_place else tok.logits, tok.target, tok.logp_old, tok.logp_ref, dl)
    torch.cuda.synchronize()
    assert st.status.item() == 0

    order = np.asarray(pk["order"], dtype=np.int64)
    adv_seg = ref["adv"].reshape(-1)[order]; w_seg = ref["prune"]["w_seq"].reshape(-1)[order]
    cu = np.asarray(pk["cu_seqlens"])
    target = tok.target.cpu().numpy(); lo = tok.logp_old.cpu().numpy(); lr = tok.logp_ref.cpu().numpy()
    # element-wise dlogits on the first and last token of every sequence plus random rows, a block at a time (a
    # block of float64 rows of the full vocabulary is already a few hundred MB on the host)
    rows_all = pick_rows(cu, T, n_sample_rows, seed)
    tol = LOGP_TOL[w.dtype]
    logp_got = st.logp_out.cpu().numpy(); lse_got = st.lse_out.cpu().numpy()
    n_stable = 0
    for a in range(0, len(rows_all), 256):
        rows = rows_all[a:a + 256]
        sub = oracle.grpo_loss(rows_to_f64(tok.logits, rows), target, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta,
                               rows=rows, chunk=64)
        stable = clip_decision_is_stable(sub["rho"], w.eps, w.eps)
        n_stable += int(stable.sum())
        assert_dlogits_close(rows_to_f64(dl, rows), sub, w.dtype, w.beta, rows_ok=stable)
        assert np.abs(logp_got[rows] - sub["logp"]).max() <= tol
        assert np.abs(lse_got[rows] - sub["lse"]).max() <= tol
    assert n_stable > 0.99 * len(rows_all)
    out = st.loss_out.cpu().numpy().astype(np.float64)
    assert out[4] == T
    if all_rows:
        full = oracle_forward_all_rows(tok.logits, target, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta,
                                       processes=0 if all_rows == "inline" else None)
        assert np.abs(st.logp_out.cpu().numpy()[:T] - full["logp"]).max() <= tol
        assert abs(out[0] - full["loss"]) <= 1e-4 * abs(full["loss"]), (out[0], full["loss"], full["abs_sum"])
        assert abs(out[0] - full["loss"]) <= 1e-4 * full["abs_sum"]
        assert abs(out[1] - full["pg"]) <= 1e-4 * full["abs_sum"]
        assert abs(out[2] - full["kl"]) <= 1e-4 * full["kl"] + 1e-9
        assert abs(out[3] - full["clip_frac"]) <= 2.0 / max(T, 1)
    return T


@pytest.mark.parametrize("history", [True, False])
def test_config0_whole_path(history):
    for seed in (0, 1, 2):
        _run_config(synth.WORKLOADS["config0"], seed, 64, all_rows="inline", use_history=history)


def test_config0_in_place():
    _run_config(synth.WORKLOADS["config0"], 0, 64, all_rows="inline", in_place=True)


def test_config1_whole_path():
    T = _run_config(synth.WORKLOADS["config1"], 1, 4096, all_rows="pool")
    assert T > 10000


def test_config3_full_size():
    # the benchmark's launch configuration: in place, full vocabulary, every retained token.  dlogits element-wise
    # on more than 4,096 sampled rows (segment boundaries + random); log-probs, lse and the loss sums against the
    # oracle over ALL rows
    free, _ = torch.cuda.mem_get_info()
    if free < 90e9:
        pytest.skip("needs ~70 GB of free device memory")
    T = _run_config(synth.WORKLOADS["config3"], 3, 4096, all_rows="pool", in_place=True)
    assert T > 60000


@pytest.mark.parametrize("dtype,V,T", [("bf16", 1024, 1000000), ("f32", 2048, 250000)])
def test_short_rows_at_the_timed_size(dtype, V, T):
    """The short-row cases the benchmark line times (`loss_sweep_other_row_lengths`), in the call form it uses: the
    library's own kernel choice (the tile kernel), device-side token count, sequence map, log-prob and lse outputs,
    2,000 sequences.  dlogits element-wise on the first and last row of every sequence plus random rows; log-probs,
    lse and the loss sums against the oracle over ALL rows."""
    from paper_2603_04135_b200 import binding as B
    S, seed = 2000, 800
    w = synth.scaled(synth.WORKLOADS["config3"], V=V, dtype=dtype)
    tok = synth.make_token_inputs(w, T, seed, device="cuda")
    rng = np.random.default_rng(seed)
    cu = np.linspace(0, T, S + 1).astype(np.int32)
    adv = rng.normal(size=S).astype(np.float32)
    wseq = np.full(S, 1.0 / S, dtype=np.float32)
    seg_map = rng.permutation(S).astype(np.int32)
    prm = B.LossParams(T, V, B.BF16 if dtype == "bf16" else B.F32, V, S, 0, w.eps, w.eps, w.beta, 1.0)
    assert B.grpo_loss_kernel_choice(prm).kernel == B.KERNEL_TILE
    nbytes = B.grpo_loss_workspace_bytes(prm)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    dl = torch.empty_like(tok.logits)
    loss_out = torch.zeros(5, device="cuda"); status = torch.zeros(1, dtype=torch.int32, device="cuda")
    logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
    ntd = torch.tensor([T], dtype=torch.int32, device="cuda")
    B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, torch.from_numpy(cu).cuda(), ntd,
                        torch.from_numpy(adv).cuda(), torch.from_numpy(wseq).cuda(), torch.from_numpy(seg_map).cuda(), dl,
                        logp_out, lse_out, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    adv_seg, w_seg = adv[seg_map], wseq[seg_map]
    target = tok.target.cpu().numpy(); lo = tok.logp_old.cpu().numpy(); lr = tok.logp_ref.cpu().numpy()
    tol = LOGP_TOL[dtype]
    logp_got = logp_out.cpu().numpy(); lse_got = lse_out.cpu().numpy()
    rows_all = pick_rows(cu, T, 1024, seed)
    n_stable = 0
    for a in range(0, len(rows_all), 1024):
        rows = rows_all[a:a + 1024]
        sub = oracle.grpo_loss(rows_to_f64(tok.logits, rows), target, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta,
                               rows=rows, chunk=256)
        stable = clip_decision_is_stable(sub["rho"], w.eps, w.eps)
        n_stable += int(stable.sum())
        assert_dlogits_close(rows_to_f64(dl, rows), sub, dtype, w.beta, rows_ok=stable)
        assert np.abs(logp_got[rows] - sub["logp"]).max() <= tol
        assert np.abs(lse_got[rows] - sub["lse"]).max() <= tol
    assert len(rows_all) > 4096 and n_stable > 0.99 * len(rows_all)
    full = oracle_forward_all_rows(tok.logits, target, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta, rows_per_task=16384)
    out = loss_out.cpu().numpy().astype(np.float64)
    assert out[4] == T
    assert np.abs(logp_got - full["logp"]).max() <= tol and np.abs(lse_got - full["lse"]).max() <= tol
    assert abs(out[0] - full["loss"]) <= 1e-4 * abs(full["loss"]) + 1e-7 * full["abs_sum"]
    assert abs(out[1] - full["pg"]) <= 1e-4 * full["abs_sum"]
    assert abs(out[2] - full["kl"]) <= 1e-4 * full["kl"] + 1e-9
    # a row whose ratio sits within the margin of a clip bound may take the other branch in f32 (same loss there)
    unstable = int((~clip_decision_is_stable(full["rho"], w.eps, w.eps)).sum())
    assert abs(out[3] - full["clip_frac"]) <= (unstable + 2.0) / T


def test_rows_sharded_over_two_ranks_add_up():
    # Rows dealt out to two ranks (dp.shard_rows), each rank's sweep run here one after the other on the one device:
    # every rank uses the sequence weights of the WHOLE batch, so the five scalars add up to the whole batch's and each
    # rank's dlogits are the whole batch's rows, bit for bit
    w = synth.scaled(synth.WORKLOADS["config0"], P=8, G=4, V=2056, L_row=192, r_q=0.3, r_o=0.3)
    seed = 9
    batch = synth.make_batch(w, seed)
    ref = oracle_prune_pack(batch, w, seed, step=1)
    T = ref["pack"]["counts"][3]
    st = _step(w, T)
    st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
    st.prune_pack(seed=seed, step=1)
    assert st.n_tokens() == T and ref["pack"]["counts"][1] >= 4
    tok = synth.make_token_inputs(w, T, seed, device="cuda", sigma_old=0.3)
    dl = torch.empty_like(tok.logits)
    st.loss(tok.logits, tok.target, tok.logp_old, tok.logp_ref, dl)
    whole = st.loss_out.double().cpu().numpy()
    order = np.asarray(ref["pack"]["order"], dtype=np.int64)
    full = oracle.grpo_loss(synth.to_f64_numpy(tok.logits), tok.target.cpu().numpy(), tok.logp_old.cpu().numpy(),
                            tok.logp_ref.cpu().numpy(), ref["pack"]["cu_seqlens"], ref["adv"].reshape(-1)[order],
                            ref["prune"]["w_seq"].reshape(-1)[order], w.eps, w.eps, w.beta, want_dlogits=False)
    assert abs(whole[0] - full["loss"]) <= 1e-4 * abs(full["loss"]) + 1e-7 * full["abs_sum"]
    parts = []
    covered = 0
    for rank in range(2):
        sh = st.shard(2, rank)
        a, b = sh["tok_lo"], sh["tok_hi"]
        assert a == covered and b > a
        covered = b
        dl_r = torch.full((b - a, w.V), 7.0, device="cuda")
        st.loss_shard(sh, tok.logits[a:b], tok.target[a:b], tok.logp_old[a:b], tok.logp_ref[a:b], dl_r)
        torch.cuda.synchronize()
        assert st.status.item() == 0
        parts.append(st.loss_out.double().cpu().numpy())
        assert torch.equal(dl_r.view(torch.int32), dl[a:b].view(torch.int32))
    assert covered == T
    total = parts[0][:3] + parts[1][:3]
    for k in range(3):
        assert abs(total[k] - whole[k]) <= 1e-6 * max(abs(whole[k]), 1e-6)
    assert parts[0][4] + parts[1][4] == T == whole[4]
    assert abs((parts[0][3] * parts[0][4] + parts[1][3] * parts[1][4]) / T - whole[3]) <= 1e-6
