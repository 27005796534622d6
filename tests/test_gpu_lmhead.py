"""Fused LM-head + loss (tcgen05 / TMEM) against the float64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_04135_b200 import synth
from parity_util import Guarded

pytestmark = pytest.mark.gpu


# Element-wise bounds on the two gradients, relative to the largest entry of the same output row.  Both are sums of
# products with bf16-rounded factors (unit roundoff 2^-9) accumulated in f32:
#   dhidden[t,:] = -f_t * sum_v E'[t,v] W[v,:]    one rounded factor per product (the stored exponential), the row
#                                                 factor applied to the f32 sum, the result stored as bf16
#   dW[v,:]      = sum_t E'[t,v] * (-f_t h[t,:])  two rounded factors per product (the exponential and the pre-scaled
#                                                 hidden entry), so up to twice the relative error per term
DH_TOL = 2.0 ** -7
DW_TOL = 2.0 ** -6


def assert_loss_close(got, ref):
    """The stated bound on the loss: 1e-4 relative to |loss|, plus the floor 1e-7 * sum_t |W_t j_t| that the other
    loss tests use (positive and negative advantages cancel in the sum, the rounding of its terms does not)."""
    assert abs(got - ref["loss"]) <= 1e-4 * abs(ref["loss"]) + 1e-7 * ref["abs_sum"], (got, ref["loss"], ref["abs_sum"])


def _run(T, V, H, S, seed, n_tokens=None, tau=1.0, backward=False, variant=0, dW_bf16=False):
    from paper_2603_04135_b200 import binding as B
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=V, H=H)
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device="cuda")
    rng = np.random.default_rng(seed)
    T_true = T if n_tokens is None else n_tokens
    cuts = np.sort(rng.choice(np.arange(1, T_true), size=min(S - 1, T_true - 1), replace=False))
    cu = np.concatenate([[0], cuts, [T_true]]).astype(np.int32)
    S_real = len(cu) - 1
    adv = rng.normal(size=S_real).astype(np.float32); wseq = (rng.random(S_real) * 0.1).astype(np.float32)
    prm = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S_real, 0, w.eps, w.eps, w.beta, tau), H, int(backward), variant, B.BF16 if dW_bf16 else B.F32)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 1024:]
    # every output sits between guard bands of sentinels (an overrun past either end fails the test)
    g_dh = Guarded((T, H), torch.bfloat16, 7.0) if backward else None
    g_dW = Guarded((V, H), torch.bfloat16 if dW_bf16 else torch.float32, 7.0) if backward else None
    g_loss = Guarded((5,), torch.float32, 0.0); g_logp = Guarded((T,), torch.float32, 0.0); g_lse = Guarded((T,), torch.float32, 0.0)
    dh = g_dh.t if backward else None
    dW = g_dW.t if backward else None
    loss_out, logp_out, lse_out = g_loss.t, g_logp.t, g_lse.t
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ntd = torch.tensor([T_true], dtype=torch.int32, device="cuda") if n_tokens is not None else None
    B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, torch.from_numpy(cu).cuda(), ntd, torch.from_numpy(adv).cuda(),
                       torch.from_numpy(wseq).cuda(), None, dh, dW, logp_out, lse_out, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for g in (g_dh, g_dW, g_loss, g_logp, g_lse):
        if g is not None:
            g.check()
    if backward:
        ref = oracle.lmhead_grpo_loss(synth.to_f64_numpy(hidden[:T_true]), synth.to_f64_numpy(W), target.cpu().numpy(),
                                      lo.cpu().numpy(), lr.cpu().numpy(), cu, adv, wseq, w.eps, w.eps, w.beta, tau)
    else:
        ref = oracle.grpo_loss(synth.to_f64_numpy(hidden[:T_true]) @ synth.to_f64_numpy(W).T, target.cpu().numpy(),
                               lo.cpu().numpy(), lr.cpu().numpy(), cu, adv, wseq, w.eps, w.eps, w.beta, tau,
                               want_dlogits=False)
    got = loss_out.cpu().numpy().astype(np.float64)
    # logits are f32 accumulations of exact bf16 products over H terms; the row sum runs in f32
    assert np.abs(lse_out.cpu().numpy()[:T_true] - ref["lse"]).max() <= 1e-4
    assert np.abs(logp_out.cpu().numpy()[:T_true] - ref["logp"]).max() <= 1e-4
    assert_loss_close(got[0], ref)
    assert abs(got[1] - ref["pg"]) <= 1e-4 * ref["abs_sum"] and abs(got[2] - ref["kl"]) <= 1e-4 * ref["kl"] + 1e-9
    assert got[4] == T_true
    if backward:
        gmax = np.abs(ref["g"]).max()
        got_dh = dh.double().cpu().numpy()
        assert (got_dh[T_true:] == 0).all()
        err = np.abs(got_dh[:T_true] - ref["dhidden"])
        bound = DH_TOL * np.abs(ref["dhidden"]).max(axis=1, keepdims=True) + 1e-6 * gmax
        assert (err <= bound).all(), "dhidden worst ratio %.3g" % (err / bound).max()
        got_dW = dW.double().cpu().numpy()
        err = np.abs(got_dW - ref["dW"])
        bound = DW_TOL * np.abs(ref["dW"]).max(axis=1, keepdims=True) + 1e-6 * gmax
        if dW_bf16:
            bound = bound + 2.0 ** -8 * np.abs(ref["dW"])            # one more rounding, of the f32 sum to bf16
        assert (err <= bound).all(), "dW worst ratio %.3g" % (err / bound).max()
    return ref


@pytest.mark.parametrize("variant", [1, 0])           # single-CTA core, CTA-pair core
def test_lmhead_small_shapes(variant):
    _run(T=200, V=1000, H=128, S=4, seed=1, variant=variant)     # ragged token tile, ragged vocabulary tile
    _run(T=128, V=256, H=64, S=1, seed=2, variant=variant)       # exactly one tile, one K slab
    _run(T=130, V=4096, H=4096, S=3, seed=3, variant=variant)    # the wider hidden size
    _run(T=300, V=777, H=192, S=5, seed=4, n_tokens=259, tau=1.3, variant=variant)
    _run(T=700, V=300, H=512, S=2, seed=6, variant=variant)      # several token tiles, an odd number of them


@pytest.mark.parametrize("variant", [1, 0])
def test_lmhead_edge_shapes(variant):
    # one token, one vocabulary entry, one more than a tile in each direction, fewer tokens than a tile
    for kw in [dict(T=1, V=8, H=64, S=1, seed=61), dict(T=5, V=300, H=64, S=2, seed=62), dict(T=2, V=1, H=64, S=1, seed=63),
               dict(T=129, V=257, H=128, S=3, seed=64), dict(T=64, V=65, H=64, S=2, seed=65)]:
        _run(backward=False, variant=variant, **kw)
        _run(backward=True, variant=variant, **kw)


@pytest.mark.parametrize("variant", [1, 0])
def test_lmhead_full_vocabulary(variant):
    _run(T=300, V=151936, H=2560, S=4, seed=5, variant=variant)


@pytest.mark.parametrize("variant", [1, 0])
def test_lmhead_backward_small_shapes(variant):
    _run(T=200, V=1000, H=128, S=4, seed=11, backward=True, variant=variant)
    _run(T=128, V=256, H=64, S=1, seed=12, backward=True, variant=variant)
    _run(T=300, V=777, H=192, S=5, seed=14, n_tokens=259, tau=1.3, backward=True, variant=variant)
    _run(T=130, V=2048, H=2560, S=3, seed=13, backward=True, variant=variant)


@pytest.mark.parametrize("variant", [1, 0])
def test_lmhead_backward_several_token_chunks(variant):
    _run(T=9472 + 9472 + 70, V=520, H=64, S=9, seed=15, backward=True, variant=variant)   # three chunks, the last ragged


def test_lmhead_backward_bf16_dW():
    _run(T=300, V=777, H=192, S=5, seed=21, n_tokens=259, backward=True, dW_bf16=True)
    _run(T=9472 + 200, V=520, H=64, S=3, seed=22, backward=True, dW_bf16=True)   # summed over two chunks in f32, rounded once


@pytest.mark.parametrize("dW_bf16", [False, True])
def test_lmhead_accumulate_dW(dW_bf16):
    """accumulate_dW = 1 adds the gradient to what dW holds: a second call on the first call's result gives twice
    the oracle's dW (dhidden is overwritten both times)."""
    from paper_2603_04135_b200 import binding as B
    T, V, H, S, seed = 9472 + 300, 520, 64, 4, 41
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=V, H=H)
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device="cuda")
    rng = np.random.default_rng(seed)
    cu = np.concatenate([[0], np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False)), [T]]).astype(np.int32)
    adv = rng.normal(size=S).astype(np.float32); wseq = (rng.random(S) * 0.1).astype(np.float32)
    dh = torch.zeros((T, H), dtype=torch.bfloat16, device="cuda")
    dW = torch.full((V, H), 7.0, dtype=torch.bfloat16 if dW_bf16 else torch.float32, device="cuda")
    loss_out = torch.zeros(5, device="cuda"); status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for acc in (0, 1):
        prm = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S, 0, w.eps, w.eps, w.beta, 1.0), H, 1, 0,
                             B.BF16 if dW_bf16 else B.F32, acc)
        nbytes = B.lmhead_workspace_bytes(prm)
        ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda"); ws = ws[(-ws.data_ptr()) % 1024:]
        B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, torch.from_numpy(cu).cuda(), None, torch.from_numpy(adv).cuda(),
                           torch.from_numpy(wseq).cuda(), None, dh, dW, None, None, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    ref = oracle.lmhead_grpo_loss(synth.to_f64_numpy(hidden), synth.to_f64_numpy(W), target.cpu().numpy(), lo.cpu().numpy(),
                                  lr.cpu().numpy(), cu, adv, wseq, w.eps, w.eps, w.beta, 1.0)
    want = 2.0 * ref["dW"]
    bound = 2.0 * (DW_TOL * np.abs(ref["dW"]).max(axis=1, keepdims=True) + 1e-6 * np.abs(ref["g"]).max())
    if dW_bf16:
        bound = bound + 2.0 ** -7 * np.abs(want)                 # the intermediate and the final rounding to bf16
    err = np.abs(dW.double().cpu().numpy() - want)
    assert (err <= bound).all(), "dW worst ratio %.3g" % (err / bound).max()


@pytest.mark.parametrize("H", [2560, 4096])
def test_config4_whole_path(H):
    """The fused LM-head configuration end to end at a size the oracle finishes: advantages -> pruning with
    probabilities 0.5 / 0.5 -> packing -> fused LM-head + loss driven by the packer's cu_seqlens, placement order
    and device-side token count, over the full vocabulary and both hidden widths, forward and backward."""
    from paper_2603_04135_b200 import binding as B
    from paper_2603_04135_b200.step import DppoStep
    from parity_util import oracle_prune_pack, assert_prune_equal, assert_pack_equal
    V = 151936 if H == 2560 else 32768                      # the oracle's float64 dW is V x H: keep the wider case small
    w = synth.scaled(synth.WORKLOADS["config4_h%d" % H], P=4, G=8, resp_len=("uniform", 4, 24), L_row=128, N_win=4, V=V)
    seed = 4
    batch = synth.make_batch(w, seed)
    ref = oracle_prune_pack(batch, w, seed, step=2)
    pk = ref["pack"]
    T = pk["counts"][3]
    assert 60 <= T <= 500
    T_cap = int(batch.loss_len.sum())                        # buffers sized for the unpruned batch
    st = DppoStep(w.P, w.G, w.L_row, w.N_win, w.r_q, w.r_o, w.V, w.dtype, T_cap, w.eps, w.eps, w.beta)
    st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, ref["H_prev"])
    st.prune_pack(seed=seed, step=2)
    assert_prune_equal(st.prune_results(), ref)
    assert_pack_equal(st.pack_results(), pk, w.P * w.G)

    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T_cap, seed, device="cuda")
    prm = B.LmheadParams(B.LossParams(T_cap, w.V, B.BF16, w.V, w.P * w.G, 0, w.eps, w.eps, w.beta, 1.0), H, 1, 0, B.F32)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda"); ws = ws[(-ws.data_ptr()) % 1024:]
    dh = torch.full((T_cap, H), 7.0, dtype=torch.bfloat16, device="cuda")
    dW = torch.full((w.V, H), 7.0, dtype=torch.float32, device="cuda")
    B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, st.cu_seqlens, st.counts[3:4], st.adv, st.w_seq, st.order,
                       dh, dW, st.logp_out, st.lse_out, st.loss_out, ws, nbytes, st.status)
    torch.cuda.synchronize()
    assert st.status.item() == 0

    order = np.asarray(pk["order"], dtype=np.int64)
    want = oracle.lmhead_grpo_loss(synth.to_f64_numpy(hidden[:T]), synth.to_f64_numpy(W), target.cpu().numpy()[:T],
                                   lo.cpu().numpy()[:T], lr.cpu().numpy()[:T], np.asarray(pk["cu_seqlens"]),
                                   ref["adv"].reshape(-1)[order], ref["prune"]["w_seq"].reshape(-1)[order],
                                   w.eps, w.eps, w.beta, 1.0)
    got = st.loss_out.cpu().numpy().astype(np.float64)
    assert got[4] == T
    assert np.abs(st.lse_out.cpu().numpy()[:T] - want["lse"]).max() <= 1e-4
    assert np.abs(st.logp_out.cpu().numpy()[:T] - want["logp"]).max() <= 1e-4
    assert_loss_close(got[0], want)
    gmax = np.abs(want["g"]).max()
    got_dh = dh.double().cpu().numpy()
    assert (got_dh[T:] == 0).all()                           # rows beyond the retained tokens are cleared
    err = np.abs(got_dh[:T] - want["dhidden"])
    bound = DH_TOL * np.abs(want["dhidden"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dhidden worst ratio %.3g" % (err / bound).max()
    err = np.abs(dW.double().cpu().numpy() - want["dW"])
    bound = DW_TOL * np.abs(want["dW"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dW worst ratio %.3g" % (err / bound).max()


@pytest.mark.parametrize("mode", ["no_length_norm", "seq_ratio"])
def test_lmhead_loss_variants(mode):
    """The objectives of Section 5.2 through the fused path: weights without the 1/|o| factor, and the
    sequence-level ratio (a forward-only call gives the current log-probs, their per-sequence mean log-ratio goes
    back in for the call with gradients)."""
    from paper_2603_04135_b200 import binding as B
    T, V, H, S, seed = 300, 1000, 128, 5, 51
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=V, H=H, sigma_old=0.3)
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device="cuda")
    rng = np.random.default_rng(seed)
    cu = np.concatenate([[0], np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False)), [T]]).astype(np.int32)
    adv = rng.normal(size=S).astype(np.float32); wseq = (rng.random(S) * 0.1).astype(np.float32)
    d_cu = torch.from_numpy(cu).cuda(); d_adv = torch.from_numpy(adv).cuda(); d_w = torch.from_numpy(wseq).cuda()
    loss_out = torch.zeros(5, device="cuda"); logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fwd = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S, 0, w.eps, w.eps, w.beta, 1.0), H, 0)
    bwd = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S, 0, w.eps, w.eps, w.beta, 1.0), H, 1, 0, B.F32)
    nbytes = max(B.lmhead_workspace_bytes(fwd), B.lmhead_workspace_bytes(bwd))
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda"); ws = ws[(-ws.data_ptr()) % 1024:]
    slr = None
    if mode == "seq_ratio":
        B.lmhead_grpo_loss(fwd, hidden, W, target, lo, lr, d_cu, None, d_adv, d_w, None, None, None, logp_out, None, loss_out,
                           ws, nbytes, status)
        slr_dev = torch.zeros(S, device="cuda")
        B.sequence_log_ratio(logp_out, lo, d_cu, S, slr_dev)
        bwd.loss.seq_log_ratio = slr_dev.data_ptr()
        z = synth.to_f64_numpy(hidden) @ synth.to_f64_numpy(W).T
        slr = oracle.sequence_log_ratio(oracle.token_logprob(z, target.cpu().numpy())[0], lo.cpu().numpy(), cu)
        assert np.abs(slr_dev.cpu().numpy() - slr).max() <= 1e-4
    else:
        bwd.loss.no_length_norm = 1
    dh = torch.zeros((T, H), dtype=torch.bfloat16, device="cuda"); dW = torch.zeros((V, H), device="cuda")
    B.lmhead_grpo_loss(bwd, hidden, W, target, lo, lr, d_cu, None, d_adv, d_w, None, dh, dW, logp_out, lse_out, loss_out,
                       ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    ref = oracle.lmhead_grpo_loss(synth.to_f64_numpy(hidden), synth.to_f64_numpy(W), target.cpu().numpy(), lo.cpu().numpy(),
                                  lr.cpu().numpy(), cu, adv, wseq, w.eps, w.eps, w.beta, 1.0,
                                  length_norm=(mode != "no_length_norm"), seq_log_ratio=slr)
    got = loss_out.cpu().numpy().astype(np.float64)
    assert_loss_close(got[0], ref)
    gmax = np.abs(ref["g"]).max()
    err = np.abs(dh.double().cpu().numpy() - ref["dhidden"])
    bound = DH_TOL * np.abs(ref["dhidden"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dhidden worst ratio %.3g" % (err / bound).max()
    err = np.abs(dW.double().cpu().numpy() - ref["dW"])
    bound = DW_TOL * np.abs(ref["dW"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dW worst ratio %.3g" % (err / bound).max()


def test_lmhead_full_size_sampled_tokens():
    """The size the benchmark times (99,030 tokens, V = 151,936, H = 2560, eleven token chunks, the last ragged):
    lse, logp and dhidden of sampled tokens against the oracle (each sampled token is given to the oracle as a
    sequence of its own carrying its sequence's advantage and w / |o|), the exact token count, zero rows of
    dhidden nowhere, and dW on sampled vocabulary rows for consistency with a float64 contraction of the
    library's own logp (not a parity claim: its input comes from the CUDA path)."""
    from paper_2603_04135_b200 import binding as B
    free, _ = torch.cuda.mem_get_info()
    if free < 20 << 30:
        pytest.skip("needs 20 GB of free device memory")
    w = synth.WORKLOADS["config4_h2560"]
    T, V, H, S, seed = 99030, w.V, w.H, 177, 31
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device="cuda")
    rng = np.random.default_rng(seed)
    cu = np.concatenate([[0], np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False)), [T]]).astype(np.int32)
    adv = rng.normal(size=S).astype(np.float32); wseq = (rng.random(S) * 0.1).astype(np.float32)
    prm = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S, 0, w.eps, w.eps, w.beta, 1.0), H, 1, 0, B.F32)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda"); ws = ws[(-ws.data_ptr()) % 1024:]
    dh = torch.full((T, H), 7.0, dtype=torch.bfloat16, device="cuda")
    dW = torch.full((V, H), 7.0, dtype=torch.float32, device="cuda")
    loss_out = torch.zeros(5, device="cuda"); logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, torch.from_numpy(cu).cuda(), None, torch.from_numpy(adv).cuda(),
                       torch.from_numpy(wseq).cuda(), None, dh, dW, logp_out, lse_out, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0 and loss_out[4].item() == T
    del ws
    # sampled tokens: around every chunk boundary, first / last of some sequences, and random ones
    edges = [t for c in range(0, T, 9472) for t in (c - 1, c, c + 127, c + 128) if 0 <= t < T]
    pick = np.unique(np.concatenate([edges, cu[:12], cu[1:13] - 1, [T - 1], rng.choice(T, size=64, replace=False)])).astype(np.int64)
    seg = np.searchsorted(cu, pick, side="right") - 1
    seg_len = (cu[seg + 1] - cu[seg]).astype(np.float64)
    idx = torch.from_numpy(pick).cuda()
    ref = oracle.lmhead_grpo_loss(synth.to_f64_numpy(hidden[idx]), synth.to_f64_numpy(W), target[idx].cpu().numpy(),
                                  lo[idx].cpu().numpy(), lr[idx].cpu().numpy(), np.arange(len(pick) + 1, dtype=np.int32),
                                  adv[seg].astype(np.float64), wseq[seg].astype(np.float64) / seg_len, w.eps, w.eps, w.beta, 1.0)
    assert np.abs(lse_out[idx].cpu().numpy() - ref["lse"]).max() <= 1e-4
    assert np.abs(logp_out[idx].cpu().numpy() - ref["logp"]).max() <= 1e-4
    gmax = np.abs(ref["g"]).max()
    err = np.abs(dh[idx].double().cpu().numpy() - ref["dhidden"])
    bound = DH_TOL * np.abs(ref["dhidden"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dhidden worst ratio %.3g" % (err / bound).max()
    assert bool((dh.float().abs().amax(dim=1) > 0).all())                      # every token got its gradient row
    # dW on sampled vocabulary rows: sum_t g_t (1[y_t = v] - exp(z_tv - lse_t)) h_t with g from the oracle's
    # token terms evaluated at the library's logp
    seg_all = np.searchsorted(cu, np.arange(T), side="right") - 1
    terms = oracle.token_terms(logp_out.cpu().numpy(), lo.cpu().numpy(), lr.cpu().numpy(), adv[seg_all], w.eps, w.eps, w.beta)
    Wt = wseq[seg_all].astype(np.float64) / (cu[seg_all + 1] - cu[seg_all])
    g = torch.from_numpy(-Wt * terms["dj"]).cuda()
    vs = torch.from_numpy(np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, V - 1], rng.choice(V, size=40, replace=False)]))).cuda()
    hd = hidden.double()
    z = hd @ W[vs].double().T                                                    # [T x |vs|]
    D = -g[:, None] * torch.exp(z - lse_out.double()[:, None])
    D += g[:, None] * (target.long()[:, None] == vs[None, :]).double()
    want = (D.T @ hd).cpu().numpy()
    got = dW[vs].double().cpu().numpy()
    bound = DW_TOL * np.abs(want).max(axis=1, keepdims=True) + 1e-6 * float(g.abs().max())
    assert (np.abs(got - want) <= bound).all(), "dW worst ratio %.3g" % (np.abs(got - want) / bound).max()


def test_lmhead_argument_checks():
    from paper_2603_04135_b200 import binding as B
    z = torch.zeros(8 * 256, dtype=torch.bfloat16, device="cuda")
    prm = B.LmheadParams(B.LossParams(8, 256, B.BF16, 256, 1, 0, 0.2, 0.2, 0.04, 1.0), 64, 0)
    with pytest.raises(B.DppoError) as e:       # gradients passed but not requested
        B.lmhead_grpo_loss(prm, z, z, z, z, z, z, None, z, z, None, z, z, None, None, z, z, 1 << 20)
    assert e.value.code == B.ERR_INVALID_ARG
    prm = B.LmheadParams(B.LossParams(8, 256, B.BF16, 256, 1, 0, 0.2, 0.2, 0.04, 1.0), 72, 0)
    with pytest.raises(B.DppoError) as e:       # H not a multiple of 64
        B.lmhead_grpo_loss(prm, z, z, z, z, z, z, None, z, z, None, None, None, None, None, z, z, 1 << 20)
    assert e.value.code == B.ERR_BAD_SHAPE


def test_lmhead_backward_out_of_range_row_is_reported():
    """The backward keeps the exponentials relative to the sampled token's own logit, in bf16.  A sampled token
    whose log-prob lies below about -66 cannot be represented that way (no sampler would have drawn it): the row
    is reported as DPPO_STATUS_RANGE, adds nothing and gets a zero gradient; every other row is unaffected.  The
    offending token forms a sequence of weight 0 here, so the oracle's result for the batch is the expected one."""
    from paper_2603_04135_b200 import binding as B
    T, V, H, seed = 150, 300, 64, 77
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=V, H=H)
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device="cuda")
    bad = 70
    hidden[bad] = 2.0                                           # z[v] = 2 * sum(W[v]): +128 for v = 5, -128 for the target
    W[5] = 1.0; W[9] = -1.0; target[bad] = 9
    cu = np.array([0, bad, bad + 1, T], dtype=np.int32)
    adv = np.array([0.7, 1.0, -0.4], dtype=np.float32); wseq = np.array([0.05, 0.0, 0.08], dtype=np.float32)
    prm = B.LmheadParams(B.LossParams(T, V, B.BF16, V, 3, 0, w.eps, w.eps, w.beta, 1.0), H, 1, 0, B.F32)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda"); ws = ws[(-ws.data_ptr()) % 1024:]
    dh = torch.full((T, H), 7.0, dtype=torch.bfloat16, device="cuda"); dW = torch.full((V, H), 7.0, device="cuda")
    loss_out = torch.zeros(5, device="cuda"); logp_out = torch.full((T,), 7.0, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, torch.from_numpy(cu).cuda(), None, torch.from_numpy(adv).cuda(),
                       torch.from_numpy(wseq).cuda(), None, dh, dW, logp_out, None, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == B.STATUS_RANGE
    assert bool((dh[bad] == 0).all()) and logp_out[bad].item() == 0.0
    assert bool(torch.isfinite(dW).all()) and bool(torch.isfinite(dh.float()).all()) and bool(torch.isfinite(loss_out).all())
    ref = oracle.lmhead_grpo_loss(synth.to_f64_numpy(hidden), synth.to_f64_numpy(W), target.cpu().numpy(), lo.cpu().numpy(),
                                  lr.cpu().numpy(), cu, adv, wseq, w.eps, w.eps, w.beta, 1.0)
    assert_loss_close(float(loss_out[0].item()), ref)
    gmax = np.abs(ref["g"]).max()
    err = np.abs(dh.double().cpu().numpy() - ref["dhidden"])
    bound = DH_TOL * np.abs(ref["dhidden"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dhidden worst ratio %.3g" % (err / bound).max()
    err = np.abs(dW.double().cpu().numpy() - ref["dW"])
    bound = DW_TOL * np.abs(ref["dW"]).max(axis=1, keepdims=True) + 1e-6 * gmax
    assert (err <= bound).all(), "dW worst ratio %.3g" % (err / bound).max()
