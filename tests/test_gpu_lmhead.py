"""Fused LM-head + loss (tcgen05 / TMEM) against the float64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_04135_b200 import synth

pytestmark = pytest.mark.gpu


def _run(T, V, H, S, seed, n_tokens=None, tau=1.0):
    from paper_2603_04135_b200 import binding as B
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=V, H=H)
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device="cuda")
    rng = np.random.default_rng(seed)
    T_true = T if n_tokens is None else n_tokens
    cuts = np.sort(rng.choice(np.arange(1, T_true), size=min(S - 1, T_true - 1), replace=False))
    cu = np.concatenate([[0], cuts, [T_true]]).astype(np.int32)
    S_real = len(cu) - 1
    adv = rng.normal(size=S_real).astype(np.float32); wseq = (rng.random(S_real) * 0.1).astype(np.float32)
    prm = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S_real, 0, w.eps, w.eps, w.beta, tau), H, 0)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    loss_out = torch.zeros(5, device="cuda"); logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ntd = torch.tensor([T_true], dtype=torch.int32, device="cuda") if n_tokens is not None else None
    B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, torch.from_numpy(cu).cuda(), ntd, torch.from_numpy(adv).cuda(),
                       torch.from_numpy(wseq).cuda(), None, None, None, logp_out, lse_out, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    ref = oracle.grpo_loss(synth.to_f64_numpy(hidden[:T_true]) @ synth.to_f64_numpy(W).T, target.cpu().numpy(),
                           lo.cpu().numpy(), lr.cpu().numpy(), cu, adv, wseq, w.eps, w.eps, w.beta, tau, want_dlogits=False)
    got = loss_out.cpu().numpy().astype(np.float64)
    # logits are f32 accumulations of exact bf16 products over H terms; the row sum runs in f32
    assert np.abs(lse_out.cpu().numpy()[:T_true] - ref["lse"]).max() <= 1e-4
    assert np.abs(logp_out.cpu().numpy()[:T_true] - ref["logp"]).max() <= 1e-4
    assert abs(got[0] - ref["loss"]) <= 1e-4 * ref["abs_sum"]
    assert abs(got[1] - ref["pg"]) <= 1e-4 * ref["abs_sum"] and abs(got[2] - ref["kl"]) <= 1e-4 * ref["kl"] + 1e-9
    assert got[4] == T_true
    return ref


def test_lmhead_small_shapes():
    _run(T=200, V=1000, H=128, S=4, seed=1)             # ragged token tile, ragged vocabulary tile
    _run(T=128, V=256, H=64, S=1, seed=2)               # exactly one tile, one K slab
    _run(T=130, V=4096, H=4096, S=3, seed=3)            # the wider hidden size
    _run(T=300, V=777, H=192, S=5, seed=4, n_tokens=259, tau=1.3)


def test_lmhead_full_vocabulary():
    _run(T=300, V=151936, H=2560, S=4, seed=5)


def test_lmhead_backward_not_built():
    from paper_2603_04135_b200 import binding as B
    prm = B.LmheadParams(B.LossParams(8, 256, B.BF16, 256, 1, 0, 0.2, 0.2, 0.04, 1.0), 64, 0)
    z = torch.zeros(8 * 256, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.DppoError) as e:
        B.lmhead_grpo_loss(prm, z, z, z, z, z, z, None, z, z, None, z, z, None, None, z, z, 1 << 20)
    assert e.value.code == B.ERR_UNSUPPORTED
