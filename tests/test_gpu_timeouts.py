"""The bounded device-side waits, made to run out on purpose (nothing hangs, nothing faults).

Every wait inside the kernels (on a bulk copy, on the other CTAs of a cluster, on a pipeline stage) gives up after
a limit, reports DPPO_STATUS_TIMEOUT through the status word and lets the kernel finish.  In normal operation that
path never runs.  The library's self-test variants make it run: a barrier is told to expect a few bytes more than
anybody sends and the limit is 1 ms, so every copy and every message still arrives in full, no thread waits for a
writer that is late, and every CTA takes the time-out exit on its own.  These tests check what that exit leaves
behind and that the next ordinary call on the same stream is unaffected.
"""
import numpy as np
import pytest
import torch

from paper_2603_04135_b200 import synth

pytestmark = pytest.mark.gpu


def _loss_call(B, prm, tok, cu, adv, wseq, T, stride, tdt):
    nbytes = B.grpo_loss_workspace_bytes(prm)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    dl = torch.full((T, stride), 7.0, dtype=tdt, device="cuda")
    loss_out = torch.full((5,), 7.0, device="cuda")
    logp_out = torch.full((T,), 7.0, device="cuda"); lse_out = torch.full((T,), 7.0, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, wseq, None, dl,
                        logp_out, lse_out, loss_out, ws, nbytes, status)
    torch.cuda.synchronize()
    return dl, loss_out, logp_out, lse_out, int(status.item())


@pytest.mark.parametrize("dtype,V,variant", [
    ("bf16", 151936, 0),          # the benchmark's shape: four CTAs per row
    ("bf16", 151936, 80128),      # eight CTAs
    ("bf16", 151936 - 5, 20512),  # two CTAs, ragged tail
    ("f32", 151936, 0),           # eight CTAs, f32 rows
    ("bf16", 16384, 10256),       # one CTA per row: the exchange with itself
    ("f32", 12, 40128),           # most slices empty
])
def test_loss_sweep_waits_run_out(dtype, V, variant):
    from paper_2603_04135_b200 import binding as B
    T, S = 37, 3
    per16 = 8 if dtype == "bf16" else 4
    stride = -(-V // per16) * per16
    w = synth.scaled(synth.WORKLOADS["config3"], V=stride, dtype=dtype)
    tok = synth.make_token_inputs(w, T, 11, device="cuda")
    tok.target.clamp_(max=V - 1)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    rng = np.random.default_rng(11)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.from_numpy((rng.random(S) * 0.1).astype(np.float32)).cuda()

    def params(v):
        return B.LossParams(T, V, B.BF16 if dtype == "bf16" else B.F32, stride, S, v, 0.2, 0.2, 0.04, 1.0)

    choice = B.grpo_loss_kernel_choice(params(variant))
    assert choice.kernel == B.KERNEL_SHARED and choice.fell_back == 0
    before = _loss_call(B, params(variant), tok, cu, adv, wseq, T, stride, tdt)
    assert before[4] == 0 and float(before[1][4]) == T

    dl, loss_out, logp_out, lse_out, status = _loss_call(B, params(B.LOSS_WAIT_SELF_TEST + variant), tok, cu, adv, wseq,
                                                         T, stride, tdt)
    assert status == B.STATUS_TIMEOUT
    assert bool((dl[:, :V] == 0).all())                       # every row written as zeros
    if stride > V:
        assert bool((dl[:, V:] == 7.0).all())                 # padding untouched
    assert bool((logp_out == 0).all()) and bool((lse_out == 0).all())
    lo = loss_out.cpu().numpy()
    assert np.isfinite(lo).all() and (lo[:4] == 0).all() and lo[4] == T

    after = _loss_call(B, params(variant), tok, cu, adv, wseq, T, stride, tdt)
    assert after[4] == 0
    for a, b in zip(before[:4], after[:4]):                   # the ordinary call is what it was: same bits
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a.view(torch.int32),
                           b.view(torch.int16) if b.dtype == torch.bfloat16 else b.view(torch.int32))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_streaming_forward_kernel_waits_run_out(dtype):
    """The forward-only streaming kernel: the first stage of every CTA's ring expects 8 bytes more than its copy
    brings, so the consumers' first wait runs out after 1 ms; every CTA reports the time-out, lets its copies land
    and leaves all of its rows as rows that add nothing."""
    from paper_2603_04135_b200 import binding as B
    T, S, V = 400, 3, 151936
    w = synth.scaled(synth.WORKLOADS["config3"], V=V, dtype=dtype)
    tok = synth.make_token_inputs(w, T, 12, device="cuda")
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    adv = torch.ones(S, device="cuda"); wseq = torch.full((S,), 0.1, device="cuda")

    def call(variant):
        prm = B.LossParams(T, V, B.BF16 if dtype == "bf16" else B.F32, V, S, variant, 0.2, 0.2, 0.04, 1.0)
        nbytes = B.grpo_loss_workspace_bytes(prm)
        ws = torch.full((nbytes,), 0x7f, dtype=torch.uint8, device="cuda")     # garbage the kernel must overwrite
        loss_out = torch.full((5,), 7.0, device="cuda")
        logp_out = torch.full((T,), 7.0, device="cuda"); lse_out = torch.full((T,), 7.0, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, None, adv, wseq, None, None,
                            logp_out, lse_out, loss_out, ws, nbytes, status)
        torch.cuda.synchronize()
        return loss_out, logp_out, lse_out, int(status.item())

    before = call(0)                                              # variant 0 takes the streaming kernel here
    assert before[3] == 0 and float(before[0][4]) == T
    loss_out, logp_out, lse_out, status = call(B.LOSS_WAIT_SELF_TEST)
    assert status == B.STATUS_TIMEOUT
    assert bool((logp_out == 0).all()) and bool((lse_out == 0).all())
    lo = loss_out.cpu().numpy()
    assert np.isfinite(lo).all() and (lo[:4] == 0).all() and lo[4] == T
    after = call(0)
    assert after[3] == 0
    for a, b in zip(before[:3], after[:3]):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


@pytest.mark.parametrize("dtype,V,T", [("bf16", 1024, 5000), ("f32", 2048, 2000), ("bf16", 64, 40000)])
def test_tile_kernel_waits_run_out(dtype, V, T):
    """The tile kernel: the first tile of every CTA is announced with 8 bytes more than its copy brings, so the
    consumers' first wait runs out after 1 ms; every CTA reports the time-out, lets its copies land and leaves all
    of its rows as rows that add nothing (dlogits of zeros)."""
    from paper_2603_04135_b200 import binding as B
    S = 5
    w = synth.scaled(synth.WORKLOADS["config3"], V=V, dtype=dtype)
    tok = synth.make_token_inputs(w, T, 13, device="cuda")
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    rng = np.random.default_rng(13)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.from_numpy((rng.random(S) * 0.1).astype(np.float32)).cuda()

    def params(v):
        return B.LossParams(T, V, B.BF16 if dtype == "bf16" else B.F32, V, S, v, 0.2, 0.2, 0.04, 1.0)

    assert B.grpo_loss_kernel_choice(params(0)).kernel == B.KERNEL_TILE
    before = _loss_call(B, params(0), tok, cu, adv, wseq, T, V, tdt)
    assert before[4] == 0 and float(before[1][4]) == T
    dl, loss_out, logp_out, lse_out, status = _loss_call(B, params(B.LOSS_WAIT_SELF_TEST), tok, cu, adv, wseq, T, V, tdt)
    assert status == B.STATUS_TIMEOUT
    assert bool((dl == 0).all())
    assert bool((logp_out == 0).all()) and bool((lse_out == 0).all())
    lo = loss_out.cpu().numpy()
    assert np.isfinite(lo).all() and (lo[:4] == 0).all() and lo[4] == T
    after = _loss_call(B, params(0), tok, cu, adv, wseq, T, V, tdt)
    assert after[4] == 0
    for a, b in zip(before[:4], after[:4]):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a.view(torch.int32),
                           b.view(torch.int16) if b.dtype == torch.bfloat16 else b.view(torch.int32))


def test_wait_self_test_needs_a_kernel_that_waits():
    from paper_2603_04135_b200 import binding as B
    prm = B.LossParams(8, 508, B.BF16, 512, 1, B.LOSS_WAIT_SELF_TEST, 0.2, 0.2, 0.04, 1.0)   # warp-per-row shape
    with pytest.raises(B.DppoError) as e:
        B.grpo_loss_kernel_choice(prm)
    assert e.value.code == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("variant", [1, 0])                   # single-CTA core, CTA-pair core
@pytest.mark.parametrize("backward", [0, 1])
def test_lmhead_waits_run_out(variant, backward):
    from paper_2603_04135_b200 import binding as B
    T, V, H, S = 700, 1000, 192, 4
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=V, H=H)
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, 9, device="cuda")
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    rng = np.random.default_rng(9)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.from_numpy((rng.random(S) * 0.1).astype(np.float32)).cuda()

    def call(v):
        prm = B.LmheadParams(B.LossParams(T, V, B.BF16, V, S, 0, 0.2, 0.2, 0.04, 1.0), H, backward, v, B.F32)
        nbytes = B.lmhead_workspace_bytes(prm)
        ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda"); ws = ws[(-ws.data_ptr()) % 1024:]
        dh = torch.zeros((T, H), dtype=torch.bfloat16, device="cuda") if backward else None
        dW = torch.zeros((V, H), device="cuda") if backward else None
        loss_out = torch.zeros(5, device="cuda"); logp_out = torch.zeros(T, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, cu, None, adv, wseq, None, dh, dW, logp_out, None, loss_out,
                           ws, nbytes, status)
        torch.cuda.synchronize()                              # the call returns: every CTA left on its own
        return [x for x in (loss_out, logp_out, dh, dW) if x is not None], int(status.item())

    before, status = call(variant)
    assert status == 0
    _, status = call(B.LMHEAD_WAIT_SELF_TEST + variant)
    assert status == B.STATUS_TIMEOUT                         # the other outputs are unspecified
    after, status = call(variant)
    assert status == 0                                        # tensor memory was freed, the device is as before
    for a, b in zip(before, after):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a.view(torch.int32),
                           b.view(torch.int16) if b.dtype == torch.bfloat16 else b.view(torch.int32))
