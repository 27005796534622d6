"""A self-contained run of the fused LM-head + loss for timing and profiler captures.

  python -m paper_2603_04135_b200.profile_case_lmhead --tokens 16384 --hidden 2560 --iters 3

Prints the event-timed duration of each call and the tensor throughput it corresponds to
(2*T*V*H flops for the forward projection; 6*T*V*H with --backward: logits, dhidden, dW).
"""
import argparse

import numpy as np
import torch

from . import binding as B
from . import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=16384)
    ap.add_argument("--hidden", type=int, default=2560)
    ap.add_argument("--vocab", type=int, default=151936)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--seqs", type=int, default=32)
    ap.add_argument("--backward", action="store_true", help="also dhidden and dW")
    ap.add_argument("--variant", type=int, default=0, help="0: CTA pairs, 1: one CTA per tile")
    args = ap.parse_args()
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=args.vocab, H=args.hidden)
    T, S = args.tokens, args.seqs
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, 0, device="cuda")
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    adv = torch.from_numpy(np.random.default_rng(0).normal(size=S).astype(np.float32)).cuda()
    wseq = torch.full((S,), 1.0 / S, device="cuda")
    prm = B.LmheadParams(B.LossParams(T, w.V, B.BF16, w.V, S, 0, w.eps, w.eps, w.beta, 1.0), w.H, int(args.backward), args.variant)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 1024:]
    dh = torch.empty((T, w.H), dtype=torch.bfloat16, device="cuda") if args.backward else None
    dW = torch.empty((w.V, w.H), dtype=torch.float32, device="cuda") if args.backward else None
    loss_out = torch.zeros(5, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flops = (6.0 if args.backward else 2.0) * T * w.V * w.H     # logits, dhidden, dW: 2 T V H each
    for it in range(args.iters):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, cu, None, adv, wseq, None, dh, dW, None, None, loss_out,
                           ws, nbytes, status)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        print("iter %d: %.3f ms  %.1f TFLOP/s executed  %.0f tokens/s  loss %.6g  status %d" % (
            it, ms, flops / ms / 1e9, T / ms * 1e3, loss_out[0].item(), status.item()))
    assert status.item() == 0


if __name__ == "__main__":
    main()
