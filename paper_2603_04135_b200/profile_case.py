"""A small, self-contained run of the loss sweep for profiler captures.

  python -m paper_2603_04135_b200.profile_case --rows 8192 --iters 3

Runs dppo_grpo_loss_fwd_bwd on `rows` token rows of the large-vocabulary workload (bf16 logits,
V = 151,936: 2.5 GB in + 2.5 GB out at 8192 rows, well above L2 yet small enough for a multi-pass
capture) and prints the event-timed duration of each call.
"""
import argparse

import numpy as np
import torch

from . import binding as B
from . import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--vocab", type=int, default=151936)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--in-place", action="store_true")
    ap.add_argument("--seqs", type=int, default=16)
    ap.add_argument("--full-call", action="store_true",
                    help="pass everything the training step passes: device token count, seg_map, logp/lse outputs")
    ap.add_argument("--back-to-back", action="store_true", help="enqueue all iterations before synchronising")
    ap.add_argument("--variant", type=int, default=0, help="kernel variant (see dppo_loss_params.variant)")
    args = ap.parse_args()
    w = synth.scaled(synth.WORKLOADS["config3"], V=args.vocab, dtype=args.dtype)
    T, S = args.rows, args.seqs
    tok = synth.make_token_inputs(w, T, 0, device="cuda")
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    rng = np.random.default_rng(0)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.full((S,), 1.0 / S, device="cuda")
    dl = tok.logits if args.in_place else torch.empty_like(tok.logits)
    prm = B.LossParams(T, w.V, B.BF16 if args.dtype == "bf16" else B.F32, w.V, S, args.variant, w.eps, w.eps, w.beta, 1.0)
    nbytes = B.grpo_loss_workspace_bytes(prm)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    loss_out = torch.zeros(5, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    esize = 2 if args.dtype == "bf16" else 4
    ntd = seg_map = logp_out = lse_out = None
    if args.full_call:
        ntd = torch.tensor([T], dtype=torch.int32, device="cuda")
        seg_map = torch.arange(S, dtype=torch.int32, device="cuda")
        logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
    events = []
    for it in range(args.iters):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, ntd, adv, wseq, seg_map, dl,
                            logp_out, lse_out, loss_out, ws, nbytes, status)
        e1.record()
        events.append((e0, e1))
        if not args.back_to_back:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    for it, (e0, e1) in enumerate(events):
        ms = e0.elapsed_time(e1)
        print("iter %d: %.3f ms  %.1f GB/s algorithmic  loss %.6g  status %d" % (
            it, ms, 2 * T * w.V * esize / ms / 1e6, loss_out[0].item(), status.item()))
    assert status.item() == 0


if __name__ == "__main__":
    main()
