"""Process-pool worker: the oracle's loss forward + backward on a block of token rows.

TEST INFRASTRUCTURE ONLY — see the package docstring.  Used by the benchmark's CPU-baseline and
reference legs to spread rows over host cores; it only calls `grpo_loss` as it stands.
"""
import numpy as np

from .dppo_oracle import grpo_loss, bf16_bits_to_f64


def fwd_bwd_rows(args):
    (chunk, is_bf16, rows, target, logp_old, logp_ref, cu, adv_seg, w_seg, eps_lo, eps_hi, beta, tau) = args
    z = bf16_bits_to_f64(chunk) if is_bf16 else np.asarray(chunk, dtype=np.float64)
    out = grpo_loss(z, target, logp_old, logp_ref, cu, adv_seg, w_seg, eps_lo, eps_hi, beta, tau,
                    want_dlogits=True, rows=rows, chunk=32)
    # the gradient block is produced and dropped here; only its checksum travels back
    return float(out["loss"]), float(np.abs(out["dlogits"]).sum()), len(rows)
