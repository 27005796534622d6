"""Worker-process side of the all-rows oracle pass (imports only numpy and the oracle)."""
import numpy as np

import oracle


def forward_rows(args):
    (chunk, is_bf16, rows, target, logp_old, logp_ref, cu, adv_seg, w_seg, eps_lo, eps_hi, beta, tau) = args
    z = oracle.bf16_bits_to_f64(chunk) if is_bf16 else chunk.astype(np.float64)
    out = oracle.grpo_loss(z, target, logp_old, logp_ref, cu, adv_seg, w_seg, eps_lo, eps_hi, beta, tau,
                           want_dlogits=False, rows=rows, chunk=64)
    return dict(rows=rows, logp=out["logp"], lse=out["lse"], loss=out["loss"], pg=out["pg"], kl=out["kl"],
                abs_sum=out["abs_sum"], n_clipped=int(out["clipped"].sum()), g=out["g"], rho=out["rho"])
