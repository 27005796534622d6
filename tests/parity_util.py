"""Helpers shared by the GPU parity tests: run the oracle on a synthetic batch, compare outputs."""
import math
import multiprocessing as mp
import os

import numpy as np
import torch

import oracle
import oracle_worker
from paper_2603_04135_b200 import synth


def oracle_prune_pack(batch, w, seed, step, use_history=True, reverse=False, best_fit=False,
                      r_q=None, r_o=None, N_win=None, L_row=None, u_q=None, u_o=None, mode=0):
    """Steps 1-5 on the CPU.  The history score is mean |A| of the earlier-epoch rewards (Eq. 16)."""
    adv, mabs = oracle.group_advantages(batch.rewards)
    H_prev = oracle.group_advantages(batch.rewards_prev)[1] if use_history else None
    pr = oracle.prune_and_rescale(adv, mabs, H_prev, w.r_q if r_q is None else r_q,
                                  w.r_o if r_o is None else r_o, seed=seed, step=step, reverse=reverse,
                                  u_q=u_q, u_o=u_o, mode=mode)
    pk = oracle.pack_prompts(batch.unit_len, w.L_row if L_row is None else L_row,
                             w.N_win if N_win is None else N_win, keep=pr["keep_o"].reshape(-1),
                             loss_len=batch.loss_len, best_fit=best_fit)
    return dict(adv=adv, mean_abs_adv=mabs, H_prev=H_prev, prune=pr, pack=pk)


def assert_prune_equal(gpu, ref):
    """gpu: DppoStep.prune_results(); ref: oracle_prune_pack() output.  Bit-exact everything."""
    P, G = ref["adv"].shape
    assert np.array_equal(gpu["adv"].view(np.uint32), ref["adv"].reshape(-1).view(np.uint32))
    assert np.array_equal(gpu["mean_abs_adv"].view(np.uint32), ref["mean_abs_adv"].view(np.uint32))
    pr = ref["prune"]
    for k in ("cand_q", "keep_q"):
        assert np.array_equal(gpu[k], pr[k]), k
    for k in ("cand_o", "keep_o"):
        assert np.array_equal(gpu[k], pr[k].reshape(-1)), k
    assert int(gpu["n_keep_q"][0]) == pr["n_keep_q"]
    assert np.array_equal(gpu["n_keep_o"], pr["n_keep_o"])
    for k in ("gamma_q", "H_next"):
        assert np.array_equal(gpu[k].view(np.uint32), pr[k].view(np.uint32)), k
    for k in ("gamma_o", "w_seq"):
        assert np.array_equal(gpu[k].view(np.uint32), pr[k].reshape(-1).view(np.uint32)), k


def assert_pack_equal(gpu, ref_pack, n_max):
    """gpu: DppoStep.pack_results(); ref_pack: oracle.pack_prompts() output.  Bit-exact."""
    n_units, n_rows = ref_pack["counts"][0], ref_pack["counts"][1]
    assert tuple(int(x) for x in gpu["counts"]) == tuple(ref_pack["counts"])
    assert list(gpu["order"][:n_units]) == list(ref_pack["order"])
    assert (gpu["order"][n_units:] == -1).all()
    assert list(gpu["row_of"]) == list(ref_pack["row_of"])
    assert list(gpu["off_in_row"]) == list(ref_pack["off_in_row"])
    assert list(gpu["row_fill"][:n_rows]) == list(ref_pack["row_fill"])
    assert (gpu["row_fill"][n_rows:] == 0).all()
    assert list(gpu["cu_seqlens"][:n_units + 1]) == list(ref_pack["cu_seqlens"])
    assert (gpu["cu_seqlens"][n_units:] == ref_pack["cu_seqlens"][-1]).all()


def rows_to_f64(logits, rows):
    """Exact float64 copy of selected rows of a device logits tensor."""
    idx = torch.as_tensor(np.asarray(rows, dtype=np.int64), device=logits.device)
    return logits.index_select(0, idx).to(torch.float64).cpu().numpy()


def pick_rows(cu_seqlens, T, n_random, seed):
    """First and last token of every sequence plus random rows."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    rows = set()
    for s in range(len(cu) - 1):
        if cu[s + 1] > cu[s]:
            rows.add(int(cu[s])); rows.add(int(cu[s + 1] - 1))
    rng = np.random.default_rng(seed)
    if T > 0:
        rows.update(int(x) for x in rng.integers(0, T, size=n_random))
    return np.array(sorted(rows), dtype=np.int64)


class Guarded:
    """An output buffer with a guard band of sentinel elements before and after it (the library writes through
    raw pointers, and no sanitizer runs in these tests): `t` is the tensor handed to the library, check() asserts
    that nothing outside it was written.  The band is 256 elements, so `t` keeps the alignment of the allocation
    up to 512 bytes."""
    GUARD = 256

    def __init__(self, shape, dtype, fill, device="cuda"):
        n = 1
        for d in shape:
            n *= int(d)
        self.sentinel = 77 if not dtype.is_floating_point else 1024.0          # exact in every dtype used here
        self.buf = torch.full((n + 2 * self.GUARD,), self.sentinel, dtype=dtype, device=device)
        self.t = self.buf[self.GUARD:self.GUARD + n].view(*shape)
        self.t.fill_(fill)

    def check(self):
        g = self.GUARD
        assert bool((self.buf[:g] == self.sentinel).all()), "write before the start of an output buffer"
        assert bool((self.buf[-g:] == self.sentinel).all()), "write past the end of an output buffer"


LOGP_TOL = {"f32": 2e-6, "bf16": 1e-5}      # |logp - oracle| with f32 accumulation of the row sum


def assert_dlogits_close(got, ref_out, dtype, beta, rows_ok=None):
    """Element-wise parity of dlogits rows.  got: device rows as float64; ref_out: oracle.grpo_loss output
    for the same rows.  With g = dloss/dlogp of the row and ref the oracle's element:

      bf16:  |d| <= (2^-8 + 2^-11) |ref| + 1e-6 |g| + s   (the bf16 rounding of the output, unit roundoff 2^-8, on
                                                          top of the fp16 rounding of the stored exponential,
                                                          unit roundoff 2^-11)                and max-abs 2e-3
      f32:   |d| <= 1e-5 |ref| + 5e-7 |g| + s      (a few f32 ulps of g*softmax)             and max-abs 1e-5

    s = LOGP_TOL * W (|A| rho + beta rho_hat) * |onehot - softmax| is what the allowed log-prob error does to
    g = -W (A rho [unclipped] + beta (rho_hat - 1)): on rows where g nearly cancels (A = 0 and rho_hat
    close to 1) it dominates the relative terms.  Rows must sum to zero up to rounding.
    """
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref_out["dlogits"], dtype=np.float64)
    g = np.asarray(ref_out["g"], dtype=np.float64)
    sens = ref_out["W"] * (np.abs(ref_out["A"]) * ref_out["rho"] + beta * ref_out["rho_hat"])
    if rows_ok is not None:
        keep = np.asarray(rows_ok, dtype=bool)
        got, ref, g, sens = got[keep], ref[keep], g[keep], sens[keep]
    ga = np.abs(g)[:, None]
    with np.errstate(divide="ignore", invalid="ignore"):
        shape = np.where(ga > 0, np.abs(ref) / ga, 0.0)             # |onehot - softmax|
    slack = LOGP_TOL[dtype] * sens[:, None] * shape
    err = np.abs(got - ref)
    if dtype == "bf16":
        bound = (2.0 ** -8 + 2.0 ** -11) * np.abs(ref) + 1e-6 * ga + slack
        assert err.max(initial=0.0) <= 2e-3
    else:
        bound = 1e-5 * np.abs(ref) + 5e-7 * ga + slack
        assert err.max(initial=0.0) <= 1e-5
    bad = err > bound
    assert not bad.any(), "dlogits: %d elements off, worst ratio %.3g" % (bad.sum(), (err / np.maximum(bound, 1e-300)).max())
    # rounding of the V terms does not cancel exactly: allow its worst case
    tol = 1e-3 * ga[:, 0] + (2.0 ** -8 * np.abs(ref).sum(axis=1) if dtype == "bf16" else 0.0)
    assert (np.abs(got.sum(axis=1)) <= tol + 1e-30).all()


def clip_decision_is_stable(rho, eps_lo, eps_hi, margin=1e-5):
    """Rows whose ratio is not within `margin` of a clip bound (there a float32-vs-float64 difference in
    the log-prob may legitimately flip the branch)."""
    rho = np.asarray(rho)
    return (np.abs(rho - (1.0 - eps_lo)) > margin) & (np.abs(rho - (1.0 + eps_hi)) > margin)


# ---- oracle over all rows of a large device tensor, in worker processes ---------------------------
def oracle_forward_all_rows(logits, target, logp_old, logp_ref, cu, adv_seg, w_seg, eps_lo, eps_hi, beta,
                            tau=1.0, rows_per_task=256, processes=None, pool=None):
    """Forward oracle (logp, lse, loss sums) over every row of a device tensor: rows are streamed to the
    host in chunks and evaluated by spawned worker processes."""
    T = logits.shape[0]
    is_bf16 = logits.dtype == torch.bfloat16
    target = np.asarray(target); logp_old = np.asarray(logp_old); logp_ref = np.asarray(logp_ref)

    def tasks():
        for a in range(0, T, rows_per_task):
            b = min(T, a + rows_per_task)
            blk = logits[a:b]
            chunk = (blk.view(torch.int16).cpu().numpy().view(np.uint16) if is_bf16 else blk.cpu().numpy())
            yield (chunk, is_bf16, np.arange(a, b), target, logp_old, logp_ref, np.asarray(cu), np.asarray(adv_seg),
                   np.asarray(w_seg), eps_lo, eps_hi, beta, tau)

    own = pool is None and processes != 0
    if processes == 0:                                   # small case: evaluate in this process
        parts = [oracle_worker.forward_rows(t) for t in tasks()]
        cores = 1
    else:
        if own:
            ctx = mp.get_context("spawn")                # never fork after CUDA has been initialised
            pool = ctx.Pool(processes or min(32, os.cpu_count() or 1))
        cores = pool._processes
        try:
            parts = list(pool.imap(oracle_worker.forward_rows, tasks()))
        finally:
            if own:
                pool.close(); pool.join()
    logp = np.zeros(T); lse = np.zeros(T); g = np.zeros(T); rho = np.zeros(T)
    for p in parts:
        logp[p["rows"]] = p["logp"]; lse[p["rows"]] = p["lse"]; g[p["rows"]] = p["g"]; rho[p["rows"]] = p["rho"]
    return dict(logp=logp, lse=lse, g=g, rho=rho,
                loss=math.fsum(p["loss"] for p in parts), pg=math.fsum(p["pg"] for p in parts),
                kl=math.fsum(p["kl"] for p in parts), abs_sum=math.fsum(p["abs_sum"] for p in parts),
                clip_frac=(sum(p["n_clipped"] for p in parts) / T) if T else 0.0, cores=cores)
