"""Float64 CPU oracle for DPPO's pruned GRPO step.

TEST INFRASTRUCTURE ONLY — see the package docstring.  Nothing here is tuned;
each function takes the steps of the paper in the paper's order and notation.
Small per-prompt quantities use plain Python floats (IEEE binary64, one
operation at a time, ascending index, never fused), so that the decisions they
feed (candidate sets, masks) are reproducible bit for bit.  The per-token pass
uses numpy float64 array primitives (max, exp, sum, log) as library steps.

Notation: P prompts per batch (|Q|), G completions per prompt (|O|),
A advantage, Abar mean |A| of a group, H history score, r_q / r_o pruning
probabilities, gamma rescaling factors, L_row row capacity, N_win window size,
T loss tokens, V vocabulary, rho = pi_theta / pi_old, rho_hat = pi_ref / pi_theta.
"""
import math

import numpy as np

from .philox import uniform53, DOMAIN_PROMPT, DOMAIN_COMPLETION

TIE_SLACK = 1e-12   # relative slack on the candidate test |A_i| <= mean|A| (see completion_candidates)


# --------------------------------------------------------------------------
# Step 1 — group-relative advantages (Eq. 2) and the threshold (Eq. 14)
# --------------------------------------------------------------------------
def group_advantages(rewards, ddof=0, std_eps=1e-6):
    """A_i = (r_i - mean(r)) / (std(r) + std_eps) within each group (Eq. 2) and
    Abar = (1/G) sum_i |A_i| (Eq. 14).

    rewards: [P, G] float32 values.  Returns (adv float32 [P,G], mean_abs_adv
    float32 [P]).  The paper writes only "std": the divisor G - ddof and the
    guard std_eps are parameters (defaults: population std, 1e-6).  A group whose
    rewards are all bitwise equal gets A = 0 exactly.  Sums run in ascending i.
    """
    r = np.asarray(rewards, dtype=np.float32)
    P, G = r.shape
    adv = np.zeros((P, G), dtype=np.float32)
    mean_abs = np.zeros(P, dtype=np.float32)
    for k in range(P):
        rk = [float(x) for x in r[k]]
        if all(x == rk[0] for x in rk) or G - ddof <= 0:
            continue
        s = 0.0
        for x in rk:
            s = s + x
        mu = s / G
        d = [x - mu for x in rk]
        ss = 0.0
        for x in d:
            ss = ss + x * x
        sigma = math.sqrt(ss / (G - ddof))
        a = [x / (sigma + std_eps) for x in d]
        sa = 0.0
        for x in a:
            sa = sa + abs(x)
        adv[k] = np.array(a, dtype=np.float64).astype(np.float32)
        mean_abs[k] = np.float32(sa / G)
    return adv, mean_abs


# --------------------------------------------------------------------------
# Step 2 — candidate sets (Eq. 15 for completions, Eq. 17 for prompts)
# --------------------------------------------------------------------------
def completion_candidates(adv, reverse=False):
    """cand_o[k,i] = |A_i| <= Abar_k (Eq. 15; Algorithm 1's candidate set C).

    Taken on the float32 advantages as stored, in binary64, as
        G*|A_i| <= (sum_j |A_j|) * (1 + 1e-12)
    so that the frequent exact tie (all |A_i| equal: half the group succeeded, or
    every reward equal) lands on "candidate" whatever the rounding of the mean.
    reverse=True is the ablation rule of Table 5 (high-|A| completions are the
    candidates): the complement.
    """
    a = np.asarray(adv, dtype=np.float32)
    P, G = a.shape
    cand = np.zeros((P, G), dtype=np.uint8)
    for k in range(P):
        absa = [abs(float(x)) for x in a[k]]
        s = 0.0
        for x in absa:
            s = s + x
        bound = s * (1.0 + TIE_SLACK)
        for i in range(G):
            low = (G * absa[i]) <= bound
            cand[k, i] = (not low) if reverse else low
    return cand


def prompt_candidates(H_prev, P, reverse=False):
    """cand_q = the floor(P/2) prompts of the batch with the lowest history score
    (Eq. 17; Algorithm 1, bottom 50% of the batch).  No history (first epoch):
    no candidates.  Ties go to the lower index; reverse=True takes the highest
    scores instead (Table 5's ablation), ties again to the lower index.
    """
    cand = np.zeros(P, dtype=np.uint8)
    if H_prev is None:
        return cand
    h = [float(x) for x in np.asarray(H_prev, dtype=np.float32)]
    if reverse:
        ranked = sorted(range(P), key=lambda k: (-h[k], k))
    else:
        ranked = sorted(range(P), key=lambda k: (h[k], k))
    for k in ranked[: P // 2]:
        cand[k] = 1
    return cand


# --------------------------------------------------------------------------
# Step 3 — dynamic pruning masks (Eq. 15, Eq. 17)
# --------------------------------------------------------------------------
def draw_uniforms(seed, step, P, G):
    """u_q[k], u_o[k,i] in [0,1) for every index, candidate or not."""
    u_q = np.array([uniform53(seed, step, DOMAIN_PROMPT, k) for k in range(P)], dtype=np.float64)
    u_o = np.array([[uniform53(seed, step, DOMAIN_COMPLETION, k * G + i) for i in range(G)]
                    for k in range(P)], dtype=np.float64)
    return u_q, u_o


def prune_masks(cand_q, cand_o, u_q, u_o, r_q, r_o, mode=0):
    """Pruning of the candidates (Eq. 15, 17).

    mode 0 — independent draws: a prompt is pruned iff cand_q and u_q < r_q; a
    completion iff cand_o and u_o < r_o.
    mode 1 — fixed fraction (Appendix A, Algorithm 1): of the prompt candidates
    B the floor(r_q*|B|) with the smallest (u, index) are pruned; of each
    prompt's completion candidates C the floor(r_o*|C|) with the smallest
    (u, index).
    Every completion of a pruned prompt goes with it.  Returns keep_q u8[P],
    keep_o u8[P,G], n_keep_q = |S^q|, n_keep_o[k] = |S^o(q_k)| (0 for a pruned
    prompt).
    """
    cand_q = np.asarray(cand_q); cand_o = np.asarray(cand_o)
    P, G = cand_o.shape
    keep_q = np.ones(P, dtype=np.uint8)
    keep_o = np.ones((P, G), dtype=np.uint8)
    if mode == 0:
        for k in range(P):
            if cand_q[k] and float(u_q[k]) < r_q:
                keep_q[k] = 0
            for i in range(G):
                if cand_o[k, i] and float(u_o[k, i]) < r_o:
                    keep_o[k, i] = 0
    else:
        B = [k for k in range(P) if cand_q[k]]
        for k in sorted(B, key=lambda k: (float(u_q[k]), k))[: int(math.floor(r_q * len(B)))]:
            keep_q[k] = 0
        for k in range(P):
            C = [i for i in range(G) if cand_o[k, i]]
            for i in sorted(C, key=lambda i: (float(u_o[k, i]), i))[: int(math.floor(r_o * len(C)))]:
                keep_o[k, i] = 0
    for k in range(P):
        if not keep_q[k]:
            keep_o[k, :] = 0
    n_keep_q = int(keep_q.sum())
    n_keep_o = keep_o.sum(axis=1).astype(np.int32)
    return keep_q, keep_o, n_keep_q, n_keep_o


# --------------------------------------------------------------------------
# Step 4 — discrete importance rescaling (Eq. 18) and the history update (Eq. 16)
# --------------------------------------------------------------------------
def rescale(cand_q, cand_o, keep_q, keep_o, r_q, r_o, mean_abs_adv, H_prev, mode=0):
    """gamma_q[k] = (|S^q|/|Q|) / (1 - P^q(q_k)),
    gamma_o[k,i] = (|S^o(q_k)|/|O|) / (1 - P^o(o_i))                      (Eq. 18)
    for retained items (0 for pruned ones), with P^q = r_q on prompt candidates
    and 0 elsewhere, P^o likewise (Eq. 15, 17).  In fixed-fraction mode the
    probability that a candidate is pruned is the realised fraction
    floor(r|C|)/|C| of its candidate set, and that is what P stands for.

    w_seq[k,i] is the weight of completion (k,i) in the pruned objective read as
    the mean over RETAINED prompts of gamma_q times the mean over RETAINED
    completions of gamma_o times the per-completion term (Eq. 9, 12, 13 are
    expectations under the pruned distributions):
        w_seq = gamma_q*gamma_o / (|S^q| |S^o(q_k)|) = 1 / (P*G*(1-P^q)*(1-P^o)),
    evaluated in that last form; 0 for pruned items, so empty sets divide nothing.

    H_next[k] = Abar_k if the prompt was retained, else H_prev[k] (Eq. 16); with
    no history every prompt was "selected", so H_next = Abar.
    """
    cand_q = np.asarray(cand_q); cand_o = np.asarray(cand_o)
    keep_q = np.asarray(keep_q); keep_o = np.asarray(keep_o)
    P, G = cand_o.shape
    n_q = int(keep_q.sum())
    gamma_q = np.zeros(P, dtype=np.float32)
    gamma_o = np.zeros((P, G), dtype=np.float32)
    w_seq = np.zeros((P, G), dtype=np.float32)
    H_next = np.zeros(P, dtype=np.float32)
    n_B = int(cand_q.sum())
    if mode == 0:
        Pq_cand = r_q
    else:
        Pq_cand = (float(int(math.floor(r_q * n_B))) / n_B) if n_B > 0 else 0.0
    for k in range(P):
        Pq = Pq_cand if cand_q[k] else 0.0
        n_o = int(keep_o[k].sum())
        n_C = int(cand_o[k].sum())
        if mode == 0:
            Po_cand = r_o
        else:
            Po_cand = (float(int(math.floor(r_o * n_C))) / n_C) if n_C > 0 else 0.0
        if keep_q[k]:
            gamma_q[k] = np.float32((n_q / P) / (1.0 - Pq))
        for i in range(G):
            if keep_o[k, i]:
                Po = Po_cand if cand_o[k, i] else 0.0
                gamma_o[k, i] = np.float32((n_o / G) / (1.0 - Po))
                w_seq[k, i] = np.float32(1.0 / ((float(P * G) * (1.0 - Pq)) * (1.0 - Po)))
        if keep_q[k] or H_prev is None:
            H_next[k] = np.float32(mean_abs_adv[k])
        else:
            H_next[k] = np.float32(H_prev[k])
    return gamma_q, gamma_o, w_seq, H_next


def prune_and_rescale(adv, mean_abs_adv, H_prev, r_q, r_o, seed=0, step=0,
                      u_q=None, u_o=None, reverse=False, mode=0):
    """Steps 2-4 in one call; u_q/u_o override the generator when given."""
    adv = np.asarray(adv, dtype=np.float32)
    P, G = adv.shape
    cand_o = completion_candidates(adv, reverse=reverse)
    cand_q = prompt_candidates(H_prev, P, reverse=reverse)
    if u_q is None or u_o is None:
        dq, do = draw_uniforms(seed, step, P, G)
        u_q = dq if u_q is None else u_q
        u_o = do if u_o is None else u_o
    keep_q, keep_o, n_keep_q, n_keep_o = prune_masks(cand_q, cand_o, u_q, u_o, r_q, r_o, mode=mode)
    gamma_q, gamma_o, w_seq, H_next = rescale(cand_q, cand_o, keep_q, keep_o, r_q, r_o,
                                              mean_abs_adv, H_prev, mode=mode)
    return dict(cand_q=cand_q, cand_o=cand_o, keep_q=keep_q, keep_o=keep_o,
                n_keep_q=n_keep_q, n_keep_o=n_keep_o, gamma_q=gamma_q, gamma_o=gamma_o,
                w_seq=w_seq, H_next=H_next)


def history_epochs(rewards_by_epoch, batches_by_epoch, N, G, r_q, r_o, seed=0, mode=0):
    """Algorithm 1's outer loops for the pruning state only: H_0 = 0 for every dataset prompt; in epoch
    t each batch (a list of dataset prompt ids) reads H_{t-1} of its prompts (no prompt pruning in the
    first epoch), prunes, and writes H_t back (Eq. 16: fresh mean |A| for retained prompts, the old score
    for pruned ones).  rewards_by_epoch[t] is [N, G]; draws use step = t * 1_000_000 + batch index.
    Returns (final table float32 [N], list of per-batch results)."""
    table = np.zeros(N, dtype=np.float32)
    log = []
    for t, (rewards, batches) in enumerate(zip(rewards_by_epoch, batches_by_epoch)):
        for b, ids in enumerate(batches):
            ids = np.asarray(ids, dtype=np.int64)
            adv, mabs = group_advantages(np.asarray(rewards)[ids])
            H_prev = None if t == 0 else table[ids].copy()
            out = prune_and_rescale(adv, mabs, H_prev, r_q, r_o, seed=seed, step=t * 1000000 + b, mode=mode)
            table[ids] = out["H_next"]
            log.append(out)
    return table, log


# --------------------------------------------------------------------------
# Step 5 — Dense Prompt Packing (Section 4.3; Algorithm 1's packing step)
# --------------------------------------------------------------------------
def pack_prompts(lens, L_row, N_win, keep=None, loss_len=None, best_fit=False):
    """Window-based greedy packing of variable-length units into rows of L_row.

    A candidate pool W of at most N_win units is filled from the stream (the
    retained units in their given order).  For each row: start an empty row;
    repeatedly take from W a unit that fits the remaining space — the first one
    in pool order (best_fit=True: the longest that fits, ties to the oldest) —
    put it at the current offset, remove it from W and fetch the next unit of
    the stream to the tail of W; when nothing in W fits, close the row.  Repeat
    until stream and pool are empty.

    Returns order[p] (unit placed p-th), row_of[u], off_in_row[u] (-1 for
    dropped units), row_fill[r], n_rows, cu_seqlens (exclusive scan of loss_len
    in placement order, length n_units + 1), counts = (n_units, n_rows,
    total_tokens, total_loss_tokens), error (True if a retained unit has length
    < 1 or > L_row: nothing is packed then).
    """
    lens = [int(x) for x in lens]
    n = len(lens)
    stream = [u for u in range(n) if keep is None or keep[u]]
    row_of = [-1] * n
    off_in_row = [-1] * n
    if any(lens[u] < 1 or lens[u] > L_row for u in stream) or N_win < 1:
        return dict(order=[], row_of=row_of, off_in_row=off_in_row, row_fill=[], n_rows=0,
                    cu_seqlens=[0], counts=(0, 0, 0, 0), error=True)
    nxt = min(N_win, len(stream))
    pool = stream[:nxt]
    order, row_fill = [], []
    while pool:
        row = len(row_fill)
        remaining = L_row
        while True:
            pick = None
            for pos, u in enumerate(pool):
                if lens[u] <= remaining:
                    if not best_fit:
                        pick = pos
                        break
                    if pick is None or lens[u] > lens[pool[pick]]:
                        pick = pos
            if pick is None:
                break
            u = pool.pop(pick)
            row_of[u] = row
            off_in_row[u] = L_row - remaining
            remaining -= lens[u]
            order.append(u)
            if nxt < len(stream):
                pool.append(stream[nxt])
                nxt += 1
        row_fill.append(L_row - remaining)
    cu = [0]
    for u in order:
        cu.append(cu[-1] + (int(loss_len[u]) if loss_len is not None else lens[u]))
    counts = (len(order), len(row_fill), sum(lens[u] for u in order), cu[-1])
    return dict(order=order, row_of=row_of, off_in_row=off_in_row, row_fill=row_fill,
                n_rows=len(row_fill), cu_seqlens=cu, counts=counts, error=False)


# --------------------------------------------------------------------------
# Steps 6-8 — per-token log-prob, GRPO terms (Eq. 1) and dlogits
# --------------------------------------------------------------------------
def bf16_bits_to_f64(bits):
    """Exact value of bfloat16 bit patterns (uint16 array) as float64."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """Round-to-nearest-even bfloat16 bit patterns of float64 values (finite)."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    # binary64 -> binary32 -> bfloat16 double-rounds only on measure-zero ties; the
    # parity tolerances are far wider than that.
    u = f.view(np.uint32).astype(np.uint64)
    u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (u >> np.uint64(16)).astype(np.uint16)


def token_logprob(z, y, tau=1.0):
    """log pi_theta(y | .) from the logit rows z [n, V] (float64): the log-softmax
    of z/tau gathered at y.  Returns (logp [n], lse [n])."""
    z = np.asarray(z, dtype=np.float64) / tau
    if z.ndim == 1:
        z = z[None, :]
    y = np.atleast_1d(np.asarray(y, dtype=np.int64))
    m = z.max(axis=1)
    lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
    logp = z[np.arange(z.shape[0]), y] - lse
    return logp, lse


def sequence_log_ratio(logp, logp_old, cu_seqlens):
    """Mean over a sequence's tokens of logp - logp_old: the log of the sequence-level likelihood ratio
    with length normalisation, (pi_theta(o|q) / pi_old(o|q))^(1/|o|), used when the method is combined with a
    sequence-level objective (Section 5.2, "Robustness Across RL Algorithms").  Empty sequences give 0."""
    d = np.asarray(logp, dtype=np.float64) - np.asarray(logp_old, dtype=np.float64)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    out = np.zeros(len(cu) - 1)
    for s in range(len(cu) - 1):
        a, b = int(cu[s]), int(cu[s + 1])
        if b > a:
            acc = 0.0
            for x in d[a:b]:
                acc = acc + float(x)
            out[s] = acc / (b - a)
    return out


def token_terms(logp, logp_old, logp_ref, A, eps_lo, eps_hi, beta, log_ratio=None):
    """Per-token pieces of the GRPO objective (Eq. 1) for advantage A:

      rho  = exp(logp - logp_old)                        probability ratio
      surr = min(rho*A, clip(rho, 1-eps_lo, 1+eps_hi)*A) clipped surrogate
      kl   = rho_hat - log(rho_hat) - 1, rho_hat = exp(logp_ref - logp)
      j    = surr - beta*kl
      dj   = d j / d logp = A*rho*[unclipped] + beta*(rho_hat - 1)
    where [unclipped] is 0 only when the clipped branch is strictly the smaller
    one.  With log_ratio given, rho = exp(log_ratio) replaces the token ratio (dj is
    then the derivative for a ratio whose log is the mean token log-ratio of the
    sequence, times the sequence length — see grpo_loss).  Returns dict of float64
    arrays (clipped as bool).
    """
    logp = np.asarray(logp, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    if log_ratio is None:
        rho = np.exp(logp - np.asarray(logp_old, dtype=np.float64))
    else:                      # a ratio shared by the tokens of a sequence (its own log is given)
        rho = np.exp(np.asarray(log_ratio, dtype=np.float64))
    d = np.asarray(logp_ref, dtype=np.float64) - logp
    rho_hat = np.exp(d)
    kl = rho_hat - d - 1.0
    s1 = rho * A
    s2 = np.clip(rho, 1.0 - eps_lo, 1.0 + eps_hi) * A
    clipped = s2 < s1
    surr = np.where(clipped, s2, s1)
    j = surr - beta * kl
    dj = np.where(clipped, 0.0, A * rho) + beta * (rho_hat - 1.0)
    return dict(rho=rho, rho_hat=rho_hat, kl=kl, surr=surr, j=j, dj=dj, clipped=clipped)


def grpo_loss(logits, target, logp_old, logp_ref, cu_seqlens, adv_seg, w_seg,
              eps_lo=0.2, eps_hi=0.2, beta=0.04, tau=1.0, want_dlogits=True, rows=None,
              chunk=256, length_norm=True, seq_log_ratio=None):
    """The pruned GRPO loss and its gradient w.r.t. the logits.

    logits [T, V] float64 (exact values of the stored fp32/bf16 logits); target
    [T]; token t belongs to sequence s with cu_seqlens[s] <= t < cu_seqlens[s+1];
    the token weight is W_t = w_seg[s] / |o_s| (Eq. 1's 1/|o_i| times the
    sequence weight of `rescale`).  loss = -sum_t W_t j_t is what a trainer
    minimises; pg = -sum W surr; kl = sum W kl_t (loss = pg + beta*kl).
    g_t = d loss / d logp_t = -W_t * dj_t and
    dlogits[t, v] = g_t * ([v == y_t] - softmax(z_t/tau)[v]) / tau.

    rows: optional index list; then only those rows of `logits` are given
    (logits[i] is token rows[i]) and loss sums are over those rows only.

    Variants for the other objectives the paper combines the method with (Section 5.2):
    length_norm=False drops Eq. 1's 1/|o_i| (W_t = w_seg[s]; a token-level mean is then a matter
    of the w the caller passes).  seq_log_ratio [S] replaces the token ratio by the sequence-level
    one, rho_s = exp(seq_log_ratio[s]) with seq_log_ratio = `sequence_log_ratio` of the current
    log-probs; since d rho_s / d logp_t = rho_s / |o_s|, the gradient keeps the token form with rho_s
    in place of rho_t when length_norm is on (asserted here).
    """
    if seq_log_ratio is not None:
        assert length_norm, "the sequence-level ratio is defined with the 1/|o| normalisation"
    logits = np.asarray(logits)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    S = len(cu) - 1
    T = int(cu[-1])
    tok = np.arange(T) if rows is None else np.asarray(rows, dtype=np.int64)
    n = len(tok)
    seg = np.searchsorted(cu, tok, side="right") - 1
    seg_len = (cu[1:] - cu[:-1]).astype(np.float64)
    A = np.asarray(adv_seg, dtype=np.float64)[seg] if n else np.zeros(0)
    W = (np.asarray(w_seg, dtype=np.float64)[seg] / (seg_len[seg] if length_norm else 1.0)) if n else np.zeros(0)
    y = np.asarray(target, dtype=np.int64)[tok]
    logp = np.zeros(n); lse = np.zeros(n)
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        logp[a:b], lse[a:b] = token_logprob(np.asarray(logits[a:b], dtype=np.float64), y[a:b], tau)
    tt = token_terms(logp, np.asarray(logp_old)[tok], np.asarray(logp_ref)[tok], A,
                     eps_lo, eps_hi, beta,
                     log_ratio=None if seq_log_ratio is None else np.asarray(seq_log_ratio, dtype=np.float64)[seg])
    g = -W * tt["dj"]
    out = dict(
        loss=-math.fsum(W * tt["j"]), pg=-math.fsum(W * tt["surr"]), kl=math.fsum(W * tt["kl"]),
        abs_sum=math.fsum(np.abs(W * tt["j"])),
        clip_frac=(float(tt["clipped"].sum()) / n) if n else 0.0, T=T,
        logp=logp, lse=lse, g=g, rho=tt["rho"], rho_hat=tt["rho_hat"], clipped=tt["clipped"], W=W, A=A, seg=seg)
    if want_dlogits:
        dl = np.empty((n, logits.shape[1]), dtype=np.float64)
        for a in range(0, n, chunk):
            b = min(n, a + chunk)
            z = np.asarray(logits[a:b], dtype=np.float64) / tau
            p = np.exp(z - lse[a:b, None])
            d = -p
            d[np.arange(b - a), y[a:b]] += 1.0
            dl[a:b] = d * (g[a:b, None] / tau)
        out["dlogits"] = dl
    return out


# --------------------------------------------------------------------------
# Step 9 — the same loss with the LM-head projection in front
# --------------------------------------------------------------------------
def lmhead_grpo_loss(hidden, W_head, target, logp_old, logp_ref, cu_seqlens, adv_seg, w_seg,
                     eps_lo=0.2, eps_hi=0.2, beta=0.04, tau=1.0, length_norm=True, seq_log_ratio=None):
    """logits = hidden @ W_head^T (float64 accumulation of the exact bf16 inputs),
    then `grpo_loss`; dhidden = D @ W_head and dW = D^T @ hidden with D the
    float64 dlogits."""
    h = np.asarray(hidden, dtype=np.float64)
    Wm = np.asarray(W_head, dtype=np.float64)
    z = h @ Wm.T
    out = grpo_loss(z, target, logp_old, logp_ref, cu_seqlens, adv_seg, w_seg,
                    eps_lo, eps_hi, beta, tau, want_dlogits=True, length_norm=length_norm,
                    seq_log_ratio=seq_log_ratio)
    D = out["dlogits"]
    out["dhidden"] = D @ Wm
    out["dW"] = D.T @ h
    out["logits"] = z
    return out
