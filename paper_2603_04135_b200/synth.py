"""Seeded synthetic inputs with the shapes of the paper's workloads.

This module only draws random inputs (rewards, lengths, logits, sampled token
ids, perturbed old/reference log-probs).  It contains none of the method's
arithmetic: no advantages, masks, packing, log-softmax or loss.  The same bytes
it returns are handed to the CUDA library and to whatever checks it.

The paper trains Qwen3-4B/8B on GSM8K / MATH rollouts (group size 5-16, at most
1024 response tokens, Section 5.1); those are not available offline, so each
config below is a synthetic stand-in with the same structure.
"""
import math
from dataclasses import dataclass, field, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    P: int                    # prompts per batch
    G: int                    # completions per prompt
    V: int                    # vocabulary
    dtype: str                # "f32" | "bf16" logits
    prompt_len: tuple         # ("uniform", lo, hi) | ("lognormal", median, log_sigma, lo, hi) | ("const", n)
    resp_len: tuple
    logit_sigma: float
    target: str               # "softmax": y ~ softmax(z);  "boost": y uniform, z[y] += 4;  "uniform": y uniform
    reward: str               # "bernoulli": r ~ B(0.5);  "beta": per-prompt rate ~ Beta(.5,.5)
    r_q: float                # prompt pruning probability  (= 1 - retention)
    r_o: float                # completion pruning probability
    L_row: int
    N_win: int
    eps: float = 0.2
    beta: float = 0.04
    sigma_old: float = 0.05
    sigma_ref: float = 0.1
    H: int = 0                # hidden width for the fused LM-head workload (0: none)


WORKLOADS = {
    # tiny case a CPU checks in seconds
    "config0": Workload("config0", 4, 4, 1024, "f32", ("uniform", 16, 48), ("uniform", 8, 64),
                        1.0, "softmax", "bernoulli", 0.5, 0.5, 512, 4),
    # Qwen3 vocabulary, bf16
    "config1": Workload("config1", 8, 8, 151936, "bf16", ("uniform", 64, 256), ("uniform", 128, 1024),
                        2.0, "boost", "beta", 0.25, 0.25, 4096, 16),
    # pruning / packing sweep shape (no logits)
    "config2": Workload("config2", 32, 8, 0, "bf16", ("lognormal", 150, 0.6, 32, 512),
                        ("lognormal", 400, 0.6, 32, 2048), 0.0, "uniform", "beta", 0.25, 0.25, 8192, 16),
    # large fused loss pass
    "config3": Workload("config3", 32, 8, 151936, "bf16", ("const", 0), ("uniform", 64, 1024),
                        2.0, "softmax", "beta", 0.25, 0.25, 8192, 16),
    # fused LM-head + loss: about 140 k retained tokens at pruning probabilities 0.5 / 0.5 (seed 4: 130,006)
    "config4_h2560": Workload("config4_h2560", 64, 8, 151936, "bf16", ("const", 0), ("uniform", 64, 1024),
                              1.0, "uniform", "beta", 0.5, 0.5, 8192, 16, H=2560),
    "config4_h4096": Workload("config4_h4096", 64, 8, 151936, "bf16", ("const", 0), ("uniform", 64, 1024),
                              1.0, "uniform", "beta", 0.5, 0.5, 8192, 16, H=4096),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (smaller V, P, ... for tests)."""
    return replace(w, **kw)


def _draw_len(rng, spec, shape):
    kind = spec[0]
    if kind == "const":
        return np.full(shape, spec[1], dtype=np.int32)
    if kind == "uniform":
        return rng.integers(spec[1], spec[2] + 1, size=shape).astype(np.int32)
    if kind == "lognormal":
        _, median, log_sigma, lo, hi = spec
        x = np.exp(rng.normal(math.log(median), log_sigma, size=shape))
        return np.clip(np.rint(x), lo, hi).astype(np.int32)
    raise ValueError(kind)


def _draw_rewards(rng, kind, P, G):
    if kind == "bernoulli":
        rate = np.full(P, 0.5)
    elif kind == "beta":
        rate = rng.beta(0.5, 0.5, size=P)
    else:
        raise ValueError(kind)
    return (rng.random((P, G)) < rate[:, None]).astype(np.float32), rate


@dataclass
class Batch:
    """Host-side per-batch inputs (everything except the logits)."""
    workload: Workload
    seed: int
    rewards: np.ndarray        # f32 [P, G]   this epoch's rewards
    rewards_prev: np.ndarray   # f32 [P, G]   an independent earlier-epoch draw with the same success
                               #              rates; its mean |A| per prompt is the history score (Eq. 16)
    prompt_len: np.ndarray     # i32 [P]
    resp_len: np.ndarray       # i32 [P, G]

    @property
    def unit_len(self):        # i32 [P*G]  prompt + response tokens of each completion
        return (self.prompt_len[:, None] + self.resp_len).reshape(-1).astype(np.int32)

    @property
    def loss_len(self):        # i32 [P*G]  response tokens (the tokens the loss runs over)
        return self.resp_len.reshape(-1).astype(np.int32)


def make_batch(w: Workload, seed: int) -> Batch:
    rng = np.random.default_rng([seed, 0xD990])
    rewards, rate = _draw_rewards(rng, w.reward, w.P, w.G)
    prompt_len = _draw_len(rng, w.prompt_len, (w.P,))
    resp_len = _draw_len(rng, w.resp_len, (w.P, w.G))
    rng_prev = np.random.default_rng([seed + 1000, 0xD990])
    rewards_prev = (rng_prev.random((w.P, w.G)) < rate[:, None]).astype(np.float32)
    return Batch(w, seed, rewards, rewards_prev, prompt_len, resp_len)


def expected_lse(w: Workload) -> float:
    """Mean log-sum-exp of V i.i.d. N(0, sigma^2) logits: sigma^2/2 + ln V.  Used only to
    centre the synthetic old/reference log-probs near the current policy's."""
    return 0.5 * w.logit_sigma ** 2 + math.log(w.V)


@dataclass
class TokenInputs:
    logits: torch.Tensor       # [T, V] f32 or bf16, on `device`
    target: torch.Tensor       # i32 [T]
    logp_old: torch.Tensor     # f32 [T]
    logp_ref: torch.Tensor     # f32 [T]


def make_token_inputs(w: Workload, T: int, seed: int, device="cpu", sigma_old=None, sigma_ref=None,
                      rows_per_chunk=512) -> TokenInputs:
    """Logits for T loss tokens, sampled token ids and perturbed old / reference log-probs.

    logits ~ N(0, logit_sigma^2) i.i.d., rounded to the workload's dtype.  Targets: "softmax" draws
    y ~ softmax(z) by the Gumbel-max trick; "boost" draws y uniformly and adds 4 to z[y]; "uniform"
    draws y uniformly.  logp_old = (z[y] - E[lse]) + N(0, sigma_old), logp_ref likewise with
    sigma_ref, stored as f32: the current policy's log-prob is z[y] - lse, and lse is within a few
    hundredths of its closed-form mean for these sizes.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed((int(seed) * 1000003 + 0x5EED) & 0x7FFFFFFFFFFF)
    tdtype = torch.float32 if w.dtype == "f32" else torch.bfloat16
    logits = torch.empty((T, w.V), dtype=tdtype, device=dev)
    target = torch.empty((T,), dtype=torch.int32, device=dev)
    zy = torch.empty((T,), dtype=torch.float32, device=dev)
    for a in range(0, T, rows_per_chunk):
        b = min(T, a + rows_per_chunk)
        z = torch.randn((b - a, w.V), generator=gen, device=dev, dtype=torch.float32) * w.logit_sigma
        z = z.to(tdtype)
        if w.target == "softmax":
            u = torch.rand((b - a, w.V), generator=gen, device=dev, dtype=torch.float32)
            gumbel = -torch.log(-torch.log(u.clamp_min(1e-20)).clamp_min(1e-20))
            y = torch.argmax(z.float() + gumbel, dim=1)
        else:
            y = torch.randint(0, w.V, (b - a,), generator=gen, device=dev)
            if w.target == "boost":
                idx = torch.arange(b - a, device=dev)
                z[idx, y] = (z[idx, y].float() + 4.0).to(tdtype)
        logits[a:b] = z
        target[a:b] = y.to(torch.int32)
        zy[a:b] = z[torch.arange(b - a, device=dev), y].float()
    so = w.sigma_old if sigma_old is None else sigma_old
    sr = w.sigma_ref if sigma_ref is None else sigma_ref
    centre = zy - expected_lse(w)
    logp_old = centre + so * torch.randn((T,), generator=gen, device=dev, dtype=torch.float32)
    logp_ref = centre + sr * torch.randn((T,), generator=gen, device=dev, dtype=torch.float32)
    return TokenInputs(logits, target, logp_old, logp_ref)


def make_lmhead_inputs(w: Workload, T: int, seed: int, device="cpu"):
    """hidden bf16 [T, H] ~ N(0,1), LM-head weight bf16 [V, H] ~ N(0, 1/H) (so logits ~ N(0,1)), uniform
    targets and old / reference log-probs = z[y] - E[lse] + N(0, sigma)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed((int(seed) * 1000003 + 0x1EAD) & 0x7FFFFFFFFFFF)
    hidden = torch.randn((T, w.H), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    W = torch.empty((w.V, w.H), dtype=torch.bfloat16, device=dev)
    step = 8192
    for a in range(0, w.V, step):
        b = min(w.V, a + step)
        W[a:b] = (torch.randn((b - a, w.H), generator=gen, device=dev, dtype=torch.float32)
                  / math.sqrt(w.H)).to(torch.bfloat16)
    target = torch.randint(0, w.V, (T,), generator=gen, device=dev).to(torch.int32)
    # the sampled token's logit (one dot product per token) minus the closed-form mean log-sum-exp of
    # N(0,1) logits centres the old / reference log-probs near the current policy's
    zy = (hidden.float() * W[target.long()].float()).sum(dim=1)
    centre = zy - expected_lse(w)
    logp_old = centre + w.sigma_old * torch.randn((T,), generator=gen, device=dev, dtype=torch.float32)
    logp_ref = centre + w.sigma_ref * torch.randn((T,), generator=gen, device=dev, dtype=torch.float32)
    return hidden, W, target, logp_old, logp_ref


def to_f64_numpy(t: torch.Tensor) -> np.ndarray:
    """Exact float64 copy of an f32 / bf16 tensor on the host (a dtype widening, nothing else)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
