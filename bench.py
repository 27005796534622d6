#!/usr/bin/env python
"""Benchmark of the pruned-GRPO hot path: valid tokens/s and fraction of the HBM roofline.

One step = one pass of the whole path over one synthetic batch: group advantages -> candidate sets,
pruning masks, rescaling -> Dense Prompt Packing -> fused loss sweep (forward + dlogits).  The
workload is the large fused-loss configuration (32 prompts x 8 completions, 64-1024 response tokens,
bf16 logits over a 151,936-token vocabulary, pruning probabilities 0.25 / 0.25).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched with torch.distributed.run, one rank per GPU; every rank works on its own batch
(no data-path collective) and rank 0 reports the whole-job throughput with the max time over ranks.
`--impl reference` times the float64 CPU oracle on the host cores instead (rank 0 only).

Side modes (each prints its own lines and is not part of the default run):
  --prune-pack-sweep            density / timing table of the pruning and packing sweep shape
  --profile-case loss           a self-contained run of the loss sweep for timing and profiler captures
                                (--rows --vocab --dtype --iters --in-place --full-call --back-to-back --variant)
  --profile-case lmhead         the same for the fused LM-head (--tokens --hidden --vocab --iters --backward --variant)
"""
import argparse
import json
import multiprocessing as mp
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2603_04135_b200 import synth

METRIC = "valid tokens/sec of pruned GRPO loss fwd+bwd"
UNIT = "tokens/s"
WORKLOAD = "config3"
WORKLOAD_TEXT = WORKLOAD + ": P=32 G=8, response 64-1024 tokens, V=151936 bf16 logits, r_q=r_o=0.25, L_row=8192, N_win=16"


# DRAM traffic of the dominant kernel from its last ncu capture:
# dram__bytes_read.sum + dram__bytes_write.sum of one launch over 8192 rows of this vocabulary.  Traffic
# grows in proportion to the rows, so a launch over T rows moves T times the per-row figure.  The record
# is tied to the kernel sources it was taken from: once they change, `traffic` is reported as null.
TRAFFIC_CAPTURE = {"rows": 8192, "dram_bytes": 2489449000 + 2432122000,
                   "source_sha256": "d86ff3052c1d82b57f08f193f805e11838b448ac96fe6cbbd238bb0b51579171"}


def captured_traffic_per_row():
    import hashlib
    base = os.path.join(ROOT, "paper_2603_04135_b200", "csrc")
    try:
        src = b"".join(open(os.path.join(base, f), "rb").read() for f in ("grpo_loss_cluster.cu", "grpo_loss.cuh"))
    except OSError:
        return None
    if hashlib.sha256(src).hexdigest() != TRAFFIC_CAPTURE["source_sha256"]:
        return None
    return TRAFFIC_CAPTURE["dram_bytes"] / TRAFFIC_CAPTURE["rows"]


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.3)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------- oracle legs
def oracle_prune_pack(w, batch, seed, step):
    import oracle
    adv, mabs = oracle.group_advantages(batch.rewards)
    H_prev = oracle.group_advantages(batch.rewards_prev)[1]
    pr = oracle.prune_and_rescale(adv, mabs, H_prev, w.r_q, w.r_o, seed=seed, step=step)
    pk = oracle.pack_prompts(batch.unit_len, w.L_row, w.N_win, keep=pr["keep_o"].reshape(-1), loss_len=batch.loss_len)
    order = np.asarray(pk["order"], dtype=np.int64)
    return pk, adv.reshape(-1)[order], pr["w_seq"].reshape(-1)[order]


def oracle_sample_tasks(w, tok_cpu, rows, pk, adv_seg, w_seg, rows_per_task):
    is_bf16 = tok_cpu.logits.dtype == torch.bfloat16
    T = pk["counts"][3]
    target = np.zeros(T, dtype=np.int64); lo = np.zeros(T); lr = np.zeros(T)
    target[rows] = tok_cpu.target.numpy(); lo[rows] = tok_cpu.logp_old.numpy(); lr[rows] = tok_cpu.logp_ref.numpy()
    cu = np.asarray(pk["cu_seqlens"])
    tasks = []
    for a in range(0, len(rows), rows_per_task):
        b = min(len(rows), a + rows_per_task)
        blk = tok_cpu.logits[a:b]
        chunk = blk.view(torch.int16).numpy().view(np.uint16) if is_bf16 else blk.numpy()
        tasks.append((chunk, is_bf16, rows[a:b], target, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta, 1.0))
    return tasks


def time_oracle(w, seed, n_rows, steps, warmup, pool, cores):
    """Times the oracle as it stands: steps 1-5 on the full batch, then loss forward + backward on a
    bounded sample of n_rows token rows spread over `cores` worker processes."""
    from oracle import rows_worker
    batch = synth.make_batch(w, seed)
    pk, adv_seg, w_seg = oracle_prune_pack(w, batch, seed, 1)
    T = pk["counts"][3]
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(T, size=min(n_rows, T), replace=False))
    tok = synth.make_token_inputs(w, len(rows), seed, device="cpu", rows_per_chunk=64)
    tasks = oracle_sample_tasks(w, tok, rows, pk, adv_seg, w_seg, max(1, len(rows) // (cores * 2)))
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        oracle_prune_pack(w, batch, seed, 1)
        done = sum(r[2] for r in pool.map(rows_worker.fwd_bwd_rows, tasks))
        dt = time.perf_counter() - t0
        assert done == len(rows)
        if it >= warmup:
            times.append(dt)
    return len(rows), T, times


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    w = synth.WORKLOADS[WORKLOAD]
    cores = min(os.cpu_count() or 1, 64)
    with mp.get_context("spawn").Pool(cores) as pool:
        n_rows, T, times = time_oracle(w, 3, args.ref_rows, args.steps, args.warmup, pool, cores)
    ms = 1e3 * sum(times) / len(times)
    value = n_rows / (ms / 1e3)
    sample = "%d of the batch's %d retained token rows per step (fwd+bwd, V=%d) plus steps 1-5 on the full batch" % (
        n_rows, T, w.V)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT + "; CPU oracle on a row sample", "rows_per_step": n_rows},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def bf16_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured sustained cuBLAS bf16"
    except Exception:
        return 1400.0, "fallback sustained"


def time_lmhead(H, dev, gpu_index, iters=10, warmup=3, sample_clocks=True):
    """The fused LM-head configuration as stated: a batch of 64 prompts x 8 completions (64-1024 response tokens)
    goes through advantages -> pruning with probabilities 0.5 / 0.5 -> packing, and the fused LM-head + loss runs on
    the retained tokens with the packer's cu_seqlens, placement order and device-side token count and the
    library's own advantages and sequence weights.  Forward + backward (dhidden, dW) and forward only, each timed
    with CUDA events over `iters` calls after `warmup`, with the clocks sampled during the timed calls."""
    from paper_2603_04135_b200 import binding as B
    from paper_2603_04135_b200.step import DppoStep
    w = synth.WORKLOADS["config4_h%d" % H]
    seed = 4
    batch = synth.make_batch(w, seed)
    T_cap = int(batch.loss_len.sum())
    st = DppoStep(w.P, w.G, w.L_row, w.N_win, w.r_q, w.r_o, w.V, w.dtype, T_cap, w.eps, w.eps, w.beta, device=dev)
    prev = torch.from_numpy(batch.rewards_prev.reshape(-1).copy()).to(dev)
    H_prev = torch.zeros(w.P, device=dev); scratch = torch.zeros(w.P * w.G, device=dev)
    st.advantages(rewards=prev, adv=scratch, mean_abs_adv=H_prev)          # history scores: the earlier epoch's mean |A|
    st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, H_prev)
    st.prune_pack(seed=seed, step=1)
    T = st.n_tokens()
    S = int(st.counts[0].item())
    assert st.status.item() == 0 and 0 < T <= T_cap
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, seed, device=dev)   # exactly the retained tokens
    V = w.V

    def params(backward):
        return B.LmheadParams(B.LossParams(T, V, B.BF16, V, w.P * w.G, 0, w.eps, w.eps, w.beta, 1.0), H, backward)

    nbytes = max(B.lmhead_workspace_bytes(params(1)), B.lmhead_workspace_bytes(params(0)))
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device=dev)
    ws = ws[(-ws.data_ptr()) % 1024:]
    dh = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
    dW = torch.empty((V, H), dtype=torch.float32, device=dev)

    def timed(backward):
        prm = params(backward)
        sampler = ClockSampler(gpu_index)
        times = []
        for it in range(warmup + iters):
            if it == warmup and sample_clocks:
                torch.cuda.synchronize()
                sampler.start()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            B.lmhead_grpo_loss(prm, hidden, W, target, lo, lr, st.cu_seqlens, st.counts[3:4], st.adv, st.w_seq, st.order,
                               dh if backward else None, dW if backward else None, None, None, st.loss_out, ws, nbytes,
                               st.status)
            e1.record()
            times.append((e0, e1))
        torch.cuda.synchronize()
        clocks = sampler.stop() if sample_clocks else None
        assert st.status.item() == 0 and st.loss_out[4].item() == T
        ms = [a.elapsed_time(b) for a, b in times[warmup:]]
        return sum(ms) / len(ms), min(ms), clocks

    ms, ms_min, clocks = timed(1)
    ms_f, ms_f_min, clocks_f = timed(0)
    peak, peak_kind = bf16_peak()
    executed = 6.0 * T * V * H / ms / 1e9
    fwd = 2.0 * T * V * H / ms_f / 1e9
    return {"config": {"workload": "config4_h%d: P=%d G=%d, response 64-1024 tokens, pruning probabilities r_q=r_o=%.2f "
                                   "(retention 0.5 / 0.5) through prune -> pack; bf16 hidden [%d x %d], W [%d x %d]"
                                   % (H, w.P, w.G, w.r_q, T, H, V, H),
                       "valid_tokens": T, "sequences_retained": S, "unpruned_tokens": T_cap,
                       "calls_timed": iters, "warmup": warmup},
            "ms": ms, "ms_min": ms_min, "tokens_per_s": T / ms * 1e3, "executed_tflops": executed, "model_tflops_6TVH": executed,
            "clocks": clocks,
            "forward_only": {"ms": ms_f, "ms_min": ms_f_min, "tokens_per_s": T / ms_f * 1e3, "executed_tflops_2TVH": fwd,
                             "frac_of_peak": fwd / peak, "clocks": clocks_f},
            "roofline": {"bound": "tensor", "achieved": executed, "peak": peak, "unit": "TFLOP/s", "frac": executed / peak,
                         "peak_source": peak_kind,
                         "note": "executed flops = 6 T V H: logits, dhidden, dW (a chunk's exponentials are kept as bf16, nothing is recomputed)"}}


def time_row_length(dtype, V, rows, dev, iters=8, warmup=3):
    """The loss sweep (forward + dlogits, the call a training step makes: device-side token count, sequence map,
    log-prob and lse outputs) on `rows` rows of another vocabulary size, with the library's own kernel choice:
    `iters` back-to-back calls after `warmup`, CUDA events around each."""
    from paper_2603_04135_b200 import binding as B
    w = synth.scaled(synth.WORKLOADS["config3"], V=V, dtype=dtype)
    S = 2000
    tok = synth.make_token_inputs(w, rows, 0, device=dev)
    rng = np.random.default_rng(0)
    cu = torch.from_numpy(np.linspace(0, rows, S + 1).astype(np.int32)).to(dev)
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).to(dev)
    wseq = torch.full((S,), 1.0 / S, device=dev)
    dl = torch.empty_like(tok.logits)
    prm = B.LossParams(rows, V, B.BF16 if dtype == "bf16" else B.F32, V, S, 0, w.eps, w.eps, w.beta, 1.0)
    ch = B.grpo_loss_kernel_choice(prm)
    nbytes = B.grpo_loss_workspace_bytes(prm)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
    loss_out = torch.zeros(5, device=dev); status = torch.zeros(1, dtype=torch.int32, device=dev)
    ntd = torch.tensor([rows], dtype=torch.int32, device=dev)
    seg_map = torch.arange(S, dtype=torch.int32, device=dev)
    logp_out = torch.zeros(rows, device=dev); lse_out = torch.zeros(rows, device=dev)
    evs = []
    for it in range(warmup + iters):
        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_.record()
        B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, ntd, adv, wseq, seg_map, dl,
                            logp_out, lse_out, loss_out, ws, nbytes, status)
        b_.record()
        evs.append((a_, b_))
    torch.cuda.synchronize()
    assert status.item() == 0
    ms = sum(x.elapsed_time(y) for x, y in evs[warmup:]) / iters
    esize = 2 if dtype == "bf16" else 4
    gbs = 2.0 * rows * V * esize / (ms / 1e3) / 1e9
    peak, _ = measured_peaks()
    return {"dtype": dtype, "V": V, "row_bytes": V * esize, "rows": rows, "kernel": B.KERNEL_NAMES[ch.kernel],
            "ctas_per_row": ch.ctas_per_row, "ms": ms, "achieved_gbs": gbs, "frac": gbs / peak,
            "tokens_per_s": rows / ms * 1e3}


# --------------------------------------------------------------------------------------- profile cases
def run_profile_case(args):
    """A small, self-contained run of one entry point for timing and profiler captures: prints the event-timed
    duration of each call.  `loss`: dppo_grpo_loss_fwd_bwd on --rows token rows of the large-vocabulary workload
    (bf16 logits, V = 151,936: 2.5 GB in + 2.5 GB out at 8192 rows, well above L2 yet small enough for a multi-pass
    capture).  `lmhead`: dppo_lmhead_grpo_loss on --tokens tokens (2 T V H flops forward, 6 T V H with --backward)."""
    from paper_2603_04135_b200 import binding as B
    torch.cuda.set_device(0)
    rng = np.random.default_rng(0)
    if args.profile_case == "loss":
        w = synth.scaled(synth.WORKLOADS["config3"], V=args.vocab, dtype=args.dtype)
        T, S = args.rows, args.seqs
        tok = synth.make_token_inputs(w, T, 0, device="cuda")
        cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
        adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
        wseq = torch.full((S,), 1.0 / S, device="cuda")
        per16 = 8 if args.dtype == "bf16" else 4                  # rows start on 16-byte boundaries: pad the pitch
        stride = -(-w.V // per16) * per16
        if stride != w.V:
            padded = torch.zeros((T, stride), dtype=tok.logits.dtype, device="cuda")
            padded[:, :w.V] = tok.logits
            tok.logits = padded
        dl = tok.logits if args.in_place else torch.empty_like(tok.logits)
        prm = B.LossParams(T, w.V, B.BF16 if args.dtype == "bf16" else B.F32, stride, S, args.variant, w.eps, w.eps, w.beta, 1.0)
        ch = B.grpo_loss_kernel_choice(prm, forward_only=args.forward_only)
        print("kernel: %s, %d CTA(s) per row, %d threads%s" % (B.KERNEL_NAMES[ch.kernel], ch.ctas_per_row, ch.threads,
                                                                  " (fell back)" if ch.fell_back else ""))
        nbytes = B.grpo_loss_workspace_bytes(prm)
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        loss_out = torch.zeros(5, device="cuda"); status = torch.zeros(1, dtype=torch.int32, device="cuda")
        esize = 2 if args.dtype == "bf16" else 4
        ntd = seg_map = logp_out = lse_out = None
        if args.full_call:      # everything the training step passes: device token count, seg_map, logp / lse outputs
            ntd = torch.tensor([T], dtype=torch.int32, device="cuda")
            seg_map = torch.arange(S, dtype=torch.int32, device="cuda")
            logp_out = torch.zeros(T, device="cuda"); lse_out = torch.zeros(T, device="cuda")
        events = []
        for it in range(args.iters):
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            B.grpo_loss_fwd_bwd(prm, tok.logits, tok.target, tok.logp_old, tok.logp_ref, cu, ntd, adv, wseq, seg_map,
                                None if args.forward_only else dl, logp_out, lse_out, loss_out, ws, nbytes, status)
            e1.record()
            events.append((e0, e1))
            if not args.back_to_back:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        per_row = (1 if args.forward_only else 2) * w.V * esize
        for it, (e0, e1) in enumerate(events):
            ms = e0.elapsed_time(e1)
            print("iter %d: %.3f ms  %.1f GB/s algorithmic  loss %.6g  status %d" % (
                it, ms, T * per_row / ms / 1e6, loss_out[0].item(), status.item()))
        assert status.item() == 0
        return 0
    w = synth.scaled(synth.WORKLOADS["config4_h2560"], V=args.vocab, H=args.hidden)
    T, S = args.tokens, args.seqs
    hidden, W, target, lo, lr = synth.make_lmhead_inputs(w, T, 0, device="cuda")
    cu = torch.from_numpy(np.linspace(0, T, S + 1).astype(np.int32)).cuda()
    adv = torch.from_numpy(rng.normal(size=S).astype(np.float32)).cuda()
    wseq = torch.full((S,), 1.0 / S, device="cuda")
    prm = B.LmheadParams(B.LossParams(T, w.V, B.BF16, w.V, S, 0, w.eps, w.eps, w.beta, 1.0), w.H, int(args.backward), args.variant)
    nbytes = B.lmhead_workspace_bytes(prm)
    ws = torch.zeros(nbytes + 1024, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 1024:]
    dh = torch.empty((T, w.H), dtype=torch.bfloat16, device="cuda") if args.backward else None
    dW = torch.empty((w.V, w.H), dtype=torch.float32, device="cuda") if args.backward else None
    loss_out = torch.zeros(5, device="cuda"); status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flops = (6.0 if args.backward else 2.0) * T * w.V * w.H          # logits, dhidden, dW: 2 T V H each
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
    return 0


# --------------------------------------------------------------------------------------- pruning / packing sweep
def run_prune_pack_sweep(args):
    """The pruning / packing sweep shape (32 x 8 completions, log-normal lengths, rows of 8192): for every
    (r_q, r_o, N_win) cell the valid-token density of the packed rows against per-sequence padding to the longest
    retained unit, the device time of advantages + prune + pack (CUDA events, median of 20) and the oracle's time
    for the same three steps on one host core.  Prints one JSON line; not part of the default run."""
    import oracle
    from paper_2603_04135_b200.step import DppoStep
    torch.cuda.set_device(0)
    w = synth.WORKLOADS["config2"]
    batch = synth.make_batch(w, 2)
    cells = []
    for r_q in (0.0, 0.25, 0.5):
        for r_o in (0.0, 0.25, 0.5):
            for N_win in (4, 16, 64):
                st = DppoStep(w.P, w.G, w.L_row, N_win, r_q, r_o, 1, "bf16", 1, w.eps, w.eps, w.beta)
                H_prev = oracle.group_advantages(batch.rewards_prev)[1]
                st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, H_prev)
                times = []
                for it in range(25):
                    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                    e0.record(); st.prune_pack(seed=2, step=11); e1.record()
                    torch.cuda.synchronize()
                    if it >= 5:
                        times.append(e0.elapsed_time(e1) * 1e3)
                n_units, n_rows, tokens, _ = (int(x) for x in st.counts.cpu().numpy())
                keep = st.keep_o.cpu().numpy() == 1
                t0 = time.perf_counter()
                for _ in range(5):
                    adv, mabs = oracle.group_advantages(batch.rewards)
                    pr = oracle.prune_and_rescale(adv, mabs, H_prev, r_q, r_o, seed=2, step=11)
                    oracle.pack_prompts(batch.unit_len, w.L_row, N_win, keep=pr["keep_o"].reshape(-1), loss_len=batch.loss_len)
                cpu_us = (time.perf_counter() - t0) / 5 * 1e6
                cells.append({"r_q": r_q, "r_o": r_o, "N_win": N_win, "units": n_units, "rows": n_rows, "tokens": tokens,
                              "density_packed": tokens / (n_rows * w.L_row) if n_rows else None,
                              "density_padded": tokens / (n_units * int(batch.unit_len[keep].max())) if n_units else None,
                              "gpu_us": statistics.median(times), "oracle_us_1core": cpu_us})
    print(json.dumps({"sweep": "config2: P=32 G=8, log-normal lengths, L_row=8192; advantages + prune + pack", "cells": cells}))
    return 0


# --------------------------------------------------------------------------------------- ours
def run_ours(args):
    if not os.path.exists(os.path.join(ROOT, "paper_2603_04135_b200", "libdppo.so")):
        from paper_2603_04135_b200 import build          # a checkout without the built library: compile it in-tree
        build.build_library()
    from paper_2603_04135_b200.step import DppoStep      # raises if libdppo.so is missing: no fallback
    from paper_2603_04135_b200 import dp

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    # CPU-baseline pool first (spawned workers; never forked after CUDA is up)
    pool, cores = None, 0
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = min(os.cpu_count() or 1, 64)
        pool = mp.get_context("spawn").Pool(cores)

    w = synth.WORKLOADS[WORKLOAD]
    seed = dp.rank_seed(3, rank)                          # every rank has its own batch (data parallel)
    batch = synth.make_batch(w, seed)

    T_cap = int(batch.loss_len.sum())                     # unpruned upper bound of loss tokens
    st = DppoStep(w.P, w.G, w.L_row, w.N_win, w.r_q, w.r_o, w.V, w.dtype, T_cap, w.eps, w.eps, w.beta, device=dev)
    # history scores: the previous epoch's mean |A| per prompt (Eq. 16), produced by the library itself
    prev = torch.from_numpy(batch.rewards_prev.reshape(-1).copy()).to(dev)
    H_prev = torch.zeros(w.P, device=dev); scratch = torch.zeros(w.P * w.G, device=dev)
    st.advantages(rewards=prev, adv=scratch, mean_abs_adv=H_prev)
    st.set_batch(batch.rewards, batch.unit_len, batch.loss_len, H_prev)
    st.prune_pack(seed=seed, step=1)
    T = st.n_tokens()
    assert st.status.item() == 0 and 0 < T <= T_cap
    free, _ = torch.cuda.mem_get_info()
    need = 2 * T * w.V * 2 + (4 << 30)
    if need > free:
        raise RuntimeError("not enough device memory for %s: need %.1f GB, free %.1f GB" % (WORKLOAD, need / 1e9, free / 1e9))
    tok = synth.make_token_inputs(w, T, seed, device=dev)
    dlogits = torch.empty_like(tok.logits)
    st.loss_params.T_max = T          # the logits hold exactly the retained tokens (the same pruning every step)

    def one_step(ev0=None, ev1=None):
        st.prune_pack(seed=seed, step=1)
        if ev0 is not None:
            ev0.record()
        st.loss(tok.logits, tok.target, tok.logp_old, tok.logp_ref, dlogits)
        if ev1 is not None:
            ev1.record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0 and not args.no_clock_sampling:
        sampler.start()
    k_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        one_step(*k_ev[i])
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = e0.elapsed_time(e1)
    loss_ms = sum(a.elapsed_time(b) for a, b in k_ev) / args.steps
    assert st.status.item() == 0
    loss_value = float(st.loss_out[0].item())

    # ---- the same kernel in its other modes (rank 0 of a single-GPU run; a few calls each, CUDA events)
    modes = other_rows = None
    if rank == 0 and world == 1 and not args.no_modes:
        from paper_2603_04135_b200 import binding as B

        def timed_calls(fn, n=5, warm=2):
            evs = []
            for it in range(warm + n):
                a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a_.record(); fn(); b_.record()
                evs.append((a_, b_))
            torch.cuda.synchronize()
            assert st.status.item() == 0
            return sum(x.elapsed_time(y) for x, y in evs[warm:]) / n

        slr = torch.zeros(w.P * w.G, device=dev)

        def seq_ratio_step():
            # sequence-level ratio: a forward-only sweep for the current log-probs, their per-sequence mean
            # log-ratio, then the gradient sweep with that ratio (the logits are read twice)
            st.loss_params.seq_log_ratio = None
            st.loss(tok.logits, tok.target, tok.logp_old, tok.logp_ref, None)
            B.sequence_log_ratio(st.logp_out, tok.logp_old, st.cu_seqlens, w.P * w.G, slr, st.status)
            st.loss_params.seq_log_ratio = slr.data_ptr()
            st.loss(tok.logits, tok.target, tok.logp_old, tok.logp_ref, dlogits)
            st.loss_params.seq_log_ratio = None

        peak_m, _ = measured_peaks()
        vb = w.V * 2
        modes = {}
        for name, fn, bytes_per_token in (
                ("forward_only", lambda: st.loss(tok.logits, tok.target, tok.logp_old, tok.logp_ref, None), vb),
                ("seq_ratio", seq_ratio_step, 3 * vb),
                ("in_place", lambda: st.loss(dlogits, tok.target, tok.logp_old, tok.logp_ref, dlogits), 2 * vb)):
            if name == "in_place":
                dlogits.copy_(tok.logits)                     # the in-place form overwrites its input
            ms_mode = timed_calls(fn)
            gbs = T * bytes_per_token / (ms_mode / 1e3) / 1e9
            modes[name] = {"ms": ms_mode, "algorithmic_bytes_per_token": bytes_per_token, "achieved_gbs": gbs,
                           "frac": gbs / peak_m, "tokens_per_s": T / ms_mode * 1e3}
        modes["in_place"]["note"] = "dlogits written over the logits; after the first call the input is the previous gradient"
        modes["seq_ratio"]["note"] = "forward-only sweep + per-sequence mean log-ratio + gradient sweep: two reads, one write"
        modes["forward_only"]["kernel"] = B.KERNEL_NAMES[B.grpo_loss_kernel_choice(st.loss_params, forward_only=True).kernel]
        ch = B.grpo_loss_kernel_choice(st.loss_params)
        modes["kernel_choice"] = {"kernel": B.KERNEL_NAMES[ch.kernel], "ctas_per_row": ch.ctas_per_row, "threads": ch.threads,
                                  "fell_back_to_general_kernel": bool(ch.fell_back)}

        # ---- the same entry point on other row lengths (about 2 GB of logits each): the short-row and mid-row kernels
        other_rows = [time_row_length(dt, V_, n_, dev) for dt, V_, n_ in
                      (("bf16", 1024, 1000000), ("bf16", 4096, 250000), ("f32", 2048, 250000), ("bf16", 32768, 40000))]
        torch.cuda.empty_cache()

    # ---- end to end: host buffers in, loss scalars out, through DppoStep.step_from_host
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    # pinned host copy of the step's inputs; when all ranks together would pin more than half of the
    # host's memory (or pinning fails) the logits come from a pinned window that is copied repeatedly
    logits_bytes = tok.logits.numel() * tok.logits.element_size()
    try:
        import psutil
        host_total = psutil.virtual_memory().total
    except Exception:
        host_total = 64 << 30
    rows_host = T
    if world * logits_bytes > host_total // 2:
        rows_host = max(1, int((host_total // (4 * world)) // (w.V * 2)))
    host_buffer = "full copy of the inputs"
    while True:
        try:
            host_tok = {k: torch.empty((min(rows_host, T),) + tuple(getattr(tok, k).shape[1:]), dtype=getattr(tok, k).dtype,
                                       pin_memory=True) for k in ("logits", "target", "logp_old", "logp_ref")}
            break
        except RuntimeError:
            if rows_host <= 1024:
                raise
            rows_host //= 2
    if rows_host < T:
        host_buffer = "pinned window of %d rows copied repeatedly (host memory)" % rows_host
    for k in host_tok:
        host_tok[k].copy_(getattr(tok, k)[:host_tok[k].shape[0]])
    dev_tok = {k: getattr(tok, k) for k in host_tok}
    host_batch = {"rewards": torch.from_numpy(batch.rewards.reshape(-1).copy()).pin_memory(),
                  "unit_len": torch.from_numpy(batch.unit_len.copy()).pin_memory(),
                  "loss_len": torch.from_numpy(batch.loss_len.copy()).pin_memory(),
                  "H_prev": H_prev.cpu().pin_memory()}
    st.step_from_host(host_batch, host_tok, dev_tok, seed, 1, dlogits)          # warm-up
    barrier()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(e2e_steps):
        out_host, h2d, d2h = st.step_from_host(host_batch, host_tok, dev_tok, seed, 1, dlogits)
    t1.record()
    barrier()
    e2e_ms = t0.elapsed_time(t1) / e2e_steps
    del host_tok

    # ---- the optional fused LM-head path on the same token count (Qwen3-4B width): forward + backward
    lm = lm_wide = None
    if rank == 0 and not args.no_lmhead:
        del tok, dlogits, dev_tok
        torch.cuda.empty_cache()
        lm = time_lmhead(2560, dev, local_rank, sample_clocks=not args.no_clock_sampling)
        torch.cuda.empty_cache()
        lm_wide = time_lmhead(4096, dev, local_rank, sample_clocks=not args.no_clock_sampling)
    # ---- max over ranks, totals over ranks
    (total_ms, loss_ms, e2e_ms), T_all = dp.combine_over_ranks([total_ms, loss_ms, e2e_ms], T, device=dev)

    if rank == 0:
        ms_per_step = total_ms / args.steps
        peak, peak_kind = measured_peaks()
        bytes_per_token = w.V * 2 + w.V * 2               # read the bf16 logits once, write bf16 dlogits once
        achieved = T * bytes_per_token / (loss_ms / 1e3) / 1e9
        line = {
            "metric": METRIC, "value": dp.throughput(T_all, ms_per_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT, "valid_tokens_per_gpu": T,
                       "sequences_retained": int(st.counts[0].item()),
                       "arithmetic": "bf16 logits and dlogits, f32 row sums, f64 per-token scalar stage and loss sum",
                       "l2": "inputs (%.1f GB) far larger than L2; no flush" % (T * w.V * 2 / 1e9),
                       "parallelism": "dp%d, independent batches" % world},
            "clocks": clocks,
            "e2e": {"value": dp.throughput(T_all, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "host_buffer": host_buffer},
            "gpu_launches": 6 * args.steps,
            "roofline": {"bound": "hbm", "kernel": "grpo loss sweep (rows kernel + its two-launch reduction)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": peak_kind + " STREAM-style copy", "kernel_ms": loss_ms,
                         "algorithmic_bytes_per_token": bytes_per_token,
                         "traffic": (captured_traffic_per_row() * T) if captured_traffic_per_row() else None,
                         "traffic_note": "ncu dram bytes of an 8192-row capture of the same kernel, scaled by rows"},
            "loss": loss_value,
        }
        if modes is not None:
            line["roofline"]["kernel_choice"] = modes.pop("kernel_choice")
            line["loss_sweep_modes"] = modes
            line["loss_sweep_other_row_lengths"] = other_rows
        if lm is not None:
            line["lmhead"] = lm
            line["lmhead_h4096"] = lm_wide
        if pool is not None:
            n_rows, _, times = time_oracle(w, seed, args.ref_rows, 1, 0, pool, cores)
            pool.close(); pool.join()
            line["cpu_baseline"] = {"value": n_rows / times[0], "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": "%d of %d retained token rows, fwd+bwd, plus steps 1-5 on the full batch"
                                              % (n_rows, T)}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-rows", type=int, default=2048, help="token rows in the oracle's timed sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lmhead", action="store_true", help="skip the fused LM-head measurement")
    ap.add_argument("--no-modes", action="store_true", help="skip the forward-only / in-place / sequence-ratio timings")
    ap.add_argument("--profile-case", choices=["loss", "lmhead"], help="instead of the benchmark: a small self-contained run")
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--tokens", type=int, default=16384)
    ap.add_argument("--hidden", type=int, default=2560)
    ap.add_argument("--vocab", type=int, default=151936)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--seqs", type=int, default=16)
    ap.add_argument("--variant", type=int, default=0, help="kernel variant of the profile case (see include/dppo.h)")
    ap.add_argument("--in-place", action="store_true")
    ap.add_argument("--forward-only", action="store_true")
    ap.add_argument("--full-call", action="store_true")
    ap.add_argument("--back-to-back", action="store_true", help="enqueue all iterations before synchronising")
    ap.add_argument("--backward", action="store_true", help="lmhead profile case: also dhidden and dW")
    ap.add_argument("--no-clock-sampling", action="store_true", help="do not poll nvidia-smi during the timed region")
    ap.add_argument("--prune-pack-sweep", action="store_true",
                    help="instead of the benchmark: density and timing table of the pruning / packing sweep shape")
    args = ap.parse_args()
    if args.prune_pack_sweep:
        sys.exit(run_prune_pack_sweep(args))
    if args.profile_case:
        sys.exit(run_profile_case(args))
    if args.impl == "ours" and args.warmup < 3:
        args.warmup = 3
    sys.exit(run_reference(args) if args.impl == "reference" else run_ours(args))


if __name__ == "__main__":
    main()
