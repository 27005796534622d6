"""The N > 1 paths on CPU, two gloo ranks each.  (1) The benchmark's form: every rank has its own batch, timings
are combined as max over ranks and tokens as a sum.  (2) Rows sharded over ranks: the small steps repeated on every
rank, each rank's loss over its own packed rows, one all-reduce of the five loss scalars (and of dW) giving the
whole batch's.  The per-rank work here is the oracle's (no GPU)."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    import oracle
    from paper_2603_04135_b200 import dp, synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.WORKLOADS["config2"]
        seed = dp.rank_seed(3, rank)
        batch = synth.make_batch(w, seed)
        adv, mabs = oracle.group_advantages(batch.rewards)
        pr = oracle.prune_and_rescale(adv, mabs, None, w.r_q, w.r_o, seed=seed, step=1)
        pk = oracle.pack_prompts(batch.unit_len, w.L_row, w.N_win, keep=pr["keep_o"].reshape(-1), loss_len=batch.loss_len)
        tokens = pk["counts"][3]
        fake_ms = [10.0 + rank, 5.0 - rank]                    # rank 1 is slower on the first, faster on the second
        times, total = dp.combine_over_ranks(fake_ms, tokens)
        out.put((rank, seed, tokens, times, total))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_combine_max_time_and_total_tokens():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, n0, t0, tot0), (r1, s1, n1, t1, tot1) = res
    assert (s0, s1) == (3, 4) and n0 != n1                      # different batches per rank
    assert t0 == t1 == [11.0, 5.0]                              # max over ranks, element-wise
    assert tot0 == tot1 == float(n0 + n1)                       # tokens add up
    from paper_2603_04135_b200 import dp
    assert dp.throughput(tot0, 10.0) == (n0 + n1) / 0.01


def test_single_process_needs_no_group():
    from paper_2603_04135_b200 import dp
    times, total = dp.combine_over_ranks([3.0, 4.0], 7)
    assert times == [3.0, 4.0] and total == 7.0


# ---- rows sharded over ranks: the five loss scalars and dW combine to the whole batch's ----------------------
def _shard_rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2603_04135_b200 import dp, synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank repeats the small steps on the WHOLE batch from the same seed (no communication) ...
        w = synth.scaled(synth.WORKLOADS["config0"], P=6, G=4, V=96, L_row=160, r_q=0.3, r_o=0.3)
        seed = 12
        batch = synth.make_batch(w, seed)
        adv, mabs = oracle.group_advantages(batch.rewards)
        H_prev = oracle.group_advantages(batch.rewards_prev)[1]
        pr = oracle.prune_and_rescale(adv, mabs, H_prev, w.r_q, w.r_o, seed=seed, step=1)
        pk = oracle.pack_prompts(batch.unit_len, w.L_row, w.N_win, keep=pr["keep_o"].reshape(-1), loss_len=batch.loss_len)
        n_units, n_rows, _, T = pk["counts"]
        order = np.asarray(pk["order"], dtype=np.int64)
        adv_seg = adv.reshape(-1)[order]; w_seg = pr["w_seq"].reshape(-1)[order]
        cu = np.asarray(pk["cu_seqlens"], dtype=np.int64)
        tok = synth.make_token_inputs(w, T, seed, device="cpu", sigma_old=0.3)
        z = tok.logits.double().numpy(); y = tok.target.numpy(); lo = tok.logp_old.numpy(); lr = tok.logp_ref.numpy()
        # ... and takes a contiguous range of the packed rows
        sh = dp.shard_rows([pk["row_of"][u] for u in pk["order"]], pk["cu_seqlens"], n_units, world, rank)
        a, b = sh["tok_lo"], sh["tok_hi"]
        rows = np.arange(a, b)
        part = oracle.grpo_loss(z[a:b], y, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta, rows=rows)
        five = torch.tensor([part["loss"], part["pg"], part["kl"], part["clip_frac"], float(b - a)], dtype=torch.float32)
        dp.all_reduce_loss(five)
        # the LM-head weight gradient of the rank's tokens: one all-reduce makes it the batch's
        rng = np.random.default_rng(5)
        hid = rng.normal(size=(T, 16))
        dW = torch.from_numpy(part["dlogits"].T @ hid[a:b]) if b > a else torch.zeros((w.V, 16), dtype=torch.float64)
        dp.reduce_dW(dW)
        whole = oracle.grpo_loss(z, y, lo, lr, cu, adv_seg, w_seg, w.eps, w.eps, w.beta)
        out.put((rank, sh, five.tolist(), [whole["loss"], whole["pg"], whole["kl"], whole["clip_frac"], float(T)],
                 float(np.abs(dW.numpy() - whole["dlogits"].T @ hid).max()), float(np.abs(whole["dlogits"].T @ hid).max()),
                 n_rows, [pk["row_of"][u] for u in pk["order"]]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_sharded_rows_reduce_to_the_whole_batch():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, sh0, five0, whole0, err0, scale0, n_rows, rows_placed), (_, sh1, five1, whole1, err1, scale1, _, _) = res
    # the two ranges tile the batch at a row boundary, both non-empty
    assert sh0["seq_lo"] == 0 and sh0["seq_hi"] == sh1["seq_lo"] and sh1["seq_hi"] == len(rows_placed)
    assert sh0["tok_hi"] == sh1["tok_lo"] and sh0["tok_hi"] > 0 and sh1["tok_hi"] > sh1["tok_lo"] and n_rows >= 2
    assert rows_placed[sh1["seq_lo"]] != rows_placed[sh1["seq_lo"] - 1] and sh0["row_hi"] == sh1["row_lo"]
    assert five0 == five1                                        # every rank ends with the same five scalars
    for got, want in zip(five0, whole0):
        assert abs(got - want) <= 2e-6 * max(abs(want), 1e-3)    # = the oracle on the whole batch (f32 transport)
    assert five0[4] == whole0[4]
    assert max(err0, err1) <= 1e-12 * scale0


def test_shard_rows_edge_cases():
    from paper_2603_04135_b200 import dp
    # three rows of two units each, 10 tokens per unit; four ranks: one rank comes out empty
    rows = [0, 0, 1, 1, 2, 2]
    cu = [0, 10, 20, 30, 40, 50, 60]
    got = [dp.shard_rows(rows, cu, 6, 4, r) for r in range(4)]
    assert [(g["seq_lo"], g["seq_hi"]) for g in got] == [(0, 2), (2, 4), (4, 6), (6, 6)]
    assert [(g["tok_lo"], g["tok_hi"]) for g in got] == [(0, 20), (20, 40), (40, 60), (60, 60)]
    assert [(g["row_lo"], g["row_hi"]) for g in got] == [(0, 1), (1, 2), (2, 3), (3, 3)]
    one = dp.shard_rows(rows, cu, 6, 1, 0)
    assert (one["seq_lo"], one["seq_hi"], one["tok_lo"], one["tok_hi"]) == (0, 6, 0, 60)
    empty = dp.shard_rows([], [0], 0, 2, 1)
    assert (empty["seq_lo"], empty["seq_hi"], empty["tok_lo"], empty["tok_hi"]) == (0, 0, 0, 0)


def test_all_reduce_loss_single_process_is_identity():
    import torch
    from paper_2603_04135_b200 import dp
    v = torch.tensor([1.0, 2.0, 3.0, 0.25, 8.0])
    assert dp.all_reduce_loss(v) is v and v.tolist() == [1.0, 2.0, 3.0, 0.25, 8.0]
    w = torch.ones(3, 2)
    assert dp.reduce_dW(w) is w
