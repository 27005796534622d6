"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own batch, timings combined as
max over ranks and tokens as a sum.  The per-rank work here is the oracle's steps 1-5 (no GPU)."""
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
