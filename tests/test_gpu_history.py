"""Several epochs of prompt / completion pruning with the dataset-wide history table (Eq. 16, Algorithm 1):
the library's epoch driver (gather -> advantages -> prune -> scatter -> pack per batch) against the oracle's loop,
bit for bit."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [0, 1])
def test_epochs_with_history_table_match_oracle(mode):
    from paper_2603_04135_b200 import binding as B
    N, G, P, epochs = 96, 8, 32, 4
    r_q, r_o, seed = 0.5, 0.5, 17
    rng = np.random.default_rng(5)
    rate = rng.beta(0.5, 0.5, size=N)
    rewards = [(rng.random((N, G)) < rate[:, None]).astype(np.float32) for _ in range(epochs)]
    batches = []
    for t in range(epochs):
        perm = rng.permutation(N)
        batches.append([perm[i:i + P].tolist() for i in range(0, N, P)])
    table_ref, log = oracle.history_epochs(rewards, batches, N, G, r_q, r_o, seed=seed, mode=mode)

    # the library's epoch driver owns the table and issues gather -> advantages -> prune -> scatter (-> pack) per batch
    from paper_2603_04135_b200.step import DppoStep
    st = DppoStep(P, G, 4096, 8, r_q, r_o, 1, "bf16", 1, mode=mode)
    lens = rng.integers(16, 400, size=(N, G)).astype(np.int32)
    seen = []

    def on_batch(t, b, step):
        ref = log[len(seen)]
        seen.append((t, b))
        assert np.array_equal(step.keep_q.cpu().numpy(), ref["keep_q"])
        assert np.array_equal(step.keep_o.cpu().numpy(), ref["keep_o"].reshape(-1))
        assert np.array_equal(step.cand_q.cpu().numpy(), ref["cand_q"])
        assert np.array_equal(step.w_seq.cpu().numpy().view(np.uint32), ref["w_seq"].reshape(-1).view(np.uint32))
        ids = batches[t][b]
        pk = oracle.pack_prompts(lens[ids].reshape(-1), 4096, 8, keep=ref["keep_o"].reshape(-1))
        assert tuple(int(x) for x in step.counts.cpu().numpy()) == tuple(pk["counts"])
        assert list(step.order.cpu().numpy()[:pk["counts"][0]]) == list(pk["order"])

    table = st.run_epochs(N, batches, lambda t, ids: rewards[t][ids], seed,
                          lengths_fn=lambda t, ids: (lens[ids].reshape(-1), lens[ids].reshape(-1)), on_batch=on_batch)
    assert len(seen) == epochs * (N // P) and st.status.item() == 0
    assert np.array_equal(table.cpu().numpy().view(np.uint32), table_ref.view(np.uint32))
    f32 = dict(dtype=torch.float32, device="cuda"); i32 = dict(dtype=torch.int32, device="cuda")
    status = st.status
    # an id outside the table is reported, not dereferenced
    bad = torch.tensor([0, N, 5, -1], **i32)
    out = torch.full((4,), 7.0, **f32)
    B.history_gather(table, N, bad, 4, out, status)
    assert status.item() == B.STATUS_BAD_INDEX and out[1].item() == 0 and out[3].item() == 0
    status.zero_()
    B.history_scatter(table, N, bad, 4, out, status)
    assert status.item() == B.STATUS_BAD_INDEX


@pytest.mark.parametrize("b,r", [(0.5, 0.7), (0.5, 0.9), (0.5, 0.5)])
def test_prompt_rescaling_second_moment_matches_theorem_d1(b, r):
    """Appendix D.3's closed form for the variance inflation of prompt-level rescaling, E_{q ~ pruned}[gamma(q)^2] =
    (1 - b r)(1 - (1 - b) r)/(1 - r), on the library's gamma_q: explicit draws retain exactly the expected number of
    candidates, so |S^q|/P = 1 - b r and the mean of gamma_q^2 over the retained prompts is the closed form."""
    from paper_2603_04135_b200 import binding as B
    P, G = 40, 2
    n_cand = P // 2                                          # the library takes floor(P/2) candidates: b = 0.5
    n_keep_c = round(n_cand * (1 - r))
    H = np.arange(P, dtype=np.float32)                       # prompts 0 .. n_cand-1 rank lowest
    u_q = np.full(P, 0.999); u_q[n_keep_c:n_cand] = 0.0      # the last candidates are pruned
    f32 = dict(dtype=torch.float32, device="cuda"); i32 = dict(dtype=torch.int32, device="cuda"); u8 = dict(dtype=torch.uint8, device="cuda")
    adv = torch.zeros(P * G, **f32); mabs = torch.zeros(P, **f32)
    cand_q = torch.zeros(P, **u8); cand_o = torch.zeros(P * G, **u8); keep_q = torch.zeros(P, **u8); keep_o = torch.zeros(P * G, **u8)
    nq = torch.zeros(1, **i32); no = torch.zeros(P, **i32)
    gq = torch.zeros(P, **f32); go = torch.zeros(P * G, **f32); ws = torch.zeros(P * G, **f32); H_next = torch.zeros(P, **f32)
    prm = B.PruneParams(P, G, r, 0.0, 0, 0, 0, 0)
    B.prune_and_rescale(prm, adv, mabs, torch.from_numpy(H).cuda(), torch.from_numpy(u_q).cuda(),
                        torch.ones(P * G, dtype=torch.float64, device="cuda"), cand_q, cand_o, keep_q, keep_o, nq, no,
                        gq, go, ws, H_next)
    kept = keep_q.cpu().numpy() == 1
    assert cand_q.cpu().numpy()[:n_cand].all() and kept.sum() == P - n_cand + n_keep_c
    factor = float((gq.cpu().numpy()[kept].astype(np.float64) ** 2).mean())
    closed = (1 - b * r) * (1 - (1 - b) * r) / (1 - r)
    assert abs(factor - closed) <= 1e-6 * closed
