"""dppo_pack_prompts_static — packing for callers that cannot supply device scratch.

Some users of this library call the packer from a place where they have nothing to allocate with: a
plug-in that a framework hands only input and output buffers, or a training loop whose device memory
is fully reserved by a pool, where cudaMalloc would fail or stall all streams.  For them the library
carries a fixed scratch array of its own.  This test drives that entry point through the C ABI and
requires exactly the layout the workspace-taking entry point produces (integer outputs: bit for bit),
on two calls in a row with different inputs, since the second call finds the first call's leftovers
in the shared array; both are also held against the CPU oracle's packing.  A further test checks what
the entry point is for: a call leaves the device's free memory and the caching allocator untouched.

The file name sorts last so that a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from parity_util import assert_pack_equal

pytestmark = pytest.mark.gpu


def _pack(B, entry, lens, keep, loss_len, L, N_win, policy):
    n = len(lens)
    i32 = dict(dtype=torch.int32, device="cuda")
    d_len = torch.from_numpy(lens).cuda()
    d_keep = torch.from_numpy(keep).cuda() if keep is not None else None
    d_loss = torch.from_numpy(loss_len).cuda() if loss_len is not None else None
    outs = [torch.full((n,), 77, **i32) for _ in range(4)]
    cu = torch.full((n + 1,), 77, **i32); counts = torch.full((4,), 77, **i32); status = torch.zeros(1, **i32)
    prm = B.PackParams(n, L, N_win, policy)
    if entry == "static":
        B.pack_prompts_static(prm, d_len, d_keep, d_loss, *outs, cu, counts, status)
    else:
        nbytes = B.pack_workspace_bytes(prm)
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        B.pack_prompts(prm, d_len, d_keep, d_loss, *outs, cu, counts, ws, nbytes, status)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in outs] + [cu.cpu().numpy(), counts.cpu().numpy(), status.cpu().numpy()]


def test_static_scratch_packer_matches_workspace_packer_twice():
    from paper_2603_04135_b200 import binding as B
    assert B.pack_static_max_units() == 8192
    rng = np.random.default_rng(2024)
    # first call: a large stream that fills most of the array; second call: a shorter, different one
    cases = [dict(n=6000, L=2048, N_win=64, policy=0), dict(n=257, L=512, N_win=7, policy=1)]
    for c in cases:
        lens = rng.integers(1, c["L"] + 1, size=c["n"]).astype(np.int32)
        keep = (rng.random(c["n"]) < 0.8).astype(np.uint8)
        loss_len = rng.integers(0, 64, size=c["n"]).astype(np.int32)
        got = _pack(B, "static", lens, keep, loss_len, c["L"], c["N_win"], c["policy"])
        want = _pack(B, "workspace", lens, keep, loss_len, c["L"], c["N_win"], c["policy"])
        assert got[-1][0] == 0 and want[-1][0] == 0
        for g, w in zip(got, want):
            assert np.array_equal(g, w)
        assert got[5][0] == int(keep.sum()) and got[5][1] > 0
        # and against the definition: the oracle's window-greedy packing of the same stream
        ref = oracle.pack_prompts(lens, c["L"], c["N_win"], keep=keep, loss_len=loss_len, best_fit=bool(c["policy"]))
        names = ("order", "row_of", "off_in_row", "row_fill", "cu_seqlens", "counts", "status")
        assert_pack_equal(dict(zip(names, got)), ref, c["n"])


def test_static_scratch_packer_allocates_nothing():
    from paper_2603_04135_b200 import binding as B
    rng = np.random.default_rng(7)
    n, L = 4000, 1024
    i32 = dict(dtype=torch.int32, device="cuda")
    d_len = torch.from_numpy(rng.integers(1, L + 1, size=n).astype(np.int32)).cuda()
    outs = [torch.zeros(n, **i32) for _ in range(4)]
    cu = torch.zeros(n + 1, **i32); counts = torch.zeros(4, **i32); status = torch.zeros(1, **i32)
    prm = B.PackParams(n, L, 16, 0)
    B.pack_prompts_static(prm, d_len, None, None, *outs, cu, counts, status)      # first call on the device: set-up
    torch.cuda.synchronize()
    first = counts.cpu().numpy().copy()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        B.pack_prompts_static(prm, d_len, None, None, *outs, cu, counts, status)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0                                                          # the driver handed out nothing
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert status.item() == 0 and np.array_equal(counts.cpu().numpy(), first) and first[0] == n


def test_static_scratch_packer_rejects_oversize():
    from paper_2603_04135_b200 import binding as B
    n = B.pack_static_max_units() + 1
    z = torch.zeros(n + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DppoError) as e:
        B.pack_prompts_static(B.PackParams(n, 64, 4, 0), z, None, None, z, z, z, z, z, z, None)
    assert e.value.code == B.ERR_BAD_SHAPE and "8192" in str(e.value)
