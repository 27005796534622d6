"""Pins for the oracle's Dense Prompt Packing (Section 4.3)."""
import itertools

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle


def check_layout(lens, L_row, out, keep=None, loss_len=None):
    n = len(lens)
    stream = [u for u in range(n) if keep is None or keep[u]]
    assert sorted(out["order"]) == stream                       # every retained unit exactly once
    fill = [0] * out["n_rows"]
    last_row = -1
    for u in out["order"]:                                      # rows are filled one after the other
        r = out["row_of"][u]
        assert r in (last_row, last_row + 1)
        last_row = r
        assert out["off_in_row"][u] == fill[r]                  # offsets are in-row prefix sums
        fill[r] += lens[u]
    assert fill == list(out["row_fill"]) and all(0 < f <= L_row for f in fill)
    for u in range(n):
        if u not in stream:
            assert out["row_of"][u] == -1 and out["off_in_row"][u] == -1
    ll = lens if loss_len is None else loss_len
    cu = [0]
    for u in out["order"]:
        cu.append(cu[-1] + ll[u])
    assert list(out["cu_seqlens"]) == cu
    assert tuple(out["counts"]) == (len(stream), out["n_rows"], sum(lens[u] for u in stream), cu[-1])


def next_fit(lens, L):          # textbook Next-Fit: keep one open bin, open a new one when the item does not fit
    rows, cur = [], []
    for u, l in enumerate(lens):
        if sum(lens[v] for v in cur) + l > L:
            rows.append(cur); cur = []
        cur.append(u)
    if cur:
        rows.append(cur)
    return rows


def first_fit(lens, L):         # textbook First-Fit: each item goes to the lowest-numbered bin with room
    rows, space = [], []
    for u, l in enumerate(lens):
        for r in range(len(rows)):
            if l <= space[r]:
                rows[r].append(u); space[r] -= l
                break
        else:
            rows.append([u]); space.append(L - l)
    return rows


def rows_of(out):
    rows = [[] for _ in range(out["n_rows"])]
    for u in out["order"]:
        rows[out["row_of"][u]].append(u)
    return rows


def window_rule_restatement(lens, L, N_win, best_fit=False):
    """No pool list: the pool is always {unplaced u < min(n, N_win + #placed)}, and pool order is index
    order, so 'first that fits' is the lowest such index."""
    n = len(lens)
    placed = [False] * n
    order, row_of = [], [-1] * n
    row, remaining, n_placed = 0, L, 0
    while n_placed < n:
        fetched = min(n, N_win + n_placed)
        fits = [u for u in range(fetched) if not placed[u] and lens[u] <= remaining]
        if not fits:
            row += 1; remaining = L
            continue
        u = fits[0] if not best_fit else max(fits, key=lambda v: (lens[v], -v))
        placed[u] = True; n_placed += 1
        order.append(u); row_of[u] = row; remaining -= lens[u]
    return order, row_of


def optimal_rows(lens, L):
    n = len(lens)
    best = n
    def rec(i, bins):
        nonlocal best
        if len(bins) >= best:
            return
        if i == n:
            best = len(bins); return
        seen = set()
        for b in range(len(bins)):
            if bins[b] + lens[i] <= L and bins[b] not in seen:
                seen.add(bins[b])
                bins[b] += lens[i]; rec(i + 1, bins); bins[b] -= lens[i]
        bins.append(lens[i]); rec(i + 1, bins); bins.pop()
    rec(0, [])
    return best


lens_strategy = st.lists(st.integers(1, 40), min_size=0, max_size=40)


@settings(max_examples=150, deadline=None)
@given(lens_strategy, st.integers(1, 12), st.booleans())
def test_layout_invariants(lens, N_win, best_fit):
    L = 40
    out = oracle.pack_prompts(lens, L, N_win, best_fit=best_fit)
    assert not out["error"]
    check_layout(lens, L, out)


@settings(max_examples=150, deadline=None)
@given(lens_strategy)
def test_window_one_is_next_fit(lens):
    out = oracle.pack_prompts(lens, 40, 1)
    assert rows_of(out) == next_fit(lens, 40)


@settings(max_examples=150, deadline=None)
@given(lens_strategy)
def test_full_window_is_first_fit(lens):
    out = oracle.pack_prompts(lens, 40, max(1, len(lens)))
    assert rows_of(out) == first_fit(lens, 40)
    out2 = oracle.pack_prompts(lens, 40, len(lens) + 7)
    assert out2["order"] == out["order"]


@settings(max_examples=200, deadline=None)
@given(lens_strategy, st.integers(1, 9), st.booleans())
def test_matches_rule_restatement(lens, N_win, best_fit):
    out = oracle.pack_prompts(lens, 40, N_win, best_fit=best_fit)
    order, row_of = window_rule_restatement(lens, 40, N_win, best_fit)
    assert out["order"] == order and out["row_of"] == row_of


def test_against_exhaustive_optimum_on_tiny_inputs():
    rng = np.random.default_rng(0)
    worst = 0
    for _ in range(120):
        n = int(rng.integers(1, 9))
        lens = [int(x) for x in rng.integers(1, 11, size=n)]
        L = 10
        opt = optimal_rows(lens, L)
        for N_win in (1, 2, 4, n):
            out = oracle.pack_prompts(lens, L, N_win)
            assert out["n_rows"] >= opt
            worst = max(worst, out["n_rows"] - opt)
        ff = oracle.pack_prompts(lens, L, n)
        assert ff["n_rows"] <= int(1.7 * opt) + 1               # First-Fit guarantee
        nf = oracle.pack_prompts(lens, L, 1)
        assert nf["n_rows"] <= 2 * opt                          # Next-Fit guarantee
    assert worst >= 1            # greedy is not optimal: the search finds at least one gap


def test_keep_mask_loss_len_and_errors():
    lens = [5, 9, 3, 7, 2, 8]
    keep = [1, 0, 1, 1, 0, 1]
    loss_len = [2, 4, 1, 3, 1, 5]
    out = oracle.pack_prompts(lens, 10, 2, keep=keep, loss_len=loss_len)
    check_layout(lens, 10, out, keep=keep, loss_len=loss_len)
    # stream 0,2,3,5 window 2: row0 = {0(5), 2(3)} then 3(7) no, 5? window after placing 0: [2,3]; after 2: [3,5]
    # remaining 2: nothing fits -> row1 = {3(7)}, window [5]: 8 no -> row2 = {5}
    assert out["order"] == [0, 2, 3, 5] and out["row_of"] == [0, -1, 0, 1, -1, 2]
    assert out["cu_seqlens"] == [0, 2, 3, 6, 11]
    assert oracle.pack_prompts([3, 11], 10, 2)["error"]
    assert oracle.pack_prompts([3, 0], 10, 2)["error"]
    assert not oracle.pack_prompts([3, 11], 10, 2, keep=[1, 0])["error"]
    empty = oracle.pack_prompts([], 10, 4)
    assert empty["n_rows"] == 0 and empty["cu_seqlens"] == [0] and not empty["error"]
    full = oracle.pack_prompts([10, 10, 4, 6], 10, 4)          # rows exactly full
    assert full["row_fill"] == [10, 10, 10]


def test_window_lookahead_example():
    # L=10, stream 6,5,4,3: window 1 -> {6},{5,4},{3}; window 2 -> {6},{5,4},{3}; window 3 -> {6,4},{5,3}
    lens = [6, 5, 4, 3]
    assert rows_of(oracle.pack_prompts(lens, 10, 1)) == [[0], [1, 2], [3]]
    assert rows_of(oracle.pack_prompts(lens, 10, 3)) == [[0, 2], [1, 3]]
    # best-fit prefers the longest fitting unit in the window
    lens = [6, 2, 4]
    assert rows_of(oracle.pack_prompts(lens, 10, 3)) == [[0, 1], [2]]
    assert rows_of(oracle.pack_prompts(lens, 10, 3, best_fit=True)) == [[0, 2], [1]]
