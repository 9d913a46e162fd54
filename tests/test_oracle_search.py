"""Pins for the oracle's PSA-Search step (Algorithm 3): hand-worked selections, the defining property
(max sparsity subject to loss <= alpha), and the loss against direct formulas."""
import itertools
import random

import numpy as np

from oracle import psa_oracle as O

INF = O.INF_STRIDE


def test_select_hand_worked_examples():
    # candidates:        0     1     2     3
    losses = [0.020, 0.001, 0.008, 0.004]
    spars = [0.90, 0.10, 0.75, 0.50]
    # alpha below every loss: nothing qualifies, the lowest-loss candidate stays
    assert O.search_select(losses, spars, 0.0005) == 1
    # alpha = 0.005: candidates 1 (0.001) and 3 (0.004) qualify -> the sparser one, 3
    assert O.search_select(losses, spars, 0.005) == 3
    # alpha = 0.01: 1, 3, 2 qualify -> 2 (75 %)
    assert O.search_select(losses, spars, 0.01) == 2
    # alpha = 0.05: all qualify -> 0 (90 %)
    assert O.search_select(losses, spars, 0.05) == 0
    # equal sparsity does not replace: the lower-loss one of two equally sparse candidates is kept
    assert O.search_select([0.002, 0.001, 0.003], [0.5, 0.5, 0.5], 1.0) == 1
    # the threshold is inclusive
    assert O.search_select([0.3, 0.1], [0.9, 0.2], 0.3) == 0


def test_select_is_max_sparsity_under_the_threshold():
    rng = random.Random(4)
    for _ in range(300):
        n = rng.randint(1, 9)
        losses = [round(rng.random(), 3) for _ in range(n)]
        spars = [rng.choice([0.1, 0.25, 0.5, 0.75, 0.9]) for _ in range(n)]
        alpha = rng.random()
        got = O.search_select(losses, spars, alpha)
        ok = [i for i in range(n) if losses[i] <= alpha]
        lowest = min(range(n), key=lambda i: (losses[i], i))
        if not ok:
            assert got == lowest
            continue
        smax = max(spars[i] for i in ok)
        if smax <= spars[lowest]:
            # nothing qualifying is strictly sparser than the lowest-loss candidate: it is kept
            assert got == lowest
        else:
            assert losses[got] <= alpha and spars[got] == smax
            # among the sparsest qualifying candidates the one met first in loss order wins
            assert got == min((i for i in ok if spars[i] == smax), key=lambda i: (losses[i], i))


def test_losses_against_direct_formulas():
    T, H, W, tile, d = 3, 4, 4, (1, 2, 2), 8
    L, scale = T * H * W, 0.4
    rng = np.random.default_rng(12)
    q, k, v = (rng.standard_normal((L, d)) for _ in range(3))
    Tp, Hp, Wp = O.block_grid(T, H, W, tile)
    cands = [(Tp, 0, INF, Hp * Wp, 0, INF),      # all-covering: loss exactly 0
             (1, 0, INF, Hp * Wp, 0, INF),       # same frame block only
             (1, 0, INF, 1, 0, INF)]             # same block only
    losses = O.search_losses(q, k, v, cands, T, H, W, tile, scale)
    assert losses[0] < 1e-28          # same numbers up to summation order
    # written out with a boolean mask and a library softmax, then the mean of squares
    import torch
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (q, k, v))
    full = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=scale)[0, 0].numpy()
    for c in (1, 2):
        em = O.element_mask(cands[c], T, H, W, tile)
        out = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(em)[None, None], scale=scale)[0, 0].numpy()
        want = float(((out - full) ** 2).sum() / (L * d))
        assert abs(losses[c] - want) < 1e-14
    assert 0 < losses[1] < losses[2]             # dropping more keys moves the output further


def test_select_at_sparsity_is_min_loss_over_the_feasible_set():
    assert O.search_select_at_sparsity([0.02, 0.001, 0.008, 0.004], [0.9, 0.1, 0.75, 0.5], 0.5) == 3
    assert O.search_select_at_sparsity([0.02, 0.001, 0.008, 0.004], [0.9, 0.1, 0.75, 0.5], 0.8) == 0
    assert O.search_select_at_sparsity([0.02, 0.001], [0.9, 0.1], 0.95) == -1
    assert O.search_select_at_sparsity([0.5, 0.5], [0.6, 0.7], 0.6) == 0      # tie: lower index
    rng = random.Random(8)
    for _ in range(300):
        n = rng.randint(1, 9)
        losses = [rng.randint(0, 20) / 20 for _ in range(n)]
        spars = [rng.choice([0.1, 0.25, 0.5, 0.75, 0.9]) for _ in range(n)]
        target = rng.random()
        got = O.search_select_at_sparsity(losses, spars, target)
        ok = [i for i in range(n) if spars[i] >= target]
        if not ok:
            assert got == -1
        else:
            # brute force over every feasible candidate
            assert got in ok and all(losses[got] <= losses[i] for i in ok)
            assert got == min(i for i in ok if losses[i] == losses[got])


def test_the_two_interfaces_agree_on_the_pareto_front():
    # choosing by threshold alpha and then asking for that candidate's sparsity returns a candidate
    # of no larger loss and no smaller sparsity
    rng = random.Random(10)
    for _ in range(200):
        n = rng.randint(2, 9)
        losses = [rng.randint(0, 50) / 50 for _ in range(n)]
        spars = [rng.choice([0.1, 0.25, 0.5, 0.75, 0.9]) for _ in range(n)]
        a = O.search_select(losses, spars, rng.random())
        b = O.search_select_at_sparsity(losses, spars, spars[a])
        assert b >= 0 and losses[b] <= losses[a] and spars[b] >= spars[a]
