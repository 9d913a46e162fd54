"""Pins for the oracle's mask side (Algorithm 1, PSABlock granularity, 3D-padding,
GetKVBlocks lists).  CPU only.  Each test checks the oracle against something other
than itself: hand-written masks, a differently written band enumeration, closed-form
counts, structural identities, or numbers the paper prints."""
import itertools
import json
import os
import random

import numpy as np
import pytest

from oracle import psa_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
INF = O.INF_STRIDE


def _load_axis_golden():
    cases = []
    with open(os.path.join(GOLDEN, "axis_masks.txt")) as f:
        lines = [ln.rstrip("\n") for ln in f if not ln.startswith("#") and ln.strip()]
    i = 0
    while i < len(lines):
        n, w, o, s, pairs = lines[i].split()
        n, w, o, pairs = int(n), int(w), int(o), int(pairs)
        s = INF if s == "inf" else int(s)
        rows = lines[i + 1:i + 1 + n]
        m = np.array([[c == "1" for c in r] for r in rows], dtype=bool)
        cases.append((n, w, o, s, pairs, m))
        i += 1 + n
    return cases


@pytest.mark.parametrize("case", _load_axis_golden(), ids=lambda c: f"n{c[0]}_w{c[1]}_o{c[2]}_s{c[3]}")
def test_axis_mask_matches_hand_derived(case):
    n, w, o, s, pairs, want = case
    got = O.axis_mask(n, w, o, s)
    assert got.shape == (n, n)
    assert np.array_equal(got, want)
    assert int(got.sum()) == pairs
    # the scalar form agrees too
    for q in range(n):
        for k in range(n):
            assert O.axis_cond(k - q, w, o, s) == bool(want[q, k])


def _band_deltas(n, w, o, s):
    """Second, differently written statement of the rule: the attended differences are
    the central band o + [-(w-1), w-1]; for a finite stride, further bands of width w
    start at o + k*s going up and are mirrored (not translated) going down."""
    deltas = set()
    if s == INF:
        for r in range(-(w - 1), w):
            deltas.add(o + r)
    else:
        kmax = (2 * n + abs(o)) // s + 2
        for kk in range(kmax + 1):
            for r in range(min(w, s)):
                deltas.add(o + kk * s + r)
                deltas.add(o - kk * s - r)
    return {d for d in deltas if -(n - 1) <= d <= n - 1}


def test_axis_mask_vs_band_enumeration():
    for n in range(1, 13):
        for w in range(1, n + 2):
            for o in range(-2, 3):
                for s in (1, 2, 3, 5, 6, INF):
                    deltas = _band_deltas(n, w, o, s)
                    m = O.axis_mask(n, w, o, s)
                    for q in range(n):
                        for k in range(n):
                            assert bool(m[q, k]) == ((k - q) in deltas), (n, w, o, s, q, k)


def _closed_form_pairs(n, w, o, s):
    """Pairs on one axis of extent n: sum over differences d of (n - |d|) * [d attended]."""
    tot = 0
    for d in range(-(n - 1), n):
        x = abs(d - o)
        if s != INF:
            x %= s
        if x <= w - 1:
            tot += n - abs(d)
    return tot


def test_closed_form_counts():
    assert int(O.axis_mask(30, 5, 0, 6).sum()) == 770 == _closed_form_pairs(30, 5, 0, 6)
    assert int(O.axis_mask(7, 3, 0, INF).sum()) == 29 == _closed_form_pairs(7, 3, 0, INF)
    assert int(O.axis_mask(11, 3, 2, INF).sum()) == 45 == _closed_form_pairs(11, 3, 2, INF)
    # single-diagonal band of half-width w-1, no offset: n + 2*sum_{d=1}^{w-1}(n-d)
    for n in range(1, 20):
        for w in range(1, n + 1):
            want = n + 2 * sum(n - d for d in range(1, w))
            assert int(O.axis_mask(n, w, 0, INF).sum()) == want


def test_special_cases_all_pass_and_infinite_stride():
    for n in range(1, 10):
        full = np.ones((n, n), dtype=bool)
        # stride 1 is all-pass; width >= stride is all-pass; a band as wide as the axis is all-pass
        assert np.array_equal(O.axis_mask(n, 1, 0, 1), full)
        assert np.array_equal(O.axis_mask(n, 3, 1, 3), full)
        assert np.array_equal(O.axis_mask(n, n, 0, INF), full)
        # a finite stride that no difference can reach behaves like infinity
        for o in (-2, 0, 1):
            for w in range(1, n + 1):
                big = n + abs(o)
                assert np.array_equal(O.axis_mask(n, w, o, big), O.axis_mask(n, w, o, INF))
    # SVG-like family: a single band per axis, i.e. |delta| <= w-1
    m = O.axis_mask(9, 3, 0, INF)
    q, k = np.indices((9, 9))
    assert np.array_equal(m, np.abs(k - q) <= 2)


def test_mirror_not_translation():
    # With offset 1, stride 4, width 2 the lower bands are mirrored: difference -3 attends
    # (|-3-1| = 4, 4 mod 4 = 0) while a translated band would start at 1-4 = -3 and also take -2.
    assert O.axis_cond(-3, 2, 1, 4)
    assert O.axis_cond(-4, 2, 1, 4)      # |-4-1| = 5 -> 1 <= 1
    assert not O.axis_cond(-2, 2, 1, 4)  # |-2-1| = 3 -> 3 > 1


def test_delta_is_key_minus_query():
    # offset +1, width 1, no stride: query q attends key q+1 only
    m = O.axis_mask(5, 1, 1, INF)
    for q in range(5):
        assert list(np.flatnonzero(m[q])) == ([q + 1] if q + 1 < 5 else [])


def test_token_order_and_alg1_on_tokens():
    T, H, W = 3, 4, 5
    # Proposition 1: i = t*H*W + h*W + w
    for t, h, w in itertools.product(range(T), range(H), range(W)):
        assert O.token_coords(t * H * W + h * W + w, H, W) == (t, h, w)
    # brick 1x1x1: Algorithm 1 verbatim, t = i // (H*W), s = i % (H*W)
    rng = random.Random(7)
    L = T * H * W
    for _ in range(40):
        p = (rng.randint(1, 3), rng.randint(-2, 2), rng.choice([1, 2, 3, INF]),
             rng.randint(1, 6), rng.randint(-1, 1), rng.choice([1, 3, 5, 6, INF]))
        em = O.element_mask(p, T, H, W, (1, 1, 1))
        for _ in range(60):
            i, j = rng.randrange(L), rng.randrange(L)
            tq, sq = i // (H * W), i % (H * W)
            tk, sk = j // (H * W), j % (H * W)
            a = abs(tk - tq - p[1])
            a = a if p[2] == INF else a % p[2]
            b = abs(sk - sq - p[4])
            b = b if p[5] == INF else b % p[5]
            want = a <= p[0] - 1 and b <= p[3] - 1
            assert bool(em[i, j]) == want == O.is_attending(i, j, p, T, H, W)


def test_padding_examples_from_paper():
    with open(os.path.join(GOLDEN, "paper_facts.json")) as f:
        facts = json.load(f)
    for ex in facts["padding_examples"]:
        assert list(O.padded_extents(*ex["grid"], tuple(ex["tile"]))) == ex["padded"], ex["cite"]
    rb = facts["range_bounds"]
    Tp, Hp, Wp = O.block_grid(*rb["grid"], tuple(rb["tile"]))
    assert Tp == rb["Tprime"] and Wp == rb["Wprime"]


def test_flop_accounting_matches_table2():
    with open(os.path.join(GOLDEN, "paper_facts.json")) as f:
        facts = json.load(f)
    for ex in facts["flop_counts"]:
        assert round(O.dense_flops(ex["L"], ex["d"], ex["heads"]) / 1e12, 2) == ex["tflop"], ex["cite"]
    sf = facts["sparse_flops"]
    assert round(sf["dense_tflop"] * (1 - sf["sparsity"]), 2) == sf["tflop"]
    # an all-pass head on an unpadded grid computes exactly the dense count
    T, H, W, tile = 4, 8, 8, (2, 4, 4)
    p = (2, 0, INF, 4, 0, INF)
    assert O.computed_flops([p], T, H, W, tile, 128) == O.dense_flops(T * H * W, 128, 1)


def _random_params(rng, Tp, Sp):
    return (rng.randint(1, Tp), rng.randint(-2, 2), rng.choice([1, 2, 3, INF]),
            rng.randint(1, max(1, Sp)), rng.randint(-1, 1), rng.choice([1, 3, 5, 6, INF]))


def test_block_mask_is_kronecker_of_axis_masks_and_uniform():
    rng = random.Random(11)
    grids = [((4, 4, 6), (2, 2, 2)), ((3, 5, 7), (1, 2, 4)), ((5, 3, 3), (2, 2, 2)), ((2, 6, 4), (1, 3, 2))]
    for (T, H, W), tile in grids:
        Tp, Hp, Wp = O.block_grid(T, H, W, tile)
        for _ in range(12):
            p = _random_params(rng, Tp, Hp * Wp)
            bm = O.block_mask(p, T, H, W, tile)
            kron = np.kron(O.axis_mask(Tp, *p[:3]), O.axis_mask(Hp * Wp, *p[3:])).astype(np.uint8)
            assert np.array_equal(bm, kron)
            slow, uniform = O.block_mask_from_elements(p, T, H, W, tile)
            assert uniform
            assert np.array_equal(bm, slow)
            assert abs(O.tile_sparsity(p, T, H, W, tile)
                       - (1 - O.axis_mask(Tp, *p[:3]).mean() * O.axis_mask(Hp * Wp, *p[3:]).mean())) < 1e-12


def test_is_attending_brute_force_vs_element_mask():
    rng = random.Random(5)
    T, H, W, tile = 3, 4, 4, (2, 2, 2)
    L = T * H * W
    for _ in range(6):
        p = _random_params(rng, 2, 4)
        em = O.element_mask(p, T, H, W, tile)
        for i in range(L):
            for j in range(L):
                assert bool(em[i, j]) == O.is_attending(i, j, p, T, H, W, tile)


def test_index_lists_are_sorted_products():
    rng = random.Random(3)
    T, H, W, tile = 6, 8, 8, (2, 4, 4)
    Tp, Hp, Wp = O.block_grid(T, H, W, tile)
    Sp, NB = Hp * Wp, Tp * Hp * Wp
    heads = [_random_params(rng, Tp, Sp) for _ in range(5)] + [(1, 1, INF, 1, 0, INF)]
    masks, row_ptr, col = O.block_index_lists(heads, T, H, W, tile)
    assert masks.shape == (len(heads), NB, NB) and row_ptr.shape == (len(heads) * NB + 1,)
    assert row_ptr[0] == 0 and row_ptr[-1] == col.size == int(masks.sum())
    for hd, p in enumerate(heads):
        MT, MS = O.axis_mask(Tp, *p[:3]), O.axis_mask(Sp, *p[3:])
        for qb in range(NB):
            tq, sq = divmod(qb, Sp)
            want = [tk * Sp + sk for tk in np.flatnonzero(MT[tq]) for sk in np.flatnonzero(MS[sq])]
            lo, hi = row_ptr[hd * NB + qb], row_ptr[hd * NB + qb + 1]
            assert list(col[lo:hi]) == want
    # the offset-only head leaves its last temporal block row empty
    last = len(heads) - 1
    for qb in range((Tp - 1) * Sp, NB):
        assert row_ptr[last * NB + qb] == row_ptr[last * NB + qb + 1]
    assert O.has_empty_row(heads[-1], T, H, W, tile)


def test_block_real_tokens_ragged():
    T, H, W, tile = 3, 5, 7, (2, 2, 4)
    real = O.block_real_tokens(T, H, W, tile)
    Tp, Hp, Wp = O.block_grid(T, H, W, tile)
    assert real.sum() == T * H * W
    want = []
    for tb in range(Tp):
        for hb in range(Hp):
            for wb in range(Wp):
                nt = min(tile[0], T - tb * tile[0])
                nh = min(tile[1], H - hb * tile[1])
                nw = min(tile[2], W - wb * tile[2])
                want.append(nt * nh * nw)
    assert list(real) == want
