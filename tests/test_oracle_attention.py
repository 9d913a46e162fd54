"""Pins for the oracle's attention side (masked safe-softmax attention in fp64).
CPU only: brute force with Python loops, the dense invariant, softmax invariants,
closed forms for zero queries, and a library routine on the dense special case."""
import math
import random

import numpy as np
import pytest
import torch

from oracle import psa_oracle as O

INF = O.INF_STRIDE


def _rand_qkv(L, d, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((L, d)), rng.standard_normal((L, d)), rng.standard_normal((L, d))


def test_bf16_bits_to_f64_exact():
    bits = np.arange(0, 65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):   # signalling-NaN patterns are in the sweep
        got = O.bf16_bits_to_f64(bits)
    want = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    ok = np.isfinite(want)
    assert np.array_equal(got[ok], want[ok])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    # spot values: 0x3F80 = 1.0, 0xC000 = -2.0, 0x3DCC = 0.099609375
    assert list(O.bf16_bits_to_f64(np.array([0x3F80, 0xC000, 0x3DCC], dtype=np.uint16))) == [1.0, -2.0, 0.099609375]


def test_brute_force_tiny():
    """Pure-Python loops straight from the definitions on a tiny grid."""
    T, H, W, tile, d = 2, 3, 4, (1, 2, 2), 8
    L = T * H * W
    scale = 1.0 / math.sqrt(d)
    q, k, v = _rand_qkv(L, d, 1)
    rng = random.Random(2)
    for _ in range(5):
        p = (rng.randint(1, 2), rng.randint(-1, 1), rng.choice([1, 2, INF]),
             rng.randint(1, 3), rng.randint(-1, 1), rng.choice([1, 3, INF]))
        out, lse = O.attention(q, k, v, p, T, H, W, tile, scale)
        for i in range(L):
            js = [j for j in range(L) if O.is_attending(i, j, p, T, H, W, tile)]
            if not js:
                assert np.all(out[i] == 0) and lse[i] == -np.inf
                continue
            a = [scale * sum(q[i][c] * k[j][c] for c in range(d)) for j in js]
            z = sum(math.exp(x) for x in a)
            for c in range(d):
                want = sum(math.exp(x) * v[j][c] for x, j in zip(a, js)) / z
                assert abs(out[i][c] - want) < 1e-12
            assert abs(lse[i] - math.log(z)) < 1e-12


@pytest.mark.parametrize("params", [
    (4, 0, INF, 6, 0, INF),   # bands as wide as the block grid
    (1, 0, 1, 1, 0, 1),       # stride 1 on both axes
    (2, 1, 2, 3, -1, 3),      # width >= stride on both axes
    (1, 2, 1, 5, 0, 5),
])
def test_dense_invariant(params):
    """An all-covering period/width reproduces dense attention exactly."""
    T, H, W, tile, d = 4, 4, 6, (1, 2, 2), 16
    L = T * H * W
    scale = 0.3
    q, k, v = _rand_qkv(L, d, 3)
    assert O.tile_sparsity(params, T, H, W, tile) == 0.0
    out, lse = O.attention(q, k, v, params, T, H, W, tile, scale)
    dout, dlse = O.dense_attention(q, k, v, scale)
    assert np.max(np.abs(out - dout)) < 1e-12
    assert np.max(np.abs(lse - dlse)) < 1e-12


def test_dense_case_vs_library_sdpa():
    L, d, scale = 96, 32, 0.2
    q, k, v = _rand_qkv(L, d, 4)
    dout, dlse = O.dense_attention(q, k, v, scale)
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=scale)[0, 0].numpy()
    assert np.max(np.abs(dout - want)) < 1e-12
    want_lse = torch.logsumexp(scale * (tq[0, 0] @ tk[0, 0].T), dim=1).numpy()
    assert np.max(np.abs(dlse - want_lse)) < 1e-12


def test_masked_case_vs_library_sdpa_with_bool_mask():
    """The masked oracle against torch SDPA given the element mask as a boolean matrix."""
    T, H, W, tile, d = 4, 4, 4, (2, 2, 2), 16
    L, scale = T * H * W, 0.25
    q, k, v = _rand_qkv(L, d, 5)
    p = (1, 0, 2, 2, 0, 3)
    em = O.element_mask(p, T, H, W, tile)
    assert em.any(axis=1).all() and not em.all()
    out, lse = O.attention(q, k, v, p, T, H, W, tile, scale)
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(
        tq, tk, tv, attn_mask=torch.from_numpy(em)[None, None], scale=scale)[0, 0].numpy()
    assert np.max(np.abs(out - want)) < 1e-12
    a = scale * (tq[0, 0] @ tk[0, 0].T)
    a = a.masked_fill(~torch.from_numpy(em), -math.inf)
    assert np.max(np.abs(lse - torch.logsumexp(a, dim=1).numpy())) < 1e-12


def test_softmax_invariants():
    T, H, W, tile, d = 3, 4, 4, (1, 2, 2), 8
    L, scale = T * H * W, 0.5
    q, k, v = _rand_qkv(L, d, 6)
    p = (2, 0, INF, 1, 0, 3)
    tb, sb, _ = O.token_block_coords(T, H, W, tile)
    out, lse = O.attention(q, k, v, p, T, H, W, tile, scale)
    for i in range(L):
        att = O.attend_row(i, p, tb, sb)
        pr = O.softmax_row(q[i], k, att, scale)
        assert abs(pr.sum() - 1.0) < 1e-12          # rows of the softmax sum to one
        assert np.all(pr[~att] == 0)
        assert np.max(np.abs(pr @ v - out[i])) < 1e-12
        idx = np.flatnonzero(att)
        # the output lies in the per-channel hull of the attended values
        assert np.all(out[i] <= v[idx].max(axis=0) + 1e-12)
        assert np.all(out[i] >= v[idx].min(axis=0) - 1e-12)
        a = scale * (k[idx] @ q[i])
        assert a.max() - 1e-12 <= lse[i] <= a.max() + math.log(idx.size) + 1e-12


def test_zero_query_closed_form_counts_real_tokens():
    """With q = 0 every score is 0: lse = ln(number of attended real keys) and the
    output is the plain mean of the attended values.  The count follows from the
    block lists and the real-token count of each block (ragged grid)."""
    T, H, W, tile, d = 3, 5, 7, (2, 2, 4), 4
    L = T * H * W
    rng = np.random.default_rng(8)
    q = np.zeros((L, d))
    k = rng.standard_normal((L, d))
    v = rng.standard_normal((L, d))
    p = (1, 0, 2, 2, 1, 3)
    out, lse = O.attention(q, k, v, p, T, H, W, tile, 1.0)
    bm = O.block_mask(p, T, H, W, tile)
    real = O.block_real_tokens(T, H, W, tile)
    _, _, blk = O.token_block_coords(T, H, W, tile)
    n_per_block = bm.astype(np.int64) @ real
    for i in range(L):
        n = n_per_block[blk[i]]
        if n == 0:
            assert lse[i] == -np.inf and np.all(out[i] == 0)
            continue
        assert abs(lse[i] - math.log(n)) < 1e-12
        keys = np.flatnonzero(bm[blk[i]][blk] == 1)
        assert keys.size == n
        assert np.max(np.abs(out[i] - v[keys].mean(axis=0))) < 1e-12
    assert O.attended_pairs(p, T, H, W, tile) == int((n_per_block[blk]).sum())


def test_empty_rows_convention():
    T, H, W, tile, d = 4, 2, 2, (1, 2, 2), 4
    L = T * H * W
    q, k, v = _rand_qkv(L, d, 9)
    p = (1, 1, INF, 1, 0, INF)   # each query block attends only the next temporal block
    out, lse = O.attention(q, k, v, p, T, H, W, tile, 1.0)
    last = np.arange(L) >= (T - 1) * H * W
    assert np.all(out[last] == 0) and np.all(lse[last] == -np.inf)
    assert np.all(np.isfinite(lse[~last]))


def test_attention_rows_subset_matches_full():
    T, H, W, tile, d = 3, 4, 4, (1, 2, 2), 8
    L = T * H * W
    q, k, v = _rand_qkv(L, d, 10)
    p = (2, -1, 3, 2, 0, INF)
    out, lse = O.attention(q, k, v, p, T, H, W, tile, 0.4)
    rows = [0, 5, 17, L - 1]
    so, sl = O.attention_rows(q, k, v, rows, p, T, H, W, tile, 0.4)
    assert np.array_equal(so, out[rows]) and np.array_equal(sl, lse[rows])
