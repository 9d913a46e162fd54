"""Pins for the oracle's joint video + text attention (the reading taken for multimodal DiTs: stripe mask
between video tokens, text keys attended by everyone, text queries attending everything)."""
import math

import numpy as np

from oracle import psa_oracle as O

INF = O.INF_STRIDE


def _inputs(L, d, seed):
    rng = np.random.default_rng(seed)
    return tuple(rng.standard_normal((L, d)) for _ in range(3))


def test_no_text_tokens_is_the_plain_masked_attention():
    T, H, W, tile = 3, 4, 4, (1, 2, 2)
    q, k, v = _inputs(T * H * W, 8, 1)
    p = (1, 0, 2, 2, 1, INF)
    a = O.attention_with_text(q, k, v, p, T, H, W, tile, 0.3, 0)
    b = O.attention(q, k, v, p, T, H, W, tile, 0.3)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_all_covering_mask_is_dense_attention_over_the_joint_sequence():
    T, H, W, tile, nt = 2, 4, 4, (1, 2, 2), 5
    L = T * H * W
    q, k, v = _inputs(L + nt, 8, 2)
    Tp, Hp, Wp = O.block_grid(T, H, W, tile)
    out, lse = O.attention_with_text(q, k, v, (Tp, 0, INF, Hp * Wp, 0, INF), T, H, W, tile, 0.5, nt)
    ro, rl = O.dense_attention(q, k, v, 0.5)
    assert np.allclose(out, ro, atol=1e-12) and np.allclose(lse, rl, atol=1e-12)


def test_text_rows_are_dense_rows_and_video_rows_merge_two_softmaxes():
    """A video row's result is the log-sum-exp merge of (masked attention over the video keys) and
    (dense attention over the text keys); a text row is a dense row.  The merge formula is independent
    of the function under test."""
    T, H, W, tile, nt = 3, 4, 6, (1, 2, 3), 7
    L = T * H * W
    q, k, v = _inputs(L + nt, 16, 3)
    p = (1, 1, INF, 1, 0, 2)     # some video rows attend no video key at all
    scale = 0.4
    out, lse = O.attention_with_text(q, k, v, p, T, H, W, tile, scale, nt)
    ro, rl = O.dense_attention(q, k, v, scale)
    assert np.allclose(out[L:], ro[L:], atol=1e-12) and np.allclose(lse[L:], rl[L:], atol=1e-12)
    ov, lv = O.attention(q[:L], k[:L], v[:L], p, T, H, W, tile, scale)
    ot, lt = O.dense_attention(q[:L], k[L:], v[L:], scale)
    assert np.isneginf(lv).any() and not np.isneginf(lv).all()
    m = np.maximum(lv, lt)
    wv, wt = np.exp(lv - m), np.exp(lt - m)
    merged = (wv[:, None] * ov + wt[:, None] * ot) / (wv + wt)[:, None]
    assert np.allclose(out[:L], merged, atol=1e-12)
    assert np.allclose(lse[:L], m + np.log(wv + wt), atol=1e-12)


def test_brute_force_loops_on_a_tiny_case():
    T, H, W, tile, nt, d = 2, 2, 4, (1, 2, 2), 3, 4
    L = T * H * W
    q, k, v = _inputs(L + nt, d, 4)
    p = (1, 0, INF, 1, 1, INF)
    scale = 0.7
    out, lse = O.attention_with_text(q, k, v, p, T, H, W, tile, scale, nt)
    Wp = -(-W // tile[2])

    def blk(i):
        t, r = divmod(i, H * W)
        h, w = divmod(r, W)
        return t // tile[0], (h // tile[1]) * Wp + w // tile[2]

    for i in range(L + nt):
        num, den = np.zeros(d), 0.0
        for j in range(L + nt):
            if i < L and j < L:
                (ti, si), (tj, sj) = blk(i), blk(j)
                ok = abs((tj - ti) - p[1]) <= p[0] - 1 and abs((sj - si) - p[4]) <= p[3] - 1
            else:
                ok = True
            if ok:
                wgt = math.exp(scale * float(q[i] @ k[j]))
                num += wgt * v[j]
                den += wgt
        assert np.allclose(out[i], num / den, atol=1e-12)
        assert abs(lse[i] - math.log(den)) < 1e-12
