"""Oracle for parameterized stripe attention (PSA) -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 CPU statement of what the PSA forward path computes, written
from the paper's definitions.  It shares no code with the CUDA library and is
never imported by it; only the tests, the smoke check and the benchmark's CPU
baseline leg call it.

What it follows
---------------
* Mask definition (Algorithm 1): a query attends a key iff the inter-frame test
  ``(|dt - T_o| mod T_s) <= T_w - 1`` and the intra-frame test
  ``(|ds - S_o| mod S_s) <= S_w - 1`` both hold, where ``dt`` / ``ds`` are
  key-minus-query differences of the temporal / flattened spatial coordinate.
* Masking granularity (Section 3.2, "Hardware-Aware Design"): the mask is applied
  per PSABlock, a ``b_t x b_h x b_w`` brick of tokens, so the coordinates fed to
  Algorithm 1 are block coordinates ``t' = t // b_t`` and
  ``s' = (h // b_h) * W' + (w // b_w)`` on the block grid ``(T', H', W')``.
  With the brick ``1 x 1 x 1`` this is Algorithm 1 on token indices verbatim.
* Token order (Appendix D, Proposition 1): ``i = t*H*W + h*W + w``.
* Infinite stride (Appendix C.2): "one diagonal only", i.e. no modulo.  Encoded as
  stride 0.
* 3D-padding (Section 3.2, Algorithm 2 "3D-Padding(S, -inf)"): padded positions
  get score -inf, i.e. they do not exist; the oracle iterates real tokens only.
* Attention (Algorithm 2, consumer): masked safe-softmax attention.  The method is
  exact given the mask, so the oracle is the plain definition
  ``out_i = sum_j softmax_j(scale * <q_i, k_j>) v_j`` over attended ``j`` and
  ``lse_i = log sum_j exp(scale * <q_i, k_j>)``.
* Rows with no attended key (the paper is silent): ``out = 0``, ``lse = -inf``.

Parity pins: every function here is pinned by tests/test_oracle_*.py (hand-derived
masks, band enumeration, closed-form counts, dense invariant, brute force, softmax
invariants).  Not pinned beyond the stated tolerances: nothing in this file -- the
exp / P rounding freedom belongs to the kernel, not to the oracle.
"""
from __future__ import annotations

import math
from typing import Iterable, Sequence, Tuple

import numpy as np

INF_STRIDE = 0  # encoding of an infinite stride: no modulo is applied

Params = Tuple[int, int, int, int, int, int]  # (T_w, T_o, T_s, S_w, S_o, S_s)
Tile = Tuple[int, int, int]                   # (b_t, b_h, b_w)


# --------------------------------------------------------------------------- #
# bf16 <-> fp64
# --------------------------------------------------------------------------- #
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns (uint16) as float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- #
# geometry: token order, block grid, 3D-padding
# --------------------------------------------------------------------------- #
def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def block_grid(T: int, H: int, W: int, tile: Tile) -> Tuple[int, int, int]:
    """Block grid (T', H', W') after 3D-padding: each extent is rounded up to a
    multiple of its brick size (Section 3.2, "3D-Padding")."""
    bt, bh, bw = tile
    return ceil_div(T, bt), ceil_div(H, bh), ceil_div(W, bw)


def padded_extents(T: int, H: int, W: int, tile: Tile) -> Tuple[int, int, int]:
    Tp, Hp, Wp = block_grid(T, H, W, tile)
    return Tp * tile[0], Hp * tile[1], Wp * tile[2]


def token_coords(i: int, H: int, W: int) -> Tuple[int, int, int]:
    """(t, h, w) of frame-major, row-major token index i (Proposition 1)."""
    t, s = divmod(i, H * W)
    h, w = divmod(s, W)
    return t, h, w


def token_block_coords(T: int, H: int, W: int, tile: Tile):
    """Per-token block coordinates: arrays tb[i] = t', sb[i] = s', blk[i] = t'*S'+s'."""
    bt, bh, bw = tile
    _, Hp, Wp = block_grid(T, H, W, tile)
    i = np.arange(T * H * W, dtype=np.int64)
    t = i // (H * W)
    s = i % (H * W)
    h = s // W
    w = s % W
    tb = t // bt
    sb = (h // bh) * Wp + (w // bw)
    return tb, sb, tb * (Hp * Wp) + sb


# --------------------------------------------------------------------------- #
# Algorithm 1
# --------------------------------------------------------------------------- #
def axis_cond(delta: int, width: int, offset: int, stride: int) -> bool:
    """One condition of Algorithm 1: (|delta - offset| mod stride) <= width - 1.
    ``delta`` is key coordinate minus query coordinate; stride 0 means infinity."""
    x = abs(delta - offset)
    if stride != INF_STRIDE:
        x = x % stride
    return x <= width - 1


def is_attending(i: int, j: int, params: Params, T: int, H: int, W: int,
                 tile: Tile = (1, 1, 1)) -> bool:
    """Algorithm 1 for query token i and key token j, with coordinates taken at
    PSABlock granularity (``tile``)."""
    Tw, To, Ts, Sw, So, Ss = params
    bt, bh, bw = tile
    _, _, Wp = block_grid(T, H, W, tile)
    tq, hq, wq = token_coords(i, H, W)
    tk, hk, wk = token_coords(j, H, W)
    tq_b, tk_b = tq // bt, tk // bt
    sq_b = (hq // bh) * Wp + (wq // bw)
    sk_b = (hk // bh) * Wp + (wk // bw)
    if not axis_cond(tk_b - tq_b, Tw, To, Ts):
        return False
    return axis_cond(sk_b - sq_b, Sw, So, Ss)


def axis_mask(n: int, width: int, offset: int, stride: int) -> np.ndarray:
    """n x n boolean matrix [q, k] of one axis condition of Algorithm 1."""
    q = np.arange(n, dtype=np.int64)[:, None]
    k = np.arange(n, dtype=np.int64)[None, :]
    x = np.abs((k - q) - offset)
    if stride != INF_STRIDE:
        x = x % stride
    return x <= width - 1


def block_mask(params: Params, T: int, H: int, W: int, tile: Tile) -> np.ndarray:
    """Block mask uint8[NB, NB]: Algorithm 1 evaluated on block ids
    ``b = t' * S' + s'`` (query block = row, key block = column)."""
    Tw, To, Ts, Sw, So, Ss = params
    Tp, Hp, Wp = block_grid(T, H, W, tile)
    Sp = Hp * Wp
    b = np.arange(Tp * Sp, dtype=np.int64)
    tb, sb = b // Sp, b % Sp
    dt = tb[None, :] - tb[:, None]
    ds = sb[None, :] - sb[:, None]
    xt = np.abs(dt - To)
    if Ts != INF_STRIDE:
        xt = xt % Ts
    xs = np.abs(ds - So)
    if Ss != INF_STRIDE:
        xs = xs % Ss
    return ((xt <= Tw - 1) & (xs <= Sw - 1)).astype(np.uint8)


def element_mask(params: Params, T: int, H: int, W: int, tile: Tile) -> np.ndarray:
    """Dense L x L boolean element mask [query token, key token] (small grids only)."""
    Tw, To, Ts, Sw, So, Ss = params
    tb, sb, _ = token_block_coords(T, H, W, tile)
    xt = np.abs((tb[None, :] - tb[:, None]) - To)
    if Ts != INF_STRIDE:
        xt = xt % Ts
    xs = np.abs((sb[None, :] - sb[:, None]) - So)
    if Ss != INF_STRIDE:
        xs = xs % Ss
    return (xt <= Tw - 1) & (xs <= Sw - 1)


def block_mask_from_elements(params: Params, T: int, H: int, W: int, tile: Tile):
    """The slow way: expand the element mask and reduce it over every block pair.
    Returns (any-reduced uint8[NB, NB], uniform flag) where ``uniform`` says every
    block pair was all-true or all-false."""
    em = element_mask(params, T, H, W, tile)
    _, _, blk = token_block_coords(T, H, W, tile)
    Tp, Hp, Wp = block_grid(T, H, W, tile)
    NB = Tp * Hp * Wp
    any_m = np.zeros((NB, NB), dtype=np.uint8)
    all_m = np.ones((NB, NB), dtype=np.uint8)
    present = np.zeros(NB, dtype=bool)
    present[np.unique(blk)] = True
    for qb in range(NB):
        rows = em[blk == qb]
        if rows.shape[0] == 0:
            continue
        for kb in range(NB):
            sub = rows[:, blk == kb]
            if sub.size == 0:
                continue
            any_m[qb, kb] = sub.any()
            all_m[qb, kb] = sub.all()
    both = present[:, None] & present[None, :]
    uniform = bool(np.all((any_m == all_m) | ~both))
    return any_m, uniform


def block_index_lists(head_params: Sequence[Params], T: int, H: int, W: int, tile: Tile):
    """What GetKVBlocks yields for every (head, query block): the ascending list of
    attended key-block ids, in CSR form over rows ordered (head, query block).

    Returns (mask uint8[heads, NB, NB], row_ptr int32[heads*NB + 1], col_idx int32[nnz]).
    """
    masks = np.stack([block_mask(p, T, H, W, tile) for p in head_params])
    nh, NB, _ = masks.shape
    counts = masks.reshape(nh * NB, NB).sum(axis=1, dtype=np.int64)
    row_ptr = np.zeros(nh * NB + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    cols = []
    for hd in range(nh):
        for qb in range(NB):
            cols.append(np.flatnonzero(masks[hd, qb]).astype(np.int32))
    col_idx = np.concatenate(cols) if cols else np.zeros(0, np.int32)
    return masks, row_ptr.astype(np.int32), col_idx.astype(np.int32)


def tile_sparsity(params: Params, T: int, H: int, W: int, tile: Tile) -> float:
    """Fraction of block pairs the mask excludes."""
    return 1.0 - float(block_mask(params, T, H, W, tile).mean())


def has_empty_row(params: Params, T: int, H: int, W: int, tile: Tile) -> bool:
    return bool((block_mask(params, T, H, W, tile).sum(axis=1) == 0).any())


def block_real_tokens(T: int, H: int, W: int, tile: Tile) -> np.ndarray:
    """Number of real (unpadded) tokens in every block, int64[NB]."""
    _, _, blk = token_block_coords(T, H, W, tile)
    Tp, Hp, Wp = block_grid(T, H, W, tile)
    return np.bincount(blk, minlength=Tp * Hp * Wp).astype(np.int64)


def attended_pairs(params: Params, T: int, H: int, W: int, tile: Tile) -> int:
    """Number of attended real (query, key) token pairs of one head."""
    real = block_real_tokens(T, H, W, tile)
    m = block_mask(params, T, H, W, tile).astype(np.int64)
    return int(real @ m @ real)


# --------------------------------------------------------------------------- #
# masked softmax attention, fp64
# --------------------------------------------------------------------------- #
def attend_row(i: int, params: Params, tb: np.ndarray, sb: np.ndarray) -> np.ndarray:
    """Boolean vector over all key tokens: does query token i attend key j."""
    Tw, To, Ts, Sw, So, Ss = params
    xt = np.abs((tb - tb[i]) - To)
    if Ts != INF_STRIDE:
        xt = xt % Ts
    xs = np.abs((sb - sb[i]) - So)
    if Ss != INF_STRIDE:
        xs = xs % Ss
    return (xt <= Tw - 1) & (xs <= Sw - 1)


def attention_rows(q: np.ndarray, k: np.ndarray, v: np.ndarray, rows: Iterable[int],
                   params: Params, T: int, H: int, W: int, tile: Tile, scale: float):
    """Masked attention of one head for the query tokens in ``rows``.

    q, k, v: float64 [L, d] (already converted from bf16).  Returns
    (out float64[len(rows), d], lse float64[len(rows)]).
    """
    rows = np.asarray(list(rows), dtype=np.int64)
    tb, sb, _ = token_block_coords(T, H, W, tile)
    d = q.shape[1]
    out = np.zeros((rows.size, d), dtype=np.float64)
    lse = np.full(rows.size, -np.inf, dtype=np.float64)
    for r, i in enumerate(rows):
        att = attend_row(int(i), params, tb, sb)
        idx = np.flatnonzero(att)
        if idx.size == 0:
            continue
        a = scale * (k[idx] @ q[i])
        m = a.max()
        e = np.exp(a - m)
        l = e.sum()
        out[r] = (e @ v[idx]) / l
        lse[r] = m + math.log(l)
    return out, lse


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, params: Params,
              T: int, H: int, W: int, tile: Tile, scale: float):
    """Masked attention of one head, all rows."""
    return attention_rows(q, k, v, range(q.shape[0]), params, T, H, W, tile, scale)


def attend_row_with_text(i: int, params: Params, tb: np.ndarray, sb: np.ndarray, n_text: int) -> np.ndarray:
    """Attended keys of query i when n_text text tokens follow the L video tokens (a multimodal DiT's
    joint sequence).  The paper defines the stripe mask on the video grid only and does not say how the
    text tokens are treated; the reading taken: the mask applies between video tokens, every query
    attends every text key, and a text query attends every key."""
    L = tb.shape[0]
    att = np.ones(L + n_text, dtype=bool)
    if i < L:
        att[:L] = attend_row(i, params, tb, sb)
    return att


def attention_rows_with_text(q: np.ndarray, k: np.ndarray, v: np.ndarray, rows: Iterable[int], params: Params,
                             T: int, H: int, W: int, tile: Tile, scale: float, n_text: int):
    """Masked attention over the joint sequence: q, k, v are float64 [L + n_text, d], video tokens first.
    Returns (out float64[len(rows), d], lse float64[len(rows)]) for the query tokens in ``rows``."""
    rows = np.asarray(list(rows), dtype=np.int64)
    tb, sb, _ = token_block_coords(T, H, W, tile)
    out = np.zeros((rows.size, q.shape[1]), dtype=np.float64)
    lse = np.full(rows.size, -np.inf, dtype=np.float64)
    for r, i in enumerate(rows):
        idx = np.flatnonzero(attend_row_with_text(int(i), params, tb, sb, n_text))
        if idx.size == 0:
            continue
        a = scale * (k[idx] @ q[i])
        m = a.max()
        e = np.exp(a - m)
        l = e.sum()
        out[r] = (e @ v[idx]) / l
        lse[r] = m + math.log(l)
    return out, lse


def attention_with_text(q: np.ndarray, k: np.ndarray, v: np.ndarray, params: Params,
                        T: int, H: int, W: int, tile: Tile, scale: float, n_text: int):
    """All rows of attention_rows_with_text."""
    return attention_rows_with_text(q, k, v, range(q.shape[0]), params, T, H, W, tile, scale, n_text)


def dense_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float):
    """Unmasked softmax attention of one head, written without any mask logic."""
    a = scale * (q @ k.T)
    m = a.max(axis=1, keepdims=True)
    e = np.exp(a - m)
    l = e.sum(axis=1, keepdims=True)
    return (e @ v) / l, (m + np.log(l))[:, 0]


def softmax_row(q_i: np.ndarray, k: np.ndarray, att: np.ndarray, scale: float) -> np.ndarray:
    """Normalised probabilities of one query over all keys (zeros where masked)."""
    p = np.zeros(k.shape[0], dtype=np.float64)
    idx = np.flatnonzero(att)
    if idx.size:
        a = scale * (k[idx] @ q_i)
        e = np.exp(a - a.max())
        p[idx] = e / e.sum()
    return p


# --------------------------------------------------------------------------- #
# FLOP accounting (Table 2 convention: 4 * d per attended real token pair)
# --------------------------------------------------------------------------- #
def dense_flops(L: int, d: int, heads: int) -> float:
    return 4.0 * L * L * d * heads


def computed_flops(head_params: Sequence[Params], T: int, H: int, W: int, tile: Tile, d: int) -> float:
    return 4.0 * d * sum(attended_pairs(p, T, H, W, tile) for p in head_params)


# --------------------------------------------------------------------------- #
# PSA-Search for one head (Algorithm 3)
# --------------------------------------------------------------------------- #
def search_losses(q: np.ndarray, k: np.ndarray, v: np.ndarray, candidates: Sequence[Params],
                  T: int, H: int, W: int, tile: Tile, scale: float) -> np.ndarray:
    """Inner loop of Algorithm 3 for one head: Loss(M) = L2Loss(PSA(h, M), FullAttn(h)) for every
    candidate mask M.  The paper does not spell the loss out; it is taken as the mean squared
    difference over all output elements.  q, k, v: float64 [L, d].  Returns float64[len(candidates)]."""
    full, _ = dense_attention(q, k, v, scale)
    losses = np.zeros(len(candidates), dtype=np.float64)
    for c, p in enumerate(candidates):
        out, _ = attention(q, k, v, p, T, H, W, tile, scale)
        losses[c] = np.mean((out - full) ** 2)
    return losses


def search_select(losses: Sequence[float], sparsities: Sequence[float], alpha: float) -> int:
    """Selection of Algorithm 3 for one head, step by step: sort the candidates by loss (ascending,
    ties by candidate index); start from the lowest-loss candidate; scan the sorted list and, among
    those whose loss does not exceed alpha, replace the current best whenever a candidate is strictly
    sparser.  Returns the index of the chosen candidate."""
    order = sorted(range(len(losses)), key=lambda i: (losses[i], i))
    best = order[0]
    for i in order:
        if losses[i] <= alpha:
            if sparsities[i] > sparsities[best]:
                best = i
    return best


def search_select_at_sparsity(losses: Sequence[float], sparsities: Sequence[float], target: float) -> int:
    """Second interface of PSA-Search (Section 3.3): given a target sparsity, the candidate with minimal
    loss among those at least that sparse (ties by candidate index); -1 when no candidate reaches the
    target."""
    best = -1
    for i in range(len(losses)):
        if sparsities[i] >= target:
            if best < 0 or losses[i] < losses[best]:
                best = i
    return best

