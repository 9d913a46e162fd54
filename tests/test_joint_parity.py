"""psa_attn_fwd_joint (video tokens followed by text tokens) against the fp64 oracle, every row.
Same tolerances as the video-only parity tests."""
import math

import numpy as np
import pytest
import torch

from oracle import psa_oracle as O
from paper_2609_37001_b200 import workloads as WL

pytestmark = pytest.mark.gpu
INF = O.INF_STRIDE
SCALE = 1.0 / math.sqrt(128.0)
OUT_MAX, OUT_MEAN, LSE_MAX, REL_L2 = 2e-2, 2e-3, 1e-3, 1e-2


@pytest.fixture(scope="module")
def B():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding
    return binding


def _to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _bf16_to_f64(t):
    return O.bf16_bits_to_f64(t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))


def _check(B, grid, tile, params, n_text, seed, gain=1.0):
    T, H, W = grid
    L, nh = T * H * W, len(params)
    Lt = L + n_text
    bits = {n: WL.tensor_bits(seed, n, nh, Lt, gain=(gain if n != "v" else 1.0)) for n in ("q", "k", "v")}
    q, k, v = (_to_dev(bits[n]) for n in ("q", "k", "v"))
    out = torch.full_like(q, float("nan"))
    lse = torch.full((nh, Lt), float("nan"), dtype=torch.float32, device="cuda")
    B.psa_attn_fwd_joint(q, k, v, params, grid, tile, SCALE, n_text, out=out, lse=lse)
    st, detail = B.psa_last_device_status()
    assert st == 0, (st, hex(detail))
    out_h, lse_h = _bf16_to_f64(out), lse.cpu().numpy().astype(np.float64)
    assert not np.isnan(out_h).any() and not np.isnan(lse_h).any()     # every row was written
    for hd in range(nh):
        qf, kf, vf = (O.bf16_bits_to_f64(bits[n][hd]) for n in ("q", "k", "v"))
        ro, rl = O.attention_with_text(qf, kf, vf, tuple(params[hd]), T, H, W, tuple(tile), SCALE, n_text)
        what = f"grid {grid} tile {tile} n_text {n_text} head {hd}"
        assert np.array_equal(np.isneginf(lse_h[hd]), np.isneginf(rl)), what
        err = np.abs(out_h[hd] - ro)
        assert err.max() <= OUT_MAX and err.mean() <= OUT_MEAN, (what, err.max(), err.mean())
        okr = ~np.isneginf(rl)
        assert np.abs(lse_h[hd][okr] - rl[okr]).max() <= LSE_MAX, what
        assert np.linalg.norm(out_h[hd] - ro) / np.linalg.norm(ro) <= REL_L2, what
    return out, lse


def test_one_ragged_text_slab_single_slab_blocks(B):
    # 77 text tokens: one text slab (split-KV text-query item), 51 masked key columns
    params = [(2, 0, INF, 2, 0, INF), (1, 1, INF, 3, 0, 2), (1, 5, INF, 1, 0, INF)]   # last: no video key at all
    _check(B, (4, 12, 16), (1, 8, 16), params, 77, seed=41, gain=2.0)


def test_three_text_slabs_two_slab_blocks(B):
    # 300 text tokens: a two-slab text item and a ragged single one; 240-token blocks (128 + 112)
    params = [(1, 0, INF, 2, 0, INF), (3, 0, INF, 1, 1, 2)]
    _check(B, (3, 30, 32), (1, 15, 16), params, 300, seed=42)


def test_exact_text_slabs_three_slab_blocks(B):
    params = [(1, 0, 2, 1, 0, INF), (2, -1, INF, 2, 0, INF)]
    _check(B, (6, 8, 32), (3, 8, 16), params, 256, seed=43)


def test_ragged_grid_with_text(B):
    params = [(2, 0, INF, 1, 0, 2), (1, 0, INF, 4, 0, INF)]
    _check(B, (5, 20, 24), (1, 8, 16), params, 130, seed=44, gain=3.0)


def test_zero_text_tokens_is_the_video_only_call_bit_for_bit(B):
    grid, tile = (4, 12, 16), (1, 8, 16)
    params = [(2, 0, INF, 2, 0, INF), (1, 1, 2, 3, 0, INF)]
    L = 4 * 12 * 16
    bits = {n: WL.tensor_bits(45, n, 2, L) for n in ("q", "k", "v")}
    q, k, v = (_to_dev(bits[n]) for n in ("q", "k", "v"))
    o1, l1 = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    o2, l2 = B.psa_attn_fwd_joint(q, k, v, params, grid, tile, SCALE, 0)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)


def test_hunyuan_768p_with_256_text_tokens_sampled_rows(B):
    """Full-size joint call (the launch configuration of the timings): HunyuanVideo 768p shape plus 256
    text tokens; four heads are generated and run, sampled video rows, a whole edge brick and sampled text
    rows of each are compared with the oracle against all keys."""
    w = WL.workload("hunyuan_768p")
    grid, tile, nt = w["grid"], w["tile"], 256
    T, H, W = grid
    L = T * H * W
    heads = [0, 7, 14, 23]
    params = [tuple(w["head_params"][h]) for h in heads]
    bits = {n: np.stack([WL.head_bits(w["seed"], n, h, L + nt) for h in heads]) for n in ("q", "k", "v")}
    q, k, v = (_to_dev(bits[n]) for n in ("q", "k", "v"))
    out, lse = B.psa_attn_fwd_joint(q, k, v, params, grid, tile, SCALE, nt)
    st, detail = B.psa_last_device_status()
    assert st == 0, (st, hex(detail))
    out_h, lse_h = _bf16_to_f64(out), lse.cpu().numpy().astype(np.float64)
    for i, hd in enumerate(heads):
        rows = set(WL.sample_rows(w["seed"], hd, L, 24))
        rows |= {L + r for r in WL.sample_rows(w["seed"] + 1, hd, nt, 12)} | {L, L + nt - 1}
        bt, bh, bw = tile     # the last brick of the grid
        rows |= {(t * H + h) * W + x for t in range(T - bt, T) for h in range(H - bh, H) for x in range(W - bw, W) if (h + x) % 4 == 0}
        rows = sorted(rows)
        qf, kf, vf = (O.bf16_bits_to_f64(bits[n][i]) for n in ("q", "k", "v"))
        ro, rl = O.attention_rows_with_text(qf, kf, vf, rows, params[i], T, H, W, tuple(tile), SCALE, nt)
        err = np.abs(out_h[i][rows] - ro)
        assert err.max() <= OUT_MAX and err.mean() <= OUT_MEAN, (hd, err.max(), err.mean())
        assert np.abs(lse_h[i][rows] - rl).max() <= LSE_MAX, hd
