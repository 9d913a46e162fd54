"""Randomised parity of psa_attn_fwd against the fp64 oracle: seeded small grids, every supported kind of
mask block (1, 2 or 3 slabs; last slab of 128/112/96/64 tokens; slabs stacked along t, h or w), parameters
from the candidate ranges including offsets that leave empty rows.  Every row is compared."""
import math
import random

import numpy as np
import pytest
import torch

from oracle import psa_oracle as O
from paper_2609_37001_b200 import workloads as WL

pytestmark = pytest.mark.gpu
INF = O.INF_STRIDE
SCALE = 1.0 / math.sqrt(128.0)
TILES = [(1, 8, 16), (2, 8, 8), (1, 16, 16), (2, 8, 16), (1, 15, 16), (1, 14, 16), (1, 12, 16), (3, 8, 16),
         (6, 8, 8), (1, 23, 16), (2, 32, 4), (1, 1, 256), (1, 4, 32), (1, 24, 16), (4, 4, 8), (1, 2, 64), (1, 3, 64)]


@pytest.fixture(scope="module")
def B():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding
    return binding


def _cases():
    rng = random.Random(0xC0FFEE)
    cases = []
    for idx in range(36):
        tile = TILES[idx % len(TILES)]
        # 1..4 blocks per axis, with a ragged remainder in about half of the cases
        dims = []
        for b in tile:
            n = rng.randint(1, 3 if b > 1 else 4)
            ext = n * b - (rng.randint(0, b - 1) if rng.random() < 0.5 else 0)
            dims.append(max(1, ext))
        T, H, W = dims
        if T * H * W > 12000:
            continue
        Tp, Hp, Wp = O.block_grid(T, H, W, tile)
        heads = []
        for _ in range(rng.randint(1, 3)):
            heads.append((rng.randint(1, Tp), rng.randint(-2, 2), rng.choice([1, 2, 3, INF]),
                          rng.randint(1, max(1, Hp * Wp)), rng.randint(-1, 1), rng.choice([1, 3, 5, 6, INF])))
        cases.append(((T, H, W), tile, heads, 0xB000 + idx, rng.choice([1.0, 1.0, 2.0])))
    return cases


@pytest.mark.parametrize("grid,tile,params,seed,gain", _cases(),
                         ids=lambda v: "x".join(map(str, v)) if isinstance(v, tuple) and len(v) == 3 and isinstance(v[0], int) else None)
def test_random_shape(B, grid, tile, params, seed, gain):
    T, H, W = grid
    L, nh = T * H * W, len(params)
    bits = {n: WL.tensor_bits(seed, n, nh, L, gain=(gain if n != "v" else 1.0), threads=1) for n in ("q", "k", "v")}
    q, k, v = (torch.from_numpy(bits[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))
    out, lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    st, detail = B.psa_last_device_status()
    assert st == 0, (st, hex(detail))
    out_h = O.bf16_bits_to_f64(out.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
    lse_h = lse.cpu().numpy().astype(np.float64)
    for hd in range(nh):
        qf, kf, vf = (O.bf16_bits_to_f64(bits[n][hd]) for n in ("q", "k", "v"))
        ro, rl = O.attention(qf, kf, vf, params[hd], T, H, W, tile, SCALE)
        empty = np.isneginf(rl)
        assert np.array_equal(np.isneginf(lse_h[hd]), empty)
        assert np.all(out_h[hd][empty] == 0)
        err = np.abs(out_h[hd] - ro)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (hd, params[hd], err.max(), err.mean())
        if (~empty).any():
            assert np.abs(lse_h[hd][~empty] - rl[~empty]).max() <= 1e-3
