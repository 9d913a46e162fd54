"""Draws the per-head stripe parameters of the synthetic workloads and writes them to
paper_2609_37001_b200/workloads.json.  Uses only this directory's oracle.

The shapes stand in for the paper's attention calls (Wan 2.1 1.3B 480p, Wan 2.1 14B 720p,
HunyuanVideo 720p: latent grids and head counts from Appendix C.2 and Table 2's FLOP
column).  Parameters are drawn from the candidate ranges of Appendix C.2
(0 < T_w <= T', T_o in {0,+-1,+-2}, T_s in {1,2,3,inf}, 0 < S_w <= W', S_o in {0,+-1},
S_s in {1,3,5,6,inf}), filtered by the tile sparsity the oracle computes, rejecting
draws that leave a query block without any key block.

Run:  python oracle/gen_workloads.py
"""
import itertools
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from oracle import psa_oracle as O  # noqa: E402

INF = O.INF_STRIDE
OUT = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                   "paper_2609_37001_b200", "workloads.json")


def axis_candidates(n, wmax, offsets, strides):
    """All (w, o, s) on one axis with density and an empty-row flag, via the oracle's axis mask."""
    out = []
    for w, o, s in itertools.product(range(1, wmax + 1), offsets, strides):
        m = O.axis_mask(n, w, o, s)
        out.append(((w, o, s), float(m.mean()), bool((m.sum(axis=1) == 0).any())))
    return out


def candidates(T, H, W, tile):
    Tp, Hp, Wp = O.block_grid(T, H, W, tile)
    Sp = Hp * Wp
    ta = axis_candidates(Tp, Tp, (0, 1, -1, 2, -2), (1, 2, 3, INF))
    sa = axis_candidates(Sp, Wp, (0, 1, -1), (1, 3, 5, 6, INF))
    cands = []
    for (tp, dt, et), (sp, ds, es) in itertools.product(ta, sa):
        if et or es:
            continue
        kind = "dense" if dt == 1.0 and ds == 1.0 else "spatial" if dt == 1.0 else "temporal" if ds == 1.0 else "joint"
        cands.append((tp + sp, 1.0 - dt * ds, kind))
    return cands


def draw_heads(rng, cands, n_heads, lo, hi, kinds=("temporal", "spatial", "joint")):
    pools = {k: sorted({c[0] for c in cands if c[2] == k and lo <= c[1] <= hi}) for k in kinds}
    heads = []
    for i in range(n_heads):
        kind = kinds[i % len(kinds)]
        pool = pools[kind] or sorted({c[0] for c in cands if lo <= c[1] <= hi})
        heads.append(list(pool[int(rng.integers(len(pool)))]))
    return heads


def closest(cands, target, kinds=("joint", "temporal", "spatial")):
    best = min((c for c in cands if c[2] in kinds), key=lambda c: (abs(c[1] - target), c[0]))
    return list(best[0])


def describe(name, grid, tile, heads, note, seed):
    T, H, W = grid
    sp = [O.tile_sparsity(tuple(p), T, H, W, tuple(tile)) for p in heads]
    L = T * H * W
    pairs = sum(O.attended_pairs(tuple(p), T, H, W, tuple(tile)) for p in heads)
    return {
        "name": name, "grid": list(grid), "tile": list(tile), "n_heads": len(heads), "head_dim": 128,
        "seed": seed, "note": note, "head_params": heads,
        "tile_sparsity_per_head": [round(x, 6) for x in sp],
        "tile_sparsity": round(float(np.mean(sp)), 6),
        "attended_pairs": int(pairs), "dense_pairs": int(L * L * len(heads)),
    }


def main():
    wl = []
    # 1. tiny: head 0 a seeded draw, head 1 all-covering (must equal dense)
    for name, tile in (("tiny", (2, 8, 8)), ("tiny_b256", (2, 8, 16))):
        grid = (8, 16, 16)
        rng = np.random.Generator(np.random.Philox(key=0x50534101))
        c = candidates(*grid, tile)
        Tp, Hp, Wp = O.block_grid(*grid, tile)
        h0 = draw_heads(rng, c, 1, 0.3, 0.9, kinds=("joint",))[0]
        wl.append(describe(name, grid, tile, [h0, [Tp, 0, INF, Hp * Wp, 0, INF]],
                           "head 0 seeded joint draw; head 1 all-covering bands", 0x50534101))
    # 2. Wan 2.1 1.3B 480p
    grid, tile = (21, 30, 52), (2, 32, 4)
    rng = np.random.Generator(np.random.Philox(key=0x50534102))
    wl.append(describe("wan13b_480p", grid, tile, draw_heads(rng, candidates(*grid, tile), 12, 0.50, 0.80),
                       "12 heads, 50-80% tile sparsity, temporal/spatial/joint in turn", 0x50534102))
    #    the same shape with a 384-token block that tiles the 21 frames exactly (only H is padded, 30 -> 32)
    tile = (3, 32, 4)
    rng = np.random.Generator(np.random.Philox(key=0x50534102))
    wl.append(describe("wan13b_480p_b3x32x4", grid, tile, draw_heads(rng, candidates(*grid, tile), 12, 0.50, 0.80),
                       "12 heads, 50-80% tile sparsity, temporal/spatial/joint in turn", 0x50534102))
    #    and with blocks that pad only W: 1x30x8 (240 tokens = a 128- and a 112-token slab, W 52 -> 56) and
    #    the 128-token 1x32x4 (H 30 -> 32)
    for name, tile in (("wan13b_480p_b1x30x8", (1, 30, 8)), ("wan13b_480p_b1x32x4", (1, 32, 4))):
        rng = np.random.Generator(np.random.Philox(key=0x50534102))
        wl.append(describe(name, grid, tile, draw_heads(rng, candidates(*grid, tile), 12, 0.50, 0.80),
                           "12 heads, 50-80% tile sparsity, temporal/spatial/joint in turn", 0x50534102))
    # 3. Wan 2.1 14B 720p (headline).  1x15x16 (240 tokens = a 128- and a 112-token slab) tiles 21x45x80
    #    exactly; 1x16x16 and the paper's 3x8x16 pad H to 48 and are kept as further test cases.
    grid = (21, 45, 80)
    for name, tile in (("wan14b_720p", (1, 15, 16)), ("wan14b_720p_b1x16x16", (1, 16, 16)),
                       ("wan14b_720p_b3x8x16", (3, 8, 16))):
        rng = np.random.Generator(np.random.Philox(key=0x50534103))
        wl.append(describe(name, grid, tile, draw_heads(rng, candidates(*grid, tile), 40, 0.60, 0.90),
                           "40 heads, 60-90% tile sparsity, temporal/spatial/joint in turn", 0x50534103))
    # 4. HunyuanVideo 720p
    grid, tile = (33, 45, 80), (1, 15, 16)
    rng = np.random.Generator(np.random.Philox(key=0x50534104))
    wl.append(describe("hunyuan_720p", grid, tile, draw_heads(rng, candidates(*grid, tile), 24, 0.50, 0.85),
                       "24 heads, 50-85% tile sparsity, temporal/spatial/joint in turn", 0x50534104))
    # 5a. sparsity sweep at the Wan 14B shape: all heads share one parameter set per level
    grid, tile = (21, 45, 80), (1, 15, 16)
    c = candidates(*grid, tile)
    Tp, Hp, Wp = O.block_grid(*grid, tile)
    for level in (0, 25, 50, 75, 90):
        p = [Tp, 0, INF, Hp * Wp, 0, INF] if level == 0 else closest(c, level / 100.0)
        wl.append(describe(f"sweep_{level:02d}", grid, tile, [p] * 40,
                           f"sparsity sweep, target {level}% (0% = all-covering bands = dense baseline)", 0x50534103))
    # 5b. ragged grid (not a tile multiple in H and W with the 1x16x16 block)
    grid, tile = (21, 45, 79), (1, 16, 16)
    c = candidates(*grid, tile)
    wl.append(describe("ragged_75", grid, tile, [closest(c, 0.75)] * 40, "ragged grid, ~75% sparsity", 0x50534105))
    Tp, Hp, Wp = O.block_grid(*grid, tile)
    wl.append(describe("ragged_dense", grid, tile, [[Tp, 0, INF, Hp * Wp, 0, INF]] * 40, "ragged grid, all-covering", 0x50534105))
    # N1. HunyuanVideo 768x1280 (30x48x80, Table 2 / Table 3b): no padding with 1x16x16 or with the paper's
    #     6x8x8 block; plus the 60/70/80/90 % levels of Table 3b (all heads share one parameter set per level)
    grid = (30, 48, 80)
    for name, tile in (("hunyuan_768p", (1, 16, 16)), ("hunyuan_768p_b6x8x8", (6, 8, 8))):
        rng = np.random.Generator(np.random.Philox(key=0x50534106))
        wl.append(describe(name, grid, tile, draw_heads(rng, candidates(*grid, tile), 24, 0.50, 0.85),
                           "24 heads, 50-85% tile sparsity, temporal/spatial/joint in turn", 0x50534106))
    tile = (1, 16, 16)
    c = candidates(*grid, tile)
    for level in (60, 70, 80, 90):
        wl.append(describe(f"hy768_sweep_{level}", grid, tile, [closest(c, level / 100.0)] * 24,
                           f"HunyuanVideo 768p sparsity sweep, target {level}%", 0x50534106))
    with open(OUT, "w") as f:
        json.dump({"_generator": "oracle/gen_workloads.py", "inf_stride": INF, "workloads": wl}, f, indent=1)
    for w in wl:
        print(f'{w["name"]:24s} grid={w["grid"]} tile={w["tile"]} heads={w["n_heads"]} sparsity={w["tile_sparsity"]:.4f}')


if __name__ == "__main__":
    main()
