"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

Holds no arithmetic of the method: it reads the committed per-head stripe parameters
(workloads.json, written by oracle/gen_workloads.py) and draws q/k/v as i.i.d. N(0,1)
values rounded to bf16, from a counter-based generator keyed by (seed, tensor, head) so
that any single head can be reproduced on its own.
"""
from __future__ import annotations

import json
import os
from typing import Dict, List

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_TENSOR_ID = {"q": 0, "k": 1, "v": 2}


def load_workloads() -> Dict[str, dict]:
    with open(os.path.join(_HERE, "workloads.json")) as f:
        doc = json.load(f)
    return {w["name"]: w for w in doc["workloads"]}


def workload(name: str) -> dict:
    return load_workloads()[name]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (uint16)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def head_bits(seed: int, tensor: str, head: int, L: int, d: int = 128, gain: float = 1.0) -> np.ndarray:
    """bf16 bit patterns uint16[L, d] of one head of tensor 'q' | 'k' | 'v'."""
    key = (int(seed) << 20) ^ (_TENSOR_ID[tensor] << 16) ^ int(head)
    gen = np.random.Generator(np.random.Philox(key=key))
    x = gen.standard_normal((L, d), dtype=np.float32)
    if gain != 1.0:
        x *= np.float32(gain)
    return f32_to_bf16_bits(x)


def tensor_bits(seed: int, tensor: str, n_heads: int, L: int, d: int = 128, gain: float = 1.0,
                threads: int = 8) -> np.ndarray:
    """uint16[n_heads, L, d]; heads are generated independently (and in parallel)."""
    out = np.empty((n_heads, L, d), dtype=np.uint16)

    def fill(h):
        out[h] = head_bits(seed, tensor, h, L, d, gain)

    if threads > 1 and n_heads > 1:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(n_heads)))
    else:
        for h in range(n_heads):
            fill(h)
    return out


def sample_rows(seed: int, head: int, L: int, n: int) -> List[int]:
    gen = np.random.Generator(np.random.Philox(key=(int(seed) << 20) ^ (7 << 16) ^ int(head)))
    return sorted(set(int(x) for x in gen.integers(0, L, size=n)))


def search_candidates(seed: int, n: int, grid: Sequence[int], tile: Sequence[int]) -> List[Tuple[int, ...]]:
    """n distinct seeded candidate masks (Tw, To, Ts, Sw, So, Ss) from the initialisation space the
    paper gives for PSA-Search: 0 < Tw < T/bt, To in {0, +-1, +-2}, Ts in {1, 2, 3, inf},
    0 < Sw < W/bw, So in {0, +-1}, Ss in {1, 3, 5, 6, inf} (inf is encoded as stride 0).  Widths are
    clamped to at least 1 on tiny grids; fewer than n are returned if the space is smaller."""
    T, H, W = (int(x) for x in grid)
    tw_hi = max(2, -(-T // int(tile[0])))
    sw_hi = max(2, -(-W // int(tile[2])))
    gen = np.random.Generator(np.random.Philox(key=(int(seed) << 20) ^ (9 << 16)))
    seen, out = set(), []
    for _ in range(200 * n):
        c = (int(gen.integers(1, tw_hi)), int(gen.choice([0, 1, -1, 2, -2])), int(gen.choice([1, 2, 3, 0])),
             int(gen.integers(1, sw_hi)), int(gen.choice([0, 1, -1])), int(gen.choice([1, 3, 5, 6, 0])))
        if c not in seen:
            seen.add(c)
            out.append(c)
            if len(out) == n:
                break
    return out
