"""The checked build of the library (-DPSA_DEBUG_CHECKS): the attention kernel verifies every global
store index, TMA coordinate, ring slot and work-item field before using it and reports a violation
through the status word instead of touching memory -- the stand-in for a memory checker on a pool
where none may run.  A spread of shapes (ragged grids, 128 / 240 / 256 / 384-token blocks, empty rows,
text tokens, more heads than SMs) must run through it with status 0 and give, bit for bit, what the
regular build gives.  Runs in a child process: a process can load only one of the two libraries."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_CHILD = r"""
import math, pickle, sys
import torch
sys.path.insert(0, sys.argv[1])
from paper_2609_37001_b200 import build, binding as B
B.LIB_PATH = build.build(checked=(sys.argv[2] == "checked"))
INF, SCALE = 0, 1.0 / math.sqrt(128.0)
CASES = [
    ((3, 13, 19), (1, 16, 16), [(2, 0, INF, 2, 0, INF), (1, 1, INF, 1, 0, INF), (1, -1, 2, 1, 0, 3)], 0),
    ((6, 8, 16), (3, 8, 16), [(1, 0, 2, 1, 0, INF), (2, 0, INF, 1, 0, INF)], 0),
    ((5, 9, 40), (1, 4, 32), [(2, 1, 3, 2, 0, 3), (5, 0, INF, 1, 0, 1)], 0),
    ((3, 45, 32), (1, 15, 16), [(2, 0, INF, 2, 0, 3), (1, 1, 2, 6, 0, INF)], 0),
    ((2, 30, 40), (1, 12, 16), [(2, 0, 2, 2, 0, 3), (1, 0, INF, 9, 0, INF)], 0),
    ((2, 16, 16), (1, 16, 16), [((h % 2) + 1, (h % 3) - 1, INF, 1, 0, INF) for h in range(160)], 0),
    ((4, 16, 32), (1, 16, 16), [(2, 0, 3, 2, 0, 3), (1, 0, INF, 2, 1, INF)], 200),
]
res = []
for grid, tile, params, n_text in CASES:
    L = grid[0] * grid[1] * grid[2]
    g = torch.Generator(device="cuda").manual_seed(L + n_text)
    q, k, v = (torch.randn((len(params), L + n_text, 128), device="cuda", generator=g).bfloat16() for _ in range(3))
    if n_text:
        out, lse = B.psa_attn_fwd_joint(q, k, v, params, grid, tile, SCALE, n_text)
    else:
        out, lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    res.append((B.psa_last_device_status(), out.view(torch.int16).cpu(), lse.view(torch.int32).cpu()))
pickle.dump(res, open(sys.argv[3], "wb"))
"""


def test_checked_build_runs_clean_and_agrees_bit_for_bit(tmp_path):
    import pickle
    import torch
    outs = {}
    for kind in ("regular", "checked"):
        f = tmp_path / f"{kind}.pkl"
        r = subprocess.run([sys.executable, "-c", _CHILD, ROOT, kind, str(f)], capture_output=True, text=True, timeout=900)
        assert r.returncode == 0, r.stderr[-2000:]
        outs[kind] = pickle.load(open(f, "rb"))
    for i, ((st_r, o_r, l_r), (st_c, o_c, l_c)) in enumerate(zip(outs["regular"], outs["checked"])):
        assert st_r == (0, 0) and st_c == (0, 0), (i, st_r, st_c)
        assert torch.equal(o_r, o_c) and torch.equal(l_r, l_c), i
