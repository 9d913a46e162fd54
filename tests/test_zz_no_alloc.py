"""psa_attn_fwd_noalloc: the entry point for callers that may not allocate device memory (their memory
belongs to a framework's pool, or they cannot afford cudaMalloc's device-wide synchronisation).  Its
scratch is a fixed array inside the library, shared by all calls, so the test runs two calls in a row
(the second with another shape and other parameters) and compares each with psa_attn_fwd, through the
C ABI, within the tolerances of the parity tests.  Collected last on purpose."""
import ctypes
import math

import numpy as np
import pytest
import torch

from paper_2609_37001_b200 import workloads as WL

pytestmark = pytest.mark.gpu
SCALE = 1.0 / math.sqrt(128.0)
OUT_MAX, OUT_MEAN, LSE_MAX = 2e-2, 2e-3, 1e-3


@pytest.fixture(scope="module")
def B():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding
    return binding


def _inputs(seed, nh, L):
    bits = {n: WL.tensor_bits(seed, n, nh, L) for n in ("q", "k", "v")}
    return tuple(torch.from_numpy(bits[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))


def _compare(B, params, grid, tile, seed):
    T, H, W = grid
    L, nh = T * H * W, len(params)
    q, k, v = _inputs(seed, nh, L)
    ref_out, ref_lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    out = torch.full_like(q, float("nan"))
    lse = torch.full((nh, L), float("nan"), dtype=torch.float32, device="cuda")
    detail = B.psa_attn_fwd_noalloc(q, k, v, out, lse, params, grid, tile, SCALE)
    assert detail == 0
    assert not torch.isnan(out).any() and not torch.isnan(lse).any()
    err = (out.float() - ref_out.float()).abs()
    assert err.max().item() <= OUT_MAX and err.mean().item() <= OUT_MEAN
    fin = torch.isfinite(ref_lse)
    assert torch.equal(torch.isfinite(lse), fin)
    assert (lse[fin] - ref_lse[fin]).abs().max().item() <= LSE_MAX


def test_two_calls_in_a_row_match_the_allocating_entry_point(B):
    INF = 0
    _compare(B, [(2, 0, INF, 2, 0, 3), (1, 1, 2, 1, 0, INF), (6, 0, INF, 4, 0, INF)], (6, 32, 32), (1, 16, 16), 0xA1)
    # a second call right behind it, smaller and ragged, with empty rows: stale scratch must not leak in
    _compare(B, [(1, 1, INF, 1, 0, INF), (2, -1, 3, 2, 1, INF)], (3, 13, 19), (1, 16, 16), 0xA2)


def test_problems_beyond_the_fixed_scratch_are_rejected(B):
    # 21 x 45 x 80 with 128-token blocks and 40 heads needs 40 * 630 = 25,200 work items > 16,384
    nh, grid, tile = 40, (21, 45, 80), (1, 8, 16)
    prob = B.make_problem(nh, tile, SCALE, 75600 * 128, 128)
    hp = B._params_array([(1, 0, 0, 1, 0, 0)] * nh)
    rc = B.lib().psa_attn_fwd_noalloc(256, 512, 768, 1024, 2048, hp, ctypes.byref(prob), *grid, None, None)
    assert rc == B.PSA_ERR_CAPACITY
    assert "capacity" in B.status_string(rc)
