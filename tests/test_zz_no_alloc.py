"""psa_attn_fwd_noalloc: the entry point for callers that may not allocate device memory (their memory
belongs to a framework's pool, or they cannot afford cudaMalloc's device-wide synchronisation).  Its
scratch is a fixed array inside the library, shared by all calls, so the test runs two calls in a row
(the second with another shape and other parameters).  Each is compared, through the C ABI, with
psa_attn_fwd -- bit for bit, since both drive the same kernels -- and the second also with the fp64
oracle within the tolerances of the parity tests.  A further test frees the library's cached
workspace and checks that a series of calls leaves the device's free memory untouched.
Collected last on purpose."""
import ctypes
import math

import numpy as np
import pytest
import torch

from oracle import psa_oracle as O
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
    return bits, tuple(torch.from_numpy(bits[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))


def _compare(B, params, grid, tile, seed, with_oracle=False):
    T, H, W = grid
    L, nh = T * H * W, len(params)
    bits, (q, k, v) = _inputs(seed, nh, L)
    ref_out, ref_lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    out = torch.full_like(q, float("nan"))
    lse = torch.full((nh, L), float("nan"), dtype=torch.float32, device="cuda")
    detail = B.psa_attn_fwd_noalloc(q, k, v, out, lse, params, grid, tile, SCALE)
    assert detail == 0
    assert not torch.isnan(out).any() and not torch.isnan(lse).any()
    # same kernels, same inputs, no cross-item reduction: the two entry points agree bit for bit
    assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16))
    assert torch.equal(lse.view(torch.int32), ref_lse.view(torch.int32))
    if with_oracle:
        out_h = O.bf16_bits_to_f64(out.view(torch.int16).cpu().numpy().view(np.uint16))
        lse_h = lse.cpu().numpy().astype(np.float64)
        for hd in range(nh):
            qf, kf, vf = (O.bf16_bits_to_f64(bits[n][hd]) for n in ("q", "k", "v"))
            ro, rl = O.attention(qf, kf, vf, tuple(params[hd]), T, H, W, tuple(tile), SCALE)
            err = np.abs(out_h[hd] - ro)
            assert err.max() <= OUT_MAX and err.mean() <= OUT_MEAN, (hd, err.max(), err.mean())
            fin = np.isfinite(rl)
            assert np.array_equal(np.isfinite(lse_h[hd]), fin)
            assert np.abs(lse_h[hd][fin] - rl[fin]).max() <= LSE_MAX


def test_two_calls_in_a_row_match_the_allocating_entry_point(B):
    INF = 0
    _compare(B, [(2, 0, INF, 2, 0, 3), (1, 1, 2, 1, 0, INF), (6, 0, INF, 4, 0, INF)], (6, 32, 32), (1, 16, 16), 0xA1)
    # a second call right behind it, smaller and ragged, with empty rows: stale scratch must not leak in
    _compare(B, [(1, 1, INF, 1, 0, INF), (2, -1, 3, 2, 1, INF)], (3, 13, 19), (1, 16, 16), 0xA2, with_oracle=True)


def test_calls_leave_the_free_device_memory_untouched(B):
    """With the library's cached workspace freed, a run of calls must not change what cudaMemGetInfo
    reports: the entry point exists for callers that cannot have a library allocate behind their back."""
    INF = 0
    params, grid, tile = [(2, 0, INF, 2, 0, 3), (1, 0, 2, 3, 0, INF)], (4, 16, 32), (1, 16, 16)
    L, nh = 4 * 16 * 32, 2
    _, (q, k, v) = _inputs(0xA3, nh, L)
    out = torch.empty_like(q)
    lse = torch.empty((nh, L), dtype=torch.float32, device="cuda")
    B.psa_attn_fwd_noalloc(q, k, v, out, lse, params, grid, tile, SCALE)   # first call: looks up the array's address
    B.psa_shutdown()                                                      # no cached cudaMalloc workspace is left
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    first = None
    for _ in range(5):
        assert B.psa_attn_fwd_noalloc(q, k, v, out, lse, params, grid, tile, SCALE) == 0
        free_now, _ = torch.cuda.mem_get_info()
        assert free_now == free0
        if first is None:
            first = out.clone()   # (a torch allocation of ours, after the reading above; cached by torch afterwards)
            free0, _ = torch.cuda.mem_get_info()
        else:
            assert torch.equal(out.view(torch.int16), first.view(torch.int16))


def test_problems_beyond_the_fixed_scratch_are_rejected(B):
    # 21 x 45 x 80 with 128-token blocks and 40 heads needs 40 * 630 = 25,200 work items > 16,384
    nh, grid, tile = 40, (21, 45, 80), (1, 8, 16)
    prob = B.make_problem(nh, tile, SCALE, 75600 * 128, 128)
    hp = B._params_array([(1, 0, 0, 1, 0, 0)] * nh)
    rc = B.lib().psa_attn_fwd_noalloc(256, 512, 768, 1024, 2048, hp, ctypes.byref(prob), *grid, None, None)
    assert rc == B.PSA_ERR_CAPACITY
    assert "capacity" in B.status_string(rc)
