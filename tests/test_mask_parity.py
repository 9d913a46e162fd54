"""psa_mask_build (CUDA, through the C ABI) against the oracle: bit-exact block mask, row_ptr and
ascending column lists on every workload, plus degenerate cases."""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as O
from paper_2609_37001_b200 import workloads as WL

pytestmark = pytest.mark.gpu
INF = O.INF_STRIDE


@pytest.fixture(scope="module")
def B():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding
    return binding


def _check(B, params, grid, tile):
    params = [tuple(p) for p in params]
    mask, row_ptr, col = B.psa_mask_build(params, grid, tile)
    torch.cuda.synchronize()
    om, orp, oc = O.block_index_lists(params, *grid, tuple(tile))
    assert np.array_equal(mask.cpu().numpy(), om)
    assert np.array_equal(row_ptr.cpu().numpy(), orp)
    assert np.array_equal(col.cpu().numpy(), oc)
    nb, nnz = B.psa_mask_sizes(params, grid, tile)
    assert nb == om.shape[1] and nnz == oc.size


@pytest.mark.parametrize("name", sorted(WL.load_workloads().keys()))
def test_workload_masks_bit_exact(B, name):
    w = WL.workload(name)
    _check(B, w["head_params"], w["grid"], w["tile"])


def test_parameter_families_and_degenerate_cases(B):
    grid, tile = (9, 20, 28), (2, 4, 8)      # ragged in every axis: T'=5, H'=5, W'=4
    fam = [
        (2, 0, INF, 3, 0, INF),    # single band per axis (SVG-like)
        (2, 0, INF, 2, 0, 5),      # single temporal band + periodic spatial (STA-like)
        (1, 1, 2, 20, 0, INF),     # temporal only
        (5, 0, INF, 1, -1, 3),     # spatial only
        (2, -2, 3, 2, 1, 6),       # all six
        (1, 1, INF, 1, 0, INF),    # leaves empty rows
        (1, 7, INF, 1, 0, INF),    # offset beyond the grid: no pair at all
        (1, 0, 1, 1, 0, 1),        # stride 1: all-pass
        (3, 0, 2, 4, 0, 3),        # width >= stride: all-pass
    ]
    _check(B, fam, grid, tile)
    _check(B, [(1, 0, INF, 1, 0, INF)], (1, 1, 1), (1, 1, 1))          # one block
    _check(B, [(2, 0, 3, 2, 0, 3)] * 3, (4, 4, 4), (1, 1, 1))          # token granularity: Algorithm 1 verbatim
    _check(B, [(3, 1, INF, 2, 0, 5)] * 130, (6, 16, 16), (2, 8, 8))    # more heads than one launch carries


def test_capacity_error_and_optional_outputs(B):
    import ctypes
    params = [(2, 0, INF, 2, 0, INF)]
    grid, tile = (4, 16, 16), (1, 8, 8)
    nb, nnz = B.psa_mask_sizes(params, grid, tile)
    prob = B.make_problem(1, tile, 1.0, 0, 128)
    rp = torch.zeros(nb + 1, dtype=torch.int32, device="cuda")
    col = torch.zeros(nnz, dtype=torch.int32, device="cuda")
    rc = B.lib().psa_mask_build(B._params_array(params), ctypes.byref(prob), *grid, None, rp.data_ptr(),
                                col.data_ptr(), nnz - 1, None)
    assert rc == B.PSA_ERR_CAPACITY
    rc = B.lib().psa_mask_build(B._params_array(params), ctypes.byref(prob), *grid, None, rp.data_ptr(), None, 0, None)
    assert rc == B.PSA_OK
    torch.cuda.synchronize()
    _, orp, _ = O.block_index_lists(params, *grid, tile)
    assert np.array_equal(rp.cpu().numpy(), orp)


@pytest.mark.parametrize("grid,tile,nh", [((4, 4, 4), (1, 1, 1), 3), ((3, 2, 2), (1, 1, 1), 5), ((5, 1, 1), (1, 1, 1), 4),
                                          ((6, 16, 24), (1, 8, 8), 2)])
def test_mask_at_any_allowed_alignment_with_guard_bytes(B, grid, tile, nh):
    """The mask is written in aligned 32-byte pieces; a base that is only 16-byte aligned (the
    contract's minimum), and rows shorter than a piece, must give the same bytes and touch nothing
    outside the array.  A base that is not 16-byte aligned is rejected."""
    import ctypes
    params = [(1 + h % 2, (h % 3) - 1, [INF, 2, 3][h % 3], 1 + (h % 3), h % 2, [INF, 3][h % 2]) for h in range(nh)]
    om, orp, oc = O.block_index_lists(params, *grid, tuple(tile))
    nb, nnz = B.psa_mask_sizes(params, grid, tile)
    prob = B.make_problem(nh, tile, 1.0, 0, 128)
    n = nh * nb * nb
    for off in (0, 16, 48, 80):
        buf = torch.full((n + 256,), 0xEE, dtype=torch.uint8, device="cuda")
        rp = torch.zeros(nh * nb + 1, dtype=torch.int32, device="cuda")
        col = torch.zeros(max(nnz, 1), dtype=torch.int32, device="cuda")
        rc = B.lib().psa_mask_build(B._params_array(params), ctypes.byref(prob), *grid, buf.data_ptr() + 64 + off,
                                    rp.data_ptr(), col.data_ptr(), col.numel(), None)
        assert rc == B.PSA_OK
        torch.cuda.synchronize()
        got = buf.cpu().numpy()
        assert np.array_equal(got[64 + off:64 + off + n].reshape(om.shape), om), off
        assert (got[:64 + off] == 0xEE).all() and (got[64 + off + n:] == 0xEE).all(), off
        assert np.array_equal(rp.cpu().numpy(), orp) and np.array_equal(col.cpu().numpy()[:nnz], oc)
    assert B.lib().psa_mask_build(B._params_array(params), ctypes.byref(prob), *grid, buf.data_ptr() + 7,
                                  rp.data_ptr(), col.data_ptr(), col.numel(), None) == B.PSA_ERR_INVALID_ARG


@pytest.mark.parametrize("grid", [(64, 4, 8), (5, 1, 7), (6, 2, 3), (9, 2, 4), (40, 1, 1), (33, 3, 5), (2, 4, 8)])
def test_extreme_block_grids_of_the_register_path(B, grid):
    """Token-granular masks that sit on the limits of the small-grid kernel: 64 temporal x 32 spatial
    coordinates, spatial extents around the threshold of its closed-form mask window (7 and 8 use it,
    6 and 1 do not), rows shorter than one 32-byte piece."""
    T, H, W = grid
    params = [(1 + h % 3, (h % 5) - 2, [INF, 2, 3, 5][h % 4], 1 + (h % 2), (h % 3) - 1, [INF, 3, 5, 6][(h // 2) % 4])
              for h in range(6)]
    params += [(T, 0, INF, H * W, 0, INF), (1, 0, INF, 1, 0, INF), (2, T, INF, 1, 0, INF)]   # all-pass, diagonal, empty
    _check(B, params, grid, (1, 1, 1))
