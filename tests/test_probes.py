"""Structure probes and robustness of the CUDA path (GPU).

With q = 0 every score is 0, so lse = ln(number of attended REAL keys) and out = mean of the attended
values: closed forms that expose any wrongly skipped or included tile and any unmasked padded key,
which i.i.d. random data at large L does not.  The expected counts come from the oracle's block
lists and real-token counts."""
import math

import numpy as np
import pytest
import torch

from oracle import psa_oracle as O
from paper_2609_37001_b200 import workloads as WL

pytestmark = pytest.mark.gpu
INF = O.INF_STRIDE
SCALE = 1.0 / math.sqrt(128.0)


@pytest.fixture(scope="module")
def B():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding
    return binding


def _expected_counts(params, grid, tile):
    T, H, W = grid
    real = O.block_real_tokens(T, H, W, tile)
    _, _, blk = O.token_block_coords(T, H, W, tile)
    return [(O.block_mask(p, T, H, W, tile).astype(np.int64) @ real)[blk] for p in params], blk, real


@pytest.mark.parametrize("grid,tile,params", [
    ((5, 13, 19), (1, 16, 16), [(2, 0, INF, 2, 0, INF), (1, 1, 2, 1, -1, 3), (1, 2, INF, 1, 0, INF)]),
    ((6, 20, 40), (3, 8, 16), [(1, 0, 2, 2, 1, 3), (2, -1, INF, 1, 0, 5)]),
    ((21, 45, 79), (1, 16, 16), [(9, 0, INF, 2, 0, 6), (1, -2, 2, 1, 0, 5)]),
    # the headline block at both 720p shapes: 128 + 112-token slabs on an unpadded 45-row grid
    ((21, 45, 80), (1, 15, 16), [(5, 0, INF, 2, 0, 6), (2, 1, 3, 1, -1, 5)]),
    ((33, 45, 80), (1, 15, 16), [(7, -1, INF, 3, 0, 6), (1, 0, 2, 2, 1, INF)]),
])
def test_zero_query_counts_and_block_code_values(B, grid, tile, params):
    T, H, W = grid
    L, nh = T * H * W, len(params)
    counts, blk, real = _expected_counts(params, grid, tile)
    q = torch.zeros((nh, L, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.from_numpy(WL.tensor_bits(0x91, "k", nh, L).view(np.int16)).cuda().view(torch.bfloat16)
    # block-code values: channel c of key j is 1 iff block(j) mod 128 == c
    code = torch.zeros((L, 128), dtype=torch.bfloat16)
    code[torch.arange(L), torch.from_numpy(blk % 128)] = 1.0
    v = code.cuda()[None].repeat(nh, 1, 1).contiguous()
    out, lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    lse = lse.cpu().numpy().astype(np.float64)
    out = out.float().cpu().numpy().astype(np.float64)
    for hd in range(nh):
        n = counts[hd].astype(np.float64)
        empty = n == 0
        assert np.array_equal(np.isneginf(lse[hd]), empty)
        assert np.all(out[hd][empty] == 0)
        ok = ~empty
        assert np.abs(lse[hd][ok] - np.log(n[ok])).max() <= 1e-3
        # out[i, c] * n_i = real tokens of the attended blocks whose id is c mod 128
        bm = O.block_mask(params[hd], T, H, W, tile).astype(np.int64)
        per_class = np.zeros((bm.shape[0], 128))
        for kb in range(bm.shape[0]):
            per_class[:, kb % 128] += bm[:, kb] * real[kb]
        want = per_class[blk][ok] / n[ok][:, None]
        got = out[hd][ok]
        assert np.abs(got - want).max() <= 4e-3      # bf16 rounding of the probabilities and of the output
        assert np.all((want == 0) == (got == 0))     # exactly the attended block classes are present


def test_every_real_row_written_once_and_nothing_else(B):
    """Outputs are pre-filled with sentinels inside guard bands: every real row must be overwritten,
    the guards must stay intact, and two runs must agree bit for bit."""
    grid, tile = (5, 13, 19), (1, 16, 16)
    params = [(2, 0, INF, 2, 0, INF), (1, 1, INF, 1, 0, INF)]
    T, H, W = grid
    L, nh, G = T * H * W, len(params), 4096
    bits = {n: WL.tensor_bits(0x92, n, nh, L) for n in ("q", "k", "v")}
    q, k, v = (torch.from_numpy(bits[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))
    results = []
    for _ in range(2):
        obuf = torch.full((G + nh * L * 128 + G,), float("nan"), dtype=torch.bfloat16, device="cuda")
        lbuf = torch.full((G + nh * L + G,), float("nan"), dtype=torch.float32, device="cuda")
        out = obuf[G:G + nh * L * 128].view(nh, L, 128)
        lse = lbuf[G:G + nh * L].view(nh, L)
        B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE, out=out, lse=lse)
        assert B.psa_last_device_status()[0] == 0
        assert torch.isnan(obuf[:G]).all() and torch.isnan(obuf[-G:]).all()
        assert torch.isnan(lbuf[:G]).all() and torch.isnan(lbuf[-G:]).all()
        assert not torch.isnan(out).any() and not torch.isnan(lse).any()
        results.append((out.clone(), lse.clone()))
    assert torch.equal(results[0][0].view(torch.int16), results[1][0].view(torch.int16))
    assert torch.equal(results[0][1].view(torch.int32), results[1][1].view(torch.int32))


def test_bounded_wait_expires_without_hanging(B):
    """A wait on a barrier nothing arrives on gives up after its limit, reports PSA_ERR_TIMEOUT through
    the status word, and leaves the context usable."""
    B.psa_selftest_wait_timeout(20)
    st, detail = B.psa_last_device_status()
    assert st == B.PSA_ERR_TIMEOUT and detail == 0x7E57
    params = [(1, 0, INF, 1, 0, INF)]
    grid, tile = (1, 8, 16), (1, 8, 16)
    bits = {n: WL.tensor_bits(0x93, n, 1, 128) for n in ("q", "k", "v")}
    q, k, v = (torch.from_numpy(bits[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))
    out, lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    assert B.psa_last_device_status() == (0, 0)
    ro, rl = O.dense_attention(*(O.bf16_bits_to_f64(bits[n][0]) for n in ("q", "k", "v")), SCALE)
    assert np.abs(out[0].float().cpu().numpy() - ro).max() <= 2e-2
    assert np.abs(lse[0].cpu().numpy() - rl).max() <= 1e-3


def test_device_errors_are_codes_not_faults(B):
    q = torch.zeros((1, 256, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.PsaError) as e:
        B.psa_attn_fwd(q, q.clone(), q.clone(), [(1, 0, 0, 1, 0, 0)], (1, 16, 16), (1, 10, 10), SCALE)
    assert e.value.status == B.PSA_ERR_UNSUPPORTED
    with pytest.raises(B.PsaError) as e:
        B.psa_attn_fwd(q, q.clone(), q.clone(), [(0, 0, 0, 1, 0, 0)], (1, 16, 16), (1, 16, 16), SCALE)
    assert e.value.status == B.PSA_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        B.psa_attn_fwd(q.cpu(), q.cpu(), q.cpu(), [(1, 0, 0, 1, 0, 0)], (1, 16, 16), (1, 16, 16), SCALE)


@pytest.mark.parametrize("tile", [(1, 16, 16), (1, 8, 16), (3, 8, 16), (1, 15, 16)])
def test_scores_growing_along_the_keys_force_rescales(B, tile):
    """Keys are scaled so that every later key slab raises each row's maximum by far more than the lazy
    rescale threshold: the running reference maximum moves, and the output accumulator is rescaled, at
    (almost) every slab.  A decreasing variant checks the opposite extreme (never after the first slab)."""
    grid = (6, 16 if tile[1] != 15 else 15, 16)
    T, H, W = grid
    L, nh = T * H * W, 2
    rng = np.random.default_rng(0x94)
    base = rng.standard_normal((L, 128)).astype(np.float32)
    ramp = np.linspace(0.2, 6.0, L, dtype=np.float32)[:, None]
    q = WL.f32_to_bf16_bits(rng.standard_normal((nh, L, 128)).astype(np.float32))
    v = WL.f32_to_bf16_bits(rng.standard_normal((nh, L, 128)).astype(np.float32))
    k = WL.f32_to_bf16_bits(np.stack([base * ramp, base * ramp[::-1]]))
    dev = [torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16) for x in (q, k, v)]
    Tp, Hp, Wp = O.block_grid(T, H, W, tile)
    params = [(Tp, 0, INF, Hp * Wp, 0, INF), (Tp, 0, INF, Hp * Wp, 0, INF)]
    out, lse = B.psa_attn_fwd(*dev, params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    out_h = O.bf16_bits_to_f64(out.view(torch.int16).cpu().numpy().view(np.uint16))
    lse_h = lse.cpu().numpy().astype(np.float64)
    for hd in range(nh):
        ro, rl = O.dense_attention(*(O.bf16_bits_to_f64(x[hd]) for x in (q, k, v)), SCALE)
        err = np.abs(out_h[hd] - ro)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (hd, err.max(), err.mean())
        assert np.abs(lse_h[hd] - rl).max() <= 1e-3, (hd, np.abs(lse_h[hd] - rl).max(), np.abs(rl).max())


def test_forward_call_replays_from_a_cuda_graph(B):
    """After a first call (which sizes the cached workspace) psa_mask_build + psa_attn_fwd allocate nothing
    and synchronise nothing, so a step can be captured in a CUDA graph and replayed: the replay must see
    new contents of the same buffers and give, bit for bit, what direct calls give."""
    grid, tile = (4, 30, 32), (1, 15, 16)
    params = [(2, 0, INF, 2, 0, 3), (1, 1, 2, 3, 0, INF), (4, 0, INF, 1, -1, INF)]
    T, H, W = grid
    L, nh = T * H * W, len(params)
    bits = [{n: WL.tensor_bits(0x95 + i, n, nh, L) for n in ("q", "k", "v")} for i in range(2)]
    dev = [{n: torch.from_numpy(b[n].view(np.int16)).cuda().view(torch.bfloat16) for n in b} for b in bits]
    direct = [B.psa_attn_fwd(d["q"], d["k"], d["v"], params, grid, tile, SCALE) for d in dev]
    assert B.psa_last_device_status()[0] == 0
    q, k, v = (torch.empty_like(dev[0][n]) for n in ("q", "k", "v"))
    out, lse = torch.empty_like(q), torch.empty((nh, L), dtype=torch.float32, device="cuda")
    nb, nnz = B.psa_mask_sizes(params, grid, tile)
    mask_out = (torch.empty((nh, nb, nb), dtype=torch.uint8, device="cuda"),
                torch.empty(nh * nb + 1, dtype=torch.int32, device="cuda"),
                torch.empty(max(nnz, 1), dtype=torch.int32, device="cuda"))
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE, out=out, lse=lse, stream=stream)   # warm-up on this stream
        torch.cuda.synchronize()
        graph.capture_begin()
        B.psa_mask_build(params, grid, tile, out=mask_out, stream=stream)
        B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE, out=out, lse=lse, stream=stream)
        graph.capture_end()
    ref_mask = B.psa_mask_build(params, grid, tile)
    for i in (0, 1, 0):
        for n, t in (("q", q), ("k", k), ("v", v)):
            t.copy_(dev[i][n])
        out.fill_(float("nan"))
        mask_out[0].fill_(255)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), direct[i][0].view(torch.int16))
        assert torch.equal(lse.view(torch.int32), direct[i][1].view(torch.int32))
        assert all(torch.equal(a, b) for a, b in zip(mask_out, ref_mask))
    assert B.psa_last_device_status()[0] == 0
