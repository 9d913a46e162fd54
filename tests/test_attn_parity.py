"""psa_attn_fwd (CUDA, through the C ABI) against the fp64 oracle on the same seeded bf16 inputs.

Tolerances (bf16 inputs, fp32 accumulation, bf16 probabilities): out max-abs <= 2e-2,
mean-abs <= 2e-3, lse max-abs <= 1e-3, plus a relative L2 bound of 1e-2 on the output.
The output is rounded to bf16 (relative precision 2^-9), so where an output element exceeds 1 in
magnitude -- only the sharply peaked test inputs produce such rows -- its error is measured
relative to that magnitude; with i.i.d. N(0,1) inputs every |out| is below 1 and the absolute
tolerances apply unchanged.
Small workloads are compared on every row; the full-size workloads on seeded sampled rows
(whole query slabs at grid corners plus random rows), each against all keys."""
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


_BITS_CACHE = {}


def _tensor_bits(seed, nh, L, gain):
    """q/k/v bit patterns; the last request is kept so workloads sharing seed and shape reuse it."""
    key = (seed, nh, L, gain)
    if key not in _BITS_CACHE:
        _BITS_CACHE.clear()
        _BITS_CACHE[key] = {n: WL.tensor_bits(seed, n, nh, L, gain=(gain if n != "v" else 1.0)) for n in ("q", "k", "v")}
    return _BITS_CACHE[key]


def _to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _bf16_to_f64(t):
    return O.bf16_bits_to_f64(t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))


def _compare(out_rows, lse_rows, ref_out, ref_lse, what):
    empty = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(lse_rows), empty), what
    assert np.all(out_rows[empty] == 0), what
    err = np.abs(out_rows - ref_out) / np.maximum(1.0, np.abs(ref_out))
    assert err.max() <= OUT_MAX, (what, err.max())
    assert err.mean() <= OUT_MEAN, (what, err.mean())
    ok = ~empty
    if ok.any():
        assert np.abs(lse_rows[ok] - ref_lse[ok]).max() <= LSE_MAX, (what, np.abs(lse_rows[ok] - ref_lse[ok]).max())
        rel = np.linalg.norm(out_rows[ok] - ref_out[ok]) / max(np.linalg.norm(ref_out[ok]), 1e-30)
        assert rel <= REL_L2, (what, rel)


def _run_and_check(B, params, grid, tile, seed, rows_per_head=None, gain=1.0, heads_to_check=None):
    params = [tuple(p) for p in params]
    T, H, W = grid
    L, nh = T * H * W, len(params)
    bits = _tensor_bits(seed, nh, L, gain)
    q, k, v = (_to_dev(bits[n]) for n in ("q", "k", "v"))
    out, lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    st, detail = B.psa_last_device_status()
    assert st == 0, (st, hex(detail))
    out_h = _bf16_to_f64(out)
    lse_h = lse.cpu().numpy().astype(np.float64)
    assert not np.isnan(out_h).any()
    for hd in (heads_to_check if heads_to_check is not None else range(nh)):
        rows = list(range(L)) if rows_per_head is None else rows_per_head(hd)
        qf, kf, vf = (O.bf16_bits_to_f64(bits[n][hd]) for n in ("q", "k", "v"))
        ro, rl = O.attention_rows(qf, kf, vf, rows, params[hd], T, H, W, tuple(tile), SCALE)
        _compare(out_h[hd][rows], lse_h[hd][rows], ro, rl, f"head {hd} params {params[hd]}")
    return out, lse


@pytest.mark.parametrize("name", ["tiny", "tiny_b256"])
def test_tiny_every_row(B, name):
    w = WL.workload(name)
    out, lse = _run_and_check(B, w["head_params"], w["grid"], w["tile"], w["seed"])
    # head 1 has an all-covering period: it must equal dense attention
    L = out.shape[1]
    bits = {n: WL.head_bits(w["seed"], n, 1, L) for n in ("q", "k", "v")}
    do, dl = O.dense_attention(*(O.bf16_bits_to_f64(bits[n]) for n in ("q", "k", "v")), SCALE)
    _compare(_bf16_to_f64(out[1]), lse[1].cpu().numpy().astype(np.float64), do, dl, "dense head")


@pytest.mark.parametrize("grid,tile,params", [
    ((1, 8, 16), (1, 8, 16), [(1, 0, INF, 1, 0, INF)]),                        # one slab, one key slab
    ((3, 13, 19), (1, 16, 16), [(2, 0, INF, 2, 0, INF), (1, 1, INF, 1, 0, INF),  # ragged; empty rows
                                (1, -1, 2, 1, 0, 3)]),
    ((6, 8, 16), (3, 8, 16), [(1, 0, 2, 1, 0, INF), (2, 0, INF, 1, 0, INF)]),     # 384-token blocks
    ((5, 9, 40), (1, 4, 32), [(2, 1, 3, 2, 0, 3), (5, 0, INF, 1, 0, 1)]),         # 128-token blocks, ragged h, w
    ((2, 30, 10), (2, 32, 4), [(1, 0, INF, 2, -1, INF), (1, 0, 1, 1, 1, 2)]),     # slab stacks along t
    ((1, 4, 100), (1, 1, 256), [(1, 0, INF, 1, 0, INF)]),                         # slab stacks along w
    ((3, 45, 32), (1, 15, 16), [(2, 0, INF, 2, 0, 3), (1, 1, 2, 6, 0, INF)]),      # 240-token blocks: 128 + 112 slabs
    ((2, 30, 40), (1, 12, 16), [(2, 0, 2, 2, 0, 3), (1, 0, INF, 9, 0, INF)]),      # 192 = 128 + 64, ragged h and w
    ((2, 28, 16), (1, 14, 16), [(1, 0, INF, 1, 1, INF)]),                          # 224 = 128 + 96
    ((4, 16, 16), (1, 16, 16), [(1, 7, INF, 1, 0, INF)]),                         # offset beyond the grid: all rows empty
])
def test_small_shapes_every_row(B, grid, tile, params):
    _run_and_check(B, params, grid, tile, seed=0x77)


def test_peaked_inputs_every_row(B):
    """q, k scaled so the softmax is concentrated: a wrongly skipped or included tile moves the output by O(1)."""
    _run_and_check(B, [(2, 0, 3, 2, 0, 3), (1, -1, INF, 3, 0, INF)], (8, 16, 32), (1, 16, 16), seed=0x78, gain=2.0)


@pytest.mark.parametrize("grid,tile", [((4, 45, 32), (1, 15, 16)), ((6, 16, 32), (3, 8, 16))])
def test_sharply_peaked_inputs_every_row(B, grid, tile):
    """q and k scaled by 4: the softmax of a row is dominated by a handful of keys, so a missing or
    extra tile, or a rescale applied to the wrong accumulator, shows as an O(1) error.  Blocks of
    128 + 112 tokens and of three 128-token slabs (two-slab and single-slab work items)."""
    _run_and_check(B, [(2, 0, 3, 2, 0, 3), (1, -1, INF, 3, 0, INF), (2, 1, INF, 1, 0, 2)], grid, tile, seed=0x7C, gain=4.0)


def test_strided_token_major_layout(B):
    """[L, heads, 128] storage: stride_token = heads*128, stride_head = 128."""
    grid, tile, nh = (4, 16, 16), (1, 16, 16), 3
    params = [(2, 0, INF, 1, 0, INF), (1, 1, 2, 1, 0, INF), (4, 0, INF, 1, 0, INF)]
    L = 4 * 16 * 16
    bits = {n: WL.tensor_bits(0x79, n, nh, L) for n in ("q", "k", "v")}
    dev = {n: _to_dev(np.ascontiguousarray(bits[n].transpose(1, 0, 2))).permute(1, 0, 2) for n in bits}
    out, lse = B.psa_attn_fwd(dev["q"], dev["k"], dev["v"], params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    assert out.stride() == dev["q"].stride()
    for hd in range(nh):
        qf, kf, vf = (O.bf16_bits_to_f64(bits[n][hd]) for n in ("q", "k", "v"))
        ro, rl = O.attention(qf, kf, vf, params[hd], *grid, tile, SCALE)
        _compare(_bf16_to_f64(out[hd]), lse[hd].cpu().numpy().astype(np.float64), ro, rl, f"head {hd}")


def _sampled_rows(grid, tile, seed):
    T, H, W = grid
    L = T * H * W

    def rows(hd):
        r = set(WL.sample_rows(seed, hd, L, 48))
        # whole bricks at the corners of the grid (edge slabs included)
        bt, bh, bw = tile
        for (t0, h0, w0) in ((0, 0, 0), (T - 1, H - 1, W - 1), (T // 2, H - 1, 0)):
            tb, hb, wb = t0 // bt, h0 // bh, w0 // bw
            if hd % 3 == (t0 + h0) % 3:
                for t in range(tb * bt, min(T, (tb + 1) * bt)):
                    for h in range(hb * bh, min(H, (hb + 1) * bh)):
                        for w in range(wb * bw, min(W, (wb + 1) * bw)):
                            r.add((t * H + h) * W + w)
        return sorted(r)
    return rows


@pytest.mark.parametrize("name,heads", [
    ("wan13b_480p", None),
    ("wan13b_480p_b3x32x4", [0, 4, 7, 11]),
    ("wan13b_480p_b1x30x8", [1, 5, 8, 10]),
    ("wan13b_480p_b1x32x4", [2, 6, 9]),
    ("wan14b_720p", list(range(0, 40, 5))),
    ("wan14b_720p_b1x16x16", [2, 17, 31]),
    ("wan14b_720p_b3x8x16", [0, 13, 26]),
    ("hunyuan_720p", [1, 8, 15, 22]),
    ("hunyuan_768p", [0, 11]),
    ("hunyuan_768p_b6x8x8", [5, 23]),
    ("sweep_00", [0]), ("sweep_25", [3]), ("sweep_50", [5]), ("sweep_75", [7]), ("sweep_90", [39]),
    ("ragged_75", [0, 39]), ("ragged_dense", [20]),
])
def test_full_size_workloads_sampled_rows(B, name, heads):
    w = WL.workload(name)
    _run_and_check(B, w["head_params"], w["grid"], w["tile"], w["seed"],
                   rows_per_head=_sampled_rows(w["grid"], w["tile"], w["seed"]), heads_to_check=heads)


@pytest.mark.parametrize("pinned", [True, False])
def test_host_tensor_entry_point_matches_device_call(B, pinned):
    """psa_attn_fwd_host (copies in, pipelined over head chunks, copies out) gives the device call's bits,
    with more heads than chunks and with fewer heads than chunks, from pinned and from pageable memory."""
    for nh, grid, tile in ((11, (4, 16, 16), (1, 16, 16)), (3, (3, 15, 32), (1, 15, 16))):
        T, H, W = grid
        L = T * H * W
        params = [(1 + (h % 3), (h % 3) - 1, [INF, 2, 3][h % 3], 1 + (h % 2), 0, [INF, 3][h % 2]) for h in range(nh)]
        bits = {n: WL.tensor_bits(0x7A + nh, n, nh, L, threads=1) for n in ("q", "k", "v")}
        host = {n: torch.from_numpy(bits[n].view(np.int16)).view(torch.bfloat16) for n in bits}
        dev = {n: host[n].cuda() for n in host}
        ref_out, ref_lse = B.psa_attn_fwd(dev["q"], dev["k"], dev["v"], params, grid, tile, SCALE)
        assert B.psa_last_device_status()[0] == 0
        hq, hk, hv = (host[n].pin_memory() if pinned else host[n].clone() for n in ("q", "k", "v"))
        hout = torch.full_like(hq, float("nan"))
        hlse = torch.full((nh, L), float("nan"), dtype=torch.float32)
        if pinned:
            hout, hlse = hout.pin_memory(), hlse.pin_memory()
        staging = tuple(torch.empty_like(dev["q"]) for _ in range(4)) + (torch.empty((nh, L), dtype=torch.float32, device="cuda"),)
        B.psa_attn_fwd_host(hq, hk, hv, hout, hlse, staging, params, grid, tile, SCALE)
        assert torch.equal(hout.view(torch.int16), ref_out.cpu().view(torch.int16))
        assert torch.equal(hlse.view(torch.int32), ref_lse.cpu().view(torch.int32))


def test_host_tensor_call_with_reordered_chunks(B):
    """40 heads of very different weight: the host call pipelines 2-head chunks, opens with single
    heads and keeps the two lightest heads for the end (here heads 17 and 5, in the middle of runs);
    the result must be the device call's, bit for bit."""
    grid, tile, nh = (4, 16, 16), (1, 16, 16), 40
    L = 4 * 16 * 16
    params = [(1 + (h % 4), (h % 3) - 1, INF, 1, 0, INF) for h in range(nh)]
    params[17] = (1, 3, INF, 1, 0, INF)     # one attended block pair per row at most: the lightest
    params[5] = (1, 2, INF, 1, 0, INF)      # the second lightest
    bits = {n: WL.tensor_bits(0x7D, n, nh, L, threads=1) for n in ("q", "k", "v")}
    host = {n: torch.from_numpy(bits[n].view(np.int16)).view(torch.bfloat16) for n in bits}
    dev = {n: host[n].cuda() for n in host}
    ref_out, ref_lse = B.psa_attn_fwd(dev["q"], dev["k"], dev["v"], params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    hq, hk, hv = (host[n].pin_memory() for n in ("q", "k", "v"))
    hout = torch.full_like(hq, float("nan")).pin_memory()
    hlse = torch.full((nh, L), float("nan"), dtype=torch.float32).pin_memory()
    staging = tuple(torch.empty_like(dev["q"]) for _ in range(4)) + (torch.empty((nh, L), dtype=torch.float32, device="cuda"),)
    B.psa_attn_fwd_host(hq, hk, hv, hout, hlse, staging, params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    assert torch.equal(hout.view(torch.int16), ref_out.cpu().view(torch.int16))
    assert torch.equal(hlse.view(torch.int32), ref_lse.cpu().view(torch.int32))


def test_more_heads_than_one_launch_carries(B):
    """130 heads: the library splits the call into launches of at most 128 heads."""
    grid, tile, nh = (2, 16, 16), (1, 16, 16), 130
    L = 2 * 16 * 16
    params = [((h % 2) + 1, (h % 3) - 1, INF, 1, 0, INF) for h in range(nh)]
    bits = {n: WL.tensor_bits(0x7B, n, nh, L) for n in ("q", "k", "v")}
    q, k, v = (_to_dev(bits[n]) for n in ("q", "k", "v"))
    out, lse = B.psa_attn_fwd(q, k, v, params, grid, tile, SCALE)
    assert B.psa_last_device_status()[0] == 0
    for hd in (0, 1, 63, 127, 128, 129):
        qf, kf, vf = (O.bf16_bits_to_f64(bits[n][hd]) for n in ("q", "k", "v"))
        ro, rl = O.attention(qf, kf, vf, params[hd], *grid, tile, SCALE)
        _compare(_bf16_to_f64(out[hd]), lse[hd].cpu().numpy().astype(np.float64), ro, rl, f"head {hd}")


@pytest.mark.parametrize("even_spacing", [True, False])
def test_batched_call_matches_oracle_per_sample(B, even_spacing):
    """psa_attn_fwd_batched: a conditional / unconditional pair with shared per-head masks, once with the
    samples laid out as evenly spaced heads (one launch sequence) and once with a padded batch stride
    (sample by sample)."""
    grid, tile = (4, 12, 16), (1, 8, 16)
    T, H, W = grid
    L, nb, nh = T * H * W, 2, 3
    params = [(2, 0, INF, 2, 0, INF), (1, 1, 2, 3, 0, INF), (4, 0, INF, 1, 0, 2)]
    bits = {n: WL.tensor_bits(77, n, nb * nh, L) for n in ("q", "k", "v")}

    def dev(n):
        full = _to_dev(bits[n]).view(nb, nh, L, 128)
        if even_spacing:
            return full
        buf = torch.zeros((nb, nh + 1, L, 128), dtype=torch.bfloat16, device="cuda")
        buf[:, :nh] = full
        return buf[:, :nh]

    q, k, v = dev("q"), dev("k"), dev("v")
    out, lse = B.psa_attn_fwd_batched(q, k, v, params, grid, tile, SCALE)
    st, detail = B.psa_last_device_status()
    assert st == 0, (st, hex(detail))
    out_h = _bf16_to_f64(out).reshape(nb, nh, L, 128)
    lse_h = lse.cpu().numpy().astype(np.float64)
    for b in range(nb):
        for hd in range(nh):
            qf, kf, vf = (O.bf16_bits_to_f64(bits[n][b * nh + hd]) for n in ("q", "k", "v"))
            ro, rl = O.attention(qf, kf, vf, params[hd], T, H, W, tuple(tile), SCALE)
            _compare(out_h[b, hd], lse_h[b, hd], ro, rl, f"sample {b} head {hd}")
