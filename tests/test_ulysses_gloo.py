"""Head-sharded attention on sequence-sharded inputs (two gloo ranks on CPU): the two all-to-all
re-layouts are inverse permutations, every rank ends up with the right heads in global token order, and
the wrapper's result equals the unsharded oracle.  The attention itself is the fp64 oracle here (the
product kernel needs a GPU); what is under test is the exchange logic."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import psa_oracle as O
from paper_2609_37001_b200 import ulysses as U

GRID, TILE, D, NH = (2, 4, 8), (1, 2, 4), 16, 4
PARAMS = [(1, 0, 0, 2, 0, 0), (2, 0, 0, 1, 1, 0), (1, 1, 0, 4, 0, 0), (2, 0, 0, 1, 0, 2)]
SCALE = 0.3


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _oracle_attn(q, k, v, params, grid, tile, scale):
    outs, lses = [], []
    for h, p in enumerate(params):
        o, l = O.attention(q[h].numpy(), k[h].numpy(), v[h].numpy(), tuple(p), *grid, tuple(tile), scale)
        outs.append(torch.from_numpy(o))
        lses.append(torch.from_numpy(l))
    return torch.stack(outs), torch.stack(lses)


def _full_inputs():
    L = GRID[0] * GRID[1] * GRID[2]
    g = torch.Generator().manual_seed(5)
    return tuple(torch.randn((NH, L, D), generator=g, dtype=torch.float64) for _ in range(3))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        q, k, v = _full_inputs()
        L = q.shape[1]
        lc = L // world
        sl = slice(rank * lc, (rank + 1) * lc)
        ql, kl, vl = (t[:, sl].contiguous() for t in (q, k, v))
        # re-layout: my heads, all tokens, global order; and back
        qh = U.seq_to_head_shards(ql)
        lo, hi = U.local_heads(NH)
        relayout_ok = torch.equal(qh, q[lo:hi]) and torch.equal(U.head_to_seq_shards(qh), ql)
        o, lse = U.psa_attn_fwd_ulysses(ql, kl, vl, PARAMS, GRID, TILE, SCALE, attn_fn=_oracle_attn)
        ro, rl = _oracle_attn(q, k, v, PARAMS, GRID, TILE, SCALE)
        out.put((rank, relayout_ok, (lo, hi), float((o - ro[:, sl]).abs().max()),
                 bool(torch.equal(torch.isinf(lse), torch.isinf(rl[:, sl]))),
                 float(torch.nan_to_num(lse - rl[:, sl], nan=0.0, posinf=0.0, neginf=0.0).abs().max()),
                 tuple(o.shape), tuple(lse.shape)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_match_the_unsharded_oracle():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    L = GRID[0] * GRID[1] * GRID[2]
    for rank, relayout_ok, heads, err_o, inf_ok, err_l, so, sl in res:
        assert relayout_ok
        assert heads == (rank * NH // 2, (rank + 1) * NH // 2)
        assert so == (NH, L // 2, D) and sl == (NH, L // 2)
        assert err_o < 1e-12 and inf_ok and err_l < 1e-12


def test_single_process_is_the_plain_call():
    q, k, v = _full_inputs()
    assert U.seq_to_head_shards(q) is q and U.head_to_seq_shards(q) is q
    o, lse = U.psa_attn_fwd_ulysses(q, k, v, PARAMS, GRID, TILE, SCALE, attn_fn=_oracle_attn)
    ro, rl = _oracle_attn(q, k, v, PARAMS, GRID, TILE, SCALE)
    assert torch.equal(o, ro) and torch.equal(lse, rl)


import pytest


@pytest.mark.gpu
def test_single_gpu_wrapper_calls_the_kernel():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding as B
    grid, tile = (4, 12, 16), (1, 8, 16)
    L = 4 * 12 * 16
    g = torch.Generator(device="cuda").manual_seed(3)
    q, k, v = (torch.randn((2, L, 128), device="cuda", generator=g).bfloat16() for _ in range(3))
    params = [(2, 0, 0, 2, 0, 0), (1, 1, 2, 3, 0, 0)]
    o1, l1 = U.psa_attn_fwd_ulysses(q, k, v, params, grid, tile, 0.088)
    o2, l2 = B.psa_attn_fwd(q, k, v, params, grid, tile, 0.088)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)
