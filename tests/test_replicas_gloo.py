"""The N > 1 path on CPU: two gloo ranks at 127.0.0.1 exercise the timing reduction that bench.py uses
(max over ranks, whole-job throughput) and the head-sharding helper."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37001_b200 import replicas as R


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = 10.0 + 5.0 * rank          # rank 1 is the slow replica
        thr, ms = R.aggregate_throughput(1000.0, ms_local)
        lo, hi = R.shard_heads(40, rank, world)
        out.put((rank, thr, ms, lo, hi))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_reduction_and_sharding():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, thr, ms, lo, hi in res:
        assert ms == 15.0                                    # the slowest replica sets the time
        assert abs(thr - 2 * 1000.0 / 15e-3) < 1e-6          # whole-job units / that time
    assert [(r[3], r[4]) for r in res] == [(0, 20), (20, 40)]


def test_single_process_identity_and_uneven_shards():
    assert R.max_over_ranks(3.5) == 3.5
    thr, ms = R.aggregate_throughput(10.0, 2.0)
    assert ms == 2.0 and thr == 10.0 / 2e-3
    cuts = [R.shard_heads(24, r, 5) for r in range(5)]
    assert cuts[0][0] == 0 and cuts[-1][1] == 24
    assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
    assert sorted(hi - lo for lo, hi in cuts) == [4, 5, 5, 5, 5]


_RANK_SCRIPT = r"""
import os, sys
import torch, torch.distributed as dist
dist.init_process_group("gloo")          # env:// rendezvous: everything comes from the launcher's environment
t = torch.tensor([float(dist.get_rank() + 1)])
dist.all_reduce(t)
ok = (t.item() == sum(range(1, dist.get_world_size() + 1)) and os.environ["LOCAL_RANK"] == os.environ["RANK"]
      and os.environ["MASTER_ADDR"] == "127.0.0.1")
if dist.get_rank() == 0:
    print("RESULT", dist.get_world_size(), int(ok), flush=True)
dist.destroy_process_group()
sys.exit(0 if ok else 3)
"""


def test_launcher_builds_rank_environments_and_starts_the_ranks(tmp_path, capfd):
    """bench.py --gpus N without a launcher starts its own ranks through replicas.launch_ranks: every rank
    must find a complete env:// rendezvous (checked with two gloo ranks), and a failing rank must surface."""
    env = R.rank_env(1, 4, 29555, base={"PATH": "/bin"})
    assert env["RANK"] == "1" and env["LOCAL_RANK"] == "1" and env["WORLD_SIZE"] == "4"
    assert env["MASTER_ADDR"] == "127.0.0.1" and env["MASTER_PORT"] == "29555" and env["PATH"] == "/bin"
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT)
    codes = R.launch_ranks([str(script)], 2, timeout=300)
    assert codes == [0, 0]
    assert "RESULT 2 1" in capfd.readouterr().out          # rank 0's stdout is inherited, the others' is dropped
    bad = tmp_path / "bad.py"
    bad.write_text("import os, sys\nsys.exit(5 if os.environ['RANK'] == '1' else 0)\n")
    assert R.launch_ranks([str(bad)], 2, timeout=60) == [0, 5]
