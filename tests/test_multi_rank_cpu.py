"""The benchmark's N > 1 path shards nothing: every rank runs an independent replica and the ranks only meet to
reduce the timing (max) and the token count (sum).  That host logic is exercised here with two gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, toks = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100 + rank, dist, "cpu")
    dist.barrier()
    out.put((rank, ms, toks, bench.replica_prompt_seed(12, rank, 3)))
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_time_by_max_and_tokens_by_sum():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]          # slowest rank's time on every rank
    assert [r[2] for r in res] == [201, 201]            # all ranks' tokens
    assert res[0][3] != res[1][3]                       # replicas decode different prompts


def test_reference_arm_exits_quietly_on_other_ranks(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        steps, warmup = 1, 0
    bench.run_reference(A())
    assert capsys.readouterr().out == ""
