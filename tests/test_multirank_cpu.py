"""The N > 1 path of bench.py on CPU: two gloo ranks, independent batches, max-over-ranks timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2608_03796_b200 import inputs as I


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.rank_config(I.CONFIGS["c1"], rank)
    h = I.hidden(cfg, rows=torch.arange(4))
    # every rank reports its own time; the job's time is the slowest rank's
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
    gathered = [torch.zeros_like(h) for _ in range(world)]
    dist.all_gather(gathered, h)
    distinct = not torch.equal(gathered[0], gathered[1])
    out.put((rank, ms, cfg.seed, distinct))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_independent_batches_and_max_time():
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
    assert [r[1] for r in res] == [15.0, 15.0]                 # both ranks see the max
    assert [r[2] for r in res] == [1234, 1235]                 # one seed per rank
    assert all(r[3] for r in res)                              # so the batches differ
    # whole-job throughput counts every rank's tokens over the slowest rank's time
    assert bench.whole_job_tokens_per_s(4096, 2, 15.0) == 2 * 4096 / 0.015


def test_reference_arm_runs_only_on_rank_zero(monkeypatch, capsys):
    class A:
        ref_rows, warmup, steps, gpus = 4, 0, 1, 2
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(A, I.CONFIGS["c1"])
    assert capsys.readouterr().out == ""
    monkeypatch.setenv("RANK", "0")
    bench.run_reference(A, I.CONFIGS["c1"])
    import json
    line = json.loads(capsys.readouterr().out)
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
